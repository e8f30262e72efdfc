// Tree-masked factorised verification on the 5th-generation tensor cores (tcgen05 + TMEM),
// the B200 form of the parallel route of Section 4.2.
//
// Mathematics.  With gamma_t the product of alpha over the root path of node t, the rule
// S_t = alpha_t S_p + u_t k_t^T unrolls to
//        S_t = gamma_t S_0 + sum_{i in path(t)} (gamma_t / gamma_i) u_i k_i^T ,
// so with the two dense products  R = K S_0^T  and  G = Q S_0^T  (node x d_v):
//        u_t = beta_t v_t - beta_t gamma_t R_t - sum_{i strict ancestor of t} beta_t (gamma_t/gamma_i) (k_t.k_i) u_i
//        o_t = scale [ gamma_t G_t + sum_{i in path(t)} (gamma_t/gamma_i) (q_t.k_i) u_i ]
// This is the factorisation of Section 4.2 (A_tree = M_tree o K_b K_a^T, T = (I - A_tree)^-1,
// O = Qhat S0^T - Attn (W S0^T) + Attn U) with the triangular solve done as a forward
// substitution along ancestor paths: a node has at most max_depth - 1 ancestors, so the
// L x L solve, W and the padded factor tensors never exist.
//
// Mapping.  One persistent CTA per SM walks units (layer, sequence, head).  Per unit:
//   * the fp32 state tile [128 value rows x d_k] is the A operand exactly as TMA lands it
//     (K-major, 128-byte swizzle); it is read by the tensor core as TF32 and never touched
//     by a CUDA core;
//   * [K;Q] of the sequence's nodes, converted bf16 -> fp32 (exact in TF32) and laid out in
//     depth-first order, is the B operand; one MMA chain per tile gives D[v, node] =
//     (R | G)^T in TMEM with value rows on TMEM lanes, so the substitution is thread-local;
//   * the same [K;Q] block times K^T gives every q.k and k.k the coefficients need;
//   * epilogue threads own one value row each, keep the u of the current depth-first path
//     in registers (a stack indexed by depth) and stream o out coalesced.
// Roles: warp 0 TMA producer, warp 1 MMA issuer + TMEM owner, warps 2-5 operand/coefficient
// preparation, warps 6-13 two epilogue groups.  Every wait is bounded; on expiry the CTA
// raises SPECA_STATUS_TIMEOUT, drains and exits.
#include <cuda.h>

#include "speca_common.cuh"

namespace speca {

namespace {

constexpr int kDK = 128;                       // key width handled by this route
constexpr int kTileRows = 128;                 // value rows per tile (= TMEM lanes = MMA M)
constexpr int kChunkK = 32;                    // floats per 128-byte swizzle row
constexpr int kChunks = kDK / kChunkK;         // 4 K-chunks per tile
constexpr int kStageBytes = kTileRows * 128;   // 16 KiB per (tile, K-chunk)
constexpr int kStages = 6;
constexpr int kMaxNodes = 64;                  // nodes per sequence handled by this route
constexpr int kMaxDepth = 8;
constexpr int kBopRows = 2 * kMaxNodes;        // [K;Q] rows
constexpr int kBopChunkBytes = kBopRows * 128; // 16 KiB per K-chunk region
constexpr int kCoefStride = 20;                // floats per position: cU[8] cO[8] cV cR cG meta
constexpr int kAccCols = 2 * kMaxNodes;        // 128 TMEM columns per accumulator
constexpr int kNumAcc = 3;
constexpr int kGramCol = kNumAcc * kAccCols;   // 384
constexpr int kTmemCols = 512;
constexpr int kThreads = 14 * 32;
constexpr int kPrepThreads = 128;
constexpr int kGramHalf = 32;                  // Gram columns parked per extraction pass
constexpr int kVBufBytes = kMaxNodes * kTileRows * 2;   // bf16 value tile of one sequence: 16 KiB

// shared memory carve-up (bytes, from a 1024-byte aligned base)
constexpr int kOffRing = 0;
constexpr int kOffBop = kOffRing + kStages * kStageBytes;                 // 98304
constexpr int kOffGram = kOffBop + kChunks * kBopChunkBytes;              // +65536
constexpr int kOffVBuf = kOffGram + kGramHalf * kTileRows * 4;            // +16384
constexpr int kOffCoef = kOffVBuf + 2 * kVBufBytes;                       // +32768
constexpr int kOffAlpha = kOffCoef + 2 * kMaxNodes * kCoefStride * 4;     // +10240
constexpr int kOffBars = kOffAlpha + 2 * kMaxNodes * 4;                   // alpha, beta by position
constexpr int kOffMisc = kOffBars + 8 * 32;
constexpr int kSmemBytes = kOffMisc + 64 + 1024;                          // + alignment slack
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

enum Bar {
    kBarFull = 0,                        // [kStages] TMA -> MMA
    kBarEmpty = kBarFull + kStages,      // [kStages] MMA -> TMA
    kBarBReady = kBarEmpty + kStages,    // prep -> MMA (and prep-internal): [K;Q] operand, alpha, beta written
    kBarBFree,                           // MMA -> prep: operand no longer read
    kBarGramFull,                        // MMA -> prep: Gram block in TMEM
    kBarCoefReady,                       // [2] prep -> epilogue
    kBarCoefFree = kBarCoefReady + 2,    // [2] epilogue -> prep
    kBarAccFull = kBarCoefFree + 2,      // [kNumAcc] MMA -> epilogue
    kBarAccFree = kBarAccFull + kNumAcc, // [kNumAcc] epilogue -> MMA
    kBarVReady = kBarAccFree + kNumAcc,  // [2] per epilogue group: staged value tile has landed
    kBarVFree = kBarVReady + 2,          // [2] per epilogue group: staged value tile no longer read
    kBarDrain = kBarVFree + 2,           // MMA warp: everything issued has completed
    kBarCount
};
static_assert(kBarCount <= 32, "barrier region too small");

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// the mbarrier receives one arrival once all earlier cp.async of this thread have landed
__device__ __forceinline__ void cp_async_arrive(uint32_t bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded, warp-uniform wait.  Returns false if the CTA is aborting (this wait or another
// one gave up); the caller must then leave its loop.  All 32 lanes must call it together.
constexpr uint64_t kWaitLimitNs = 2000000000ull;       // 2 s
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        const bool ok = mbar_try_wait(bar, parity);
        if (__any_sync(0xffffffffu, ok)) return true;
        if ((it & 255u) == 255u) {
            if (__any_sync(0xffffffffu, *abort_flag != 0)) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            if (__any_sync(0xffffffffu, now - t0 > kWaitLimitNs)) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&r)[8])
{
    uint32_t x[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3]), "=r"(x[4]), "=r"(x[5]), "=r"(x[6]), "=r"(x[7])
                 : "r"(taddr)
                 : "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) r[i] = __uint_as_float(x[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major operand descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= uint64_t((smem_addr >> 4) & 0x3fffu);          // start address
    d |= uint64_t(1) << 16;                              // leading byte offset (unused for swizzled K-major)
    d |= uint64_t(1024 >> 4) << 32;                      // stride byte offset between 8-row groups
    d |= uint64_t(1) << 46;                              // descriptor version (Blackwell)
    d |= uint64_t(2) << 61;                              // SWIZZLE_128B
    return d;
}
// kind::tf32, fp32 accumulate, both operands K-major, M = 128
__device__ __forceinline__ uint32_t make_idesc(int n)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | (uint32_t(n >> 3) << 17) | (uint32_t(kTileRows >> 4) << 24);
}

struct FParams {
    Params p;
    int32_t tiles_per_unit;      // d_v / 128
    long n_units;
};

// Byte offset of (row r, float e) inside the swizzled [K;Q] operand.
__device__ __forceinline__ uint32_t bop_offset(int r, int e)
{
    const int c = e >> 5, w = (e >> 2) & 7;
    return uint32_t(c * kBopChunkBytes + (r >> 3) * 1024 + (r & 7) * 128 + ((w ^ (r & 7)) << 4) + ((e & 3) << 2));
}

template <int D>
__device__ __forceinline__ void node_step(float (&ustk)[kMaxDepth], const float *cf, float Rv, float Gv, float vv,
                                          float &u_out, float &o_out)
{
    // cf: cU[0..7] cO[0..7] cV cR cG
    const float4 a0 = *reinterpret_cast<const float4 *>(cf + 0), a1 = *reinterpret_cast<const float4 *>(cf + 4);
    const float4 b0 = *reinterpret_cast<const float4 *>(cf + 8), b1 = *reinterpret_cast<const float4 *>(cf + 12);
    const float4 s = *reinterpret_cast<const float4 *>(cf + 16);
    const float cU[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    const float cO[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
    float u = fmaf(s.x, vv, s.y * Rv);
    float o = s.z * Gv;
#pragma unroll
    for (int j = 0; j < D - 1; ++j) {
        u = fmaf(cU[j], ustk[j], u);
        o = fmaf(cO[j], ustk[j], o);
    }
    ustk[D - 1] = u;
    o_out = fmaf(cO[D - 1], u, o);
    u_out = u;
}

__device__ __forceinline__ int anc_byte(const int4 &meta, int j)
{
    return int((j < 4 ? (uint32_t(meta.y) >> (8 * j)) : (uint32_t(meta.z) >> (8 * (j - 4)))) & 0xffu);
}

__global__ void __launch_bounds__(kThreads, 1)
verify_factorized_kernel(const __grid_constant__ CUtensorMap s0_map, FParams fp)
{
    extern __shared__ uint8_t smem_raw[];
    const Params &p = fp.p;
    // 1024-byte alignment for the swizzled operand regions
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + kOffBars;
    auto bar = [&](int i) { return bars + 8u * uint32_t(i); };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffMisc);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + kOffMisc + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int TPU = fp.tiles_per_unit;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kStages; ++s) { mbar_init(bar(kBarFull + s), 1); mbar_init(bar(kBarEmpty + s), 1); }
        mbar_init(bar(kBarBReady), kPrepThreads);
        mbar_init(bar(kBarBFree), 1);
        mbar_init(bar(kBarGramFull), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(kBarCoefReady + i), kPrepThreads);
            mbar_init(bar(kBarCoefFree + i), 128 * TPU);
            mbar_init(bar(kBarVReady + i), 128);
            mbar_init(bar(kBarVFree + i), 128);
        }
        for (int i = 0; i < kNumAcc; ++i) { mbar_init(bar(kBarAccFull + i), 1); mbar_init(bar(kBarAccFree + i), 128); }
        mbar_init(bar(kBarDrain), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Every role walks the same list of units: u = blockIdx.x, += gridDim.x, skipping
    // sequences that failed validation or are empty.
    struct Unit { long u; int b, l, h, n, npad, base; };
    auto load_unit = [&](long u, Unit &x) {
        x.u = u;
        x.h = int(u % p.H); x.b = int((u / p.H) % p.B); x.l = int(u / (long(p.H) * p.B));
        x.n = p.ws.seq_n[x.b];
        x.npad = (x.n + 15) & ~15;
        x.base = __ldg(p.node_offsets + x.b);
    };
    auto next_unit = [&](long from, Unit &x) {         // first valid unit at or after `from`; false at the end
        for (long u = from; u < fp.n_units; u += gridDim.x) {
            load_unit(u, x);
            if (x.n > 0) return true;
        }
        x.u = fp.n_units; x.n = 0;
        return false;
    };

    if (warp == 0) {
        // ------------------------------------------------------------- TMA producer
        uint32_t it = 0;
        Unit x;
        bool ok = true;
        for (bool have = next_unit(blockIdx.x, x); have && ok; have = next_unit(x.u + gridDim.x, x)) {
            for (int t = 0; t < TPU && ok; ++t) {
                const int row = int(x.u * p.DV) + t * kTileRows;      // row in the [units*d_v, d_k] view of S0
                for (int c = 0; c < kChunks; ++c, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1;
                    if (!(ok = mbar_wait(bar(kBarEmpty + s), ph ^ 1, abort_flag))) break;
                    if (lane == 0) {
                        mbar_arrive_expect_tx(bar(kBarFull + s), kStageBytes);
                        tma_load_2d(sbase + kOffRing + s * kStageBytes, &s0_map, c * kChunkK, row, bar(kBarFull + s));
                    }
                    __syncwarp();
                }
            }
        }
        // let copies still in flight land before the CTA's shared memory goes away
        if (*abort_flag) {
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------- MMA issuer
        uint32_t it = 0, unit_seq = 0, tile_seq = 0;
        Unit x;
        bool ok = true;
        const uint32_t bop = sbase + kOffBop;
        for (bool have = next_unit(blockIdx.x, x); have && ok; have = next_unit(x.u + gridDim.x, x), ++unit_seq) {
            if (!(ok = mbar_wait(bar(kBarBReady), unit_seq & 1, abort_flag))) break;
            tc_fence_after();
            if (lane == 0) {
                // Gram block: [K;Q] (128 rows) x K^T (npad columns)
                const uint32_t idg = make_idesc(x.npad);
#pragma unroll 1
                for (int c = 0; c < kChunks; ++c)
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t d = make_desc(bop + c * kBopChunkBytes + k * 32);
                        mma_tf32(tmem_base + kGramCol, d, d, idg, (c | k) != 0);
                    }
                mma_commit(bar(kBarGramFull));
            }
            __syncwarp();
            const uint32_t idm = make_idesc(2 * x.npad);
            for (int t = 0; t < TPU && ok; ++t, ++tile_seq) {
                const int a = tile_seq % kNumAcc;
                const uint32_t aph = (tile_seq / kNumAcc) & 1;
                if (!(ok = mbar_wait(bar(kBarAccFree + a), aph ^ 1, abort_flag))) break;
                tc_fence_after();
                for (int c = 0; c < kChunks; ++c, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1;
                    if (!(ok = mbar_wait(bar(kBarFull + s), ph, abort_flag))) break;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t sa = sbase + kOffRing + s * kStageBytes;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_tf32(tmem_base + a * kAccCols, make_desc(sa + k * 32),
                                     make_desc(bop + c * kBopChunkBytes + k * 32), idm, (c | k) != 0);
                        mma_commit(bar(kBarEmpty + s));
                    }
                    __syncwarp();
                }
                if (ok && lane == 0) mma_commit(bar(kBarAccFull + a));
                __syncwarp();
            }
            if (ok && lane == 0) mma_commit(bar(kBarBFree));
            __syncwarp();
        }
        // everything this warp issued must have completed before TMEM is released
        if (lane == 0) mma_commit(bar(kBarDrain));
        __syncwarp();
        mbar_wait(bar(kBarDrain), 0, abort_flag);
    } else if (warp < 6) {
        // ------------------------------------------------------------- operand + coefficient preparation
        const int tid = threadIdx.x - 64;                        // 0..127
        const int row = 32 * (warp & 3) + lane;                  // Gram row (= TMEM lane) of this thread
        const uint32_t lane_addr = uint32_t(32 * (warp & 3)) << 16;
        float *gram = reinterpret_cast<float *>(smem + kOffGram);
        float *alpha_s = reinterpret_cast<float *>(smem + kOffAlpha);
        float *beta_s = alpha_s + kMaxNodes;
        const int sub = tid >> 4, e = (tid & 15) * 8;            // row within a group of 8, first of 8 floats

        // raw bf16 rows of [K;Q] for the unit about to be written, fetched one unit ahead
        uint4 raw[16];
        float my_alpha = 0.f, my_beta = 0.f;
        auto prefetch = [&](const Unit &x) {
            const int4 *anc = reinterpret_cast<const int4 *>(p.ws.anc) + x.base;
            int node[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int r = 8 * i + sub;
                const int pos = r < x.npad ? r : r - x.npad;
                node[i] = (r < 2 * x.npad && pos < x.n) ? ((__ldg(&anc[pos].x) >> 8) & 0xffff) : -1;
            }
            const int my_node = tid < x.n ? ((__ldg(&anc[tid].x) >> 8) & 0xffff) : -1;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int r = 8 * i + sub;
                if (node[i] >= 0) {
                    const long rec = (long(x.l) * p.T + x.base + node[i]) * p.H + x.h;
                    raw[i] = __ldg(reinterpret_cast<const uint4 *>((r < x.npad ? p.k : p.q) + rec * kDK + e));
                } else {
                    raw[i] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
            if (my_node >= 0) {
                const long rec = (long(x.l) * p.T + x.base + my_node) * p.H + x.h;
                my_alpha = __ldg(p.alpha + rec);
                my_beta = __ldg(p.beta + rec);
            }
        };

        uint32_t unit_seq = 0;
        Unit x, nx;
        bool ok = true;
        bool have = next_unit(blockIdx.x, x);
        if (have) prefetch(x);
        for (; have && ok; ++unit_seq) {
            const int par = unit_seq & 1;
            // the previous unit's MMAs must be done reading the operand, and every prep thread
            // must be done reading alpha/beta of the previous unit
            if (unit_seq > 0) {
                if (!(ok = mbar_wait(bar(kBarBFree), (unit_seq - 1) & 1, abort_flag))) break;
                if (!(ok = mbar_wait(bar(kBarCoefReady + (par ^ 1)), ((unit_seq - 1) >> 1) & 1, abort_flag))) break;
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int r = 8 * i + sub;
                if (r < 2 * x.npad) {
                    const uint4 w = raw[i];
                    *reinterpret_cast<float4 *>(smem + kOffBop + bop_offset(r, e)) =
                        make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u),
                                    __uint_as_float(w.y << 16), __uint_as_float(w.y & 0xffff0000u));
                    *reinterpret_cast<float4 *>(smem + kOffBop + bop_offset(r, e + 4)) =
                        make_float4(__uint_as_float(w.z << 16), __uint_as_float(w.z & 0xffff0000u),
                                    __uint_as_float(w.w << 16), __uint_as_float(w.w & 0xffff0000u));
                }
            }
            if (tid < x.n) { alpha_s[tid] = my_alpha; beta_s[tid] = my_beta; }
            fence_proxy_async();
            mbar_arrive(bar(kBarBReady));
            // start fetching the next unit's rows while this unit's Gram block is produced
            const bool have_next = next_unit(x.u + gridDim.x, nx);
            if (have_next) prefetch(nx);
            // all prep threads have written alpha/beta (the operand barrier doubles as the prep barrier)
            if (!(ok = mbar_wait(bar(kBarBReady), unit_seq & 1, abort_flag))) break;
            // the coefficient buffer of this parity must have been released by the epilogue
            if (unit_seq >= 2 && !(ok = mbar_wait(bar(kBarCoefFree + par), ((unit_seq >> 1) - 1) & 1, abort_flag))) break;
            if (!(ok = mbar_wait(bar(kBarGramFull), unit_seq & 1, abort_flag))) break;
            tc_fence_after();

            float *coef = reinterpret_cast<float *>(smem + kOffCoef) + par * kMaxNodes * kCoefStride;
            const int4 *anc = reinterpret_cast<const int4 *>(p.ws.anc) + x.base;
            const bool is_k = row < x.npad;
            const int pos = is_k ? row : row - x.npad;
            const bool active = row < 2 * x.npad && pos < x.n;
            int4 meta = make_int4(0, 0, 0, 0);
            if (active) meta = __ldg(&anc[pos]);
            const int d = meta.x & 0xff;
            float *cf = coef + pos * kCoefStride;
            const float sgn = is_k ? -beta_s[active ? pos : 0] : p.scale;
            for (int half = 0; half * kGramHalf < x.npad; ++half) {
                // park this thread's Gram row (32 columns) in its private scratch column
#pragma unroll
                for (int c0 = 0; c0 < kGramHalf; c0 += 8) {
                    float g[8];
                    tmem_ld8(tmem_base + lane_addr + kGramCol + half * kGramHalf + c0, g);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 8; ++i) gram[(c0 + i) * kTileRows + row] = g[i];
                }
                if (active) {
                    float ratio = alpha_s[pos];
                    if (!is_k && (pos >> 5) == half) cf[8 + d - 1] = sgn * gram[(pos & 31) * kTileRows + row];
                    for (int j = d - 2; j >= 0; --j) {
                        const int a = anc_byte(meta, j);
                        if ((a >> 5) == half) cf[(is_k ? 0 : 8) + j] = sgn * ratio * gram[(a & 31) * kTileRows + row];
                        ratio *= alpha_s[a];
                    }
                    if (half == 0) {
                        if (is_k) { cf[16] = -sgn; cf[17] = sgn * ratio; }          // cV = beta, cR = -beta gamma
                        else { cf[18] = sgn * ratio; cf[19] = __int_as_float(meta.x); }   // cG = scale gamma, depth|node<<8
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar(kBarCoefReady + par));
            x = nx;
            have = have_next;
        }
    } else {
        // ------------------------------------------------------------- epilogue groups
        const int grp = (warp - 6) >> 2;
        const int gtid = threadIdx.x - (6 + 4 * grp) * 32;       // 0..127 within the group
        const int row = 32 * (warp & 3) + lane;
        const uint32_t lane_addr = uint32_t(32 * (warp & 3)) << 16;
        const uint32_t vbuf = sbase + kOffVBuf + grp * kVBufBytes;
        const unsigned short *vbuf_g = reinterpret_cast<const unsigned short *>(smem + kOffVBuf + grp * kVBufBytes);

        struct Tile { Unit x; int t; uint32_t unit_seq, tile_seq; bool valid; };
        // advance to the next tile owned by this group (tile_seq parity == grp)
        auto advance = [&](Tile &tl, bool first) {
            if (first) {
                tl.valid = next_unit(blockIdx.x, tl.x);
                tl.t = 0; tl.unit_seq = 0; tl.tile_seq = 0;
                if (!tl.valid || int(tl.tile_seq & 1) == grp) return;
            }
            while (tl.valid) {
                ++tl.tile_seq;
                if (++tl.t == TPU) {
                    tl.t = 0;
                    ++tl.unit_seq;
                    Unit nx;
                    tl.valid = next_unit(tl.x.u + gridDim.x, nx);
                    tl.x = nx;
                }
                if (tl.valid && int(tl.tile_seq & 1) == grp) return;
            }
        };
        // stage the bf16 value tile [n][128 rows] of a tile into this group's buffer
        auto stage_values = [&](const Tile &tl) {
            if (tl.valid) {
                const int4 *anc = reinterpret_cast<const int4 *>(p.ws.anc) + tl.x.base;
                const long rec0 = (long(tl.x.l) * p.T + tl.x.base) * p.H + tl.x.h;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int idx = gtid + 128 * i, pos = idx >> 4, seg = idx & 15;
                    if (pos < tl.x.n) {
                        const int node = (__ldg(&anc[pos].x) >> 8) & 0xffff;
                        const __nv_bfloat16 *src = p.v + (rec0 + long(node) * p.H) * p.DV + tl.t * kTileRows + seg * 8;
                        cp_async_16(vbuf + pos * 256 + seg * 16, src);
                    }
                }
            }
            cp_async_arrive(bar(kBarVReady + grp));
        };

        Tile cur;
        advance(cur, true);
        stage_values(cur);
        uint32_t my_seq = 0;                                     // tiles processed by this group
        bool ok = true;
        while (cur.valid && ok) {
            const Unit &x = cur.x;
            const int par = cur.unit_seq & 1;
            const float *coef = reinterpret_cast<const float *>(smem + kOffCoef) + par * kMaxNodes * kCoefStride;
            if (!(ok = mbar_wait(bar(kBarCoefReady + par), (cur.unit_seq >> 1) & 1, abort_flag))) break;
            if (!(ok = mbar_wait(bar(kBarVReady + grp), my_seq & 1, abort_flag))) break;
            const int a = cur.tile_seq % kNumAcc;
            if (!(ok = mbar_wait(bar(kBarAccFull + a), (cur.tile_seq / kNumAcc) & 1, abort_flag))) break;
            tc_fence_after();
            const long rec0 = (long(x.l) * p.T + x.base) * p.H + x.h;          // record of node 0
            const int vrow = cur.t * kTileRows + row;
            float ustk[kMaxDepth];
#pragma unroll
            for (int j = 0; j < kMaxDepth; ++j) ustk[j] = 0.f;
            for (int p0 = 0; p0 < x.n; p0 += 8) {
                float Rv[8], Gv[8];
                tmem_ld8(tmem_base + lane_addr + a * kAccCols + p0, Rv);
                tmem_ld8(tmem_base + lane_addr + a * kAccCols + x.npad + p0, Gv);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (p0 + i < x.n) {
                        const float *cf = coef + (p0 + i) * kCoefStride;
                        const int meta = __float_as_int(cf[19]);
                        const int d = meta & 0xff, node = (meta >> 8) & 0xffff;
                        const float vv = __uint_as_float(uint32_t(vbuf_g[(p0 + i) * kTileRows + row]) << 16);
                        float uo, oo;
                        switch (d) {
                        case 1: node_step<1>(ustk, cf, Rv[i], Gv[i], vv, uo, oo); break;
                        case 2: node_step<2>(ustk, cf, Rv[i], Gv[i], vv, uo, oo); break;
                        case 3: node_step<3>(ustk, cf, Rv[i], Gv[i], vv, uo, oo); break;
                        case 4: node_step<4>(ustk, cf, Rv[i], Gv[i], vv, uo, oo); break;
                        case 5: node_step<5>(ustk, cf, Rv[i], Gv[i], vv, uo, oo); break;
                        case 6: node_step<6>(ustk, cf, Rv[i], Gv[i], vv, uo, oo); break;
                        case 7: node_step<7>(ustk, cf, Rv[i], Gv[i], vv, uo, oo); break;
                        default: node_step<8>(ustk, cf, Rv[i], Gv[i], vv, uo, oo); break;
                        }
                        const long out = (rec0 + long(node) * p.H) * p.DV + vrow;
                        p.o[out] = oo;
                        if (p.u != nullptr) p.u[out] = uo;
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar(kBarAccFree + a));
            mbar_arrive(bar(kBarCoefFree + par));
            mbar_arrive(bar(kBarVFree + grp));
            // next tile of this group: refill the value buffer once every thread has left it
            advance(cur, false);
            if (!(ok = mbar_wait(bar(kBarVFree + grp), my_seq & 1, abort_flag))) break;
            ++my_seq;
            stage_values(cur);
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, SPECA_STATUS_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = [] {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            sym = nullptr;
        return reinterpret_cast<EncodeTiledFn>(sym);
    }();
    return fn;
}

}  // namespace

bool factorized_supported(const speca_dims *d)
{
    return d->d_k == kDK && d->d_v % kTileRows == 0 && d->max_nodes <= kMaxNodes && d->max_depth <= kMaxDepth;
}

int launch_verify_factorized(const Params &p, cudaStream_t st)
{
    EncodeTiledFn encode = encode_tiled_fn();
    if (encode == nullptr) return int(cudaErrorNotSupported);
    const long n_units = long(p.L) * p.B * p.H;
    CUtensorMap map;
    const cuuint64_t gdim[2] = {cuuint64_t(kDK), cuuint64_t(n_units) * cuuint64_t(p.DV)};
    const cuuint64_t gstride[1] = {cuuint64_t(kDK) * sizeof(float)};
    const cuuint32_t box[2] = {kChunkK, kTileRows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(p.S0), gdim, gstride, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return int(cudaErrorInvalidValue);

    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (sm_count <= 0) sm_count = 148;
    }
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(verify_factorized_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kSmemBytes);
        if (e != cudaSuccess) return int(e);
        attr_set = true;
    }
    FParams fp;
    fp.p = p;
    fp.tiles_per_unit = p.DV / kTileRows;
    fp.n_units = n_units;
    const int grid = int(n_units < sm_count ? n_units : sm_count);
    verify_factorized_kernel<<<grid, kThreads, kSmemBytes, st>>>(map, fp);
    return int(cudaGetLastError());
}

}  // namespace speca
