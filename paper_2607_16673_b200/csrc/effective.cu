// Tree-masked verification with effective queries on the 5th-generation tensor cores
// (tcgen05 + TMEM): the parallel route of Section 4.2 with every coefficient matrix moved to
// the small side of ONE accumulation chain, at fp32 accuracy.
//
// Mathematics.  With gamma_t the product of alpha over the root path of node t, a_0 .. a_{d-1}
// that path (a_{d-1} = t) and rho_t[j] = gamma_t / gamma_{a_j}, the factorisation of Section 4.2
// (A_tree = M_tree o K_b K_a^T, T = (I + A)^-1, O = Qhat S0^T - Attn (W S0^T) + Attn U) regroups as
//        o_t = S0 qeff_t + sum_j Mq[t][a_j] v_{a_j} ,      u_t = -S0 weff_t + sum_j Mk[t][a_j] v_{a_j}
// with, per node, two short coefficient rows taken from the gate-free triangular system
// X = (I + Ahat)^-1, Ahat[t][i] = beta_t (k_t.k_i) over strict ancestors, and C = Phat X,
// Phat[t][i] = q_t.k_i over the path:
//        qeff_t = scale gamma_t ( q_t - sum_j C[t][j] beta_{a_j} k_{a_j} )   Mq[t][a_j] = scale rho_t[j] C[t][j] beta_{a_j}
//        weff_t =       gamma_t   sum_j X[t][j] beta_{a_j} k_{a_j}           Mk[t][a_j] =       rho_t[j] X[t][j] beta_{a_j}
// (W and Attn of the paper are these rows; the triangular solve is a forward substitution along
// ancestor paths, at most 15 steps).  Everything that depends on the state is then one dense
// contraction of the state tile with N effective vectors, plus a small product with the value
// rows; the epilogue only adds two accumulator columns and stores.
//
// Accuracy.  The tensor core reads fp32 operands as TF32 (top 19 bits).  Both operands are
// therefore split: the state slice as landed (its TF32 head, free) and its exact remainder
// S - tf32(S), rewritten in place by a CUDA-core role once the first pass has read the slice;
// the effective vectors as a TF32-rounded head and the exact remainder, stacked as 2R operand
// rows.  Pass 1: S x [head; tail] -> accumulator columns [0,R) and [R,2R); pass 2: (S - tf32(S)) x
// head -> columns [0,R).  The dropped term is 2^-22 of the result.  Mq / Mk are split into three
// bf16 pieces (24 bits) and multiply the bf16 value rows exactly.
//
// Mapping.  One persistent CTA per SM walks units (layer, sequence, head); 18 warps:
//   warp 0       streams the fp32 state, K-slice by K-slice over both value tiles (TMA, 128-byte swizzle);
//   warp 1       issues every tcgen05.mma and owns TMEM (two units of accumulators in flight);
//   warps 2-9    preparation: Gram rows out of TMEM, the two substitutions, one record per operand
//                row, the three bf16 pieces of M, then the effective vectors one K-slice at a time
//                into a double-buffered operand (so they never exist whole);
//   warps 10-13  rewrite each state slice as its TF32 remainder between the two passes;
//   warps 14-17  epilogue: o (or u) = column t + column R + t, streamed out coalesced.
// Nodes keep their index order everywhere.  When u is requested a unit is walked twice (first the
// o rows, then the u rows); the second walk finds the state tile in L2.
// Every wait is bounded; on expiry the CTA raises SPECA_STATUS_TIMEOUT, drains and exits.
#include <cuda.h>

#include "speca_common.cuh"
#include "tc_ptx.cuh"

namespace speca {

namespace {

using namespace tc;

constexpr int kRows = 128;                      // value rows per tile (= TMEM lanes = MMA M)
constexpr int kSliceBytes = kRows * 128;        // one K-slice of a tile: 128 rows x 32 fp32
constexpr int kMaxD = 16;                       // tree depth taken
constexpr int kAccCols = 128;                   // accumulator columns per tile: [head R | tail R], R <= 64
constexpr int kPairCols = 2 * kAccCols;
constexpr int kTmemCols = 512;
constexpr int kThreads = 18 * 32;
constexpr int kSolveThreads = 128;
constexpr int kSplitThreads = 128;
constexpr int kRecBytes = 112;                  // per operand row: count, 17 weights, 17 staging offsets
constexpr int kRecW = 4, kRecOff = 72;
constexpr int kWalkSeqs = 128;

// shared-memory carve-up per instantiation
template <int TP, int DK> struct Lay {
    static constexpr int MAXN = DK == 128 ? 64 : 32;            // nodes per sequence
    static constexpr int NC = DK / 32;                          // K-slices per tile
    static constexpr int SC = DK / 64;                          // 64-column regions of the staged bf16 rows
    static constexpr int SCB = 2 * MAXN * 128;                  // bytes per region: key rows, then query rows
    static constexpr int STAGE = SC * SCB;
    static constexpr int BBUF = 2 * MAXN * 128;                 // one K-slice of the operand: head rows, tail rows
    static constexpr int MPIECE = MAXN * 128;                   // one bf16 piece of M: R rows x 64 columns
    static constexpr int VBLK = MAXN * 128;                     // 64 values of all nodes
    static constexpr int VBYTES = TP * 2 * VBLK;
    static constexpr int kTemp = MAXN * kRows * 4;              // whole Gram block of a unit, parked in the value-row buffer
    static constexpr int VREG = VBYTES > kTemp ? VBYTES : kTemp;
    static constexpr int kFixed = 2 * BBUF + 2 * STAGE + 3 * MPIECE + VREG + 64 * kRecBytes + 2 * 64 * 4 + 512 + 64 +
                                  5 * kWalkSeqs;
    static constexpr int kRoom = (227 * 1024 - kFixed - 1024) / kSliceBytes;
    static constexpr int NS = kRoom > 6 ? 6 : kRoom;            // ring depth
    static constexpr int OffRing = 0;
    static constexpr int OffB = OffRing + NS * kSliceBytes;
    static constexpr int OffStage = OffB + 2 * BBUF;
    static constexpr int OffM = OffStage + 2 * STAGE;
    static constexpr int OffV = OffM + 3 * MPIECE;
    static constexpr int OffTemp = OffV;
    static constexpr int OffRec = OffV + VREG;
    static constexpr int OffAlpha = OffRec + 64 * kRecBytes;
    static constexpr int OffBars = OffAlpha + 2 * 64 * 4;
    static constexpr int OffMisc = OffBars + 512;
    static constexpr int OffWalk = OffMisc + 64;
    static constexpr int Bytes = OffWalk + 5 * kWalkSeqs;
    static_assert(NS >= 4, "ring too shallow");
    static_assert(Bytes <= 227 * 1024, "shared memory budget");
};

enum Bar {
    kFull = 0,                 // [6] TMA -> MMA (and split): slice landed
    kEmpty = kFull + 6,        // [6] MMA -> TMA: second pass has read the slice
    kP1Done = kEmpty + 6,      // [6] MMA -> split: first pass has read the slice
    kLo = kP1Done + 6,         // [6] split -> MMA: slice rewritten as its remainder
    kKQFull = kLo + 6,         // [2] TMA -> MMA, prep: staged bf16 key / query rows of a unit
    kGramFull = kKQFull + 2,   // MMA -> prep: Gram block in TMEM
    kGramDone,                 // prep -> MMA: Gram rows read, the columns may be overwritten
    kBReady,                   // [2] prep -> MMA: operand slice written
    kBFree = kBReady + 2,      // [2] MMA -> prep: operand slice no longer read
    kMReady = kBFree + 2,      // prep -> MMA: pieces of M written
    kMFree,                    // MMA -> prep
    kVFull,                    // TMA -> MMA: value rows staged
    kVFree,                    // MMA -> prep (which issues the copy)
    kAccFull,                  // [2] MMA -> epilogue
    kPairFree = kAccFull + 2,  // [2] epilogue -> MMA
    kRecReady = kPairFree + 2, // solver -> vector warps: records of a unit written
    kRecFree,                  // vector warps -> solver
    kSolveSync,                // role-internal
    kVecSync,
    kDrain,
    kBarCount
};
static_assert(kBarCount * 8 <= 512, "barrier region too small");

struct EMaps { CUtensorMap k[4], q[4], v[4]; };       // one per box height: 16, 32, 48, 64 nodes

struct EParams {
    Params p;
    int32_t heads_per_group;
    int32_t withhold_first_load;     // failure-detection test: CTA 0 never requests its first state slice
    int32_t want_u;
    long n_units;
};

// A unit is one (layer, sequence, head); with u requested it is walked twice (kind 0: o rows, kind 1: u rows).
struct VUnit { int grp, hi, u, b, l, h, n, npad, base, kind; };
struct Walk {
    int HG, gpl, n_groups, H, B, grid, two;
    const int32_t *seq_n; const int32_t *offs;
    const uint8_t *tab;
};

__device__ __forceinline__ bool load_group(const Walk &w, int G, VUnit &x)
{
    for (; G < w.n_groups; G += w.grid) {
        const int lb = G / w.gpl;
        x.b = lb % w.B;
        const bool in_tab = x.b < kWalkSeqs;
        x.n = in_tab ? int(reinterpret_cast<const int8_t *>(w.tab + 4 * kWalkSeqs)[x.b]) : w.seq_n[x.b];
        if (x.n > 0) {
            x.grp = G; x.hi = 0; x.kind = 0;
            x.l = lb / w.B;
            x.h = (G - lb * w.gpl) * w.HG;
            x.u = lb * w.H + x.h;
            x.npad = (x.n + 15) & ~15;
            x.base = in_tab ? reinterpret_cast<const int32_t *>(w.tab)[x.b] : __ldg(w.offs + x.b);
            return true;
        }
    }
    x.n = 0; x.grp = w.n_groups;
    return false;
}
__device__ __forceinline__ bool first_unit(const Walk &w, VUnit &x) { return load_group(w, int(blockIdx.x), x); }
__device__ __forceinline__ bool next_unit(const Walk &w, VUnit &x)
{
    if (w.two && x.kind == 0) { x.kind = 1; return true; }
    x.kind = 0;
    if (++x.hi < w.HG) { ++x.h; ++x.u; return true; }
    return load_group(w, x.grp + w.grid, x);
}

// ancestor (node index) of level j (0 = child of the committed state) from the plan kernel's two records
__device__ __forceinline__ int anc_at(const int4 &meta, int meta2, int j)
{
    const uint32_t w = j < 4 ? uint32_t(meta.y) : j < 8 ? uint32_t(meta.z) : j < 12 ? uint32_t(meta.w) : uint32_t(meta2);
    return int((w >> (8 * (j & 3))) & 0xffu);
}

// one arrival for the whole warp: every lane's earlier writes are ordered before it
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane)
{
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
}

__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }


// Optional self-profiling build (-DSPECA_PROF): cycles CTA 0 spends in each kind of wait, per warp,
// written to the control words of the workspace ([8 + 9 warp .. ): 8 slots and the warp's lifetime).
#ifdef SPECA_PROF
#define PROF_DECL long long prof_w[8] = {0, 0, 0, 0, 0, 0, 0, 0}; const long long prof_t0 = clock64();
#define WAIT(slot, b, ph) prof_wait(prof_w[slot], b, ph, abort_flag)
#define PROF_T0() const long long prof_seg0 = clock64();
#define PROF_ADD(slot) prof_w[slot] += clock64() - prof_seg0;
#define PROF_STORE()                                                                              \
    if (blockIdx.x == 0 && lane == 0) {                                                           \
        long long *dst = reinterpret_cast<long long *>(p.ws.ctrl) + 8 + warp * 9;                \
        for (int i_ = 0; i_ < 8; ++i_) dst[i_] = prof_w[i_];                                      \
        dst[8] = clock64() - prof_t0;                                                             \
    }
__device__ __forceinline__ bool prof_wait(long long &acc, uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    const long long t = clock64();
    const bool r = wait_fast(bar, parity, abort_flag);
    acc += clock64() - t;
    return r;
}
#else
#define PROF_DECL
#define PROF_T0()
#define PROF_ADD(slot)
#define WAIT(slot, b, ph) wait_fast(b, ph, abort_flag)
#define PROF_STORE()
#endif

// TP = value tiles per unit (d_v / 128), DK = key width.
template <int TP, int DK>
__global__ void __launch_bounds__(kThreads, 1)
verify_effective_kernel(const __grid_constant__ CUtensorMap s0_map, const __grid_constant__ EMaps maps, EParams ep)
{
    using LY = Lay<TP, DK>;
    constexpr int NS = LY::NS, NC = LY::NC, SC = LY::SC, SCB = LY::SCB;
    extern __shared__ __align__(1024) uint8_t smem[];
    const Params &p = ep.p;
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {                                 // never expected; refuse to run rather than corrupt
        if (threadIdx.x == 0) atomicOr(p.status, SPECA_STATUS_TIMEOUT);
        return;
    }
    const uint32_t bars = sbase + LY::OffBars;
    auto bar = [&](int i) { return bars + 8u * uint32_t(i); };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + LY::OffMisc);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + LY::OffMisc + 8);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < 6; ++s) {
            mbar_init(bar(kFull + s), 1);
            mbar_init(bar(kEmpty + s), 1);
            mbar_init(bar(kP1Done + s), 1);
            mbar_init(bar(kLo + s), kSplitThreads / 32);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(kKQFull + i), 1);
            mbar_init(bar(kBReady + i), 4);
            mbar_init(bar(kBFree + i), 1);
            mbar_init(bar(kAccFull + i), 1);
            mbar_init(bar(kPairFree + i), 4);
        }
        mbar_init(bar(kGramFull), 1);
        mbar_init(bar(kGramDone), kSolveThreads / 32);
        mbar_init(bar(kMReady), kSolveThreads / 32);
        mbar_init(bar(kMFree), 1);
        mbar_init(bar(kVFull), 1);
        mbar_init(bar(kVFree), 1);
        mbar_init(bar(kRecReady), 4);
        mbar_init(bar(kRecFree), 4);
        mbar_init(bar(kSolveSync), 4);
        mbar_init(bar(kVecSync), 4);
        mbar_init(bar(kDrain), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int b = threadIdx.x; b < p.B && b < kWalkSeqs; b += blockDim.x) {
        const int n = p.ws.seq_n[b];
        reinterpret_cast<int32_t *>(smem + LY::OffWalk)[b] = p.node_offsets[b];
        reinterpret_cast<int8_t *>(smem + LY::OffWalk + 4 * kWalkSeqs)[b] = int8_t(n < 0 ? -1 : n);
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    Walk walk;
    walk.HG = ep.heads_per_group; walk.gpl = p.H / ep.heads_per_group;
    walk.n_groups = int(ep.n_units / ep.heads_per_group);
    walk.H = p.H; walk.B = p.B; walk.grid = int(gridDim.x);
    walk.two = ep.want_u;
    walk.seq_n = p.ws.seq_n; walk.offs = p.node_offsets;
    walk.tab = smem + LY::OffWalk;

    if (warp == 0) {
        // ------------------------------------------------------------- state producer
        uint32_t it = 0;
        VUnit x;
        bool ok = true;
        PROF_DECL
        for (bool have = first_unit(walk, x); have && ok; have = next_unit(walk, x)) {
            for (int c = 0; c < NC && ok; ++c) {
                for (int t = 0; t < TP; ++t, ++it) {
                    const int s = it % NS;
                    if (!(ok = WAIT(0, bar(kEmpty + s), ((it / NS) & 1) ^ 1))) break;
                    if (lane == 0 && !(ep.withhold_first_load && blockIdx.x == 0 && it == 0)) {
                        mbar_arrive_expect_tx(bar(kFull + s), kSliceBytes);
                        tma_load_3d(sbase + LY::OffRing + s * kSliceBytes, &s0_map, c * 32, t * kRows, x.u, bar(kFull + s));
                    }
                    __syncwarp();
                }
            }
        }
        PROF_STORE()
        // let copies still in flight land before the CTA's shared memory goes away
        if (*abort_flag) {
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------- MMA issuer
        // Two cursors walk the same sequence of slices: the first pass is issued as soon as a slice and its
        // operand have landed, the second pass as soon as the slice has been rewritten as its remainder.
        // Neither blocks the other: the warp polls and serves whichever is ready.
        struct Cur { VUnit x; uint32_t useq, it, cc; int c, t; bool have; };
        auto advance = [&](Cur &q) {
            ++q.it;
            if (++q.t == TP) {
                q.t = 0; ++q.cc;
                if (++q.c == NC) { q.c = 0; ++q.useq; q.have = next_unit(walk, q.x); }
            }
        };
        bool ok = true;
        PROF_DECL
        // Gram block of a unit: [K;Q] (128 rows) x K^T (npad columns) from the staged bf16 rows, parked in the
        // unit's own accumulator columns until its state MMAs overwrite them.
        auto gram_ready = [&](uint32_t seq) -> bool {
            const int pr = seq & 1;
            return __all_sync(0xffffffffu, mbar_test_wait(bar(kKQFull + pr), (seq >> 1) & 1) &&
                                               mbar_test_wait(bar(kPairFree + pr), ((seq >> 1) & 1) ^ 1));
        };
        auto issue_gram = [&](uint32_t seq, int npad) {
            const int pr = seq & 1;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t idg = make_idesc_bf16(npad);
                const uint32_t stage = sbase + LY::OffStage + pr * LY::STAGE;
#pragma unroll
                for (int c = 0; c < SC; ++c)
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t d = make_desc(stage + c * SCB + k * 32);
                        mma_bf16(tmem_base + pr * kPairCols, d, d, idg, (c | k) != 0);
                    }
                mma_commit(bar(kGramFull));
            }
            __syncwarp();
        };
        Cur c1, c2;
        c1.useq = c1.it = c1.cc = 0; c1.c = c1.t = 0;
        c1.have = first_unit(walk, c1.x);
        c2 = c1;
        VUnit nx = c1.x;
        bool have_next = c1.have && next_unit(walk, nx);
        uint32_t gram_seq = 0;                                   // Gram blocks issued so far
        uint64_t t0 = 0;
        uint32_t spin = 0;
        while (ok && (c1.have || c2.it < c1.it)) {
            bool prog = false;
            // the Gram block of the unit the first cursor is in, or of the one after it
            if (c1.have && gram_seq == c1.useq && gram_ready(gram_seq)) {
                issue_gram(gram_seq, c1.x.npad);
                ++gram_seq;
                prog = true;
            } else if (c1.have && have_next && gram_seq == c1.useq + 1 && (c1.c > 0 || c1.t > 0) && gram_ready(gram_seq)) {
                issue_gram(gram_seq, nx.npad);
                ++gram_seq;
                prog = true;
            }
            // second pass
            if (c2.it < c1.it) {
                const int s = c2.it % NS;
                if (__all_sync(0xffffffffu, mbar_test_wait(bar(kLo + s), (c2.it / NS) & 1))) {
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t sa = sbase + LY::OffRing + s * kSliceBytes;
                        const uint32_t ba = sbase + LY::OffB + (c2.cc & 1) * LY::BBUF;
                        const uint32_t acc = tmem_base + (c2.useq & 1) * kPairCols + c2.t * kAccCols;
                        const uint32_t id2 = make_idesc(c2.x.npad);
#pragma unroll
                        for (int k = 0; k < 4; ++k) mma_tf32(acc, make_desc(sa + k * 32), make_desc(ba + k * 32), id2, 1);
                        mma_commit(bar(kEmpty + s));
                        if (c2.t == TP - 1) mma_commit(bar(kBFree + (c2.cc & 1)));
                        if (c2.t == TP - 1 && c2.c == NC - 1) mma_commit(bar(kAccFull + (c2.useq & 1)));
                    }
                    __syncwarp();
                    advance(c2);
                    prog = true;
                }
            }
            // first pass
            if (c1.have && gram_seq > c1.useq) {
                const int s = c1.it % NS;
                bool ready = mbar_test_wait(bar(kBReady + (c1.cc & 1)), (c1.cc >> 1) & 1) &&
                             mbar_test_wait(bar(kFull + s), (c1.it / NS) & 1);
                if (c1.c == 0 && c1.t == 0) ready = ready && mbar_test_wait(bar(kGramDone), c1.useq & 1);
                if (c1.c == 1 && c1.t == 0)
                    ready = ready && mbar_test_wait(bar(kMReady), c1.useq & 1) && mbar_test_wait(bar(kVFull), c1.useq & 1);
                // the last slice of a unit waits for the next unit's Gram block to be on its way, so that the
                // preparation of that unit is never queued behind a whole unit of state MMAs
                if (c1.c == NC - 1 && c1.t == TP - 1 && have_next && gram_seq < c1.useq + 2) ready = false;
                if (__all_sync(0xffffffffu, ready)) {
                    tc_fence_after();
                    const int R = c1.x.npad;
                    const uint32_t acc = tmem_base + (c1.useq & 1) * kPairCols + c1.t * kAccCols;
                    if (lane == 0) {
                        const uint32_t sa = sbase + LY::OffRing + s * kSliceBytes;
                        const uint32_t ba = sbase + LY::OffB + (c1.cc & 1) * LY::BBUF;
                        const uint32_t id1 = make_idesc(2 * R);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_tf32(acc, make_desc(sa + k * 32), make_desc(ba + k * 32), id1, (c1.c | k) != 0);
                        mma_commit(bar(kP1Done + s));
                        if (c1.c == 1) {
                            // value term of this tile: V^T (128 values x R nodes, as landed) x M^T, three bf16 pieces
                            const uint32_t idv = make_idesc_bf16_amn(R);
                            const uint32_t vb = sbase + LY::OffV + c1.t * 2 * LY::VBLK, mb = sbase + LY::OffM;
                            for (int piece = 0; piece < 3; ++piece)
                                for (int ks = 0; ks < R / 16; ++ks)
                                    mma_bf16(acc, make_desc_mn(vb + ks * 2048, LY::VBLK),
                                             make_desc(mb + piece * LY::MPIECE + ks * 32), idv, 1);
                            if (c1.t == TP - 1) { mma_commit(bar(kVFree)); mma_commit(bar(kMFree)); }
                        }
                    }
                    __syncwarp();
                    const uint32_t was = c1.useq;
                    advance(c1);
                    if (c1.useq != was) {
                        nx = c1.x;
                        have_next = c1.have && next_unit(walk, nx);
                    }
                    prog = true;
                }
            }
            if (prog) {
                spin = 0; t0 = 0;
            } else {
                __nanosleep(20);
                if ((++spin & 255u) == 0u) {
                    if (__any_sync(0xffffffffu, *abort_flag != 0)) ok = false;
                    const uint64_t now = global_timer_ns();
                    if (t0 == 0) t0 = now;
                    if (__any_sync(0xffffffffu, now - t0 > kWaitLimitNs)) { *abort_flag = 1; ok = false; }
                }
            }
        }
        PROF_STORE()
        // everything this warp issued must have completed before TMEM is released
        if (lane == 0) mma_commit(bar(kDrain));
        __syncwarp();
        mbar_wait(bar(kDrain), 0, abort_flag);
    } else if (warp < 6) {
        // ------------------------------------------------------------- solver: Gram block -> records and M
        const int stid = threadIdx.x - 64;                       // 0..127
        const int grow = 32 * (warp & 3) + lane;                 // Gram row (= TMEM lane) of this thread
        const uint32_t lane_addr = uint32_t(32 * (warp & 3)) << 16;
        float *G = reinterpret_cast<float *>(smem + LY::OffTemp);   // whole Gram block, [column][128 rows]
        uint8_t *rec = smem + LY::OffRec;
        float *alpha_s = reinterpret_cast<float *>(smem + LY::OffAlpha);
        float *beta_s = alpha_s + 64;
        uint32_t ssync = 0, useq = 0;
        PROF_DECL
        auto solve_sync = [&]() -> bool {
            warp_arrive(bar(kSolveSync), lane);
            const bool r = WAIT(0, bar(kSolveSync), ssync & 1);
            ++ssync;
            return r;
        };
        // per-thread topology and gates of a unit, fetched one unit ahead
        int4 meta_n = make_int4(0, 0, 0, 0);
        int meta2_n = 0;
        float alpha_n = 0.f, beta_n = 0.f;
        auto fetch_topo = [&](const VUnit &y) {
            const int node = grow < y.npad ? grow : grow - y.npad;
            const bool act = grow < 2 * y.npad && node < y.n;
            meta_n = act ? __ldg(reinterpret_cast<const int4 *>(p.ws.anc) + y.base + node) : make_int4(0, 0, 0, 0);
            meta2_n = act ? __ldg(p.ws.anc2 + 4 * (y.base + node)) : 0;
            if (stid < y.n) {
                const int r = (y.l * p.T + y.base + stid) * p.H + y.h;
                alpha_n = __ldg(p.alpha + r);
                beta_n = __ldg(p.beta + r);
            }
        };
        VUnit x, nx;
        bool ok = true;
        bool have = first_unit(walk, x);
        if (have) fetch_topo(x);
        while (have && ok) {
            const int R = x.npad;
            const int4 meta = meta_n;
            const int meta2 = meta2_n;
            const float my_alpha = alpha_n, my_beta = beta_n;
            nx = x;
            const bool have_next = next_unit(walk, nx);
            if (have_next) fetch_topo(nx);
            // ancestors by level, one byte each
            const unsigned long long anc_lo = (unsigned long long)(uint32_t(meta.y)) | ((unsigned long long)(uint32_t(meta.z)) << 32);
            const unsigned long long anc_hi = (unsigned long long)(uint32_t(meta.w)) | ((unsigned long long)(uint32_t(meta2)) << 32);
            const bool is_k = grow < R;
            const int node = is_k ? grow : grow - R;
            const bool in_rows = grow < 2 * R;
            const bool active = in_rows && node < x.n;
            const int d = active ? (meta.x & 0xff) : 0;
            auto anc = [&](int j) -> int {
                const int a = int(((j < 8 ? anc_lo : anc_hi) >> (8 * (j & 7))) & 0xffull);
                return j < d - 1 ? a : node;
            };
            // The scratch below sits in the value-row buffer: the previous unit's value term must have read it.
            if (!(ok = WAIT(2, bar(kVFree), (useq & 1) ^ 1))) break;
            if (!(ok = WAIT(4, bar(kGramFull), useq & 1))) break;
            tc_fence_after();
            PROF_T0()
            {
                // whole Gram row of this thread -> G[column][row]
                const uint32_t gaddr = tmem_base + (useq & 1) * kPairCols + lane_addr;
#pragma unroll 1
                for (int c0 = 0; c0 < R; c0 += 16) {
                    float t8[8], u8[8];
                    tmem_ld8(gaddr + c0, t8);
                    tmem_ld8(gaddr + c0 + 8, u8);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 8; ++i) G[(c0 + i) * kRows + grow] = t8[i];
#pragma unroll
                    for (int i = 0; i < 8; ++i) G[(c0 + 8 + i) * kRows + grow] = u8[i];
                }
                tc_fence_before();
                warp_arrive(bar(kGramDone), lane);               // the state MMAs may now overwrite these columns
            }
            if (stid < x.n) { alpha_s[stid] = my_alpha; beta_s[stid] = my_beta; }
            PROF_ADD(1)
            if (!(ok = solve_sync())) break;                     // Gram block and gates visible

            // Row of X = (I + Ahat)^-1 (key rows, right-hand side e_t) or of C = Phat X (query rows, right-hand
            // side the row's own q.k entries) by back substitution along the path:
            //     c_j = rhs_j - sum_{m > j} c_m beta_{a_m} (k_{a_m} . k_{a_j}).
            float cf[kMaxD];
            {
                PROF_T0()
                if (active) {
#pragma unroll 1
                    for (int j = d - 1; j >= 0; --j) {
                        const int aj = anc(j);
                        float acc = is_k ? (j == d - 1 ? 1.f : 0.f) : G[aj * kRows + grow];
                        if (!p.no_erase) {
#pragma unroll 1
                            for (int m = j + 1; m < d; ++m) {
                                const int am = anc(m);
                                acc = fmaf(-cf[m] * beta_s[am], G[aj * kRows + am], acc);
                            }
                        }
                        cf[j] = acc;
                    }
                }
                PROF_ADD(7)
            }
            // record and M row of operand row `node`: query-row threads on the o walk, key-row threads on the u
            // walk.  The previous unit's effective vectors must have been formed, its value term issued.
            if (!(ok = WAIT(3, bar(kRecFree), (useq & 1) ^ 1))) break;
            if (!(ok = WAIT(5, bar(kMFree), (useq & 1) ^ 1))) break;
            const bool mine = in_rows && (x.kind == 0 ? !is_k : is_k);
            if (mine) {
                uint8_t *rr = rec + node * kRecBytes;
                uint8_t *mrow = smem + LY::OffM + (node >> 3) * 1024 + (node & 7) * 128;
#pragma unroll
                for (int pc = 0; pc < 3; ++pc)
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        *reinterpret_cast<uint4 *>(mrow + pc * LY::MPIECE + i * 16) = make_uint4(0u, 0u, 0u, 0u);
                int cnt = 0;
                if (active) {
                    float gamma = 1.f;
#pragma unroll 1
                    for (int j = 0; j < d; ++j) gamma *= alpha_s[anc(j)];
                    const float front = x.kind == 0 ? p.scale : 1.f;
                    float rho = 1.f;
#pragma unroll 1
                    for (int j = d - 1; j >= 0; --j) {
                        const int a = anc(j);
                        const float cb = cf[j] * beta_s[a];
                        // weight of k_a in the effective vector (zero without the erase term) ...
                        *reinterpret_cast<float *>(rr + kRecW + 4 * j) = p.no_erase ? 0.f : -front * gamma * cb;
                        *reinterpret_cast<unsigned short *>(rr + kRecOff + 2 * j) =
                            (unsigned short)((a >> 3) * 1024 + (a & 7) * 128);
                        // ... and of v_a in the value term, split into three bf16 pieces
                        float mv = front * rho * cb;
                        const uint32_t moff = uint32_t((((a >> 3) ^ (node & 7)) << 4) + (a & 7) * 2);
#pragma unroll
                        for (int pc = 0; pc < 3; ++pc) {
                            const __nv_bfloat16 bq = __float2bfloat16_rn(mv);
                            *reinterpret_cast<__nv_bfloat16 *>(mrow + pc * LY::MPIECE + moff) = bq;
                            mv -= __bfloat162float(bq);
                        }
                        rho *= alpha_s[a];
                    }
                    cnt = d;
                    if (x.kind == 0) {                           // the node's own query row
                        const int sr = R + node;
                        *reinterpret_cast<float *>(rr + kRecW + 4 * d) = p.scale * gamma;
                        *reinterpret_cast<unsigned short *>(rr + kRecOff + 2 * d) =
                            (unsigned short)((sr >> 3) * 1024 + (sr & 7) * 128);
                        cnt = d + 1;
                    }
                }
                *reinterpret_cast<int *>(rr) = cnt;
            }
            fence_proxy_async();
            warp_arrive(bar(kMReady), lane);
            warp_arrive(bar(kRecReady), lane);
            if (!(ok = solve_sync())) break;                     // nobody reads the Gram block any more
            if (stid == 0) {
                // value rows of this unit, as two 64-value blocks per tile, over the scratch
                const int m = (R >> 4) - 1;
                const int z = x.l * p.T + x.base;
                fence_proxy_async();
                mbar_arrive_expect_tx(bar(kVFull), uint32_t(TP * 2 * R * 128));
#pragma unroll
                for (int t = 0; t < TP; ++t)
#pragma unroll
                    for (int j = 0; j < 2; ++j)
                        tma_load_3d(sbase + LY::OffV + (t * 2 + j) * LY::VBLK, &maps.v[m], t * kRows + j * 64, x.h, z,
                                    bar(kVFull));
            }
            x = nx;
            have = have_next;
            ++useq;
        }
        PROF_STORE()
    } else if (warp < 10) {
        // ------------------------------------------------------------- effective vectors, one K-slice at a time
        const int vtid = threadIdx.x - 192;                      // 0..127
        const int cg = vtid & 3;                                 // 8-column group of the slice
        const uint8_t *rec = smem + LY::OffRec;
        uint32_t useq = 0, cc = 0, vsync = 0;
        PROF_DECL
        auto load_kq = [&](const VUnit &y, int par) {           // one thread
            const int m = (y.npad >> 4) - 1;
            const int z = y.l * p.T + y.base;
            const uint32_t stage = sbase + LY::OffStage + par * LY::STAGE;
            mbar_arrive_expect_tx(bar(kKQFull + par), uint32_t(4 * y.npad * DK));
#pragma unroll
            for (int c = 0; c < SC; ++c) {
                tma_load_3d(stage + c * SCB, &maps.k[m], c * 64, y.h, z, bar(kKQFull + par));
                tma_load_3d(stage + c * SCB + y.npad * 128, &maps.q[m], c * 64, y.h, z, bar(kKQFull + par));
            }
        };
        VUnit x, nx, nx2;
        bool ok = true;
        bool have = first_unit(walk, x);
        if (have && vtid == 0) {
            nx = x;
            load_kq(x, 0);
            if (next_unit(walk, nx)) load_kq(nx, 1);
        }
        while (have && ok) {
            const int par = useq & 1;
            const int R = x.npad;
            nx = x;
            const bool have_next = next_unit(walk, nx);
            nx2 = nx;
            const bool have_next2 = have_next && next_unit(walk, nx2);
            if (!(ok = WAIT(3, bar(kKQFull + par), (useq >> 1) & 1))) break;
            if (!(ok = WAIT(4, bar(kRecReady), useq & 1))) break;
            const uint8_t *stage = smem + LY::OffStage + par * LY::STAGE;
            for (int c = 0; c < NC; ++c, ++cc) {
                const int bb = cc & 1;
                if (!(ok = WAIT(6, bar(kBFree + bb), ((cc >> 1) & 1) ^ 1))) break;
                PROF_T0()
                const uint8_t *region = stage + (c >> 1) * SCB;
                const uint32_t slot = uint32_t((c & 1) * 4 + cg);
                uint8_t *bbuf = smem + LY::OffB + bb * LY::BBUF;
#pragma unroll 1
                for (int crow = vtid >> 2; crow < R; crow += 32) {
                    const uint8_t *rr = rec + crow * kRecBytes;
                    const int cnt = *reinterpret_cast<const int *>(rr);
                    float acc[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll 2
                    for (int j = 0; j < cnt; ++j) {
                        const float w = *reinterpret_cast<const float *>(rr + kRecW + 4 * j);
                        const uint32_t off = *reinterpret_cast<const unsigned short *>(rr + kRecOff + 2 * j);
                        const uint4 raw = *reinterpret_cast<const uint4 *>(region + off + ((slot ^ ((off >> 7) & 7u)) << 4));
                        acc[0] = fmaf(w, bf_lo(raw.x), acc[0]); acc[1] = fmaf(w, bf_hi(raw.x), acc[1]);
                        acc[2] = fmaf(w, bf_lo(raw.y), acc[2]); acc[3] = fmaf(w, bf_hi(raw.y), acc[3]);
                        acc[4] = fmaf(w, bf_lo(raw.z), acc[4]); acc[5] = fmaf(w, bf_hi(raw.z), acc[5]);
                        acc[6] = fmaf(w, bf_lo(raw.w), acc[6]); acc[7] = fmaf(w, bf_hi(raw.w), acc[7]);
                    }
                    float hi[8], lo[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) { hi[i] = round_tf32(acc[i]); lo[i] = acc[i] - hi[i]; }
                    const int r0 = crow, r1 = R + crow;
                    uint8_t *d0 = bbuf + (r0 >> 3) * 1024 + (r0 & 7) * 128;
                    uint8_t *d1 = bbuf + (r1 >> 3) * 1024 + (r1 & 7) * 128;
                    *reinterpret_cast<float4 *>(d0 + (((2 * cg) ^ (r0 & 7)) << 4)) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<float4 *>(d0 + (((2 * cg + 1) ^ (r0 & 7)) << 4)) = make_float4(hi[4], hi[5], hi[6], hi[7]);
                    *reinterpret_cast<float4 *>(d1 + (((2 * cg) ^ (r1 & 7)) << 4)) = make_float4(lo[0], lo[1], lo[2], lo[3]);
                    *reinterpret_cast<float4 *>(d1 + (((2 * cg + 1) ^ (r1 & 7)) << 4)) = make_float4(lo[4], lo[5], lo[6], lo[7]);
                }
                fence_proxy_async();
                warp_arrive(bar(kBReady + bb), lane);
                PROF_ADD(7)
            }
            if (!ok) break;
            warp_arrive(bar(kRecFree), lane);                    // the records of this unit are dead
            // every warp of the role has left the staged rows of this unit: request those of the unit after next
            warp_arrive(bar(kVecSync), lane);
            if (!(ok = WAIT(0, bar(kVecSync), vsync & 1))) break;
            ++vsync;
            if (vtid == 0 && have_next2) load_kq(nx2, par);
            x = nx;
            have = have_next;
            ++useq;
        }
        PROF_STORE()
    } else if (warp < 14) {
        // ------------------------------------------------------------- TF32 remainder of every slice, in place
        const int stid = threadIdx.x - 10 * 32;
        uint32_t it = 0;
        VUnit x;
        bool ok = true;
        PROF_DECL
        for (bool have = first_unit(walk, x); have && ok; have = next_unit(walk, x)) {
            for (int i = 0; i < TP * NC; ++i, ++it) {
                const int s = it % NS;
                const uint32_t ph = (it / NS) & 1;
                if (!(ok = WAIT(0, bar(kFull + s), ph))) break;
                if (!(ok = WAIT(1, bar(kP1Done + s), ph))) break;
                float4 *sl = reinterpret_cast<float4 *>(smem + LY::OffRing + s * kSliceBytes);
#pragma unroll
                for (int k = 0; k < kSliceBytes / 16 / kSplitThreads; ++k) {
                    float4 v = sl[stid + k * kSplitThreads];
                    v.x -= __uint_as_float(__float_as_uint(v.x) & 0xffffe000u);
                    v.y -= __uint_as_float(__float_as_uint(v.y) & 0xffffe000u);
                    v.z -= __uint_as_float(__float_as_uint(v.z) & 0xffffe000u);
                    v.w -= __uint_as_float(__float_as_uint(v.w) & 0xffffe000u);
                    sl[stid + k * kSplitThreads] = v;
                }
                fence_proxy_async();
                warp_arrive(bar(kLo + s), lane);
            }
        }
        PROF_STORE()
    } else {
        // ------------------------------------------------------------- epilogue
        const int row = 32 * (warp & 3) + lane;
        const uint32_t lane_addr = uint32_t(32 * (warp & 3)) << 16;
        uint32_t useq = 0;
        VUnit x;
        bool ok = true;
        PROF_DECL
        for (bool have = first_unit(walk, x); have && ok; have = next_unit(walk, x), ++useq) {
            const int pr = useq & 1;
            if (!(ok = WAIT(0, bar(kAccFull + pr), (useq >> 1) & 1))) break;
            tc_fence_after();
            const int R = x.npad, n = x.n;
            const size_t rec0 = size_t((x.l * p.T + x.base) * p.H + x.h);
            float *dst = (x.kind == 0 ? p.o : p.u) + rec0 * p.DV + row;
            const size_t stride = size_t(p.H) * p.DV;
#pragma unroll
            for (int t = 0; t < TP; ++t) {
                const uint32_t acc = tmem_base + pr * kPairCols + t * kAccCols + lane_addr;
#pragma unroll 1
                for (int j0 = 0; j0 < n; j0 += 8) {
                    float a[8], b[8];
                    tmem_ld8(acc + j0, a);
                    tmem_ld8(acc + R + j0, b);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (j0 + i < n) dst[(j0 + i) * stride + t * kRows] = a[i] + b[i];
                }
            }
            tc_fence_before();
            warp_arrive(bar(kPairFree + pr), lane);
        }
        PROF_STORE()
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, SPECA_STATUS_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

struct DeviceInfo { int sm_count; bool attr_set; };
DeviceInfo g_dev[64] = {};

}  // namespace

bool effective_supported(const speca_dims *d)
{
    if (d->d_k != 128 && d->d_k != 256) return false;
    if (d->d_v != kRows && d->d_v != 2 * kRows) return false;
    if (d->max_depth > kMaxD) return false;
    return d->max_nodes <= (d->d_k == 128 ? 64 : 32);
}

static int g_withhold_first_load = 0;
void effective_set_withhold(int on) { g_withhold_first_load = on; }

int launch_verify_effective(const Params &p, int d_k, cudaStream_t st)
{
    if (d_k != 128 && d_k != 256) return int(cudaErrorInvalidValue);
    EncodeTiledFn encode = encode_tiled_fn();
    if (encode == nullptr) return int(cudaErrorNotSupported);
    const long n_units = long(p.L) * p.B * p.H;
    const cuuint32_t es[3] = {1, 1, 1};
    CUtensorMap map;
    {
        const cuuint64_t gdim[3] = {cuuint64_t(d_k), cuuint64_t(p.DV), cuuint64_t(n_units)};
        const cuuint64_t gstride[2] = {cuuint64_t(d_k) * sizeof(float), cuuint64_t(p.DV) * d_k * sizeof(float)};
        const cuuint32_t box[3] = {32, kRows, 1};
        CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(p.S0), gdim, gstride, box, es,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return int(cudaErrorInvalidValue);
    }
    EMaps em;
    {
        const cuuint64_t gd[3] = {cuuint64_t(d_k), cuuint64_t(p.H), cuuint64_t(p.L) * cuuint64_t(p.T)};
        const cuuint64_t gs[2] = {cuuint64_t(d_k) * 2, cuuint64_t(p.H) * d_k * 2};
        const cuuint64_t vd[3] = {cuuint64_t(p.DV), cuuint64_t(p.H), cuuint64_t(p.L) * cuuint64_t(p.T)};
        const cuuint64_t vs[2] = {cuuint64_t(p.DV) * 2, cuuint64_t(p.H) * p.DV * 2};
        for (int m = 0; m < 4; ++m) {
            const cuuint32_t bx[3] = {64, 1, cuuint32_t(16 * (m + 1))};
            CUresult r1 = encode(&em.k[m], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16 *>(p.k), gd, gs, bx,
                                 es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            CUresult r2 = encode(&em.q[m], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16 *>(p.q), gd, gs, bx,
                                 es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            CUresult r3 = encode(&em.v[m], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16 *>(p.v), vd, vs, bx,
                                 es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r1 != CUDA_SUCCESS || r2 != CUDA_SUCCESS || r3 != CUDA_SUCCESS) return int(cudaErrorInvalidValue);
        }
    }

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return int(cudaErrorInvalidDevice);
    DeviceInfo &di = g_dev[dev];
    if (di.sm_count == 0) {
        int n = 0;
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        di.sm_count = n > 0 ? n : 148;
    }
    if (!di.attr_set) {
        cudaError_t e;
        e = cudaFuncSetAttribute(verify_effective_kernel<1, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<1, 128>::Bytes);
        if (e != cudaSuccess) return int(e);
        e = cudaFuncSetAttribute(verify_effective_kernel<2, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<2, 128>::Bytes);
        if (e != cudaSuccess) return int(e);
        e = cudaFuncSetAttribute(verify_effective_kernel<1, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<1, 256>::Bytes);
        if (e != cudaSuccess) return int(e);
        e = cudaFuncSetAttribute(verify_effective_kernel<2, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<2, 256>::Bytes);
        if (e != cudaSuccess) return int(e);
        di.attr_set = true;
    }
    EParams ep;
    ep.p = p;
    ep.n_units = n_units;
    ep.want_u = p.u != nullptr ? 1 : 0;
    ep.withhold_first_load = g_withhold_first_load;
    // consecutive heads of one (layer, sequence) a CTA takes together: as many as divide H while every SM still gets a group
    ep.heads_per_group = 1;
    for (int hg = 4; hg > 1; hg >>= 1)
        if (p.H % hg == 0 && n_units / hg >= di.sm_count) { ep.heads_per_group = hg; break; }
    const long n_groups = n_units / ep.heads_per_group;
    const int grid = int(n_groups < di.sm_count ? n_groups : di.sm_count);
    const bool one_tile = p.DV == kRows;
    if (d_k == 128) {
        if (one_tile) verify_effective_kernel<1, 128><<<grid, kThreads, Lay<1, 128>::Bytes, st>>>(map, em, ep);
        else verify_effective_kernel<2, 128><<<grid, kThreads, Lay<2, 128>::Bytes, st>>>(map, em, ep);
    } else {
        if (one_tile) verify_effective_kernel<1, 256><<<grid, kThreads, Lay<1, 256>::Bytes, st>>>(map, em, ep);
        else verify_effective_kernel<2, 256><<<grid, kThreads, Lay<2, 256>::Bytes, st>>>(map, em, ep);
    }
    return int(cudaGetLastError());
}

}  // namespace speca
