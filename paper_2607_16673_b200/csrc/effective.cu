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
// (W and Attn of the paper are these rows; the triangular solve is a back substitution along
// ancestor paths, at most 15 steps).  Everything that depends on the state is then one dense
// contraction of the state tile with N effective vectors, plus a small product with the value
// rows; the epilogue only adds two accumulator columns and stores.
//
// Accuracy.  The tensor core reads fp32 operands as TF32 (top 19 bits).  Both operands are
// therefore split: the state slice as landed (its TF32 head, free) and its exact remainder
// S - tf32(S), rewritten in place by a CUDA-core role once the first pass has read the slice;
// the effective vectors as a TF32-rounded head and the exact remainder.  First pass: S x head ->
// accumulator columns [0,R); correction passes: S x tail and then (S - tf32(S)) x head -> columns
// [R,2R).  The dropped term is 2^-22 of the result.  Mq / Mk are split into three bf16 pieces
// (24 bits) and multiply the bf16 value rows exactly.
//
// Mapping.  One persistent CTA per SM walks units (layer, sequence, head); 21 warps:
//   warp 0        TMA producer: per unit the K-slices of the fp32 state (128-byte swizzle), slice by slice
//                 over both value tiles, and, after the first slice pair, the unit's bf16 value rows --
//                 all through one ring of 16 KiB slots;
//   warps 1, 18   issue the first-pass tcgen05.mma of value tile 0 / 1 and the value-row product (an
//                 instruction costs its issuer about 130 cycles and a unit needs about a hundred of
//                 them, hence several issuers); warp 1 owns TMEM (two units of accumulators in flight)
//                 and issues the Gram blocks;
//   warps 19, 20  issue the correction passes of tile 0 / 1, each following two cursors (the tail
//                 operand, ready as soon as the slice has landed; the rewritten slice, ready once the
//                 split role is done with it) and releasing the ring slot;
//   warps 2-5     solver: ancestor entries of the Gram block out of TMEM, the two back substitutions,
//                 one record per operand row, the three bf16 pieces of M -- one unit ahead;
//   warps 6-9     effective vectors from the records and the staged bf16 keys / queries, one K-slice
//                 at a time into a ring of operand slices (so they never exist whole);
//   warps 10-13   rewrite each state slice as its TF32 remainder between the passes;
//   warps 14-17   epilogue: o (or u) = column t + column R + t, streamed out coalesced.
// Every visit of a ring slot, state slice or value rows, completes the same four barriers in the
// same order (landed, first pass read, rewritten, released), so that their phase parities stay in step.
// Nodes keep their index order everywhere.  When u is requested a unit is walked twice (first the
// o rows, then the u rows); the second walk finds the state tile in L2.  The order in which the
// passes reach an accumulator column is not fixed, so two runs may differ in the last bit.
// Every wait is bounded; on expiry the CTA raises SPECA_STATUS_TIMEOUT, drains and exits.
#include <cuda.h>

#include "speca_common.cuh"
#include "tc_ptx.cuh"

namespace speca {

namespace {

using namespace tc;

constexpr int kRows = 128;                      // value rows per tile (= TMEM lanes = MMA M)
constexpr int kSliceBytes = kRows * 128;        // one ring slot: a K-slice of a tile (128 rows x 32 fp32)
constexpr int kMaxD = 16;                       // tree depth taken
constexpr int kAccCols = 128;                   // accumulator columns per tile: [head R | tail R], R <= 64
constexpr int kPairCols = 2 * kAccCols;
constexpr int kTmemCols = 512;
constexpr int kThreads = 21 * 32;
constexpr int kRecBytes = 112;                  // per operand row: count, 17 weights, 17 staging offsets
constexpr int kRecW = 4, kRecOff = 72;
constexpr int kRecBuf = 64 * kRecBytes;
constexpr int kWalkSeqs = 128;
constexpr int kVBlock = 8192;                   // the two 64-value blocks of a staged value tile sit this far apart

// shared-memory carve-up per instantiation
template <int TP, int DK, int MAXN_> struct Lay {
    static constexpr int MAXN = MAXN_;                          // nodes per sequence
    static constexpr int NC = DK / 32;                          // K-slices per tile
    static constexpr int SC = DK / 64;                          // 64-column regions of the staged bf16 rows
    static constexpr int SCB = 2 * MAXN * 128;                  // bytes per region: key rows, then query rows
    static constexpr int STAGE = SC * SCB;
    static constexpr int BBUF = 2 * MAXN * 128;                 // one K-slice of the operand: head rows, tail rows
    static constexpr int MPIECE = MAXN * 128;                   // one bf16 piece of M: R rows x 64 columns
    static constexpr int GS = kMaxD * kRows * 4;                // Gram entries of every row against its own path
    static constexpr int NB = MAXN > 32 ? 3 : 4;                // operand slices in flight
    static constexpr int kFixed = NB * BBUF + 2 * STAGE + 3 * MPIECE + GS + 2 * kRecBuf + 2 * 64 * 4 + 512 + 128 +
                                  5 * kWalkSeqs;
    static constexpr int kRoom = (227 * 1024 - kFixed - 1024) / kSliceBytes;
    static constexpr int NS = kRoom > 8 ? 8 : kRoom;            // ring depth
    static constexpr int OffRing = 0;
    static constexpr int OffB = OffRing + NS * kSliceBytes;
    static constexpr int OffStage = OffB + NB * BBUF;
    static constexpr int OffM = OffStage + 2 * STAGE;
    static constexpr int OffGs = OffM + 3 * MPIECE;
    static constexpr int OffRec = OffGs + GS;
    static constexpr int OffAlpha = OffRec + 2 * kRecBuf;
    static constexpr int OffBars = OffAlpha + 2 * 64 * 4;
    static constexpr int OffMisc = OffBars + 512;               // abort flag, TMEM base, node depths
    static constexpr int OffWalk = OffMisc + 128;
    static constexpr int Bytes = OffWalk + 5 * kWalkSeqs;
    static_assert(NS >= 4, "ring too shallow");
    static_assert(Bytes <= 227 * 1024, "shared memory budget");
};

constexpr int kMaxSlots = 8;
enum Bar {
    kFull = 0,                         // [8] TMA -> MMA (and split): slot landed
    kEmpty = kFull + kMaxSlots,        // [8] MMA -> TMA: slot no longer read
    kP1Done = kEmpty + kMaxSlots,      // [8] MMA -> split: first pass has read the slice
    kLo = kP1Done + kMaxSlots,         // [8] split -> MMA: slice rewritten as its remainder
    kKQFull = kLo + kMaxSlots,         // [2] TMA -> MMA, vector warps: staged bf16 key / query rows of a unit
    kGramFull = kKQFull + 2,           // MMA -> solver: Gram block in TMEM
    kGramDone,                         // solver -> MMA: Gram rows read, the columns may be overwritten
    kBReady,                           // [4] vector warps -> MMA: operand slice written
    kBFree = kBReady + 4,              // [4] MMA -> vector warps: operand slice no longer read
    kMReady = kBFree + 4,              // solver -> MMA: pieces of M written
    kMFree,                            // MMA -> solver: value term issued and done
    kAccFull,                          // [2] MMA -> epilogue
    kPairFree = kAccFull + 2,          // [2] epilogue -> MMA
    kRecReady = kPairFree + 2,         // [2] solver -> vector warps: records of a unit written
    kRecFree = kRecReady + 2,          // [2] vector warps -> solver
    kSolveSync = kRecFree + 2,         // role-internal
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

// one arrival for the whole warp: every lane's earlier writes are ordered before it
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane)
{
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
}

__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
// what the tensor core's TF32 reading of x (low 13 mantissa bits dropped) leaves out; exact
__device__ __forceinline__ float tf32_rest(float x) { return x - __uint_as_float(__float_as_uint(x) & 0xffffe000u); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&r)[16])
{
    uint32_t x[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3]), "=r"(x[4]), "=r"(x[5]), "=r"(x[6]), "=r"(x[7]),
                   "=r"(x[8]), "=r"(x[9]), "=r"(x[10]), "=r"(x[11]), "=r"(x[12]), "=r"(x[13]), "=r"(x[14]), "=r"(x[15])
                 : "r"(taddr)
                 : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) r[i] = __uint_as_float(x[i]);
}

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
//
// Ring entries of a unit, in order: slices (c = 0; t = 0 .. TP-1), value tiles (t = 0 .. TP-1), then slices
// (c = 1 .. NC-1; t).  For tile t the q-th entry (q = 0: slice 0, q = 1: value tile, q >= 2: slice q - 1) is
// entry q * TP + t of the unit.
template <int TP, int DK, int MAXN>
__global__ void __launch_bounds__(kThreads, 1)
verify_effective_kernel(const __grid_constant__ CUtensorMap s0_map, const __grid_constant__ EMaps maps, EParams ep)
{
    using LY = Lay<TP, DK, MAXN>;
    constexpr int NS = LY::NS, NC = LY::NC, SC = LY::SC, SCB = LY::SCB, NB = LY::NB;
    constexpr int NQ = NC + 1;                                    // ring entries per tile and unit
    constexpr int NE = TP * NQ;                                   // ring entries per unit
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
    uint8_t *depth_s = smem + LY::OffMisc + 64;          // depth of every node of the unit in the solver's hands
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kMaxSlots; ++s) {
            mbar_init(bar(kFull + s), 1);
            mbar_init(bar(kEmpty + s), 1);
            mbar_init(bar(kP1Done + s), 2);
            mbar_init(bar(kLo + s), 4);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(kKQFull + i), 1);
            mbar_init(bar(kAccFull + i), TP);
            mbar_init(bar(kPairFree + i), 4);
            mbar_init(bar(kRecReady + i), 4);
            mbar_init(bar(kRecFree + i), 4);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(bar(kBReady + i), 4);
            mbar_init(bar(kBFree + i), TP);
        }
        mbar_init(bar(kGramFull), 1);
        mbar_init(bar(kGramDone), 4);
        mbar_init(bar(kMReady), 4);
        mbar_init(bar(kMFree), TP);
        mbar_init(bar(kSolveSync), 4);
        mbar_init(bar(kVecSync), 4);
        mbar_init(bar(kDrain), 2 * TP);
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
        // ------------------------------------------------------------- TMA producer
        uint32_t it = 0;
        VUnit x;
        bool ok = true;
        PROF_DECL
        for (bool have = first_unit(walk, x); have && ok; have = next_unit(walk, x)) {
            for (int e = 0; e < NE; ++e, ++it) {
                const int s = it % NS;
                if (!(ok = WAIT(0, bar(kEmpty + s), ((it / NS) & 1) ^ 1))) break;
                const uint32_t dst = sbase + LY::OffRing + s * kSliceBytes;
                if (lane == 0 && !(ep.withhold_first_load && blockIdx.x == 0 && it == 0)) {
                    if (e >= TP && e < 2 * TP) {
                        // value rows of tile t: two blocks of 64 values, nodes down the rows
                        const int t = e - TP;
                        mbar_arrive_expect_tx(bar(kFull + s), uint32_t(2 * x.npad * 128));
                        const CUtensorMap *vm = &maps.v[(x.npad >> 4) - 1];
                        tma_load_3d(dst, vm, t * kRows, x.h, x.l * p.T + x.base, bar(kFull + s));
                        tma_load_3d(dst + kVBlock, vm, t * kRows + 64, x.h, x.l * p.T + x.base, bar(kFull + s));
                    } else {
                        const int c = e < TP ? 0 : (e - TP) / TP, t = e % TP;
                        mbar_arrive_expect_tx(bar(kFull + s), kSliceBytes);
                        tma_load_3d(dst, &s0_map, c * 32, t * kRows, x.u, bar(kFull + s));
                    }
                }
                __syncwarp();
            }
        }
        PROF_STORE()
        // let copies still in flight land before the CTA's shared memory goes away
        if (*abort_flag) {
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
    } else if (warp == 1 || warp == 18) {
        // ------------------------------------------------------------- first-pass MMA issuers, one warp per value tile
        // Issuing a tcgen05 instruction costs its thread on the order of a hundred cycles and a unit needs about
        // a hundred of them, so the work is spread over four warps that never wait for one another and write
        // disjoint accumulator columns: per tile, this warp issues S x head -> columns [0,R) (kind::tf32, the
        // slice as landed) and the value term, the second-pass warp the two correction products -> [R,2R).
        // Warp 1 also issues the Gram blocks.
        const int mt = warp == 1 ? 0 : 1;                        // tile of this warp
        bool ok = mt < TP;
        PROF_DECL
        // Gram block of a unit: [K;Q] (128 rows) x K^T (npad columns) from the staged bf16 rows, parked in the
        // unit's own accumulator columns (tile 0) until its state MMAs overwrite them.
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
        auto gram_ready = [&](uint32_t seq) -> bool {
            const int pr = seq & 1;
            const bool a = mbar_test_wait(bar(kKQFull + pr), (seq >> 1) & 1);
            const bool b = mbar_test_wait(bar(kPairFree + pr), ((seq >> 1) & 1) ^ 1);
            return __all_sync(0xffffffffu, a && b);
        };
        auto gram_wait = [&](uint32_t seq) -> bool {
            const int pr = seq & 1;
            return WAIT(5, bar(kKQFull + pr), (seq >> 1) & 1) && WAIT(6, bar(kPairFree + pr), ((seq >> 1) & 1) ^ 1);
        };
        VUnit x, nx;
        uint32_t useq = 0, gram_seq = 0;
        bool have = ok && first_unit(walk, x);
        while (have && ok) {
            nx = x;
            const bool have_next = next_unit(walk, nx);
            const int R = x.npad;
            const uint32_t acc = tmem_base + (useq & 1) * kPairCols + mt * kAccCols;
            const uint32_t id1 = make_idesc(R);
            if (mt == 0 && gram_seq == useq) {                   // first unit only: later ones are issued ahead
                if (!(ok = gram_wait(gram_seq))) break;
                issue_gram(gram_seq, R);
                ++gram_seq;
            }
            for (int q = 0; q < NQ && ok; ++q) {
                const uint32_t it = useq * NE + q * TP + mt;
                const int s = it % NS;
                const uint32_t ph = (it / NS) & 1;
                const uint32_t sa = sbase + LY::OffRing + s * kSliceBytes;
                if (mt == 0 && have_next && gram_seq == useq + 1 && q > 0) {
                    // the next unit's Gram block: as soon as its rows are staged and its accumulators released, at
                    // the latest before this unit's last slice, so that the preparation of that unit is never
                    // queued behind a whole unit of state MMAs
                    if (q == NQ - 1) {
                        if (!(ok = gram_wait(gram_seq))) break;
                        issue_gram(gram_seq, nx.npad);
                        ++gram_seq;
                    } else if (gram_ready(gram_seq)) {
                        issue_gram(gram_seq, nx.npad);
                        ++gram_seq;
                    }
                }
                if (q == 1) {
                    // value term: V^T (128 values x R nodes, as landed) x M^T, three bf16 pieces
                    if (!(ok = WAIT(1, bar(kMReady), useq & 1))) break;
                    if (!(ok = WAIT(0, bar(kFull + s), ph))) break;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t idv = make_idesc_bf16_amn(R);
                        const uint32_t mb = sbase + LY::OffM;
                        for (int piece = 0; piece < 3; ++piece)
                            for (int ks = 0; ks < R / 16; ++ks)
                                mma_bf16(acc, make_desc_mn(sa + ks * 2048, kVBlock),
                                         make_desc(mb + piece * LY::MPIECE + ks * 32), idv, 1);
                        // every slot visit completes each of its four barriers once, in the same order as for a
                        // slice (a slot must not come round again before every waiter has seen this visit)
                        mma_commit(bar(kP1Done + s));
                        mma_commit(bar(kP1Done + s));
                        mma_commit(bar(kMFree));
                    }
                    __syncwarp();
                } else {
                    const int c = q == 0 ? 0 : q - 1;
                    const uint32_t cc = useq * NC + c;
                    if (q == 0) {
                        // the accumulator pair must be released by the epilogue, and the Gram block parked in it read
                        if (!(ok = WAIT(2, bar(kPairFree + (useq & 1)), ((useq >> 1) & 1) ^ 1))) break;
                        // (tile 0 only: that is where it is parked, and only this warp keeps step with the solver)
                        if (mt == 0 && !(ok = WAIT(3, bar(kGramDone), useq & 1))) break;
                    }
                    if (!(ok = WAIT(4, bar(kBReady + (cc % NB)), (cc / NB) & 1))) break;
                    if (!(ok = WAIT(0, bar(kFull + s), ph))) break;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t ba = sbase + LY::OffB + (cc % NB) * LY::BBUF;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_tf32(acc, make_desc(sa + k * 32), make_desc(ba + k * 32), id1, (c | k) != 0);
                        mma_commit(bar(kP1Done + s));
                    }
                    __syncwarp();
                }
            }
            x = nx;
            have = have_next;
            ++useq;
        }
        PROF_STORE()
        // everything this warp issued must have completed before TMEM is released
        if (mt < TP) {
            if (lane == 0) mma_commit(bar(kDrain));
            __syncwarp();
            mbar_wait(bar(kDrain), 0, abort_flag);
        }
    } else if (warp == 19 || warp == 20) {
        // ------------------------------------------------------------- correction MMA issuers, one warp per value tile
        // Columns [R,2R) collect the two small products: S x tail while the slice is as landed, then
        // (S - tf32(S)) x head once it has been rewritten in place.  Two cursors over the tile's slices: whichever
        // product is ready is issued, so the rewrite of one slice is never waited for while another can go.
        const int mt = warp - 19;
        bool ok = mt < TP;
        PROF_DECL
        struct Cur { VUnit x; uint32_t useq; int q; bool have; };
        auto advance = [&](Cur &c, bool skip_values) {
            if (++c.q == 1 && skip_values) ++c.q;                // value tiles have no product for this warp
            if (c.q == NQ) { c.q = 0; ++c.useq; c.have = next_unit(walk, c.x); }
        };
        Cur f, g;
        f.useq = 0; f.q = 0;
        f.have = ok && first_unit(walk, f.x);
        g = f;
        uint64_t t0 = 0;
        uint32_t spin = 0;
        while (ok && (f.have || g.useq * NQ + g.q < f.useq * NQ + f.q)) {
            bool prog = false;
            if (g.useq * NQ + g.q < f.useq * NQ + f.q) {
                const uint32_t it = g.useq * NE + g.q * TP + mt;
                const int s = it % NS;
                if (__all_sync(0xffffffffu, mbar_test_wait(bar(kLo + s), (it / NS) & 1))) {
                    const int c = g.q == 0 ? 0 : g.q - 1;
                    const uint32_t cc = g.useq * NC + c;
                    tc_fence_after();
                    if (g.q == 1) {
                        // a value tile: its term has completed (the split warps saw that) and every waiter has seen
                        // this visit of the slot, so it may come round again
                        if (lane == 0) mbar_arrive(bar(kEmpty + s));
                    } else if (lane == 0) {
                        const int R = g.x.npad;
                        const uint32_t acc = tmem_base + (g.useq & 1) * kPairCols + mt * kAccCols + R;
                        const uint32_t sa = sbase + LY::OffRing + s * kSliceBytes;
                        const uint32_t ba = sbase + LY::OffB + (cc % NB) * LY::BBUF;
                        const uint32_t idc = make_idesc(R);
#pragma unroll
                        for (int k = 0; k < 4; ++k) mma_tf32(acc, make_desc(sa + k * 32), make_desc(ba + k * 32), idc, 1);
                        mma_commit(bar(kEmpty + s));
                        mma_commit(bar(kBFree + (cc % NB)));
                        if (c == NC - 1) mma_commit(bar(kAccFull + (g.useq & 1)));
                    }
                    __syncwarp();
                    advance(g, false);
                    prog = true;
                }
            }
            if (f.have) {
                const uint32_t it = f.useq * NE + f.q * TP + mt;
                const int s = it % NS;
                const int c = f.q == 0 ? 0 : f.q - 1;
                const uint32_t cc = f.useq * NC + c;
                const bool r0 = mbar_test_wait(bar(kFull + s), (it / NS) & 1);
                const bool r1 = mbar_test_wait(bar(kBReady + (cc % NB)), (cc / NB) & 1);
                // first slice of a unit: the accumulator pair must be released by the epilogue
                const bool r2 = f.q != 0 || mbar_test_wait(bar(kPairFree + (f.useq & 1)), ((f.useq >> 1) & 1) ^ 1);
                if (__all_sync(0xffffffffu, r0 && r1 && r2)) {
                    tc_fence_after();
                    if (lane == 0) {
                        const int R = f.x.npad;
                        const uint32_t acc = tmem_base + (f.useq & 1) * kPairCols + mt * kAccCols + R;
                        const uint32_t sa = sbase + LY::OffRing + s * kSliceBytes;
                        const uint32_t ba = sbase + LY::OffB + (cc % NB) * LY::BBUF + LY::MAXN * 128;
                        const uint32_t idc = make_idesc(R);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_tf32(acc, make_desc(sa + k * 32), make_desc(ba + k * 32), idc, (c | k) != 0);
                        mma_commit(bar(kP1Done + s));
                    }
                    __syncwarp();
                    advance(f, true);
                    prog = true;
                }
            }
            if (prog) {
                spin = 0; t0 = 0;
            } else {
                // nothing to issue: sleep (up to 400 ns) on the barrier that is due next
                if (g.useq * NQ + g.q < f.useq * NQ + f.q) {
                    const uint32_t it = g.useq * NE + g.q * TP + mt;
                    mbar_try_wait_for(bar(kLo + it % NS), (it / NS) & 1, 400);
                } else if (f.have) {
                    const uint32_t it = f.useq * NE + f.q * TP + mt;
                    mbar_try_wait_for(bar(kFull + it % NS), (it / NS) & 1, 400);
                }
                if ((++spin & 255u) == 0u) {
                    if (__any_sync(0xffffffffu, *abort_flag != 0)) ok = false;
                    const uint64_t now = global_timer_ns();
                    if (t0 == 0) t0 = now;
                    if (__any_sync(0xffffffffu, now - t0 > kWaitLimitNs)) { *abort_flag = 1; ok = false; }
                }
            }
        }
        PROF_STORE()
        if (mt < TP) {
            if (lane == 0) mma_commit(bar(kDrain));
            __syncwarp();
            mbar_wait(bar(kDrain), 0, abort_flag);
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------- solver: Gram block -> records and M
        const int stid = threadIdx.x - 64;                       // 0..127
        const int grow = 32 * (warp & 3) + lane;                 // Gram row (= TMEM lane) of this thread
        const uint32_t lane_addr = uint32_t(32 * (warp & 3)) << 16;
        float *Gs = reinterpret_cast<float *>(smem + LY::OffGs);    // [level][128 rows]: (row) . k_{a_level}
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
            const int par = useq & 1;
            const int R = x.npad;
            const int4 meta = meta_n;
            const int meta2 = meta2_n;
            const float my_alpha = alpha_n, my_beta = beta_n;
            nx = x;
            const bool have_next = next_unit(walk, nx);
            if (have_next) fetch_topo(nx);
            // ancestors by level, one byte each; the nodes of the path as a bit set
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
            unsigned long long path = 0ull;
#pragma unroll 1
            for (int j = 0; j < d; ++j) path |= 1ull << anc(j);
            // gates and depths of this unit's nodes (the previous unit's readers are behind the last sync)
            if (stid < x.n) { alpha_s[stid] = my_alpha; beta_s[stid] = my_beta; }
            if (is_k && active) depth_s[node] = uint8_t(d);
            if (!(ok = solve_sync())) break;
            if (!(ok = WAIT(4, bar(kGramFull), useq & 1))) break;
            tc_fence_after();
            {
                PROF_T0()
                // Gram row of this thread, 16 columns at a time: keep the entries against the nodes of its own
                // path, filed by the level of that node
                const uint32_t gaddr = tmem_base + par * kPairCols + lane_addr;
#pragma unroll 1
                for (int c0 = 0; c0 < R; c0 += 16) {
                    float g16[16];
                    tmem_ld16(gaddr + c0, g16);
                    const uint4 dep = *reinterpret_cast<const uint4 *>(depth_s + c0);
                    tmem_ld_wait();
                    const uint32_t dw[4] = {dep.x, dep.y, dep.z, dep.w};
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int lev = int((dw[i >> 2] >> (8 * (i & 3))) & 0xffu) - 1;
                        if ((path >> (c0 + i)) & 1ull) Gs[lev * kRows + grow] = g16[i];
                    }
                }
                tc_fence_before();
                warp_arrive(bar(kGramDone), lane);               // the state MMAs may now overwrite these columns
                PROF_ADD(1)
            }
            if (!(ok = solve_sync())) break;                     // every row's entries visible

            // Row of X = (I + Ahat)^-1 (key rows, right-hand side e_t) or of C = Phat X (query rows, right-hand
            // side the row's own q.k entries) by back substitution along the path:
            //     c_j = rhs_j - sum_{m > j} c_m beta_{a_m} (k_{a_m} . k_{a_j}).
            // Then the record of operand row `node` (query-row threads on the o walk, key-row threads on the u
            // walk): weight of k_{a_j} in the effective vector, -front gamma c_j beta_{a_j} (zero without the erase
            // term), and the row of M: weight of v_{a_j} in the value term, front rho_j c_j beta_{a_j}, as three bf16
            // pieces.
            const bool mine = in_rows && (x.kind == 0 ? !is_k : is_k);
            const float front = x.kind == 0 ? p.scale : 1.f;
            uint8_t *rr = smem + LY::OffRec + par * kRecBuf + node * kRecBytes;
            uint8_t *mrow = smem + LY::OffM + (node >> 3) * 1024 + (node & 7) * 128;
            auto zero_mrow = [&]() {
#pragma unroll
                for (int pc = 0; pc < 3; ++pc)
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        *reinterpret_cast<uint4 *>(mrow + pc * LY::MPIECE + i * 16) = make_uint4(0u, 0u, 0u, 0u);
            };
            auto put_m = [&](int a, float mv) {
                const uint32_t moff = uint32_t((((a >> 3) ^ (node & 7)) << 4) + (a & 7) * 2);
#pragma unroll
                for (int pc = 0; pc < 3; ++pc) {
                    const __nv_bfloat16 bq = __float2bfloat16_rn(mv);
                    *reinterpret_cast<__nv_bfloat16 *>(mrow + pc * LY::MPIECE + moff) = bq;
                    mv -= __bfloat162float(bq);
                }
            };
            auto put_rec = [&](int j, int a, float w) {
                *reinterpret_cast<float *>(rr + kRecW + 4 * j) = w;
                *reinterpret_cast<unsigned short *>(rr + kRecOff + 2 * j) = (unsigned short)((a >> 3) * 1024 + (a & 7) * 128);
            };
            float cf[kMaxD];
            {
                PROF_T0()
                if (active) {
#pragma unroll 1
                    for (int j = d - 1; j >= 0; --j) {
                        float acc = is_k ? (j == d - 1 ? 1.f : 0.f) : Gs[j * kRows + grow];
                        if (!p.no_erase) {
#pragma unroll 1
                            for (int m = j + 1; m < d; ++m) {
                                const int am = anc(m);
                                acc = fmaf(-cf[m] * beta_s[am], Gs[j * kRows + am], acc);
                            }
                        }
                        cf[j] = acc;
                    }
                }
                PROF_ADD(7)
            }
            if (!(ok = WAIT(3, bar(kRecFree + par), ((useq >> 1) & 1) ^ 1))) break;
            float gamma = 1.f;
            if (mine) {
                int cnt = 0;
                if (active) {
#pragma unroll 1
                    for (int j = 0; j < d; ++j) gamma *= alpha_s[anc(j)];
#pragma unroll 1
                    for (int j = 0; j < d; ++j) {
                        const int a = anc(j);
                        put_rec(j, a, p.no_erase ? 0.f : -front * gamma * cf[j] * beta_s[a]);
                    }
                    cnt = d;
                    if (x.kind == 0) { put_rec(d, R + node, p.scale * gamma); cnt = d + 1; }
                }
                *reinterpret_cast<int *>(rr) = cnt;
            }
            warp_arrive(bar(kRecReady + par), lane);
            if (!(ok = WAIT(5, bar(kMFree), (useq & 1) ^ 1))) break;
            if (mine) {
                zero_mrow();
                if (active) {
                    float rho = 1.f;
#pragma unroll 1
                    for (int j = d - 1; j >= 0; --j) {
                        const int a = anc(j);
                        put_m(a, front * rho * cf[j] * beta_s[a]);
                        rho *= alpha_s[a];
                    }
                }
            }
            fence_proxy_async();
            warp_arrive(bar(kMReady), lane);
            if (!(ok = solve_sync())) break;                     // gates, depths and Gram entries of this unit are dead
            x = nx;
            have = have_next;
            ++useq;
        }
        PROF_STORE()
    } else if (warp < 10) {
        // ------------------------------------------------------------- effective vectors, one K-slice at a time
        const int vtid = threadIdx.x - 192;                      // 0..127
        const int cg = vtid & 3;                                 // 8-column group of the slice
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
        const bool shallow = p.max_depth <= 8;                  // at most 9 terms per row: fully unrolled form
        while (have && ok) {
            const int par = useq & 1;
            const int R = x.npad;
            nx = x;
            const bool have_next = next_unit(walk, nx);
            nx2 = nx;
            const bool have_next2 = have_next && next_unit(walk, nx2);
            if (!(ok = WAIT(3, bar(kKQFull + par), (useq >> 1) & 1))) break;
            if (!(ok = WAIT(4, bar(kRecReady + par), (useq >> 1) & 1))) break;
            const uint8_t *stage = smem + LY::OffStage + par * LY::STAGE;
            const uint8_t *rec = smem + LY::OffRec + par * kRecBuf;
            for (int c = 0; c < NC; ++c, ++cc) {
                const int bb = cc % NB;
                if (!(ok = WAIT(6, bar(kBFree + bb), ((cc / NB) & 1) ^ 1))) break;
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
                    auto term = [&](float w, uint32_t off) {
                        const uint4 raw = *reinterpret_cast<const uint4 *>(region + off + ((slot ^ ((off >> 7) & 7u)) << 4));
                        acc[0] = fmaf(w, bf_lo(raw.x), acc[0]); acc[1] = fmaf(w, bf_hi(raw.x), acc[1]);
                        acc[2] = fmaf(w, bf_lo(raw.y), acc[2]); acc[3] = fmaf(w, bf_hi(raw.y), acc[3]);
                        acc[4] = fmaf(w, bf_lo(raw.z), acc[4]); acc[5] = fmaf(w, bf_hi(raw.z), acc[5]);
                        acc[6] = fmaf(w, bf_lo(raw.w), acc[6]); acc[7] = fmaf(w, bf_hi(raw.w), acc[7]);
                    };
                    if (shallow) {
                        // all nine loads in flight at once; terms past the end of the record weigh nothing
#pragma unroll
                        for (int j = 0; j < 9; ++j) {
                            const float w = j < cnt ? *reinterpret_cast<const float *>(rr + kRecW + 4 * j) : 0.f;
                            const uint32_t off = j < cnt ? *reinterpret_cast<const unsigned short *>(rr + kRecOff + 2 * j) : 0u;
                            term(w, off);
                        }
                    } else {
#pragma unroll 2
                        for (int j = 0; j < cnt; ++j)
                            term(*reinterpret_cast<const float *>(rr + kRecW + 4 * j),
                                 *reinterpret_cast<const unsigned short *>(rr + kRecOff + 2 * j));
                    }
                    // head (TF32-rounded) and exact tail, one fp32 row each
                    float hi[8], lo[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) { hi[i] = round_tf32(acc[i]); lo[i] = acc[i] - hi[i]; }
                    const uint32_t sw = uint32_t(crow & 7);
                    uint8_t *d0 = bbuf + (crow >> 3) * 1024 + (crow & 7) * 128;
                    uint8_t *d1 = d0 + LY::MAXN * 128;
                    *reinterpret_cast<float4 *>(d0 + (((2 * cg) ^ sw) << 4)) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<float4 *>(d0 + (((2 * cg + 1) ^ sw) << 4)) = make_float4(hi[4], hi[5], hi[6], hi[7]);
                    *reinterpret_cast<float4 *>(d1 + (((2 * cg) ^ sw) << 4)) = make_float4(lo[0], lo[1], lo[2], lo[3]);
                    *reinterpret_cast<float4 *>(d1 + (((2 * cg + 1) ^ sw) << 4)) = make_float4(lo[4], lo[5], lo[6], lo[7]);
                }
                fence_proxy_async();
                warp_arrive(bar(kBReady + bb), lane);
                PROF_ADD(7)
            }
            if (!ok) break;
            warp_arrive(bar(kRecFree + par), lane);              // the records of this unit are dead
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
            for (int e = 0; e < NE; ++e, ++it) {
                const int s = it % NS;
                const uint32_t ph = (it / NS) & 1;
                if (!(ok = WAIT(0, bar(kFull + s), ph))) break;
                if (e >= TP && e < 2 * TP) {                     // value tiles are not split
                    if (!(ok = WAIT(1, bar(kP1Done + s), ph))) break;
                    warp_arrive(bar(kLo + s), lane);
                    continue;
                }
                // the remainders are formed while the first products are still reading the slice; only the stores wait
                float4 *sl = reinterpret_cast<float4 *>(smem + LY::OffRing + s * kSliceBytes);
                float4 v[kSliceBytes / 16 / 128];
#pragma unroll
                for (int k = 0; k < kSliceBytes / 16 / 128; ++k) {
                    v[k] = sl[stid + k * 128];
                    v[k].x = tf32_rest(v[k].x); v[k].y = tf32_rest(v[k].y); v[k].z = tf32_rest(v[k].z); v[k].w = tf32_rest(v[k].w);
                }
                if (!(ok = WAIT(1, bar(kP1Done + s), ph))) break;
#pragma unroll
                for (int k = 0; k < kSliceBytes / 16 / 128; ++k) sl[stid + k * 128] = v[k];
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
        cudaError_t e = cudaSuccess;
        auto opt_in = [&](const void *k, int bytes) {
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        };
        opt_in(reinterpret_cast<const void *>(verify_effective_kernel<1, 128, 64>), Lay<1, 128, 64>::Bytes);
        opt_in(reinterpret_cast<const void *>(verify_effective_kernel<2, 128, 64>), Lay<2, 128, 64>::Bytes);
        opt_in(reinterpret_cast<const void *>(verify_effective_kernel<1, 128, 32>), Lay<1, 128, 32>::Bytes);
        opt_in(reinterpret_cast<const void *>(verify_effective_kernel<2, 128, 32>), Lay<2, 128, 32>::Bytes);
        opt_in(reinterpret_cast<const void *>(verify_effective_kernel<1, 256, 32>), Lay<1, 256, 32>::Bytes);
        opt_in(reinterpret_cast<const void *>(verify_effective_kernel<2, 256, 32>), Lay<2, 256, 32>::Bytes);
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
    // a smaller node budget leaves room for a deeper ring of state slices
    if (d_k == 128 && p.max_nodes > 32) {
        if (one_tile) verify_effective_kernel<1, 128, 64><<<grid, kThreads, Lay<1, 128, 64>::Bytes, st>>>(map, em, ep);
        else verify_effective_kernel<2, 128, 64><<<grid, kThreads, Lay<2, 128, 64>::Bytes, st>>>(map, em, ep);
    } else if (d_k == 128) {
        if (one_tile) verify_effective_kernel<1, 128, 32><<<grid, kThreads, Lay<1, 128, 32>::Bytes, st>>>(map, em, ep);
        else verify_effective_kernel<2, 128, 32><<<grid, kThreads, Lay<2, 128, 32>::Bytes, st>>>(map, em, ep);
    } else {
        if (one_tile) verify_effective_kernel<1, 256, 32><<<grid, kThreads, Lay<1, 256, 32>::Bytes, st>>>(map, em, ep);
        else verify_effective_kernel<2, 256, 32><<<grid, kThreads, Lay<2, 256, 32>::Bytes, st>>>(map, em, ep);
    }
    return int(cudaGetLastError());
}

}  // namespace speca
