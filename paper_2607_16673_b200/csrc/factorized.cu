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
//   * the same [K;Q] block times K^T gives every q.k and k.k the coefficients need; that
//     Gram block borrows the unit's own accumulator columns before the state MMAs start;
//   * an epilogue thread owns one value row of EACH tile of the unit (same TMEM lane), so the
//     per-node coefficients are fetched from shared memory once per two rows; it keeps the u
//     of the current depth-first path in registers (a stack indexed by depth) and streams o
//     out coalesced.
// Roles: warp 0 TMA producer, warp 1 MMA issuer + TMEM owner, warps 2-5 operand/coefficient
// preparation, warps 6-9 and 10-13 two epilogue groups that alternate units.  Shared-memory
// bandwidth (operand reads by the tensor core, coefficient broadcasts) is the scarce on-chip
// resource, which is what the two-rows-per-thread epilogue is for.  Every wait is bounded; on
// expiry the CTA raises SPECA_STATUS_TIMEOUT, drains and exits.
//
// Fused commit-and-verify (the delayed state update of Section 5).  A second instantiation
// adds one role, the warps after the epilogue groups: between the TMA landing a state slice and the tensor core
// reading it, they advance the slice in place over the pending accepted path,
//        S <- gamma_A S + sum_{i < A} (gamma_A / gamma_i) u_i k_i^T ,
// with the u_i the previous verification wrote, and send the slice back to HBM with a TMA
// store.  The tensor core then reads the committed state, so everything downstream is the
// plain verification; the state crosses HBM twice per round (one read, one write) instead
// of three times.
#include <cuda.h>

#include <cstdlib>
#include <mutex>

#include <type_traits>

#include "speca_common.cuh"
#include "tc_ptx.cuh"

namespace speca {

namespace {

using namespace tc;

constexpr int kDK = 128;                       // key width handled by this route
constexpr int kTileRows = 128;                 // value rows per tile (= TMEM lanes = MMA M)
constexpr int kChunkK = 32;                    // floats per 128-byte swizzle row
constexpr int kChunks = kDK / kChunkK;         // 4 K-chunks per tile
constexpr int kStageBytes = kTileRows * 128;   // 16 KiB per (tile, K-chunk)
constexpr int kStages = 6;
constexpr int kStagesFused = 5;                // the fused kernel's ring: its sixth slot holds the staged u rows of the pending
                                               // paths (the kernel reads the state at about half of its total traffic)
constexpr int kPollNs = 100;                   // pause of the fused producer when neither a load nor a store is ready
constexpr int kMaxNodes = 64;                  // nodes per sequence handled by this route
constexpr int kMaxDepth = 8;
constexpr int kBopRows = 2 * kMaxNodes;        // [K;Q] rows
constexpr int kBopChunkBytes = kBopRows * 128; // 16 KiB per K-chunk region
constexpr int kCoefStride = 20;                // floats per position: cU[7] cV cO[8] cR cG depth-1 out-offset
constexpr int kAccCols = 2 * kMaxNodes;        // 128 TMEM columns per tile accumulator (R | G)
constexpr int kPairCols = 2 * kAccCols;        // a unit's two tiles
constexpr int kTmemCols = 512;                 // two units in flight
constexpr int kThreads = 14 * 32;
constexpr int kUpdWarps = 2;                   // state-update role of the fused kernel
constexpr int kUpdThreads = kUpdWarps * 32;
constexpr int kThreadsFused = kThreads + kUpdThreads;
#ifndef SPECA_SPLIT_WARPS
#define SPECA_SPLIT_WARPS 4
#endif
constexpr int kSplitWarps = SPECA_SPLIT_WARPS;      // warps that rewrite slices as their remainder
constexpr int kSplitThreads = kSplitWarps * 32;
constexpr int kThreadsComp = kThreads + (1 + kSplitWarps) * 32;  // compensated form: a second MMA issuer and the split warps
constexpr int kPrepThreads = 128;
// The tensor core reads an fp32 state element as TF32 by dropping its low 13 mantissa bits, i.e. it
// rounds every element toward zero: on average a value with mantissa m in [1, 2) loses 2^-11 / m of
// itself, and E[1/m] is 0.69 .. 0.72 for any smooth distribution that spans a few binades.  The
// products R = K S0^T and G = Q S0^T are therefore short by that fraction on average; the coefficients
// that multiply them carry the expected-value correction.  It halves the typical error of the route
// (measured 4.0e-4 -> 2.1e-4 at S0 ~ N(0, 0.02^2)); on a state whose elements happen to be exact in TF32
// it costs at most the same 3.5e-4 of |R|, far inside the 2e-3 bar.
constexpr float kDebias = 1.0f + 0.71f / 2048.0f;
constexpr int kEpiChunk = 4;                   // nodes per TMEM read in the epilogue
constexpr int kGramHalf = 32;                  // Gram columns parked per extraction pass
constexpr int kStageChunkBytes = kBopRows * 128; // 64 bf16 columns of all [K;Q] rows: 16 KiB

// shared memory carve-up (bytes, from a 1024-byte aligned base)
constexpr int kOffRing = 0;
constexpr int kOffBop = kOffRing + kStages * kStageBytes;
constexpr int kOffStage = kOffBop + kChunks * kBopChunkBytes;              // raw bf16 [K;Q] rows of the next unit
constexpr int kOffGram = kOffStage + 2 * kStageChunkBytes;
constexpr int kOffCoef = kOffGram + kGramHalf * kTileRows * 4;
constexpr int kOffAlpha = kOffCoef + 2 * kMaxNodes * kCoefStride * 4;
constexpr int kOffBars = kOffAlpha + 2 * kMaxNodes * 4;                   // alpha, beta by position
constexpr int kOffMisc = kOffBars + 8 * 56;
constexpr int kOffPendK = kOffMisc + 64;                                  // bf16 keys of the pending path [2][8][d_k + 8]
constexpr int kKeyStride = kDK * 2 + 16;                                   // bytes per staged pending key (bank padding)
constexpr int kKeyBuf = kMaxDepth * kKeyStride;
constexpr int kOffWalk = kOffPendK + 2 * kKeyBuf;                          // per-sequence walk table
// fused kernel: u rows of the pending path, [2][8][256] fp32, in the sixth ring slot
constexpr int kOffPendU = kOffRing + kStagesFused * kStageBytes;
constexpr int kPendUStride = 2 * kTileRows * 4;
constexpr int kPendUBuf = kMaxDepth * kPendUStride;
static_assert(2 * kPendUBuf <= (kStages - kStagesFused) * kStageBytes, "pending u rows do not fit the spare ring slots");
constexpr int kWalkSeqs = 192;                                            // sequences the table holds
constexpr int kWalkOffs = 0, kWalkPBase = 4 * kWalkSeqs, kWalkPNode = 8 * kWalkSeqs, kWalkN = 16 * kWalkSeqs,
              kWalkA = 17 * kWalkSeqs;
constexpr int kSmemBytes = kOffWalk + 18 * kWalkSeqs;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

enum Bar {
    kBarFull = 0,                        // [kStages] TMA -> MMA
    kBarEmpty = kBarFull + kStages,      // [kStages] MMA -> TMA
    kBarBReady = kBarEmpty + kStages,    // prep -> MMA (and prep-internal): [K;Q] operand, alpha, beta written
    kBarBFree,                           // MMA -> prep: operand no longer read
    kBarStageReady,                      // prep -> MMA: raw bf16 rows of a unit staged (Gram operand)
    kBarGramFull,                        // MMA -> prep: Gram block in TMEM
    kBarGramDone,                        // prep -> MMA: Gram block read, its columns may be overwritten
    kBarCoefReady,                       // [2] prep -> epilogue group
    kBarCoefFree = kBarCoefReady + 2,    // [2] epilogue group -> prep
    kBarAccFull = kBarCoefFree + 2,      // [2] MMA -> epilogue group: the unit's accumulators are complete
    kBarPairFree = kBarAccFull + 2,      // [2] epilogue group -> MMA: accumulator columns released
    kBarDrain = kBarPairFree + 2,        // MMA warp: everything issued has completed
    kBarUpd,                             // [kStages] fused only: update role -> MMA, slice advanced in place
    kBarPendFull = kBarUpd + kStages,    // [2] fused only: TMA producer -> update role, pending u rows and keys staged
    kBarPendFree = kBarPendFull + 2,     // [2] fused only: update role -> TMA producer
    kBarP1Done = kBarPendFree + 2,       // [kStages] compensated form: MMA -> split warps, first pass has read the slice
    kBarLo = kBarP1Done + kStages,       // [kStages] compensated form: split warps -> MMA, slice rewritten as its remainder
    kBarCount
};
static_assert(kBarCount <= 56, "barrier region too small");


// Optional self-profiling build (-DSPECA_PROF): cycles spent in each kind of wait per role.
#ifdef SPECA_PROF
#define PROF_DECL long long prof_w[8] = {0, 0, 0, 0, 0, 0, 0, 0}; const long long prof_t0 = clock64(); long long prof_mark = prof_t0;
#define PROF_MARK() prof_mark = clock64();
#define PROF_SEG(slot) { const long long t_ = clock64(); prof_w[slot] += t_ - prof_mark; prof_mark = t_; }
#define WAIT(slot, b, ph) prof_wait(prof_w[slot], b, ph, abort_flag)
#define PROF_STORE()                                                                              \
    if (blockIdx.x == 0 && lane == 0) {                                                           \
        long long *dst = reinterpret_cast<long long *>(p.ws.ctrl) + 8 + warp * 9;                \
        for (int i_ = 0; i_ < 8; ++i_) dst[i_] = prof_w[i_];                                      \
        dst[8] = clock64() - prof_t0;                                                             \
    }
__device__ __forceinline__ bool prof_wait(long long &acc, uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    const long long t = clock64();
    const bool r = mbar_wait(bar, parity, abort_flag);
    acc += clock64() - t;
    return r;
}
#else
#define PROF_DECL
#define PROF_MARK()
#define PROF_SEG(slot)
#define WAIT(slot, b, ph) wait_fast(b, ph, abort_flag)
#define PROF_STORE()
#endif


// Tensor maps of the bf16 key / query records, view [L*T][H][d_k], one per box height
// (16, 32, 48, 64 nodes): a unit's rows are fetched with the smallest box that covers them.
struct KQMaps { CUtensorMap k[4], q[4], v[4]; };

struct FParams {
    Params p;
    int32_t heads_per_group;     // consecutive heads of one (layer, sequence) a CTA takes together
    int32_t withhold_first_load; // test hook: CTA 0 never issues its first state load, so that its waits run out
    long n_units;
};

__device__ __forceinline__ int anc_byte(const int4 &meta, int j)
{
    return int((j < 4 ? (uint32_t(meta.y) >> (8 * j)) : (uint32_t(meta.z) >> (8 * (j - 4)))) & 0xffu);
}
// levels 0..14 (trees up to 16 deep): levels 8..11 in the first record's last word, 12..14 in the second record
__device__ __forceinline__ int anc_byte16(const int4 &meta, int meta2, int j)
{
    const uint32_t w = j < 4 ? uint32_t(meta.y) : j < 8 ? uint32_t(meta.z) : j < 12 ? uint32_t(meta.w) : uint32_t(meta2);
    return int((w >> (8 * (j & 3))) & 0xffu);
}


// Units are taken in groups of HG consecutive heads of one (layer, sequence): group
// G = blockIdx.x, += gridDim.x.  Inside a group the topology-dependent data (node count,
// order, ancestors) is loaded once.  Sequences that failed validation or are empty are
// skipped.  Every role walks the same list; unit number i of a CTA (unit_seq) uses
// accumulator pair, coefficient buffer and epilogue group i & 1.
// Fused walk: a is the length of the sequence's pending accepted path; a sequence whose new
// tree is empty or was rejected still gets its commit (a unit with no nodes).
struct Unit { int grp, hi, u, b, l, h, n, npad, base, a; };
// What the walk needs per sequence (node count, offset, pending path) is copied into shared
// memory when the kernel starts, for the first kWalkSeqs sequences: a global load on the
// per-unit control path costs a full memory round trip under a saturated HBM.
struct UnitWalk {
    int HG, gpl, n_groups, H, B, grid;
    const int32_t *seq_n; const int32_t *offs; const int32_t *pend;
    const uint8_t *tab;
};

__device__ __forceinline__ bool load_group(const UnitWalk &w, int G, Unit &x)
{
    for (; G < w.n_groups; G += w.grid) {
        const int lb = G / w.gpl;                        // (layer, sequence) pair
        x.b = lb % w.B;
        const bool in_tab = x.b < kWalkSeqs;
        if (in_tab) {
            x.n = reinterpret_cast<const int8_t *>(w.tab + kWalkN)[x.b];
            x.a = reinterpret_cast<const int8_t *>(w.tab + kWalkA)[x.b];
        } else {
            x.n = w.seq_n[x.b];
            x.a = w.pend != nullptr ? __ldg(w.pend + x.b * kPendWords) : 0;
        }
        if (x.a > 0 && x.n < 0) x.n = 0;
        if (x.n > 0 || x.a > 0) {
            x.grp = G;
            x.hi = 0;
            x.l = lb / w.B;
            x.h = (G - lb * w.gpl) * w.HG;
            x.u = lb * w.H + x.h;
            x.npad = x.n > 0 ? (x.n + 15) & ~15 : 16;
            x.base = in_tab ? reinterpret_cast<const int32_t *>(w.tab + kWalkOffs)[x.b] : __ldg(w.offs + x.b);
            return true;
        }
    }
    x.n = 0; x.a = 0; x.grp = w.n_groups;
    return false;
}
__device__ __forceinline__ bool first_unit(const UnitWalk &w, Unit &x) { return load_group(w, int(blockIdx.x), x); }
__device__ __forceinline__ bool next_unit(const UnitWalk &w, Unit &x)
{
    if (++x.hi < w.HG) { ++x.h; ++x.u; return true; }
    return load_group(w, x.grp + w.grid, x);
}


// One node of the forward substitution for TP value rows (one per tile of the unit),
// branch-free.  The u of the nodes on the current depth-first path live in ustk[.][depth-1];
// coefficients of levels that are not ancestors of this node are zero.
//   cf[0..6] cU   cf[7] cV   cf[8..15] cO   cf[16] cR   cf[17] cG   cf[18] depth-1   cf[19] output offset
// SELF: the coefficient of the node's own u (q.k) sits in cO[7] whatever the depth and the last stack slot always
// takes the node's own u (a node at depth 8 has no children, so that slot is never an ancestor's): one select and one
// compare fewer per row, and a leaf can stay out of the stack altogether (level -1 in its record), so that the sums
// of the node after it do not depend on it (64-node trees 10.8 -> 10.5 us per unit in the compensated kernel, 9.4 ->
// 9.15 in the single-pass one).  A form of the step on packed two-wide fp32 FMAs was measured equal on trees, 1.5 %
// better on 8-node chains and spills at the compensated kernel's 96 registers; it is not kept.
template <int TP, bool SELF = false>
__device__ __forceinline__ void node_step(float (&ustk)[TP][kMaxDepth], const float *cf, const float (&Rv)[TP],
                                          const float (&Gv)[TP], const float (&vv)[TP], float (&u_out)[TP],
                                          float (&o_out)[TP], int &off)
{
    const float4 a0 = *reinterpret_cast<const float4 *>(cf + 0), a1 = *reinterpret_cast<const float4 *>(cf + 4);
    const float4 b0 = *reinterpret_cast<const float4 *>(cf + 8), b1 = *reinterpret_cast<const float4 *>(cf + 12);
    const float4 s = *reinterpret_cast<const float4 *>(cf + 16);
    const int d1 = __float_as_int(s.z);
    off = __float_as_int(s.w);
#pragma unroll
    for (int t = 0; t < TP; ++t) {
        float u0 = fmaf(a1.w, vv[t], s.x * Rv[t]);
        float u1 = a0.y * ustk[t][1];
        u0 = fmaf(a0.x, ustk[t][0], u0);
        u1 = fmaf(a0.w, ustk[t][3], u1);
        u0 = fmaf(a0.z, ustk[t][2], u0);
        u1 = fmaf(a1.y, ustk[t][5], u1);
        u0 = fmaf(a1.x, ustk[t][4], u0);
        u0 = fmaf(a1.z, ustk[t][6], u0);
        const float u = u0 + u1;
#pragma unroll
        for (int j = 0; j < kMaxDepth - (SELF ? 1 : 0); ++j) ustk[t][j] = (d1 == j) ? u : ustk[t][j];
        if (SELF) ustk[t][kMaxDepth - 1] = u;
        float o0 = fmaf(b0.x, ustk[t][0], s.y * Gv[t]);
        float o1 = b0.y * ustk[t][1];
        o0 = fmaf(b0.z, ustk[t][2], o0);
        o1 = fmaf(b0.w, ustk[t][3], o1);
        o0 = fmaf(b1.x, ustk[t][4], o0);
        o1 = fmaf(b1.y, ustk[t][5], o1);
        o0 = fmaf(b1.z, ustk[t][6], o0);
        o1 = fmaf(b1.w, ustk[t][7], o1);
        o_out[t] = o0 + o1;
        u_out[t] = u;
    }
}

// The same step for trees up to MAXD levels deep (the coefficient record is cU[MAXD-1] cV cO[MAXD] cR cG
// depth-1 offset).  Used for MAXD = 16; the 8-level form above is kept as it is because the shape of its
// two accumulation chains was tuned.
template <int TP, int MAXD, bool SELF = false>
__device__ __forceinline__ void node_step_deep(float (&ustk)[TP][MAXD], const float *cf, const float (&Rv)[TP],
                                               const float (&Gv)[TP], const float (&vv)[TP], float (&u_out)[TP],
                                               float (&o_out)[TP], int &off)
{
    float cu[MAXD], co[MAXD];
#pragma unroll
    for (int i = 0; i < MAXD / 4; ++i) {
        const float4 a = *reinterpret_cast<const float4 *>(cf + 4 * i), b = *reinterpret_cast<const float4 *>(cf + MAXD + 4 * i);
        cu[4 * i] = a.x; cu[4 * i + 1] = a.y; cu[4 * i + 2] = a.z; cu[4 * i + 3] = a.w;
        co[4 * i] = b.x; co[4 * i + 1] = b.y; co[4 * i + 2] = b.z; co[4 * i + 3] = b.w;
    }
    const float4 s = *reinterpret_cast<const float4 *>(cf + 2 * MAXD);
    const int d1 = __float_as_int(s.z);
    off = __float_as_int(s.w);
#pragma unroll
    for (int t = 0; t < TP; ++t) {
        float u0 = fmaf(cu[MAXD - 1], vv[t], s.x * Rv[t]), u1 = 0.f;
#pragma unroll
        for (int j = 0; j < MAXD - 1; ++j) {
            if (j & 1) u1 = fmaf(cu[j], ustk[t][j], u1);
            else u0 = fmaf(cu[j], ustk[t][j], u0);
        }
        const float u = u0 + u1;
#pragma unroll
        for (int j = 0; j < MAXD - (SELF ? 1 : 0); ++j) ustk[t][j] = (d1 == j) ? u : ustk[t][j];
        if (SELF) ustk[t][MAXD - 1] = u;
        float o0 = s.y * Gv[t], o1 = 0.f;
#pragma unroll
        for (int j = 0; j < MAXD; ++j) {
            if (j & 1) o1 = fmaf(co[j], ustk[t][j], o1);
            else o0 = fmaf(co[j], ustk[t][j], o0);
        }
        o_out[t] = o0 + o1;
        u_out[t] = u;
    }
}

// TP = value tiles per unit (d_v / 128): 1 or 2.  FUSED adds the state-update role (d_k = 128 only).
// DK = key width, 128 or 256.  The operand buffers have a fixed size, so the wider key halves
// the number of [K;Q] rows they hold: up to 64 nodes per sequence at d_k = 128, 32 at d_k = 256.
// DEEP: trees up to 16 levels deep (up to 32 nodes per sequence at either key width; not with FUSED).
// COMP: compensated form (not with FUSED).  The tensor core reads the fp32 state as TF32, i.e. its top 19 bits;
// every slice is therefore multiplied twice: as landed, and, rewritten in place as its exact remainder
// S - tf32(S) by two extra warps, once more into the same accumulator.  [K;Q] is exact in TF32, so R and G carry
// fp32 accuracy (the dropped part is 2^-21 of the state).  The two value tiles are then issued by two warps.
template <int TP, bool FUSED, int DK = kDK, bool DEEP = false, bool COMP = false>
__global__ void __launch_bounds__(FUSED ? kThreadsFused : (COMP ? kThreadsComp : kThreads), 1)
verify_factorized_kernel(const __grid_constant__ CUtensorMap s0_map, const __grid_constant__ KQMaps kq, FParams fp)
{
    // The swizzled operand regions need 1024-byte alignment.  The array is declared with that
    // alignment and used directly, so every access below stays a shared-memory access for the
    // compiler (address space known, no aliasing with the global output pointers).
    extern __shared__ __align__(1024) uint8_t smem[];
    const Params &p = fp.p;
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {                                 // never expected; refuse to run rather than corrupt
        if (threadIdx.x == 0) atomicOr(p.status, SPECA_STATUS_TIMEOUT);
        return;
    }
    const uint32_t bars = sbase + kOffBars;
    auto bar = [&](int i) { return bars + 8u * uint32_t(i); };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffMisc);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + kOffMisc + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar(kBarFull + s), 1);
            mbar_init(bar(kBarEmpty + s), 1);
            mbar_init(bar(kBarUpd + s), kUpdThreads);
            mbar_init(bar(kBarP1Done + s), 1);
            mbar_init(bar(kBarLo + s), kSplitWarps);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(bar(kBarPendFull + i), 1); mbar_init(bar(kBarPendFree + i), kUpdThreads); }
        mbar_init(bar(kBarBReady), kPrepThreads);
        mbar_init(bar(kBarBFree), COMP ? TP : 1);
        mbar_init(bar(kBarStageReady), 1);
        mbar_init(bar(kBarGramFull), 1);
        mbar_init(bar(kBarGramDone), kPrepThreads);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(kBarCoefReady + i), kPrepThreads);
            mbar_init(bar(kBarCoefFree + i), 128);
            mbar_init(bar(kBarAccFull + i), COMP ? TP : 1);
            mbar_init(bar(kBarPairFree + i), 128);
        }
        mbar_init(bar(kBarDrain), COMP ? TP : 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int b = threadIdx.x; b < p.B && b < kWalkSeqs; b += blockDim.x) {
        const int n = p.ws.seq_n[b];
        reinterpret_cast<int8_t *>(smem + kOffWalk + kWalkN)[b] = int8_t(n < 0 ? -1 : n);       // n <= kMaxNodes
        reinterpret_cast<int32_t *>(smem + kOffWalk + kWalkOffs)[b] = p.node_offsets[b];
        int a = 0;
        if (FUSED) {
            const int32_t *rec = p.ws.pend + b * kPendWords;
            a = rec[0];
            reinterpret_cast<int32_t *>(smem + kOffWalk + kWalkPBase)[b] = rec[9];
            for (int i = 0; i < kMaxDepth; ++i) smem[kOffWalk + kWalkPNode + b * kMaxDepth + i] = uint8_t(rec[1 + i]);
        }
        reinterpret_cast<int8_t *>(smem + kOffWalk + kWalkA)[b] = int8_t(a);
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    constexpr int NS = FUSED ? kStagesFused : kStages;            // ring depth in use
    constexpr bool kSelfSlot = true;                              // see node_step
    static_assert(DK == 128 || DK == 256, "key width");
    constexpr int NC = DK / kChunkK;                              // K-chunks (state slices) per tile
    constexpr int BROWS = DK == 128 ? kBopRows : kBopRows / 2;    // [K;Q] rows the operand buffers hold
    constexpr int BCB = BROWS * 128;                              // bytes of one K-chunk region of the fp32 operand
    constexpr int SC = DK / 64;                                   // 64-column chunks of the staged bf16 rows
    constexpr int SCB = BROWS * 128;                              // bytes of one such chunk
    static_assert(NC * BCB == kChunks * kBopChunkBytes && SC * SCB == 2 * kStageChunkBytes, "operand buffers keep their size");
    static_assert(!(FUSED && DEEP), "the fused kernel takes pending paths and trees of at most 8 levels");
    static_assert(!(FUSED && COMP), "the fused kernel reads the state in a single TF32 pass");
    constexpr int MAXD = DEEP ? 2 * kMaxDepth : kMaxDepth;        // tree depth this instantiation takes
    constexpr int CS = 2 * MAXD + 4;                              // floats of a coefficient record
    constexpr int MAXN = DEEP ? kMaxNodes / 2 : BROWS / 2;        // nodes per sequence; also the stride of the coefficient buffers
    static_assert(2 * MAXN * CS * 4 <= 2 * kMaxNodes * kCoefStride * 4 && CS % 4 == 0, "coefficient records do not fit");
    // Fused kernel: staged bf16 keys of the pending path, two buffers of 8 padded rows.  At d_k = 128 both
    // sit in their own region; at d_k = 256 a buffer is twice as large, and the second one takes the half
    // of the coefficient region that 32-node sequences leave unused.
    constexpr int KSTRIDE = DK * 2 + 16, KBUF = kMaxDepth * KSTRIDE;
    static_assert(DK == kDK ? 2 * KBUF <= kOffWalk - kOffPendK
                            : (KBUF <= kOffWalk - kOffPendK && KBUF <= kMaxNodes * kCoefStride * 4), "pending keys do not fit");
    auto key_buf = [](int pb) -> int {
        return DK == kDK ? kOffPendK + pb * KBUF : (pb == 0 ? kOffPendK : kOffCoef + 2 * MAXN * CS * 4);
    };
    UnitWalk walk;
    walk.HG = fp.heads_per_group; walk.gpl = p.H / fp.heads_per_group;
    walk.n_groups = int(fp.n_units / fp.heads_per_group);
    walk.H = p.H; walk.B = p.B; walk.grid = int(gridDim.x);
    walk.seq_n = p.ws.seq_n; walk.offs = p.node_offsets;
    walk.pend = FUSED ? p.ws.pend : nullptr;
    walk.tab = smem + kOffWalk;

    if (warp == 0 && FUSED) {
        // ------------------------------------------------------------- TMA producer of the fused kernel
        // Besides loading state slices it sends the advanced slices back: a TMA store needs a good
        // fraction of a microsecond to read its 16 KiB out of shared memory under load, so nobody
        // may block on one.  The warp keeps two cursors over the same sequence of slices, one for
        // loads and one (behind it) for stores, and serves whichever is ready; a slot is reloaded
        // once the tensor core has read it and the store of its previous content has read it.
        // Stores are committed one bulk group per slice (an empty group for slices of units with
        // nothing pending), so group age equals slice age.
        uint32_t it = 0, ist = 0, pseq = 0;                      // slices loaded, slices stored, staged units
        Unit x, nx, xs = {};                                     // unit being loaded, the one after it, unit being stored
        int js = 0;                                              // slice of xs the store cursor is at
        bool ok = true;
        auto stage_pending = [&](const Unit &y) -> bool {
            if (y.a == 0) return true;
            const int pb = pseq & 1;
            if (!wait_fast(bar(kBarPendFree + pb), ((pseq >> 1) & 1) ^ 1, abort_flag)) return false;
            if (lane == 0) mbar_arrive_expect_tx(bar(kBarPendFull + pb), uint32_t(y.a) * uint32_t(p.DV * 4 + DK * 2));
            __syncwarp();
            if (lane < y.a) {
                const int node = y.b < kWalkSeqs
                    ? reinterpret_cast<const int32_t *>(smem + kOffWalk + kWalkPBase)[y.b] +
                          int(smem[kOffWalk + kWalkPNode + y.b * kMaxDepth + lane])
                    : __ldg(p.ws.pend + y.b * kPendWords + 9) + __ldg(p.ws.pend + y.b * kPendWords + 1 + lane);
                const size_t rec = (size_t(y.l) * p.Tp + node) * p.H + y.h;
                bulk_load(sbase + kOffPendU + pb * kPendUBuf + lane * kPendUStride, p.pu + rec * p.DV, uint32_t(p.DV * 4),
                          bar(kBarPendFull + pb));
                bulk_load(sbase + key_buf(pb) + lane * KSTRIDE, p.pk + rec * DK, uint32_t(DK * 2),
                          bar(kBarPendFull + pb));
            }
            ++pseq;
            return true;
        };
        // store (or skip) slice ist, which the update role has finished, and advance the store cursor
        auto issue_store = [&]() {
            if (lane == 0) {
                if (xs.a > 0)
                    tma_store_3d_nocommit(&s0_map, (js % NC) * kChunkK, js / NC, xs.u * kTileRows,
                                          sbase + kOffRing + (ist % NS) * kStageBytes);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            __syncwarp();
            ++ist;
            if (++js == TP * NC) { js = 0; next_unit(walk, xs); }
        };
        auto updated = [&](uint32_t i, bool blocking) -> int {   // 1 ready, 0 not yet, -1 abort
            if (xs.a == 0) return 1;
            const uint32_t b = bar(kBarUpd + i % NS), ph = (i / NS) & 1;
            if (!blocking) return __all_sync(0xffffffffu, mbar_test_wait(b, ph)) ? 1 : 0;
            return wait_fast(b, ph, abort_flag) ? 1 : -1;
        };
        bool have = first_unit(walk, x);
        xs = x;
        if (have) ok = stage_pending(x);
        for (; have && ok; x = nx) {
            nx = x;
            const bool have_next = next_unit(walk, nx);
            have = have_next;
            if (lane == 0 && x.n > 0) tma_prefetch_3d(&kq.v[(x.npad >> 4) - 1], 0, x.h, x.l * p.T + x.base);
            for (int j = 0; j < TP * NC && ok; ++j, ++it) {
                // halfway through the unit the update role has left the unit before it, whose
                // staging buffer the next unit's pending path takes
                if (have_next && j == TP * NC / 2 && !(ok = stage_pending(nx))) break;
                const int s = it % NS;
                if (it >= uint32_t(NS)) {
                    // the slot's previous content (slice it - NS) must have been stored ...
                    while (ok && ist <= it - NS) {
                        if (updated(ist, true) < 0) ok = false;
                        else issue_store();
                    }
                    if (!ok) break;
                    // ... and that store must have read it: at most ist - 1 - (it - NS) younger groups pending
                    if (lane == 0) {
                        switch (int(ist - 1 - (it - NS))) {
                        case 0: tma_store_wait_read<0>(); break;
                        case 1: tma_store_wait_read<1>(); break;
                        case 2: tma_store_wait_read<2>(); break;
                        case 3: tma_store_wait_read<3>(); break;
                        default: tma_store_wait_read<4>(); break;
                        }
                    }
                    __syncwarp();
                }
                // wait for the tensor core to release the slot, serving stores that become ready meanwhile
                {
                    const uint32_t be = bar(kBarEmpty + s), pe = ((it / NS) & 1) ^ 1;
                    uint64_t t0 = 0;
                    for (uint32_t spin = 0; ok; ++spin) {
                        if (__all_sync(0xffffffffu, mbar_test_wait(be, pe))) break;
                        if (ist < it && updated(ist, false) == 1) issue_store();
                        else __nanosleep(kPollNs);         // nothing to do: leave the issue slots to the other warps
                        if ((spin & 255u) == 255u) {
                            if (__any_sync(0xffffffffu, *abort_flag != 0)) ok = false;
                            const uint64_t now = global_timer_ns();
                            if (t0 == 0) t0 = now;
                            if (__any_sync(0xffffffffu, now - t0 > kWaitLimitNs)) { *abort_flag = 1; ok = false; }
                        }
                    }
                    if (!ok) break;
                }
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(kBarFull + s), kStageBytes);
                    tma_load_3d(sbase + kOffRing + s * kStageBytes, &s0_map, (j % NC) * kChunkK, j / NC,
                                x.u * kTileRows, bar(kBarFull + s));
                }
                __syncwarp();
            }
        }
        // drain: store what is left, then let every store finish
        while (ok && ist < it) {
            if (updated(ist, true) < 0) ok = false;
            else issue_store();
        }
        if (lane == 0) tma_store_wait_all();
        __syncwarp();
        if (*abort_flag) {
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
    } else if (warp == 0) {
        // ------------------------------------------------------------- TMA producer
        uint32_t it = 0;
        Unit x;
        bool ok = true;
        PROF_DECL
        for (bool have = first_unit(walk, x); have && ok; have = next_unit(walk, x)) {
            // the value rows of this unit's nodes are read by the epilogue with plain loads a
            // couple of units from now: pull them into L2 meanwhile
            if (lane == 0 && x.n > 0) tma_prefetch_3d(&kq.v[(x.npad >> 4) - 1], 0, x.h, x.l * p.T + x.base);
            // tile t of a unit holds its value rows t, t + TP, t + 2 TP, ... (interleaved tiles:
            // an epilogue thread then owns TP ADJACENT value rows, one per tile).  Slices go tile by tile,
            // or, in the compensated form (one MMA issuer per tile), K-slice by K-slice over both tiles.
            const int row = x.u * kTileRows;                          // row-group in the [units*128][TP][d_k] view of S0
            for (int o = 0; o < TP && ok; ++o) {
                for (int i = 0; i < NC; ++i, ++it) {
                    const int lin = o * NC + i;
                    const int t = COMP ? lin % TP : o, c = COMP ? lin / TP : i;
                    const int s = it % NS;
                    const uint32_t ph = (it / NS) & 1;
                    if (!(ok = WAIT(0, bar(kBarEmpty + s), ph ^ 1))) break;
                    if (lane == 0 && !(fp.withhold_first_load && blockIdx.x == 0 && it == 0)) {
                        mbar_arrive_expect_tx(bar(kBarFull + s), kStageBytes);
                        tma_load_3d(sbase + kOffRing + s * kStageBytes, &s0_map, c * kChunkK, t, row, bar(kBarFull + s));
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
    } else if (COMP && (warp == 1 || warp == 14)) {
        // ------------------------------------------------------------- MMA issuers of the compensated form
        // One warp per value tile (disjoint accumulator columns); warp 1 also issues the Gram blocks.  Per slice:
        // first pass as landed, then -- one slice later, so that the rewrite in between is rarely waited for --
        // the second pass over the remainder, which releases the slot.
        const int mt = warp == 1 ? 0 : 1;
        uint32_t unit_seq = 0;
        Unit x;
        bool ok = mt < TP;
        const uint32_t bop = sbase + kOffBop, stage = sbase + kOffStage;
        PROF_DECL
        auto issue_gram = [&](uint32_t seq, int npad) -> bool {
            const int pr = seq & 1;
            if (!wait_fast(bar(kBarStageReady), seq & 1, abort_flag)) return false;
            if (!wait_fast(bar(kBarPairFree + pr), ((seq >> 1) & 1) ^ 1, abort_flag)) return false;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t idg = make_idesc_bf16(npad);
#pragma unroll
                for (int c = 0; c < SC; ++c)
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t d = make_desc(stage + c * SCB + k * 32);
                        mma_bf16(tmem_base + pr * kPairCols, d, d, idg, (c | k) != 0);
                    }
                mma_commit(bar(kBarGramFull));
            }
            __syncwarp();
            return true;
        };
        bool have = ok && first_unit(walk, x);
        if (have && mt == 0) ok = issue_gram(0, x.npad);
        while (have && ok) {
            const int pr = unit_seq & 1;
            const uint32_t acc = tmem_base + pr * kPairCols + mt * kAccCols;
            if (!(ok = WAIT(0, bar(kBarBReady), unit_seq & 1))) break;
            if (mt == 0) {
                if (!(ok = WAIT(1, bar(kBarGramDone), unit_seq & 1))) break;
            } else if (!(ok = WAIT(1, bar(kBarPairFree + pr), ((unit_seq >> 1) & 1) ^ 1))) {
                break;
            }
            tc_fence_after();
            const uint32_t idm = make_idesc(2 * x.npad);
            int ps = -1;
            uint32_t pph = 0;
            for (int c = 0; c <= NC && ok; ++c) {
                if (c < NC) {
                    const uint32_t it = (unit_seq * NC + c) * TP + mt;
                    const int s = it % NS;
                    const uint32_t ph = (it / NS) & 1;
                    if (!(ok = WAIT(2, bar(kBarFull + s), ph))) break;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t sa = sbase + kOffRing + s * kStageBytes;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_tf32(acc, make_desc(sa + k * 32), make_desc(bop + c * BCB + k * 32), idm, (c | k) != 0);
                        mma_commit(bar(kBarP1Done + s));
                    }
                    __syncwarp();
                    if (ps >= 0) {
                        if (!(ok = WAIT(3, bar(kBarLo + ps), pph))) break;
                        tc_fence_after();
                        if (lane == 0) {
                            const uint32_t sa = sbase + kOffRing + ps * kStageBytes;
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                mma_tf32(acc, make_desc(sa + k * 32), make_desc(bop + (c - 1) * BCB + k * 32), idm, 1);
                            mma_commit(bar(kBarEmpty + ps));
                        }
                        __syncwarp();
                    }
                    ps = s; pph = ph;
                } else {
                    // the last slice's second pass closes the tile
                    if (!(ok = WAIT(3, bar(kBarLo + ps), pph))) break;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t sa = sbase + kOffRing + ps * kStageBytes;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_tf32(acc, make_desc(sa + k * 32), make_desc(bop + (NC - 1) * BCB + k * 32), idm, 1);
                        mma_commit(bar(kBarEmpty + ps));
                        mma_commit(bar(kBarAccFull + pr));
                        mma_commit(bar(kBarBFree));
                    }
                    __syncwarp();
                }
            }
            if (!ok) break;
            ++unit_seq;
            have = next_unit(walk, x);
            if (have && mt == 0) ok = issue_gram(unit_seq, x.npad);
        }
        PROF_STORE()
        // everything this warp issued must have completed before TMEM is released
        if (mt < TP) {
            if (lane == 0) mma_commit(bar(kBarDrain));
            __syncwarp();
            mbar_wait(bar(kBarDrain), 0, abort_flag);
        }
    } else if (COMP && warp >= 15) {
        // ------------------------------------------------------------- compensated form: remainder of every slice, in place
        const int stid = threadIdx.x - 15 * 32;                  // 0..127
        uint32_t it = 0;
        Unit x;
        bool ok = true;
        PROF_DECL
        for (bool have = first_unit(walk, x); have && ok; have = next_unit(walk, x)) {
            for (int i = 0; i < TP * NC; ++i, ++it) {
                const int s = it % NS;
                const uint32_t ph = (it / NS) & 1;
                // the remainders are formed while the first pass is still reading the slice; only the stores wait
                if (!(ok = WAIT(0, bar(kBarFull + s), ph))) break;
                float4 *sl = reinterpret_cast<float4 *>(smem + kOffRing + s * kStageBytes);
                float4 v[kStageBytes / 16 / kSplitThreads];
#pragma unroll
                for (int k = 0; k < kStageBytes / 16 / kSplitThreads; ++k) {
                    v[k] = sl[stid + k * kSplitThreads];
                    v[k].x -= __uint_as_float(__float_as_uint(v[k].x) & 0xffffe000u);
                    v[k].y -= __uint_as_float(__float_as_uint(v[k].y) & 0xffffe000u);
                    v[k].z -= __uint_as_float(__float_as_uint(v[k].z) & 0xffffe000u);
                    v[k].w -= __uint_as_float(__float_as_uint(v[k].w) & 0xffffe000u);
                }
                if (!(ok = WAIT(1, bar(kBarP1Done + s), ph))) break;
#pragma unroll
                for (int k = 0; k < kStageBytes / 16 / kSplitThreads; ++k) sl[stid + k * kSplitThreads] = v[k];
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarLo + s));
            }
        }
        PROF_STORE()
    } else if (warp == 1) {
        // ------------------------------------------------------------- MMA issuer
        uint32_t it = 0, unit_seq = 0;
        Unit x;
        bool ok = true;
        const uint32_t bop = sbase + kOffBop, stage = sbase + kOffStage;
        PROF_DECL
        // Gram block of a unit: [K;Q] (128 rows) x K^T (npad columns) from the raw bf16 rows,
        // parked in the unit's own accumulator columns until the state MMAs overwrite them.
        auto issue_gram = [&](uint32_t seq, int npad) -> bool {
            const int pr = seq & 1;
            if (!WAIT(0, bar(kBarStageReady), seq & 1)) return false;
            // the epilogue group must have released this pair of accumulators (unit seq - 2)
            if (!WAIT(1, bar(kBarPairFree + pr), ((seq >> 1) & 1) ^ 1)) return false;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t idg = make_idesc_bf16(npad);
#pragma unroll
                for (int c = 0; c < SC; ++c)
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t d = make_desc(stage + c * SCB + k * 32);
                        mma_bf16(tmem_base + pr * kPairCols, d, d, idg, (c | k) != 0);
                    }
                mma_commit(bar(kBarGramFull));
            }
            __syncwarp();
            return true;
        };
        bool have = first_unit(walk, x);
        if (have) ok = issue_gram(0, x.npad);
        while (have && ok) {
            const int pr = unit_seq & 1;
            const uint32_t acc = tmem_base + pr * kPairCols;
            if (!(ok = WAIT(2, bar(kBarBReady), unit_seq & 1))) break;
            if (!(ok = WAIT(3, bar(kBarGramDone), unit_seq & 1))) break;
            tc_fence_after();
            const uint32_t idm = make_idesc(2 * x.npad);
            for (int t = 0; t < TP && ok; ++t) {
                for (int c = 0; c < NC; ++c, ++it) {
                    const int s = it % NS;
                    const uint32_t ph = (it / NS) & 1;
                    if (!(ok = WAIT(4, bar((FUSED ? kBarUpd : kBarFull) + s), ph))) break;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t sa = sbase + kOffRing + s * kStageBytes;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_tf32(acc + t * kAccCols, make_desc(sa + k * 32),
                                     make_desc(bop + c * BCB + k * 32), idm, (c | k) != 0);
                        mma_commit(bar(kBarEmpty + s));
                    }
                    __syncwarp();
                }
            }
            if (!ok) break;
            if (lane == 0) { mma_commit(bar(kBarAccFull + pr)); mma_commit(bar(kBarBFree)); }
            __syncwarp();
            ++unit_seq;
            have = next_unit(walk, x);
            if (have) ok = issue_gram(unit_seq, x.npad);
        }
        PROF_STORE()
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
        // Raw bf16 rows of [K;Q] of the NEXT unit are fetched by TMA, in node-index order, into a
        // staging buffer laid out as a bf16 K-major 128-byte-swizzled operand: rows [0, npad) keys,
        // [npad, 2 npad) queries.  The Gram MMA reads it directly; the conversion below gathers
        // its rows in depth-first order into the fp32 operand of the state MMAs.
        // This thread converts, for operand rows r = sub, sub + RSTEP, ..., the 16-byte piece seg of
        // the row (bf16 columns 8 seg .. 8 seg + 7).
        const uint32_t stage = sbase + kOffStage;
        constexpr int PPR = DK / 8;                              // 16-byte bf16 pieces per row
        constexpr int RSTEP = kPrepThreads / PPR;                // rows converted per pass: 8 (d_k 128) or 4 (d_k 256)
        const int sub = tid / PPR, seg = tid % PPR;
        // staging piece of node nd: chunk (seg >> 3) of 64 bf16, 16-byte slot (seg & 7) ^ (nd & 7)
        const uint32_t stage_chunk = uint32_t((seg >> 3) * SCB);
        // fp32 operand: floats 8 seg .. 8 seg + 7 -> chunk seg >> 2, 16-byte slots 2 (seg & 3), +1 (swizzled by r & 7)
        const uint32_t bop_chunk = uint32_t((seg >> 2) * BCB);

        float my_alpha = 0.f, my_beta = 0.f;
        unsigned long long node_lo = ~0ull, node_hi = ~0ull;   // node at the position of each handled row (0xff = none)
        int topo_grp = -1;
        int4 meta_nxt = make_int4(0, 0, 0, 0);
        int meta2_nxt = 0;                                       // DEEP: ancestors of levels 12..14
        // start the TMA copies of unit x's rows (one thread), fetch alpha / beta and, when the
        // sequence changes, the topology this thread needs
        auto prefetch = [&](const Unit &x) {
            if (tid == 0) {
                const int m = (x.npad >> 4) - 1;             // box height 16 (m + 1)
                const int z = x.l * p.T + x.base;
                mbar_arrive_expect_tx(bar(kBarStageReady), uint32_t(4 * x.npad * DK));
#pragma unroll
                for (int c = 0; c < SC; ++c) {
                    tma_load_3d(stage + c * SCB, &kq.k[m], c * 64, x.h, z, bar(kBarStageReady));
                    tma_load_3d(stage + c * SCB + x.npad * 128, &kq.q[m], c * 64, x.h, z, bar(kBarStageReady));
                }
            }
            if (x.grp != topo_grp) {
                topo_grp = x.grp;
                node_lo = node_hi = 0ull;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int r = RSTEP * i + sub;
                    const int pos = r < x.npad ? r : r - x.npad;
                    const unsigned long long nd =
                        (r < 2 * x.npad && pos < x.n) ? (unsigned long long)(__ldg(p.ws.plan + x.base + pos) & 0xff) : 0xffull;
                    if (i < 8) node_lo |= nd << (8 * i);
                    else node_hi |= nd << (8 * (i - 8));
                }
                const int node = row < x.npad ? row : row - x.npad;
                meta_nxt = (row < 2 * x.npad && node < x.n)
                               ? __ldg(reinterpret_cast<const int4 *>(p.ws.anc) + x.base + node) : make_int4(0, 0, 0, 0);
                if (DEEP) meta2_nxt = (row < 2 * x.npad && node < x.n) ? __ldg(p.ws.anc2 + 4 * (x.base + node)) : 0;
            }
            if (tid < x.n) {
                const int rec = (x.l * p.T + x.base + tid) * p.H + x.h;
                my_alpha = __ldg(p.alpha + rec);
                my_beta = __ldg(p.beta + rec);
            }
        };

        uint32_t unit_seq = 0;
        Unit x, nx;
        bool ok = true;
        bool have = first_unit(walk, x);
        if (have) prefetch(x);
        int4 meta = meta_nxt;
        int meta2 = meta2_nxt;
        unsigned long long cur_lo = node_lo, cur_hi = node_hi;
        PROF_DECL
        for (; have && ok; ++unit_seq) {
            const int par = unit_seq & 1;
            // the previous unit's MMAs must be done reading the operand, and every prep thread
            // must be done reading alpha/beta of the previous unit
            if (unit_seq > 0) {
                if (!(ok = WAIT(0, bar(kBarBFree), (unit_seq - 1) & 1))) break;
                if (!(ok = WAIT(1, bar(kBarCoefReady + (par ^ 1)), ((unit_seq - 1) >> 1) & 1))) break;
            }
            PROF_MARK()
            // the staged rows of this unit have landed (the Gram MMA may still be reading them)
            if (!(ok = WAIT(2, bar(kBarStageReady), unit_seq & 1))) break;
            {
                // bf16 -> fp32 (exact): operand row r (depth-first position) <- staged row of its node
                const int iters = 2 * x.npad / RSTEP;
                const int nk = x.npad / RSTEP;               // rows [0, npad) keys, then queries
#pragma unroll 4
                for (int i = 0; i < iters; ++i) {
                    const int r = RSTEP * i + sub;
                    uint8_t *dst = smem + kOffBop + bop_chunk + r * 128;
                    const uint32_t bop_off0 = uint32_t(((2 * (seg & 3)) ^ (r & 7)) << 4);
                    const uint32_t bop_off1 = uint32_t(((2 * (seg & 3) + 1) ^ (r & 7)) << 4);
                    const int nd = int(((i < 8 ? cur_lo : cur_hi) >> (8 * (i & 7))) & 0xffull);
                    uint4 w = make_uint4(0u, 0u, 0u, 0u);
                    if (nd != 0xff) {
                        const int sr = i < nk ? nd : x.npad + nd;
                        w = *reinterpret_cast<const uint4 *>(smem + kOffStage + stage_chunk + (sr >> 3) * 1024 + (sr & 7) * 128 +
                                                            (((seg & 7) ^ (sr & 7)) << 4));
                    }
                    *reinterpret_cast<float4 *>(dst + bop_off0) =
                        make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u),
                                    __uint_as_float(w.y << 16), __uint_as_float(w.y & 0xffff0000u));
                    *reinterpret_cast<float4 *>(dst + bop_off1) =
                        make_float4(__uint_as_float(w.z << 16), __uint_as_float(w.z & 0xffff0000u),
                                    __uint_as_float(w.w << 16), __uint_as_float(w.w & 0xffff0000u));
                }
            }
            if (tid < x.n) { alpha_s[tid] = my_alpha; beta_s[tid] = my_beta; }
            fence_proxy_async();
            mbar_arrive(bar(kBarBReady));
            PROF_SEG(5)
            if (!(ok = WAIT(3, bar(kBarGramFull), unit_seq & 1))) break;
            tc_fence_after();
            PROF_MARK()

            // this thread's Gram row belongs to node `node` (keys: row, queries: row - npad)
            const bool is_k = row < x.npad;
            const int node = is_k ? row : row - x.npad;
            const bool in_rows = row < 2 * x.npad;
            const bool active = in_rows && node < x.n;
            const int d = meta.x & 0xff;
            const int pos = active ? ((meta.x >> 8) & 0xff) : node;       // padding rows: any unused record (n <= node < npad)
            // ancestors by level (level d-1 is the node itself), their alpha, and this row's Gram entries
            int anc_pos[MAXD];
            float anc_alpha[MAXD], gsel[MAXD];
#pragma unroll
            for (int j = 0; j < MAXD; ++j)
                anc_pos[j] = !active ? 0 : ((j < d - 1) ? (DEEP ? anc_byte16(meta, meta2, j) : anc_byte(meta, j)) : node);

            // park this thread's Gram row in its private scratch column (32 columns per pass),
            // then pick the entries it needs
            const uint32_t gaddr = tmem_base + par * kPairCols + lane_addr;
#pragma unroll
            for (int j = 0; j < MAXD; ++j) gsel[j] = 0.f;
#pragma unroll 1
            for (int half = 0; half * kGramHalf < x.npad; ++half) {
#pragma unroll 1
                for (int c0 = 0; c0 < kGramHalf; c0 += 16) {
                    float g0[8], g1[8];
                    tmem_ld8(gaddr + half * kGramHalf + c0, g0);
                    tmem_ld8(gaddr + half * kGramHalf + c0 + 8, g1);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 8; ++i) gram[(c0 + i) * kTileRows + row] = g0[i];
#pragma unroll
                    for (int i = 0; i < 8; ++i) gram[(c0 + 8 + i) * kTileRows + row] = g1[i];
                }
#pragma unroll
                for (int j = 0; j < MAXD; ++j)
                    if ((anc_pos[j] >> 5) == half) gsel[j] = gram[(anc_pos[j] & 31) * kTileRows + row];
            }
            tc_fence_before();
            mbar_arrive(bar(kBarGramDone));                  // the state MMAs may now overwrite these columns
            PROF_SEG(7)
            // every prep thread has written alpha / beta and converted its rows (the operand barrier
            // doubles as the prep-internal barrier)
            if (!(ok = WAIT(3, bar(kBarBReady), unit_seq & 1))) break;
#pragma unroll
            for (int j = 0; j < MAXD; ++j) anc_alpha[j] = alpha_s[anc_pos[j]];
            const float my_a = alpha_s[active ? node : 0];
            const float sgn = is_k ? -beta_s[active ? node : 0] : p.scale;
            // the coefficient buffer of this parity must have been released by the epilogue
            if (unit_seq >= 2 && !(ok = WAIT(4, bar(kBarCoefFree + par), ((unit_seq >> 1) - 1) & 1))) break;
            // coefficient record of this row's node; levels that are not ancestors stay zero, rows
            // past the last node (padding up to a multiple of 16) become no-op records
            if (in_rows) {
                float *cf = reinterpret_cast<float *>(smem + kOffCoef) + (par * MAXN + pos) * CS;
                float c[MAXD];
                float ratio = my_a;
#pragma unroll
                for (int j = MAXD - 2; j >= 0; --j) {
                    const bool is_anc = active && j < d - 1;
                    // without the erase term u_t = beta_t v_t: the key rows contribute nothing but cV
                    c[j] = (is_anc && !(is_k && p.no_erase)) ? sgn * ratio * gsel[j] : 0.f;
                    if (is_anc) ratio *= anc_alpha[j];
                }
                // after the loop ratio = gamma (product of alpha over the whole root path)
                // record: cU[MAXD-1] cV | cO[MAXD] | cR cG depth-1 offset
                if (is_k) {
                    c[MAXD - 1] = active ? -sgn : 0.f;                                // cV = beta
#pragma unroll
                    for (int i = 0; i < MAXD / 4; ++i)
                        reinterpret_cast<float4 *>(cf)[i] = make_float4(c[4 * i], c[4 * i + 1], c[4 * i + 2], c[4 * i + 3]);
                    cf[2 * MAXD] = (active && !p.no_erase) ? sgn * ratio * (COMP ? 1.f : kDebias) : 0.f;      // cR = -beta gamma
                } else {
                    // level d-1 is the node itself: (q_t . k_t) with ratio 1 (kSelfSlot: kept in the last slot)
                    c[MAXD - 1] = 0.f;
#pragma unroll
                    for (int j = 0; j < MAXD; ++j)
                        if (active && j == d - 1) c[kSelfSlot ? MAXD - 1 : j] = sgn * gsel[j];
#pragma unroll
                    for (int i = 0; i < MAXD / 4; ++i)
                        reinterpret_cast<float4 *>(cf)[MAXD / 4 + i] = make_float4(c[4 * i], c[4 * i + 1], c[4 * i + 2], c[4 * i + 3]);
                    cf[2 * MAXD + 1] = active ? sgn * ratio * (COMP ? 1.f : kDebias) : 0.f;                  // cG = scale gamma
                    // (kSelfSlot: a leaf's u is nobody's ancestor term -- level -1 keeps it out of the stack, so that the
                    // next node's sums do not wait for it)
                    cf[2 * MAXD + 2] = __int_as_float((active && !(kSelfSlot && ((meta.x >> 16) & 1))) ? d - 1 : -1);
                    cf[2 * MAXD + 3] = __int_as_float(active ? node * p.H * p.DV : 0);        // offset of the node's row
                }
            }
            mbar_arrive(bar(kBarCoefReady + par));
            PROF_SEG(7)
            // The staging buffer may be refilled now: the Gram block of this unit is complete (the
            // tensor core no longer reads the staged rows) and every prep thread has converted its rows.
            nx = x;
            const bool have_next = next_unit(walk, nx);
            if (have_next) prefetch(nx);
            PROF_SEG(6)
            x = nx;
            have = have_next;
            meta = meta_nxt;
            meta2 = meta2_nxt;
            cur_lo = node_lo; cur_hi = node_hi;
        }
        PROF_STORE()
    } else if (warp < 14) {
        // ------------------------------------------------------------- epilogue groups
        const int grp = (warp - 6) >> 2;
        const int row = 32 * (warp & 3) + lane;
        const uint32_t lane_addr = uint32_t(32 * (warp & 3)) << 16;
        const uint32_t acc = tmem_base + grp * kPairCols + lane_addr;
        const float *coef = reinterpret_cast<const float *>(smem + kOffCoef) + grp * MAXN * CS;

        // this group's units: unit_seq == grp (mod 2)
        Unit x;
        bool have = first_unit(walk, x);
        if (have && grp == 1) have = next_unit(walk, x);
        uint32_t my_seq = 0;
        bool ok = true;
        PROF_DECL
        // Two register buffers (A, B) of kEpiChunk nodes each: TMEM columns R, G and the bf16
        // value rows.  While one chunk is processed the loads of the next one are in flight.
        float RA[TP][kEpiChunk], GA[TP][kEpiChunk], RB[TP][kEpiChunk], GB[TP][kEpiChunk];
        // value rows: TP adjacent bf16 values per node, fetched with one load
        using VPack = typename std::conditional<TP == 2, uint32_t, unsigned short>::type;
        VPack vA[kEpiChunk], vB[kEpiChunk];
        const VPack *vraw = reinterpret_cast<const VPack *>(p.v);
        // value rows of the first chunk of a unit, fetched ahead (node order from the plan)
        auto fetch_first_values = [&](const Unit &y) {
            if (y.n == 0) return;                            // commit-only unit: no records to read
            const int rec0 = (y.l * p.T + y.base) * p.H + y.h;
#pragma unroll
            for (int i = 0; i < kEpiChunk; ++i) {
                const int node = i < y.n ? (__ldg(p.ws.plan + y.base + i) & 0xffff) : 0;
                vA[i] = __ldg(vraw + size_t(rec0 + node * p.H) * kTileRows + row);
            }
        };
        if (have) fetch_first_values(x);
        while (have && ok) {
            // look up this group's next unit now: its global loads overlap with this unit's work
            Unit nx = x;
            bool have_next = next_unit(walk, nx);
            if (have_next) have_next = next_unit(walk, nx);
            if (!(ok = WAIT(0, bar(kBarCoefReady + grp), my_seq & 1))) break;
            if (!(ok = WAIT(2, bar(kBarAccFull + grp), my_seq & 1))) break;
            tc_fence_after();
            const size_t rec0 = size_t((x.l * p.T + x.base) * p.H + x.h);        // record of node 0
            // this thread's TP adjacent value rows: row*TP .. row*TP + TP-1
            const VPack *v_row = vraw + rec0 * kTileRows + row;
            float *o_row = p.o + rec0 * p.DV + row * TP;
            float *u_row = p.u != nullptr ? p.u + rec0 * p.DV + row * TP : nullptr;
            float ustk[TP][MAXD];
#pragma unroll
            for (int t = 0; t < TP; ++t)
#pragma unroll
                for (int j = 0; j < MAXD; ++j) ustk[t][j] = 0.f;
            const int npad = x.npad, n = x.n;
            auto load_tmem = [&](int p0, float (&R)[TP][kEpiChunk], float (&G)[TP][kEpiChunk]) {
#pragma unroll
                for (int t = 0; t < TP; ++t) {
                    tmem_ld4(acc + t * kAccCols + p0, R[t]);
                    tmem_ld4(acc + t * kAccCols + npad + p0, G[t]);
                }
            };
            auto load_values = [&](int p0, VPack (&vv)[kEpiChunk]) {
#pragma unroll
                for (int i = 0; i < kEpiChunk; ++i) {
                    const int off = __float_as_int(coef[(p0 + i) * CS + CS - 1]);        // p0 + i < npad; in floats of o
                    vv[i] = __ldg(v_row + off / TP);
                }
                // the value rows of the chunk after this one: into L1 now, so that their loads are short
                // (a global load takes a microsecond or more while the state stream saturates HBM)
                if (p0 + kEpiChunk < n) {
#pragma unroll
                    for (int i = 0; i < kEpiChunk; ++i) {
                        const int offn = __float_as_int(coef[(p0 + kEpiChunk + i) * CS + CS - 1]);
                        asm volatile("prefetch.global.L1 [%0];" ::"l"(v_row + offn / TP));
                    }
                }
            };
            auto process = [&](int p0, const float (&R)[TP][kEpiChunk], const float (&G)[TP][kEpiChunk],
                               const VPack (&vv)[kEpiChunk]) {
#pragma unroll
                for (int i = 0; i < kEpiChunk; ++i) {
                    float r_[TP], g_[TP], v_[TP], uo[TP], oo[TP];
                    int off;
#pragma unroll
                    for (int t = 0; t < TP; ++t) {
                        r_[t] = R[t][i]; g_[t] = G[t][i];
                    }
                    if (TP == 2) {
                        v_[0] = __uint_as_float(uint32_t(vv[i]) << 16);
                        v_[TP - 1] = __uint_as_float(uint32_t(vv[i]) & 0xffff0000u);
                    } else {
                        v_[0] = __uint_as_float(uint32_t(vv[i]) << 16);
                    }
                    if constexpr (DEEP) node_step_deep<TP, MAXD, kSelfSlot>(ustk, coef + (p0 + i) * CS, r_, g_, v_, uo, oo, off);
                    else node_step<TP, kSelfSlot>(ustk, coef + (p0 + i) * CS, r_, g_, v_, uo, oo, off);
                    if (p0 + i < n) {
                        if (TP == 2) {
                            *reinterpret_cast<float2 *>(o_row + off) = make_float2(oo[0], oo[TP - 1]);
                            if (u_row != nullptr) *reinterpret_cast<float2 *>(u_row + off) = make_float2(uo[0], uo[TP - 1]);
                        } else {
                            o_row[off] = oo[0];
                            if (u_row != nullptr) u_row[off] = uo[0];
                        }
                    }
                }
            };
            // Software pipeline, one chunk deep: buffer A is processed while buffer B (the next
            // chunk's TMEM columns and value rows) is in flight; B is then moved into A.
            if (n > 0) load_tmem(0, RA, GA);
#pragma unroll 1
            for (int p0 = 0; p0 < n; p0 += kEpiChunk) {
                tmem_ld_wait();
                const bool more = p0 + kEpiChunk < n;
                if (more) { load_tmem(p0 + kEpiChunk, RB, GB); load_values(p0 + kEpiChunk, vB); }
                process(p0, RA, GA, vA);
                if (more) {
                    tmem_ld_wait();
#pragma unroll
                    for (int t = 0; t < TP; ++t)
#pragma unroll
                        for (int i = 0; i < kEpiChunk; ++i) { RA[t][i] = RB[t][i]; GA[t][i] = GB[t][i]; }
#pragma unroll
                    for (int i = 0; i < kEpiChunk; ++i) vA[i] = vB[i];
                }
            }
            tc_fence_before();
            mbar_arrive(bar(kBarPairFree + grp));
            mbar_arrive(bar(kBarCoefFree + grp));
            ++my_seq;
            x = nx;
            have = have_next;
            if (have) fetch_first_values(x);
        }
        PROF_STORE()
    } else if (FUSED) {
        // ------------------------------------------------------------- state update (fused commit)
        // The pending update of a slice, S <- gA S + W Kp (W[r][i] = (gamma_A / gamma_i) u_i[r],
        // Kp[i][c] = k_i[c], i < A <= 8), is a rank-8 product: each warp applies it to its rows
        // with warp-level m16n8k8 TF32 MMAs whose accumulator fragment is the slice itself, read
        // from and written back to the shared-memory slot.  Keys are bf16 (exact in TF32); W is
        // split into a TF32 head and tail (two MMAs), so the products carry fp32 accuracy and the
        // accumulation is fp32.  The cost does not depend on A and the only shared-memory round
        // trip per batch of rows is the slice itself.
        // The u rows and keys of the path are staged in shared memory by the TMA producer (double
        // buffered by unit); the gates are fetched here, one unit ahead, lane l keeping the gate
        // of path node l & 7.  Nothing on this role's path waits on a global load issued in the
        // same unit: under a saturated HBM such a wait costs microseconds.
        const int ut = threadIdx.x - kThreads;
        const int uw = ut >> 5;                                  // warp of the role
        const int g = lane >> 2, t4 = lane & 3;                  // MMA fragment coordinates
        const int li = lane & 7;
        constexpr int kRowsPerWarp = kTileRows / kUpdWarps, kMT = kRowsPerWarp / 16;
        const int rowbase = uw * kRowsPerWarp;
        float alpha_c = 1.f, alpha_n = 1.f;
        auto fetch_alpha = [&](const Unit &y) {
            if (y.a == 0) return;
            const int node = y.b < kWalkSeqs
                ? reinterpret_cast<const int32_t *>(smem + kOffWalk + kWalkPBase)[y.b] +
                      int(smem[kOffWalk + kWalkPNode + y.b * kMaxDepth + li])
                : __ldg(p.ws.pend + y.b * kPendWords + 9) + (li < y.a ? __ldg(p.ws.pend + y.b * kPendWords + 1 + li) : 0);
            alpha_n = li < y.a ? __ldg(p.palpha + (size_t(y.l) * p.Tp + node) * p.H + y.h) : 1.f;
        };

        uint32_t it = 0, pseq = 0;
        Unit x, nx;
        bool ok = true;
        bool have = first_unit(walk, x);
        if (have) { fetch_alpha(x); alpha_c = alpha_n; }
        PROF_DECL
        while (have && ok) {
            const int A = x.a;
            const int pb = pseq & 1;
            PROF_MARK()
            // my_ratio = product of alpha over the path nodes after node li; gA over all of them
            float my_ratio = 1.f, gA = 1.f;
#pragma unroll
            for (int j = 0; j < kMaxDepth; ++j) {
                const float aj = __shfl_sync(0xffffffffu, alpha_c, j);
                if (j < A) {
                    gA *= aj;
                    if (j > li) my_ratio *= aj;
                }
            }
            const float ratio0 = __shfl_sync(0xffffffffu, my_ratio, t4), ratio1 = __shfl_sync(0xffffffffu, my_ratio, t4 + 4);
            PROF_SEG(1)
            nx = x;
            const bool have_next = next_unit(walk, nx);
            if (have_next) fetch_alpha(nx);
            PROF_SEG(2)
            // the staged u rows and keys of this unit have landed
            if (A > 0 && !(ok = WAIT(3, bar(kBarPendFull + pb), (pseq >> 1) & 1))) break;
            const float *ub = reinterpret_cast<const float *>(smem + kOffPendU + pb * kPendUBuf);
            for (int t = 0; t < TP && ok; ++t) {
                // A fragments of this tile, W = ratio * u: [m][0..3] = (row g, node t4), (row g + 8, node t4),
                // (row g, node t4 + 4), (row g + 8, node t4 + 4) of m-tile m; zero past the end of the path
                float w[kMT][4];
#pragma unroll
                for (int m = 0; m < kMT; ++m) {
                    const int r0 = (rowbase + 16 * m + g) * TP + t, r1 = r0 + 8 * TP;
                    const float *u0 = ub + t4 * (kPendUStride / 4), *u1 = ub + (t4 + 4) * (kPendUStride / 4);
                    const float x0 = u0[r0], x1 = u0[r1], x2 = u1[r0], x3 = u1[r1];
                    w[m][0] = t4 < A ? ratio0 * x0 : 0.f;
                    w[m][1] = t4 < A ? ratio0 * x1 : 0.f;
                    w[m][2] = t4 + 4 < A ? ratio1 * x2 : 0.f;
                    w[m][3] = t4 + 4 < A ? ratio1 * x3 : 0.f;
                }
                PROF_SEG(4)
                for (int c = 0; c < NC; ++c, ++it) {
                    const int s = it % NS;
                    const uint32_t ph = (it / NS) & 1;
                    if (!(ok = WAIT(0, bar(kBarFull + s), ph))) break;
                    PROF_MARK()
                    if (A > 0) {
                        uint8_t *slot = smem + kOffRing + s * kStageBytes;
                        // B fragments: keys t4 and t4 + 4 at column 8 n + g of this chunk
                        const uint8_t *kb = smem + key_buf(pb) + (c * kChunkK + g) * 2;
                        uint32_t b0[4], b1[4];
#pragma unroll
                        for (int n = 0; n < 4; ++n) {
                            const uint32_t lo = *reinterpret_cast<const unsigned short *>(kb + t4 * KSTRIDE + n * 16);
                            const uint32_t hi = *reinterpret_cast<const unsigned short *>(kb + (t4 + 4) * KSTRIDE + n * 16);
                            b0[n] = t4 < A ? lo << 16 : 0u;
                            b1[n] = t4 + 4 < A ? hi << 16 : 0u;
                        }
#pragma unroll
                        for (int mb = 0; mb < kMT; mb += 2) {
                            // accumulator fragments of two m-tiles: rows R, R + 8; columns 8 n + 2 t4, + 1
                            float cf[2][4][4];
#pragma unroll
                            for (int m2 = 0; m2 < 2; ++m2) {
                                const int R = rowbase + 16 * (mb + m2) + g;
#pragma unroll
                                for (int n = 0; n < 4; ++n) {
                                    const uint32_t off = ((uint32_t(2 * n + (t4 >> 1)) ^ uint32_t(R & 7)) << 4) | uint32_t((t4 & 1) * 8);
                                    const float2 v0 = *reinterpret_cast<const float2 *>(slot + R * 128 + off);
                                    const float2 v1 = *reinterpret_cast<const float2 *>(slot + (R + 8) * 128 + off);
                                    cf[m2][n][0] = v0.x; cf[m2][n][1] = v0.y; cf[m2][n][2] = v1.x; cf[m2][n][3] = v1.y;
                                }
                            }
#pragma unroll
                            for (int m2 = 0; m2 < 2; ++m2) {
                                uint32_t ah[4], al[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float wv = w[mb + m2][e];
                                    ah[e] = __float_as_uint(wv) & 0xffffe000u;
                                    al[e] = __float_as_uint(wv - __uint_as_float(ah[e]));
                                }
#pragma unroll
                                for (int n = 0; n < 4; ++n) {
#pragma unroll
                                    for (int e = 0; e < 4; ++e) cf[m2][n][e] *= gA;
                                    mma_tf32_sync(cf[m2][n], ah, b0[n], b1[n]);
                                    mma_tf32_sync(cf[m2][n], al, b0[n], b1[n]);
                                }
                            }
#pragma unroll
                            for (int m2 = 0; m2 < 2; ++m2) {
                                const int R = rowbase + 16 * (mb + m2) + g;
#pragma unroll
                                for (int n = 0; n < 4; ++n) {
                                    const uint32_t off = ((uint32_t(2 * n + (t4 >> 1)) ^ uint32_t(R & 7)) << 4) | uint32_t((t4 & 1) * 8);
                                    *reinterpret_cast<float2 *>(slot + R * 128 + off) = make_float2(cf[m2][n][0], cf[m2][n][1]);
                                    *reinterpret_cast<float2 *>(slot + (R + 8) * 128 + off) = make_float2(cf[m2][n][2], cf[m2][n][3]);
                                }
                            }
                        }
                        PROF_SEG(5)
                        fence_proxy_async();                 // the tensor core and the TMA store read this slice
                    }
                    mbar_arrive(bar(kBarUpd + s));
                    PROF_SEG(7)
                    PROF_SEG(6)
                }
            }
            // the staged rows may be refilled
            if (A > 0) { mbar_arrive(bar(kBarPendFree + pb)); ++pseq; }
            x = nx;
            have = have_next;
            alpha_c = alpha_n;
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


}  // namespace

bool factorized_supported(const speca_dims *d)
{
    if (d->d_k != kDK && d->d_k != 2 * kDK) return false;
    if (d->d_v != kTileRows && d->d_v != 2 * kTileRows) return false;
    // trees of at most 8 levels: 64 nodes per sequence at d_k = 128, 32 at d_k = 256; up to 16 levels: 32 nodes
    if (d->max_depth <= kMaxDepth) return d->max_nodes <= (d->d_k == kDK ? kMaxNodes : kMaxNodes / 2);
    return d->max_depth <= 2 * kMaxDepth && d->max_nodes <= kMaxNodes / 2;
}

bool factorized_fused_supported(const speca_dims *d) { return factorized_supported(d) && d->max_depth <= kMaxDepth; }

namespace {

struct DeviceState { int sm_count; bool attr_set; };
DeviceState g_device[64] = {};
int g_withhold_first_load = 0;

template <int TP, bool FUSED, int DK, bool DEEP, bool COMP>
cudaError_t opt_in_smem()
{
    return cudaFuncSetAttribute(verify_factorized_kernel<TP, FUSED, DK, DEEP, COMP>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

template <bool FUSED, bool DEEP, bool COMP>
void launch_one(bool one_tile, int d_k, int grid, cudaStream_t st, const CUtensorMap &map, const KQMaps &kq, const FParams &fp)
{
    constexpr int threads = FUSED ? kThreadsFused : (COMP ? kThreadsComp : kThreads);
    if (d_k == kDK) {
        if (one_tile) verify_factorized_kernel<1, FUSED, 128, DEEP, COMP><<<grid, threads, kSmemBytes, st>>>(map, kq, fp);
        else verify_factorized_kernel<2, FUSED, 128, DEEP, COMP><<<grid, threads, kSmemBytes, st>>>(map, kq, fp);
    } else {
        if (one_tile) verify_factorized_kernel<1, FUSED, 256, DEEP, COMP><<<grid, threads, kSmemBytes, st>>>(map, kq, fp);
        else verify_factorized_kernel<2, FUSED, 256, DEEP, COMP><<<grid, threads, kSmemBytes, st>>>(map, kq, fp);
    }
}

}  // namespace

namespace {

struct MapKey {
    const void *s, *q, *k, *v;
    long units;
    int L, T, H, DV, dk;
    bool operator==(const MapKey &o) const
    {
        return s == o.s && q == o.q && k == o.k && v == o.v && units == o.units && L == o.L && T == o.T && H == o.H &&
               DV == o.DV && dk == o.dk;
    }
};
struct MapSet { CUtensorMap state; KQMaps kq; };
// last kSets distinct (pointers, shape) keys, replaced round robin; a handful of entries, searched linearly
class MapCache {
public:
    bool find(const MapKey &key, MapSet &out)
    {
        std::lock_guard<std::mutex> lock(mu_);
        for (int i = 0; i < kSets; ++i)
            if (used_[i] && keys_[i] == key) { out = sets_[i]; return true; }
        return false;
    }
    void insert(const MapKey &key, const MapSet &set)
    {
        std::lock_guard<std::mutex> lock(mu_);
        keys_[next_] = key; sets_[next_] = set; used_[next_] = true;
        next_ = (next_ + 1) % kSets;
    }
private:
    static constexpr int kSets = 16;
    std::mutex mu_;
    MapKey keys_[kSets];
    MapSet sets_[kSets];
    bool used_[kSets] = {};
    int next_ = 0;
};
MapCache g_map_cache;

int launch_with_maps(const Params &p, int d_k, bool fused, bool comp, cudaStream_t st, long n_units, const CUtensorMap &map,
                     const KQMaps &kq);

}  // namespace

// Test hook of the failure-detection test (not part of the public header): with `on` the producer of CTA 0
// never requests its first state slice, so that CTA's bounded waits run out and the call reports
// SPECA_STATUS_TIMEOUT.  Plain (non-fused) verification only.
void factorized_set_withhold(int on) { g_withhold_first_load = on; }

// comp: the compensated (fp32-grade) form; fused: commit-and-verify in one pass (single TF32 pass only).
int launch_verify_factorized(const Params &p, int d_k, bool fused, bool comp, cudaStream_t st)
{
    if (d_k != kDK && d_k != 2 * kDK) return int(cudaErrorInvalidValue);
    if (fused && comp) return int(cudaErrorInvalidValue);
    EncodeTiledFn encode = encode_tiled_fn();
    if (encode == nullptr) return int(cudaErrorNotSupported);
    const long n_units = long(p.L) * p.B * p.H;
    // The 13 tensor maps depend only on the four base pointers and the shape: a serving loop calls with the same
    // ones round after round, so the last few sets are kept (a map holds addresses and strides, nothing of the data).
    const MapKey key{p.S0, p.q, p.k, p.v, n_units, p.L, p.T, p.H, p.DV, d_k};
    MapSet cached;
    if (g_map_cache.find(key, cached)) return launch_with_maps(p, d_k, fused, comp, st, n_units, cached.state, cached.kq);
    CUtensorMap map;
    const int tiles = p.DV / kTileRows;
    const cuuint64_t gdim[3] = {cuuint64_t(d_k), cuuint64_t(tiles), cuuint64_t(n_units) * kTileRows};
    const cuuint64_t gstride[2] = {cuuint64_t(d_k) * sizeof(float), cuuint64_t(tiles) * d_k * sizeof(float)};
    const cuuint32_t box[3] = {kChunkK, 1, kTileRows};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(p.S0), gdim, gstride, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return int(cudaErrorInvalidValue);

    KQMaps kq;
    {
        const cuuint64_t gd[3] = {cuuint64_t(d_k), cuuint64_t(p.H), cuuint64_t(p.L) * cuuint64_t(p.T)};
        const cuuint64_t gs[2] = {cuuint64_t(d_k) * 2, cuuint64_t(p.H) * d_k * 2};
        const cuuint32_t es[3] = {1, 1, 1};
        for (int m = 0; m < 4; ++m) {
            const cuuint32_t bx[3] = {64, 1, cuuint32_t(16 * (m + 1))};
            CUresult r1 = encode(&kq.k[m], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16 *>(p.k), gd, gs, bx,
                                 es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            CUresult r2 = encode(&kq.q[m], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16 *>(p.q), gd, gs, bx,
                                 es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r1 != CUDA_SUCCESS || r2 != CUDA_SUCCESS) return int(cudaErrorInvalidValue);
            const cuuint64_t vd[3] = {cuuint64_t(p.DV), cuuint64_t(p.H), cuuint64_t(p.L) * cuuint64_t(p.T)};
            const cuuint64_t vs[2] = {cuuint64_t(p.DV) * 2, cuuint64_t(p.H) * p.DV * 2};
            const cuuint32_t vb[3] = {cuuint32_t(p.DV), 1, cuuint32_t(16 * (m + 1))};
            CUresult r3 = encode(&kq.v[m], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16 *>(p.v), vd, vs, vb,
                                 es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r3 != CUDA_SUCCESS) return int(cudaErrorInvalidValue);
        }
    }

    g_map_cache.insert(key, MapSet{map, kq});
    return launch_with_maps(p, d_k, fused, comp, st, n_units, map, kq);
}

namespace {

int launch_with_maps(const Params &p, int d_k, bool fused, bool comp, cudaStream_t st, long n_units, const CUtensorMap &map,
                     const KQMaps &kq)
{
    // the SM count and the opt-in to large dynamic shared memory belong to a device, not to the process
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return int(cudaErrorInvalidDevice);
    DeviceState &ds = g_device[dev];
    if (ds.sm_count == 0) {
        int n = 0;
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        ds.sm_count = n > 0 ? n : 148;
    }
    if (!ds.attr_set) {
        cudaError_t e[] = {
            opt_in_smem<1, false, 128, false, false>(), opt_in_smem<2, false, 128, false, false>(),
            opt_in_smem<1, false, 256, false, false>(), opt_in_smem<2, false, 256, false, false>(),
            opt_in_smem<1, true, 128, false, false>(),  opt_in_smem<2, true, 128, false, false>(),
            opt_in_smem<1, true, 256, false, false>(),  opt_in_smem<2, true, 256, false, false>(),
            opt_in_smem<1, false, 128, true, false>(),  opt_in_smem<2, false, 128, true, false>(),
            opt_in_smem<1, false, 256, true, false>(),  opt_in_smem<2, false, 256, true, false>(),
            opt_in_smem<1, false, 128, false, true>(),  opt_in_smem<2, false, 128, false, true>(),
            opt_in_smem<1, false, 256, false, true>(),  opt_in_smem<2, false, 256, false, true>(),
            opt_in_smem<1, false, 128, true, true>(),   opt_in_smem<2, false, 128, true, true>(),
            opt_in_smem<1, false, 256, true, true>(),   opt_in_smem<2, false, 256, true, true>()};
        for (cudaError_t x : e)
            if (x != cudaSuccess) return int(x);
        ds.attr_set = true;
    }
    FParams fp;
    fp.p = p;
    fp.n_units = n_units;
    fp.withhold_first_load = g_withhold_first_load;
    // consecutive heads of one (layer, sequence) a CTA takes together: as many as divide H while
    // every SM still gets a group
    fp.heads_per_group = 1;
    for (int hg = 4; hg > 1; hg >>= 1)
        if (p.H % hg == 0 && n_units / hg >= ds.sm_count) { fp.heads_per_group = hg; break; }
    const long n_groups = n_units / fp.heads_per_group;
    const int grid = int(n_groups < ds.sm_count ? n_groups : ds.sm_count);
    const bool one_tile = p.DV == kTileRows;
    const bool deep = p.max_depth > kMaxDepth;
    if (fused) launch_one<true, false, false>(one_tile, d_k, grid, st, map, kq, fp);
    else if (comp && deep) launch_one<false, true, true>(one_tile, d_k, grid, st, map, kq, fp);
    else if (comp) launch_one<false, false, true>(one_tile, d_k, grid, st, map, kq, fp);
    else if (deep) launch_one<false, true, false>(one_tile, d_k, grid, st, map, kq, fp);
    else launch_one<false, false, false>(one_tile, d_k, grid, st, map, kq, fp);
    return int(cudaGetLastError());
}

}  // namespace

}  // namespace speca
