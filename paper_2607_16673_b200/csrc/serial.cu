// State-resident serial kernels: single-token decode, serial chain / tree verification
// and commit.  All three keep a value-tile of the fp32 state in registers with the
// full key dimension inside the CTA (V-dimension tiling, Section 4.1), so a row's dot
// products with k and q never leave a sub-warp and there is no cross-block reduction.
//
// Thread mapping.  A row of d_k floats is spread over G = d_k/16 adjacent lanes, each
// holding 16 floats as four float4 taken at stride G (so a sub-warp reads a row with
// fully coalesced 128-bit loads).  One warp covers 32/G rows per "row set" and RS row
// sets; k and q are converted from bf16 once per node per lane.  The two row dot
// products S_p k and S_p q are taken in ONE pass over the registers, then
//        u = beta (v - alpha S_p k),   o = scale (alpha S_p q + u (k.q)),   S = alpha S_p + u k^T
// which is the rule of Section 2.2 with o read from the updated state.  Leaves of a
// draft tree need no state update at all.
#include "speca_common.cuh"

namespace speca {

namespace {

template <int DK> struct Map {
    static constexpr int G = DK / 16;          // lanes per row
    static constexpr int RPS = 32 / G;         // rows per warp per row set
};

template <int G> __device__ __forceinline__ float group_sum(float x)
{
#pragma unroll
    for (int off = G / 2; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
}

// 16 of a row's d_k values for this lane, from a bf16 vector in global memory.
// The 16 values a lane holds of a row are kept as 8 float2 so that the arithmetic can use the
// packed two-wide fp32 instructions of sm_100 (each lane of a pair is an ordinary IEEE fp32 op).
template <int G> __device__ __forceinline__ void load_vec(const __nv_bfloat16 *p, int g, float2 (&x)[8])
{
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(p) + g + G * c);
        x[2 * c + 0] = make_float2(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u));
        x[2 * c + 1] = make_float2(__uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u));
    }
}

template <int G> __device__ __forceinline__ void load_row(const float *row, int g, float2 (&s)[8])
{
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const float4 t = *(reinterpret_cast<const float4 *>(row) + g + G * c);
        s[2 * c + 0] = make_float2(t.x, t.y);
        s[2 * c + 1] = make_float2(t.z, t.w);
    }
}

template <int G> __device__ __forceinline__ void store_row(float *row, int g, const float2 (&s)[8])
{
#pragma unroll
    for (int c = 0; c < 4; ++c)
        *(reinterpret_cast<float4 *>(row) + g + G * c) =
            make_float4(s[2 * c + 0].x, s[2 * c + 0].y, s[2 * c + 1].x, s[2 * c + 1].y);
}

__device__ __forceinline__ float dot16(const float2 (&a)[8], const float2 (&b)[8])
{
    float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 8; i += 2) { acc0 = __ffma2_rn(a[i], b[i], acc0); acc1 = __ffma2_rn(a[i + 1], b[i + 1], acc1); }
    const float2 acc = __fadd2_rn(acc0, acc1);
    return acc.x + acc.y;
}

// s <- alpha s + u k   (the rank-1 write of the rule)
__device__ __forceinline__ void axpy16(float2 (&s)[8], const float2 (&k)[8], float alpha, float u)
{
    const float2 a2 = make_float2(alpha, alpha), u2 = make_float2(u, u);
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] = __ffma2_rn(a2, s[i], __fmul2_rn(u2, k[i]));
}

__device__ __forceinline__ float bf16_to_float(const __nv_bfloat16 *p)
{
    return __uint_as_float(uint32_t(__ldg(reinterpret_cast<const unsigned short *>(p))) << 16);
}

// ---------------------------------------------------------------------------
// decode step: S in place, one token per sequence
// ---------------------------------------------------------------------------
template <int DK, int RS, int WARPS>
__global__ void __launch_bounds__(WARPS * 32)
decode_kernel(Params p)
{
    constexpr int G = Map<DK>::G, RPS = Map<DK>::RPS, ROWS = WARPS * RS * RPS;
    const int tiles = p.DV / ROWS;
    const long unit = blockIdx.x / tiles;                       // (l*B + b)*H + h == record index (T == B)
    const int row0 = (blockIdx.x % tiles) * ROWS + (threadIdx.x >> 5) * RS * RPS;
    const int lane = threadIdx.x & 31, g = lane % G, sub = lane / G;

    float *Su = p.S + unit * p.DV * DK;
    float2 s[RS][8];
#pragma unroll
    for (int r = 0; r < RS; ++r) load_row<G>(Su + long(row0 + r * RPS + sub) * DK, g, s[r]);
    float2 kx[8], qx[8];
    load_vec<G>(p.k + unit * DK, g, kx);
    load_vec<G>(p.q + unit * DK, g, qx);
    const float alpha = __ldg(p.alpha + unit), beta = __ldg(p.beta + unit);
    const float kq = group_sum<G>(dot16(kx, qx));
#pragma unroll
    for (int r = 0; r < RS; ++r) {
        const int row = row0 + r * RPS + sub;
        const float sk = group_sum<G>(dot16(s[r], kx));
        const float sq = group_sum<G>(dot16(s[r], qx));
        const float vv = bf16_to_float(p.v + unit * p.DV + row);
        const float u = p.no_erase ? beta * vv : beta * (vv - alpha * sk);
        axpy16(s[r], kx, alpha, u);
        store_row<G>(Su + long(row) * DK, g, s[r]);
        if (g == 0) p.o[unit * p.DV + row] = p.scale * fmaf(alpha, sq, u * kq);
    }
}

// ---------------------------------------------------------------------------
// serial verification (chain: nodes in index order; tree: plan order with slots)
// ---------------------------------------------------------------------------
template <int DK, int RS, int WARPS, bool CHAIN>
__global__ void __launch_bounds__(WARPS * 32)
verify_serial_kernel(Params p)
{
    constexpr int G = Map<DK>::G, RPS = Map<DK>::RPS, ROWS = WARPS * RS * RPS;
    extern __shared__ float4 slot_mem[];                         // [n_slots][ROWS][DK] floats
    const int tiles = p.DV / ROWS;
    const long unit = blockIdx.x / tiles;
    const int h = int(unit % p.H), b = int((unit / p.H) % p.B), l = int(unit / (long(p.H) * p.B));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane % G, sub = lane / G;
    const int row0 = (blockIdx.x % tiles) * ROWS + warp * RS * RPS;

    const int base = __ldg(p.node_offsets + b);
    int n;
    if (CHAIN) {
        n = __ldg(p.node_offsets + b + 1) - base;
        int fault = 0;
        if (base < 0 || n < 0 || base + n > p.T) fault = SPECA_STATUS_BAD_OFFSETS;
        else if (n > p.max_nodes) fault = SPECA_STATUS_TOO_MANY;
        else if (n > p.max_depth) fault = SPECA_STATUS_TOO_DEEP;      // a chain of n nodes is n levels deep, on every route
        if (fault) {
            if (threadIdx.x == 0 && blockIdx.x % tiles == 0 && h == 0 && l == 0) atomicOr(p.status, fault);
            return;
        }
    } else {
        n = p.ws.seq_n[b];
    }
    if (n <= 0) return;

    const float *S0u = p.S0 + unit * p.DV * DK;
    float2 s[RS][8];
#pragma unroll
    for (int r = 0; r < RS; ++r) load_row<G>(S0u + long(row0 + r * RPS + sub) * DK, g, s[r]);
    float *my_slot = reinterpret_cast<float *>(slot_mem) + size_t(warp) * RS * RPS * DK;
    const size_t slot_stride = size_t(ROWS) * DK;

    for (int j = 0; j < n; ++j) {
        int t = j, load = 0, save = 0;
        bool leaf = (j == n - 1);
        if (!CHAIN) {
            const int e = __ldg(p.ws.plan + base + j);
            t = e & 0xffff;
            load = (e >> kPlanLoadShift) & 15;
            save = (e >> kPlanSaveShift) & 15;
            leaf = (e & kPlanLeafBit) != 0;
            if (load == kLoadFromS0) {
#pragma unroll
                for (int r = 0; r < RS; ++r) load_row<G>(S0u + long(row0 + r * RPS + sub) * DK, g, s[r]);
            } else if (load) {
                const float *src = my_slot + slot_stride * (load - 1);
#pragma unroll
                for (int r = 0; r < RS; ++r) load_row<G>(src + (r * RPS + sub) * DK, g, s[r]);
            }
        }
        const long rec = (long(l) * p.T + base + t) * p.H + h;
        float2 kx[8], qx[8];
        load_vec<G>(p.k + rec * DK, g, kx);
        load_vec<G>(p.q + rec * DK, g, qx);
        const float alpha = __ldg(p.alpha + rec), beta = __ldg(p.beta + rec);
        const float kq = group_sum<G>(dot16(kx, qx));
#pragma unroll
        for (int r = 0; r < RS; ++r) {
            const int row = row0 + r * RPS + sub;
            const float sk = group_sum<G>(dot16(s[r], kx));
            const float sq = group_sum<G>(dot16(s[r], qx));
            const float vv = bf16_to_float(p.v + rec * p.DV + row);
            const float u = p.no_erase ? beta * vv : beta * (vv - alpha * sk);
            if (!leaf) axpy16(s[r], kx, alpha, u);
            if (g == 0) {
                p.o[rec * p.DV + row] = p.scale * fmaf(alpha, sq, u * kq);
                if (p.u != nullptr) p.u[rec * p.DV + row] = u;
            }
        }
        if (!CHAIN && save) {
            float *dst = my_slot + slot_stride * (save - 1);
#pragma unroll
            for (int r = 0; r < RS; ++r) store_row<G>(dst + (r * RPS + sub) * DK, g, s[r]);
        }
    }
}

// ---------------------------------------------------------------------------
// commit: advance S in place over the accepted factor records
// ---------------------------------------------------------------------------
template <int DK, int RS, int WARPS>
__global__ void __launch_bounds__(WARPS * 32, 2048 / (WARPS * 32) / 2)
commit_kernel(Params p)
{
    constexpr int G = Map<DK>::G, RPS = Map<DK>::RPS, ROWS = WARPS * RS * RPS;
    const int tiles = p.DV / ROWS;
    const long unit = blockIdx.x / tiles;
    const int h = int(unit % p.H), b = int((unit / p.H) % p.B), l = int(unit / (long(p.H) * p.B));
    const int lane = threadIdx.x & 31, g = lane % G, sub = lane / G;
    const int row0 = (blockIdx.x % tiles) * ROWS + (threadIdx.x >> 5) * RS * RPS;

    // path_len == 0: the sequence's state is neither read nor written
    const int len = __ldg(p.path_len + b);
    const int base = __ldg(p.node_offsets + b);
    const int n = __ldg(p.node_offsets + b + 1) - base;
    if (len == 0) return;
    // paths the tensor-core commit takes (it validates them itself)
    if (p.long_min > 0 && len >= p.long_min && len <= 8 && len <= p.max_depth) return;

    // Start streaming the state tile right away; the accepted path is validated in the
    // shadow of these loads (one thread per path step), and nothing is stored if it is bad.
    float *Su = p.S + unit * p.DV * DK;
    float2 s[RS][8];
    const bool len_ok = len > 0 && len <= p.max_depth;
    if (len_ok) {
#pragma unroll
        for (int r = 0; r < RS; ++r) load_row<G>(Su + long(row0 + r * RPS + sub) * DK, g, s[r]);
    }
    // The factor records of the whole accepted path (k rows, alpha, beta, the tile's v values)
    // are staged in shared memory while the state tile is in flight, so that the token-by-token
    // recurrence below never waits on global memory.
    __shared__ int s_path[16];
    __shared__ __align__(16) __nv_bfloat16 s_k[16][DK];
    __shared__ float s_alpha[16], s_beta[16];
    __shared__ __nv_bfloat16 s_v[16][ROWS];
    int fault = 0;
    if (!len_ok) fault = SPECA_STATUS_TOO_DEEP;
    else if (base < 0 || n < 0 || base + n > p.T) fault = SPECA_STATUS_BAD_OFFSETS;
    else {
        if (int(threadIdx.x) < len) {
            const int d = threadIdx.x;
            const int t = __ldg(p.path_idx + b * p.max_depth + d);
            const int prev = d > 0 ? __ldg(p.path_idx + b * p.max_depth + d - 1) : -1;
            if (t < 0 || t >= n) fault = SPECA_STATUS_BAD_PATH;
            else if (p.parent != nullptr && __ldg(p.parent + base + t) != prev) fault = SPECA_STATUS_BAD_PATH;
            s_path[d] = t;
            if (!fault) {
                const long rec = (long(l) * p.T + base + t) * p.H + h;
                s_alpha[d] = __ldg(p.alpha + rec);
                s_beta[d] = __ldg(p.beta + rec);
            }
        }
        constexpr int PIECES = DK / 8;                       // 16-byte pieces per k row
        const int row_base = (blockIdx.x % tiles) * ROWS;
        for (int idx = threadIdx.x; idx < len * PIECES; idx += WARPS * 32) {
            const int d = idx / PIECES, piece = idx % PIECES;
            const int t = __ldg(p.path_idx + b * p.max_depth + d);
            if (t >= 0 && t < n) {
                const long rec = (long(l) * p.T + base + t) * p.H + h;
                const uint32_t dst = uint32_t(__cvta_generic_to_shared(&s_k[d][piece * 8]));
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(p.k + rec * DK + piece * 8)
                             : "memory");
            }
        }
        for (int idx = threadIdx.x; idx < len * ROWS; idx += WARPS * 32) {
            const int d = idx / ROWS, r = idx % ROWS;
            const int t = __ldg(p.path_idx + b * p.max_depth + d);
            if (t >= 0 && t < n) {
                const long rec = (long(l) * p.T + base + t) * p.H + h;
                s_v[d][r] = p.v[rec * p.DV + row_base + r];
            }
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    }
    fault = __syncthreads_or(fault);
    if (fault) {
        // report one of the faults seen by the CTA (BAD_PATH is the only per-thread one)
        if (threadIdx.x == 0 && blockIdx.x % tiles == 0 && h == 0 && l == 0)
            atomicOr(p.status, !len_ok ? SPECA_STATUS_TOO_DEEP
                                       : ((base < 0 || n < 0 || base + n > p.T) ? SPECA_STATUS_BAD_OFFSETS
                                                                                : SPECA_STATUS_BAD_PATH));
        return;
    }

    const int tile_row = (threadIdx.x >> 5) * RS * RPS + sub;        // row inside the CTA's tile (row set 0)
    for (int d = 0; d < len; ++d) {
        float2 kx[8];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint2 raw = *(reinterpret_cast<const uint2 *>(&s_k[d][0]) + g + G * c);
            kx[2 * c + 0] = make_float2(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u));
            kx[2 * c + 1] = make_float2(__uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u));
        }
        const float alpha = s_alpha[d], beta = s_beta[d];
#pragma unroll
        for (int r = 0; r < RS; ++r) {
            const float sk = group_sum<G>(dot16(s[r], kx));
            const float vv = __bfloat162float(s_v[d][tile_row + r * RPS]);
            const float u = p.no_erase ? beta * vv : beta * (vv - alpha * sk);
            axpy16(s[r], kx, alpha, u);
        }
    }
#pragma unroll
    for (int r = 0; r < RS; ++r) store_row<G>(Su + long(row0 + r * RPS + sub) * DK, g, s[r]);
}

// Rows covered by one CTA for a given d_k: the largest of {32,16,8,4,2} rows (RS in
// {2,1}) that divides d_v is chosen by the launchers below.
template <int DK, int RS, int WARPS> constexpr int rows_per_cta() { return WARPS * RS * Map<DK>::RPS; }

template <int DK, template <int, int, int> class Launch>
int pick_tile(const Params &p, cudaStream_t st)
{
    // prefer 2 row sets x 4 warps; fall back to smaller tiles when d_v is not a multiple
    if (p.DV % rows_per_cta<DK, 2, 4>() == 0) return Launch<DK, 2, 4>::run(p, st);
    if (p.DV % rows_per_cta<DK, 2, 2>() == 0) return Launch<DK, 2, 2>::run(p, st);
    if (p.DV % rows_per_cta<DK, 1, 2>() == 0) return Launch<DK, 1, 2>::run(p, st);
    if (p.DV % rows_per_cta<DK, 1, 1>() == 0) return Launch<DK, 1, 1>::run(p, st);
    return int(cudaErrorInvalidValue);
}

inline long n_units(const Params &p) { return long(p.L) * p.B * p.H; }

template <int DK, int RS, int WARPS> struct LaunchDecode {
    static int run(const Params &p, cudaStream_t st)
    {
        const long blocks = n_units(p) * (p.DV / rows_per_cta<DK, RS, WARPS>());
        decode_kernel<DK, RS, WARPS><<<unsigned(blocks), WARPS * 32, 0, st>>>(p);
        return int(cudaGetLastError());
    }
};

template <int DK, int RS, int WARPS> struct LaunchCommit {
    static int run(const Params &p, cudaStream_t st)
    {
        const long blocks = n_units(p) * (p.DV / rows_per_cta<DK, RS, WARPS>());
        commit_kernel<DK, RS, WARPS><<<unsigned(blocks), WARPS * 32, 0, st>>>(p);
        return int(cudaGetLastError());
    }
};

template <int DK, int RS, int WARPS> struct LaunchChain {
    static int run(const Params &p, cudaStream_t st)
    {
        const long blocks = n_units(p) * (p.DV / rows_per_cta<DK, RS, WARPS>());
        verify_serial_kernel<DK, RS, WARPS, true><<<unsigned(blocks), WARPS * 32, 0, st>>>(p);
        return int(cudaGetLastError());
    }
};

template <int DK, int RS, int WARPS> struct LaunchTree {
    static int run(const Params &p, cudaStream_t st)
    {
        constexpr int ROWS = rows_per_cta<DK, RS, WARPS>();
        const long blocks = n_units(p) * (p.DV / ROWS);
        const size_t smem = size_t(p.n_slots) * ROWS * DK * sizeof(float);
        auto kern = verify_serial_kernel<DK, RS, WARPS, false>;
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
            if (e != cudaSuccess) return int(e);
        }
        kern<<<unsigned(blocks), WARPS * 32, smem, st>>>(p);
        return int(cudaGetLastError());
    }
};

// The tree walk parks whole tiles on chip, so it uses a smaller tile (2 warps) to keep
// several CTAs resident per SM.
template <int DK>
int pick_tree_tile(const Params &p, cudaStream_t st)
{
    if (p.DV % rows_per_cta<DK, 2, 2>() == 0) return LaunchTree<DK, 2, 2>::run(p, st);
    if (p.DV % rows_per_cta<DK, 1, 2>() == 0) return LaunchTree<DK, 1, 2>::run(p, st);
    if (p.DV % rows_per_cta<DK, 1, 1>() == 0) return LaunchTree<DK, 1, 1>::run(p, st);
    return int(cudaErrorInvalidValue);
}

}  // namespace

int launch_decode(const Params &p, int d_k, cudaStream_t st)
{
    switch (d_k) {
    case 64: return pick_tile<64, LaunchDecode>(p, st);
    case 128: return pick_tile<128, LaunchDecode>(p, st);
    case 256: return pick_tile<256, LaunchDecode>(p, st);
    }
    return int(cudaErrorInvalidValue);
}

// Accepted paths of kCommitLongMin nodes or more go to the tensor-core kernel where it takes the shape: from there
// on the token-by-token form is bound by its arithmetic, not by HBM.
constexpr int kCommitLongMin = 4;

int launch_commit(const Params &p_in, int d_k, cudaStream_t st)
{
    Params p = p_in;
    p.long_min = (p.max_depth >= kCommitLongMin && commit_long_supported(p, d_k)) ? kCommitLongMin : 0;
    if (p.long_min > 0) {
        const int rc = launch_commit_long(p, d_k, st);
        if (rc != 0) return rc;
    }
    switch (d_k) {
    case 64: return pick_tile<64, LaunchCommit>(p, st);
    case 128: return pick_tile<128, LaunchCommit>(p, st);
    case 256: return pick_tile<256, LaunchCommit>(p, st);
    }
    return int(cudaErrorInvalidValue);
}

int launch_verify_serial(const Params &p, int d_k, bool chain, cudaStream_t st)
{
    if (chain) {
        switch (d_k) {
        case 64: return pick_tile<64, LaunchChain>(p, st);
        case 128: return pick_tile<128, LaunchChain>(p, st);
        case 256: return pick_tile<256, LaunchChain>(p, st);
        }
    } else {
        switch (d_k) {
        case 64: return pick_tree_tile<64>(p, st);
        case 128: return pick_tree_tile<128>(p, st);
        case 256: return pick_tree_tile<256>(p, st);
        }
    }
    return int(cudaErrorInvalidValue);
}

}  // namespace speca
