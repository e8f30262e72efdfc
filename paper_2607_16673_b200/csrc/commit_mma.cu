// Commit of long accepted paths on warp-level tensor-core MMAs (Section 5.1 factor buffering, Eq. 3;
// Section 5.2 immediate update).
//
// The token-by-token commit costs three fp32 FMAs per state element and accepted node, each node's
// update waiting for the previous one's row reduction: beyond about four nodes the arithmetic, not
// HBM, sets its speed.  For a path of A nodes (4 <= A <= 8) the same result is, per state row r,
//        R[r][i] = S0[r,:] . k_i                                          (one product with all keys)
//        u_i[r]  = beta_i v_i[r] - beta_i gamma_i R[r][i] - sum_{j<i} beta_i (gamma_i/gamma_j) (k_j.k_i) u_j[r]
//        S_A     = gamma_A S0 + sum_j (gamma_A/gamma_j) u_j k_j^T         (one rank-A update)
// with gamma_i the product of alpha over nodes 0..i -- the unrolled recurrence of Section 4.2 on a
// chain.  The two dense products run as mma.sync m16n8k8 TF32 with the fp32 operand (S0, then
// W = ratio * u) split into its TF32 head and the exact remainder (two MMAs; keys are bf16 and exact
// in TF32), so products carry fp32 accuracy; the recurrence in between is scalar work per row.
//
// One warp owns a 16-row tile with the full key width.  The contraction index of the first product
// and the output column of the second are both free to permute, so the state stays in the registers
// it was loaded into (coalesced 128-bit loads: lane (g, t) holds rows g and g + 8, the 16-byte
// chunks t, t + 4, ...) through both products and is stored from the same registers.  Key fragments
// in that permuted order are built once per work item in warp-private shared memory; the Gram block
// of the keys falls out of the same fragments.  Sequences with shorter (or longer) paths are left to
// the token-by-token kernel, which skips the ones taken here.
#include <atomic>

#include "speca_common.cuh"
#include "tc_ptx.cuh"

namespace speca {

namespace {

using tc::mma_tf32_sync;

constexpr int kCtasPerSm = 4;                // 128 registers per thread: the state tile alone takes 64
constexpr int kLongMax = 8;                  // path lengths [long_min, kLongMax] are taken here
constexpr int kWarps = 4;
constexpr int kListCap = 2048;               // sequences whose indices the per-CTA list can hold

__device__ __forceinline__ uint32_t tf32_head(float x) { return __float_as_uint(x) & 0xffffe000u; }
__device__ __forceinline__ uint32_t tf32_tail(float x) { return __float_as_uint(x - __uint_as_float(tf32_head(x))); }

template <int DK>
__global__ void __launch_bounds__(kWarps * 32, kCtasPerSm)
commit_long_kernel(Params p)
{
    constexpr int NME = DK / 8;              // permuted k-steps of the first product = column blocks of the second
    constexpr int NM = DK / 16;              // 16-byte chunks of a row per lane
    __shared__ uint16_t s_long[kListCap];
    __shared__ int s_nlong;
    __shared__ __align__(16) float2 s_tab1[kWarps][NME][32];
    __shared__ __align__(16) float2 s_tab2[kWarps][NME][32];
    __shared__ __align__(16) float s_cf[kWarps][kLongMax][12];     // per node i: C[i][0..7], cR, beta, ratio to the end, -

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;

    // the sequences this kernel takes, in index order (every CTA builds the same list)
    if (warp == 0) {
        int count = 0;
        for (int b0 = 0; b0 < p.B; b0 += 32) {
            const int b = b0 + lane;
            const int len = b < p.B ? __ldg(p.path_len + b) : 0;
            const bool take = len >= p.long_min && len <= kLongMax && len <= p.max_depth;
            const unsigned m = __ballot_sync(0xffffffffu, take);
            if (take) s_long[count + __popc(m & ((1u << lane) - 1u))] = uint16_t(b);
            count += __popc(m);
        }
        if (lane == 0) s_nlong = count;
    }
    __syncthreads();
    // Rows per work item: the whole value dimension (the per-item set-up is then paid once per unit) when the
    // sequences taken here give every warp several items, fewer 16-row tiles otherwise.
    const int n_warps = gridDim.x * kWarps;
    int passes = p.DV / 16;
    while (passes > 1 && (passes & 1) == 0 && long(s_nlong) * p.L * p.H * (p.DV / 16 / passes) < 4L * n_warps) passes >>= 1;
    const int parts = p.DV / (16 * passes);
    const long total = long(s_nlong) * p.L * p.H * parts;

    float2(*tab1)[32] = s_tab1[warp];
    float2(*tab2)[32] = s_tab2[warp];
    float(*cf)[12] = s_cf[warp];

    for (long item = long(blockIdx.x) * kWarps + warp; item < total; item += n_warps) {
        const int part = int(item % parts);
        long rest = item / parts;
        const int h = int(rest % p.H); rest /= p.H;
        const int l = int(rest % p.L);
        const int b = s_long[rest / p.L];
        const int len = __ldg(p.path_len + b);
        const int base = __ldg(p.node_offsets + b);
        const int n = __ldg(p.node_offsets + b + 1) - base;

        // validate the path as the token-by-token kernel does; a bad path leaves the state untouched
        int fault = 0;
        long rec = 0;
        if (base < 0 || n < 0 || base + n > p.T) fault = SPECA_STATUS_BAD_OFFSETS;
        else if (lane < len) {
            const int node = __ldg(p.path_idx + b * p.max_depth + lane);
            const int prev = lane > 0 ? __ldg(p.path_idx + b * p.max_depth + lane - 1) : -1;
            if (node < 0 || node >= n) fault = SPECA_STATUS_BAD_PATH;
            else if (p.parent != nullptr && __ldg(p.parent + base + node) != prev) fault = SPECA_STATUS_BAD_PATH;
            rec = (long(l) * p.T + base + node) * p.H + h;
        }
        const unsigned bad = __ballot_sync(0xffffffffu, fault != 0);
        if (bad) {
            if (l == 0 && h == 0 && part == 0 && lane == __ffs(bad) - 1) atomicOr(p.status, fault);
            continue;
        }
        const float alpha = lane < len ? __ldg(p.alpha + rec) : 1.f;
        const float beta = lane < len ? __ldg(p.beta + rec) : 0.f;

        // key fragments in the permuted order, and the Gram block of the keys from the same values
        const long rec_g = __shfl_sync(0xffffffffu, rec, g);
        const long rec_t = __shfl_sync(0xffffffffu, rec, t), rec_t4 = __shfl_sync(0xffffffffu, rec, t + 4);
        float gram[4] = {0.f, 0.f, 0.f, 0.f};
        __syncwarp();                                        // the previous item's reads of the tables are done
#pragma unroll
        for (int me = 0; me < NME; ++me) {
            const int m = me >> 1, e = me & 1;
            uint32_t w = 0;
            if (g < len) w = __ldg(reinterpret_cast<const uint32_t *>(p.k + rec_g * DK + 4 * (t + 4 * m) + 2 * e));
            const uint32_t b0 = w << 16, b1 = w & 0xffff0000u;
            tab1[me][lane] = make_float2(__uint_as_float(b0), __uint_as_float(b1));
            const uint32_t a[4] = {b0, 0u, b1, 0u};
            mma_tf32_sync(gram, a, b0, b1);
            const int col2 = 4 * ((g >> 1) + 4 * m) + 2 * e + (g & 1);
            const unsigned short x0 = t < len ? __ldg(reinterpret_cast<const unsigned short *>(p.k + rec_t * DK + col2)) : 0;
            const unsigned short x1 = t + 4 < len ? __ldg(reinterpret_cast<const unsigned short *>(p.k + rec_t4 * DK + col2)) : 0;
            tab2[me][lane] = make_float2(__uint_as_float(uint32_t(x0) << 16), __uint_as_float(uint32_t(x1) << 16));
        }
        // coefficient rows: lane i (< 8) builds row i from the Gram entries k_j . k_i, which sit in lanes
        // (j, i / 2) as gram[i & 1]
        float gA = 1.f;
        {
            float c[kLongMax];
            float ratio = alpha;                             // gamma_i / gamma_j for j = i - 1, then further down
#pragma unroll
            for (int j = kLongMax - 2; j >= 0; --j) {
                const float e0 = __shfl_sync(0xffffffffu, gram[0], 4 * j + (lane >> 1) % 4);
                const float e1 = __shfl_sync(0xffffffffu, gram[1], 4 * j + (lane >> 1) % 4);
                const float a_j = __shfl_sync(0xffffffffu, alpha, j);
                const bool is_prev = j < lane && lane < len;
                c[j] = (is_prev && !p.no_erase) ? beta * ratio * ((lane & 1) ? e1 : e0) : 0.f;
                if (j < lane) ratio *= a_j;
            }
            c[kLongMax - 1] = 0.f;
            // ratio is now gamma_i; the ratio from node i to the end of the path is the product of the later alphas
            float tail = 1.f;
#pragma unroll
            for (int j = kLongMax - 1; j >= 1; --j) {
                const float a_j = __shfl_sync(0xffffffffu, alpha, j);
                if (j > lane) tail *= a_j;
                gA *= a_j;
            }
            gA *= __shfl_sync(0xffffffffu, alpha, 0);
            if (lane < kLongMax) {
                *reinterpret_cast<float4 *>(&cf[lane][0]) = make_float4(c[0], c[1], c[2], c[3]);
                *reinterpret_cast<float4 *>(&cf[lane][4]) = make_float4(c[4], c[5], c[6], c[7]);
                *reinterpret_cast<float4 *>(&cf[lane][8]) =
                    make_float4((lane < len && !p.no_erase) ? beta * ratio : 0.f, beta, lane < len ? tail : 0.f, 0.f);
            }
        }
        __syncwarp();

        const bool low = t < 2;                              // lanes t = 0, 1 carry row g through the recurrence, t = 2, 3 row g + 8
        for (int pass = 0; pass < passes; ++pass) {
            const int row0 = (part * passes + pass) * 16;
            float *Su = p.S + ((long(l) * p.B + b) * p.H + h) * long(p.DV) * DK;
            float4 sa[NM], sb[NM];
#pragma unroll
            for (int m = 0; m < NM; ++m) {
                sa[m] = __ldcs(reinterpret_cast<const float4 *>(Su + long(row0 + g) * DK) + t + 4 * m);
                sb[m] = __ldcs(reinterpret_cast<const float4 *>(Su + long(row0 + g + 8) * DK) + t + 4 * m);
            }
            const int my_row = row0 + (low ? g : g + 8);
            float vv[kLongMax];
#pragma unroll
            for (int i = 0; i < kLongMax; ++i) {
                const long rec_i = __shfl_sync(0xffffffffu, rec, i);
                vv[i] = i < len ? __uint_as_float(uint32_t(__ldg(reinterpret_cast<const unsigned short *>(p.v + rec_i * p.DV + my_row))) << 16)
                                : 0.f;
            }
            // R = S0 K^T
            // (four accumulation chains, so that consecutive MMAs do not wait for one another)
            float R[4] = {0.f, 0.f, 0.f, 0.f}, R1[4] = {0.f, 0.f, 0.f, 0.f}, R2[4] = {0.f, 0.f, 0.f, 0.f}, R3[4] = {0.f, 0.f, 0.f, 0.f};
            if (!p.no_erase) {
#pragma unroll
                for (int me = 0; me < NME; ++me) {
                    const int m = me >> 1;
                    const float2 kb = tab1[me][lane];
                    const float x0 = (me & 1) ? sa[m].z : sa[m].x, x2 = (me & 1) ? sa[m].w : sa[m].y;
                    const float x1 = (me & 1) ? sb[m].z : sb[m].x, x3 = (me & 1) ? sb[m].w : sb[m].y;
                    const uint32_t hi[4] = {tf32_head(x0), tf32_head(x1), tf32_head(x2), tf32_head(x3)};
                    const uint32_t lo[4] = {tf32_tail(x0), tf32_tail(x1), tf32_tail(x2), tf32_tail(x3)};
                    mma_tf32_sync((me & 1) ? R1 : R, hi, __float_as_uint(kb.x), __float_as_uint(kb.y));
                    mma_tf32_sync((me & 1) ? R3 : R2, lo, __float_as_uint(kb.x), __float_as_uint(kb.y));
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) R[i] = (R[i] + R1[i]) + (R2[i] + R3[i]);
            }
            // this lane's row of R: nodes 2s, 2s + 1 come from lane s of the quad
            float Rr[kLongMax];
#pragma unroll
            for (int s = 0; s < 4; ++s) {
                const int src = (lane & ~3) | s;
                const float p0 = __shfl_sync(0xffffffffu, R[0], src), p1 = __shfl_sync(0xffffffffu, R[1], src);
                const float p2 = __shfl_sync(0xffffffffu, R[2], src), p3 = __shfl_sync(0xffffffffu, R[3], src);
                Rr[2 * s] = low ? p0 : p2;
                Rr[2 * s + 1] = low ? p1 : p3;
            }
            // the recurrence along the path, then W = ratio * u
            float u[kLongMax];
#pragma unroll
            for (int i = 0; i < kLongMax; ++i) {
                const float4 c0 = *reinterpret_cast<const float4 *>(&cf[i][0]), c1 = *reinterpret_cast<const float4 *>(&cf[i][4]);
                const float4 sc = *reinterpret_cast<const float4 *>(&cf[i][8]);
                const float c[kLongMax] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
                float acc = fmaf(sc.y, vv[i], -sc.x * Rr[i]);
#pragma unroll
                for (int j = 0; j < i; ++j) acc = fmaf(-c[j], u[j], acc);
                u[i] = acc;
            }
#pragma unroll
            for (int i = 0; i < kLongMax; ++i) u[i] *= cf[i][10];
            // A fragment of the update: W[g][t], W[g+8][t], W[g][t+4], W[g+8][t+4]; the other row's come from lane t ^ 2
            const int tp = t ^ 2;
            float own_a = u[0], own_b = u[4], oth_a = u[0], oth_b = u[4];
#pragma unroll
            for (int i = 1; i < 4; ++i) {
                own_a = t == i ? u[i] : own_a; own_b = t == i ? u[i + 4] : own_b;
                oth_a = tp == i ? u[i] : oth_a; oth_b = tp == i ? u[i + 4] : oth_b;
            }
            const float got_a = __shfl_xor_sync(0xffffffffu, oth_a, 2), got_b = __shfl_xor_sync(0xffffffffu, oth_b, 2);
            const float w0 = low ? own_a : got_a, w1 = low ? got_a : own_a, w2 = low ? own_b : got_b, w3 = low ? got_b : own_b;
            const uint32_t whi[4] = {tf32_head(w0), tf32_head(w1), tf32_head(w2), tf32_head(w3)};
            const uint32_t wlo[4] = {tf32_tail(w0), tf32_tail(w1), tf32_tail(w2), tf32_tail(w3)};
            // S_A = gamma_A S0 + W K, column block by column block, in the registers the state was loaded into
#pragma unroll
            for (int me = 0; me < NME; ++me) {
                const int m = me >> 1;
                const float2 kb = tab2[me][lane];
                float acc[4];
                if (me & 1) { acc[0] = gA * sa[m].z; acc[1] = gA * sa[m].w; acc[2] = gA * sb[m].z; acc[3] = gA * sb[m].w; }
                else { acc[0] = gA * sa[m].x; acc[1] = gA * sa[m].y; acc[2] = gA * sb[m].x; acc[3] = gA * sb[m].y; }
                mma_tf32_sync(acc, whi, __float_as_uint(kb.x), __float_as_uint(kb.y));
                mma_tf32_sync(acc, wlo, __float_as_uint(kb.x), __float_as_uint(kb.y));
                if (me & 1) { sa[m].z = acc[0]; sa[m].w = acc[1]; sb[m].z = acc[2]; sb[m].w = acc[3]; }
                else { sa[m].x = acc[0]; sa[m].y = acc[1]; sb[m].x = acc[2]; sb[m].y = acc[3]; }
            }
#pragma unroll
            for (int m = 0; m < NM; ++m) {
                __stcs(reinterpret_cast<float4 *>(Su + long(row0 + g) * DK) + t + 4 * m, sa[m]);
                __stcs(reinterpret_cast<float4 *>(Su + long(row0 + g + 8) * DK) + t + 4 * m, sb[m]);
            }
        }
    }
}

// Batch size from which the second launch pays: its tail (about 25 us) against what the long paths save (about a
// seventh of their own time, for the third or so of the sequences that accept four nodes or more), i.e. from about
// half a millisecond of commit on -- 128 16-row tiles per resident warp.
constexpr int kMinTilesPerWarp = 128;
std::atomic<int> g_min_tiles_per_warp{kMinTilesPerWarp};

// SM count per device (asked once per device)
int sm_count_of_current_device()
{
    static std::atomic<int> cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    const bool cached = dev >= 0 && dev < 64;
    int sms = cached ? cache[dev].load(std::memory_order_relaxed) : 0;
    if (sms == 0) {
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        if (cached) cache[dev].store(sms, std::memory_order_relaxed);
    }
    return sms;
}

}  // namespace

// Shapes and sizes the long-path kernel takes; everything else stays with the token-by-token kernel.  A small batch
// is latency, not throughput: there one kernel with a CTA per tile is quicker than two launches and a per-item set-up.
bool commit_long_supported(const Params &p, int d_k)
{
    if (!((d_k == 64 || d_k == 128) && p.DV % 16 == 0 && p.B <= kListCap)) return false;
    const long tiles = long(p.L) * p.B * p.H * (p.DV / 16);
    return tiles >= long(g_min_tiles_per_warp.load(std::memory_order_relaxed)) * sm_count_of_current_device() * kCtasPerSm * kWarps;
}

// Test hook: 16-row tiles per resident warp from which the long-path kernel is used (0: always, where the shape fits).
void commit_long_set_min_tiles_per_warp(int n) { g_min_tiles_per_warp.store(n < 0 ? kMinTilesPerWarp : n, std::memory_order_relaxed); }

int launch_commit_long(const Params &p, int d_k, cudaStream_t st)
{
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return int(cudaErrorInvalidDevice);
    const int grid = sms * kCtasPerSm;
    if (d_k == 64) commit_long_kernel<64><<<grid, kWarps * 32, 0, st>>>(p);
    else commit_long_kernel<128><<<grid, kWarps * 32, 0, st>>>(p);
    return int(cudaGetLastError());
}

}  // namespace speca
