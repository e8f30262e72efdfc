// Integer kernels: topology validation + walk schedule ("plan"), and greedy acceptance.
//
// The plan is computed once per verify call and shared by every layer, head and
// value tile of a sequence.  It turns the parent-pointer array (Section 4.2) into a
// depth-first processing order in which, at every node, children are visited in
// ascending order of subtree size.  This is the heavy-path idea of the
// chain-decomposed schedule (Section 4.3) used as a traversal order: the state of a
// branching node is parked on chip only while its lighter subtrees are walked and is
// released when its heaviest child starts, so a handful of slots suffice and no
// boundary state ever goes to HBM.
#include "speca_common.cuh"

namespace speca {

namespace {

constexpr int kPlanThreads = 128;

// One CTA per sequence.  Dynamic smem: 6 int32 arrays of max_nodes (+1).
__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(const int32_t *__restrict__ node_offsets, const int32_t *__restrict__ parent,
            const int32_t *__restrict__ depth_in, int32_t B, int32_t T, int32_t max_depth,
            int32_t max_nodes, int32_t n_slots, Workspace ws, int32_t *status)
{
    extern __shared__ int32_t sm[];
    const int b = blockIdx.x;
    const int tid = threadIdx.x;
    __shared__ int32_t s_flag;

    if (b == 0 && tid < 64) ws.ctrl[tid] = 0;          // reset the work-queue counters
    const int base = node_offsets[b];
    const int n = node_offsets[b + 1] - base;
    int fault = 0;
    if (base < 0 || n < 0 || base + n > T || (b == B - 1 && base + n != T) || (b == 0 && base != 0))
        fault = SPECA_STATUS_BAD_OFFSETS;
    else if (n > max_nodes)
        fault = SPECA_STATUS_TOO_MANY;
    if (fault) {
        if (tid == 0) { atomicOr(status, fault); ws.seq_n[b] = -1; }
        return;
    }
    int32_t *par = sm;                       // [n]
    int32_t *size = par + max_nodes;         // [n]   subtree size
    int32_t *bef = size + max_nodes;         // [n]   total size of siblings visited before this node
    int32_t *nlc = bef + max_nodes;          // [n+1] children with children, index shifted by one (slot 0 = committed state)
    int32_t *ldf = nlc + max_nodes + 1;      // [n]   1 if an earlier sibling has children (register state lost)
    int32_t *posn = ldf + max_nodes;         // [n]   position of node i in the processing order

    if (tid == 0) s_flag = 0;
    for (int i = tid; i < n; i += kPlanThreads) { size[i] = 0; nlc[i + 1] = 0; }
    if (tid == 0) nlc[0] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += kPlanThreads) {
        int p = parent != nullptr ? parent[base + i] : i - 1;      // no parent array: chain
        par[i] = p;
        if (p < -1 || p >= i) atomicOr(&s_flag, SPECA_STATUS_BAD_PARENT);
    }
    __syncthreads();
    if (s_flag) {
        if (tid == 0) { atomicOr(status, s_flag); ws.seq_n[b] = -1; }
        return;
    }
    // depth and subtree sizes: every node adds itself to all nodes on its root path
    for (int i = tid; i < n; i += kPlanThreads) {
        int d = 0;
        for (int a = i; a >= 0; a = par[a]) { atomicAdd(&size[a], 1); ++d; }
        ws.depth[base + i] = d;
        if (d > max_depth) atomicOr(&s_flag, SPECA_STATUS_TOO_DEEP);
        if (depth_in != nullptr && depth_in[base + i] != d) atomicOr(&s_flag, SPECA_STATUS_BAD_DEPTH);
    }
    __syncthreads();
    if (s_flag) {
        if (tid == 0) { atomicOr(status, s_flag); ws.seq_n[b] = -1; }
        return;
    }
    for (int i = tid; i < n; i += kPlanThreads) {
        const int p = par[i], sz = size[i];
        if (sz > 1) atomicAdd(&nlc[p + 1], 1);
        int before = 0, lost = 0;
        for (int s = 0; s < n; ++s) {
            if (s == i || par[s] != p) continue;
            const int ss = size[s];
            if (ss < sz || (ss == sz && s < i)) { before += ss; lost |= (ss > 1); }
        }
        bef[i] = before;
        ldf[i] = lost;
    }
    __syncthreads();
    for (int i = tid; i < n; i += kPlanThreads) {
        int pos = -1, slot = 0, first = 0;
        for (int c = i; c >= 0; c = par[c]) {
            pos += 1 + bef[c];
            const int a = par[c];
            if (a >= 0 && nlc[a + 1] >= 2 && bef[c] + size[c] != size[a] - 1) {
                ++slot;                                   // a's parked state is live while we are below c
                if (c == i) first = 1;
            }
        }
        const int leaf = (size[i] == 1);
        int entry = i;
        if (ldf[i]) {
            const int p = par[i];
            entry |= (p < 0 ? kLoadFromS0 : 1 + (slot - first)) << kPlanLoadShift;
        }
        if (!leaf && nlc[i + 1] >= 2) {
            entry |= (1 + slot) << kPlanSaveShift;
            if (1 + slot > n_slots) atomicOr(&s_flag, SPECA_STATUS_TOO_MANY);
        }
        if (leaf) entry |= kPlanLeafBit;
        ws.plan[base + pos] = entry;
        posn[i] = pos;
    }
    __syncthreads();
    // Per node: depth, position in the processing order, a leaf flag, and the node's ancestors by depth
    // (one byte each; meaningful for sequences of <= 256 nodes and depth <= 16, which is all
    // the factorised route accepts).  Level j (0 = child of the committed state) of the first
    // record sits in byte j % 4 of word 1 + j / 4 for j < 12; levels 12..14 are in the second.
    for (int i = tid; i < n; i += kPlanThreads) {
        int d = 0;
        for (int a = i; a >= 0; a = par[a]) ++d;
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        int j = d - 1;
        for (int a = par[i]; a >= 0; a = par[a]) {
            --j;
            if (j < 16) w[j >> 2] |= (uint32_t(a) & 0xffu) << (8 * (j & 3));
        }
        int4 rec, rec2;
        rec.x = d | (posn[i] << 8) | (size[i] == 1 ? 1 << 16 : 0);         // bit 16: leaf (its u is nobody's ancestor term)
        rec.y = int(w[0]);
        rec.z = int(w[1]);
        rec.w = int(w[2]);
        rec2.x = int(w[3]);
        rec2.y = rec2.z = rec2.w = 0;
        reinterpret_cast<int4 *>(ws.anc)[base + i] = rec;
        reinterpret_cast<int4 *>(ws.anc2)[base + i] = rec2;
    }
    __syncthreads();
    if (tid == 0) {
        if (s_flag) { atomicOr(status, s_flag); ws.seq_n[b] = -1; }
        else ws.seq_n[b] = n;
    }
}

// One warp per sequence.  Each lane takes nodes t = lane, lane+32, ... and walks t's
// root path checking every token against the prediction made at its parent.
__global__ void __launch_bounds__(128)
accept_kernel(int32_t B, int32_t max_depth, const int32_t *__restrict__ node_offsets,
              const int32_t *__restrict__ parent, const int32_t *__restrict__ draft_tok,
              const int32_t *__restrict__ target_tok, const int32_t *__restrict__ root_target_tok,
              int32_t *__restrict__ path_idx, int32_t *__restrict__ path_len,
              int32_t *__restrict__ next_tok, int32_t *status)
{
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (b >= B) return;
    const int base = node_offsets[b];
    const int n = node_offsets[b + 1] - base;
    const int root_pred = root_target_tok[b];
    int fault = 0;
    if (base < 0 || n < 0) fault = SPECA_STATUS_BAD_OFFSETS;
    // best = (depth << 16) | (0xffff - index): max picks the deepest, then the lowest index
    int best = -1;
    if (!fault) {
        for (int t = lane; t < n; t += 32) {
            int d = 0, ok = 1;
            for (int a = t; a >= 0;) {
                const int p = parent[base + a];
                if (p < -1 || p >= a) { fault |= SPECA_STATUS_BAD_PARENT; ok = 0; break; }
                const int pred = (p < 0) ? root_pred : target_tok[base + p];
                if (draft_tok[base + a] != pred) { ok = 0; break; }
                if (++d > max_depth) { fault |= SPECA_STATUS_TOO_DEEP; ok = 0; break; }
                a = p;
            }
            if (ok && t <= 0xffff) best = max(best, (d << 16) | (0xffff - t));
        }
    }
    if (n > 0x10000) fault |= SPECA_STATUS_TOO_MANY;
    for (int off = 16; off; off >>= 1) {
        best = max(best, __shfl_xor_sync(0xffffffffu, best, off));
        fault |= __shfl_xor_sync(0xffffffffu, fault, off);
    }
    if (lane != 0) return;
    if (fault) {                       // skip the sequence: nothing accepted
        atomicOr(status, fault);
        best = -1;
    }
    const int len = best < 0 ? 0 : (best >> 16);
    int node = best < 0 ? -1 : 0xffff - (best & 0xffff);
    path_len[b] = len;
    next_tok[b] = (node < 0) ? root_pred : target_tok[base + node];
    for (int d = max_depth - 1; d >= 0; --d) {
        if (d < len) { path_idx[b * max_depth + d] = node; node = parent[base + node]; }
        else path_idx[b * max_depth + d] = -1;
    }
}

// Stochastic posterior selection given per-node probabilities: one warp per sequence.
// Node t passes its own test iff uniform[t] * p_draft[t] < p_target[t] (uniform < min(1, p/q),
// written without the division; one fp32 product and one comparison).  From the committed state
// the walk takes, among the children of the current node in ascending index, the first that
// passes, and stops when none does.  A node is therefore on the accepted path iff it and all
// its ancestors are "chosen": passing, with no passing sibling of lower index.
__global__ void __launch_bounds__(128)
stochastic_accept_kernel(int32_t B, int32_t max_depth, const int32_t *__restrict__ node_offsets,
                         const int32_t *__restrict__ parent, const float *__restrict__ p_target,
                         const float *__restrict__ p_draft, const float *__restrict__ uniform,
                         int32_t *__restrict__ path_idx, int32_t *__restrict__ path_len, int32_t *status)
{
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (b >= B) return;
    const int base = node_offsets[b];
    const int n = node_offsets[b + 1] - base;
    int fault = 0;
    if (base < 0 || n < 0) fault = SPECA_STATUS_BAD_OFFSETS;
    if (n > 0x10000) fault |= SPECA_STATUS_TOO_MANY;
    auto passes = [&](int t) { return __fmul_rn(uniform[base + t], p_draft[base + t]) < p_target[base + t]; };
    int best = -1;                     // (depth << 16) | (0xffff - index) of the deepest node whose root path is all chosen
    if (!fault) {
        for (int t = lane; t < n; t += 32) {
            int d = 0, ok = 1;
            for (int a = t; a >= 0;) {
                const int pa = parent[base + a];
                if (pa < -1 || pa >= a) { fault |= SPECA_STATUS_BAD_PARENT; ok = 0; break; }
                if (!passes(a)) { ok = 0; break; }
                // a lower-index sibling that passes is taken instead
                for (int s2 = pa + 1; s2 < a; ++s2)
                    if (parent[base + s2] == pa && passes(s2)) { ok = 0; break; }
                if (!ok) break;
                if (++d > max_depth) { fault |= SPECA_STATUS_TOO_DEEP; ok = 0; break; }
                a = pa;
            }
            if (ok) best = max(best, (d << 16) | (0xffff - t));
        }
    }
    for (int off = 16; off; off >>= 1) {
        best = max(best, __shfl_xor_sync(0xffffffffu, best, off));
        fault |= __shfl_xor_sync(0xffffffffu, fault, off);
    }
    if (lane != 0) return;
    if (fault) {                       // skip the sequence: nothing accepted
        atomicOr(status, fault);
        best = -1;
    }
    const int len = best < 0 ? 0 : (best >> 16);
    int node = best < 0 ? -1 : 0xffff - (best & 0xffff);
    path_len[b] = len;
    for (int d = max_depth - 1; d >= 0; --d) {
        if (d < len) { path_idx[b * max_depth + d] = node; node = parent[base + node]; }
        else path_idx[b * max_depth + d] = -1;
    }
}

// Pending accepted paths of the fused commit-and-verify call, one thread per sequence:
// the same checks the stand-alone commit makes (length, node range, parent chain when the
// parent array is given), plus a node count within max_nodes.  A bad path is reported and
// recorded with length 0, so the sequence's state is not advanced; a good one is stored as
// local node indices (words 1..8) and the sequence's offset in the previous draft's packed
// arrays (word 9).
__global__ void __launch_bounds__(128)
pending_check_kernel(int32_t B, int32_t Tp, int32_t max_depth, int32_t max_len, int32_t max_nodes,
                     const int32_t *__restrict__ pnode_offsets, const int32_t *__restrict__ pparent,
                     const int32_t *__restrict__ path_idx, const int32_t *__restrict__ path_len,
                     int32_t *__restrict__ pend, int32_t *status)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int32_t *rec = pend + b * kPendWords;
    const int len = path_len[b];
    const int base = pnode_offsets[b];
    const int n = pnode_offsets[b + 1] - base;
    int fault = 0;
    if (len < 0 || len > max_depth || len > max_len) fault = SPECA_STATUS_TOO_DEEP;
    else if (len > 0 && (base < 0 || n < 0 || base + n > Tp)) fault = SPECA_STATUS_BAD_OFFSETS;
    else if (len > 0 && n > max_nodes) fault = SPECA_STATUS_TOO_MANY;
    int prev = -1;
    for (int d = 0; d < len && !fault; ++d) {
        const int t = path_idx[b * max_depth + d];
        if (t < 0 || t >= n) fault = SPECA_STATUS_BAD_PATH;
        else if (pparent != nullptr && pparent[base + t] != prev) fault = SPECA_STATUS_BAD_PATH;
        if (!fault) rec[1 + d] = t;
        prev = t;
    }
    if (fault) atomicOr(status, fault);
    rec[0] = fault ? 0 : len;
    rec[9] = base;
}

// Convolution-state commit: one CTA per (layer, sequence), a thread per 8 channels.  A thread reads the
// W rows that make up the new register (old rows and accepted inputs) into registers, then writes them,
// so the in-place update never reads a row it has already overwritten.
constexpr int kConvMaxWidth = 8;
__global__ void __launch_bounds__(256)
conv_commit_kernel(int32_t B, int32_t channels, int32_t W, int32_t T, int32_t max_depth, uint4 *__restrict__ C,
                   const uint4 *__restrict__ x, const int32_t *__restrict__ node_offsets,
                   const int32_t *__restrict__ path_idx, const int32_t *__restrict__ path_len, int32_t *status)
{
    const int l = blockIdx.x / B, b = blockIdx.x % B;
    const int A = path_len[b];
    if (A == 0) return;
    const int base = node_offsets[b], n = node_offsets[b + 1] - base;
    int fault = 0;
    if (A < 0 || A > max_depth) fault = SPECA_STATUS_TOO_DEEP;
    else if (base < 0 || n < 0 || base + n > T) fault = SPECA_STATUS_BAD_OFFSETS;
    else
        for (int d = 0; d < A; ++d) {
            const int t = path_idx[b * max_depth + d];
            if (t < 0 || t >= n) fault = SPECA_STATUS_BAD_PATH;
        }
    if (fault) {
        if (threadIdx.x == 0 && l == 0) atomicOr(status, fault);
        return;
    }
    const int vec = channels / 8;                       // 16-byte pieces per row
    uint4 *Cb = C + (size_t(l) * B + b) * W * vec;
    for (int c = threadIdx.x; c < vec; c += blockDim.x) {
        uint4 row[kConvMaxWidth];
#pragma unroll
        for (int w = 0; w < kConvMaxWidth; ++w) {
            if (w < W) {
                const int s = A + w;                    // index in (old rows, accepted rows); the last W are kept
                if (s < W) row[w] = Cb[s * vec + c];
                else row[w] = __ldg(x + (size_t(l) * T + base + path_idx[b * max_depth + (s - W)]) * vec + c);
            }
        }
#pragma unroll
        for (int w = 0; w < kConvMaxWidth; ++w)
            if (w < W) Cb[w * vec + c] = row[w];
    }
}

// Proposal converter: tree attention mask -> parent array.  One CTA per sequence, thread i owns node i:
// its parent is the strict ancestor with the most ancestors of its own.  The mask is checked to be the mask
// of a tree in topological order (self bit set, no later node among the ancestors, parent exactly one
// level up); otherwise the sequence gets STATUS_BAD_PARENT and its parents are left untouched.
__global__ void __launch_bounds__(256)
mask_to_parent_kernel(int32_t N, const uint8_t *__restrict__ mask, const int32_t *__restrict__ node_offsets,
                      int32_t *__restrict__ parent, int32_t *status)
{
    extern __shared__ int32_t sm[];                     // [N] ancestors-or-self per node, [N] parent
    __shared__ int32_t s_flag;
    const int b = blockIdx.x;
    const int base = node_offsets[b], n = node_offsets[b + 1] - base;
    if (threadIdx.x == 0) s_flag = 0;
    __syncthreads();
    if (n < 0 || n > N) {
        if (threadIdx.x == 0) atomicOr(status, n < 0 ? SPECA_STATUS_BAD_OFFSETS : SPECA_STATUS_TOO_MANY);
        return;
    }
    const uint8_t *m = mask + size_t(b) * N * N;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        int cnt = 0, bad = m[size_t(i) * N + i] == 0;
        for (int j = 0; j < n; ++j) {
            const int on = m[size_t(i) * N + j] != 0;
            cnt += on;
            bad |= on && j > i;
        }
        sm[i] = cnt;
        if (bad) atomicOr(&s_flag, 1);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        int best = -1;
        for (int j = 0; j < n; ++j)
            if (j != i && m[size_t(i) * N + j] != 0 && (best < 0 || sm[j] > sm[best])) best = j;
        if (best >= 0 ? sm[best] != sm[i] - 1 : sm[i] != 1) atomicOr(&s_flag, 1);
        sm[N + i] = best;
    }
    __syncthreads();
    if (s_flag) {
        if (threadIdx.x == 0) atomicOr(status, SPECA_STATUS_BAD_PARENT);
        return;
    }
    for (int i = threadIdx.x; i < n; i += blockDim.x) parent[base + i] = sm[N + i];
}

// Heavy-light chain decomposition (Section 4.3): one CTA per sequence, thread i owns node i.  The heavy
// child of a node is its child with the largest subtree (lowest index on ties); a node continues its
// parent's chain iff it is that heavy child, otherwise it heads a chain of its own (so does every child
// of the committed state).  Subtree sizes are integer sums over ancestor walks, the heavy child an
// integer maximum: both are exact whatever the order of the atomics.
__global__ void __launch_bounds__(256)
chain_decompose_kernel(int32_t N, const int32_t *__restrict__ node_offsets, const int32_t *__restrict__ parent,
                       int32_t *__restrict__ chain_head, int32_t *__restrict__ n_chains, int32_t *status)
{
    extern __shared__ int32_t sm[];                     // [N] subtree size, [N] key of the heavy child
    __shared__ int32_t s_flag, s_count;
    const int b = blockIdx.x;
    const int base = node_offsets[b], n = node_offsets[b + 1] - base;
    if (threadIdx.x == 0) { s_flag = 0; s_count = 0; }
    __syncthreads();
    if (n < 0 || n > N || n > 0x10000) {
        if (threadIdx.x == 0) {
            atomicOr(status, n < 0 ? SPECA_STATUS_BAD_OFFSETS : SPECA_STATUS_TOO_MANY);
            n_chains[b] = 0;
        }
        return;
    }
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        sm[i] = 1;
        sm[N + i] = -1;
        const int pa = parent[base + i];
        if (pa < -1 || pa >= i) atomicOr(&s_flag, 1);
    }
    __syncthreads();
    if (s_flag) {
        if (threadIdx.x == 0) { atomicOr(status, SPECA_STATUS_BAD_PARENT); n_chains[b] = 0; }
        return;
    }
    for (int i = threadIdx.x; i < n; i += blockDim.x)
        for (int a = parent[base + i]; a >= 0; a = parent[base + a]) atomicAdd(&sm[a], 1);
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int pa = parent[base + i];
        if (pa >= 0) atomicMax(&sm[N + pa], (sm[i] << 16) | (0xffff - i));       // largest subtree, then lowest index
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        int h = i;
        for (;;) {
            const int pa = parent[base + h];
            if (pa < 0 || 0xffff - (sm[N + pa] & 0xffff) != h) break;            // h heads its chain
            h = pa;
        }
        chain_head[base + i] = h;
        if (h == i) atomicAdd(&s_count, 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) n_chains[b] = s_count;
}

// Confidence-guided pruning, step 1: one CTA per sequence selects its nodes and writes them, already
// re-indexed, at the sequence's INPUT offset; out_offsets[b + 1] receives the count.  Scores are
// accumulated in fp32 in node order, which adds every path root first, exactly as the definition does.
__global__ void __launch_bounds__(128)
prune_select_kernel(int32_t N, float tau, int32_t budget, const int32_t *__restrict__ node_offsets,
                    const int32_t *__restrict__ parent, const float *__restrict__ logp, int32_t *__restrict__ out_offsets,
                    int32_t *__restrict__ out_parent, int32_t *__restrict__ out_index, int32_t *status)
{
    extern __shared__ int32_t sm[];
    float *q = reinterpret_cast<float *>(sm);           // [N]
    int32_t *keep = sm + N, *newidx = sm + 2 * N;       // [N], [N]
    __shared__ float s_thr;
    __shared__ int32_t s_fault;
    const int b = blockIdx.x;
    const int base = node_offsets[b], n = node_offsets[b + 1] - base;
    if (threadIdx.x == 0) {
        s_fault = 0;
        if (n < 0 || base < 0) s_fault = SPECA_STATUS_BAD_OFFSETS;
        else if (n > N) s_fault = SPECA_STATUS_TOO_MANY;
        else {
            float best = 0.f;
            for (int i = 0; i < n; ++i) {
                const int p = parent[base + i];
                if (p < -1 || p >= i) { s_fault = SPECA_STATUS_BAD_PARENT; break; }
                q[i] = (p >= 0 ? q[p] : 0.f) + logp[base + i];
                best = (i == 0 || q[i] > best) ? q[i] : best;
            }
            s_thr = best - tau;
        }
    }
    __syncthreads();
    if (s_fault) {
        if (threadIdx.x == 0) { atomicOr(status, s_fault); out_offsets[b + 1] = 0; }
        return;
    }
    const float thr = s_thr;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const float qi = q[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const float qj = q[j];
            rank += (qj >= thr) && (qj > qi || (qj == qi && j < i));
        }
        keep[i] = (qi >= thr) && rank < budget;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int c = 0;
        for (int i = 0; i < n; ++i) {
            const int p = parent[base + i];
            if (p >= 0 && !keep[p]) keep[i] = 0;
            newidx[i] = c;
            c += keep[i];
        }
        out_offsets[b + 1] = c;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x)
        if (keep[i]) {
            const int p = parent[base + i];
            out_parent[base + newidx[i]] = p < 0 ? -1 : newidx[p];
            out_index[base + newidx[i]] = i;
        }
}

// Step 2: one CTA turns the counts into offsets and closes the gaps, sequence by sequence in order
// (a sequence only ever moves toward the front, over space earlier sequences have already left).
__global__ void __launch_bounds__(256)
prune_pack_kernel(int32_t B, const int32_t *__restrict__ node_offsets, int32_t *__restrict__ out_offsets,
                  int32_t *__restrict__ out_parent, int32_t *__restrict__ out_index)
{
    __shared__ int32_t s_out;
    if (threadIdx.x == 0) { s_out = 0; out_offsets[0] = 0; }
    __syncthreads();
    for (int b = 0; b < B; ++b) {
        const int base = node_offsets[b], cnt = out_offsets[b + 1], dst = s_out;
        __syncthreads();                                 // everyone has read the count before it becomes an offset
        if (dst != base)
            for (int i0 = 0; i0 < cnt; i0 += blockDim.x) {
                const int i = i0 + threadIdx.x;
                int vp = 0, vi = 0;
                if (i < cnt) { vp = out_parent[base + i]; vi = out_index[base + i]; }
                __syncthreads();                         // dst < base: a slice is read before it can be overwritten
                if (i < cnt) { out_parent[dst + i] = vp; out_index[dst + i] = vi; }
                __syncthreads();
            }
        if (threadIdx.x == 0) { s_out = dst + cnt; out_offsets[b + 1] = dst + cnt; }
        __syncthreads();
    }
}

}  // namespace

int launch_mask_to_parent(int32_t B, int32_t N, const uint8_t *mask, const int32_t *node_offsets, int32_t *parent,
                          int32_t *status, cudaStream_t st)
{
    mask_to_parent_kernel<<<B, 256, size_t(2 * N) * sizeof(int32_t), st>>>(N, mask, node_offsets, parent, status);
    return int(cudaGetLastError());
}

int launch_chain_decompose(int32_t B, int32_t N, const int32_t *node_offsets, const int32_t *parent,
                           int32_t *chain_head, int32_t *n_chains, int32_t *status, cudaStream_t st)
{
    chain_decompose_kernel<<<B, 256, size_t(2 * N) * sizeof(int32_t), st>>>(N, node_offsets, parent, chain_head, n_chains,
                                                                         status);
    return int(cudaGetLastError());
}

int launch_prune(int32_t B, int32_t N, float tau, int32_t budget, const int32_t *node_offsets, const int32_t *parent,
                 const float *logp, int32_t *out_offsets, int32_t *out_parent, int32_t *out_index, int32_t *status,
                 cudaStream_t st)
{
    prune_select_kernel<<<B, 128, size_t(3 * N) * sizeof(int32_t), st>>>(N, tau, budget, node_offsets, parent, logp,
                                                                        out_offsets, out_parent, out_index, status);
    int e = int(cudaGetLastError());
    if (e != 0) return e;
    prune_pack_kernel<<<1, 256, 0, st>>>(B, node_offsets, out_offsets, out_parent, out_index);
    return int(cudaGetLastError());
}

int launch_conv_commit(int32_t L, int32_t B, int32_t channels, int32_t W, int32_t T, int32_t max_depth, void *C,
                       const void *x, const int32_t *node_offsets, const int32_t *path_idx, const int32_t *path_len,
                       int32_t *status, cudaStream_t st)
{
    conv_commit_kernel<<<L * B, 256, 0, st>>>(B, channels, W, T, max_depth, static_cast<uint4 *>(C),
                                              static_cast<const uint4 *>(x), node_offsets, path_idx, path_len, status);
    return int(cudaGetLastError());
}

int launch_pending_check(const Params &p, int max_len, cudaStream_t st)
{
    pending_check_kernel<<<(p.B + 127) / 128, 128, 0, st>>>(p.B, p.Tp, p.max_depth, max_len, p.max_nodes, p.pnode_offsets,
                                                            p.pparent, p.path_idx, p.path_len, p.ws.pend, p.status);
    return int(cudaGetLastError());
}

int launch_plan(const Params &p, cudaStream_t st)
{
    const size_t smem = size_t(6 * p.max_nodes + 1) * sizeof(int32_t);
    plan_kernel<<<p.B, kPlanThreads, smem, st>>>(p.node_offsets, p.parent, p.depth_in, p.B, p.T,
                                                  p.max_depth, p.max_nodes, p.n_slots, p.ws, p.status);
    return int(cudaGetLastError());
}

int launch_accept(int32_t B, int32_t max_depth, const int32_t *node_offsets, const int32_t *parent,
                  const int32_t *draft_tok, const int32_t *target_tok, const int32_t *root_target_tok,
                  int32_t *path_idx, int32_t *path_len, int32_t *next_tok, int32_t *status,
                  cudaStream_t st)
{
    const int warps = 4;
    accept_kernel<<<(B + warps - 1) / warps, warps * 32, 0, st>>>(
        B, max_depth, node_offsets, parent, draft_tok, target_tok, root_target_tok, path_idx, path_len,
        next_tok, status);
    return int(cudaGetLastError());
}

int launch_stochastic_accept(int32_t B, int32_t max_depth, const int32_t *node_offsets, const int32_t *parent,
                             const float *p_target, const float *p_draft, const float *uniform,
                             int32_t *path_idx, int32_t *path_len, int32_t *status, cudaStream_t st)
{
    const int warps = 4;
    stochastic_accept_kernel<<<(B + warps - 1) / warps, warps * 32, 0, st>>>(
        B, max_depth, node_offsets, parent, p_target, p_draft, uniform, path_idx, path_len, status);
    return int(cudaGetLastError());
}

}  // namespace speca
