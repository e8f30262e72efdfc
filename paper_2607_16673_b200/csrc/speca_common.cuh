// Shared declarations of the libspeca translation units (device helpers, launch
// parameter blocks, workspace layout).  Nothing here is visible at the C ABI.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/speca.h"

namespace speca {

// ---------------------------------------------------------------------------
// Workspace layout (device scratch handed in by the caller).
//   [0, 2048)                    control words (work-queue counters, optional profiling slots)
//   [2048, 2048 + 4*Bpad)        seq_n[b]: node count of sequence b, or -1 if the
//                                sequence failed validation and must be skipped
//   then int32 arrays of Tpad words: plan[T], depth[T], anc[T][4], anc2[T][4]
//   after the kNodeWords node arrays, used only by the fused commit-and-verify call:
//   pend[B][kPendWords]: validated length of the pending accepted path, its local node
//   indices, and the sequence's offset in the previous draft's packed arrays
// Every region starts on a 256-byte boundary.
// ---------------------------------------------------------------------------
constexpr size_t kCtrlBytes = 2048;
constexpr int kNodeWords = 16;          // int32 words of scratch reserved per packed node
constexpr int kPendWords = 12;          // per sequence: path length, 8 local node indices, offset, spare

__host__ __device__ inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

struct Workspace {
    int32_t *ctrl;      // [64]
    int32_t *seq_n;     // [B]
    int32_t *plan;      // [T]   packed schedule entries, in processing order per sequence
    int32_t *depth;     // [T]   depth computed from parent[]
    int32_t *anc;       // [T][4] per node: depth | position << 8, ancestor node indices of levels 1..12 (one byte each)
    int32_t *anc2;      // [T][4] per node: ancestor node indices of levels 13..15, spare
    int32_t *pend;      // [B][kPendWords] pending accepted path (fused commit-and-verify only)
};

inline size_t workspace_bytes(int32_t batch, int32_t total_nodes)
{
    return kCtrlBytes + align256(size_t(batch) * 4) + align256(size_t(total_nodes) * 4) * kNodeWords +
           align256(size_t(batch) * kPendWords * 4);
}

inline Workspace carve_workspace(void *base, int32_t batch, int32_t total_nodes)
{
    Workspace w;
    char *p = static_cast<char *>(base);
    w.ctrl = reinterpret_cast<int32_t *>(p);
    p += kCtrlBytes;
    w.seq_n = reinterpret_cast<int32_t *>(p);
    p += align256(size_t(batch) * 4);
    size_t tb = align256(size_t(total_nodes) * 4);
    w.plan = reinterpret_cast<int32_t *>(p);
    w.depth = reinterpret_cast<int32_t *>(p + tb);
    w.anc = reinterpret_cast<int32_t *>(p + 2 * tb);
    w.anc2 = reinterpret_cast<int32_t *>(p + 6 * tb);
    w.pend = reinterpret_cast<int32_t *>(p + kNodeWords * tb);
    return w;
}

// Packed schedule entry written by the plan kernel, one per node, in the order
// the serial tree walk processes the nodes of a sequence.
//   bits  0..15  node index (local to the sequence)
//   bits 16..19  load code: 0 = parent state is already in registers,
//                1..14 = reload from on-chip slot (code-1), 15 = reload S0 from HBM
//   bits 20..23  save code: 0 = none, 1..14 = store the new state to slot (code-1)
//   bit  24      leaf: emit o only, leave the register state at the parent's
constexpr int kPlanLoadShift = 16, kPlanSaveShift = 20, kPlanLeafBit = 1 << 24;
constexpr int kLoadFromS0 = 15;

// Launch parameter block shared by the kernels.
struct Params {
    int32_t L, B, H, T, DV;
    float scale;
    int32_t max_depth, max_nodes;
    int32_t no_erase;            // SPECA_RULE_GATED_NO_ERASE: the corrected value is u = beta v (no read-out of the state)
    float *S;                    // in/out for decode and commit
    const float *S0;             // read-only for verify
    const __nv_bfloat16 *q, *k, *v;
    const float *alpha, *beta;
    float *o, *u;
    const int32_t *node_offsets, *parent, *depth_in;
    const int32_t *path_idx, *path_len;
    // pending commit of the fused call: records of the previous draft (keys, gates, u) and its packing
    const __nv_bfloat16 *pk;
    const float *palpha, *pu;
    const int32_t *pnode_offsets, *pparent;
    int32_t Tp;
    int32_t *status;
    Workspace ws;
    int32_t n_slots;             // on-chip state slots available to the tree walk
    int32_t long_min;            // commit: accepted paths of long_min..8 nodes are taken by the tensor-core kernel (0: none)
};

// Launchers implemented per translation unit; each returns a cudaError_t-compatible int.
int launch_plan(const Params &p, cudaStream_t st);
int launch_decode(const Params &p, int d_k, cudaStream_t st);
int launch_verify_serial(const Params &p, int d_k, bool chain, cudaStream_t st);
int launch_commit(const Params &p, int d_k, cudaStream_t st);
// commit of paths of p.long_min..8 nodes on warp-level MMAs (the token-by-token kernel skips those sequences)
bool commit_long_supported(const Params &p, int d_k);
int launch_commit_long(const Params &p, int d_k, cudaStream_t st);
void commit_long_set_min_tiles_per_warp(int n);
bool factorized_supported(const speca_dims *d);
bool factorized_fused_supported(const speca_dims *d);
int launch_verify_factorized(const Params &p, int d_k, bool fused, bool comp, cudaStream_t st);
void factorized_set_withhold(int on);
bool effective_supported(const speca_dims *d);
int launch_verify_effective(const Params &p, int d_k, cudaStream_t st);
void effective_set_withhold(int on);
int launch_pending_check(const Params &p, int max_len, cudaStream_t st);
int launch_mask_to_parent(int32_t B, int32_t N, const uint8_t *mask, const int32_t *node_offsets, int32_t *parent,
                          int32_t *status, cudaStream_t st);
int launch_chain_decompose(int32_t B, int32_t N, const int32_t *node_offsets, const int32_t *parent,
                           int32_t *chain_head, int32_t *n_chains, int32_t *status, cudaStream_t st);
int launch_prune(int32_t B, int32_t N, float tau, int32_t budget, const int32_t *node_offsets, const int32_t *parent,
                 const float *logp, int32_t *out_offsets, int32_t *out_parent, int32_t *out_index, int32_t *status,
                 cudaStream_t st);
int launch_conv_commit(int32_t L, int32_t B, int32_t channels, int32_t W, int32_t T, int32_t max_depth, void *C,
                       const void *x, const int32_t *node_offsets, const int32_t *path_idx, const int32_t *path_len,
                       int32_t *status, cudaStream_t st);
int launch_accept(int32_t B, int32_t max_depth, const int32_t *node_offsets, const int32_t *parent,
                  const int32_t *draft_tok, const int32_t *target_tok, const int32_t *root_target_tok,
                  int32_t *path_idx, int32_t *path_len, int32_t *next_tok, int32_t *status,
                  cudaStream_t st);
int launch_stochastic_accept(int32_t B, int32_t max_depth, const int32_t *node_offsets, const int32_t *parent,
                             const float *p_target, const float *p_draft, const float *uniform,
                             int32_t *path_idx, int32_t *path_len, int32_t *status, cudaStream_t st);

// Number of on-chip state slots the light-children-first walk can need for a tree of
// at most n nodes: a node saves its state only if it has two children with
// children of their own (subtree >= 5 nodes) and every live slot at least halves
// the remaining subtree.
inline int tree_slots_needed(int n)
{
    int s = 0;
    while (n >= 5) { ++s; n = (n - 1) / 2; }
    return s;
}

}  // namespace speca
