// extern "C" entry points of libspeca: argument validation and kernel dispatch only.
#include <atomic>

#include "speca_common.cuh"

using namespace speca;

namespace {

inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

int check_dims(const speca_dims *d)
{
    if (d == nullptr) return SPECA_ERR_NULL;
    if (d->n_layers < 1 || d->batch < 1 || d->heads < 1) return SPECA_ERR_RANGE;
    if (d->d_k != 64 && d->d_k != 128 && d->d_k != 256) return SPECA_ERR_UNSUPPORTED;
    if (d->d_v < 32 || d->d_v > 1024 || d->d_v % 32 != 0) return SPECA_ERR_UNSUPPORTED;
    if (d->max_depth < 1 || d->max_depth > 16) return SPECA_ERR_RANGE;
    if (d->max_nodes < 1 || d->max_nodes > 1024) return SPECA_ERR_RANGE;
    if (d->route < SPECA_ROUTE_AUTO || d->route > SPECA_ROUTE_EFFECTIVE) return SPECA_ERR_UNSUPPORTED;
    if (d->rule != SPECA_RULE_GATED_DELTA && d->rule != SPECA_RULE_GATED_NO_ERASE) return SPECA_ERR_UNSUPPORTED;
    const long long units = 1LL * d->n_layers * d->batch * d->heads;
    if (units * (d->d_v / 2) > 0x7fffffffLL) return SPECA_ERR_RANGE;       // grid size bound
    return SPECA_OK;
}

Params base_params(const speca_dims *d, int32_t total_nodes)
{
    Params p{};
    p.L = d->n_layers; p.B = d->batch; p.H = d->heads; p.T = total_nodes; p.DV = d->d_v;
    p.scale = d->scale; p.max_depth = d->max_depth; p.max_nodes = d->max_nodes;
    p.no_erase = d->rule == SPECA_RULE_GATED_NO_ERASE;
    return p;
}

inline int cuda_rc(int e) { return e == 0 ? SPECA_OK : SPECA_ERR_CUDA; }

int verify_common(const speca_dims *dims, const float *S0, const uint16_t *q, const uint16_t *k,
                  const uint16_t *v, const float *alpha, const float *beta,
                  const int32_t *node_offsets, int32_t total_nodes, const int32_t *parent,
                  const int32_t *depth, bool chain, float *o, float *u, void *workspace,
                  size_t workspace_bytes, int32_t *status_word, void *stream)
{
    int rc = check_dims(dims);
    if (rc != SPECA_OK) return rc;
    if (!S0 || !q || !k || !v || !alpha || !beta || !node_offsets || !o || !status_word) return SPECA_ERR_NULL;
    if (!chain && !parent) return SPECA_ERR_NULL;
    if (total_nodes < 0) return SPECA_ERR_RANGE;
    if (1LL * total_nodes > 1LL * dims->batch * dims->max_nodes) return SPECA_ERR_RANGE;
    if (misaligned(S0) || misaligned(q) || misaligned(k) || misaligned(v) || misaligned(alpha) ||
        misaligned(beta) || misaligned(o) || (u && misaligned(u)) || misaligned(node_offsets) ||
        (parent && misaligned(parent)) || (depth && misaligned(depth)))
        return SPECA_ERR_ALIGN;
    if (!workspace || misaligned(workspace) ||
        workspace_bytes < speca::workspace_bytes(dims->batch, total_nodes))
        return SPECA_ERR_WORKSPACE;
    if (total_nodes == 0) return SPECA_OK;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Params p = base_params(dims, total_nodes);
    p.S0 = S0;
    p.q = reinterpret_cast<const __nv_bfloat16 *>(q);
    p.k = reinterpret_cast<const __nv_bfloat16 *>(k);
    p.v = reinterpret_cast<const __nv_bfloat16 *>(v);
    p.alpha = alpha; p.beta = beta; p.o = o; p.u = u;
    p.node_offsets = node_offsets; p.parent = parent; p.depth_in = depth;
    p.status = status_word;
    p.ws = carve_workspace(workspace, dims->batch, total_nodes);
    p.n_slots = tree_slots_needed(dims->max_nodes);
    // AUTO: an fp32-grade tensor-core route where the shape fits -- the factorised kernel in its compensated form,
    // or, for shapes it does not take (more than 32 nodes below 16 levels), the effective-query kernel -- else the
    // serial walk.  The single-pass TF32 kernel runs only when asked for by name.
    const bool tf32 = dims->route == SPECA_ROUTE_TF32;
    if (tf32 && !factorized_supported(dims)) return SPECA_ERR_UNSUPPORTED;
    const bool tensor = dims->route == SPECA_ROUTE_AUTO || dims->route == SPECA_ROUTE_FACTORIZED;
    const bool fact = tensor && factorized_supported(dims);
    if (dims->route == SPECA_ROUTE_EFFECTIVE && !effective_supported(dims)) return SPECA_ERR_UNSUPPORTED;
    const bool eff = dims->route == SPECA_ROUTE_EFFECTIVE || (tensor && !fact && effective_supported(dims));
    if (dims->route == SPECA_ROUTE_FACTORIZED && !fact && !eff) return SPECA_ERR_UNSUPPORTED;
    if (!chain || fact || eff || tf32) {
        // with parent == NULL (chain entry point) the plan kernel assumes parent[i] = i - 1
        rc = cuda_rc(launch_plan(p, st));
        if (rc != SPECA_OK) return rc;
    }
    if (fact) return cuda_rc(launch_verify_factorized(p, dims->d_k, false, true, st));
    if (eff) return cuda_rc(launch_verify_effective(p, dims->d_k, st));
    if (tf32) return cuda_rc(launch_verify_factorized(p, dims->d_k, false, false, st));
    return cuda_rc(launch_verify_serial(p, dims->d_k, chain, st));
}

// ---------------------------------------------------------------------------
// Built-in scratch of speca_verify_tree_noalloc.  The array lives in the library image
// on every device that loads it.  In host code its name is only a handle: the device
// address has to be asked for, once per device, with that device current.
// ---------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[SPECA_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::atomic<void *> g_noalloc_scratch_addr[kMaxDevices];

// Device address of the built-in scratch for the current device (nullptr on failure).  The lookup is
// idempotent, so two threads that race on the first call of a device store the same value.
void *noalloc_scratch_for_current_device()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    void *ptr = g_noalloc_scratch_addr[dev].load(std::memory_order_acquire);
    if (ptr == nullptr) {
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess) return nullptr;
        g_noalloc_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    return ptr;
}

}  // namespace

extern "C" {

int speca_version(void) { return SPECA_VERSION; }

/* Test hook, deliberately absent from speca.h: makes the next tensor-core verifications withhold the first
 * state slice of CTA 0, so that its bounded waits expire and the call reports SPECA_STATUS_TIMEOUT without
 * faulting anything.  The failure-detection test switches it on for one call and off again. */
void speca_test_withhold_first_load(int on)
{
    factorized_set_withhold(on);
    effective_set_withhold(on);
}

/* Test hook, deliberately absent from speca.h: speca_commit hands accepted paths of four to eight nodes to its
 * tensor-core kernel only when the batch is large enough for throughput to matter (n 16-row tiles per resident
 * warp; default 128).  n = 0 makes every batch of a supported shape take it, n < 0 restores the default. */
void speca_test_commit_long_min_tiles(int n) { commit_long_set_min_tiles_per_warp(n); }

/* Not in speca.h: 1 if the library was compiled with -DSPECA_PROF (the tensor-core kernels then record, for CTA 0,
 * the cycles each role spends in each kind of wait at the start of the workspace; bench.py --sweep role-waits
 * reads them). */
int speca_test_profiling_build(void)
{
#ifdef SPECA_PROF
    return 1;
#else
    return 0;
#endif
}

const char *speca_strerror(int code)
{
    switch (code) {
    case SPECA_OK: return "ok";
    case SPECA_ERR_NULL: return "a required pointer is NULL";
    case SPECA_ERR_UNSUPPORTED: return "unsupported shape or route";
    case SPECA_ERR_ALIGN: return "a tensor base is not 16-byte aligned";
    case SPECA_ERR_RANGE: return "a count is out of range";
    case SPECA_ERR_CUDA: return "CUDA launch error";
    case SPECA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case SPECA_ERR_TOO_LARGE: return "batch or node count exceeds the built-in scratch of the _noalloc entry point";
    }
    return "unknown speca error code";
}

size_t speca_workspace_bytes(const speca_dims *dims, int32_t total_nodes)
{
    if (dims == nullptr || total_nodes < 0 || dims->batch < 1) return 0;
    return speca::workspace_bytes(dims->batch, total_nodes);
}

int speca_decode_step(const speca_dims *dims, float *S, const uint16_t *q, const uint16_t *k,
                      const uint16_t *v, const float *alpha, const float *beta, float *o, void *stream)
{
    int rc = check_dims(dims);
    if (rc != SPECA_OK) return rc;
    if (!S || !q || !k || !v || !alpha || !beta || !o) return SPECA_ERR_NULL;
    if (misaligned(S) || misaligned(q) || misaligned(k) || misaligned(v) || misaligned(alpha) ||
        misaligned(beta) || misaligned(o))
        return SPECA_ERR_ALIGN;
    Params p = base_params(dims, dims->batch);
    p.S = S;
    p.q = reinterpret_cast<const __nv_bfloat16 *>(q);
    p.k = reinterpret_cast<const __nv_bfloat16 *>(k);
    p.v = reinterpret_cast<const __nv_bfloat16 *>(v);
    p.alpha = alpha; p.beta = beta; p.o = o;
    return cuda_rc(launch_decode(p, dims->d_k, static_cast<cudaStream_t>(stream)));
}

int speca_verify_chain(const speca_dims *dims, const float *S0, const uint16_t *q, const uint16_t *k,
                       const uint16_t *v, const float *alpha, const float *beta,
                       const int32_t *node_offsets, int32_t total_nodes, float *o, float *u_or_null,
                       void *workspace, size_t workspace_bytes, int32_t *status_word, void *stream)
{
    return verify_common(dims, S0, q, k, v, alpha, beta, node_offsets, total_nodes, nullptr, nullptr, true,
                         o, u_or_null, workspace, workspace_bytes, status_word, stream);
}

int speca_verify_tree(const speca_dims *dims, const float *S0, const uint16_t *q, const uint16_t *k,
                      const uint16_t *v, const float *alpha, const float *beta,
                      const int32_t *node_offsets, int32_t total_nodes, const int32_t *parent,
                      const int32_t *depth_or_null, float *o, float *u_or_null, void *workspace,
                      size_t workspace_bytes, int32_t *status_word, void *stream)
{
    return verify_common(dims, S0, q, k, v, alpha, beta, node_offsets, total_nodes, parent, depth_or_null,
                         false, o, u_or_null, workspace, workspace_bytes, status_word, stream);
}

int speca_verify_tree_noalloc(const speca_dims *dims, const float *S0, const uint16_t *q, const uint16_t *k,
                              const uint16_t *v, const float *alpha, const float *beta,
                              const int32_t *node_offsets, int32_t total_nodes, const int32_t *parent,
                              const int32_t *depth_or_null, float *o, float *u_or_null,
                              int32_t *status_word, void *stream)
{
    if (dims == nullptr) return SPECA_ERR_NULL;
    if (dims->batch > SPECA_NOALLOC_MAX_BATCH || total_nodes > SPECA_NOALLOC_MAX_NODES) return SPECA_ERR_TOO_LARGE;
    static_assert(SPECA_NOALLOC_SCRATCH_BYTES >= kCtrlBytes + 4 * SPECA_NOALLOC_MAX_BATCH +
                                                     size_t(kNodeWords) * 4 * SPECA_NOALLOC_MAX_NODES +
                                                     size_t(kPendWords) * 4 * SPECA_NOALLOC_MAX_BATCH,
                  "built-in scratch smaller than the workspace of the largest accepted problem");
    // all argument checks first (they need no device); only then touch the CUDA runtime
    void *scratch = nullptr;
    if (total_nodes > 0 && dims->batch >= 1) {
        scratch = noalloc_scratch_for_current_device();
        if (scratch == nullptr) return SPECA_ERR_CUDA;
    } else {
        scratch = reinterpret_cast<void *>(uintptr_t(256));      // never dereferenced: nothing is launched
    }
    return verify_common(dims, S0, q, k, v, alpha, beta, node_offsets, total_nodes, parent, depth_or_null, false,
                         o, u_or_null, scratch, SPECA_NOALLOC_SCRATCH_BYTES, status_word, stream);
}

int speca_greedy_accept(int32_t batch, int32_t max_depth, const int32_t *node_offsets,
                        const int32_t *parent, const int32_t *draft_tok, const int32_t *target_tok,
                        const int32_t *root_target_tok, int32_t *path_idx, int32_t *path_len,
                        int32_t *next_tok, int32_t *status_word, void *stream)
{
    if (!node_offsets || !parent || !draft_tok || !target_tok || !root_target_tok || !path_idx || !path_len ||
        !next_tok || !status_word)
        return SPECA_ERR_NULL;
    if (batch < 1 || max_depth < 1 || max_depth > 16) return SPECA_ERR_RANGE;
    return cuda_rc(launch_accept(batch, max_depth, node_offsets, parent, draft_tok, target_tok,
                                 root_target_tok, path_idx, path_len, next_tok, status_word,
                                 static_cast<cudaStream_t>(stream)));
}

int speca_stochastic_accept(int32_t batch, int32_t max_depth, const int32_t *node_offsets,
                            const int32_t *parent, const float *p_target, const float *p_draft,
                            const float *uniform, int32_t *path_idx, int32_t *path_len,
                            int32_t *status_word, void *stream)
{
    if (!node_offsets || !parent || !p_target || !p_draft || !uniform || !path_idx || !path_len || !status_word)
        return SPECA_ERR_NULL;
    if (batch < 1 || max_depth < 1 || max_depth > 16) return SPECA_ERR_RANGE;
    return cuda_rc(launch_stochastic_accept(batch, max_depth, node_offsets, parent, p_target, p_draft, uniform,
                                            path_idx, path_len, status_word, static_cast<cudaStream_t>(stream)));
}

int speca_commit(const speca_dims *dims, float *S, const uint16_t *k, const uint16_t *v,
                 const float *alpha, const float *beta, const int32_t *node_offsets, int32_t total_nodes,
                 const int32_t *parent_or_null, const int32_t *path_idx, const int32_t *path_len,
                 int32_t *status_word, void *stream)
{
    int rc = check_dims(dims);
    if (rc != SPECA_OK) return rc;
    if (!S || !k || !v || !alpha || !beta || !node_offsets || !path_idx || !path_len || !status_word)
        return SPECA_ERR_NULL;
    if (total_nodes < 0) return SPECA_ERR_RANGE;
    if (misaligned(S) || misaligned(k) || misaligned(v) || misaligned(alpha) || misaligned(beta))
        return SPECA_ERR_ALIGN;
    if (total_nodes == 0) return SPECA_OK;
    Params p = base_params(dims, total_nodes);
    p.S = S;
    p.k = reinterpret_cast<const __nv_bfloat16 *>(k);
    p.v = reinterpret_cast<const __nv_bfloat16 *>(v);
    p.alpha = alpha; p.beta = beta;
    p.node_offsets = node_offsets; p.parent = parent_or_null;
    p.path_idx = path_idx; p.path_len = path_len; p.status = status_word;
    return cuda_rc(launch_commit(p, dims->d_k, static_cast<cudaStream_t>(stream)));
}

int speca_tree_mask_to_parent(int32_t batch, int32_t max_nodes, const uint8_t *mask, const int32_t *node_offsets,
                              int32_t *parent, int32_t *status_word, void *stream)
{
    if (!mask || !node_offsets || !parent || !status_word) return SPECA_ERR_NULL;
    if (batch < 1 || max_nodes < 1 || max_nodes > 1024) return SPECA_ERR_RANGE;
    return cuda_rc(launch_mask_to_parent(batch, max_nodes, mask, node_offsets, parent, status_word,
                                         static_cast<cudaStream_t>(stream)));
}

int speca_prune_tree(int32_t batch, int32_t max_nodes, float tau, int32_t budget, const int32_t *node_offsets,
                     const int32_t *parent, const float *logp, int32_t *out_offsets, int32_t *out_parent,
                     int32_t *out_index, int32_t *status_word, void *stream)
{
    if (!node_offsets || !parent || !logp || !out_offsets || !out_parent || !out_index || !status_word)
        return SPECA_ERR_NULL;
    if (batch < 1 || max_nodes < 1 || max_nodes > 1024 || budget < 0 || !(tau >= 0.f)) return SPECA_ERR_RANGE;
    return cuda_rc(launch_prune(batch, max_nodes, tau, budget, node_offsets, parent, logp, out_offsets, out_parent,
                                out_index, status_word, static_cast<cudaStream_t>(stream)));
}

int speca_chain_decompose(int32_t batch, int32_t max_nodes, const int32_t *node_offsets, const int32_t *parent,
                          int32_t *chain_head, int32_t *n_chains, int32_t *status_word, void *stream)
{
    if (!node_offsets || !parent || !chain_head || !n_chains || !status_word) return SPECA_ERR_NULL;
    if (batch < 1 || max_nodes < 1 || max_nodes > 1024) return SPECA_ERR_RANGE;
    return cuda_rc(launch_chain_decompose(batch, max_nodes, node_offsets, parent, chain_head, n_chains, status_word,
                                          static_cast<cudaStream_t>(stream)));
}

int speca_commit_conv(int32_t n_layers, int32_t batch, int32_t channels, int32_t width, int32_t max_depth,
                      uint16_t *C, const uint16_t *x, const int32_t *node_offsets, int32_t total_nodes,
                      const int32_t *path_idx, const int32_t *path_len, int32_t *status_word, void *stream)
{
    if (!C || !x || !node_offsets || !path_idx || !path_len || !status_word) return SPECA_ERR_NULL;
    if (n_layers < 1 || batch < 1 || total_nodes < 0 || max_depth < 1 || max_depth > 16) return SPECA_ERR_RANGE;
    if (1LL * n_layers * batch > 0x7fffffffLL) return SPECA_ERR_RANGE;
    if (channels < 8 || channels % 8 != 0 || width < 1 || width > 8) return SPECA_ERR_UNSUPPORTED;
    if (misaligned(C) || misaligned(x)) return SPECA_ERR_ALIGN;
    if (total_nodes == 0) return SPECA_OK;
    return cuda_rc(launch_conv_commit(n_layers, batch, channels, width, total_nodes, max_depth, C, x, node_offsets,
                                      path_idx, path_len, status_word, static_cast<cudaStream_t>(stream)));
}

int speca_commit_verify_tree(const speca_dims *dims, float *S, const uint16_t *k_prev, const uint16_t *v_prev,
                             const float *alpha_prev, const float *beta_prev, const float *u_prev_or_null,
                             const int32_t *node_offsets_prev, int32_t total_nodes_prev,
                             const int32_t *parent_prev_or_null, const int32_t *path_idx, const int32_t *path_len,
                             const uint16_t *q, const uint16_t *k, const uint16_t *v, const float *alpha,
                             const float *beta, const int32_t *node_offsets, int32_t total_nodes,
                             const int32_t *parent, const int32_t *depth_or_null, float *o, float *u_or_null,
                             void *workspace, size_t workspace_bytes, int32_t *status_word, void *stream)
{
    int rc = check_dims(dims);
    if (rc != SPECA_OK) return rc;
    if (!S || !status_word) return SPECA_ERR_NULL;
    if (total_nodes_prev < 0 || total_nodes < 0) return SPECA_ERR_RANGE;
    const bool have_commit = total_nodes_prev > 0;
    if (have_commit && (!k_prev || !v_prev || !alpha_prev || !beta_prev || !node_offsets_prev || !path_idx || !path_len))
        return SPECA_ERR_NULL;
    if (have_commit && (misaligned(k_prev) || misaligned(v_prev) || misaligned(alpha_prev) || misaligned(beta_prev) ||
                        (u_prev_or_null && misaligned(u_prev_or_null))))
        return SPECA_ERR_ALIGN;
    if (total_nodes > 0 && workspace_bytes < speca::workspace_bytes(dims->batch, total_nodes))
        return SPECA_ERR_WORKSPACE;

    // One pass over the state on the single-pass TF32 route, when the previous verification left its
    // u; otherwise the commit and verify kernels run back to back on the stream (same results, fp32-grade).
    const bool one_pass = have_commit && total_nodes > 0 && u_prev_or_null != nullptr && factorized_fused_supported(dims) &&
                          dims->route == SPECA_ROUTE_TF32;
    if (!one_pass) {
        if (have_commit) {
            rc = speca_commit(dims, S, k_prev, v_prev, alpha_prev, beta_prev, node_offsets_prev, total_nodes_prev,
                              parent_prev_or_null, path_idx, path_len, status_word, stream);
            if (rc != SPECA_OK) return rc;
        }
        if (total_nodes == 0) return SPECA_OK;
        return verify_common(dims, S, q, k, v, alpha, beta, node_offsets, total_nodes, parent, depth_or_null, false, o,
                             u_or_null, workspace, workspace_bytes, status_word, stream);
    }

    if (!q || !k || !v || !alpha || !beta || !node_offsets || !parent || !o) return SPECA_ERR_NULL;
    if (1LL * total_nodes > 1LL * dims->batch * dims->max_nodes) return SPECA_ERR_RANGE;
    if (misaligned(S) || misaligned(q) || misaligned(k) || misaligned(v) || misaligned(alpha) || misaligned(beta) ||
        misaligned(o) || (u_or_null && misaligned(u_or_null)) || misaligned(node_offsets) || misaligned(parent) ||
        (depth_or_null && misaligned(depth_or_null)))
        return SPECA_ERR_ALIGN;
    if (!workspace || misaligned(workspace)) return SPECA_ERR_WORKSPACE;
    if (u_or_null != nullptr && u_or_null == u_prev_or_null) return SPECA_ERR_RANGE;     // read and written in one pass

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Params p = base_params(dims, total_nodes);
    p.S = S; p.S0 = S;
    p.q = reinterpret_cast<const __nv_bfloat16 *>(q);
    p.k = reinterpret_cast<const __nv_bfloat16 *>(k);
    p.v = reinterpret_cast<const __nv_bfloat16 *>(v);
    p.alpha = alpha; p.beta = beta; p.o = o; p.u = u_or_null;
    p.node_offsets = node_offsets; p.parent = parent; p.depth_in = depth_or_null;
    p.path_idx = path_idx; p.path_len = path_len;
    p.pk = reinterpret_cast<const __nv_bfloat16 *>(k_prev);
    p.palpha = alpha_prev; p.pu = u_prev_or_null;
    p.pnode_offsets = node_offsets_prev; p.pparent = parent_prev_or_null; p.Tp = total_nodes_prev;
    p.status = status_word;
    p.ws = carve_workspace(workspace, dims->batch, total_nodes);
    p.n_slots = tree_slots_needed(dims->max_nodes);
    rc = cuda_rc(launch_plan(p, st));
    if (rc != SPECA_OK) return rc;
    rc = cuda_rc(launch_pending_check(p, 8, st));
    if (rc != SPECA_OK) return rc;
    return cuda_rc(launch_verify_factorized(p, dims->d_k, true, false, st));
}

}  // extern "C"
