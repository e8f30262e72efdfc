/*
 * gdn_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of what the speculative verify / accept /
 * commit path over a gated-delta-rule (GDN) recurrent state computes.  It is
 * the yardstick the CUDA library is compared with; it shares no code, header,
 * table or helper with that library, and nothing in the product may call it.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Every function is the definition written out: no blocking, no fusion, no
 * prefix sharing between draft nodes, no reordering.
 *
 *   gated delta rule      S' = S * alpha (I - beta k k^T) + beta v k^T ,  o = scale * S' q
 *                         (GDN layer, Section 2.2; the minimal un-gated form is Eq. 1)
 *   verification          every draft node sees the state obtained by applying
 *                         the rule along its own ancestor path from the committed
 *                         state S_0; siblings never influence each other
 *                         (Section 4.2: updates propagate only along ancestor paths)
 *   greedy acceptance     longest root path whose draft tokens equal the
 *                         target's greedy tokens (Section 2.1, Section 8 setup)
 *   commit                S_A = the rule applied token by token over the accepted
 *                         factor records f_t = (k_t, v_t, alpha_t, beta_t)
 *                         (Section 5.1, Eq. 3; Section 5.2 "immediate update")
 *
 * Parity pins: all four entry points are pinned by tests/test_oracle_pins.py
 * (closed forms, a dense-matrix restatement, the tree-masked factorised form of
 * Section 4.2 solved densely, snapshot-propagation brute force over every
 * forest of <= 4 nodes, brute-force path enumeration for acceptance).
 *
 * Layouts (row-major, last index fastest):
 *   S        double [L][B][H][d_v][d_k]
 *   q, k     bf16 bits (uint16) [L][T][H][d_k]
 *   v        bf16 bits (uint16) [L][T][H][d_v]
 *   alpha,beta float [L][T][H]
 *   o        double [L][T][H][d_v]
 *   node_offsets int32 [B+1]; parent int32 [T] (index local to the sequence,
 *   -1 = child of the committed state).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* Which recurrence the entry points apply (Section 5.1, remark on other layer types):
 *   0  gated delta rule (GDN; a DeltaNet layer is its alpha = 1 case)
 *   1  gated rule without the erase term,  S' = alpha S + beta v k^T  (GLA-style layers, which keep
 *      key, value and gate but no delta-rule read-out)
 * Set between calls with oracle_set_rule; read-only while a call runs. */
static int g_rule = 0;
void oracle_set_rule(int rule) { g_rule = rule; }

/* One application of the rule to one head's state, in place.
 * Order of the definition: decay the state, read it with the key, erase that
 * read-out (rule 0 only), write the new value.  S is [d_v][d_k]. */
static void gdn_rule(int d_k, int d_v, double *S, const double *k, const double *v,
                     double alpha, double beta)
{
    for (int i = 0; i < d_v; ++i) {
        double *row = S + (size_t)i * d_k;
        for (int j = 0; j < d_k; ++j) row[j] *= alpha;          /* S alpha            */
        double read = 0.0;
        if (g_rule == 0)
            for (int j = 0; j < d_k; ++j) read += row[j] * k[j];    /* (S alpha) k        */
        for (int j = 0; j < d_k; ++j)                            /* - beta (.) k^T + beta v k^T */
            row[j] += beta * (v[i] - read) * k[j];
    }
}

static void gdn_readout(int d_k, int d_v, double scale, const double *S, const double *q, double *o)
{
    for (int i = 0; i < d_v; ++i) {
        double acc = 0.0;
        const double *row = S + (size_t)i * d_k;
        for (int j = 0; j < d_k; ++j) acc += row[j] * q[j];
        o[i] = scale * acc;
    }
}

static void widen(int n, const uint16_t *src, double *dst)
{
    for (int j = 0; j < n; ++j) dst[j] = bf16_to_double(src[j]);
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Threads the unit loops below may use (timing only: no result depends on it). */
void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Single-token decode step for every (layer, sequence, head): T == B, one token
 * per sequence.  S is updated in place, o = scale * S_new q. */
int oracle_decode_step(int L, int B, int H, int d_k, int d_v, double scale,
                       double *S, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                       const float *alpha, const float *beta, double *o)
{
    long units = (long)L * B * H;
#pragma omp parallel
    {
        double *kk = malloc(sizeof(double) * d_k), *qq = malloc(sizeof(double) * d_k);
        double *vv = malloc(sizeof(double) * d_v);
#pragma omp for schedule(static)
        for (long u = 0; u < units; ++u) {
            widen(d_k, k + u * d_k, kk);
            widen(d_k, q + u * d_k, qq);
            widen(d_v, v + u * d_v, vv);
            double *Su = S + (size_t)u * d_v * d_k;
            gdn_rule(d_k, d_v, Su, kk, vv, (double)alpha[u], (double)beta[u]);
            gdn_readout(d_k, d_v, scale, Su, qq, o + u * d_v);
        }
        free(kk); free(qq); free(vv);
    }
    return 0;
}

/* Verification of a packed batch of draft forests.  For EVERY node on its own:
 * follow parent[] up to the committed state, copy S_0, apply the rule down the
 * path, read out with the node's query.  S0 is never modified.
 * Returns 0, or -1 when a parent pointer is not a valid earlier node. */
int oracle_verify_tree(int L, int B, int H, int d_k, int d_v, double scale,
                       const double *S0, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                       const float *alpha, const float *beta,
                       const int32_t *node_offsets, const int32_t *parent, double *o)
{
    int T = node_offsets[B];
    for (int b = 0; b < B; ++b)
        for (int t = node_offsets[b]; t < node_offsets[b + 1]; ++t) {
            int local = t - node_offsets[b];
            if (parent[t] < -1 || parent[t] >= local) return -1;
        }
    long units = (long)L * B * H;
#pragma omp parallel
    {
        double *St = malloc(sizeof(double) * (size_t)d_v * d_k);
        double *kk = malloc(sizeof(double) * d_k), *qq = malloc(sizeof(double) * d_k);
        double *vv = malloc(sizeof(double) * d_v);
        int32_t *path = malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
#pragma omp for schedule(dynamic, 1)
        for (long u = 0; u < units; ++u) {
            int h = (int)(u % H), b = (int)((u / H) % B), l = (int)(u / ((long)H * B));
            int base = node_offsets[b], n = node_offsets[b + 1] - base;
            const double *S0u = S0 + (size_t)u * d_v * d_k;
            for (int t = 0; t < n; ++t) {
                int len = 0;
                for (int a = t; a != -1; a = parent[base + a]) path[len++] = a;
                memcpy(St, S0u, sizeof(double) * (size_t)d_v * d_k);
                for (int s = len - 1; s >= 0; --s) {            /* root first */
                    size_t rec = ((size_t)l * T + base + path[s]) * H + h;
                    widen(d_k, k + rec * d_k, kk);
                    widen(d_v, v + rec * d_v, vv);
                    gdn_rule(d_k, d_v, St, kk, vv, (double)alpha[rec], (double)beta[rec]);
                }
                size_t rec = ((size_t)l * T + base + t) * H + h;
                widen(d_k, q + rec * d_k, qq);
                gdn_readout(d_k, d_v, scale, St, qq, o + rec * d_v);
            }
        }
        free(St); free(kk); free(qq); free(vv); free(path);
    }
    return 0;
}

/* Greedy acceptance.  pred(-1) = root_target_tok[b], pred(i) = target_tok[i].
 * A node is matched iff its draft token equals pred(parent) and its parent is
 * matched (children of the committed state only need the first condition).
 * The accepted path is the root path of the deepest matched node, lowest index
 * on ties; it may be empty.  next_tok = pred(last accepted node).
 * path_idx is [B][max_depth], unused entries are set to -1.
 * Returns 0, -1 on a bad parent pointer, -2 if a matched path exceeds max_depth. */
int oracle_greedy_accept(int B, int max_depth, const int32_t *node_offsets, const int32_t *parent,
                         const int32_t *draft_tok, const int32_t *target_tok,
                         const int32_t *root_target_tok,
                         int32_t *path_idx, int32_t *path_len, int32_t *next_tok)
{
    for (int b = 0; b < B; ++b) {
        int base = node_offsets[b], n = node_offsets[b + 1] - base;
        int *mdepth = calloc((size_t)(n > 0 ? n : 1), sizeof(int));   /* 0 = not matched */
        int best = -1, best_depth = 0;
        for (int t = 0; t < n; ++t) {
            int p = parent[base + t];
            if (p < -1 || p >= t) { free(mdepth); return -1; }
            int pred = (p == -1) ? root_target_tok[b] : target_tok[base + p];
            int parent_ok = (p == -1) || mdepth[p] > 0;
            if (parent_ok && draft_tok[base + t] == pred) {
                mdepth[t] = (p == -1 ? 0 : mdepth[p]) + 1;
                if (mdepth[t] > best_depth) { best_depth = mdepth[t]; best = t; }
            }
        }
        free(mdepth);
        if (best_depth > max_depth) return -2;
        for (int d = 0; d < max_depth; ++d) path_idx[(size_t)b * max_depth + d] = -1;
        path_len[b] = best_depth;
        int a = best;
        for (int d = best_depth - 1; d >= 0; --d) {
            path_idx[(size_t)b * max_depth + d] = a;
            a = parent[base + a];
        }
        next_tok[b] = (best < 0) ? root_target_tok[b] : target_tok[base + best];
    }
    return 0;
}

/* Commit: advance the durable state over the accepted factor records, token by
 * token, in place.  path_len[b] == 0 leaves the state of sequence b untouched. */
int oracle_commit(int L, int B, int H, int d_k, int d_v, int max_depth,
                  double *S, const uint16_t *k, const uint16_t *v,
                  const float *alpha, const float *beta,
                  const int32_t *node_offsets, const int32_t *path_idx, const int32_t *path_len)
{
    int T = node_offsets[B];
    for (int b = 0; b < B; ++b) {
        int n = node_offsets[b + 1] - node_offsets[b];
        if (path_len[b] < 0 || path_len[b] > max_depth) return -2;
        for (int d = 0; d < path_len[b]; ++d) {
            int a = path_idx[(size_t)b * max_depth + d];
            if (a < 0 || a >= n) return -1;
        }
    }
    long units = (long)L * B * H;
#pragma omp parallel
    {
        double *kk = malloc(sizeof(double) * d_k), *vv = malloc(sizeof(double) * d_v);
#pragma omp for schedule(dynamic, 1)
        for (long u = 0; u < units; ++u) {
            int h = (int)(u % H), b = (int)((u / H) % B), l = (int)(u / ((long)H * B));
            double *Su = S + (size_t)u * d_v * d_k;
            for (int d = 0; d < path_len[b]; ++d) {
                int a = path_idx[(size_t)b * max_depth + d];
                size_t rec = ((size_t)l * T + node_offsets[b] + a) * H + h;
                widen(d_k, k + rec * d_k, kk);
                widen(d_v, v + rec * d_v, vv);
                gdn_rule(d_k, d_v, Su, kk, vv, (double)alpha[rec], (double)beta[rec]);
            }
        }
        free(kk); free(vv);
    }
    return 0;
}
