/*
 * CPU oracle for the Speculative-Streaming decode hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain C, fp64 arithmetic, one pass, no blocking, no fusion: every function is the
 * definition it cites, written out so that it can be checked against the paper by eye.
 * It shares no code, header, table or helper with the CUDA library; only tests, the smoke
 * check and the benchmark's CPU-baseline leg may link or call it.
 *
 * Parity pins (tests/test_oracle_*.py): dense-mask brute force written independently in
 * numpy; chain tree with gamma = 0 against a library causal attention; single-query softmax;
 * mask-cardinality closed form; one-hot membership sweep; the mask example printed with the
 * attention-mask figure of App. A; causality invariants; verification closed forms and path
 * enumeration; sequential-copy brute force for the compaction; next-draft construction against
 * numpy's stable sort, the size formula of Sec. 3.2.3 and the k = 1 chain of App. D; pruning and
 * soft matching against scipy's softmax / entropy and hand-built trees; sampled verification
 * against numpy's cumulative sums; stream insertion and value rotation against numpy float32
 * arithmetic, the rotation's norm and composition laws.  Nothing here is unpinned.
 *
 * bf16 values arrive as raw 16-bit patterns; widening to double is exact.
 * OpenMP only distributes independent (head) / (node) / (layer) iterations; the arithmetic
 * order inside one output is the sequential order of the definition.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SSOR_OK 0
#define SSOR_BAD_TREE -2
#define SSOR_BAD_ARG -1

static double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* A draft tree is given by parent[]: node 0 is the root (the correction token of the previous
 * pass, App. A.1), parent[i] in [0, i).  depth(root) = 0.  is_anc[t*n + a] = 1 iff a lies on
 * the path root..t, t itself included: a node sees every node on its root path and itself
 * (attention-mask figure of App. A). */
int ssor_tree_build(const int32_t* parent, int32_t n, int32_t* depth, uint8_t* is_anc,
                    int32_t* max_depth) {
    if (n < 1 || parent[0] != -1) return SSOR_BAD_TREE;
    for (int32_t i = 1; i < n; ++i)
        if (parent[i] < 0 || parent[i] >= i) return SSOR_BAD_TREE;
    int32_t md = 0;
    for (int32_t t = 0; t < n; ++t) {
        int32_t dep = 0;
        if (is_anc) memset(is_anc + (size_t)t * n, 0, (size_t)n);
        for (int32_t a = t; a != -1; a = parent[a]) {   /* walk t, parent(t), ..., root */
            if (is_anc) is_anc[(size_t)t * n + a] = 1;
            if (a != t) ++dep;
        }
        if (depth) depth[t] = dep;
        if (dep > md) md = dep;
    }
    if (max_depth) *max_depth = md;
    return SSOR_OK;
}

/* softmax(sm_scale * q.K^T) V over an explicit key list (Eq. 1 / Eq. 2 with the MHA of
 * Vaswani et al.): x_i = s * <q, k_i>, m = max x, p_i = exp(x_i - m), o = sum p_i v_i / sum p_i,
 * lse = m + log sum p_i. */
static void attend_row(int d, double s, const uint16_t* q, int n_keys, const uint16_t** kp,
                       const uint16_t** vp, double* x, double* o, double* lse) {
    double m = -INFINITY;
    for (int i = 0; i < n_keys; ++i) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += bf16_to_f64(q[c]) * bf16_to_f64(kp[i][c]);
        x[i] = s * acc;
        if (x[i] > m) m = x[i];
    }
    double sum = 0.0;
    for (int c = 0; c < d; ++c) o[c] = 0.0;
    for (int i = 0; i < n_keys; ++i) {
        double p = exp(x[i] - m);
        sum += p;
        for (int c = 0; c < d; ++c) o[c] += p * bf16_to_f64(vp[i][c]);
    }
    for (int c = 0; c < d; ++c) o[c] /= sum;
    if (lse) *lse = m + log(sum);
}

/* One layer, one sequence.
 *   main row t   (Eq. 1):  keys = prefix slots 0..L-1, then tree nodes a (ascending) with a in anc*(t);
 *   stream (t,j) (Eq. 2):  the keys of main row t, then stream keys (t,1)..(t,j)  [j = 1..gamma].
 * Only main-stream K/V live in the cache (prefix at slots 0..L-1, tree node a at slot L+a);
 * stream K/V come from the transient k_spec/v_spec (Sec. 3.2.1: stream K/V are never cached).
 * Layouts (elements): q_main,o_main [T][H][d]; q_spec,k_spec,v_spec,o_spec [T][gamma][H][d];
 * cache slot s, head h at k_cache + s*slot_stride + h*head_stride.  lse_* may be NULL.
 * node_sel (may be NULL): compute only rows of nodes with node_sel[t] != 0; heads [h0,h1). */
int ssor_msa_attention(int32_t n_heads, int32_t head_dim, int32_t L, int32_t T, int32_t gamma,
                       double sm_scale, const int32_t* parent, const uint16_t* q_main,
                       const uint16_t* q_spec, const uint16_t* k_cache, const uint16_t* v_cache,
                       int64_t slot_stride, int64_t head_stride, const uint16_t* k_spec,
                       const uint16_t* v_spec, double* o_main, double* lse_main, double* o_spec,
                       double* lse_spec, const uint8_t* node_sel, int32_t h0, int32_t h1) {
    if (T < 1 || L < 0 || gamma < 0 || head_dim < 1) return SSOR_BAD_ARG;
    uint8_t* is_anc = (uint8_t*)malloc((size_t)T * T);
    int rc = ssor_tree_build(parent, T, NULL, is_anc, NULL);
    if (rc != SSOR_OK) { free(is_anc); return rc; }
    const int H = n_heads, d = head_dim;
    const int max_keys = L + T + gamma;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = h0; h < h1; ++h) {
        const uint16_t** kp = (const uint16_t**)malloc(sizeof(void*) * (size_t)max_keys);
        const uint16_t** vp = (const uint16_t**)malloc(sizeof(void*) * (size_t)max_keys);
        double* x = (double*)malloc(sizeof(double) * (size_t)max_keys);
        for (int t = 0; t < T; ++t) {
            if (node_sel && !node_sel[t]) continue;
            int n = 0;
            for (int s = 0; s < L; ++s, ++n) {
                kp[n] = k_cache + (int64_t)s * slot_stride + (int64_t)h * head_stride;
                vp[n] = v_cache + (int64_t)s * slot_stride + (int64_t)h * head_stride;
            }
            for (int a = 0; a < T; ++a)
                if (is_anc[(size_t)t * T + a]) {
                    kp[n] = k_cache + (int64_t)(L + a) * slot_stride + (int64_t)h * head_stride;
                    vp[n] = v_cache + (int64_t)(L + a) * slot_stride + (int64_t)h * head_stride;
                    ++n;
                }
            attend_row(d, sm_scale, q_main + ((size_t)t * H + h) * d, n, kp, vp, x,
                       o_main + ((size_t)t * H + h) * d, lse_main ? lse_main + (size_t)t * H + h : NULL);
            for (int j = 1; j <= gamma; ++j) {          /* stream j appends stream key (t,j) */
                size_t idx = (((size_t)t * gamma + (j - 1)) * H + h);
                kp[n] = k_spec + idx * d;
                vp[n] = v_spec + idx * d;
                ++n;
                attend_row(d, sm_scale, q_spec + idx * d, n, kp, vp, x, o_spec + idx * d,
                           lse_spec ? lse_spec + idx : NULL);
            }
        }
        free(kp); free(vp); free(x);
    }
    free(is_anc);
    return SSOR_OK;
}

/* Lowest index maximising row[.]: ascending scan, replaced only on strict '>'.  A NaN is never
 * selected while a comparable value exists (a NaN candidate is replaced by the first comparable
 * entry); a row without any comparable value reports index 0.  Comparisons are IEEE fp32 (-0 == +0,
 * subnormals are ordinary values). */
static int32_t argmax_lowest(const float* row, int32_t n) {
    int32_t best = 0;
    for (int32_t v = 1; v < n; ++v)
        if (row[v] > row[best] || (row[best] != row[best] && row[v] == row[v])) best = v;
    return best;
}

/* Greedy ("hard" matching, App. A.2) verification of one tree draft (Sec. 3.2.2, App. A.1):
 * am[t] = lowest index maximising logits[t][.]; the root is always accepted; node c is valid iff
 * its parent is valid and its draft token equals am[parent]; the deepest valid node wins
 * (lowest index among equally deep ones); the accepted path is root..best, accept_len counts its
 * nodes, the correction token is am[best].  path is padded with -1 up to path_cap entries. */
int ssor_tree_verify(const float* logits, const int32_t* tokens, const int32_t* parent, int32_t T,
                     int32_t vocab, int32_t* accept_len, int32_t* path, int32_t path_cap,
                     int32_t* last_node, int32_t* bonus_token, int32_t* node_argmax) {
    if (T < 1 || vocab < 1) return SSOR_BAD_ARG;
    int32_t* depth = (int32_t*)malloc(sizeof(int32_t) * (size_t)T);
    int32_t* am = (int32_t*)malloc(sizeof(int32_t) * (size_t)T);
    uint8_t* valid = (uint8_t*)malloc((size_t)T);
    int rc = ssor_tree_build(parent, T, depth, NULL, NULL);
    if (rc != SSOR_OK) { free(depth); free(am); free(valid); return rc; }
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const float* row = logits + (size_t)t * vocab;
        am[t] = argmax_lowest(row, vocab);
    }
    valid[0] = 1;
    for (int c = 1; c < T; ++c) valid[c] = (uint8_t)(valid[parent[c]] && tokens[c] == am[parent[c]]);
    int32_t best = 0;
    for (int c = 1; c < T; ++c)
        if (valid[c] && depth[c] > depth[best]) best = c;
    int32_t len = depth[best] + 1;
    if (len > path_cap) { free(depth); free(am); free(valid); return SSOR_BAD_ARG; }
    for (int i = 0; i < path_cap; ++i) path[i] = -1;
    for (int32_t a = best, i = len - 1; a != -1; a = parent[a], --i) path[i] = a;
    *accept_len = len;
    *last_node = best;
    *bonus_token = am[best];
    if (node_argmax) memcpy(node_argmax, am, sizeof(int32_t) * (size_t)T);
    free(depth); free(am); free(valid);
    return SSOR_OK;
}

/* Lazy KV backtracking (App. A.1) of one sequence: in every layer the K/V of accepted node
 * path[i] (slot L+path[i]) moves to slot L+i; the new length is L+len.  Written out of place:
 * dst must already hold a copy of src.  Layer l, slot s, head h, element c sit at
 * base + l*layer_stride + s*slot_stride + h*head_stride + c (elements of 16 bits). */
int ssor_kv_compact(const uint16_t* k_src, const uint16_t* v_src, uint16_t* k_dst, uint16_t* v_dst,
                    int32_t n_layers, int64_t layer_stride, int64_t slot_stride, int64_t head_stride,
                    int32_t n_heads, int32_t head_dim, int32_t L, int32_t len, const int32_t* path,
                    int32_t* new_len) {
    if (len < 1) return SSOR_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int l = 0; l < n_layers; ++l)
        for (int i = 0; i < len; ++i)
            for (int h = 0; h < n_heads; ++h) {
                int64_t from = (int64_t)l * layer_stride + (int64_t)(L + path[i]) * slot_stride + (int64_t)h * head_stride;
                int64_t to = (int64_t)l * layer_stride + (int64_t)(L + i) * slot_stride + (int64_t)h * head_stride;
                for (int c = 0; c < head_dim; ++c) {
                    k_dst[to + c] = k_src[from + c];
                    v_dst[to + c] = v_src[from + c];
                }
            }
    *new_len = L + len;
    return SSOR_OK;
}


/* ------------------------------------------------------------------------------------------------
 * The k best entries of row[.] in descending order, equal values by ascending index; a NaN ranks
 * below every comparable value (rule of argmax_lowest).  Selection by k scans, each taking the best
 * entry not taken yet. */
static void topk_lowest(const float* row, int32_t n, int32_t k, int32_t* idx) {
    for (int32_t r = 0; r < k; ++r) {
        int32_t best = -1;
        for (int32_t v = 0; v < n; ++v) {
            int taken = 0;
            for (int32_t q = 0; q < r; ++q) taken |= (idx[q] == v);
            if (taken) continue;
            if (best < 0 || row[v] > row[best] || (row[best] != row[best] && row[v] == row[v])) best = v;
        }
        idx[r] = best;
    }
}

/* Next draft (Sec. 3.2.2, App. A.1): the correction token is the root; the k best tokens of stream g's
 * logits (the streams of the last accepted node) are the children of every node of level g - 1, so that
 * tokens drawn from stream n are the predecessors of those drawn from stream n + 1.  Nodes are numbered
 * level by level, children of a node in rank order, so parent[i] < i; the full tree has
 * 1 + sum_g k^g nodes (Sec. 3.2.3) and is cut after max_nodes nodes in that order.
 * stream_logits [gamma][vocab]; tokens / parent [max_nodes]. */
int ssor_next_draft(const float* stream_logits, int32_t gamma, int32_t vocab, int32_t k, int32_t bonus_token,
                    int32_t max_nodes, int32_t* n_nodes, int32_t* tokens, int32_t* parent) {
    if (gamma < 0 || vocab < 1 || k < 1 || k > vocab || max_nodes < 1) return SSOR_BAD_ARG;
    int32_t* top = (int32_t*)malloc(sizeof(int32_t) * (size_t)(gamma > 0 ? gamma : 1) * (size_t)k);
    for (int32_t g = 0; g < gamma; ++g) topk_lowest(stream_logits + (size_t)g * vocab, vocab, k, top + (size_t)g * k);
    int32_t n = 0;
    tokens[n] = bonus_token; parent[n] = -1; ++n;
    int32_t level_begin = 0, level_end = 1;                 /* nodes of level g - 1 */
    for (int32_t g = 1; g <= gamma && n < max_nodes; ++g) {
        for (int32_t p = level_begin; p < level_end && n < max_nodes; ++p)
            for (int32_t r = 0; r < k && n < max_nodes; ++r) {
                tokens[n] = top[(size_t)(g - 1) * k + r];
                parent[n] = p;
                ++n;
            }
        level_begin = level_end;
        level_end = n;
    }
    *n_nodes = n;
    free(top);
    return SSOR_OK;
}

/* log of the softmax denominator and (optionally) the entropy of softmax(row), in fp64:
 * m = max x, Z = sum exp(x - m), lse = m + log Z, H = -sum p log p with p = exp(x - m) / Z. */
static double row_lse(const float* row, int32_t n, double* entropy) {
    double m = -INFINITY;
    for (int32_t v = 0; v < n; ++v) if ((double)row[v] > m) m = (double)row[v];
    double z = 0.0, w = 0.0;                                /* w = sum (x - m) exp(x - m) */
    for (int32_t v = 0; v < n; ++v) {
        const double d = (double)row[v] - m, e = exp(d);
        z += e;
        if (e > 0.0) w += d * e;
    }
    if (entropy) *entropy = log(z) - w / z;                 /* -sum p (d - log Z) */
    return m + log(z);
}

/* Re-indexing of a tree after some sub-trees are dropped: keep[c] is cleared for every node with a
 * dropped ancestor, kept nodes are numbered in their old order. */
static int32_t compact_tree(const int32_t* parent, int32_t T, uint8_t* keep, int32_t* new_index, int32_t* kept_nodes,
                            int32_t* new_parent) {
    int32_t n = 0;
    for (int32_t c = 0; c < T; ++c) {
        if (c > 0) keep[c] = (uint8_t)(keep[c] && keep[parent[c]]);
        new_index[c] = keep[c] ? n : -1;
        if (keep[c]) {
            kept_nodes[n] = c;
            new_parent[n] = c == 0 ? -1 : new_index[parent[c]];
            ++n;
        }
    }
    return n;
}

/* Parallel tree pruning (Sec. 3.2.3, App. A.1): the transition probability of the edge parent -> child is
 * the early-exit probability of the child's token at the parent, softmax(z~[parent])[token[child]]; an edge
 * below the threshold drops the child's whole sub-tree; the survivors are re-indexed in their old order.
 * The root is always kept.  decide (may be NULL) replaces the threshold test per node, so that a test can
 * hand in decisions taken elsewhere and check everything that follows from them.
 * logits [T][vocab] early-exit logits; edge_prob [T] (root: 1); keep, new_index, kept_nodes, new_parent [T]. */
int ssor_tree_prune(const float* logits, const int32_t* tokens, const int32_t* parent, int32_t T, int32_t vocab,
                    double threshold, const uint8_t* decide, double* edge_prob, uint8_t* keep, int32_t* new_index,
                    int32_t* n_kept, int32_t* kept_nodes, int32_t* new_parent) {
    if (T < 1 || vocab < 1) return SSOR_BAD_ARG;
    int rc = ssor_tree_build(parent, T, NULL, NULL, NULL);
    if (rc != SSOR_OK) return rc;
    double* lse = (double*)malloc(sizeof(double) * (size_t)T);
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) lse[t] = row_lse(logits + (size_t)t * vocab, vocab, NULL);
    edge_prob[0] = 1.0;
    keep[0] = 1;
    for (int32_t c = 1; c < T; ++c) {
        if (tokens[c] < 0 || tokens[c] >= vocab) { free(lse); return SSOR_BAD_ARG; }
        edge_prob[c] = exp((double)logits[(size_t)parent[c] * vocab + tokens[c]] - lse[parent[c]]);
        keep[c] = decide ? decide[c] : (uint8_t)(edge_prob[c] >= threshold);
    }
    *n_kept = compact_tree(parent, T, keep, new_index, kept_nodes, new_parent);
    free(lse);
    return SSOR_OK;
}

/* The walk shared by the verification variants: given, per node, whether its edge from the parent
 * matches, the deepest node whose whole root path matches wins (lowest index among equally deep ones). */
static int accept_walk(const int32_t* parent, int32_t T, const uint8_t* edge_ok, int32_t* accept_len, int32_t* path,
                       int32_t path_cap, int32_t* last_node) {
    int32_t* depth = (int32_t*)malloc(sizeof(int32_t) * (size_t)T);
    uint8_t* valid = (uint8_t*)malloc((size_t)T);
    int rc = ssor_tree_build(parent, T, depth, NULL, NULL);
    if (rc != SSOR_OK) { free(depth); free(valid); return rc; }
    valid[0] = 1;
    for (int c = 1; c < T; ++c) valid[c] = (uint8_t)(valid[parent[c]] && edge_ok[c]);
    int32_t best = 0;
    for (int c = 1; c < T; ++c)
        if (valid[c] && depth[c] > depth[best]) best = c;
    const int32_t len = depth[best] + 1;
    if (len > path_cap) { free(depth); free(valid); return SSOR_BAD_ARG; }
    for (int i = 0; i < path_cap; ++i) path[i] = -1;
    for (int32_t a = best, i = len - 1; a != -1; a = parent[a], --i) path[i] = a;
    *accept_len = len;
    *last_node = best;
    free(depth); free(valid);
    return SSOR_OK;
}

/* "Soft" matching (App. A.2 names it as the relaxation of the hard criterion, after Medusa's typical
 * acceptance): a draft token is accepted when the main stream gives it a probability of at least
 * min(eps, delta * exp(-H)), H the entropy of the main stream's distribution at the parent.  The
 * correction token is the arg-max of the last accepted node.  decide (may be NULL) replaces the
 * threshold test per node.  edge_prob, node_entropy [T] are outputs (root edge: 1). */
int ssor_tree_verify_soft(const float* logits, const int32_t* tokens, const int32_t* parent, int32_t T, int32_t vocab,
                          double eps, double delta, const uint8_t* decide, int32_t* accept_len, int32_t* path,
                          int32_t path_cap, int32_t* last_node, int32_t* bonus_token, double* edge_prob,
                          double* node_entropy) {
    if (T < 1 || vocab < 1) return SSOR_BAD_ARG;
    int rc = ssor_tree_build(parent, T, NULL, NULL, NULL);
    if (rc != SSOR_OK) return rc;
    double* lse = (double*)malloc(sizeof(double) * (size_t)T);
    uint8_t* ok = (uint8_t*)malloc((size_t)T);
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) lse[t] = row_lse(logits + (size_t)t * vocab, vocab, node_entropy + t);
    edge_prob[0] = 1.0;
    ok[0] = 1;
    for (int32_t c = 1; c < T; ++c) {
        if (tokens[c] < 0 || tokens[c] >= vocab) { free(lse); free(ok); return SSOR_BAD_ARG; }
        const int32_t u = parent[c];
        edge_prob[c] = exp((double)logits[(size_t)u * vocab + tokens[c]] - lse[u]);
        const double bar = fmin(eps, delta * exp(-node_entropy[u]));
        ok[c] = decide ? decide[c] : (uint8_t)(edge_prob[c] >= bar);
    }
    rc = accept_walk(parent, T, ok, accept_len, path, path_cap, last_node);
    if (rc == SSOR_OK) *bonus_token = argmax_lowest(logits + (size_t)(*last_node) * vocab, vocab);
    free(lse); free(ok);
    return rc;
}

/* Verification under top-k sampling at temperature 1 (App. B): the main stream's token at node t is
 * drawn from the softmax over its k largest logits (order of topk_lowest), by inversion with the uniform
 * number u[t] in [0, 1) handed in by the caller: the first rank whose cumulative probability exceeds u[t]
 * (the last rank if rounding leaves none).  A draft token is accepted when it equals the token drawn at
 * its parent; the correction token is the token drawn at the last accepted node.  drawn_in (may be NULL)
 * replaces the draw per node.  node_token [T] is an output. */
int ssor_tree_verify_sampled(const float* logits, const int32_t* tokens, const int32_t* parent, int32_t T, int32_t vocab,
                             int32_t k, const float* u, const int32_t* drawn_in, int32_t* accept_len, int32_t* path,
                             int32_t path_cap, int32_t* last_node, int32_t* bonus_token, int32_t* node_token) {
    if (T < 1 || vocab < 1 || k < 1 || k > vocab) return SSOR_BAD_ARG;
    int rc = ssor_tree_build(parent, T, NULL, NULL, NULL);
    if (rc != SSOR_OK) return rc;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        if (drawn_in) { node_token[t] = drawn_in[t]; continue; }
        const float* row = logits + (size_t)t * vocab;
        int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)k);
        topk_lowest(row, vocab, k, idx);
        double z = 0.0;
        for (int32_t r = 0; r < k; ++r) z += exp((double)row[idx[r]] - (double)row[idx[0]]);
        double cdf = 0.0;
        int32_t pick = k - 1;
        for (int32_t r = 0; r < k; ++r) {
            cdf += exp((double)row[idx[r]] - (double)row[idx[0]]) / z;
            if (cdf > (double)u[t]) { pick = r; break; }
        }
        node_token[t] = idx[pick];
        free(idx);
    }
    uint8_t* ok = (uint8_t*)malloc((size_t)T);
    ok[0] = 1;
    for (int32_t c = 1; c < T; ++c) ok[c] = (uint8_t)(tokens[c] == node_token[parent[c]]);
    rc = accept_walk(parent, T, ok, accept_len, path, path_cap, last_node);
    if (rc == SSOR_OK) *bonus_token = node_token[*last_node];
    free(ok);
    return rc;
}

/* fp32 -> bf16, round to nearest even (finite inputs) */
static uint16_t f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}
static float bf16_to_f32(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* Stream insertion (Eq. 3) with the identity for f, as in all of the paper's experiments (App. A.2):
 * S_tj = M_t + P_j.  One fp32 addition per element, rounded to bf16.
 * m [rows][hidden], p [gamma][hidden], out [rows][gamma][hidden]. */
int ssor_stream_insert(const uint16_t* m, const uint16_t* p, uint16_t* out, int64_t rows, int32_t gamma, int32_t hidden) {
    if (rows < 0 || gamma < 1 || hidden < 1) return SSOR_BAD_ARG;
    for (int64_t t = 0; t < rows; ++t)
        for (int32_t j = 0; j < gamma; ++j)
            for (int32_t c = 0; c < hidden; ++c) {
                const float s = bf16_to_f32(m[t * hidden + c]) + bf16_to_f32(p[(int64_t)j * hidden + c]);
                out[(t * gamma + j) * hidden + c] = f32_to_bf16(s);
            }
    return SSOR_OK;
}

/* Value rotation (App. B, Eq. 7): V_tn = V_t e^{i eps n}, n = 1..gamma.  Consecutive pairs of a value
 * vector are the real and imaginary part of a complex number; stream n's value is the main stream's
 * rotated by the angle eps * n.  cos_sin [gamma][2] holds cos and sin of eps * n as fp32; each product,
 * difference and sum is one fp32 operation, the results are rounded to bf16.
 * v [rows][width] (width even), out [rows][gamma][width]. */
int ssor_value_rotate(const uint16_t* v, uint16_t* out, int64_t rows, int32_t gamma, int32_t width, const float* cos_sin) {
    if (rows < 0 || gamma < 1 || width < 2 || (width & 1)) return SSOR_BAD_ARG;
    for (int64_t t = 0; t < rows; ++t)
        for (int32_t n = 0; n < gamma; ++n) {
            const float cs = cos_sin[2 * n], sn = cos_sin[2 * n + 1];
            for (int32_t c = 0; c < width; c += 2) {
                const float re = bf16_to_f32(v[t * width + c]), im = bf16_to_f32(v[t * width + c + 1]);
                const float a = re * cs, b = im * sn, d = re * sn, e = im * cs;
                out[(t * gamma + n) * width + c] = f32_to_bf16(a - b);
                out[(t * gamma + n) * width + c + 1] = f32_to_bf16(d + e);
            }
        }
    return SSOR_OK;
}

int ssor_max_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void ssor_set_threads(int n) {
#ifdef _OPENMP
    extern void omp_set_num_threads(int);
    omp_set_num_threads(n);
#else
    (void)n;
#endif
}
