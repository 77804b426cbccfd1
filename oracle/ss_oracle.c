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
 * enumeration; sequential-copy brute force for the compaction.  Nothing here is unpinned.
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
 * the path root..t, t itself included ("child tokens attend to all predecessors starting
 * from root ... and itself", attention-mask figure of App. A). */
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
        int32_t best = 0;
        for (int32_t v = 1; v < vocab; ++v)
            if (row[v] > row[best]) best = v;          /* strict '>' keeps the lowest index */
        am[t] = best;
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
