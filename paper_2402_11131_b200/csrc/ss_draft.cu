// Draft management around the attention: the next tree draft (Sec. 3.2.2, App. A.1), parallel tree pruning
// (Sec. 3.2.3), and the soft / sampled variants of the verification (App. A.2, App. B).
//
// All of them are one HBM-bound pass over rows of fp32 logits followed by a few dozen integer steps per
// sequence.  One kernel per call: a (chunk, row, sequence) grid scans the rows with 128-bit loads and leaves
// a small partial per chunk (the k best entries, or the maximum with the softmax sums); the last CTA to
// finish a sequence (arrival counter, nobody waits) merges the partials and does the sequence's tail.
//
// Order of logits.  Entries are ranked by an integer key that is monotone in the IEEE order of fp32 values,
// with -0 == +0 and every NaN below -inf, and equal keys by ascending index: the rule of the arg-max of the
// verification, as a total order.  Compiled without fast-math: nothing is flushed or reassociated.
#include "ss_common.cuh"

namespace ss {

constexpr int kScanThreads = 256;
constexpr int kScanChunk = 4096;          // logits per CTA
constexpr int kScanPerThread = kScanChunk / kScanThreads;
constexpr int kMaxTopK = SS_MAX_TOPK;

__device__ __forceinline__ uint32_t order_key(float x) {
    if (x != x) return 0u;
    x += 0.0f;                                         // -0 -> +0
    const uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_value(uint32_t key) {
    if (key == 0u) return __uint_as_float(0x7fc00000u);
    return __uint_as_float((key & 0x80000000u) ? (key ^ 0x80000000u) : ~key);
}
// larger = better: (key, lower index first)
__device__ __forceinline__ unsigned long long entry(float x, int idx) {
    return (static_cast<unsigned long long>(order_key(x)) << 32) | (0xFFFFFFFFu - static_cast<uint32_t>(idx));
}
__device__ __forceinline__ int entry_index(unsigned long long e) { return static_cast<int>(0xFFFFFFFFu - static_cast<uint32_t>(e)); }
__device__ __forceinline__ float entry_value(unsigned long long e) { return key_value(static_cast<uint32_t>(e >> 32)); }

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
    #pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, v, off);
        v = o > v ? o : v;
    }
    return v;
}

// the chunk's elements of this thread: 4 consecutive floats per step (or one by one when the row is not 16-byte aligned)
template <typename F>
__device__ __forceinline__ void for_chunk(const float* row, int vocab, int chunk, F&& f) {
    const int lo = chunk * kScanChunk, hi = min(vocab, lo + kScanChunk);
    if ((vocab & 3) == 0) {
        const float4* row4 = reinterpret_cast<const float4*>(row);
        #pragma unroll
        for (int s = 0; s < kScanPerThread / 4; ++s) {
            const int i = lo / 4 + s * kScanThreads + static_cast<int>(threadIdx.x);
            if (i < hi / 4) {
                const float4 x = __ldcs(row4 + i);
                f(x.x, 4 * i); f(x.y, 4 * i + 1); f(x.z, 4 * i + 2); f(x.w, 4 * i + 3);
            }
        }
    } else {
        #pragma unroll
        for (int s = 0; s < kScanPerThread; ++s) {
            const int i = lo + s * kScanThreads + static_cast<int>(threadIdx.x);
            if (i < hi) f(row[i], i);
        }
    }
}

// ---- scan 1: the k best entries of a chunk -> part[k] (descending; 0 = none) ---------------------------------
__device__ void chunk_topk(const float* row, int vocab, int chunk, int k, unsigned long long* part) {
    unsigned long long best[kMaxTopK];
    #pragma unroll
    for (int r = 0; r < kMaxTopK; ++r) best[r] = 0ull;
    for_chunk(row, vocab, chunk, [&](float x, int i) {
        unsigned long long e = entry(x, i);
        #pragma unroll
        for (int r = 0; r < kMaxTopK; ++r) {            // insertion into the sorted list
            if (e > best[r]) { const unsigned long long t = best[r]; best[r] = e; e = t; }
        }
    });
    // k rounds over the block: the best head wins and its owner moves on
    __shared__ unsigned long long s_w[kScanThreads / 32];
    __shared__ unsigned long long s_pick;
    int pos = 0;
    for (int r = 0; r < k; ++r) {
        unsigned long long head = 0ull;
        #pragma unroll
        for (int q = 0; q < kMaxTopK; ++q) head = (q == pos) ? best[q] : head;
        const unsigned long long wmax = warp_max_u64(head);
        if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = wmax;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long m = s_w[0];
            for (int w = 1; w < kScanThreads / 32; ++w) m = s_w[w] > m ? s_w[w] : m;
            s_pick = m;
            part[r] = m;
        }
        __syncthreads();
        if (head != 0ull && head == s_pick) ++pos;        // entries are unique (the index is part of them)
    }
}

// ---- scan 2: maximum (lowest index), Z = sum exp(x - m), W = sum (x - m) exp(x - m) of a chunk -----------------
struct Stats {
    unsigned long long best;      // entry of the maximum
    float z, w;
};
__device__ __forceinline__ Stats merge_stats(const Stats& a, const Stats& b) {
    Stats r;
    r.best = a.best > b.best ? a.best : b.best;
    const float m = entry_value(r.best), ma = entry_value(a.best), mb = entry_value(b.best);
    r.z = 0.f; r.w = 0.f;
    if (a.z > 0.f) { const float e = expf(ma - m); r.z += a.z * e; r.w += (a.w + (ma - m) * a.z) * e; }
    if (b.z > 0.f) { const float e = expf(mb - m); r.z += b.z * e; r.w += (b.w + (mb - m) * b.z) * e; }
    return r;
}
__device__ Stats chunk_stats(const float* row, int vocab, int chunk) {
    float x[kScanPerThread];
    int n = 0;
    Stats s;
    s.best = 0ull; s.z = 0.f; s.w = 0.f;
    for_chunk(row, vocab, chunk, [&](float v, int i) {
        const unsigned long long e = entry(v, i);
        s.best = e > s.best ? e : s.best;
        #pragma unroll
        for (int q = 0; q < kScanPerThread; ++q) x[q] = (q == n) ? v : x[q];
        ++n;
    });
    if (n > 0) {
        const float m = entry_value(s.best);
        #pragma unroll
        for (int q = 0; q < kScanPerThread; ++q)
            if (q < n) { const float d = x[q] - m, e = expf(d); s.z += e; if (e > 0.f) s.w += d * e; }
    }
    #pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Stats o;
        o.best = __shfl_xor_sync(0xffffffffu, s.best, off);
        o.z = __shfl_xor_sync(0xffffffffu, s.z, off);
        o.w = __shfl_xor_sync(0xffffffffu, s.w, off);
        s = merge_stats(s, o);
    }
    __shared__ Stats s_st[kScanThreads / 32];
    if ((threadIdx.x & 31) == 0) s_st[threadIdx.x >> 5] = s;
    __syncthreads();
    Stats r = s_st[0];
    for (int w = 1; w < kScanThreads / 32; ++w) r = merge_stats(r, s_st[w]);
    return r;
}

// The k best of n_cand chunk candidates (kMaxTopK per chunk, the first k of each meaningful), by one warp: the lanes
// share the candidates (four each in registers, more are read again in every round) and k rounds of a warp
// maximum pick them in order (candidates are unique: the next best is the largest one below the last).
// Every lane gets top[0 .. k).
__device__ __forceinline__ void warp_topk(const unsigned long long* cand, int n_cand, int k, unsigned long long (&top)[kMaxTopK]) {
    const int lane = threadIdx.x & 31;
    unsigned long long mine[4];
    #pragma unroll
    for (int q = 0; q < 4; ++q) {
        const int j = lane + 32 * q;
        mine[q] = (j < n_cand && (j % kMaxTopK) < k) ? __ldcg(cand + j) : 0ull;
    }
    unsigned long long below = ~0ull;
    #pragma unroll
    for (int r = 0; r < kMaxTopK; ++r) top[r] = 0ull;
    for (int q = 0; q < k; ++q) {
        unsigned long long m = 0ull;
        #pragma unroll
        for (int r = 0; r < 4; ++r)
            if (mine[r] < below && mine[r] > m) m = mine[r];
        for (int j = lane + 128; j < n_cand; j += 32) {
            const unsigned long long e = (j % kMaxTopK) < k ? __ldcg(cand + j) : 0ull;
            if (e < below && e > m) m = e;
        }
        m = warp_max_u64(m);
        #pragma unroll
        for (int r = 0; r < kMaxTopK; ++r) top[r] = (r == q) ? m : top[r];
        below = m;
    }
}

// the last CTA of a sequence to get here returns true (its threads then see every other CTA's partials)
__device__ bool arrive_last(int32_t* counter, int expected) {
    __shared__ bool s_last;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(counter, 1) == expected - 1;
    }
    __syncthreads();
    if (s_last) __threadfence();
    return s_last;
}

// deepest node whose whole root path is ok (lowest index among equally deep ones); one thread
__device__ void accept_walk(int T, const int32_t* parent, const int32_t* depth, unsigned long long ok, int32_t* path, int* best_out,
                            int* len_out) {
    unsigned long long valid = 1ull;
    int best = 0, best_depth = 0;
    for (int c = 1; c < T; ++c) {
        const int p = parent[c];
        if (p >= 0 && ((valid >> p) & 1ull) && ((ok >> c) & 1ull)) {
            valid |= 1ull << c;
            if (depth[c] > best_depth) { best = c; best_depth = depth[c]; }
        }
    }
    const int len = best_depth + 1;
    for (int a = best, i = len - 1; a >= 0 && i >= 0; a = parent[a], --i) path[i] = a;
    for (int i = len; i < SS_PATH_STRIDE; ++i) path[i] = -1;
    *best_out = best; *len_out = len;
}

// =============================================================================================================
// Next draft: the k best tokens of each of the gamma stream-logit rows of the last accepted node; tree of
// 1 + sum_g k^g nodes (cut after max_nodes), level by level, children of a node in rank order.
__global__ void __launch_bounds__(kScanThreads)
next_draft_kernel(const float* __restrict__ stream_logits, int n_rows, const int32_t* __restrict__ row_index,
                  const int32_t* __restrict__ bonus_token, int gamma, int vocab, int k, int max_nodes, int n_chunks,
                  int32_t* __restrict__ draft_tokens, ss_tree_desc* __restrict__ trees, int32_t* __restrict__ counters,
                  unsigned long long* __restrict__ partials) {
    const int chunk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    wait_for_previous_kernel();
    int r = row_index ? row_index[b] : 0;
    r = min(max(r, 0), n_rows - 1);
    const float* row = stream_logits + ((static_cast<size_t>(b) * n_rows + r) * gamma + g) * vocab;
    unsigned long long* part = partials + ((static_cast<size_t>(b) * gamma + g) * n_chunks + chunk) * kMaxTopK;
    chunk_topk(row, vocab, chunk, k, part);
    if (!arrive_last(&counters[b], n_chunks * gamma)) return;

    __shared__ int32_t s_top[SS_MAX_GAMMA][kMaxTopK];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp < gamma) {                                   // one warp per stream: k rounds over its chunks' candidates
        unsigned long long top[kMaxTopK];
        warp_topk(partials + (static_cast<size_t>(b) * gamma + warp) * n_chunks * kMaxTopK, n_chunks * kMaxTopK, k, top);
        #pragma unroll
        for (int q = 0; q < kMaxTopK; ++q)
            if (lane == 0 && q < k) s_top[warp][q] = entry_index(top[q]);
    }
    __syncthreads();
    // node i of the full k-ary tree: level g (1-based), offset o within the level; parent = level(g-1) start + o / k
    __shared__ int32_t s_parent[SS_MAX_NODES], s_depth[SS_MAX_NODES];
    int total = 1;
    {
        long long sz = 1, acc = 1;
        for (int lev = 1; lev <= gamma; ++lev) { sz *= k; acc += sz; if (acc >= max_nodes) { acc = max_nodes; break; } }
        total = static_cast<int>(acc);
    }
    const int i = threadIdx.x;
    if (i < SS_MAX_NODES) {
        int par = -1, dep = 0, tok = bonus_token[b];
        if (i > 0 && i < total) {
            long long start = 1, sz = k, prev_start = 0;
            int lev = 1;
            while (i >= start + sz) { prev_start = start; start += sz; sz *= k; ++lev; }
            const int o = static_cast<int>(i - start);
            par = static_cast<int>(prev_start) + o / k;
            dep = lev;
            tok = s_top[lev - 1][o % k];
        }
        s_parent[i] = i < total ? par : -1;
        s_depth[i] = i < total ? dep : 0;
        if (i < max_nodes) draft_tokens[static_cast<size_t>(b) * max_nodes + i] = i < total ? tok : -1;
    }
    __syncthreads();
    if (i < SS_MAX_NODES) {
        unsigned long long anc = 0ull;
        if (i < total) for (int a2 = i; a2 >= 0; a2 = s_parent[a2]) anc |= 1ull << a2;
        trees[b].parent[i] = s_parent[i];
        trees[b].depth[i] = s_depth[i];
        trees[b].anc_mask[i] = anc;
    }
    if (i == 0) {
        int md = 0;
        for (int q = 0; q < total; ++q) md = max(md, s_depth[q]);
        trees[b].n_nodes = total; trees[b].gamma = gamma; trees[b].max_depth = md; trees[b].reserved = 0;
        counters[b] = 0;                                  // leave the workspace ready for the next call
    }
}

// =============================================================================================================
// Row statistics of every node's logits, then per sequence either the pruning of the tree (mode 0) or the
// soft verification (mode 1).
struct NodeTailArgs {
    int mode;
    float threshold, eps, delta;
    float* edge_prob;                 // [B][max_nodes]
    float* node_entropy;              // mode 1, may be null
    int32_t *new_index, *kept_nodes, *kept_tokens;     // mode 0
    ss_tree_desc* pruned_trees;                         // mode 0
    int32_t *accept_len, *accept_path, *last_node, *bonus_token;   // mode 1
};

// Pruning, after the edges are judged: a node survives when every edge of its root path is ok; survivors keep
// their order.  One thread sweeps the nodes (parent[c] < c) over shared-memory copies; all threads write the
// results out.  Called by every thread of the CTA.
__device__ void prune_tail(int T, int max_nodes, int b, unsigned long long ok, const int32_t* s_parent, const int32_t* s_depth,
                           const int32_t* s_tok, int gamma, const NodeTailArgs& ta) {
    __shared__ int32_t s_new[SS_MAX_NODES], s_kept[SS_MAX_NODES], s_np[SS_MAX_NODES];
    __shared__ unsigned long long s_anc[SS_MAX_NODES];
    __shared__ int s_n, s_md;
    const int i = threadIdx.x;
    if (i == 0) {
        unsigned long long keep = T > 0 ? 1ull : 0ull;
        int n = 0, md = 0;
        for (int c = 0; c < T; ++c) {
            const bool kp = c == 0 || (((keep >> s_parent[c]) & 1ull) && ((ok >> c) & 1ull));
            if (kp) {
                keep |= 1ull << c;
                const int np = c == 0 ? -1 : s_new[s_parent[c]];
                s_new[c] = n;
                s_kept[n] = c;
                s_np[n] = np;
                s_anc[n] = (np >= 0 ? s_anc[np] : 0ull) | (1ull << n);
                md = max(md, s_depth[c]);
                ++n;
            } else {
                s_new[c] = -1;
            }
        }
        s_n = n; s_md = md;
    }
    __syncthreads();
    const int n = s_n;
    ss_tree_desc* out = ta.pruned_trees + b;
    if (i < max_nodes) ta.new_index[static_cast<size_t>(b) * max_nodes + i] = i < T ? s_new[i] : -1;
    if (i < SS_MAX_NODES) {
        const bool live = i < n;
        const int c = live ? s_kept[i] : 0;
        out->parent[i] = live ? s_np[i] : -1;
        out->depth[i] = live ? s_depth[c] : 0;
        out->anc_mask[i] = live ? s_anc[i] : 0ull;
        if (i < max_nodes) {
            ta.kept_nodes[static_cast<size_t>(b) * max_nodes + i] = live ? c : -1;
            ta.kept_tokens[static_cast<size_t>(b) * max_nodes + i] = live ? s_tok[c] : -1;
        }
    }
    if (i == 0) { out->n_nodes = n; out->gamma = gamma; out->max_depth = s_md; out->reserved = 0; }
}

__global__ void __launch_bounds__(kScanThreads)
node_stats_kernel(const float* __restrict__ logits, const int32_t* __restrict__ tokens, const ss_tree_desc* __restrict__ trees,
                  int max_nodes, int vocab, int n_chunks, NodeTailArgs ta, int32_t* __restrict__ counters, Stats* __restrict__ partials) {
    const int chunk = blockIdx.x, t = blockIdx.y, b = blockIdx.z;
    wait_for_previous_kernel();
    const int T = min(max(trees[b].n_nodes, 0), max_nodes);
    if (t < T) {
        const Stats s = chunk_stats(logits + (static_cast<size_t>(b) * max_nodes + t) * vocab, vocab, chunk);
        if (threadIdx.x == 0) partials[(static_cast<size_t>(b) * max_nodes + t) * n_chunks + chunk] = s;
    }
    if (!arrive_last(&counters[b], n_chunks * max_nodes)) return;

    __shared__ float s_lse[SS_MAX_NODES], s_ent[SS_MAX_NODES];
    __shared__ int32_t s_am[SS_MAX_NODES], s_parent[SS_MAX_NODES], s_depth[SS_MAX_NODES], s_tok[SS_MAX_NODES];
    __shared__ unsigned long long s_ok;
    const int i = threadIdx.x;
    if (i == 0) s_ok = 1ull;
    if (i < T) {
        const Stats* p = partials + (static_cast<size_t>(b) * max_nodes + i) * n_chunks;
        Stats s;
        s.best = 0ull; s.z = 0.f; s.w = 0.f;
        for (int q0 = 0; q0 < n_chunks; q0 += 8) {          // eight partials' loads in flight at once, merged in order
            Stats o[8];
            #pragma unroll
            for (int q = 0; q < 8; ++q) {
                o[q].best = 0ull; o[q].z = 0.f; o[q].w = 0.f;
                if (q0 + q < n_chunks) { o[q].best = __ldcg(&p[q0 + q].best); o[q].z = __ldcg(&p[q0 + q].z); o[q].w = __ldcg(&p[q0 + q].w); }
            }
            #pragma unroll
            for (int q = 0; q < 8; ++q)
                if (q0 + q < n_chunks) s = merge_stats(s, o[q]);
        }
        const float logz = logf(s.z);
        s_lse[i] = entry_value(s.best) + logz;
        s_ent[i] = logz - s.w / s.z;
        s_am[i] = s.best == 0ull ? 0 : entry_index(s.best);
        s_parent[i] = trees[b].parent[i];
        s_depth[i] = trees[b].depth[i];
        s_tok[i] = tokens[static_cast<size_t>(b) * max_nodes + i];
        if (ta.node_entropy) ta.node_entropy[static_cast<size_t>(b) * max_nodes + i] = s_ent[i];
    }
    __syncthreads();
    if (i < T) {
        float prob = 1.f;
        bool ok = true;
        if (i > 0) {
            const int u = s_parent[i], tk = s_tok[i];
            const bool legal = u >= 0 && u < i && tk >= 0 && tk < vocab;
            prob = legal ? expf(__ldcg(logits + (static_cast<size_t>(b) * max_nodes + u) * vocab + tk) - s_lse[u]) : 0.f;
            const float bar = ta.mode == 0 ? ta.threshold : fminf(ta.eps, ta.delta * expf(-s_ent[legal ? u : 0]));
            ok = legal && prob >= bar;
        }
        ta.edge_prob[static_cast<size_t>(b) * max_nodes + i] = prob;
        if (ok && i > 0) atomicOr(&s_ok, 1ull << i);
    }
    __syncthreads();
    const unsigned long long ok = s_ok;
    if (ta.mode == 1) {
        if (i != 0) return;
        int best = 0, len = 1;
        accept_walk(T, s_parent, s_depth, ok, ta.accept_path + static_cast<size_t>(b) * SS_PATH_STRIDE, &best, &len);
        ta.accept_len[b] = len;
        ta.last_node[b] = best;
        ta.bonus_token[b] = s_am[best];
    } else {
        prune_tail(T, max_nodes, b, ok, s_parent, s_depth, s_tok, trees[b].gamma, ta);
        if (i != 0) return;
    }
    counters[b] = 0;
}

// =============================================================================================================
// Verification against tokens drawn from the softmax over each node's k largest logits (temperature 1).
__global__ void __launch_bounds__(kScanThreads)
sampled_verify_kernel(const float* __restrict__ logits, const int32_t* __restrict__ tokens, const ss_tree_desc* __restrict__ trees,
                      const float* __restrict__ uniforms, int max_nodes, int vocab, int k, int n_chunks,
                      int32_t* __restrict__ accept_len, int32_t* __restrict__ accept_path, int32_t* __restrict__ last_node,
                      int32_t* __restrict__ bonus_token, int32_t* __restrict__ node_token, int32_t* __restrict__ counters,
                      unsigned long long* __restrict__ partials) {
    const int chunk = blockIdx.x, t = blockIdx.y, b = blockIdx.z;
    wait_for_previous_kernel();
    const int T = min(max(trees[b].n_nodes, 0), max_nodes);
    if (t < T)
        chunk_topk(logits + (static_cast<size_t>(b) * max_nodes + t) * vocab, vocab, chunk, k,
                   partials + ((static_cast<size_t>(b) * max_nodes + t) * n_chunks + chunk) * kMaxTopK);
    if (!arrive_last(&counters[b], n_chunks * max_nodes)) return;

    __shared__ int32_t s_draw[SS_MAX_NODES], s_parent[SS_MAX_NODES], s_depth[SS_MAX_NODES], s_tok[SS_MAX_NODES];
    const int i = threadIdx.x;
    // a warp per node picks the node's k best; its lane 0 draws the token
    const int lane = i & 31, n_cand = n_chunks * kMaxTopK;
    for (int node = i >> 5; node < T; node += kScanThreads / 32) {                     // warp-uniform
        unsigned long long top[kMaxTopK];
        warp_topk(partials + (static_cast<size_t>(b) * max_nodes + node) * n_chunks * kMaxTopK, n_cand, k, top);
        if (lane != 0) continue;
        float x0 = 0.f, z = 0.f, ex[kMaxTopK];
        #pragma unroll
        for (int r = 0; r < kMaxTopK; ++r) {
            if (r == 0) x0 = entry_value(top[0]);
            ex[r] = r < k ? expf(entry_value(top[r]) - x0) : 0.f;
            z += ex[r];
        }
        const float u = uniforms[static_cast<size_t>(b) * max_nodes + node];
        float cdf = 0.f;
        int pick = k - 1;
        bool found = false;
        #pragma unroll
        for (int r = 0; r < kMaxTopK; ++r) {
            if (r < k && !found) {
                cdf += ex[r] / z;
                if (cdf > u) { pick = r; found = true; }
            }
        }
        unsigned long long e = 0ull;
        #pragma unroll
        for (int r = 0; r < kMaxTopK; ++r) e = (r == pick) ? top[r] : e;
        s_draw[node] = entry_index(e);
        if (node_token) node_token[static_cast<size_t>(b) * max_nodes + node] = s_draw[node];
    }
    if (i < T) {
        s_parent[i] = trees[b].parent[i];
        s_depth[i] = trees[b].depth[i];
        s_tok[i] = tokens[static_cast<size_t>(b) * max_nodes + i];
    }
    __syncthreads();
    if (i != 0) return;
    unsigned long long ok = 1ull;
    for (int c = 1; c < T; ++c) {
        const int p = s_parent[c];
        if (p >= 0 && p < c && s_tok[c] == s_draw[p]) ok |= 1ull << c;
    }
    int best = 0, len = 1;
    accept_walk(T, s_parent, s_depth, ok, accept_path + static_cast<size_t>(b) * SS_PATH_STRIDE, &best, &len);
    accept_len[b] = len;
    last_node[b] = best;
    bonus_token[b] = s_draw[best];
    counters[b] = 0;
}

static size_t scan_workspace(int32_t batch, int32_t rows, int32_t vocab, size_t per_chunk) {
    if (batch < 1 || rows < 1 || vocab < 1) return 0;
    const size_t n_chunks = (static_cast<size_t>(vocab) + kScanChunk - 1) / kScanChunk;
    const size_t counters = (static_cast<size_t>(batch) * sizeof(int32_t) + 255) / 256 * 256;
    return kWsHeaderBytes + counters + static_cast<size_t>(batch) * rows * n_chunks * per_chunk;
}

}  // namespace ss

extern "C" size_t ss_next_draft_workspace_bytes(int32_t batch, int32_t gamma, int32_t vocab) {
    return ss::scan_workspace(batch, gamma < 1 ? 1 : gamma, vocab, ss::kMaxTopK * sizeof(unsigned long long));
}

extern "C" int32_t ss_next_draft(const float* stream_logits, int32_t n_rows, const int32_t* row_index, const int32_t* bonus_token,
                                 int32_t batch, int32_t gamma, int32_t vocab, int32_t top_k, int32_t max_nodes,
                                 int32_t* draft_tokens, ss_tree_desc* trees, void* workspace, size_t workspace_bytes, void* stream) {
    if (!stream_logits || !bonus_token || !draft_tokens || !trees || !workspace) return SS_ERR_INVALID_ARG;
    if (batch < 1 || batch > 65535 || n_rows < 1 || vocab < 1 || gamma < 1 || top_k < 1 || max_nodes < 1) return SS_ERR_INVALID_ARG;
    if (gamma > SS_MAX_GAMMA || top_k > SS_MAX_TOPK || top_k > vocab || max_nodes > SS_MAX_NODES) return SS_ERR_UNSUPPORTED;
    if (!ss::aligned16(stream_logits) || !ss::aligned16(workspace)) return SS_ERR_INVALID_ARG;
    if (workspace_bytes < ss_next_draft_workspace_bytes(batch, gamma, vocab)) return SS_ERR_WORKSPACE;
    const int n_chunks = (vocab + ss::kScanChunk - 1) / ss::kScanChunk;
    char* ws = static_cast<char*>(workspace);
    const size_t counter_bytes = (static_cast<size_t>(batch) * sizeof(int32_t) + 255) / 256 * 256;
    int32_t* counters = reinterpret_cast<int32_t*>(ws + ss::kWsHeaderBytes);
    unsigned long long* partials = reinterpret_cast<unsigned long long*>(ws + ss::kWsHeaderBytes + counter_bytes);
    const cudaError_t err = ss::launch_after_previous(ss::next_draft_kernel, dim3(n_chunks, gamma, batch), dim3(ss::kScanThreads),
                                                      static_cast<cudaStream_t>(stream), stream_logits, n_rows, row_index, bonus_token,
                                                      gamma, vocab, top_k, max_nodes, n_chunks, draft_tokens, trees, counters, partials);
    return err == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}

extern "C" size_t ss_tree_prune_workspace_bytes(int32_t batch, int32_t max_nodes, int32_t vocab) {
    return ss::scan_workspace(batch, max_nodes, vocab, sizeof(ss::Stats));
}

static int32_t launch_node_stats(const float* logits, const int32_t* tokens, const ss_tree_desc* trees, int32_t batch,
                                 int32_t max_nodes, int32_t vocab, const ss::NodeTailArgs& ta, void* workspace, size_t workspace_bytes,
                                 void* stream) {
    if (!logits || !tokens || !trees || !workspace || !ta.edge_prob) return SS_ERR_INVALID_ARG;
    if (batch < 1 || batch > 65535 || max_nodes < 1 || vocab < 1) return SS_ERR_INVALID_ARG;
    if (max_nodes > SS_MAX_NODES) return SS_ERR_UNSUPPORTED;
    if (!ss::aligned16(logits) || !ss::aligned16(workspace)) return SS_ERR_INVALID_ARG;
    if (workspace_bytes < ss_tree_prune_workspace_bytes(batch, max_nodes, vocab)) return SS_ERR_WORKSPACE;
    const int n_chunks = (vocab + ss::kScanChunk - 1) / ss::kScanChunk;
    char* ws = static_cast<char*>(workspace);
    const size_t counter_bytes = (static_cast<size_t>(batch) * sizeof(int32_t) + 255) / 256 * 256;
    int32_t* counters = reinterpret_cast<int32_t*>(ws + ss::kWsHeaderBytes);
    ss::Stats* partials = reinterpret_cast<ss::Stats*>(ws + ss::kWsHeaderBytes + counter_bytes);
    const cudaError_t err = ss::launch_after_previous(ss::node_stats_kernel, dim3(n_chunks, max_nodes, batch), dim3(ss::kScanThreads),
                                                      static_cast<cudaStream_t>(stream), logits, tokens, trees, max_nodes, vocab,
                                                      n_chunks, ta, counters, partials);
    return err == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}

extern "C" int32_t ss_tree_prune(const float* exit_logits, const int32_t* draft_tokens, const ss_tree_desc* trees, int32_t batch,
                                 int32_t max_nodes, int32_t vocab, float threshold, float* edge_prob, int32_t* new_index,
                                 int32_t* kept_nodes, int32_t* kept_tokens, ss_tree_desc* pruned_trees, void* workspace,
                                 size_t workspace_bytes, void* stream) {
    if (!new_index || !kept_nodes || !kept_tokens || !pruned_trees) return SS_ERR_INVALID_ARG;
    if (!(threshold == threshold)) return SS_ERR_INVALID_ARG;
    ss::NodeTailArgs ta = {};
    ta.mode = 0; ta.threshold = threshold; ta.edge_prob = edge_prob;
    ta.new_index = new_index; ta.kept_nodes = kept_nodes; ta.kept_tokens = kept_tokens; ta.pruned_trees = pruned_trees;
    return launch_node_stats(exit_logits, draft_tokens, trees, batch, max_nodes, vocab, ta, workspace, workspace_bytes, stream);
}

extern "C" int32_t ss_tree_verify_soft(const float* logits, const int32_t* draft_tokens, const ss_tree_desc* trees, int32_t batch,
                                       int32_t max_nodes, int32_t vocab, float eps, float delta, int32_t* accept_len,
                                       int32_t* accept_path, int32_t* last_node, int32_t* bonus_token, float* edge_prob,
                                       float* node_entropy, void* workspace, size_t workspace_bytes, void* stream) {
    if (!accept_len || !accept_path || !last_node || !bonus_token) return SS_ERR_INVALID_ARG;
    if (!(eps == eps) || !(delta == delta)) return SS_ERR_INVALID_ARG;
    ss::NodeTailArgs ta = {};
    ta.mode = 1; ta.eps = eps; ta.delta = delta; ta.edge_prob = edge_prob; ta.node_entropy = node_entropy;
    ta.accept_len = accept_len; ta.accept_path = accept_path; ta.last_node = last_node; ta.bonus_token = bonus_token;
    return launch_node_stats(logits, draft_tokens, trees, batch, max_nodes, vocab, ta, workspace, workspace_bytes, stream);
}

extern "C" size_t ss_tree_verify_sampled_workspace_bytes(int32_t batch, int32_t max_nodes, int32_t vocab) {
    return ss::scan_workspace(batch, max_nodes, vocab, ss::kMaxTopK * sizeof(unsigned long long));
}

extern "C" int32_t ss_tree_verify_sampled(const float* logits, const int32_t* draft_tokens, const ss_tree_desc* trees,
                                          const float* uniforms, int32_t batch, int32_t max_nodes, int32_t vocab, int32_t top_k,
                                          int32_t* accept_len, int32_t* accept_path, int32_t* last_node, int32_t* bonus_token,
                                          int32_t* node_token, void* workspace, size_t workspace_bytes, void* stream) {
    if (!logits || !draft_tokens || !trees || !uniforms || !accept_len || !accept_path || !last_node || !bonus_token || !workspace)
        return SS_ERR_INVALID_ARG;
    if (batch < 1 || batch > 65535 || max_nodes < 1 || vocab < 1 || top_k < 1) return SS_ERR_INVALID_ARG;
    if (max_nodes > SS_MAX_NODES || top_k > SS_MAX_TOPK || top_k > vocab) return SS_ERR_UNSUPPORTED;
    if (!ss::aligned16(logits) || !ss::aligned16(workspace)) return SS_ERR_INVALID_ARG;
    if (workspace_bytes < ss_tree_verify_sampled_workspace_bytes(batch, max_nodes, vocab)) return SS_ERR_WORKSPACE;
    const int n_chunks = (vocab + ss::kScanChunk - 1) / ss::kScanChunk;
    char* ws = static_cast<char*>(workspace);
    const size_t counter_bytes = (static_cast<size_t>(batch) * sizeof(int32_t) + 255) / 256 * 256;
    int32_t* counters = reinterpret_cast<int32_t*>(ws + ss::kWsHeaderBytes);
    unsigned long long* partials = reinterpret_cast<unsigned long long*>(ws + ss::kWsHeaderBytes + counter_bytes);
    const cudaError_t err = ss::launch_after_previous(ss::sampled_verify_kernel, dim3(n_chunks, max_nodes, batch), dim3(ss::kScanThreads),
                                                      static_cast<cudaStream_t>(stream), logits, draft_tokens, trees, uniforms, max_nodes,
                                                      vocab, top_k, n_chunks, accept_len, accept_path, last_node, bonus_token, node_token,
                                                      counters, partials);
    return err == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}
