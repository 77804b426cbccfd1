// Greedy tree verification (Sec. 3.2.2, App. A.1): per-node arg-max over the vocabulary, then a
// scan of the tree for the deepest node whose whole root path matches.
//
// HBM-bound: 4*T*V bytes of logits are read exactly once.  One launch: a (chunk, node, sequence)
// grid scans the logits with 128-bit loads; the last CTA to finish a sequence (arrival counter, no
// waiting) reduces the per-chunk candidates and walks the tree.
#include "ss_common.cuh"

namespace ss {

constexpr int kVerifyThreads = 256;
constexpr int kVerifyChunk = 4096;   // logits per CTA

struct Cand {
    float v;
    int32_t i;
};

// "a is better than b": larger value, or equal value at a lower index (lowest-index arg-max)
__device__ __forceinline__ bool better(float av, int32_t ai, float bv, int32_t bi) {
    return av > bv || (av == bv && ai < bi);
}

__global__ void __launch_bounds__(kVerifyThreads)
tree_verify_kernel(const float* __restrict__ logits, const int32_t* __restrict__ tokens,
                   const ss_tree_desc* __restrict__ trees, int max_nodes, int vocab, int n_chunks,
                   int32_t* __restrict__ accept_len, int32_t* __restrict__ accept_path,
                   int32_t* __restrict__ last_node, int32_t* __restrict__ bonus_token,
                   int32_t* __restrict__ node_argmax, int32_t* __restrict__ counters,
                   Cand* __restrict__ partials) {
    const int chunk = blockIdx.x, t = blockIdx.y, b = blockIdx.z;
    wait_for_previous_kernel();
    const int T = min(max(trees[b].n_nodes, 0), max_nodes);     // a descriptor is never trusted beyond the arrays' extent
    __shared__ Cand s_red[kVerifyThreads / 32];
    __shared__ int32_t s_am[SS_MAX_NODES];
    __shared__ bool s_last;

    if (t < T) {
        const float* row = logits + (static_cast<size_t>(b) * max_nodes + t) * vocab;
        const int lo = chunk * kVerifyChunk;
        const int hi = min(vocab, lo + kVerifyChunk);
        float bv = -INFINITY;
        int32_t bi = 0x7fffffff;
        if ((vocab & 3) == 0) {
            const float4* row4 = reinterpret_cast<const float4*>(row);
            #pragma unroll 4
            for (int i = lo / 4 + threadIdx.x; i < hi / 4; i += kVerifyThreads) {
                const float4 x = __ldcs(row4 + i);
                const int base = i * 4;
                if (better(x.x, base, bv, bi)) { bv = x.x; bi = base; }
                if (better(x.y, base + 1, bv, bi)) { bv = x.y; bi = base + 1; }
                if (better(x.z, base + 2, bv, bi)) { bv = x.z; bi = base + 2; }
                if (better(x.w, base + 3, bv, bi)) { bv = x.w; bi = base + 3; }
            }
        } else {
            for (int i = lo + threadIdx.x; i < hi; i += kVerifyThreads) {
                const float x = row[i];
                if (better(x, i, bv, bi)) { bv = x; bi = i; }
            }
        }
        #pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int32_t oi = __shfl_xor_sync(0xffffffffu, bi, off);
            if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = Cand{bv, bi};
        __syncthreads();
        if (threadIdx.x == 0) {
            Cand c = s_red[0];
            for (int w = 1; w < kVerifyThreads / 32; ++w)
                if (better(s_red[w].v, s_red[w].i, c.v, c.i)) c = s_red[w];
            partials[(static_cast<size_t>(b) * max_nodes + t) * n_chunks + chunk] = c;
        }
    }
    // arrival: every CTA of the sequence counts, the last one finishes the job
    if (threadIdx.x == 0) {
        __threadfence();
        const int expected = n_chunks * max_nodes;
        const int prev = atomicAdd(&counters[b], 1);
        s_last = (prev == expected - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // the tree walk below is one thread's serial loop: its inputs go to shared memory first, loaded by
    // T threads at once, so that no step of the loop waits for global memory
    __shared__ int32_t s_parent[SS_MAX_NODES], s_depth[SS_MAX_NODES], s_tok[SS_MAX_NODES];
    if (threadIdx.x < T) {
        const Cand* p = partials + (static_cast<size_t>(b) * max_nodes + threadIdx.x) * n_chunks;
        float bv = -INFINITY;
        int32_t bi = 0x7fffffff;
        for (int k0 = 0; k0 < n_chunks; k0 += 8) {             // eight candidates' loads in flight at once
            long long raw[8];
            #pragma unroll
            for (int k = 0; k < 8; ++k) raw[k] = k0 + k < n_chunks ? __ldcg(reinterpret_cast<const long long*>(p + k0 + k)) : 0ll;
            #pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (k0 + k < n_chunks) {
                    const float v = __int_as_float(static_cast<int>(raw[k] & 0xffffffffll));
                    const int32_t i = static_cast<int32_t>(raw[k] >> 32);
                    if (better(v, i, bv, bi)) { bv = v; bi = i; }
                }
            }
        }
        // a row without any comparable value (all NaN) reports index 0, like a strict '>' scan
        if (bi == 0x7fffffff) bi = 0;
        s_am[threadIdx.x] = bi;
        if (node_argmax) node_argmax[static_cast<size_t>(b) * max_nodes + threadIdx.x] = bi;
        s_parent[threadIdx.x] = trees[b].parent[threadIdx.x];
        s_depth[threadIdx.x] = trees[b].depth[threadIdx.x];
        s_tok[threadIdx.x] = tokens[static_cast<size_t>(b) * max_nodes + threadIdx.x];
    }
    __syncthreads();
    int32_t* const path = accept_path + static_cast<size_t>(b) * SS_PATH_STRIDE;
    if (threadIdx.x < 32) {
        // validity needs the parent's validity, so sweep in index order (parent[i] < i) with one
        // thread; T <= 64 keeps this trivial
        int best = 0, len = 1;
        if (threadIdx.x == 0) {
            uint64_t valid = 1ull;
            int best_depth = 0;
            for (int c = 1; c < T; ++c) {
                const int p = s_parent[c];
                if (p >= 0 && ((valid >> p) & 1ull) && s_tok[c] == s_am[p]) {
                    valid |= 1ull << c;
                    const int dep = s_depth[c];
                    if (dep > best_depth) { best = c; best_depth = dep; }
                }
            }
            len = best_depth + 1;
            for (int a = best, i = len - 1; a >= 0 && i >= 0; a = s_parent[a], --i) path[i] = a;
            accept_len[b] = len;
            last_node[b] = best;
            bonus_token[b] = s_am[best];
            counters[b] = 0;   // leave the workspace ready for the next call
        }
        len = __shfl_sync(0xffffffffu, len, 0);
        for (int i = len + static_cast<int>(threadIdx.x); i < SS_PATH_STRIDE; i += 32) path[i] = -1;
    }
}

}  // namespace ss

extern "C" size_t ss_tree_verify_workspace_bytes(int32_t batch, int32_t max_nodes, int32_t vocab) {
    if (batch < 1 || max_nodes < 1 || vocab < 1) return 0;
    const size_t n_chunks = (static_cast<size_t>(vocab) + ss::kVerifyChunk - 1) / ss::kVerifyChunk;
    const size_t counters = (static_cast<size_t>(batch) * sizeof(int32_t) + 255) / 256 * 256;
    return ss::kWsHeaderBytes + counters + static_cast<size_t>(batch) * max_nodes * n_chunks * sizeof(ss::Cand);
}

extern "C" int32_t ss_tree_verify(const float* logits, const int32_t* draft_tokens, const ss_tree_desc* trees,
                                  int32_t batch, int32_t max_nodes, int32_t vocab, int32_t* accept_len,
                                  int32_t* accept_path, int32_t* last_node, int32_t* bonus_token,
                                  int32_t* node_argmax, void* workspace, size_t workspace_bytes, void* stream) {
    if (!logits || !draft_tokens || !trees || !accept_len || !accept_path || !last_node || !bonus_token ||
        !workspace)
        return SS_ERR_INVALID_ARG;
    if (batch < 1 || max_nodes < 1 || vocab < 1 || batch > 65535) return SS_ERR_INVALID_ARG;
    if (max_nodes > SS_MAX_NODES) return SS_ERR_UNSUPPORTED;
    if (!ss::aligned16(logits) || !ss::aligned16(workspace)) return SS_ERR_INVALID_ARG;
    if (workspace_bytes < ss_tree_verify_workspace_bytes(batch, max_nodes, vocab)) return SS_ERR_WORKSPACE;
    const int n_chunks = (vocab + ss::kVerifyChunk - 1) / ss::kVerifyChunk;
    char* ws = static_cast<char*>(workspace);
    int32_t* counters = reinterpret_cast<int32_t*>(ws + ss::kWsHeaderBytes);
    const size_t counter_bytes = (static_cast<size_t>(batch) * sizeof(int32_t) + 255) / 256 * 256;
    ss::Cand* partials = reinterpret_cast<ss::Cand*>(ws + ss::kWsHeaderBytes + counter_bytes);
    dim3 grid(n_chunks, max_nodes, batch);
    const cudaError_t err = ss::launch_after_previous(ss::tree_verify_kernel, grid, dim3(ss::kVerifyThreads),
                                                      static_cast<cudaStream_t>(stream), logits, draft_tokens, trees, max_nodes,
                                                      vocab, n_chunks, accept_len, accept_path, last_node, bonus_token,
                                                      node_argmax, counters, partials);
    return err == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Verification without a caller-provided workspace.
//
// Some callers cannot hand this library scratch memory: code that runs where allocating device
// memory is not allowed (inside a region that forbids cudaMalloc, a plug-in that owns no allocator,
// a real-time loop whose memory was fixed at start-up).  For them the scratch of the verification
// kernel lives in this fixed device array, which every GPU that loads the library holds until the
// process exits.  All calls on a device share it, so calls that overlap on that device race.
namespace ss {

static __device__ __align__(256) unsigned char g_verify_static_scratch[SS_VERIFY_STATIC_SCRATCH_BYTES];

// Device address of the array, looked up once per device.  In host code the array's name is only a
// host-side handle, never a device address: the address must come from cudaGetSymbolAddress, taken
// with the device current.
static void* verify_static_scratch_ptr(int32_t* status) {
    static void* cached[64] = {nullptr};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        *status = SS_ERR_CUDA;
        return nullptr;
    }
    if (cached[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_verify_static_scratch) != cudaSuccess || p == nullptr) {
            *status = SS_ERR_CUDA;
            return nullptr;
        }
        cached[dev] = p;
    }
    *status = SS_OK;
    return cached[dev];
}

}  // namespace ss

extern "C" int32_t ss_tree_verify_static(const float* logits, const int32_t* draft_tokens,
                                         const ss_tree_desc* trees, int32_t batch, int32_t max_nodes,
                                         int32_t vocab, int32_t* accept_len, int32_t* accept_path,
                                         int32_t* last_node, int32_t* bonus_token, int32_t* node_argmax,
                                         void* stream) {
    if (!logits || !draft_tokens || !trees || !accept_len || !accept_path || !last_node || !bonus_token)
        return SS_ERR_INVALID_ARG;
    if (batch < 1 || max_nodes < 1 || vocab < 1 || batch > 65535) return SS_ERR_INVALID_ARG;
    if (max_nodes > SS_MAX_NODES) return SS_ERR_UNSUPPORTED;
    if (!ss::aligned16(logits)) return SS_ERR_INVALID_ARG;
    const size_t need = ss_tree_verify_workspace_bytes(batch, max_nodes, vocab);
    if (need == 0 || need > SS_VERIFY_STATIC_SCRATCH_BYTES) return SS_ERR_WORKSPACE;   // beyond the fixed scratch
    int32_t st = SS_OK;
    char* ws = static_cast<char*>(ss::verify_static_scratch_ptr(&st));
    if (ws == nullptr) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array keeps the previous call's contents: the status word and the arrival counters must
    // start at zero (the per-chunk candidates are fully rewritten before they are read)
    const size_t counter_bytes = (static_cast<size_t>(batch) * sizeof(int32_t) + 255) / 256 * 256;
    if (cudaMemsetAsync(ws, 0, ss::kWsHeaderBytes + counter_bytes, s) != cudaSuccess) return SS_ERR_CUDA;
    const int n_chunks = (vocab + ss::kVerifyChunk - 1) / ss::kVerifyChunk;
    int32_t* counters = reinterpret_cast<int32_t*>(ws + ss::kWsHeaderBytes);
    ss::Cand* partials = reinterpret_cast<ss::Cand*>(ws + ss::kWsHeaderBytes + counter_bytes);
    dim3 grid(n_chunks, max_nodes, batch);
    ss::tree_verify_kernel<<<grid, ss::kVerifyThreads, 0, s>>>(
        logits, draft_tokens, trees, max_nodes, vocab, n_chunks, accept_len, accept_path, last_node,
        bonus_token, node_argmax, counters, partials);
    return cudaGetLastError() == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}
