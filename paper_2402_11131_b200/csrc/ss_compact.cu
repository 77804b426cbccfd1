// Lazy KV-cache backtracking (App. A.1): gather the accepted path's K/V into slots L..L+len-1,
// in place, in every layer, with one launch.
//
// Each thread owns one 16-byte column (a slice of one head's row) of one (layer, sequence, K|V) and
// walks the path in ascending order.  path[i] >= i and the path is strictly increasing, so a
// destination slot L+i is never a source of a later copy; a thread batches kBatch loads before its
// stores, which stays safe because every source of a later batch lies past every slot written so far.
#include "ss_common.cuh"

namespace ss {

constexpr int kCompactThreads = 128;
constexpr int kBatch = 8;

__global__ void __launch_bounds__(kCompactThreads)
kv_compact_kernel(uint4* __restrict__ k_all, uint4* __restrict__ v_all, int n_heads, int chunks_per_head,
                  int64_t layer_stride16, int64_t slot_stride16, int64_t head_stride16,
                  const int64_t* __restrict__ kv_start, const int32_t* __restrict__ kv_len_in,
                  const int32_t* __restrict__ accept_len, const int32_t* __restrict__ accept_path) {
    const int layer = blockIdx.y, b = blockIdx.z;
    const int cols = n_heads * chunks_per_head;          // 16-byte columns per K (or V) slot
    const int col2 = blockIdx.x * kCompactThreads + threadIdx.x;
    wait_for_previous_kernel();
    const int L = kv_len_in[b];
    int len = accept_len[b];
    len = max(0, min(len, SS_PATH_STRIDE));
    if (col2 < 2 * cols) {
        uint4* base = (col2 < cols) ? k_all : v_all;
        const int col = (col2 < cols) ? col2 : col2 - cols;
        const int h = col / chunks_per_head, c = col - h * chunks_per_head;
        base += layer * layer_stride16 + (kv_start[b] + L) * slot_stride16 + h * head_stride16 + c;
        const int32_t* path = accept_path + static_cast<size_t>(b) * SS_PATH_STRIDE;
        for (int i0 = 0; i0 < len; i0 += kBatch) {
            uint4 regs[kBatch];
            int src[kBatch];
            #pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int i = i0 + k;
                src[k] = (i < len) ? path[i] : -1;
                if (src[k] >= 0 && src[k] != i) regs[k] = base[src[k] * slot_stride16];
            }
            #pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int i = i0 + k;
                if (src[k] >= 0 && src[k] != i) base[i * slot_stride16] = regs[k];
            }
        }
    }
}

// kv_len_out may alias kv_len_in, which every CTA of the gather reads: the lengths are updated by
// a second, stream-ordered launch.

__global__ void kv_len_update_kernel(const int32_t* __restrict__ kv_len_in, const int32_t* __restrict__ accept_len,
                                     int32_t* __restrict__ kv_len_out, int batch) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    wait_for_previous_kernel();      // the gather has read the old lengths
    if (b < batch) kv_len_out[b] = kv_len_in[b] + max(0, min(accept_len[b], SS_PATH_STRIDE));
}

}  // namespace ss

extern "C" int32_t ss_kv_compact(void* k_cache_all, void* v_cache_all, const ss_cache_layout* layout,
                                 int32_t batch, const int64_t* kv_start, const int32_t* kv_len_in,
                                 const int32_t* accept_len, const int32_t* accept_path, int32_t* kv_len_out,
                                 void* stream) {
    if (!k_cache_all || !v_cache_all || !layout || !kv_start || !kv_len_in || !accept_len || !accept_path ||
        !kv_len_out)
        return SS_ERR_INVALID_ARG;
    const ss_cache_layout& lo = *layout;
    if (batch < 1 || batch > 65535 || lo.n_layers < 1 || lo.n_layers > 65535 || lo.n_heads < 1 || lo.head_dim < 1)
        return SS_ERR_INVALID_ARG;
    // 16-byte columns: head rows, and all strides, must be multiples of 8 bf16 elements
    if ((lo.head_dim & 7) || (lo.layer_stride & 7) || (lo.slot_stride & 7) || (lo.head_stride & 7))
        return SS_ERR_UNSUPPORTED;
    if (!ss::aligned16(k_cache_all) || !ss::aligned16(v_cache_all)) return SS_ERR_INVALID_ARG;
    const int chunks_per_head = lo.head_dim / 8;
    const int cols2 = 2 * lo.n_heads * chunks_per_head;
    dim3 grid((cols2 + ss::kCompactThreads - 1) / ss::kCompactThreads, lo.n_layers, batch);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // both launches may be scheduled while their predecessor drains; each waits for it before touching memory
    if (ss::launch_after_previous(ss::kv_compact_kernel, grid, dim3(ss::kCompactThreads), s, static_cast<uint4*>(k_cache_all),
                                  static_cast<uint4*>(v_cache_all), lo.n_heads, chunks_per_head, lo.layer_stride / 8,
                                  lo.slot_stride / 8, lo.head_stride / 8, kv_start, kv_len_in, accept_len,
                                  accept_path) != cudaSuccess)
        return SS_ERR_CUDA;
    return ss::launch_after_previous(ss::kv_len_update_kernel, dim3((batch + 127) / 128), dim3(128), s, kv_len_in, accept_len,
                                     kv_len_out, batch) == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}
