// Stream initialisation (Eq. 3 with the identity transformation) and the value-rotation stream variant
// (App. B, Eq. 7): element-wise, HBM-bound, 16 bytes per thread and step.  Compiled without fast-math: each
// product, difference and sum is one IEEE fp32 operation, so the results are defined bit by bit.
#include <cuda_bf16.h>
#include <math.h>

#include "ss_common.cuh"

namespace ss {

struct RotTable {
    float cs[SS_MAX_GAMMA], sn[SS_MAX_GAMMA];
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// out[t][j][c] = m[t][c] + p[j][c]; one thread per (row, stream, 8 elements)
__global__ void __launch_bounds__(256)
stream_insert_kernel(const uint4* __restrict__ m, const uint4* __restrict__ p, uint4* __restrict__ out, long long rows, int gamma, int vec) {
    wait_for_previous_kernel();
    const long long total = rows * gamma * vec;
    for (long long w = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; w < total; w += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int c = static_cast<int>(w % vec);
        const long long tj = w / vec;
        const int j = static_cast<int>(tj % gamma);
        const long long t = tj / gamma;
        const uint4 a = m[t * vec + c], b = __ldg(p + static_cast<long long>(j) * vec + c);
        uint4 r;
        r.x = pack2(__fadd_rn(bf16_lo(a.x), bf16_lo(b.x)), __fadd_rn(bf16_hi(a.x), bf16_hi(b.x)));
        r.y = pack2(__fadd_rn(bf16_lo(a.y), bf16_lo(b.y)), __fadd_rn(bf16_hi(a.y), bf16_hi(b.y)));
        r.z = pack2(__fadd_rn(bf16_lo(a.z), bf16_lo(b.z)), __fadd_rn(bf16_hi(a.z), bf16_hi(b.z)));
        r.w = pack2(__fadd_rn(bf16_lo(a.w), bf16_lo(b.w)), __fadd_rn(bf16_hi(a.w), bf16_hi(b.w)));
        out[w] = r;
    }
}

// a 32-bit word holds one complex number (re in the low half, im in the high half)
__device__ __forceinline__ uint32_t rotate_word(uint32_t w, float cs, float sn) {
    const float re = bf16_lo(w), im = bf16_hi(w);
    return pack2(__fsub_rn(__fmul_rn(re, cs), __fmul_rn(im, sn)), __fadd_rn(__fmul_rn(re, sn), __fmul_rn(im, cs)));
}

// out[t][n][c] = v[t][c] rotated by eps * (n + 1); one thread per (row, 8 elements), all streams
__global__ void __launch_bounds__(256)
value_rotate_kernel(const uint4* __restrict__ v, uint4* __restrict__ out, long long rows, int gamma, int vec, RotTable tab) {
    wait_for_previous_kernel();
    const long long total = rows * vec;
    for (long long w = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; w < total; w += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int c = static_cast<int>(w % vec);
        const long long t = w / vec;
        const uint4 a = v[w];
        for (int n = 0; n < gamma; ++n) {
            const float cs = tab.cs[n], sn = tab.sn[n];
            uint4 r;
            r.x = rotate_word(a.x, cs, sn); r.y = rotate_word(a.y, cs, sn);
            r.z = rotate_word(a.z, cs, sn); r.w = rotate_word(a.w, cs, sn);
            out[(t * gamma + n) * vec + c] = r;
        }
    }
}

static int grid_for(long long items) {
    long long g = (items + 255) / 256;
    const long long cap = static_cast<long long>(sm_count()) * 8;
    if (g > cap) g = cap;
    return g < 1 ? 1 : static_cast<int>(g);
}

}  // namespace ss

extern "C" int32_t ss_stream_insert(const void* main_hidden, const void* stream_emb, void* out, int64_t rows, int32_t gamma,
                                    int32_t hidden, void* stream) {
    if (rows < 0 || gamma < 1 || hidden < 8) return SS_ERR_INVALID_ARG;
    if (gamma > SS_MAX_GAMMA || (hidden & 7)) return SS_ERR_UNSUPPORTED;
    if (rows == 0) return SS_OK;                                   // nothing to do: the buffers may be empty
    if (!main_hidden || !stream_emb || !out) return SS_ERR_INVALID_ARG;
    if (!ss::aligned16(main_hidden) || !ss::aligned16(stream_emb) || !ss::aligned16(out)) return SS_ERR_INVALID_ARG;
    const int vec = hidden / 8;
    const cudaError_t err = ss::launch_after_previous(ss::stream_insert_kernel, dim3(ss::grid_for(rows * gamma * vec)), dim3(256),
                                                      static_cast<cudaStream_t>(stream), static_cast<const uint4*>(main_hidden),
                                                      static_cast<const uint4*>(stream_emb), static_cast<uint4*>(out),
                                                      static_cast<long long>(rows), gamma, vec);
    return err == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}

extern "C" int32_t ss_value_rotate(const void* v_main, void* v_streams, int64_t rows, int32_t gamma, int32_t width, float epsilon,
                                   void* stream) {
    if (rows < 0 || gamma < 1 || width < 8 || !(epsilon == epsilon)) return SS_ERR_INVALID_ARG;
    if (gamma > SS_MAX_GAMMA || (width & 7)) return SS_ERR_UNSUPPORTED;
    if (rows == 0) return SS_OK;                                   // nothing to do: the buffers may be empty
    if (!v_main || !v_streams) return SS_ERR_INVALID_ARG;
    if (!ss::aligned16(v_main) || !ss::aligned16(v_streams)) return SS_ERR_INVALID_ARG;
    ss::RotTable tab = {};
    for (int n = 0; n < gamma; ++n) {
        const double ang = static_cast<double>(epsilon) * (n + 1);
        tab.cs[n] = static_cast<float>(cos(ang));
        tab.sn[n] = static_cast<float>(sin(ang));
    }
    const int vec = width / 8;
    const cudaError_t err = ss::launch_after_previous(ss::value_rotate_kernel, dim3(ss::grid_for(rows * vec)), dim3(256),
                                                      static_cast<cudaStream_t>(stream), static_cast<const uint4*>(v_main),
                                                      static_cast<uint4*>(v_streams), static_cast<long long>(rows), gamma, vec, tab);
    return err == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}
