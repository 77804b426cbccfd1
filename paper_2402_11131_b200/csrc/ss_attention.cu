// Tree-masked multi-stream attention, one layer (Eq. 1, Eq. 2): split-KV flash-decode.
//
// Work decomposition.  For sequence b the "extended key sequence" of a head is
//     [0, L_b)                      cached prefix,
//     [L_b, L_b + T_b)              this step's tree nodes (already in the cache, masked by ancestry),
//     [L_b + T_b, L_b + T_b(1+g))   the transient stream keys, node-major: (t,1)..(t,g), (t+1,1)...
// All (sequence, head) pairs are laid end to end in units of 16 keys and the persistent grid cuts
// that line into equal spans, so every CTA streams the same number of K/V bytes whatever the
// batch's length mix.  The cut points are computed on the device from kv_len[], so the host never
// needs the lengths.  A span crossing a pair boundary yields several segments; each segment of a
// pair that is split over CTAs leaves an un-normalised partial (m, l, O) in the workspace, and the
// last CTA to arrive on the pair's counter merges them (no CTA ever waits for another).
//
// Inside a CTA: all (node x stream) query rows of the head are processed against each staged K/V
// tile, 64 rows per pass; warp (rb, kh) owns 16 rows x one 32-key half of the 64-key tile, S = QK^T
// and O += PV run on bf16 tensor-core MMAs with fp32 accumulators, the online softmax lives in
// registers, and the tree / stream mask is evaluated from the node's 64-bit ancestor word only for
// tiles that reach past the prefix.
#include <cuda_bf16.h>

#include "ss_common.cuh"

namespace ss {

constexpr int kThreads = 256;
constexpr int kTileKeys = 64;      // keys per staged tile
constexpr int kUnit = 16;          // scheduling granularity (keys)
constexpr int kRowChunk = 64;      // query rows per pass
constexpr int kStages = 3;
constexpr int kMinUnitsPerCta = 4; // do not spread less than 64 keys per CTA

struct AttnArgs {
    int batch, n_heads, gamma, max_nodes;
    float scale_log2;              // sm_scale * log2(e)
    const __nv_bfloat16* q_main;
    __nv_bfloat16* o_main;
    const __nv_bfloat16* q_spec;
    const __nv_bfloat16* k_spec;
    const __nv_bfloat16* v_spec;
    __nv_bfloat16* o_spec;
    const __nv_bfloat16* k_cache;
    const __nv_bfloat16* v_cache;
    long long slot_stride, head_stride;
    const long long* kv_start;
    const int* kv_len;
    const int* kv_capacity;
    const ss_tree_desc* trees;
    float* lse_main;
    float* lse_spec;
    int* status;                   // workspace word 0
    int* counters;                 // [batch * n_heads]
    float* partials;               // [2 * grid][m_pad][HD + 2]
    int m_pad;                     // rows per partial slot
};

// ---------------------------------------------------------------------------------------------
// small PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int n = valid ? 16 : 0;   // n = 0 zero-fills the 16 bytes
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(n));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// ---------------------------------------------------------------------------------------------
// schedule: the line of 16-key units over all (sequence, head) pairs
struct Schedule {
    long long total_units;
    int g_eff;
};

__device__ __forceinline__ int ext_keys(const AttnArgs& a, int b) {
    return a.kv_len[b] + a.trees[b].n_nodes * (1 + a.gamma);
}
__device__ __forceinline__ long long span_begin(long long total, int g_eff, int c) { return total * c / g_eff; }
// the CTA whose span holds unit x
__device__ __forceinline__ int cta_of(long long total, int g_eff, long long x) {
    return static_cast<int>(((x + 1) * g_eff - 1) / total);
}

template <int HD>
struct Smem {
    static constexpr int kPitch = HD * 2 + 16;                  // bytes per staged row (bank-conflict padding)
    static constexpr int kTileBytes = kTileKeys * kPitch;       // one K (or V) tile
    static constexpr int kStageBytes = 2 * kTileBytes;          // K + V
    static constexpr int kQBytes = kRowChunk * kPitch;
    static constexpr int kPipeBytes = kStages * kStageBytes;
    static constexpr int kMergeBytes = 4 * 16 * (HD + 2) * 4;   // (m, l, O) of the four kh = 1 warps
    static_assert(kMergeBytes <= kPipeBytes, "merge buffer aliases the pipeline stages");
    static constexpr int kTotal = kPipeBytes + kQBytes;
};

template <int HD>
__global__ void __launch_bounds__(kThreads, 1) msa_attention_kernel(const AttnArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
    using S = Smem<HD>;
    __shared__ unsigned long long s_anc[SS_MAX_NODES];
    __shared__ int s_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, q = lane & 3;
    const int rb = warp & 3, kh = warp >> 2;
    const int H = a.n_heads, gamma = a.gamma, rows_per_node = 1 + gamma;

    // ---- schedule ------------------------------------------------------------------------------
    long long total = 0;
    for (int b = 0; b < a.batch; ++b) total += static_cast<long long>(H) * ((ext_keys(a, b) + kUnit - 1) / kUnit);
    if (total == 0) return;
    const int g_eff = static_cast<int>(min(static_cast<long long>(gridDim.x), max(1ll, total / kMinUnitsPerCta)));
    const int cta = blockIdx.x;
    if (cta >= g_eff) return;
    long long u = span_begin(total, g_eff, cta);
    const long long u_end = span_begin(total, g_eff, cta + 1);

    const uint32_t smem_base = smem_u32(smem);
    const uint32_t q_base = smem_base + S::kPipeBytes;

    int b = 0;
    long long pair_base = 0;   // first unit of sequence b
    while (u < u_end) {
        // locate the pair that holds unit u
        int units_b = (ext_keys(a, b) + kUnit - 1) / kUnit;
        while (u >= pair_base + static_cast<long long>(H) * units_b) {
            pair_base += static_cast<long long>(H) * units_b;
            ++b;
            units_b = (ext_keys(a, b) + kUnit - 1) / kUnit;
        }
        const int h = static_cast<int>((u - pair_base) / units_b);
        const long long p0 = pair_base + static_cast<long long>(h) * units_b;   // pair's first unit
        const long long p1 = p0 + units_b;
        const long long seg_end_u = min(u_end, p1);
        const int L = a.kv_len[b];
        const int T = a.trees[b].n_nodes;
        const int M = T * rows_per_node;
        const int E = L + M;                                   // extended keys of the pair
        const int e0 = static_cast<int>(u - p0) * kUnit;
        const int e1 = min(E, static_cast<int>(seg_end_u - p0) * kUnit);
        const bool continuation = (u > p0);
        const int c_first = cta_of(total, g_eff, p0), c_last = cta_of(total, g_eff, p1 - 1);
        const int n_splits = c_last - c_first + 1;
        const bool over_capacity = a.kv_capacity != nullptr && L + T > a.kv_capacity[b];
        if (over_capacity && tid == 0) set_status(a.status, SS_ERR_CAPACITY);
        u = seg_end_u;
        if (over_capacity) continue;

        __syncthreads();   // previous segment is completely done with shared memory
        if (tid < SS_MAX_NODES) s_anc[tid] = a.trees[b].anc_mask[tid];

        const long long seq_slot0 = a.kv_start[b];
        const __nv_bfloat16* kc = a.k_cache + seq_slot0 * a.slot_stride + static_cast<long long>(h) * a.head_stride;
        const __nv_bfloat16* vc = a.v_cache + seq_slot0 * a.slot_stride + static_cast<long long>(h) * a.head_stride;
        const long long spec_row0 = static_cast<long long>(b) * a.max_nodes * gamma;   // [b][0][0]
        float* part = a.partials + static_cast<size_t>(2 * cta + (continuation ? 0 : 1)) * a.m_pad * (HD + 2);

        const int n_tiles = (e1 - e0 + kTileKeys - 1) / kTileKeys;
        const int n_chunks = (M + kRowChunk - 1) / kRowChunk;

        for (int rc = 0; rc < n_chunks; ++rc) {
            const int row_base = rc * kRowChunk;
            __syncthreads();   // shared memory of the previous pass is free; s_anc is visible
            // ---- stage the query rows of this pass -------------------------------------------
            for (int i = tid; i < kRowChunk * (HD / 8); i += kThreads) {
                const int r = i / (HD / 8), ch = i - r * (HD / 8);
                const int row = row_base + r;
                const bool valid = row < M;
                const __nv_bfloat16* src = a.q_main;
                if (valid) {
                    const int t = row / rows_per_node, j = row - t * rows_per_node;
                    if (j == 0)
                        src = a.q_main + ((static_cast<long long>(b) * a.max_nodes + t) * H + h) * HD + ch * 8;
                    else
                        src = a.q_spec + ((spec_row0 + static_cast<long long>(t) * gamma + (j - 1)) * H + h) * HD + ch * 8;
                }
                cp_async16(q_base + r * S::kPitch + ch * 16, src, valid);
            }
            // ---- K/V tile loader ---------------------------------------------------------------
            auto issue_tile = [&](int tile) {
                const uint32_t kdst = smem_base + (tile % kStages) * S::kStageBytes;
                const uint32_t vdst = kdst + S::kTileBytes;
                const int eb = e0 + tile * kTileKeys;
                for (int i = tid; i < kTileKeys * (HD / 8); i += kThreads) {
                    const int r = i / (HD / 8), ch = i - r * (HD / 8);
                    const int e = eb + r;
                    const bool valid = e < e1;
                    const __nv_bfloat16 *ks = kc, *vs = vc;
                    if (valid) {
                        if (e < L + T) {
                            ks = kc + static_cast<long long>(e) * a.slot_stride + ch * 8;
                            vs = vc + static_cast<long long>(e) * a.slot_stride + ch * 8;
                        } else {
                            const long long off = ((spec_row0 + (e - L - T)) * H + h) * HD + ch * 8;
                            ks = a.k_spec + off;
                            vs = a.v_spec + off;
                        }
                    }
                    cp_async16(kdst + r * S::kPitch + ch * 16, ks, valid);
                    cp_async16(vdst + r * S::kPitch + ch * 16, vs, valid);
                }
            };
            #pragma unroll
            for (int s = 0; s < kStages - 1; ++s) {
                if (s < n_tiles) issue_tile(s);
                cp_async_commit();
            }

            // ---- per-thread row info ----------------------------------------------------------
            // thread rows: r_lo = row_base + rb*16 + g, r_hi = r_lo + 8
            int row_id[2];
            unsigned long long anc[2];
            int s_lo[2], s_hi[2];   // visible stream-key range [s_lo, s_hi) in extended key indices
            #pragma unroll
            for (int x = 0; x < 2; ++x) {
                const int row = row_base + rb * 16 + g + 8 * x;
                row_id[x] = row;
                if (row < M) {
                    const int t = row / rows_per_node, j = row - t * rows_per_node;
                    anc[x] = s_anc[t];
                    s_lo[x] = L + T + t * gamma;
                    s_hi[x] = s_lo[x] + j;
                } else {
                    anc[x] = 0ull;
                    s_lo[x] = s_hi[x] = 0;
                }
            }

            uint32_t qf[HD / 16][4];
            float o[HD / 8][4];
            float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
            #pragma unroll
            for (int i = 0; i < HD / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

            const bool warp_active = (row_base + rb * 16) < M;

            for (int tile = 0; tile < n_tiles; ++tile) {
                cp_async_wait<kStages - 2>();
                __syncthreads();
                if (tile + kStages - 1 < n_tiles) issue_tile(tile + kStages - 1);
                cp_async_commit();
                if (tile == 0) {
                    #pragma unroll
                    for (int ks = 0; ks < HD / 16; ++ks)
                        ldmatrix_x4(qf[ks], q_base + (rb * 16 + (lane & 15)) * S::kPitch + ks * 32 + (lane >> 4) * 16);
                }
                if (!warp_active) continue;
                const uint32_t kbase = smem_base + (tile % kStages) * S::kStageBytes;
                const uint32_t vbase = kbase + S::kTileBytes;
                const int eb = e0 + tile * kTileKeys + kh * 32;   // first key of this warp's half tile
                if (eb >= e1) continue;                            // warp-uniform

                // ---- S = Q K^T over 32 keys ------------------------------------------------------
                float s[4][4];
                #pragma unroll
                for (int i = 0; i < 4; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
                const int mid = lane >> 3;
                #pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    #pragma unroll
                    for (int kp = 0; kp < 2; ++kp) {
                        uint32_t bf[4];
                        const int key = kh * 32 + kp * 16 + (mid >> 1) * 8 + (lane & 7);
                        ldmatrix_x4(bf, kbase + key * S::kPitch + ks * 32 + (mid & 1) * 16);
                        mma_bf16(s[2 * kp], qf[ks], bf[0], bf[1]);
                        mma_bf16(s[2 * kp + 1], qf[ks], bf[2], bf[3]);
                    }
                }
                // ---- scale + mask -----------------------------------------------------------------
                const bool need_mask = (eb + 32 > L) || (eb + 32 > e1);
                #pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    #pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        float v = s[nt][x] * a.scale_log2;
                        if (need_mask) {
                            const int e = eb + nt * 8 + 2 * q + (x & 1);
                            const int rr = x >> 1;
                            bool vis;
                            if (e >= e1) vis = false;
                            else if (e < L) vis = true;
                            else if (e < L + T) vis = (anc[rr] >> (e - L)) & 1ull;
                            else vis = (e >= s_lo[rr]) && (e < s_hi[rr]);
                            if (!vis) v = -INFINITY;
                        }
                        s[nt][x] = v;
                    }
                }
                // ---- online softmax ---------------------------------------------------------------
                uint32_t pa[2][4];
                #pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    float mx = -INFINITY;
                    #pragma unroll
                    for (int nt = 0; nt < 4; ++nt) mx = fmaxf(mx, fmaxf(s[nt][2 * rr], s[nt][2 * rr + 1]));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                    const float m_new = fmaxf(m_run[rr], mx);
                    const float m_use = (m_new == -INFINITY) ? 0.f : m_new;   // all-masked row: every p is 0
                    const float corr = exp2f(m_run[rr] - m_use);
                    float sum = 0.f;
                    #pragma unroll
                    for (int nt = 0; nt < 4; ++nt) {
                        const float p0 = exp2f(s[nt][2 * rr] - m_use), p1 = exp2f(s[nt][2 * rr + 1] - m_use);
                        sum += p0 + p1;
                        s[nt][2 * rr] = p0;
                        s[nt][2 * rr + 1] = p1;
                    }
                    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                    l_run[rr] = l_run[rr] * corr + sum;
                    m_run[rr] = m_new;
                    #pragma unroll
                    for (int i = 0; i < HD / 8; ++i) {
                        o[i][2 * rr] *= corr;
                        o[i][2 * rr + 1] *= corr;
                    }
                }
                #pragma unroll
                for (int kp = 0; kp < 2; ++kp) {
                    pa[kp][0] = pack_bf16(s[2 * kp][0], s[2 * kp][1]);
                    pa[kp][1] = pack_bf16(s[2 * kp][2], s[2 * kp][3]);
                    pa[kp][2] = pack_bf16(s[2 * kp + 1][0], s[2 * kp + 1][1]);
                    pa[kp][3] = pack_bf16(s[2 * kp + 1][2], s[2 * kp + 1][3]);
                }
                // ---- O += P V ---------------------------------------------------------------------
                #pragma unroll
                for (int kp = 0; kp < 2; ++kp) {
                    #pragma unroll
                    for (int dn = 0; dn < HD / 16; ++dn) {
                        uint32_t bf[4];
                        const int key = kh * 32 + kp * 16 + (mid & 1) * 8 + (lane & 7);
                        ldmatrix_x4_trans(bf, vbase + key * S::kPitch + dn * 32 + (mid >> 1) * 16);
                        mma_bf16(o[2 * dn], pa[kp], bf[0], bf[1]);
                        mma_bf16(o[2 * dn + 1], pa[kp], bf[2], bf[3]);
                    }
                }
            }
            cp_async_wait<0>();
            __syncthreads();   // all tiles consumed: the stage buffers may be reused for the merge

            // ---- merge the two key halves (kh = 1 -> kh = 0) through shared memory -------------
            float* mrg = reinterpret_cast<float*>(smem) + rb * 16 * (HD + 2);
            if (kh == 1) {
                #pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    float* dst = mrg + (g + 8 * rr) * (HD + 2);
                    if (q == 0) { dst[HD] = m_run[rr]; dst[HD + 1] = l_run[rr]; }
                    #pragma unroll
                    for (int i = 0; i < HD / 8; ++i) {
                        dst[i * 8 + 2 * q] = o[i][2 * rr];
                        dst[i * 8 + 2 * q + 1] = o[i][2 * rr + 1];
                    }
                }
            }
            __syncthreads();
            if (kh == 0 && warp_active) {
                #pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    const float* src = mrg + (g + 8 * rr) * (HD + 2);
                    const float m2 = src[HD], l2 = src[HD + 1];
                    const float m_new = fmaxf(m_run[rr], m2);
                    const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                    const float c1 = exp2f(m_run[rr] - m_use), c2 = exp2f(m2 - m_use);
                    l_run[rr] = l_run[rr] * c1 + l2 * c2;
                    m_run[rr] = m_new;
                    #pragma unroll
                    for (int i = 0; i < HD / 8; ++i) {
                        o[i][2 * rr] = o[i][2 * rr] * c1 + src[i * 8 + 2 * q] * c2;
                        o[i][2 * rr + 1] = o[i][2 * rr + 1] * c1 + src[i * 8 + 2 * q + 1] * c2;
                    }
                }
                // ---- write: final rows when the pair is not split, else the partial -----------
                #pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    const int row = row_id[rr];
                    if (row >= M) continue;
                    if (n_splits == 1) {
                        const int t = row / rows_per_node, j = row - t * rows_per_node;
                        const float inv = 1.f / l_run[rr];
                        __nv_bfloat16* dst;
                        float* lse = nullptr;
                        if (j == 0) {
                            const long long idx = (static_cast<long long>(b) * a.max_nodes + t) * H + h;
                            dst = a.o_main + idx * HD;
                            if (a.lse_main) lse = a.lse_main + idx;
                        } else {
                            const long long idx = (spec_row0 + static_cast<long long>(t) * gamma + (j - 1)) * H + h;
                            dst = a.o_spec + idx * HD;
                            if (a.lse_spec) lse = a.lse_spec + idx;
                        }
                        #pragma unroll
                        for (int i = 0; i < HD / 8; ++i)
                            *reinterpret_cast<uint32_t*>(dst + i * 8 + 2 * q) =
                                pack_bf16(o[i][2 * rr] * inv, o[i][2 * rr + 1] * inv);
                        if (lse && q == 0) *lse = (m_run[rr] + log2f(l_run[rr])) * 0.6931471805599453f;
                    } else {
                        float* dst = part + static_cast<size_t>(row) * (HD + 2);
                        if (q == 0) { dst[HD] = m_run[rr]; dst[HD + 1] = l_run[rr]; }
                        #pragma unroll
                        for (int i = 0; i < HD / 8; ++i)
                            *reinterpret_cast<float2*>(dst + i * 8 + 2 * q) = make_float2(o[i][2 * rr], o[i][2 * rr + 1]);
                    }
                }
            }
        }   // row chunks

        // ---- split pair: arrive; the last CTA merges every partial of the pair ------------------
        if (n_splits > 1) {
            __syncthreads();
            if (tid == 0) {
                __threadfence();
                const int prev = atomicAdd(&a.counters[b * H + h], 1);
                s_flag = (prev == n_splits - 1);
                if (s_flag) a.counters[b * H + h] = 0;   // ready for the next call
            }
            __syncthreads();
            if (s_flag) {
                __threadfence();
                for (int i = tid; i < M * (HD / 4); i += kThreads) {
                    const int row = i / (HD / 4), c4 = i - row * (HD / 4);
                    float mx = -INFINITY;
                    for (int c = c_first; c <= c_last; ++c) {
                        const float* ps = a.partials + (static_cast<size_t>(2 * c + (c == c_first ? 1 : 0)) * a.m_pad + row) * (HD + 2);
                        mx = fmaxf(mx, __ldcg(ps + HD));
                    }
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    float l = 0.f;
                    for (int c = c_first; c <= c_last; ++c) {
                        const float* ps = a.partials + (static_cast<size_t>(2 * c + (c == c_first ? 1 : 0)) * a.m_pad + row) * (HD + 2);
                        const float w = exp2f(__ldcg(ps + HD) - mx);
                        l += w * __ldcg(ps + HD + 1);
                        const float2 lo = __ldcg(reinterpret_cast<const float2*>(ps + c4 * 4));
                        const float2 hi = __ldcg(reinterpret_cast<const float2*>(ps + c4 * 4 + 2));
                        acc.x += w * lo.x; acc.y += w * lo.y; acc.z += w * hi.x; acc.w += w * hi.y;
                    }
                    const float inv = 1.f / l;
                    const int t = row / rows_per_node, j = row - t * rows_per_node;
                    __nv_bfloat16* dst;
                    float* lse = nullptr;
                    if (j == 0) {
                        const long long idx = (static_cast<long long>(b) * a.max_nodes + t) * H + h;
                        dst = a.o_main + idx * HD;
                        if (a.lse_main) lse = a.lse_main + idx;
                    } else {
                        const long long idx = (spec_row0 + static_cast<long long>(t) * gamma + (j - 1)) * H + h;
                        dst = a.o_spec + idx * HD;
                        if (a.lse_spec) lse = a.lse_spec + idx;
                    }
                    uint2 packed;
                    packed.x = pack_bf16(acc.x * inv, acc.y * inv);
                    packed.y = pack_bf16(acc.z * inv, acc.w * inv);
                    *reinterpret_cast<uint2*>(dst + c4 * 4) = packed;
                    if (lse && c4 == 0) *lse = (mx + log2f(l)) * 0.6931471805599453f;
                }
            }
        }
    }   // segments
}

// ---------------------------------------------------------------------------------------------
struct AttnPlan {
    int grid;
    int m_pad;
    size_t counter_bytes, partial_bytes;
};

static bool make_plan(const ss_attn_params& p, AttnPlan* plan) {
    if (p.batch < 1 || p.n_heads < 1 || p.max_nodes < 1 || p.gamma < 0) return false;
    plan->grid = sm_count();
    plan->m_pad = (p.max_nodes * (1 + p.gamma) + 15) / 16 * 16;
    plan->counter_bytes = (static_cast<size_t>(p.batch) * p.n_heads * sizeof(int32_t) + 255) / 256 * 256;
    plan->partial_bytes = static_cast<size_t>(2) * plan->grid * plan->m_pad * (p.head_dim + 2) * sizeof(float);
    return true;
}

template <int HD>
static int32_t launch(const AttnArgs& args, int grid, cudaStream_t stream) {
    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SS_ERR_CUDA;
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(msa_attention_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 Smem<HD>::kTotal) != cudaSuccess)
            return SS_ERR_CUDA;
        configured[dev] = true;
    }
    msa_attention_kernel<HD><<<grid, kThreads, Smem<HD>::kTotal, stream>>>(args);
    return cudaGetLastError() == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}

}  // namespace ss

extern "C" size_t ss_msa_attention_workspace_bytes(const ss_attn_params* p) {
    ss::AttnPlan plan;
    if (p == nullptr || !ss::make_plan(*p, &plan)) return 0;
    return ss::kWsHeaderBytes + plan.counter_bytes + plan.partial_bytes;
}

extern "C" int32_t ss_msa_attention(const ss_attn_params* p, void* stream) {
    if (p == nullptr) return SS_ERR_INVALID_ARG;
    ss::AttnPlan plan;
    if (!ss::make_plan(*p, &plan)) return SS_ERR_INVALID_ARG;
    if (p->head_dim != 64 && p->head_dim != 80 && p->head_dim != 128) return SS_ERR_UNSUPPORTED;
    if (p->max_nodes > SS_MAX_NODES || p->gamma > SS_MAX_GAMMA) return SS_ERR_UNSUPPORTED;
    if (!p->q_main || !p->o_main || !p->k_cache || !p->v_cache || !p->kv_start || !p->kv_len || !p->trees ||
        !p->workspace)
        return SS_ERR_INVALID_ARG;
    if (p->gamma > 0 && (!p->q_spec || !p->k_spec || !p->v_spec || !p->o_spec)) return SS_ERR_INVALID_ARG;
    if (p->kv_slot_stride < p->head_dim || p->kv_head_stride < 0 || p->kv_total_slots < 1) return SS_ERR_INVALID_ARG;
    if ((p->kv_slot_stride & 7) || (p->kv_head_stride & 7)) return SS_ERR_INVALID_ARG;
    const void* ptrs[] = {p->q_main, p->o_main, p->k_cache, p->v_cache, p->workspace,
                          p->gamma ? p->q_spec : nullptr, p->gamma ? p->k_spec : nullptr,
                          p->gamma ? p->v_spec : nullptr, p->gamma ? p->o_spec : nullptr};
    for (const void* q : ptrs)
        if (!ss::aligned16(q)) return SS_ERR_INVALID_ARG;
    if (!(p->sm_scale == p->sm_scale)) return SS_ERR_INVALID_ARG;
    if (p->workspace_bytes < ss_msa_attention_workspace_bytes(p)) return SS_ERR_WORKSPACE;

    ss::AttnArgs a;
    a.batch = p->batch; a.n_heads = p->n_heads; a.gamma = p->gamma; a.max_nodes = p->max_nodes;
    a.scale_log2 = p->sm_scale * 1.4426950408889634f;
    a.q_main = static_cast<const __nv_bfloat16*>(p->q_main);
    a.o_main = static_cast<__nv_bfloat16*>(p->o_main);
    a.q_spec = static_cast<const __nv_bfloat16*>(p->q_spec);
    a.k_spec = static_cast<const __nv_bfloat16*>(p->k_spec);
    a.v_spec = static_cast<const __nv_bfloat16*>(p->v_spec);
    a.o_spec = static_cast<__nv_bfloat16*>(p->o_spec);
    a.k_cache = static_cast<const __nv_bfloat16*>(p->k_cache);
    a.v_cache = static_cast<const __nv_bfloat16*>(p->v_cache);
    a.slot_stride = p->kv_slot_stride; a.head_stride = p->kv_head_stride;
    a.kv_start = reinterpret_cast<const long long*>(p->kv_start);
    a.kv_len = p->kv_len; a.kv_capacity = p->kv_capacity; a.trees = p->trees;
    a.lse_main = p->lse_main; a.lse_spec = p->lse_spec;
    char* ws = static_cast<char*>(p->workspace);
    a.status = reinterpret_cast<int*>(ws);
    a.counters = reinterpret_cast<int*>(ws + ss::kWsHeaderBytes);
    a.partials = reinterpret_cast<float*>(ws + ss::kWsHeaderBytes + plan.counter_bytes);
    a.m_pad = plan.m_pad;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (p->head_dim) {
        case 64: return ss::launch<64>(a, plan.grid, s);
        case 80: return ss::launch<80>(a, plan.grid, s);
        default: return ss::launch<128>(a, plan.grid, s);
    }
}
