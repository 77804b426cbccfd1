// Tree-masked multi-stream attention for heads of at most 64 query rows (Eq. 1, Eq. 2): the keys lie on
// the TMEM lanes and the query rows on the columns.  Included by ss_attention.cu after its helpers.
//
//   S^T = K Q^T     A = a K tile (128 keys x d, K-major), B = the head's query tile (64 rows x d, K-major)
//   O^T += V^T P^T  A = the V tile (d x 128 keys, read MN-major from the [key][d] tile), B = P (128 keys x 64
//                   rows, MN-major: one 128-byte row of bf16 per key, written by the key's softmax thread)
//
// Nothing is duplicated and nothing is padded on the row side: the 64 rows are the N of both MMAs, a CTA
// has one accumulator (64 TMEM columns) and two score buffers (64 columns each), and its shared memory is
// the query tile plus a short ring of K/V tiles, so two CTAs -- of two consecutive layers -- fit on an SM:
// while one layer computes and merges, the CTAs of the next one are already resident, have requested
// their first tiles and have asked the L2 for the rest of their prefix.
//
// Softmax without a row reduction.  A thread owns one key and 32 of the 64 rows (two warpgroups share
// the columns).  Row r is exponentiated against a reference m_ref[r] held in shared memory; any reference
// at or above the row's scores (and not absurdly far above) gives the same result after normalisation.
// The reference is the row's maximum over the CTA's first tile; a later score that exceeds it by more
// than 2^8 raises it: all softmax threads agree on that through one reducing barrier per tile, the column
// maxima come from warp reductions, the accumulator and the row sums are rescaled, and the tile's P is
// recomputed.  The row sums are taken over the bf16 P that the MMA reads, by a separate warp.
//
// Roles (384 threads): warp 0 lane 0 requests tiles (TMA) into the ring, K and V tiles alternating;
// warp 1 lane 0 issues S^T; warp 2 lane 0 issues O^T and hands ring slots back; warp 3 sums P's columns;
// warps 4..11 are the softmax threads.  P of tile j is written into the first 16 KB of the ring slot that
// held K tile j (the MMA that read K is complete by then), so P needs no shared memory of its own.
#pragma once

namespace ss {

// developer trace of this kernel: worker CTAs are numbered after the prefetch CTAs
#ifdef SS_TRACE
#define SS_TRC(role, slot)                                                                                       \
    do {                                                                                                         \
        const int tr_cta_ = static_cast<int>(blockIdx.x) - a.n_prefetch;                                         \
        if (tr_cta_ >= 0 && tr_cta_ < ss::kTraceCtas && (slot) < ss::kTraceSlots) ss::g_trace[tr_cta_][role][slot] = clock64(); \
    } while (0)
#else
#define SS_TRC(role, slot) do { } while (0)
#endif

constexpr int kColsRows = 64;                     // query rows (columns of S^T and O^T) of the variant
constexpr int kColsThreads = 384;
constexpr int kColsMaxSlots = 6;
constexpr int kColsSmemLimit = 232448 - 1024;     // one CTA per SM: 227 KB less the control block

template <int HD>
struct GeoC {
    static constexpr int kHalves = HD > 64 ? 2 : 1;               // 64-element boxes along head_dim
    static constexpr int kBoxBytes = kTileKeys * 128;             // one TMA box: 128 keys x 128 B
    static constexpr int kSlotBytes = kHalves * kBoxBytes;        // a K tile or a V tile
    static constexpr int kQHalfBytes = kColsRows * 128;
    static constexpr int kQBytes = kHalves * kQHalfBytes;
    static constexpr int kKSteps = HD / 16;
    // the V tile feeds an M = 128 MMA: with one 64-element box the upper 64 lanes read whatever follows the
    // slot (their results are never looked at), so the ring is followed by one box of padding
    static constexpr int kPadBytes = kHalves == 1 ? kBoxBytes : 0;
    static constexpr uint32_t kTmemCols = 256;                    // S^T (2 x 64), O^T (64); two CTAs share an SM's 512
    static constexpr int kMergePitch = HD + 4;
};

struct CtrlC {
    unsigned long long q_full;
    // A slot's K fills and V fills complete on barriers of their own: each is awaited by one thread, which then
    // sees every phase of its barrier (K and V tiles alternate in a slot when the ring has an odd number of
    // slots, and a parity wait that is two phases behind would pass at once).
    unsigned long long slot_full[2][kColsMaxSlots], slot_empty[kColsMaxSlots];
    unsigned long long s_full[2], s_free[2];   // S^T buffer written / read by the eight softmax warps
    unsigned long long p_full[2];              // P of tile j written (eight warps), by tile parity
    unsigned long long o_done[2];              // O^T += V^T P^T of tile j complete, by tile parity
    alignas(16) float m_ref[kColsRows];        // per query row: the reference its exponentials are taken against
    unsigned long long anc[SS_MAX_NODES];
    uint32_t tmem_base;
    int abort;
    int merge_ok;
    int raised[4];                             // tile j raised a reference: [j & 3], read by the column-sum warp
    int wait_limit;                            // bound of every wait, in units of 1024 cycles
};
static_assert(sizeof(CtrlC) <= 1024, "control block and dynamic shared memory must fit two CTAs per SM");

__device__ __forceinline__ uint32_t bar_red_or(int id, int threads, bool pred) {
    uint32_t out;
    asm volatile("{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, %2, %3, q;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(out) : "r"(pred ? 1u : 0u), "r"(id), "r"(threads) : "memory");
    return out;
}
__device__ __forceinline__ float warp_max_f32(float v) {
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ void tma_prefetch_l2_3d(const CUtensorMap* map, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(map), "r"(c0), "r"(c1), "r"(c2)
                 : "memory");
}
// waits whose limit comes from the control block (the caller may shorten it through the workspace header)
__device__ __noinline__ bool mbar_wait_slow_c(uint32_t bar, uint32_t parity, CtrlC* c, int* status) {
    const long long t0 = clock64();
    volatile int* abort = &c->abort;
    const long long limit = static_cast<long long>(*reinterpret_cast<volatile int*>(&c->wait_limit)) << 10;
    for (;;) {
        for (int i = 0; i < 256; ++i) {
            if (mbar_try(bar, parity)) return true;
            if (*abort) return false;
        }
        if (clock64() - t0 > limit) {
            *abort = 1;
            set_status(status, SS_ERR_DEVICE_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait_c(uint32_t bar, uint32_t parity, CtrlC* c, int* status) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow_c(bar, parity, c, status);
}
__device__ __forceinline__ bool mbar_wait_warp_c(uint32_t bar, uint32_t parity, CtrlC* c, int* status) {
    return __all_sync(0xffffffffu, mbar_wait_c(bar, parity, c, status));
}

template <int HD>
__global__ void __launch_bounds__(kColsThreads, 1) msa_attention_cols_kernel(const __grid_constant__ AttnArgs a) {
    using G = GeoC<HD>;
    constexpr int TK = kTileKeys;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(16) CtrlC c;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int C = a.cluster;
    // The first n_prefetch CTAs of the grid compute nothing: they are dispatched first, to the SMs that the
    // worker CTAs of the previous launch leave free, while that launch is still at work, and ask the L2 for
    // every K/V tile and query tile of this call.  A prefetch has no architectural effect, so it needs no
    // ordering against the kernels before it; the lengths it reads are covered by the caller's promise.
    if (static_cast<int>(blockIdx.x) < a.n_prefetch) {
        const int me = static_cast<int>(blockIdx.x) * kColsThreads + tid, n_me = a.n_prefetch * kColsThreads;
        constexpr int kRowBytes = HD * 2, kLines = (kRowBytes + 127) / 128;
        auto touch = [](const char* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p) : "memory"); };
        for (int b = 0; b < a.batch; ++b) {
            int L, T;
            long long slot0;
            asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(L) : "l"(a.kv_len + b) : "memory");
            asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(T) : "l"(&a.trees[b].n_nodes) : "memory");
            asm volatile("ld.global.cg.s64 %0, [%1];" : "=l"(slot0) : "l"(a.kv_start + b) : "memory");
            T = min(max(T, 0), a.max_nodes);
            if (L < 0) continue;
            const int rows = L + T;
            // cached rows: (kind, head, slot); one thread per row, a line at a time
            for (long long w = me; w < 2ll * a.n_heads * rows; w += n_me) {
                const int kind = static_cast<int>(w / (static_cast<long long>(a.n_heads) * rows));
                const long long rem = w - static_cast<long long>(kind) * a.n_heads * rows;
                const int r = static_cast<int>(rem / a.n_heads), h = static_cast<int>(rem - static_cast<long long>(r) * a.n_heads);
                const char* p = (kind ? a.v_ptr : a.k_ptr) + ((slot0 + r) * a.kv_slot_stride + static_cast<long long>(h) * a.kv_head_stride) * 2;
                #pragma unroll
                for (int i = 0; i < kLines; ++i) touch(p + i * 128);
            }
            // the contiguous per-step tensors of the sequence: queries, stream queries / keys / values
            const long long qm_bytes = static_cast<long long>(T) * a.n_heads * kRowBytes;
            const char* qm = a.q_ptr + static_cast<long long>(b) * a.max_nodes * a.n_heads * kRowBytes;
            for (long long o = static_cast<long long>(me) * 128; o < qm_bytes; o += static_cast<long long>(n_me) * 128) touch(qm + o);
            if (a.gamma > 0) {
                const long long sp_bytes = qm_bytes * a.gamma, sp_off = static_cast<long long>(b) * a.max_nodes * a.gamma * a.n_heads * kRowBytes;
                for (long long o = static_cast<long long>(me) * 128; o < sp_bytes; o += static_cast<long long>(n_me) * 128) {
                    touch(a.qs_ptr + sp_off + o); touch(a.ks_ptr + sp_off + o); touch(a.vs_ptr + sp_off + o);
                }
            }
        }
        return;
    }
    const int blk = static_cast<int>(blockIdx.x) - a.n_prefetch;
    const uint32_t rank = blk & (C - 1);
    const int group = blk >> a.cluster_shift;              // (sequence, head)
    int b = group / a.n_heads;
    const int h = group - b * a.n_heads;
    const int n_slots = a.n_kslots;
    if (tid == 0) SS_TRC(0, 0);
#ifdef SS_TRACE
    __shared__ unsigned int s_launch;
    if (tid == 0) {
        const unsigned long long key = reinterpret_cast<unsigned long long>(a.o_main);
        s_launch = 0;
        for (unsigned int i = 0; i < 8; ++i) {
            const unsigned long long old = atomicCAS(&g_key[i], 0ull, key);
            if (old == 0ull || old == key) { s_launch = i; break; }
        }
        atomicMin(&g_wall[s_launch & 7][0], wall_ns());
        atomicMax(&g_wall[s_launch & 7][2], wall_ns());
        if (blk < kTraceCtas) g_trace[blk][0][150] = static_cast<long long>(wall_ns());
    }
#endif

    const uint32_t base = smem_u32(smem_raw);              // 1024-byte aligned (checked below): swizzle atoms
    const uint32_t q_base = base;                          // [half][64 rows][128 B]
    const uint32_t ring_base = q_base + G::kQBytes;        // [slot][half][128 keys][128 B]
    // scratch of a raise at tile j: the upper box of K tile j's slot, free once S^T of the tile is complete
    // (one-box slots: the padding behind the ring)
    auto slot_addr = [&](int s) { return ring_base + static_cast<uint32_t>(s) * G::kSlotBytes; };
    // 2 KB of scratch for tile j whose K tile sits in ring slot s: column maxima per warp (1 KB), then the
    // 64 rescale factors
    auto scratch_addr = [&](int s, int j) {
        return G::kHalves == 2 ? slot_addr(s) + G::kBoxBytes
                               : ring_base + static_cast<uint32_t>(n_slots) * G::kSlotBytes + static_cast<uint32_t>(j & 3) * 2048u;
    };

    // ---- prologue (see msa_attention_kernel: the same launch protocol) ------------------------------
    int L = 0, T = 0, cap = 0x7fffffff;
    long long slot0 = 0;
    const bool by_length = a.batch > 1 && a.batch <= 32 && C == 1;
    auto load_scalars = [&]() {
        if (by_length) {
            int len = -1;
            if (lane < a.batch) asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(len) : "l"(a.kv_len + lane) : "memory");
            int longer = 0;
            for (int o = 0; o < a.batch; ++o) {
                const int other = __shfl_sync(0xffffffffu, len, o);
                longer += (other > len || (other == len && o < lane)) ? 1 : 0;
            }
            b = __ffs(__ballot_sync(0xffffffffu, lane < a.batch && longer == b)) - 1;
        }
        asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(L) : "l"(a.kv_len + b) : "memory");
        asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(T) : "l"(&a.trees[b].n_nodes) : "memory");
        asm volatile("ld.global.cg.s64 %0, [%1];" : "=l"(slot0) : "l"(a.kv_start + b) : "memory");
        if (a.kv_capacity != nullptr) asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(cap) : "l"(a.kv_capacity + b) : "memory");
    };
    if (a.prefix_stable) load_scalars();
    if (tid == 0) {
        mbar_init(smem_u32(&c.q_full), 1);
        for (int s = 0; s < kColsMaxSlots; ++s) { mbar_init(smem_u32(&c.slot_full[0][s]), 1); mbar_init(smem_u32(&c.slot_full[1][s]), 1); }
        c.abort = 0;
        c.wait_limit = static_cast<int>(kWaitCycles >> 10);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&a.tm_qm); tma_prefetch_desc(&a.tm_k); tma_prefetch_desc(&a.tm_v);
        if (a.gamma > 0) { tma_prefetch_desc(&a.tm_qs); tma_prefetch_desc(&a.tm_ks); tma_prefetch_desc(&a.tm_vs); }
    } else if (tid == 64) {
        // a slot is handed back by two arrivals: the MMA that last read it, and the column-sum warp (K
        // slots, which hold P) or the issuing thread itself (V slots)
        for (int s = 0; s < kColsMaxSlots; ++s) mbar_init(smem_u32(&c.slot_empty[s]), 2);
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&c.s_full[s]), 1);
            mbar_init(smem_u32(&c.s_free[s]), 8);
            mbar_init(smem_u32(&c.p_full[s]), 8);
            mbar_init(smem_u32(&c.o_done[s]), 1);
        }
        for (int i = 0; i < 4; ++i) c.raised[i] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    auto dependency_wait = [&]() {
        if (tid == 0) {
            SS_TRC(0, 2);
            asm volatile("griddepcontrol.wait;" ::: "memory");
            SS_TRC(0, 3);
#ifdef SS_TRACE
            atomicMin(&g_wall[s_launch & 7][3], wall_ns());
            atomicMax(&g_wall[s_launch & 7][4], wall_ns());
            if (blk < kTraceCtas) g_trace[blk][0][151] = static_cast<long long>(wall_ns());
#endif
            asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        }
        __syncthreads();
    };
    if (!a.prefix_stable) {
        dependency_wait();
        load_scalars();
    }
    const long long spec_row0 = static_cast<long long>(b) * a.max_nodes * a.gamma;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&c.tmem_base)), "r"(G::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    T = min(max(T, 0), a.max_nodes);
    bool skip = false;
    const bool bad_smem = (base & 1023u) != 0u;           // never expected: nothing is copied to shared memory then
    if (L < 0 || L + T > cap || bad_smem) {
        skip = true;
        L = 0; T = 0;
    }
    const Span sp = make_span(a, L, T, static_cast<int>(rank), 0, kTileKeys);

    // ring entry i: K tile i/2 (even) or V tile i/2 (odd)
    auto load_entry = [&](int i, int st) {
        const int j = i >> 1;
        const bool is_v = (i & 1) != 0;
        const uint32_t bar = smem_u32(&c.slot_full[i & 1][st]);
        mbar_expect_tx(bar, G::kSlotBytes);
        const uint32_t dst = slot_addr(st);
        const int x = sp.first_key(j);
        #pragma unroll
        for (int hh = 0; hh < G::kHalves; ++hh) {
            if (sp.is_cache(j)) tma_load_3d(dst + hh * G::kBoxBytes, is_v ? &a.tm_v : &a.tm_k, hh * 64, h * a.head_coord, static_cast<int>(slot0 + x), bar);
            else tma_load_3d(dst + hh * G::kBoxBytes, is_v ? &a.tm_vs : &a.tm_ks, hh * 64, h, static_cast<int>(spec_row0 + x), bar);
        }
    };
    const int n_entries = 2 * sp.n_tiles;
    const int n_early = min(n_entries, n_slots);
    auto prefix_only = [&](int j) { return sp.is_cache(j) && sp.first_key(j) + TK <= sp.L; };
    int n_pre = 0;
    if (a.prefix_stable) {
        if (tid == 0) {
            // the first tiles that lie wholly inside the cached prefix
            while (n_pre < n_early && prefix_only(n_pre >> 1)) { load_entry(n_pre, n_pre); ++n_pre; }
        }
        dependency_wait();
    }
    if (tid == 0) {
        if (skip) set_status(a.status, bad_smem ? SS_ERR_CUDA : SS_ERR_CAPACITY);
        // the caller may shorten the bound of the device-side waits (workspace word 1, units of 1024 cycles)
        int lim;
        asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(lim) : "l"(a.status + 1) : "memory");
        if (lim > 0) c.wait_limit = lim;
        for (int i = n_pre; i < n_early; ++i) load_entry(i, i);
        const uint32_t qbar = smem_u32(&c.q_full);
        const bool with_spec = a.gamma > 0 && a.s0rows > 0;
        const uint32_t rows = a.tmax8 + (with_spec ? a.s0rows : 0);
        mbar_expect_tx(qbar, bad_smem ? 0u : G::kHalves * rows * 128u);
        #pragma unroll
        for (int hh = 0; hh < G::kHalves; ++hh) {
            if (bad_smem) break;
            const uint32_t dst = q_base + hh * G::kQHalfBytes;
            tma_load_3d(dst, &a.tm_qm, hh * 64, h, b * a.max_nodes, qbar);
            if (with_spec) tma_load_3d(dst + a.tmax8 * 128u, &a.tm_qs, hh * 64, h, static_cast<int>(spec_row0), qbar);
        }
        SS_TRC(0, 5);
    }
    if (tid >= kAuxThreads && tid < kAuxThreads + SS_MAX_NODES) c.anc[tid - kAuxThreads] = __ldcg(&a.trees[b].anc_mask[tid - kAuxThreads]);
    if (tid >= kAuxThreads + 64 && tid < kAuxThreads + 128) c.m_ref[tid - kAuxThreads - 64] = -INFINITY;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (tid == 0) SS_TRC(0, 6);
    const uint32_t tmem = c.tmem_base;
    const uint32_t tmem_o = tmem;                          // 64 columns
    const uint32_t tmem_s = tmem + 64;                     // two buffers of 64 columns
    int* const status = a.status;
    // fill number of a slot's barrier of one kind: with an odd number of slots the kinds alternate in a slot
    const bool odd_ring = (n_slots & 1) != 0;
    auto fill_parity = [&](const Ring& r) { return static_cast<uint32_t>((odd_ring ? r.round >> 1 : r.round) & 1); };
    auto wait_slot_full = [&](int kind, const Ring& r) {
        return mbar_wait_c(smem_u32(&c.slot_full[kind][r.slot]), fill_parity(r), &c, status);
    };

    // =============================== warp 0: tile requests =======================================
    if (warp == 0) {
        if (lane == 0 && n_entries > n_early) {
            Ring r;
            r.start();
            for (int i = 0; i < n_early; ++i) r.advance(n_slots);
            bool ok = true;
            for (int i = n_early; ok && i < n_entries; ++i) {
                ok = mbar_wait_c(smem_u32(&c.slot_empty[r.slot]), (r.round - 1) & 1, &c, status);
                SS_TRC(0, 8 + i);
                if (ok) { load_entry(i, r.slot); r.advance(n_slots); }
            }
            if (!ok) {                 // gave up: let the copies already in flight land before the CTA leaves
                Ring d;
                d.start();
                for (int i = 0; i < n_entries; ++i, d.advance(n_slots))
                    if (d.slot + d.round * n_slots >= r.slot + r.round * n_slots - n_slots && d.slot + d.round * n_slots < r.slot + r.round * n_slots)
                        mbar_drain(smem_u32(&c.slot_full[i & 1][d.slot]), fill_parity(d));
            }
        }
    }
    // =============================== warp 1: S^T = K Q^T ==========================================
    else if (warp == 1) {
        if (lane == 0) {
            bool ok = mbar_wait_c(smem_u32(&c.q_full), 0, &c, status);
            if (!ok) mbar_drain(smem_u32(&c.q_full), 0);
            SS_TRC(1, 0);
            Ring r;
            r.start();
            const uint64_t dq = desc_k_major(q_base);
            for (int j = 0; ok && j < sp.n_tiles; ++j) {
                const int buf = j & 1;
                if (!wait_slot_full(0, r)) break;
                SS_TRC(1, 8 + 4 * j);
                if (j >= 2 && !mbar_wait_c(smem_u32(&c.s_free[buf]), ((j >> 1) - 1) & 1, &c, status)) break;
                SS_TRC(1, 9 + 4 * j);
                tc_fence_after();
                const uint64_t dk = desc_k_major(slot_addr(r.slot));
                #pragma unroll
                for (int ks = 0; ks < G::kKSteps; ++ks) {
                    const uint32_t hh = ks >> 2, off = (ks & 3) * 32u;
                    tc_mma(tmem_s + buf * kColsRows, dk + ((hh * G::kBoxBytes + off) >> 4), dq + ((hh * G::kQHalfBytes + off) >> 4),
                           idesc_bf16(kColsRows, false, false), ks > 0);
                }
                tc_commit(smem_u32(&c.s_full[buf]));
                SS_TRC(1, 10 + 4 * j);
                r.advance(n_slots); r.advance(n_slots);
            }
        }
    }
    // =============================== warp 2: O^T += V^T P^T =======================================
    else if (warp == 2) {
        if (lane == 0) {
            Ring rk, rv;
            rk.start(); rv.start();
            rv.advance(n_slots);
            for (int j = 0; j < sp.n_tiles; ++j) {
                if (!wait_slot_full(1, rv)) break;
                SS_TRC(2, 8 + 4 * j);
                if (!mbar_wait_c(smem_u32(&c.p_full[j & 1]), (j >> 1) & 1, &c, status)) break;
                SS_TRC(2, 9 + 4 * j);
                tc_fence_after();
                const uint64_t dv = desc_mn_major(slot_addr(rv.slot), G::kBoxBytes);
                const uint64_t dp = desc_mn_major(slot_addr(rk.slot), G::kBoxBytes);
                #pragma unroll
                for (int ks = 0; ks < TK / 16; ++ks)
                    tc_mma(tmem_o, dv + ((ks * 2048u) >> 4), dp + ((ks * 2048u) >> 4), idesc_bf16(kColsRows, true, true),
                           (j > 0 || ks > 0) ? 1u : 0u);
                tc_commit(smem_u32(&c.o_done[j & 1]));
                tc_commit(smem_u32(&c.slot_empty[rk.slot]));
                tc_commit(smem_u32(&c.slot_empty[rv.slot]));
                mbar_arrive(smem_u32(&c.slot_empty[rv.slot]));
                SS_TRC(2, 10 + 4 * j);
                rk.advance(n_slots); rk.advance(n_slots);
                rv.advance(n_slots); rv.advance(n_slots);
            }
        }
    }
    // =============================== warp 3: column sums of P =====================================
    // lane = (key parity, four columns): l of row r is the sum over keys of the bf16 P the MMA reads
    float lsum[4] = {0.f, 0.f, 0.f, 0.f};
    if (warp == 3) {
        Ring rk;
        rk.start();
        const int q = lane & 15, kp = lane >> 4;
        for (int j = 0; j < sp.n_tiles; ++j) {
            if (!mbar_wait_warp_c(smem_u32(&c.p_full[j & 1]), (j >> 1) & 1, &c, status)) break;
            const uint32_t p_base = slot_addr(rk.slot);
            if (lane == 0) SS_TRC(4, 8 + 2 * j);
            if (*reinterpret_cast<volatile int*>(&c.raised[j & 3])) {
                const uint32_t corr = scratch_addr(rk.slot, j) + 1024u;
                const float4 f = ld_shared_v4(corr + q * 16u);
                lsum[0] *= f.x; lsum[1] *= f.y; lsum[2] *= f.z; lsum[3] *= f.w;
            }
            #pragma unroll 8
            for (int r = 0; r < TK / 2; ++r) {
                const int key = 2 * r + kp;
                const uint32_t addr = p_base + key * 128u + ((((q >> 1) ^ (key & 7)) << 4) | ((q & 1) << 3));
                uint32_t w0, w1;
                asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(w0), "=r"(w1) : "r"(addr) : "memory");
                lsum[0] += __uint_as_float(w0 << 16); lsum[1] += __uint_as_float(w0 & 0xffff0000u);
                lsum[2] += __uint_as_float(w1 << 16); lsum[3] += __uint_as_float(w1 & 0xffff0000u);
            }
            __syncwarp();
            if (lane == 0) SS_TRC(4, 9 + 2 * j);
            if (lane == 0) mbar_arrive(smem_u32(&c.slot_empty[rk.slot]));
            rk.advance(n_slots); rk.advance(n_slots);
        }
        #pragma unroll
        for (int i = 0; i < 4; ++i) lsum[i] += __shfl_xor_sync(0xffffffffu, lsum[i], 16);
    }
    // =============================== warps 4..11: softmax =========================================
    const int wg = warp >= 4 ? (warp - 4) >> 2 : 0;                           // column half
    const int kl = ((warp & 3) << 5) | lane;                                  // TMEM lane: key of a tile, later head_dim index
    const int col0 = wg * 32;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    uint32_t valid_cols = 0u;                                                 // my 32 columns that are query rows of the head
    if (warp >= 4) {
        #pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int cc = col0 + i;
            const bool v = cc < sp.T || (cc >= sp.tmax8 && cc - sp.tmax8 < sp.n_stream);
            valid_cols |= v ? (1u << i) : 0u;
        }
        const uint32_t m_ref_addr = smem_u32(&c.m_ref[col0]);
        Ring rk;
        rk.start();
        bool failed = false;
        for (int j = 0; j < sp.n_tiles; ++j) {
            const int buf = j & 1;
            // every phase of the completion barriers is looked at (two tiles late), so a parity wait is never
            // more than one phase behind
            bool have_s = j < 2 || mbar_wait_warp_c(smem_u32(&c.o_done[buf]), ((j - 2) >> 1) & 1, &c, status);
            have_s = mbar_wait_warp_c(smem_u32(&c.s_full[buf]), (j >> 1) & 1, &c, status) && have_s;
            if (tid == kAuxThreads) SS_TRC(3, 8 + 6 * j);
            tc_fence_after();
            const uint32_t s_addr = tmem_s + lane_base + buf * kColsRows + col0;
            const uint32_t k_slot = slot_addr(rk.slot);
            const uint32_t p_row = k_slot + kl * 128u;
            const uint32_t scratch = scratch_addr(rk.slot, j);
            const int x0 = sp.first_key(j), nvk = sp.valid_keys(j);
            const bool cache = sp.is_cache(j);
            const bool masked = !cache || x0 + TK > sp.L || nvk < TK;
            // the rows (my 32 columns) that see this thread's key (Eq. 1 / Eq. 2 with the tree mask of App. A)
            uint32_t vis = valid_cols;
            if (masked) {
                const int x = x0 + kl;
                if (kl >= nvk) {
                    vis = 0u;
                } else if (cache) {
                    if (x >= sp.L) {                                          // tree node x - L: its descendants and itself
                        const int node_a = x - sp.L;
                        uint32_t m = 0u;
                        #pragma unroll 4
                        for (int i = 0; i < 32; ++i) {
                            const int cc = col0 + i;
                            const int node = cc < sp.tmax8 ? cc : ((cc - sp.tmax8) * a.gamma_magic) >> 16;
                            m |= static_cast<uint32_t>((c.anc[node & (SS_MAX_NODES - 1)] >> node_a) & 1ull) << i;
                        }
                        vis = m & valid_cols;
                    }
                } else {                                                      // stream key x = (node, i): streams i.. of its node
                    const int node = (x * a.gamma_magic) >> 16;
                    const int lo = sp.tmax8 + x - col0, hi = sp.tmax8 + (node + 1) * sp.gamma - col0;   // columns [lo, hi)
                    const uint32_t below_hi = hi >= 32 ? ~0u : (hi <= 0 ? 0u : ((1u << hi) - 1u));
                    const uint32_t below_lo = lo >= 32 ? ~0u : (lo <= 0 ? 0u : ((1u << lo) - 1u));
                    vis = below_hi & ~below_lo & valid_cols;
                }
            }
            if (tid == kAuxThreads) c.raised[j & 3] = 0;

            // Raises the references to the column maxima of this tile, rescales what was accumulated so far.
            auto raise = [&]() {
                float mine = -INFINITY;
                #pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    uint32_t sr[16];
                    tmem_ld16<0>(s_addr + ch * 16, sr);
                    tmem_wait_ld();
                    #pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        float v = __uint_as_float(sr[i]) * a.scale_log2;
                        v = ((vis >> (ch * 16 + i)) & 1u) ? v : -INFINITY;
                        const float r = warp_max_f32(v);
                        if (lane == ch * 16 + i) mine = r;
                    }
                }
                asm volatile("st.shared.f32 [%0], %1;" ::"r"(scratch + static_cast<uint32_t>((warp - 4) * 32 + lane) * 4u), "f"(mine) : "memory");
                named_barrier(5, 256);
                const int ts = tid - kAuxThreads;
                if (ts < kColsRows) {
                    const uint32_t src = scratch + static_cast<uint32_t>((ts >> 5) * 128 + (ts & 31)) * 4u;
                    float mx = -INFINITY;
                    #pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        float v;
                        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(src + w * 128u) : "memory");
                        mx = fmaxf(mx, v);
                    }
                    const bool colv = ts < sp.T || (ts >= sp.tmax8 && ts - sp.tmax8 < sp.n_stream);
                    const float m_old = c.m_ref[ts];
                    const float m_new = colv ? fmaxf(m_old, mx) : INFINITY;
                    const float corr = m_new == m_old ? 1.f : exp2f(m_old - m_new);      // 0 when nothing was visible so far
                    c.m_ref[ts] = m_new;
                    asm volatile("st.shared.f32 [%0], %1;" ::"r"(scratch + 1024u + ts * 4u), "f"(corr) : "memory");
                    if (ts == 0) c.raised[j & 3] = 1;
                }
                named_barrier(5, 256);
                bool ok = true;
                if (j > 0) {
                    ok = mbar_wait_warp_c(smem_u32(&c.o_done[(j - 1) & 1]), ((j - 1) >> 1) & 1, &c, status);
                    tc_fence_after();
                    if (ok) {
                        #pragma unroll
                        for (int ch = 0; ch < 2; ++ch) {
                            uint32_t orr[16];
                            tmem_ld16<0>(tmem_o + lane_base + col0 + ch * 16, orr);
                            tmem_wait_ld();
                            #pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4) {
                                const float4 f = ld_shared_v4(scratch + 1024u + static_cast<uint32_t>(col0 + ch * 16 + q4 * 4) * 4u);
                                orr[q4 * 4 + 0] = __float_as_uint(__uint_as_float(orr[q4 * 4 + 0]) * f.x);
                                orr[q4 * 4 + 1] = __float_as_uint(__uint_as_float(orr[q4 * 4 + 1]) * f.y);
                                orr[q4 * 4 + 2] = __float_as_uint(__uint_as_float(orr[q4 * 4 + 2]) * f.z);
                                orr[q4 * 4 + 3] = __float_as_uint(__uint_as_float(orr[q4 * 4 + 3]) * f.w);
                            }
                            tmem_st16<0>(tmem_o + lane_base + col0 + ch * 16, orr);
                        }
                        tmem_wait_st();
                    }
                }
                return ok;
            };

            bool ok = have_s;
            if (j == 0) raise();                                              // every thread, so the barriers inside match
            bool leave = false;
            for (int attempt = 0; attempt < 3; ++attempt) {
                float tmax = -INFINITY;
                if (ok) {
                    #pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        uint32_t sr[16];
                        tmem_ld16<0>(s_addr + ch * 16, sr);
                        float mr[16];
                        #pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const float4 f = ld_shared_v4(m_ref_addr + static_cast<uint32_t>(ch * 16 + q4 * 4) * 4u);
                            mr[q4 * 4 + 0] = f.x; mr[q4 * 4 + 1] = f.y; mr[q4 * 4 + 2] = f.z; mr[q4 * 4 + 3] = f.w;
                        }
                        tmem_wait_ld();
                        uint32_t pk[8];
                        #pragma unroll
                        for (int i = 0; i < 16; i += 2) {
                            float t0 = fmaf(__uint_as_float(sr[i]), a.scale_log2, -mr[i]);
                            float t1 = fmaf(__uint_as_float(sr[i + 1]), a.scale_log2, -mr[i + 1]);
                            float e0 = exp2f(t0), e1 = exp2f(t1);
                            if (masked) {
                                const bool v0 = (vis >> (ch * 16 + i)) & 1u, v1 = (vis >> (ch * 16 + i + 1)) & 1u;
                                t0 = v0 ? t0 : -INFINITY; t1 = v1 ? t1 : -INFINITY;
                                e0 = v0 ? e0 : 0.f; e1 = v1 ? e1 : 0.f;
                            }
                            tmax = fmaxf(tmax, fmaxf(t0, t1));
                            pk[i >> 1] = pack_bf16(e0, e1);
                        }
                        // columns col0 + 16 ch .. + 15 = 16-byte pieces 4 wg + 2 ch, + 1 of the key's row
                        const uint32_t piece = static_cast<uint32_t>(wg * 4 + ch * 2);
                        st_shared_v4(p_row + (((piece) ^ (kl & 7)) << 4), pk[0], pk[1], pk[2], pk[3]);
                        st_shared_v4(p_row + (((piece + 1) ^ (kl & 7)) << 4), pk[4], pk[5], pk[6], pk[7]);
                    }
                }
                if (tid == kAuxThreads) SS_TRC(3, 9 + 6 * j + (attempt > 0 ? 3 : 0));
                // one reducing barrier per tile: did a score outgrow its reference, or did a wait run out
                const uint32_t any = bar_red_or(4, 256, !ok || tmax > kRescaleStep);
                if (tid == kAuxThreads) SS_TRC(3, 10 + 6 * j);
                if (!any) break;
                if (*reinterpret_cast<volatile int*>(&c.abort)) { leave = true; break; }
                ok = raise();
            }
            if (leave) { failed = true; break; }
            // V rows past the end of the sequence's keys may hold anything (even NaN patterns): P is 0 there,
            // but 0 * NaN is NaN, so they are cleared (warpgroup w: box w of the key's row)
            const int region_left = (cache ? sp.L + sp.T : sp.n_stream) - x0;
            if (region_left < TK) {
                Ring rv = rk;
                rv.advance(n_slots);
                if (mbar_wait_warp_c(smem_u32(&c.slot_full[1][rv.slot]), fill_parity(rv), &c, status)) {
                    if (kl >= region_left && wg < G::kHalves) {
                        const uint32_t dst = slot_addr(rv.slot) + wg * G::kBoxBytes + kl * 128u;
                        #pragma unroll
                        for (int i = 0; i < 8; ++i) st_shared_v4(dst + i * 16, 0u, 0u, 0u, 0u);
                    }
                }
            }
            fence_async_smem();
            tc_fence_before();
            __syncwarp();
            // P of the tile is published, then the score buffer handed back (S^T of tile j + 2 may overwrite it):
            // in this order no warp can reach tile j + 2 and arrive on p_full[j & 1] before every warp has
            // arrived there for tile j
            if (lane == 0) {
                mbar_arrive(smem_u32(&c.p_full[j & 1]));
                mbar_arrive(smem_u32(&c.s_free[buf]));
            }
            if (tid == kAuxThreads) SS_TRC(3, 11 + 6 * j);
            rk.advance(n_slots); rk.advance(n_slots);
        }
        if (!failed && sp.n_tiles > 0) {
            const int n = sp.n_tiles;
            if (n > 1) mbar_wait_warp_c(smem_u32(&c.o_done[(n - 2) & 1]), ((n - 2) >> 1) & 1, &c, status);
            mbar_wait_warp_c(smem_u32(&c.o_done[(n - 1) & 1]), ((n - 1) >> 1) & 1, &c, status);
            tc_fence_after();
        }
    }
    __syncwarp();
    if (tid == kAuxThreads) SS_TRC(5, 0);

    // ======================================== epilogue ==========================================
    // Everything in the ring and the query tile is dead now (the last MMA is complete): the row sums go to
    // the start of the query tile.
    const uint32_t l_base = q_base;
    if (warp >= 3) {
        mbar_wait_warp_c(smem_u32(&c.q_full), 0, &c, status);                         // the query copy has landed
        if (warp == 3 && lane < 16)
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(l_base + lane * 16u), "f"(lsum[0]), "f"(lsum[1]), "f"(lsum[2]), "f"(lsum[3]) : "memory");
        named_barrier(6, 288);
    }
    if (tid == kAuxThreads) SS_TRC(5, 1);
    constexpr int RP = G::kMergePitch;
    constexpr int rows_cap = kColsRows;
    constexpr int wg_threads = 256;
    float* const part_group = a.partials + static_cast<size_t>(group) * C * rows_cap * RP;
    float* const part_mine = part_group + static_cast<size_t>(rank) * rows_cap * RP;
    const bool aborted = *reinterpret_cast<volatile int*>(&c.abort) != 0;
    if (warp >= 4 && !aborted) {
        const bool has_acc = sp.n_tiles > 0;
        #pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
            uint32_t orr[16];
            #pragma unroll
            for (int i = 0; i < 16; ++i) orr[i] = 0u;
            if (has_acc) {
                tmem_ld16<0>(tmem_o + lane_base + col0 + ch * 16, orr);
                tmem_wait_ld();
            }
            if (kl < HD && !skip) {
                #pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int cc = col0 + ch * 16 + i;
                    if (!((valid_cols >> (ch * 16 + i)) & 1u)) continue;
                    if (C == 1) {
                        float l;
                        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(l) : "r"(l_base + cc * 4u) : "memory");
                        RowInfo r = row_info(sp, cc);
                        const OutPtr dst = out_ptr<HD>(a, b, h, spec_row0, r);
                        dst.o[kl] = __float2bfloat16_rn(__uint_as_float(orr[i]) / l);
                        if (dst.lse && kl == 0) *dst.lse = (c.m_ref[cc] + log2f(l)) * 0.6931471805599453f;
                    } else {
                        __stcg(part_mine + cc * RP + kl, __uint_as_float(orr[i]));
                    }
                }
            }
        }
        if (C > 1 && kl < 32 && !skip) {
            const int cc = col0 + kl;
            float l;
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(l) : "r"(l_base + cc * 4u) : "memory");
            const float m = has_acc ? c.m_ref[cc] : -INFINITY;
            __stcg(reinterpret_cast<float2*>(part_mine + cc * RP + HD), make_float2(m == INFINITY ? -INFINITY : m, has_acc ? l : 0.f));
        }
    }
    if (C > 1 && warp >= 4) {
        // Publication and merge as in msa_attention_kernel: every thread's partial values precede its release
        // arrival on the block's counter; one thread waits (bounded) for the other CTAs of the head, which were
        // launched with this one and need nothing from it; each CTA then combines its share of the rows.
        const int t = tid - kAuxThreads;
        if (tid == kAuxThreads) SS_TRC(5, 2);
        unsigned int* cnt = reinterpret_cast<unsigned int*>(a.counters) + group;
        asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(cnt), "r"(8u >> a.cluster_shift) : "memory");
        if (tid == kAuxThreads) {
            bool ok = !aborted;
            const long long t0 = clock64();
            const long long limit = c.wait_limit;
            while (ok) {
                unsigned int now;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(now) : "l"(cnt) : "memory");
                if ((now & 2047u) == 0u) break;
                if (clock64() - t0 > limit) ok = false;
            }
            if (!ok) { c.abort = 1; set_status(a.status, SS_ERR_DEVICE_TIMEOUT); }
            c.merge_ok = ok ? 1 : 0;
        }
        named_barrier(3, wg_threads);
        if (tid == kAuxThreads) SS_TRC(5, 4);
        if (c.merge_ok && !skip) {
            const int share = rows_cap >> a.cluster_shift;
            const int first = static_cast<int>(rank) * share;
            const size_t cta_stride = static_cast<size_t>(rows_cap) * RP;
            for (int w = t; w < share * (HD / 4); w += wg_threads) {
                const int rr = w / (HD / 4), g = w - rr * (HD / 4);
                const RowInfo r = row_info(sp, first + rr);
                if (!r.valid) continue;
                const float* src = part_group + static_cast<size_t>(first + rr) * RP;
                float4 v[8];
                float2 ml[8];
                #pragma unroll
                for (int sidx = 0; sidx < 8; ++sidx) {
                    if (sidx < C) {
                        v[sidx] = __ldcg(reinterpret_cast<const float4*>(src + sidx * cta_stride + g * 4));
                        ml[sidx] = __ldcg(reinterpret_cast<const float2*>(src + sidx * cta_stride + HD));
                    }
                }
                float mx = -INFINITY;
                #pragma unroll
                for (int sidx = 0; sidx < 8; ++sidx)
                    if (sidx < C) mx = fmaxf(mx, ml[sidx].x);
                float l = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                #pragma unroll
                for (int sidx = 0; sidx < 8; ++sidx) {
                    if (sidx < C) {
                        const float wgt = ml[sidx].x == -INFINITY ? 0.f : exp2f(ml[sidx].x - mx);
                        l += wgt * ml[sidx].y;
                        acc.x += wgt * v[sidx].x; acc.y += wgt * v[sidx].y; acc.z += wgt * v[sidx].z; acc.w += wgt * v[sidx].w;
                    }
                }
                const OutPtr dst = out_ptr<HD>(a, b, h, spec_row0, r);
                const float inv = 1.f / l;
                uint2 o;
                o.x = pack_bf16(acc.x * inv, acc.y * inv);
                o.y = pack_bf16(acc.z * inv, acc.w * inv);
                *reinterpret_cast<uint2*>(dst.o + g * 4) = o;
                if (dst.lse && g == 0) *dst.lse = (mx + log2f(l)) * 0.6931471805599453f;
            }
        }
    }
    if (tid == kAuxThreads) SS_TRC(5, 5);
#ifdef SS_TRACE
    if (tid == 0) atomicMax(&g_wall[s_launch & 7][1], wall_ns());
    if (tid == 0) atomicMin(&g_wall[s_launch & 7][5], wall_ns());
    if (tid == 0 && blk < kTraceCtas) g_trace[blk][0][152] = static_cast<long long>(wall_ns());
#endif
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(G::kTmemCols) : "memory");
    }
}

}  // namespace ss
