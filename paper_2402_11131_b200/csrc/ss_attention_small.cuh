// Tree-masked multi-stream attention for heads of at most 64 query rows (Eq. 1, Eq. 2).  Included by
// ss_attention.cu after its helpers.
//
// A tile of 128 keys costs an SM 64 KB of TMA writes into shared memory and at least 64 KB of MMA operand
// reads out of it (128 B per cycle in total), so P never goes through shared memory: it is written to TMEM as
// bf16 and is the A operand of its MMA (tcgen05.mma with A in TMEM).
//
//   S = Q K^T     A = the query tile in shared memory (K-major), B = a K tile (K-major), N = 128 keys
//   O += P V      A = P in TMEM, B = the V tile (MN-major), N = head_dim
//
// The 64 rows fill half of the 128 rows of an MMA; the other half holds the rows a second time (copy 1).  The
// copies take alternate tiles: copy c exponentiates tiles c, c + 2, .. from a score buffer of its own into a P
// buffer of its own, in which the other copy's lanes stay zero, so one tile's exponentials overlap the other
// tile's MMAs, and each copy accumulates its own partial row, over its own tiles.  A copy moves its scores to
// registers (four softmax threads share a lane, 32 scores each) and hands the score buffer back at once.
//
// Softmax with a shared reference.  The four threads of a lane exponentiate against one reference m_ref (any
// value at or above the lane's scores, and not absurdly far above, gives the same result after
// normalisation): the lane's maximum over the first tile.  A later score that exceeds it by more than 2^8
// raises it: the copy's softmax threads agree on that through one reducing barrier per tile (each votes on the
// sum of its 32 exponentials), exchange their maxima through shared memory, rescale the lane's accumulator and
// their row sums, and redo the tile's P.
//
// Roles (640 threads): warp 0 lane 0 requests the query tile and the K tiles (TMA), warp 3 lane 0 the V tiles,
// into rings of their own (a K slot is free again after S, a V slot only after P V, so K runs ahead); warp 1
// lane 0 issues S and hands K slots back; warp 2 lane 0 issues P V and hands V slots back; warps 4..19 are the
// softmax threads, four to a TMEM lane.
//
// End of a CTA.  The copies exchange halves of their partial rows (O, m, l) through shared memory and each
// combines the half it keeps.  C = 1: normalise and write bf16.  Split heads (C > 1): the combined rows go to the
// workspace by bulk copy, and each CTA combines its share of the rows from all C partials as they arrive
// (publish_partial_rows, merge_partial_rows).
#pragma once

namespace ss {

// developer trace of this kernel
#ifdef SS_TRACE
#define SS_TRC(role, slot)                                                                                       \
    do {                                                                                                         \
        const int tr_cta_ = static_cast<int>(blockIdx.x) - ss::g_trace_base;                                                        \
        if (tr_cta_ >= 0 && tr_cta_ < ss::kTraceCtas && (slot) < ss::kTraceSlots) ss::g_trace[tr_cta_][role][slot] = clock64(); \
    } while (0)
#else
#define SS_TRC(role, slot) do { } while (0)
#endif

constexpr int kSmRows = 64;                       // query rows of the variant
constexpr int kSmThreads = 640;
constexpr int kSmSoftmax = 512;                   // four threads per TMEM lane
constexpr int kSmMaxSlots = 6;
constexpr int kSmDynSmem = 224 * 1024;            // one CTA per SM: with the 3 KB control block, all of its 227 KB

template <int HD>
struct GeoS {
    static constexpr int kHalves = HD > 64 ? 2 : 1;               // 64-element boxes along head_dim
    static constexpr int kBoxBytes = kTileKeys * 128;             // one TMA box: 128 keys x 128 B
    static constexpr int kSlotBytes = kHalves * kBoxBytes;        // a K tile or a V tile
    static constexpr int kQHalfBytes = 2 * kSmRows * 128;         // the 64 rows twice (copy 0, copy 1): M = 128
    static constexpr int kQBytes = kHalves * kQHalfBytes;
    static constexpr int kKSteps = HD / 16;
    static constexpr int kCpt = HD / 4;                           // accumulator columns a thread finishes
    static constexpr uint32_t kTmemCols = 512;                    // O (128), two score buffers (128 each), two P buffers (64 each)
    static constexpr int kPitch = HD + 4;                         // floats of a partial row: O, m, l, pad
    static constexpr size_t kCtaFloats = static_cast<size_t>(kSmRows) * kPitch;         // workspace of one CTA of a split head
};

struct CtrlS {
    unsigned long long q_full, q_ready;        // query tile in shared memory / the P buffers' constant zeros in place (16 warps)
    // K tiles and V tiles have rings of their own ([0] K, [1] V; tile j in slot j mod depth): a K slot is free
    // again when S of its tile is complete, a V slot only when P V is, so K tiles run ahead of V tiles
    unsigned long long slot_full[2][kSmMaxSlots / 2], slot_empty[2][kSmMaxSlots / 2];
    // by tile parity = copy that consumes the tile; each barrier is then looked at in every phase by its waiters
    unsigned long long s_full[2];              // S of a tile complete
    unsigned long long s_free[2];              // its scores are in registers (the copy's 8 warps): the copy's score buffer is free
    unsigned long long p_full[2];              // P of a tile written to the copy's P buffer (8 warps)
    // P V of tile t complete, on barrier t mod 4 (its phase is t / 4): a waiter derives the parity from t and never
    // counts phases.  Whoever waits for tile t does so before it publishes a P that tile t + 4 depends on, and
    // after it has seen a tile later than t - 4 complete (MMAs complete in issue order), so the barrier is
    // neither two phases ahead of the wait nor behind it.  With one barrier per copy a copy could find the other
    // copy's barrier two phases ahead (tiles j - 3 and j - 1 both complete), and its parity wait then never ends.
    unsigned long long pv_done[4];
    unsigned long long anc[SS_MAX_NODES];
    alignas(16) float xch[4][2 * kSmRows];     // exchange between the four threads of a lane (maxima, row sums)
    uint32_t tmem_base;
    int abort;
    int wait_limit;                            // bound of every wait, in units of 1024 cycles
};

__device__ __forceinline__ uint32_t bar_red_or(int id, int threads, bool pred) {
    uint32_t out;
    asm volatile("{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, %2, %3, q;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(out) : "r"(pred ? 1u : 0u), "r"(id), "r"(threads) : "memory");
    return out;
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                 ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(taddr) : "memory");
}
// waits whose limit comes from the control block (the caller may shorten it through the workspace header)
__device__ __noinline__ bool mbar_wait_slow_s(uint32_t bar, uint32_t parity, CtrlS* c, int* status) {
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
__device__ __forceinline__ bool mbar_wait_s(uint32_t bar, uint32_t parity, CtrlS* c, int* status) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow_s(bar, parity, c, status);
}
__device__ __forceinline__ bool mbar_wait_warp_s(uint32_t bar, uint32_t parity, CtrlS* c, int* status) {
    return __all_sync(0xffffffffu, mbar_wait_s(bar, parity, c, status));
}

template <int HD>
__global__ void __launch_bounds__(kSmThreads, 1) msa_attention_small_kernel(const __grid_constant__ AttnArgs a) {
    using G = GeoS<HD>;
    constexpr int TK = kTileKeys;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(16) CtrlS c;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int C = a.cluster;
    const int blk = static_cast<int>(blockIdx.x);
    const uint32_t rank = blk & (C - 1);
    const int group = blk >> a.cluster_shift;              // (sequence, head)
    int b = group / a.n_heads;
    const int h = group - b * a.n_heads;
    const int n_ring = a.n_kslots >> 1;                    // depth of the K ring and of the V ring
    if (tid == 0) SS_TRC(0, 0);
#ifdef SS_TRACE
    __shared__ unsigned int s_launch;
    if (tid == 0) {
        const unsigned long long key = reinterpret_cast<unsigned long long>(a.o_main);
        unsigned int found = 8;
        for (unsigned int i = 0; i < 8 && found == 8; ++i)
            if (*reinterpret_cast<volatile unsigned long long*>(&g_key[i]) == key) found = i;
        for (unsigned int i = 0; i < 8 && found == 8; ++i) {
            const unsigned long long old = atomicCAS(&g_key[i], 0ull, key);
            if (old == 0ull || old == key) found = i;
        }
        s_launch = found & 7;
        unsigned int smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        if (blk < 256) { g_cta_wall[s_launch][blk][0] = wall_ns(); g_cta_wall[s_launch][blk][3] = smid; }
    }
#endif

    const uint32_t base = smem_u32(smem_raw);              // 1024-byte aligned (checked below): swizzle atoms
    const uint32_t q_base = base;                          // [half][64 rows][128 B]: the query tile on its way to TMEM
    const uint32_t ring_base = q_base + G::kQBytes;        // [slot][K, V][half][128 keys][128 B]
    auto slot_addr = [&](int kind, int s) { return ring_base + static_cast<uint32_t>(2 * s + kind) * G::kSlotBytes; };

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
        for (int s = 0; s < kSmMaxSlots / 2; ++s) { mbar_init(smem_u32(&c.slot_full[0][s]), 1); mbar_init(smem_u32(&c.slot_full[1][s]), 1); }
        c.abort = 0;
        c.wait_limit = static_cast<int>(kWaitCycles >> 10);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&a.tm_qm); tma_prefetch_desc(&a.tm_k); tma_prefetch_desc(&a.tm_v);
        if (a.gamma > 0) { tma_prefetch_desc(&a.tm_qs); tma_prefetch_desc(&a.tm_ks); tma_prefetch_desc(&a.tm_vs); }
    } else if (tid == 64) {
        mbar_init(smem_u32(&c.q_ready), 16);
        for (int s = 0; s < kSmMaxSlots / 2; ++s) { mbar_init(smem_u32(&c.slot_empty[0][s]), 1); mbar_init(smem_u32(&c.slot_empty[1][s]), 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&c.s_full[s]), 1);
            mbar_init(smem_u32(&c.s_free[s]), 8);
            mbar_init(smem_u32(&c.p_full[s]), 8);
        }
        for (int s = 0; s < 4; ++s) mbar_init(smem_u32(&c.pv_done[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    auto dependency_wait = [&]() {
        if (tid == 0) {
            SS_TRC(0, 2);
            asm volatile("griddepcontrol.wait;" ::: "memory");
            SS_TRC(0, 3);
#ifdef SS_TRACE
            if (blk < 256) g_cta_wall[s_launch][blk][1] = wall_ns();
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
    // whole tiles are dealt out, the first CTAs of a head taking the odd ones: the last CTA has the masked tiles
    const Span sp = make_span(a, L, T, static_cast<int>(rank), 0, kTileKeys, true);

    // the K tile (kind 0) or the V tile (kind 1) of the CTA's tile j into slot st of its ring
    auto load_tile = [&](int kind, int j, int st) {
        const bool is_v = kind != 0;
        const uint32_t bar = smem_u32(&c.slot_full[kind][st]);
        mbar_expect_tx(bar, G::kSlotBytes);
        const uint32_t dst = slot_addr(kind, st);
        const int x = sp.first_key(j);
        #pragma unroll
        for (int hh = 0; hh < G::kHalves; ++hh) {
            if (sp.is_cache(j)) tma_load_3d(dst + hh * G::kBoxBytes, is_v ? &a.tm_v : &a.tm_k, hh * 64, h * a.head_coord, static_cast<int>(slot0 + x), bar);
            else tma_load_3d(dst + hh * G::kBoxBytes, is_v ? &a.tm_vs : &a.tm_ks, hh * 64, h, static_cast<int>(spec_row0 + x), bar);
        }
    };
    // The K tiles of the first two tiles are requested right away (before the dependency wait, under the caller's
    // promise): S of a tile needs only K and Q.  After the wait come the query rows, then the third K tile, then the
    // V tiles of the first two tiles (a CTA that starts late passes the wait at once, and its query rows then queue
    // behind two K tiles instead of four tiles); the rest follows once the query rows have arrived
    const int n_early = min(sp.n_tiles, min(n_ring, 2));
    const int n_early_k = min(sp.n_tiles, n_ring);          // K tiles requested by thread 0: the ring's depth
    auto prefix_only = [&](int j) { return sp.is_cache(j) && sp.first_key(j) + TK <= sp.L; };
    int n_pre = 0;
    if (a.prefix_stable) {
        if (tid == 0) {
            // the K tiles that lie wholly inside the cached prefix
            while (n_pre < n_early && prefix_only(n_pre)) { load_tile(0, n_pre, n_pre); ++n_pre; }
        }
        dependency_wait();
    }
    if (tid == 0) {
        if (skip) set_status(a.status, bad_smem ? SS_ERR_CUDA : SS_ERR_CAPACITY);
        // the query tile first: nothing can be computed before it is there
        const uint32_t qbar = smem_u32(&c.q_full);
        const bool with_spec = a.gamma > 0 && a.s0rows > 0;
        const uint32_t rows = a.tmax8 + (with_spec ? a.s0rows : 0);
        mbar_expect_tx(qbar, bad_smem ? 0u : 2u * G::kHalves * rows * 128u);
        #pragma unroll
        for (int hh = 0; hh < G::kHalves; ++hh) {
            #pragma unroll
            for (int cp = 0; cp < 2; ++cp) {
                if (bad_smem) break;
                const uint32_t dst = q_base + hh * G::kQHalfBytes + cp * (kSmRows * 128u);
                tma_load_3d(dst, &a.tm_qm, hh * 64, h, b * a.max_nodes, qbar);
                if (with_spec) tma_load_3d(dst + a.tmax8 * 128u, &a.tm_qs, hh * 64, h, static_cast<int>(spec_row0), qbar);
            }
        }
        for (int j = n_pre; j < n_early_k; ++j) load_tile(0, j, j);
        for (int j = 0; j < n_early; ++j) load_tile(1, j, j);
        SS_TRC(0, 5);
    }
    if (tid >= kAuxThreads && tid < kAuxThreads + SS_MAX_NODES) c.anc[tid - kAuxThreads] = __ldcg(&a.trees[b].anc_mask[tid - kAuxThreads]);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (tid == 0) SS_TRC(0, 6);
    const uint32_t tmem = c.tmem_base;
    const uint32_t tmem_o = tmem;                          // 128 columns
    const uint32_t tmem_s = tmem + 128;                    // two score buffers of 128 columns, one per copy
    const uint32_t tmem_p = tmem + 384;                    // two P buffers of 64 columns (128 keys as bf16), one per copy
    int* const status = a.status;
    // tile j of a kind: slot j mod depth, filled for the (j / depth)-th time
    auto wait_tile_full = [&](int kind, const Ring& r) {
        return mbar_wait_s(smem_u32(&c.slot_full[kind][r.slot]), static_cast<uint32_t>(r.round & 1), &c, status);
    };
    // the tiles after the early ones, each as soon as its slot is free; a producer that gives up lets the
    // copies already in flight land before the CTA leaves
    auto produce = [&](int kind) {
        Ring r;
        r.start();
        const int first = kind ? n_early : n_early_k;
        for (int j = 0; j < first; ++j) r.advance(n_ring);
        bool ok = mbar_wait_s(smem_u32(&c.q_full), 0, &c, status);
        int j = first;
        for (; ok && j < sp.n_tiles; ++j) {
            if (r.round > 0) ok = mbar_wait_s(smem_u32(&c.slot_empty[kind][r.slot]), (r.round - 1) & 1, &c, status);
            if (kind == 0) SS_TRC(0, 8 + j);
            if (ok) { load_tile(kind, j, r.slot); r.advance(n_ring); }
        }
        if (!ok) {
            const int issued = r.slot + r.round * n_ring;
            Ring d;
            d.start();
            for (int i = 0; i < issued; ++i, d.advance(n_ring))
                if (i >= issued - n_ring) mbar_drain(smem_u32(&c.slot_full[kind][d.slot]), static_cast<uint32_t>(d.round & 1));
        }
    };

    // =============================== warps 0 and 3: tile requests ================================
    if (warp == 0) {
        if (lane == 0 && sp.n_tiles > n_early_k) produce(0);
    } else if (warp == 3) {
        if (lane == 0) {
            // the caller may shorten the bound of the device-side waits (workspace word 1, units of 1024 cycles)
            int lim;
            asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(lim) : "l"(a.status + 1) : "memory");
            if (lim > 0) *reinterpret_cast<volatile int*>(&c.wait_limit) = lim;
            if (sp.n_tiles > n_early) produce(1);
        }
    }
    // =============================== warp 1: S = Q K^T, A from TMEM ================================
    else if (warp == 1) {
        if (lane == 0) {
            bool ok = mbar_wait_s(smem_u32(&c.q_full), 0, &c, status);
            if (!ok) mbar_drain(smem_u32(&c.q_full), 0);
            SS_TRC(1, 0);
            const uint64_t dq = desc_k_major(q_base);
            Ring r;
            r.start();
            for (int j = 0; ok && j < sp.n_tiles; ++j) {
                const int buf = j & 1;
                if (!wait_tile_full(0, r)) break;
                SS_TRC(1, 8 + 4 * j);
                // the copy's scores of its tile before must be in registers
                if (j >= 2 && !mbar_wait_s(smem_u32(&c.s_free[buf]), ((j >> 1) - 1) & 1, &c, status)) break;
                SS_TRC(1, 9 + 4 * j);
                tc_fence_after();
                const uint64_t dk = desc_k_major(slot_addr(0, r.slot));
                #pragma unroll
                for (int ks = 0; ks < G::kKSteps; ++ks) {
                    const uint32_t hh = ks >> 2, off = (ks & 3) * 32u;
                    tc_mma(tmem_s + buf * TK, dq + ((hh * G::kQHalfBytes + off) >> 4), dk + ((hh * G::kBoxBytes + off) >> 4),
                           idesc_bf16(TK, false, false), ks > 0);
                }
                tc_commit(smem_u32(&c.s_full[buf]));
                tc_commit(smem_u32(&c.slot_empty[0][r.slot]));                // K may go when S is complete
                SS_TRC(1, 10 + 4 * j);
                r.advance(n_ring);
            }
        }
    }
    // =============================== warp 2: O += P V, A from TMEM ================================
    else if (warp == 2) {
        if (lane == 0) {
            Ring rv;
            rv.start();
            bool okq = mbar_wait_s(smem_u32(&c.q_ready), 0, &c, status);     // the P buffers' constant zeros are in place
            for (int j = 0; okq && j < sp.n_tiles; ++j) {
                const int buf = j & 1;
                if (!wait_tile_full(1, rv)) break;
                SS_TRC(2, 8 + 4 * j);
                if (!mbar_wait_s(smem_u32(&c.p_full[buf]), (j >> 1) & 1, &c, status)) break;
                SS_TRC(2, 9 + 4 * j);
                tc_fence_after();
                const uint64_t dv = desc_mn_major(slot_addr(1, rv.slot), G::kBoxBytes);
                // P of the tile: the copy's buffer, keys 16 ks .. 16 ks + 15 in columns 8 ks .. 8 ks + 7 (zero in the
                // other copy's lanes)
                #pragma unroll
                for (int ks = 0; ks < TK / 16; ++ks)
                    tc_mma_ts(tmem_o, tmem_p + buf * 64u + 8u * ks, dv + ((ks * 2048u) >> 4), idesc_bf16(HD, false, true),
                              (j > 0 || ks > 0) ? 1u : 0u);
                tc_commit(smem_u32(&c.pv_done[j & 3]));
                tc_commit(smem_u32(&c.slot_empty[1][rv.slot]));
                SS_TRC(2, 10 + 4 * j);
                rv.advance(n_ring);
            }
        }
    }
    // =============================== warps 4..19: softmax =========================================
    const int w4 = warp >= 4 ? (warp - 4) >> 2 : 0;                           // which 32 keys of a tile (and which quarter of a row)
    const int tl = ((warp & 3) << 5) | lane;                                  // TMEM lane = (copy, row)
    const int copy = tl >> 6, row = tl & 63;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    float m_ref = -INFINITY, l_part = 0.f;
    RowInfo ri;
    ri.valid = false; ri.node = 0; ri.stream = 0;
    if (warp >= 4) {
        ri = row_info(sp, row);
        const unsigned long long anc = ri.valid ? c.anc[ri.node] : 0ull;
        // ---- the lane's part of the other copy's P buffer is zero for the whole kernel
        {
            uint32_t zr[16];
            #pragma unroll
            for (int i = 0; i < 16; ++i) zr[i] = 0u;
            tmem_st16<0>(tmem_p + lane_base + static_cast<uint32_t>((1 - copy) * 64 + 16 * w4), zr);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&c.q_ready));
        }
        if (tid == kAuxThreads) SS_TRC(5, 6);
        const bool leader = (tid == kAuxThreads) || (tid == kAuxThreads + 64);      // lane 0 of each copy's first warp
        const uint32_t p_addr = tmem_p + lane_base + static_cast<uint32_t>(copy * 64 + 16 * w4);   // my 32 keys of a tile as bf16
        const uint32_t o_addr = tmem_o + lane_base + 32u * w4;
        auto wait_pv_tile = [&](int t) {                                       // P V of tile t complete
            return mbar_wait_warp_s(smem_u32(&c.pv_done[t & 3]), static_cast<uint32_t>((t >> 2) & 1), &c, status);
        };
        bool failed = false;
        // copy c takes the tiles j = c, c + 2, ..: all 128 keys of the tile for its 64 rows
        for (int j = copy; j < sp.n_tiles; j += 2) {
            bool ok = mbar_wait_warp_s(smem_u32(&c.s_full[copy]), (j >> 1) & 1, &c, status);
            if (leader) SS_TRC(3, 8 + 6 * j);
            tc_fence_after();
            const int x0 = sp.first_key(j), nvk = sp.valid_keys(j);
            const bool cache = sp.is_cache(j);
            const bool masked = !cache || x0 + TK > sp.L || nvk < TK;
            const uint32_t vis = masked ? static_cast<uint32_t>(visible_mask(cache, x0 + 32 * w4, nvk - 32 * w4, sp.L, sp.gamma, ri, anc) & 0xffffffffull)
                                        : 0xffffffffu;
            uint32_t sr[32];
            if (ok) {
                tmem_ld32<0>(tmem_s + lane_base + static_cast<uint32_t>(copy * TK) + 32u * w4, sr);
                tmem_wait_ld();
            }
            // the scores are in registers: S of the copy's next tile may overwrite the buffer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&c.s_free[copy]));

            // Raises the lane's reference to its maximum over this tile and rescales what it has accumulated.  The
            // P V of the tile before this one is the last that can have been issued (they are issued in tile order
            // and this tile's P is not published yet): once it is complete the accumulator is at rest.
            auto raise = [&]() {
                float mx = -INFINITY;
                #pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float v = __uint_as_float(sr[i]) * a.scale_log2;
                    mx = fmaxf(mx, ((vis >> i) & 1u) ? v : -INFINITY);
                }
                c.xch[w4][tl] = mx;
                named_barrier(6 + copy, 256);
                const float m_new = ri.valid ? fmaxf(fmaxf(m_ref, fmaxf(c.xch[0][tl], c.xch[1][tl])), fmaxf(c.xch[2][tl], c.xch[3][tl]))
                                             : INFINITY;       // a lane without a row never asks for a raise again
                const float corr = m_new == m_ref ? 1.f : exp2f(m_ref - m_new);          // 0 when nothing was visible so far
                m_ref = m_new;
                l_part *= corr;
                bool ok2 = true;
                if (j >= 2) {
                    ok2 = wait_pv_tile(j - 1);
                    tc_fence_after();
                    if (ok2) {
                        uint32_t orr[32];
                        tmem_ld32<0>(o_addr, orr);
                        tmem_wait_ld();
                        #pragma unroll
                        for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * corr);
                        tmem_st32(o_addr, orr);
                        tmem_wait_st();
                    }
                }
                // the copy's reducing barrier of this tile lies between these reads and the next raise's writes
                return ok2;
            };

            if (j < 2) raise();                                               // every thread of the copy, so the barriers inside match
            bool leave = false;
            for (int attempt = 0; attempt < 3; ++attempt) {
                float lsum = 0.f;
                if (ok) {
                    // two scores per instruction (packed fp32 pairs) for the scaling and for the row sum
                    uint32_t pk[16];
                    const unsigned long long scale2 = pack_f32x2(a.scale_log2, a.scale_log2), shift2 = pack_f32x2(-m_ref, -m_ref);
                    unsigned long long sum2 = pack_f32x2(0.f, 0.f);
                    #pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float t0, t1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sr[i]), __uint_as_float(sr[i + 1])), scale2, shift2), t0, t1);
                        float e0 = exp2f(t0), e1 = exp2f(t1);
                        if (masked) {
                            e0 = ((vis >> i) & 1u) ? e0 : 0.f;
                            e1 = ((vis >> (i + 1)) & 1u) ? e1 : 0.f;
                        }
                        sum2 = add_f32x2(sum2, pack_f32x2(e0, e1));
                        pk[i >> 1] = pack_bf16(e0, e1);
                    }
                    float s0, s1;
                    unpack_f32x2(sum2, s0, s1);
                    lsum = s0 + s1;
                    // P of this copy's previous tile must have been read before it is overwritten
                    if (attempt == 0 && j >= 2) ok = wait_pv_tile(j - 2);
                    if (ok) tmem_st16<0>(p_addr, pk);
                }
                if (leader) SS_TRC(3, 9 + 6 * j + (attempt > 0 ? 3 : 0));
                // one reducing barrier per tile: did a score outgrow its reference, or did a wait run out
                // (a thread's 32 exponentials sum to at most 32 unless a score is above the reference; past
                // 32 * 2^8 one of them is more than 2^8 above it)
                const uint32_t any = bar_red_or(4 + copy, 256, !ok || lsum > 32.f * 256.f);
                if (leader) SS_TRC(3, 10 + 6 * j);
                if (!any) { l_part += lsum; break; }
                if (*reinterpret_cast<volatile int*>(&c.abort)) { leave = true; break; }
                ok = raise() && ok;
                if (attempt == 2) l_part += lsum;
            }
            if (leave) { failed = true; break; }
            // V rows past the end of the sequence's keys may hold anything (even NaN patterns): P is 0 there,
            // but 0 * NaN is NaN, so they are cleared: a thread looks after rows (row, row + 64) of the tile
            const int region_left = (cache ? sp.L + sp.T : sp.n_stream) - x0;
            if (region_left < TK) {
                const int vs = j % n_ring;
                if (mbar_wait_warp_s(smem_u32(&c.slot_full[1][vs]), static_cast<uint32_t>((j / n_ring) & 1), &c, status)) {
                    #pragma unroll
                    for (int up = 0; up < 2; ++up) {
                        const int vr = row + 64 * up;
                        if (vr >= region_left && (w4 >> 1) < G::kHalves) {
                            const uint32_t dst = slot_addr(1, vs) + (w4 >> 1) * G::kBoxBytes + vr * 128u + (w4 & 1) * 64u;
                            #pragma unroll
                            for (int i = 0; i < 4; ++i) st_shared_v4(dst + i * 16, 0u, 0u, 0u, 0u);
                        }
                    }
                    fence_async_smem();
                }
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&c.p_full[copy]));
            if (leader) SS_TRC(3, 11 + 6 * j);
        }
        // every P V must be complete before the accumulator is read: they complete in issue order, so the last one
        if (!failed && sp.n_tiles > 0) {
            wait_pv_tile(sp.n_tiles - 1);
            tc_fence_after();
        }
    }
    __syncwarp();
    if (tid == kAuxThreads) SS_TRC(5, 0);

    // ======================================== epilogue ==========================================
    // A lane's partial over the keys of its copy: O in TMEM, the reference, and the sum of its four threads' row
    // sums.  The copies exchange halves of their rows through shared memory (the rings are idle: every copy has
    // landed and every MMA is complete) and each combines the half it keeps.  C = 1: normalise and write bf16.
    // Split head: the combined rows are staged in shared memory, the copy engine takes them to the workspace (they
    // stay in L2), and each CTA combines its share of the rows as they arrive from the CTAs of the head.
    constexpr int CPT = G::kCpt;
    constexpr uint32_t YB = G::kPitch * 4;                                    // bytes of a staged row
    const uint32_t y_base = ring_base;                                        // [64 rows][kPitch floats]
    float* const part_group = a.partials + static_cast<size_t>(group) * C * G::kCtaFloats;
    float* const part_mine = part_group + static_cast<size_t>(rank) * G::kCtaFloats;
    const bool has_acc = sp.n_tiles > 0;
    if (warp >= 4) {
        c.xch[w4][tl] = l_part;
        named_barrier(8, kSmSoftmax);
        float l_lane = (c.xch[0][tl] + c.xch[1][tl]) + (c.xch[2][tl] + c.xch[3][tl]);
        const bool aborted = *reinterpret_cast<volatile int*>(&c.abort) != 0;
        uint32_t orr[32];
        #pragma unroll
        for (int i = 0; i < 32; ++i) orr[i] = 0u;
        if (has_acc && !aborted) {
            tmem_ld32<0>(tmem_o + lane_base + static_cast<uint32_t>(CPT * w4), orr);
            tmem_wait_ld();
        }
        if (!has_acc || !ri.valid) { m_ref = -INFINITY; l_lane = 0.f; }
        if (tid == kAuxThreads) SS_TRC(5, 1);
        // The two threads that hold a row's columns [CPT w4, CPT w4 + CPT) -- one per copy -- each hand one half of
        // them to the other through shared memory (X) and combine the half they keep: copy 0 the first CPT / 2
        // columns, copy 1 the rest.
        constexpr int HC = CPT / 2;                                           // columns a thread keeps
        constexpr int VW = HC % 4 == 0 ? 4 : 2;                               // words per shared-memory access
        const uint32_t x_base = y_base + kSmRows * YB;                        // [64 rows][kPitch floats], then (m, l) of both copies per row
        const uint32_t xml = x_base + kSmRows * YB + static_cast<uint32_t>(row) * 16u;
        const uint32_t yrow = y_base + static_cast<uint32_t>(row) * YB, xrow = x_base + static_cast<uint32_t>(row) * YB;
        const int keep0 = copy == 0 ? 0 : HC, give0 = copy == 0 ? HC : 0;     // first kept / given column of my CPT
        #pragma unroll
        for (int i = 0; i < HC; ++i) {                                        // registers: kept columns first, then the given ones
            const uint32_t lo = orr[i], hi = orr[HC + i];
            orr[i] = copy == 0 ? lo : hi;
            orr[HC + i] = copy == 0 ? hi : lo;
        }
        #pragma unroll
        for (int i = 0; i < HC; i += VW) {
            const uint32_t at = xrow + static_cast<uint32_t>(CPT * w4 + give0 + i) * 4u;
            if constexpr (VW == 4) st_shared_v4(at, orr[HC + i], orr[HC + i + 1], orr[HC + i + 2], orr[HC + i + 3]);
            else st_shared_v2(at, orr[HC + i], orr[HC + i + 1]);
        }
        if (w4 == 0) st_shared_v2(xml + copy * 8u, __float_as_uint(m_ref), __float_as_uint(l_lane));
        named_barrier(8, kSmSoftmax);
        if (tid == kAuxThreads) SS_TRC(5, 8);
        const float2 z = ld_shared_v2(xml + (1 - copy) * 8u);                 // the other copy's (m, l)
        const float m_out = fmaxf(m_ref, z.x);
        const float wa = m_ref == -INFINITY ? 0.f : exp2f(m_ref - m_out), wb = z.x == -INFINITY ? 0.f : exp2f(z.x - m_out);
        const float l_out = wa * l_lane + wb * z.y;
        float keep[HC];
        #pragma unroll
        for (int i = 0; i < HC; i += VW) {
            const uint32_t at = xrow + static_cast<uint32_t>(CPT * w4 + keep0 + i) * 4u;
            if constexpr (VW == 4) {
                const float4 t4 = ld_shared_v4(at);
                keep[i] = wa * __uint_as_float(orr[i]) + wb * t4.x;
                keep[i + 1] = wa * __uint_as_float(orr[i + 1]) + wb * t4.y;
                keep[i + 2] = wa * __uint_as_float(orr[i + 2]) + wb * t4.z;
                keep[i + 3] = wa * __uint_as_float(orr[i + 3]) + wb * t4.w;
            } else {
                const float2 t2 = ld_shared_v2(at);
                keep[i] = wa * __uint_as_float(orr[i]) + wb * t2.x;
                keep[i + 1] = wa * __uint_as_float(orr[i + 1]) + wb * t2.y;
            }
        }
        if (C == 1) {
            if (ri.valid && !skip && !aborted) {
                const float inv = 1.f / l_out;
                const OutPtr dst = out_ptr<HD>(a, b, h, spec_row0, ri);
                #pragma unroll
                for (int i = 0; i < HC; i += VW) {
                    __nv_bfloat16* at = dst.o + CPT * w4 + keep0 + i;
                    if constexpr (VW == 4) {
                        uint2 o;
                        o.x = pack_bf16(keep[i] * inv, keep[i + 1] * inv);
                        o.y = pack_bf16(keep[i + 2] * inv, keep[i + 3] * inv);
                        *reinterpret_cast<uint2*>(at) = o;
                    } else {
                        *reinterpret_cast<uint32_t*>(at) = pack_bf16(keep[i] * inv, keep[i + 1] * inv);
                    }
                }
                if (dst.lse && w4 == 0 && copy == 0) *dst.lse = (m_out + log2f(l_out)) * 0.6931471805599453f;
            }
        } else {
            // the combined row, staged for the copy engine (never +0: a word of a partial row that reads zero in the
            // workspace has not arrived)
            #pragma unroll
            for (int i = 0; i < HC; i += VW) {
                const uint32_t at = yrow + static_cast<uint32_t>(CPT * w4 + keep0 + i) * 4u;
                if constexpr (VW == 4)
                    st_shared_v4(at, never_plus_zero(__float_as_uint(keep[i])), never_plus_zero(__float_as_uint(keep[i + 1])),
                                 never_plus_zero(__float_as_uint(keep[i + 2])), never_plus_zero(__float_as_uint(keep[i + 3])));
                else
                    st_shared_v2(at, never_plus_zero(__float_as_uint(keep[i])), never_plus_zero(__float_as_uint(keep[i + 1])));
            }
            if (w4 == 0 && copy == 0) st_shared_v4(yrow + HD * 4u, never_plus_zero(__float_as_uint(m_out)), never_plus_zero(__float_as_uint(l_out)), 0u, 0u);
            fence_async_smem();                           // the copy engine reads these rows
        }
        if (C > 1) {
            named_barrier(8, kSmSoftmax);                                     // the staged rows are complete
            if (tid == kAuxThreads) SS_TRC(5, 9);
            const int t = tid - kAuxThreads;
            const bool live = __all_sync(0xffffffffu, !skip && !aborted);
            const int share = kSmRows >> a.cluster_shift, first = static_cast<int>(rank) * share;
            if (live && t == 0) publish_partial_rows<HD>(sp, 0, kSmRows, y_base, part_mine, first, share);
            if (tid == kAuxThreads) SS_TRC(5, 2);
            // the other CTAs of the head were launched with this one and need nothing from it: the wait is short
            const long long limit = static_cast<long long>(*reinterpret_cast<volatile int*>(&c.wait_limit)) << 10;
            if (live && !merge_partial_rows<HD>(a, sp, 0, b, h, spec_row0, C, static_cast<int>(rank), y_base, part_group, G::kCtaFloats, first,
                                                share, t, kSmSoftmax, limit, &c.abort)) {
                c.abort = 1;
                set_status(a.status, SS_ERR_DEVICE_TIMEOUT);
            }
            if (live && t == 0) bulk_copies_read();
        }
    }
    if (tid == kAuxThreads) SS_TRC(5, 5);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(G::kTmemCols) : "memory");
    }
#ifdef SS_TRACE
    if (tid == kAuxThreads && blk < 256) g_cta_wall[s_launch][blk][2] = wall_ns();
#endif
}

}  // namespace ss
