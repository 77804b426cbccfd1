// Tree-masked multi-stream attention, one layer (Eq. 1, Eq. 2): flash-decode for sm_100a.
//
// Work decomposition.  The query rows of a (sequence, head) pair -- T main rows, then the T*gamma
// stream rows -- form one tile when there are at most 64 of them (msa_attention_small_kernel, in
// ss_attention_small.cuh), else blocks of 128 rows that go to separate CTAs (msa_attention_kernel, here;
// a block streams the keys it can see: the cached slots, and the stream keys of its own nodes).  C CTAs
// (a power of two, chosen so that the grid fills the SMs once) share the keys of a block: the cached
// slots [0, L+T) (prefix, then this step's tree nodes, masked by ancestry) and the block's transient
// stream keys (node-major) are cut into 16-key units and CTA r takes units [U*r/C, U*(r+1)/C), so every
// CTA of a block streams the same number of bytes.  The CTAs of a pair run in the same wave, so a K/V
// tile crosses HBM once and is served from L2 to the other row blocks.  A batch (up to 32 sequences, no
// key split) is dispatched longest prefix first.
//
// Inside a CTA of msa_attention_kernel.
//   threads 0, 96  TMA producers of the K ring and of the V ring (mbarrier complete_tx); swizzle-128B
//               boxes straight from the caller's strided tensors.  A K slot is handed back as soon
//               as S is queued, a V slot after P V.  Thread 0 also requests Q once.
//   warp 1      tcgen05 issuer of S = Q K^T (128 x 128 keys x d) into one of two TMEM buffers;
//   warp 2      tcgen05 issuer of O += P V (A = P in TMEM) into the TMEM accumulator of a warpgroup;
//               tcgen05.commit arrives on the mbarriers that hand buffers back.
//   warps 4..11 two softmax warpgroups, one thread per TMEM lane: tcgen05.ld of the row's scores, tree /
//               stream mask from the node's 64-bit ancestor word, exponentials and row sums in fp32
//               registers, P as bf16 back to TMEM, from where the second MMA takes it.  Two pipelines:
//               - a block whose keys are not split (C == 1, the long key sequences): the warpgroups take
//                 alternate tiles against one reference per row, the maximum of the row's first tile
//                 (any reference not absurdly far from the row's maximum gives the same result after
//                 normalisation); one accumulator; P in TMEM buffers of its own, so a score buffer goes
//                 back to the S issuer as soon as its scores are in registers and one tile's exponentials
//                 run beside the other tile's MMAs.  If a later tile's exponentials would leave the range
//                 of fp32 (a tile's row sum above 2^64), the CTA lets everything in flight land, sets its
//                 barriers up anew and runs its tiles again on the other pipeline;
//               - a split block (short key spans), or a block that started over: of every tile warpgroup 0
//                 takes keys 0..63 and warpgroup 1 keys 64..127, each with its own running maximum (raised
//                 only when it would grow by more than 2^8) and accumulator; P is written over the first
//                 32 of the score columns just read.
//
// Split-KV merge.  Each CTA ends with un-normalised (m, l, O) per row, combines what it holds for a
// row locally, and -- when the keys were split -- leaves one partial row in the workspace (it stays in
// L2).  The rows are their own arrival flags (the area is zero between calls and +0 is never stored):
// each CTA polls, bounded, the rows of its own share from all CTAs of the block (launched with it,
// needing nothing from it), combines them, writes bf16 output and stores zeros over what it read.
//
// Launch.  Programmatic dependent launch: one thread of each CTA waits for the previous kernel of
// the stream; before that wait the kernel touches global memory only under the caller's
// SS_ATTN_PREFIX_STABLE promise (lengths, trees and wholly-prefix K/V tiles).  Every wait in the
// kernel is bounded and reports SS_ERR_DEVICE_TIMEOUT.
#include <cuda.h>
#include <cuda_bf16.h>
#include <type_traits>

#include "ss_common.cuh"

namespace ss {

// Developer build (-DSS_TRACE): per-role clock64 timestamps of the first CTAs, read back with
// ss_trace_read.  Compiled out of the product library.
#ifdef SS_TRACE
constexpr int kTraceCtas = 16, kTraceRoles = 6, kTraceSlots = 160;
__device__ long long g_trace[kTraceCtas][kTraceRoles][kTraceSlots];
__device__ int g_trace_base;
__device__ unsigned long long g_cta_wall[8][256][4];   // per launch and CTA: start, wait released, end (globaltimer ns), SM id
__device__ unsigned long long g_wall[8][6];      // first CTA start / last CTA end (globaltimer ns) of the last 8 launches
__device__ unsigned long long g_key[8];           // launch identity: the output pointer
__device__ __forceinline__ unsigned long long wall_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define SS_TR(role, slot)                                                                                   \
    do {                                                                                                    \
        if (blockIdx.x < ss::kTraceCtas && (slot) < ss::kTraceSlots) ss::g_trace[blockIdx.x][role][slot] = clock64(); \
    } while (0)
#else
#define SS_TR(role, slot) do { } while (0)
#endif

constexpr int kUnit = 16;            // split granularity (keys)
constexpr int kBlockRows = 128;      // query rows per block (M of both MMAs)
constexpr int kTileKeys = 128;       // keys per tile: N = 128 MMAs run at the full tensor rate
constexpr int kMaxSlots = 4;         // slots per ring (K ring, V ring)
constexpr int kAuxThreads = 128;     // warps 0..3: producers and MMA issuers
constexpr int kPairMaxDynSmem = 232448 - 2048;   // 227 KB per CTA less the static control block (up to 2 KB) of msa_attention_kernel
// Row blocks that are not split take the shared-reference pipeline: a row's exponentials are taken against the
// maximum of its first tile for as long as a tile's 128 of them sum to at most 2^64 (no overflow anywhere: bf16
// and fp32 reach 2^127); past that the CTA starts over with a running maximum per warpgroup.
constexpr float kSharedRefLimit = 18446744073709551616.f;
constexpr float kRescaleStep = 8.f;  // raise the running maximum only when it grows by more than 2^8
constexpr long long kWaitCycles = 2000000000ll;   // bound of every mbarrier wait (~1 s)

struct alignas(64) AttnArgs {
    CUtensorMap tm_k, tm_v;          // cache slab    dims (d, H, slots)        box (64, 1, 128)
    CUtensorMap tm_qm;               // q_main        dims (d, H, B*Tmax)       box (64, 1, tmax8)
    CUtensorMap tm_qs;               // q_spec        dims (d, H, B*Tmax*g)     box (64, 1, s0rows): stream rows of block 0
    CUtensorMap tm_qs1;              // q_spec        the same tensor           box (64, 1, 128): later row blocks
    CUtensorMap tm_ks, tm_vs;        // k_spec/v_spec dims (d, H, B*Tmax*g)     box (64, 1, 128)
    int batch, n_heads, gamma, max_nodes;
    int tmax8;                       // max_nodes rounded up to 8: first stream row of the head's query tile
    int s0rows;                      // stream rows that share block 0 with the main rows
    int n_blocks;                    // 128-row blocks per head (1 for heads of at most 64 rows)
    int cluster, cluster_shift;      // CTAs that share a block's keys; cluster = 1 << cluster_shift
    int n_kslots, n_vslots;          // ring depths
    int head_coord;                  // 1, or 0 when all heads share one K/V (head stride 0)
    int gamma_magic;                 // ceil(65536 / gamma): x / gamma == (x * gamma_magic) >> 16 for x < 256
    int prefix_stable;               // the caller's SS_ATTN_PREFIX_STABLE promise
    float scale_log2;                // sm_scale * log2(e)
    __nv_bfloat16* o_main;
    __nv_bfloat16* o_spec;
    float* lse_main;
    float* lse_spec;
    const long long* kv_start;
    const int* kv_len;
    const int* kv_capacity;
    const ss_tree_desc* trees;
    int* status;
    float* partials;                 // [groups][splits][rows][head_dim + 4]
};

struct Ctrl {
    unsigned long long q_full;
    unsigned long long k_full[kMaxSlots], k_empty[kMaxSlots], v_full[kMaxSlots], v_empty[kMaxSlots];
    unsigned long long s_full[2][2];            // per (warpgroup, S buffer): a warpgroup sees every phase of its own
    unsigned long long s_free[2];
    // P of a warpgroup written: [w][tile & 1], one arrival per warp: a warp can only be two tiles ahead of another
    // once the P V between them is complete, so it never arrives twice in a phase
    unsigned long long p_full[2][2];
    // P V of a warpgroup complete: [w][tile & 1]: a warpgroup that does not look at every phase is then never more
    // than one phase behind, which a parity wait needs
    unsigned long long o_done[2][2];
    unsigned long long anc[SS_MAX_NODES];
    // shared-reference pipeline: the reference of each row (warpgroup 0 sets it from the first tile, one barrier per
    // warp of 32 rows), and the barriers on which the MMA issuers wait for their last MMAs when the CTA starts over
    unsigned long long mref_full[4], drain[2];
    float m_ref[kBlockRows];
    uint32_t tmem_base;
    int abort;                                  // 1: a wait ran out of time; 2: the shared reference did not hold, start over
#ifdef SS_TRACE
    unsigned int trace_launch;
#endif
};
static_assert(sizeof(Ctrl) + 16 <= 232448 - kPairMaxDynSmem, "control block and dynamic shared memory exceed an SM");

// ---------------------------------------------------------------------------------------------
// PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ float4 ld_shared_v4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up when another thread of the CTA already gave up, or after kWaitCycles.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort, int* status) {
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 256; ++i) {
            if (mbar_try(bar, parity)) return true;
            if (*abort) return false;
        }
        if (clock64() - t0 > kWaitCycles) {
            *abort = 1;
            set_status(status, SS_ERR_DEVICE_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort, int* status) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort, status);
}
// the same for a whole warp: either every lane saw the phase complete or every lane gives up
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort, int* status) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort, status));
}
// after giving up: a short bounded wait that lets a copy already in flight land
__device__ __noinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!mbar_try(bar, parity) && clock64() - t0 < kWaitCycles / 16) {}
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
__device__ __forceinline__ void named_barrier(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void st_shared_v2(uint32_t addr, uint32_t x, uint32_t y) {
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ float2 ld_shared_v2(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]: A is 128 lanes x 16 bf16, two to a 32-bit column (8 columns per step)
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

#define SS_R16(r, o) "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), \
                     "=r"(r[o + 6]), "=r"(r[o + 7]), "=r"(r[o + 8]), "=r"(r[o + 9]), "=r"(r[o + 10]), "=r"(r[o + 11]), \
                     "=r"(r[o + 12]), "=r"(r[o + 13]), "=r"(r[o + 14]), "=r"(r[o + 15])
#define SS_W16(r, o) "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), \
                     "r"(r[o + 6]), "r"(r[o + 7]), "r"(r[o + 8]), "r"(r[o + 9]), "r"(r[o + 10]), "r"(r[o + 11]), \
                     "r"(r[o + 12]), "r"(r[o + 13]), "r"(r[o + 14]), "r"(r[o + 15])
// N consecutive fp32 columns of this thread's TMEM lane <-> registers r[O .. O+N-1]
template <int O, int N>
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[N]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : SS_R16(r, O) : "r"(taddr) : "memory");
}
template <int O, int N>
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[N]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : SS_R16(r, O), SS_R16(r, O + 16) : "r"(taddr) : "memory");
}
template <int O, int N>
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[N]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
        ::SS_W16(r, O), "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"
        ::SS_W16(r, 0), SS_W16(r, 16), "r"(taddr) : "memory");
}
// 64 columns starting at taddr
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t (&r)[64]) {
    tmem_ld32<0>(taddr, r);
    tmem_ld32<32>(taddr + 32, r);
}

// packed pairs of fp32 (one instruction for two values)
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
    unsigned long long v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.ftz.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long add_f32x2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.ftz.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Shared-memory matrix descriptors (swizzle-128B canonical layouts, 8-row groups 1024 B apart).
//   K-major  (Q, K, P): rows of 128 B, the contraction index contiguous; a 16-element step is +32 B.
//   MN-major (V): rows of 128 B are keys (contraction), the 64 contiguous elements are head_dim;
//                 the next 64 elements of head_dim start `lbo` bytes further; a 16-key step is +2048 B.
__device__ __forceinline__ uint64_t desc_k_major(uint32_t addr) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (1ull << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint64_t desc_mn_major(uint32_t addr, uint32_t lbo) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo >> 4) << 16) |
           (static_cast<uint64_t>(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, M = 128
__host__ __device__ constexpr uint32_t idesc_bf16(int n, bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (a_mn_major ? (1u << 15) : 0u) | (b_mn_major ? (1u << 16) : 0u) |
           (static_cast<uint32_t>(n >> 3) << 17) |
           (static_cast<uint32_t>(kBlockRows >> 4) << 24);
}

// ---------------------------------------------------------------------------------------------
// The CTA's share of its row block's keys, as a list of tiles of kTileKeys keys.  Every role derives
// it from the same few numbers, so no tile list is ever stored.
struct Span {
    int L, T, n_stream;            // prefix length, tree nodes, stream keys of the sequence (T * gamma)
    int kc0, kc1;                  // cache keys [kc0, kc1) (indices into [0, L+T))
    int ks0, ks1;                  // stream keys [ks0, ks1) (indices into [0, T*gamma))
    int n_cache_tiles, n_tiles;
    int tmax8, gamma;
    int spec_end;                  // valid rows of the head: [0, T) and [tmax8, spec_end)
    int row0;                      // first row of this CTA's block

    __device__ __forceinline__ bool is_cache(int j) const { return j < n_cache_tiles; }
    __device__ __forceinline__ int first_key(int j) const {
        return j < n_cache_tiles ? kc0 + j * kTileKeys : ks0 + (j - n_cache_tiles) * kTileKeys;
    }
    __device__ __forceinline__ int valid_keys(int j) const {
        return min(kTileKeys, (j < n_cache_tiles ? kc1 : ks1) - first_key(j));
    }
};

// position in a ring of n slots: slot index and the number of completed rounds
struct Ring {
    int slot, round;
    __device__ __forceinline__ void start() { slot = 0; round = 0; }
    __device__ __forceinline__ void advance(int n) {
        if (++slot == n) { slot = 0; ++round; }
    }
};

__device__ __forceinline__ Span make_span(const AttnArgs& a, int L, int T, int rank, int rb, int unit, bool front_heavy = false) {
    Span s;
    s.L = L; s.T = T; s.gamma = a.gamma; s.tmax8 = a.tmax8;
    s.n_stream = T * a.gamma;
    s.spec_end = a.tmax8 + s.n_stream;
    s.row0 = rb * kBlockRows;
    // stream rows [x0, x1) of the block (numbered from the first stream row); row x = (node, stream) sees
    // the stream keys node*gamma .. x, so the block sees the keys from its first node's first stream on
    const int x0 = max(s.row0, s.tmax8) - s.tmax8, x1 = min(s.row0 + kBlockRows, s.spec_end) - s.tmax8;
    int slo = 0, shi = 0;
    if (x1 > x0) { slo = x0 / a.gamma * a.gamma; shi = x1; }
    const bool any_row = s.row0 < T || x1 > x0;           // a block without a valid row streams nothing
    const int ec = any_row ? L + T : 0;
    const int uc = (ec + unit - 1) / unit, us = (shi - slo + unit - 1) / unit;
    const int u = uc + us;
    // u < 2^28 and rank < 8: the products fit 32 bits; the split factor is a power of two
    // front_heavy: the odd units go to the first CTAs (rounding up instead of down)
    const unsigned round_up = front_heavy ? static_cast<unsigned>(a.cluster - 1) : 0u;
    const int u0 = static_cast<int>((static_cast<unsigned>(u) * static_cast<unsigned>(rank) + round_up) >> a.cluster_shift);
    const int u1 = static_cast<int>((static_cast<unsigned>(u) * static_cast<unsigned>(rank + 1) + round_up) >> a.cluster_shift);
    s.kc0 = min(u0, uc) * unit;
    s.kc1 = min(min(u1, uc) * unit, ec);
    s.ks0 = slo + (max(u0, uc) - uc) * unit;
    s.ks1 = min(slo + (max(u1, uc) - uc) * unit, shi);
    s.n_cache_tiles = s.kc1 > s.kc0 ? (s.kc1 - s.kc0 + kTileKeys - 1) / kTileKeys : 0;
    const int nst = s.ks1 > s.ks0 ? (s.ks1 - s.ks0 + kTileKeys - 1) / kTileKeys : 0;
    s.n_tiles = s.n_cache_tiles + nst;
    return s;
}

// Row r of the head's query tile: rows [0, T) are the main-stream rows of nodes 0..T-1, rows
// [tmax8, tmax8 + T*gamma) the stream rows in (node, stream) order; everything else is padding.
struct RowInfo {
    bool valid;
    int node, stream;              // stream 0 = main row, 1..gamma = speculative stream
};
__device__ __forceinline__ RowInfo row_info(const Span& s, int row) {
    RowInfo r;
    if (row < s.tmax8) {
        r.valid = row < s.T; r.node = row; r.stream = 0;
    } else {
        const int x = row - s.tmax8;
        r.valid = x < s.n_stream;
        r.node = s.gamma > 0 ? x / s.gamma : 0;
        r.stream = x - r.node * s.gamma + 1;
    }
    return r;
}

// Bit i set <=> key x+i (i < 64) is visible to the row (Eq. 1 / Eq. 2 with the tree mask of App. A).
// `cache`: x indexes the cached slots [0, L+T), else the stream keys; nv = valid keys from x on.
__device__ __forceinline__ unsigned long long visible_mask(bool cache, int x, int nv, int L, int gamma, const RowInfo& r,
                                                            unsigned long long anc) {
    if (!r.valid || nv <= 0) return 0ull;
    const unsigned long long in_tile = nv >= 64 ? ~0ull : ((1ull << nv) - 1ull);
    unsigned long long m;
    if (cache) {
        if (x >= L) {                          // tree keys only: key x+i is node (x - L + i)
            const int sh = x - L;
            m = sh >= 64 ? 0ull : (anc >> sh);
        } else {                               // prefix keys (all visible), then tree keys
            const int np = L - x;
            m = np >= 64 ? ~0ull : (((1ull << np) - 1ull) | (anc << np));
        }
    } else {                                   // stream keys: (node, 1..stream) of the row's own node
        if (r.stream == 0) return 0ull;
        const int lo = r.node * gamma - x, hi = lo + r.stream;        // visible positions [lo, hi)
        const unsigned long long below_hi = hi >= 64 ? ~0ull : (hi <= 0 ? 0ull : ((1ull << hi) - 1ull));
        const unsigned long long below_lo = lo >= 64 ? ~0ull : (lo <= 0 ? 0ull : ((1ull << lo) - 1ull));
        m = below_hi & ~below_lo;
    }
    return m & in_tile;
}

// max over 64 scores of (visible ? s * scale : -inf), four independent chains
template <bool MASKED>
__device__ __forceinline__ float chunk_max(const uint32_t (&v)[64], float scale, unsigned long long vis) {
    const uint32_t vlo = static_cast<uint32_t>(vis), vhi = static_cast<uint32_t>(vis >> 32);
    if (!MASKED) {
        // every score counts: the extreme of the raw scores, scaled once (the minimum if the scale is negative)
        float hi[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (scale >= 0.f) {
            #pragma unroll
            for (int i = 0; i < 64; ++i) hi[i & 3] = fmaxf(hi[i & 3], __uint_as_float(v[i]));
            return fmaxf(fmaxf(hi[0], hi[1]), fmaxf(hi[2], hi[3])) * scale;
        }
        float lo[4] = {INFINITY, INFINITY, INFINITY, INFINITY};
        #pragma unroll
        for (int i = 0; i < 64; ++i) lo[i & 3] = fminf(lo[i & 3], __uint_as_float(v[i]));
        return fminf(fminf(lo[0], lo[1]), fminf(lo[2], lo[3])) * scale;
    }
    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    #pragma unroll
    for (int i = 0; i < 64; ++i) {
        float s = __uint_as_float(v[i]) * scale;
        s = (((i < 32 ? vlo : vhi) >> (i & 31)) & 1u) ? s : -INFINITY;
        mx[i & 3] = fmaxf(mx[i & 3], s);
    }
    return fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
}
// p = exp2(s * scale - m) for 64 scores, packed two bf16 to a word (key 2c in the low half of word c); returns the sum of p
template <bool MASKED>
__device__ __forceinline__ float chunk_exp_pack(const uint32_t (&v)[64], float scale, float m_use, unsigned long long vis,
                                                uint32_t (&pk)[32]) {
    // two scores per instruction (packed fp32 pairs) for the scaling and for the row sum
    const uint32_t vlo = static_cast<uint32_t>(vis), vhi = static_cast<uint32_t>(vis >> 32);
    const unsigned long long scale2 = pack_f32x2(scale, scale), shift2 = pack_f32x2(-m_use, -m_use);
    unsigned long long sum2[2] = {pack_f32x2(0.f, 0.f), pack_f32x2(0.f, 0.f)};
    #pragma unroll
    for (int k = 0; k < 64; k += 2) {
        const unsigned long long t2 = fma_f32x2(pack_f32x2(__uint_as_float(v[k]), __uint_as_float(v[k + 1])), scale2, shift2);
        float t0, t1;
        unpack_f32x2(t2, t0, t1);
        float e0 = exp2f(t0), e1 = exp2f(t1);
        if (MASKED) {
            e0 = (((k < 32 ? vlo : vhi) >> (k & 31)) & 1u) ? e0 : 0.f;
            e1 = (((k < 32 ? vlo : vhi) >> ((k + 1) & 31)) & 1u) ? e1 : 0.f;
        }
        sum2[(k >> 1) & 1] = add_f32x2(sum2[(k >> 1) & 1], pack_f32x2(e0, e1));
        pk[k >> 1] = pack_bf16(e0, e1);
    }
    float s0, s1, s2, s3;
    unpack_f32x2(sum2[0], s0, s1);
    unpack_f32x2(sum2[1], s2, s3);
    return (s0 + s1) + (s2 + s3);
}

// Which kernel a call takes: kCols, heads of at most 64 rows (msa_attention_small_kernel); kPair, blocks of up to
// 128 rows of larger heads (msa_attention_kernel: warpgroup w takes keys 64w .. 64w+63 of every tile, with its own
// running maximum and accumulator; the two partials a row then has inside the CTA are combined before the merge
// across CTAs).
enum Mode { kPair = 0, kCols = 1 };

template <int HD>
struct Geo {
    static constexpr int kHalves = HD > 64 ? 2 : 1;               // 64-element boxes along head_dim
    static constexpr int kBoxBytes = kTileKeys * 128;             // one TMA box: 128 keys x 128 B
    static constexpr int kSlotBytes = kHalves * kBoxBytes;        // one K tile (or one V tile)
    static constexpr int kKSteps = HD / 16;                       // MMA K steps of S = Q K^T
    static constexpr int kMergePitch = HD + 4;                    // floats per partial row: O, m, l, pad
    static constexpr uint32_t kIdescS = idesc_bf16(kTileKeys, false, false);
    static constexpr uint32_t kIdescPV = idesc_bf16(HD, false, true);
    static constexpr int kOCols = 128;                            // TMEM columns reserved per accumulator
    static constexpr int kThreads = kAuxThreads + 2 * kBlockRows; // two softmax warpgroups
    static constexpr int kRowsCap = kBlockRows;                   // partial rows a CTA ships
    static constexpr int kSplitCol = ((HD / 16 + 1) / 2) * 16;    // warpgroup 0 finishes columns [0, kSplitCol)
};

// destination of a row's output and log-sum-exp
struct OutPtr {
    __nv_bfloat16* o;
    float* lse;
};
template <int HD>
__device__ __forceinline__ OutPtr out_ptr(const AttnArgs& a, int b, int h, long long spec_row0, const RowInfo& r) {
    OutPtr p;
    if (r.stream == 0) {
        const long long idx = (static_cast<long long>(b) * a.max_nodes + r.node) * a.n_heads + h;
        p.o = a.o_main + idx * HD;
        p.lse = a.lse_main ? a.lse_main + idx : nullptr;
    } else {
        const long long idx = (spec_row0 + static_cast<long long>(r.node) * a.gamma + (r.stream - 1)) * a.n_heads + h;
        p.o = a.o_spec + idx * HD;
        p.lse = a.lse_spec ? a.lse_spec + idx : nullptr;
    }
    return p;
}

// ---- combining the partial rows of the CTAs that share a block's keys ---------------------------
// A partial row is HD floats of O, then m, l and two floats of padding, relative to the row's reference m
// (in log2 units).  Between calls the workspace's partial-row area is all zero, and a value is never stored
// there as +0 (the writer stores -0 instead): a word that reads non-zero has arrived.  So the rows need no
// flag, no counter and no fence: a reader polls the words it needs (bounded), combines them, and stores zeros
// over what it has read, which leaves the area as the next call expects it.  Rows that no node owns are
// neither written nor read.
__device__ __forceinline__ uint32_t never_plus_zero(uint32_t bits) { return bits == 0u ? 0x80000000u : bits; }
#ifndef SS_ST_KIND
#define SS_ST_KIND "st.relaxed.gpu.global"
#endif
__device__ __forceinline__ void st_relaxed_v4(float* p, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
    asm volatile(SS_ST_KIND ".v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void st_relaxed_v2(float* p, uint32_t x, uint32_t y) {
    asm volatile(SS_ST_KIND ".v2.b32 [%0], {%1, %2};" ::"l"(p), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ uint4 ld_relaxed_v4(const float* p) {
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint2 ld_relaxed_v2(const float* p) {
    uint2 v;
    asm volatile("ld.relaxed.gpu.global.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
    return v;
}

// Step 1: the staged rows (shared memory at y_base, `rows` rows of HD + 4 floats, no +0 among them) go to this
// CTA's rows in the workspace as a few bulk copies (the copy engine moves them faster than the threads' stores
// would -- those reach about 22 B per cycle and SM -- and leaves the load / store path to the polling that
// follows): the rows that nodes own, [0, T) and [tmax8, spec_end) of the head, except those of this CTA's own
// share [first, first + share), which it combines straight from shared memory.  Called by one thread once the
// staged rows are complete (every thread that staged a row has executed fence.proxy.async before the barrier
// that says so); bulk_copies_read() must follow before the shared memory is given up.
__device__ __forceinline__ void bulk_copy_rows(float* dst, uint32_t src, int lo, int hi, uint32_t row_bytes) {
    if (hi <= lo) return;
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst + static_cast<size_t>(lo) * (row_bytes / 4)), "r"(src + static_cast<uint32_t>(lo) * row_bytes),
                   "r"(static_cast<uint32_t>(hi - lo) * row_bytes) : "memory");
}
__device__ __forceinline__ void bulk_copies_read() {
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
template <int HD>
__device__ __forceinline__ void publish_partial_rows(const Span& sp, int row0, int rows, uint32_t y_base, float* part_mine, int first, int share) {
    constexpr uint32_t kRowBytes = (HD + 4) * 4;
    // the two ranges of owned rows, in rows of this block
    const int a0 = 0, a1 = min(max(sp.T - row0, 0), rows);
    const int b0 = max(min(max(sp.tmax8 - row0, 0), rows), a1), b1 = min(max(sp.spec_end - row0, 0), rows);
    const int own0 = first, own1 = first + share;
    // each range minus the own share: the part before it and the part after it
    bulk_copy_rows(part_mine, y_base, a0, min(a1, own0), kRowBytes);
    bulk_copy_rows(part_mine, y_base, max(a0, own1), a1, kRowBytes);
    bulk_copy_rows(part_mine, y_base, b0, min(b1, own0), kRowBytes);
    bulk_copy_rows(part_mine, y_base, max(b0, own1), b1, kRowBytes);
}

// Step 2: this CTA's share of the block's rows, rows [first, first + share): its own partial from shared memory,
// the others' from the workspace (part_group, one CTA's rows `cta_stride` floats after the previous one's).  A
// row's items (four columns each) lie in one warp, so that one lane can clear the row's (m, l) once every lane
// of the warp has read it.  A lane has the loads of BATCH rows x SLOTS sources in flight at once (the more rows
// the fewer sources there are: every pass over a warp's rows costs a round trip to L2).  Returns false when the
// wait ran out (limit in cycles) or another thread of the CTA had given up.
template <int HD, int SLOTS, int BATCH>
__device__ __forceinline__ bool merge_partial_rows_impl(const AttnArgs& a, const Span& sp, int row0, int b, int h, long long spec_row0, int C,
                                                        int rank, uint32_t y_base, const float* part_group, size_t cta_stride, int first,
                                                        int share, int t, int threads, long long limit, volatile int* abort_flag) {
    constexpr int kItems = HD / 4;                                   // items of a row
    constexpr int kLanes = kItems <= 16 ? 16 : 32;                   // lanes a row takes in a warp
    constexpr int kRowsPerWarp = 32 / kLanes;
    constexpr int kPitch = HD + 4;
    const int lane = t & 31, warp_t = t >> 5, n_warps = threads >> 5;
    const int sub = lane / kLanes, g4 = lane - sub * kLanes;
    for (int rbase = warp_t * kRowsPerWarp * BATCH; rbase < share; rbase += n_warps * kRowsPerWarp * BATCH) {     // warp-uniform
        uint4 v[BATCH][SLOTS];
        uint2 ml[BATCH][SLOTS];
        uint32_t pending[BATCH];
        float* src[BATCH];
        RowInfo r[BATCH];
        #pragma unroll
        for (int bi = 0; bi < BATCH; ++bi) {
            const int rr = rbase + bi * kRowsPerWarp + sub;
            r[bi] = row_info(sp, row0 + first + (rr < share ? rr : 0));
            const bool mine = rr < share && g4 < kItems && r[bi].valid;
            r[bi].valid = mine;
            src[bi] = const_cast<float*>(part_group) + static_cast<size_t>(first + (mine ? rr : 0)) * kPitch;
            pending[bi] = mine ? ((1u << C) - 1u) & ~(1u << rank) : 0u;
            if (mine) {
                const uint32_t own = y_base + static_cast<uint32_t>(first + rr) * (kPitch * 4u);
                const float4 ov = ld_shared_v4(own + static_cast<uint32_t>(g4) * 16u);
                const float2 oml = ld_shared_v2(own + HD * 4u);
                #pragma unroll
                for (int sidx = 0; sidx < SLOTS; ++sidx) {
                    if (sidx == rank) {
                        v[bi][sidx] = make_uint4(__float_as_uint(ov.x), __float_as_uint(ov.y), __float_as_uint(ov.z), __float_as_uint(ov.w));
                        ml[bi][sidx] = make_uint2(__float_as_uint(oml.x), __float_as_uint(oml.y));
                    }
                }
            }
        }
        const long long t0 = clock64();
        for (;;) {
            #pragma unroll
            for (int bi = 0; bi < BATCH; ++bi) {
                #pragma unroll
                for (int sidx = 0; sidx < SLOTS; ++sidx) {
                    if ((pending[bi] >> sidx) & 1u) {
                        v[bi][sidx] = ld_relaxed_v4(src[bi] + sidx * cta_stride + g4 * 4);
                        ml[bi][sidx] = ld_relaxed_v2(src[bi] + sidx * cta_stride + HD);
                    }
                }
            }
            uint32_t left = 0u;
            #pragma unroll
            for (int bi = 0; bi < BATCH; ++bi) {
                #pragma unroll
                for (int sidx = 0; sidx < SLOTS; ++sidx)
                    if (((pending[bi] >> sidx) & 1u) && v[bi][sidx].x != 0u && v[bi][sidx].y != 0u && v[bi][sidx].z != 0u && v[bi][sidx].w != 0u &&
                        ml[bi][sidx].x != 0u && ml[bi][sidx].y != 0u)
                        pending[bi] &= ~(1u << sidx);
                left |= pending[bi];
            }
            if (!__any_sync(0xffffffffu, left != 0u)) break;
            if (__any_sync(0xffffffffu, *abort_flag != 0 || clock64() - t0 > limit)) return false;
        }
        #pragma unroll
        for (int bi = 0; bi < BATCH; ++bi) {
            if (!r[bi].valid) continue;
            float mx = -INFINITY;
            #pragma unroll
            for (int sidx = 0; sidx < SLOTS; ++sidx)
                if (sidx < C) mx = fmaxf(mx, __uint_as_float(ml[bi][sidx].x));
            float l = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            #pragma unroll
            for (int sidx = 0; sidx < SLOTS; ++sidx) {
                if (sidx < C) {
                    const float ms = __uint_as_float(ml[bi][sidx].x);
                    const float wgt = ms == -INFINITY ? 0.f : exp2f(ms - mx);       // 0: saw no visible key
                    l += wgt * __uint_as_float(ml[bi][sidx].y);
                    acc.x += wgt * __uint_as_float(v[bi][sidx].x); acc.y += wgt * __uint_as_float(v[bi][sidx].y);
                    acc.z += wgt * __uint_as_float(v[bi][sidx].z); acc.w += wgt * __uint_as_float(v[bi][sidx].w);
                }
            }
            const OutPtr dst = out_ptr<HD>(a, b, h, spec_row0, r[bi]);
            const float inv = 1.f / l;
            uint2 o;
            o.x = pack_bf16(acc.x * inv, acc.y * inv);
            o.y = pack_bf16(acc.z * inv, acc.w * inv);
            *reinterpret_cast<uint2*>(dst.o + g4 * 4) = o;
            if (dst.lse && g4 == 0) *dst.lse = (mx + log2f(l)) * 0.6931471805599453f;
            // what was read goes back to zero: every lane its own columns, one lane the row's (m, l)
            #pragma unroll
            for (int sidx = 0; sidx < SLOTS; ++sidx) {
                if (sidx < C && sidx != rank) {
                    st_relaxed_v4(src[bi] + sidx * cta_stride + g4 * 4, 0u, 0u, 0u, 0u);
                    if (g4 == 0) st_relaxed_v2(src[bi] + sidx * cta_stride + HD, 0u, 0u);
                }
            }
        }
    }
    return true;
}
template <int HD>
__device__ __forceinline__ bool merge_partial_rows(const AttnArgs& a, const Span& sp, int row0, int b, int h, long long spec_row0, int C, int rank,
                                                   uint32_t y_base, const float* part_group, size_t cta_stride, int first, int share, int t,
                                                   int threads, long long limit, volatile int* abort_flag) {
    if (C > 4) return merge_partial_rows_impl<HD, 8, 1>(a, sp, row0, b, h, spec_row0, C, rank, y_base, part_group, cta_stride, first, share, t, threads, limit, abort_flag);
    if (C > 2) return merge_partial_rows_impl<HD, 4, 2>(a, sp, row0, b, h, spec_row0, C, rank, y_base, part_group, cta_stride, first, share, t, threads, limit, abort_flag);
    return merge_partial_rows_impl<HD, 2, 4>(a, sp, row0, b, h, spec_row0, C, rank, y_base, part_group, cta_stride, first, share, t, threads, limit, abort_flag);
}

// 16 fp32 values scaled and packed to bf16 -> 32 bytes at dst
__device__ __forceinline__ void store_bf16x16(__nv_bfloat16* dst, const float (&v)[16]) {
    uint4 lo, hi;
    lo.x = pack_bf16(v[0], v[1]);   lo.y = pack_bf16(v[2], v[3]);   lo.z = pack_bf16(v[4], v[5]);   lo.w = pack_bf16(v[6], v[7]);
    hi.x = pack_bf16(v[8], v[9]);   hi.y = pack_bf16(v[10], v[11]); hi.z = pack_bf16(v[12], v[13]); hi.w = pack_bf16(v[14], v[15]);
    *reinterpret_cast<uint4*>(dst) = lo;
    *reinterpret_cast<uint4*>(dst + 8) = hi;
}

// ---------------------------------------------------------------------------------------------
// The barriers that hand score buffers, P and accumulators around, for either pipeline of msa_attention_kernel.
//   running maximum per warpgroup: s_full[w][b] S of buffer b complete (seen by warpgroup w); p_full[w][b] the
//     warpgroup's half of P written (4 warps); s_free[b] the P V that read the buffer complete; o_done[w][b] the
//     warpgroup's P V of a tile of parity b complete.
//   shared reference (tile j: buffer b = j & 1, warpgroup b): s_full[0][b] S complete; s_free[b] the scores are in
//     registers (4 warps); p_full[0][b] P written (4 warps); o_done[b][(j >> 1) & 1] P V of tile j complete.
__device__ __forceinline__ void init_tile_barriers(Ctrl& c, bool shared_ref) {
    for (int s = 0; s < 2; ++s) {
        mbar_init(smem_u32(&c.s_free[s]), shared_ref ? 4 : 1);
        mbar_init(smem_u32(&c.s_full[0][s]), 1);
        mbar_init(smem_u32(&c.s_full[1][s]), 1);
        mbar_init(smem_u32(&c.p_full[s][0]), 4);
        mbar_init(smem_u32(&c.p_full[s][1]), 4);
        mbar_init(smem_u32(&c.o_done[s][0]), 1);
        mbar_init(smem_u32(&c.o_done[s][1]), 1);
    }
}
__device__ __forceinline__ void mbar_inval(uint32_t bar) {
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

// SHARED: the instantiation for blocks whose keys are not split (it starts on the shared-reference pipeline and holds
// the other one for a block that has to start over); the instantiation for split blocks holds only the other one.
template <int HD, bool SHARED>
__global__ void __launch_bounds__(Geo<HD>::kThreads, 1) msa_attention_kernel(const __grid_constant__ AttnArgs a) {
    using G = Geo<HD>;
    constexpr int TK = kTileKeys;
    extern __shared__ unsigned char smem_raw[];
    __shared__ Ctrl c;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int C = a.cluster;
    const uint32_t rank = blockIdx.x & (C - 1);            // C is a power of two
    const int group = blockIdx.x >> a.cluster_shift;       // (pair, row block): the CTAs that share its keys
    const int rb = group % a.n_blocks;
    const int pair = group / a.n_blocks;
    int b = pair / a.n_heads;                              // the sequence (for a batch: its place in the dispatch order, see below)
    const int h = pair - b * a.n_heads;
    const int nk = a.n_kslots, nv_slots = a.n_vslots;
    volatile int* abort_flag = &c.abort;
    // Row blocks that are not split start on the shared-reference pipeline (see kSharedRefLimit)
    bool shared_ref = SHARED;

    if (tid == 0) SS_TR(0, 0);
#ifdef SS_TRACE
    unsigned int& s_launch = c.trace_launch;
    if (tid == 0) {
        const unsigned long long key = reinterpret_cast<unsigned long long>(a.o_main);
        s_launch = 0;
        for (unsigned int i = 0; i < 8; ++i) {
            const unsigned long long old = atomicCAS(&g_key[i], 0ull, key);
            if (old == 0ull || old == key) { s_launch = i; break; }
        }
        atomicMin(&g_wall[s_launch & 7][0], wall_ns());
        atomicMax(&g_wall[s_launch & 7][2], wall_ns());      // last CTA start
        if (blockIdx.x == 0) { g_wall[s_launch & 7][3] = wall_ns(); g_wall[s_launch & 7][4] = clock64(); }
    }
#endif
    // ---- shared-memory carve-up (1024-byte aligned: swizzle atoms) ----------------------------
    // The query tile always has room for 128 rows; rows past the ones that exist hold whatever shared
    // memory held, which only ever reaches padding rows of S and O.
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    constexpr uint32_t kQHalfBytes = kBlockRows * 128u;
    const uint32_t q_base = base;                                       // [half][128 rows][128 B]
    const uint32_t k_base = q_base + G::kHalves * kQHalfBytes;          // [slot][half][128 keys][128 B]
    const uint32_t v_base = k_base + nk * G::kSlotBytes;                // [slot][half][128 keys][128 B]
    const uint32_t merge_base = base;                                   // aliases everything above, after the main loop

    // ---- prologue ---------------------------------------------------------------------------------
    // Per-sequence scalars (every thread reads them; through L2: under an early launch the SM's L1 may predate
    // the previous kernel's last writes).  Under the caller's promise they are requested first of all, so that
    // their latency passes while the barriers are set up (volatile: the loads stay where they are written).
    int L = 0, T = 0, cap = 0x7fffffff;
    long long slot0 = 0;
    // A batch whose grid takes several waves is dispatched longest sequence first (CTAs start in the order of
    // their index), so that the last wave holds the short ones: place s of the order goes to the sequence with
    // the s-th longest prefix.  Every warp ranks the (at most 32) lengths for itself.
    const bool by_length = a.batch > 1 && a.batch <= 32 && C == 1;
    auto load_scalars = [&]() {
        if (by_length) {
            int len = -1;
            if (lane < a.batch) asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(len) : "l"(a.kv_len + lane) : "memory");
            int longer = 0;                                // sequences that come before this lane's in the order
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
    // Everything up to the dependency wait touches no global memory, so under programmatic dependent
    // launch it overlaps the tail of the previous kernel in the stream.
    if (tid == 0) {                                       // Q / K producer: the barriers its copies complete on
        mbar_init(smem_u32(&c.q_full), 1);
        for (int s = 0; s < kMaxSlots; ++s) mbar_init(smem_u32(&c.k_full[s]), 1);
        c.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&a.tm_qm); tma_prefetch_desc(&a.tm_k);
        if (a.gamma > 0) { tma_prefetch_desc(&a.tm_qs); tma_prefetch_desc(&a.tm_qs1); tma_prefetch_desc(&a.tm_ks); }
    } else if (tid == 96) {                               // V producer
        for (int s = 0; s < kMaxSlots; ++s) mbar_init(smem_u32(&c.v_full[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&a.tm_v);
        if (a.gamma > 0) tma_prefetch_desc(&a.tm_vs);
    } else if (tid == 64) {                               // every other barrier (first used after the CTA-wide sync)
        for (int s = 0; s < kMaxSlots; ++s) { mbar_init(smem_u32(&c.k_empty[s]), 1); mbar_init(smem_u32(&c.v_empty[s]), 1); }
        init_tile_barriers(c, shared_ref);
        for (int s = 0; s < 4; ++s) mbar_init(smem_u32(&c.mref_full[s]), 1);
        for (int s = 0; s < 2; ++s) mbar_init(smem_u32(&c.drain[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid == 0) SS_TR(0, 1);
    // One thread waits for the previous kernel of the stream; the others sleep on the CTA barrier (a
    // whole parked grid polling the dependency slows the kernel it waits for).  Only then may the next
    // kernel be scheduled: every CTA of this grid is resident and past its wait, so CTAs of a later
    // grid can never hold an SM that this grid still needs.
    auto dependency_wait = [&]() {
        if (tid == 0) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        }
        __syncthreads();
    };
    // Without the caller's promise nothing is read before the wait.  With it (prefix_stable: nothing
    // still in flight writes the cached prefix, the lengths or the trees) the lengths are read and the
    // first prefix tiles requested right away, so HBM streams while the previous kernel drains.
    if (!a.prefix_stable) {
        dependency_wait();
        load_scalars();
    }
    const long long spec_row0 = static_cast<long long>(b) * a.max_nodes * a.gamma;   // first stream row of the sequence
    if (tid == 0) SS_TR(0, 2);
    constexpr uint32_t kTmemCols = 512;                   // two accumulators and two S buffers of 128 columns
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&c.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    T = min(max(T, 0), a.max_nodes);
    bool skip = false;                                    // sequence over its slot capacity: nothing read or written
    if (L < 0 || L + T > cap) {
        skip = true;
        L = 0; T = 0;
    }
    if (tid == 0) SS_TR(0, 3);

    const Span sp = make_span(a, L, T, static_cast<int>(rank), rb, kUnit);

    // K tile j / V tile j of the span -> ring slot st (K: thread 0, V: thread 96)
    auto load_k = [&](int j, int st) {
        const uint32_t bar = smem_u32(&c.k_full[st]);
        mbar_expect_tx(bar, G::kSlotBytes);
        const uint32_t dst = k_base + st * G::kSlotBytes;
        const int x = sp.first_key(j);
        #pragma unroll
        for (int hh = 0; hh < G::kHalves; ++hh) {
            if (sp.is_cache(j)) tma_load_3d(dst + hh * G::kBoxBytes, &a.tm_k, hh * 64, h * a.head_coord, static_cast<int>(slot0 + x), bar);
            else tma_load_3d(dst + hh * G::kBoxBytes, &a.tm_ks, hh * 64, h, static_cast<int>(spec_row0 + x), bar);
        }
    };
    auto load_v = [&](int j, int st) {
        const uint32_t bar = smem_u32(&c.v_full[st]);
        mbar_expect_tx(bar, G::kSlotBytes);
        const uint32_t dst = v_base + st * G::kSlotBytes;
        const int x = sp.first_key(j);
        #pragma unroll
        for (int hh = 0; hh < G::kHalves; ++hh) {
            if (sp.is_cache(j)) tma_load_3d(dst + hh * G::kBoxBytes, &a.tm_v, hh * 64, h * a.head_coord, static_cast<int>(slot0 + x), bar);
            else tma_load_3d(dst + hh * G::kBoxBytes, &a.tm_vs, hh * 64, h, static_cast<int>(spec_row0 + x), bar);
        }
    };
    // the producers start before the CTA-wide synchronisation: the first tiles need no hand-back
    const int n_early_k = min(sp.n_tiles, nk), n_early_v = min(sp.n_tiles, nv_slots);
    // before the dependency wait only tiles that lie wholly inside the cached prefix may be requested
    auto prefix_only = [&](int j) { return sp.is_cache(j) && sp.first_key(j) + TK <= sp.L; };
    int n_pre = 0;                                        // early tiles this producer thread has requested
    if (a.prefix_stable) {
        if (tid == 0) {
            while (n_pre < n_early_k && prefix_only(n_pre)) { load_k(n_pre, n_pre); ++n_pre; }
        } else if (tid == 96) {
            while (n_pre < n_early_v && prefix_only(n_pre)) { load_v(n_pre, n_pre); ++n_pre; }
        }
        dependency_wait();
    }
    if (skip && tid == 0) set_status(a.status, SS_ERR_CAPACITY);
    if (tid == 0) {
        // the rest of the first tiles, then the queries of the block
        for (int j = n_pre; j < n_early_k; ++j) load_k(j, j);
        const uint32_t qbar = smem_u32(&c.q_full);
        const bool with_spec = a.gamma > 0 && a.s0rows > 0;
        const uint32_t rows = rb > 0 ? kBlockRows : a.tmax8 + (with_spec ? a.s0rows : 0);
        mbar_expect_tx(qbar, G::kHalves * rows * 128u);
        #pragma unroll
        for (int hh = 0; hh < G::kHalves; ++hh) {
            const uint32_t dst = q_base + hh * kQHalfBytes;
            if (rb > 0) {
                tma_load_3d(dst, &a.tm_qs1, hh * 64, h, static_cast<int>(spec_row0 + rb * kBlockRows - a.tmax8), qbar);
            } else {
                tma_load_3d(dst, &a.tm_qm, hh * 64, h, b * a.max_nodes, qbar);
                if (with_spec) tma_load_3d(dst + a.tmax8 * 128u, &a.tm_qs, hh * 64, h, static_cast<int>(spec_row0), qbar);
            }
        }
    } else if (tid == 96) {
        for (int j = n_pre; j < n_early_v; ++j) load_v(j, j);
    }
    if (tid >= kAuxThreads && tid < kAuxThreads + SS_MAX_NODES) c.anc[tid - kAuxThreads] = __ldcg(&a.trees[b].anc_mask[tid - kAuxThreads]);
    if (tid == 0) SS_TR(0, 5);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = c.tmem_base;
    const uint32_t tmem_s = tmem + 2 * G::kOCols;         // two S buffers of 128 columns
    if (tid == 0) SS_TR(0, 6);

    // per-thread partial of this CTA's key span, kept for the merge (softmax warps only)
    float m_run = -INFINITY, l_run = 0.f;
    int n_own = 0;
    const int wg = (warp - 4) >> 2;                                           // softmax warpgroup 0 / 1
    const int row_in_blk = ((warp & 3) << 5) | lane;                          // TMEM lane of this thread
    const int lrow = row_in_blk;                                              // row of the block this thread works for
    const int chunk = wg;                                                     // 64-key half of a tile this thread handles
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    RowInfo ri;
    ri.valid = false; ri.node = 0; ri.stream = 0;

    // The tile loops of all roles, for either pipeline; early_k / early_v tiles have been requested already.
    // n_requested: what a producer thread has requested in all (for the wait when the CTA starts over).
    int n_requested = 0;
    const uint32_t tmem_s1 = tmem + G::kOCols;            // shared reference: O, two S buffers, two P buffers of 64 columns
    const uint32_t tmem_p1 = tmem_s1 + 2 * TK;
    auto run_tiles = [&](auto mode_tag, const int early_k, const int early_v) {
    constexpr bool kShared = decltype(mode_tag)::value;
    // ============================ warp 0: K producer, warp 3: V producer ==========================
    // Two rings, two threads: a K slot comes back as soon as S is queued, a V slot only after P V, and
    // neither request waits behind the other.
    if (warp == 0) {
        if (lane == 0 && sp.n_tiles > early_k) {
            Ring rk;
            rk.start();
            for (int i = 0; i < early_k; ++i) rk.advance(nk);
            bool ok = true;
            for (int j = early_k; ok && j < sp.n_tiles; ++j) {
                ok = mbar_wait(smem_u32(&c.k_empty[rk.slot]), (rk.round - 1) & 1, abort_flag, a.status);
                SS_TR(0, 8 + 2 * j);
                if (ok) { load_k(j, rk.slot); rk.advance(nk); n_requested = j + 1; }
            }
            // gave up: let the copies already in flight land before shared memory is reused or released
            if (!ok) for (int s = 0; s < nk; ++s) mbar_drain(smem_u32(&c.k_full[s]), (s < rk.slot ? rk.round : rk.round - 1) & 1);
        }
    } else if (warp == 3) {
        if (lane == 0 && sp.n_tiles > early_v) {
            Ring rv;
            rv.start();
            for (int i = 0; i < early_v; ++i) rv.advance(nv_slots);
            bool ok = true;
            for (int j = early_v; ok && j < sp.n_tiles; ++j) {
                ok = mbar_wait(smem_u32(&c.v_empty[rv.slot]), (rv.round - 1) & 1, abort_flag, a.status);
                SS_TR(0, 9 + 2 * j);
                if (ok) { load_v(j, rv.slot); rv.advance(nv_slots); n_requested = j + 1; }
            }
            if (!ok) for (int s = 0; s < nv_slots; ++s) mbar_drain(smem_u32(&c.v_full[s]), (s < rv.slot ? rv.round : rv.round - 1) & 1);
        }
    }
    // ============================ warp 1: issues S = Q K^T, one MMA group per tile ================
    else if (warp == 1) {
        if (lane == 0) {
            // the query tile is always requested, so it is always awaited (shared memory is reused later)
            bool ok = mbar_wait(smem_u32(&c.q_full), 0, abort_flag, a.status);
            if (!ok) mbar_drain(smem_u32(&c.q_full), 0);
            SS_TR(1, 0);
            Ring rk;
            rk.start();
            // A descriptor's low word is (address >> 4): a step inside the tile is an addition to the descriptor
            // (shared memory ends below 2^18, so nothing carries out of the field), and the issuing thread
            // spends its cycles on the MMAs, not on rebuilding descriptors
            const uint64_t dq = desc_k_major(q_base);
            for (int j = 0; ok && j < sp.n_tiles; ++j, rk.advance(nk)) {
                const int buf = j & 1;
                if (!mbar_wait(smem_u32(&c.k_full[rk.slot]), rk.round & 1, abort_flag, a.status)) break;
                SS_TR(1, 8 + 4 * j);
                if (j >= 2 && !mbar_wait(smem_u32(&c.s_free[buf]), ((j >> 1) - 1) & 1, abort_flag, a.status)) break;
                SS_TR(1, 9 + 4 * j);
                tc_fence_after();
                const uint64_t dk = desc_k_major(k_base + rk.slot * G::kSlotBytes);
                const uint32_t sd = (kShared ? tmem_s1 : tmem_s) + buf * TK;
                #pragma unroll
                for (int ks = 0; ks < G::kKSteps; ++ks) {
                    const uint32_t hh = ks >> 2, off = (ks & 3) * 32u;
                    tc_mma(sd, dq + ((hh * kQHalfBytes + off) >> 4), dk + ((hh * G::kBoxBytes + off) >> 4), G::kIdescS, ks > 0);
                }
                SS_TR(1, 10 + 4 * j);
                tc_commit(smem_u32(&c.s_full[0][buf]));
                if (!kShared) tc_commit(smem_u32(&c.s_full[1][buf]));
                tc_commit(smem_u32(&c.k_empty[rk.slot]));                // S of tile j is queued: K may go
                SS_TR(1, 11 + 4 * j);
            }
        }
    }
    // ============================ warp 2: issues O += P V ==========================================
    else if (warp == 2) {
        if (lane == 0) {
            Ring rv;
            rv.start();
            bool ok = true;
            for (int j = 0; ok && j < sp.n_tiles; ++j, rv.advance(nv_slots)) {
                if (!mbar_wait(smem_u32(&c.v_full[rv.slot]), rv.round & 1, abort_flag, a.status)) break;
                SS_TR(2, 8 + 4 * j);
                const uint32_t va = v_base + rv.slot * G::kSlotBytes;
                if constexpr (kShared) {
                    // the tile's 128 keys into the one accumulator; P is read from its own TMEM buffer
                    const int buf = j & 1;
                    const uint64_t dv = desc_mn_major(va, G::kBoxBytes);
                    if (!mbar_wait(smem_u32(&c.p_full[0][buf]), (j >> 1) & 1, abort_flag, a.status)) break;
                    SS_TR(2, 9 + 4 * j);
                    tc_fence_after();
                    const uint32_t pa = tmem_p1 + buf * (TK / 2);
                    #pragma unroll
                    for (int ks = 0; ks < TK / 16; ++ks)
                        tc_mma_ts(tmem, pa + ks * 8u, dv + ((ks * 2048u) >> 4), G::kIdescPV, (j > 0 || ks > 0) ? 1u : 0u);
                    tc_commit(smem_u32(&c.o_done[buf][(j >> 1) & 1]));   // P of the buffer may be overwritten
                } else {
                    // keys 64w .. 64w+63 into the accumulator of warpgroup w; P is read from TMEM, where the
                    // warpgroup left it over the first 32 columns of its half of the S buffer
                    const int buf = j & 1;
                    const uint64_t dv = desc_mn_major(va, G::kBoxBytes);
                    #pragma unroll
                    for (int w = 0; w < 2; ++w) {
                        if (!mbar_wait(smem_u32(&c.p_full[w][buf]), (j >> 1) & 1, abort_flag, a.status)) { ok = false; break; }
                        if (w == 0) SS_TR(2, 9 + 4 * j);
                        tc_fence_after();
                        const uint32_t pa = tmem_s + buf * TK + w * 64;
                        #pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            tc_mma_ts(tmem + w * G::kOCols, pa + ks * 8u, dv + (((w * 4 + ks) * 2048u) >> 4), G::kIdescPV, (j > 0 || ks > 0) ? 1u : 0u);
                        tc_commit(smem_u32(&c.o_done[w][buf]));
                    }
                    if (!ok) break;
                    tc_commit(smem_u32(&c.s_free[buf]));                 // both halves of P have been read: S may be overwritten
                }
                SS_TR(2, 10 + 4 * j);
                tc_commit(smem_u32(&c.v_empty[rv.slot]));                // P V of tile j is queued: V may go when it completes
                SS_TR(2, 11 + 4 * j);
            }
        }
    }
    // ============================ warps 4..11: softmax warpgroups ==============================
    else if (warp >= 4) {
        ri = row_info(sp, sp.row0 + lrow);
        const unsigned long long anc = ri.valid ? c.anc[ri.node] : 0ull;
        // a warp whose 32 rows are all padding skips the arithmetic but keeps the barrier protocol
        const bool warp_active = __any_sync(0xffffffffu, ri.valid);
        Ring rv;                                       // V ring position of tile j
        rv.start();
        int v_tile = 0;
        // V rows past the end of the sequence's keys may hold anything (even NaN patterns): P is 0 there, but
        // 0 * NaN is NaN, so the rows [lo, hi) of tile j that lie past the end are cleared before P V reads them.
        // Rows that only lie past this CTA's share of the keys are real data.  (false: a wait gave up)
        auto clear_v_tail = [&](int j, int lo, int hi) {
            const int region_left = (sp.is_cache(j) ? sp.L + sp.T : sp.n_stream) - sp.first_key(j);      // real rows in the tile
            const int fix_lo = max(region_left, lo), fix_hi = hi;
            if (fix_lo >= fix_hi) return true;
            if (!mbar_wait_warp(smem_u32(&c.v_full[rv.slot]), rv.round & 1, abort_flag, a.status)) return false;
            const uint32_t vdst = v_base + rv.slot * G::kSlotBytes;
            constexpr int kPieceShift = G::kHalves == 2 ? 4 : 3;                  // 16-byte pieces per row: 8 per half
            const int n_pieces = (fix_hi - fix_lo) << kPieceShift;
            for (int i = row_in_blk; i < n_pieces; i += kBlockRows) {
                const int r = fix_lo + (i >> kPieceShift), pc = i & ((1 << kPieceShift) - 1);
                const uint32_t dst = vdst + (pc >> 3) * G::kBoxBytes + r * 128u + ((pc & 7) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0u) : "memory");
            }
            return true;
        };
        if constexpr (kShared) {
            // ---- shared reference: the warpgroups take alternate tiles (warpgroup w: tiles w, w + 2, ..., all 128
            // keys, one thread per row) from their own score buffer into their own P buffer; one accumulator.
            // A score buffer goes back to the S issuer as soon as its scores are in registers, so the only
            // thing a warpgroup ever waits for is its next scores.
            const uint32_t s_addr = tmem_s1 + lane_base + wg * TK, p_addr = tmem_p1 + lane_base + wg * (TK / 2);
            const int quad = warp & 3;
            bool ok = true;
            if (wg == 1 && sp.n_tiles > 0) {
                // the reference comes from warpgroup 0's first tile
                ok = mbar_wait_warp(smem_u32(&c.mref_full[quad]), 0, abort_flag, a.status);
                if (ok) m_run = c.m_ref[row_in_blk];
            }
            for (int j = wg; ok && j < sp.n_tiles; j += 2) {
                while (v_tile < j) { rv.advance(nv_slots); ++v_tile; }
                if (!mbar_wait_warp(smem_u32(&c.s_full[0][wg]), n_own & 1, abort_flag, a.status)) break;
                [[maybe_unused]] const int trole = 3 + wg;
                [[maybe_unused]] const bool tr_on = row_in_blk == 0;
                if (tr_on) SS_TR(trole, 8 + 6 * n_own);
                tc_fence_after();
                const int x = sp.first_key(j), nvk = sp.valid_keys(j);
                const bool cache = sp.is_cache(j);
                const bool masked = !cache || x + TK > sp.L || nvk < TK;
                const unsigned long long vis0 = masked ? visible_mask(cache, x, nvk, sp.L, sp.gamma, ri, anc) : ~0ull;
                const unsigned long long vis1 = masked ? visible_mask(cache, x + 64, nvk - 64, sp.L, sp.gamma, ri, anc) : ~0ull;
                bool bad = false;
                if (warp_active) {
                    uint32_t sr[64], pk[32];
                    if (j == 0) {
                        // the row maximum of the first tile is the reference of the row for the whole CTA
                        tmem_ld64(s_addr + 64, sr);
                        tmem_wait_ld();
                        float mx = masked ? chunk_max<true>(sr, a.scale_log2, vis1) : chunk_max<false>(sr, a.scale_log2, 0ull);
                        tmem_ld64(s_addr, sr);
                        tmem_wait_ld();
                        mx = fmaxf(mx, masked ? chunk_max<true>(sr, a.scale_log2, vis0) : chunk_max<false>(sr, a.scale_log2, 0ull));
                        m_run = mx;
                        c.m_ref[row_in_blk] = mx;
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&c.mref_full[quad]));   // (release: the lanes' references are written)
                        bad = ri.valid && !(mx > -INFINITY && mx < INFINITY);     // a row that sees no key here, or a NaN
                    } else {
                        tmem_ld64(s_addr, sr);
                        tmem_wait_ld();
                    }
                    if (tr_on) SS_TR(trole, 9 + 6 * n_own);
                    const float m_use = (m_run > -INFINITY && m_run < INFINITY) ? m_run : 0.f;
                    float sum = masked ? chunk_exp_pack<true>(sr, a.scale_log2, m_use, vis0, pk) : chunk_exp_pack<false>(sr, a.scale_log2, m_use, 0ull, pk);
                    // the P buffer is free once the P V of the warpgroup's previous tile has completed
                    if (n_own > 0 && !mbar_wait_warp(smem_u32(&c.o_done[wg][(n_own - 1) & 1]), ((n_own - 1) >> 1) & 1, abort_flag, a.status)) break;
                    tc_fence_after();
                    tmem_st32(p_addr, pk);
                    tmem_ld64(s_addr + 64, sr);
                    tmem_wait_ld();
                    // the scores are in registers: the S issuer may overwrite the buffer
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&c.s_free[wg]));
                    if (tr_on) SS_TR(trole, 10 + 6 * n_own);
                    sum += masked ? chunk_exp_pack<true>(sr, a.scale_log2, m_use, vis1, pk) : chunk_exp_pack<false>(sr, a.scale_log2, m_use, 0ull, pk);
                    tmem_st32(p_addr + 32, pk);
                    tmem_wait_st();
                    l_run += sum;
                    bad = bad || (ri.valid && !(sum <= kSharedRefLimit));
                } else {
                    // (a warp without rows keeps the protocol, this wait included: it must see every phase of
                    // the barrier, or the wait after the loop could take an earlier phase for the last)
                    if (n_own > 0 && !mbar_wait_warp(smem_u32(&c.o_done[wg][(n_own - 1) & 1]), ((n_own - 1) >> 1) & 1, abort_flag, a.status)) break;
                    if (lane == 0) {
                        mbar_arrive(smem_u32(&c.s_free[wg]));
                        if (j == 0) mbar_arrive(smem_u32(&c.mref_full[quad]));
                    }
                }
                if (__any_sync(0xffffffffu, bad)) {
                    // the reference does not hold for some row: every role leaves its loop and the CTA starts over
                    if (lane == 0) atomicCAS(&c.abort, 0, 2);
                    break;
                }
                if (tr_on) SS_TR(trole, 11 + 6 * n_own);
                if (!clear_v_tail(j, 0, TK)) break;
                fence_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&c.p_full[0][wg]));
                if (tr_on) SS_TR(trole, 13 + 6 * n_own);
                ++n_own;
            }
            // The CTA's last P V must have landed before the accumulator is read and before shared memory is reused
            // (commits complete in order, so the last stands for all).  Its barrier has completed every earlier
            // phase by now: this warpgroup's last P store came after the P V four tiles before the CTA's last.
            if (sp.n_tiles > 0) {
                const int jl = sp.n_tiles - 1;
                mbar_wait_warp(smem_u32(&c.o_done[jl & 1][(jl >> 1) & 1]), (jl >> 2) & 1, abort_flag, a.status);
                tc_fence_after();
            }
        } else {
        const uint32_t o_addr = tmem + lane_base + wg * G::kOCols;
        for (int j = 0; j < sp.n_tiles; ++j) {
            while (v_tile < j) { rv.advance(nv_slots); ++v_tile; }
            const int buf = j & 1;
            // uses of (warpgroup, buffer) so far: j >> 1
            if (!mbar_wait_warp(smem_u32(&c.s_full[wg][buf]), (j >> 1) & 1, abort_flag, a.status)) break;
            [[maybe_unused]] const int trole = 3 + wg;
            [[maybe_unused]] const bool tr_on = row_in_blk == 0;
            if (tr_on) SS_TR(trole, 8 + 6 * n_own);
            tc_fence_after();
            const uint32_t s_addr = tmem_s + lane_base + buf * TK + chunk * 64;
            const int x = sp.first_key(j), nvk = sp.valid_keys(j);
            const bool cache = sp.is_cache(j);
            const bool masked = !cache || x + TK > sp.L || nvk < TK;
            const unsigned long long vis = masked ? visible_mask(cache, x + chunk * 64, nvk - chunk * 64, sp.L, sp.gamma, ri, anc) : ~0ull;

            uint32_t sr[64];
            float corr = 1.f;
            bool need = false;
            // ---- pass 1: the maximum of this thread's 64 scores ----------------------------------------
            if (warp_active) {
                tmem_ld64(s_addr, sr);
                tmem_wait_ld();
                const float mx = masked ? chunk_max<true>(sr, a.scale_log2, vis) : chunk_max<false>(sr, a.scale_log2, 0ull);
                need = mx > m_run + kRescaleStep;
                if (need) {
                    corr = exp2f(m_run - mx);           // 0 when nothing was visible so far
                    m_run = mx;
                    l_run *= corr;
                }
            }
            if (tr_on) SS_TR(trole, 9 + 6 * n_own);
            const bool rescale = n_own > 0 && __any_sync(0xffffffffu, need);
            if (rescale) {
                // P goes to the S buffer itself (handed back by the P V that reads it), so only a raised
                // maximum waits for the previous P V: it rescales the accumulator that P V wrote
                // (S of this tile exists, so the P V two tiles back is complete: the barrier is at most one phase behind)
                if (!mbar_wait_warp(smem_u32(&c.o_done[wg][(j - 1) & 1]), ((j - 1) >> 1) & 1, abort_flag, a.status)) break;
                tc_fence_after();
            }
            if (tr_on) SS_TR(trole, 10 + 6 * n_own);
            if (warp_active) {
                if (rescale) {
                    #pragma unroll
                    for (int c0 = 0; c0 < HD; c0 += 16) {
                        uint32_t orr[16];
                        tmem_ld16<0>(o_addr + c0, orr);
                        tmem_wait_ld();
                        #pragma unroll
                        for (int i = 0; i < 16; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * corr);
                        tmem_st16<0>(o_addr + c0, orr);
                    }
                    tmem_wait_st();
                }
                // ---- pass 2: P = exp2(S - m) as bf16, row sum -------------------------------------------
                const float m_use = (m_run == -INFINITY) ? 0.f : m_run;
                // two bf16 to a column, over the first 32 of the 64 score columns this thread has read
                uint32_t pk[32];
                l_run += masked ? chunk_exp_pack<true>(sr, a.scale_log2, m_use, vis, pk) : chunk_exp_pack<false>(sr, a.scale_log2, m_use, 0ull, pk);
                tmem_st32(s_addr, pk);
                tmem_wait_st();
            }
            if (tr_on) SS_TR(trole, 11 + 6 * n_own);
            // the warpgroup clears the V rows past the end that its P V reads (its half of the tile)
            if (!clear_v_tail(j, wg * 64, wg * 64 + 64)) break;
            if (tr_on) SS_TR(trole, 12 + 6 * n_own);
            fence_async_smem();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&c.p_full[wg][buf]));
            if (tr_on) SS_TR(trole, 13 + 6 * n_own);
            ++n_own;
        }
        // the warpgroup's last PV must have landed in TMEM before the accumulator is read
        if (n_own > 0) {
            // the last two P V may both be outstanding: one barrier each
            if (n_own > 1) mbar_wait_warp(smem_u32(&c.o_done[wg][(n_own - 2) & 1]), ((n_own - 2) >> 1) & 1, abort_flag, a.status);
            mbar_wait_warp(smem_u32(&c.o_done[wg][(n_own - 1) & 1]), ((n_own - 1) >> 1) & 1, abort_flag, a.status);
            tc_fence_after();
        }
        }   // running maximum per warpgroup
    }
    };  // run_tiles
    if (tid == 0) n_requested = n_early_k; else if (tid == 96) n_requested = n_early_v;
    if constexpr (SHARED) {
        run_tiles(std::true_type{}, n_early_k, n_early_v);
        __syncwarp();
        tc_fence_before();
        __syncthreads();                                  // every role has left its loop
        tc_fence_after();
        if (c.abort == 2) {
            // The shared reference did not hold for some row.  What is in flight lands first: the producers wait
            // for the last copy they requested into every slot, the MMA issuers for their last MMA; then the
            // barriers are set up anew (all but the query tile's) and the tiles run again from the first.
            if (tid == 0 || tid == 96) {
                const int slots = tid == 0 ? nk : nv_slots;
                unsigned long long* const full = tid == 0 ? c.k_full : c.v_full;
                for (int sl = 0; sl < slots; ++sl)
                    if (n_requested > sl) mbar_drain(smem_u32(&full[sl]), ((n_requested - 1 - sl) / slots) & 1);
                if (tid == 0) mbar_drain(smem_u32(&c.q_full), 0);
            } else if (tid == 32 || tid == 64) {
                const uint32_t bar = smem_u32(&c.drain[tid == 64 ? 1 : 0]);
                tc_commit(bar);
                mbar_drain(bar, 0);
            }
            __syncwarp();
            if (warp >= 4) { tmem_wait_ld(); tmem_wait_st(); }
            tc_fence_before();
            __syncthreads();
            tc_fence_after();
            if (tid == 0) {
                for (int sl = 0; sl < kMaxSlots; ++sl) {
                    unsigned long long* const ring[4] = {&c.k_full[sl], &c.k_empty[sl], &c.v_full[sl], &c.v_empty[sl]};
                    for (int i = 0; i < 4; ++i) { mbar_inval(smem_u32(ring[i])); mbar_init(smem_u32(ring[i]), 1); }
                }
                for (int i = 0; i < 2; ++i) {
                    mbar_inval(smem_u32(&c.s_free[i]));
                    for (int k = 0; k < 2; ++k) {
                        mbar_inval(smem_u32(&c.s_full[i][k])); mbar_inval(smem_u32(&c.p_full[i][k])); mbar_inval(smem_u32(&c.o_done[i][k]));
                    }
                }
                init_tile_barriers(c, false);
                c.abort = 0;
                atomicAdd(a.status + 2, 1);               // diagnostics: blocks that started over
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            }
            shared_ref = false;
            m_run = -INFINITY; l_run = 0.f; n_own = 0; n_requested = 0;
            __syncthreads();
            run_tiles(std::false_type{}, 0, 0);
        }
    } else {
        run_tiles(std::false_type{}, n_early_k, n_early_v);
    }
    if (tid == kAuxThreads) SS_TR(5, 0);
    __syncwarp();     // the single-lane roles of warps 0..3 rejoin their warps

    // ======================================== epilogue ==========================================
    // The softmax warpgroups combine the partials a row has inside the CTA.  Not split (C == 1): that
    // is the result.  Split: every CTA leaves one un-normalised partial row (O, m, l) per query row in
    // the workspace (it stays in L2) and combines its own share of the rows as they arrive from all CTAs.
    // (shared reference: one accumulator, which both threads of a lane read; the reference is the row's m for both)
    const bool has_acc = (warp >= 4) && (shared_ref ? sp.n_tiles > 0 : n_own > 0);     // otherwise the partial is (m = -inf, l = 0, O = 0)
    const uint32_t o_addr = tmem + lane_base + ((warp >= 4 && !shared_ref) ? wg : 0) * G::kOCols;
    constexpr int RP = G::kMergePitch;                                         // floats per partial row: O, m, l, pad
    constexpr uint32_t RB = RP * 4;                                            // bytes of a partial row
    constexpr int rows_cap = G::kRowsCap;                                      // partial rows per CTA
    constexpr int wg_threads = 2 * kBlockRows;
    float* const part_group = a.partials + static_cast<size_t>(group) * C * rows_cap * RP;
    float* const part_mine = part_group + static_cast<size_t>(rank) * rows_cap * RP;

    // Shared memory after the main loop: 2 KB in which the warpgroups exchange their (m, l) (the first thing
    // a finished warpgroup writes: it has seen the last S land, so the query tile under merge_base is free);
    // then Y, the outgoing partial rows of this CTA as they lie in the workspace.
    const uint32_t ml_base = merge_base;                                       // [warpgroup][128 lanes] (m, l)
    const uint32_t y_base = merge_base + 2048u;                                // [rows_cap][RP floats]
    if (warp >= 4) {
        // What is written below (except the (m, l)) overlaps the query tile and the K/V slots: the query copy
        // must have landed and every MMA of the CTA must be complete (each warpgroup has seen its last P V land).
        mbar_wait_warp(smem_u32(&c.q_full), 0, abort_flag, a.status);
        const bool any_valid = __any_sync(0xffffffffu, ri.valid);
        // Both accumulators of a TMEM lane can be read by either of the lane's two threads (one per
        // warpgroup).  The two exchange (m, l) through shared memory; then warpgroup 0 combines columns
        // [0, kSplitCol) of the lane's two partials and warpgroup 1 the rest.
        asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(ml_base + static_cast<uint32_t>(wg * kBlockRows + row_in_blk) * 8u),
                     "f"(m_run), "f"(l_run) : "memory");
        tc_fence_before();
        named_barrier(2, wg_threads);
        tc_fence_after();
        if (tid == kAuxThreads) SS_TR(5, 1);
        const float2 other = ld_shared_v2(ml_base + static_cast<uint32_t>((wg ^ 1) * kBlockRows + row_in_blk) * 8u);
        float m_out = fmaxf(m_run, other.x);
        const float w_me = m_run != -INFINITY ? exp2f(m_run - m_out) : 0.f;      // 0: saw no visible key
        const float w_ot = other.x != -INFINITY ? exp2f(other.x - m_out) : 0.f;
        float l_out = w_me * l_run + w_ot * other.y;
        // an accumulator that no MMA has written holds anything: it is not read
        const bool has_ot = has_acc && !shared_ref;
        const uint32_t o_other = tmem + lane_base + (wg ^ 1) * G::kOCols;
        const int c_lo = wg == 0 ? 0 : G::kSplitCol, c_hi = wg == 0 ? G::kSplitCol : HD;
        float v[G::kSplitCol];                                                   // this thread's columns of the lane's combined partial
        #pragma unroll
        for (int cc = 0; cc < G::kSplitCol; cc += 16) {
            const int c0 = c_lo + cc;
            uint32_t mine[16], theirs[16];
            #pragma unroll
            for (int i = 0; i < 16; ++i) { mine[i] = 0u; theirs[i] = 0u; }
            if (any_valid && c0 < c_hi) {                                        // warp-uniform
                if (has_acc) tmem_ld16<0>(o_addr + c0, mine);
                if (has_ot) tmem_ld16<0>(o_other + c0, theirs);
                tmem_wait_ld();
            }
            #pragma unroll
            for (int i = 0; i < 16; ++i) v[cc + i] = w_me * __uint_as_float(mine[i]) + w_ot * __uint_as_float(theirs[i]);
        }
        // the thread now holds its columns of the row's partial over all keys of this CTA
        {
            if (C == 1) {
                if (ri.valid && !skip) {
                    const OutPtr dst = out_ptr<HD>(a, b, h, spec_row0, ri);
                    const float inv = 1.f / l_out;
                    #pragma unroll
                    for (int cc = 0; cc < G::kSplitCol; cc += 16) {
                        if (c_lo + cc < c_hi) {
                            float o[16];
                            #pragma unroll
                            for (int i = 0; i < 16; ++i) o[i] = v[cc + i] * inv;
                            store_bf16x16(dst.o + c_lo + cc, o);
                        }
                    }
                    if (dst.lse && wg == 0) *dst.lse = (m_out + log2f(l_out)) * 0.6931471805599453f;
                }
            } else {
                // (never +0: a word of a partial row that reads zero in the workspace has not arrived)
                const uint32_t yrow = y_base + static_cast<uint32_t>(lrow) * RB;
                #pragma unroll
                for (int cc = 0; cc < G::kSplitCol; cc += 4)
                    if (c_lo + cc < c_hi)
                        st_shared_v4(yrow + (c_lo + cc) * 4u, never_plus_zero(__float_as_uint(v[cc])), never_plus_zero(__float_as_uint(v[cc + 1])),
                                     never_plus_zero(__float_as_uint(v[cc + 2])), never_plus_zero(__float_as_uint(v[cc + 3])));
                if (wg == 0) st_shared_v4(yrow + HD * 4u, never_plus_zero(__float_as_uint(m_out)), never_plus_zero(__float_as_uint(l_out)), 0u, 0u);
                fence_async_smem();                       // the copy engine reads these rows
            }
        }
        if (tid == kAuxThreads) SS_TR(5, 3);
    }

    if (C > 1 && warp >= 4) {
        // The partial rows wait in Y.  The other CTAs of the block were launched with this one and need nothing
        // from it, so the (bounded) wait for their rows is short.
        named_barrier(3, wg_threads);                                 // Y is complete
        const int t = tid - kAuxThreads;
        const bool live = __all_sync(0xffffffffu, !skip && *abort_flag == 0);
        const int share = rows_cap >> a.cluster_shift, first = static_cast<int>(rank) * share;
        if (live && t == 0) publish_partial_rows<HD>(sp, sp.row0, rows_cap, y_base, part_mine, first, share);
        if (tid == kAuxThreads) SS_TR(5, 4);
        if (live && !merge_partial_rows<HD>(a, sp, sp.row0, b, h, spec_row0, C, static_cast<int>(rank), y_base, part_group,
                                            static_cast<size_t>(rows_cap) * RP, first, share, t, wg_threads, kWaitCycles, abort_flag)) {
            c.abort = 1;
            set_status(a.status, SS_ERR_DEVICE_TIMEOUT);
        }
        if (live && t == 0) bulk_copies_read();
    }
    if (tid == kAuxThreads) SS_TR(5, 5);

#ifdef SS_TRACE
    if (tid == 0) atomicMax(&g_wall[s_launch & 7][1], wall_ns());
    if (tid == 0) atomicMin(&g_wall[s_launch & 7][5], wall_ns());      // first CTA end
    if (tid == 0 && blockIdx.x == 0) { g_wall[s_launch & 7][3] = wall_ns() - g_wall[s_launch & 7][3]; g_wall[s_launch & 7][4] = clock64() - g_wall[s_launch & 7][4]; }
#endif
    // ---- release TMEM ---------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace ss

#include "ss_attention_small.cuh"

namespace ss {

// ---------------------------------------------------------------------------------------------
// host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 tensor (d, n1, n2) with element strides (1, s1, s2); box (64, 1, box_rows); swizzle 128 B
static bool make_map(CUtensorMap* out, const void* basep, int d, long long n1, long long s1, long long n2, long long s2,
                     int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(n1), static_cast<cuuint64_t>(n2)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(s1) * 2u, static_cast<cuuint64_t>(s2) * 2u};
    cuuint32_t box[3] = {64u, 1u, static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(basep), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct AttnPlan {
    int tmax8, spec_rows, s0rows, n_blocks, mode, n_kslots, n_vslots, cluster;
    long long groups;                          // (sequence, head, row block) triples
    size_t smem;
    size_t partial_bytes;                      // workspace after its header
};

static bool make_plan(const ss_attn_params& p, AttnPlan* plan) {
    if (p.batch < 1 || p.n_heads < 1 || p.max_nodes < 1 || p.gamma < 0) return false;
    if (p.head_dim != 64 && p.head_dim != 80 && p.head_dim != 128) return false;
    if (p.max_nodes > SS_MAX_NODES || p.gamma > SS_MAX_GAMMA) return false;
    const int halves = p.head_dim > 64 ? 2 : 1;
    plan->tmax8 = (p.max_nodes + 7) / 8 * 8;
    plan->spec_rows = p.gamma > 0 ? (p.max_nodes * p.gamma + 7) / 8 * 8 : 0;
    const int q_rows = plan->tmax8 + plan->spec_rows;
    plan->mode = q_rows <= kSmRows ? kCols : kPair;
    plan->n_blocks = plan->mode != kPair ? 1 : (q_rows + kBlockRows - 1) / kBlockRows;
    // stream rows that share block 0 with the main rows
    plan->s0rows = plan->spec_rows < kBlockRows - plan->tmax8 ? plan->spec_rows : kBlockRows - plan->tmax8;
    // CTAs per (sequence, head, row block): the largest power of two that still fits the grid on the SMs in one wave
    plan->groups = static_cast<long long>(p.batch) * p.n_heads * plan->n_blocks;
    int c = 1;
    while (c < 8 && plan->groups * (c * 2) <= sm_count()) c *= 2;
    plan->cluster = c;
    if (plan->mode == kCols) {
        // the query tile (its 64 rows twice), then the K and V rings (at the end they stage 64 partial rows)
        const size_t q_bytes = static_cast<size_t>(halves) * 2 * kSmRows * 128, slot = static_cast<size_t>(halves) * kTileKeys * 128;
        int slots = static_cast<int>((kSmDynSmem - q_bytes) / slot);
        if (slots > kSmMaxSlots) slots = kSmMaxSlots;
        slots &= ~1;                                          // a K ring and a V ring of the same depth
        if (slots < 4) return false;
        plan->n_kslots = slots;
        plan->n_vslots = 0;
        plan->smem = q_bytes + static_cast<size_t>(slots) * slot;
        // a split head leaves the partial rows (O, m, l) of each of its CTAs in the workspace
        plan->partial_bytes = c > 1 ? static_cast<size_t>(plan->groups) * c * kSmRows * (p.head_dim + 4) * 4 : 0;
        return true;
    }
    // row blocks: the query tile, then the K ring and the V ring (P lives in TMEM)
    const size_t qp = static_cast<size_t>(halves) * kBlockRows * 128;
    const size_t slot = static_cast<size_t>(halves) * kTileKeys * 128;
    int slots = static_cast<int>((kPairMaxDynSmem - 1024 - qp) / slot);
    if (slots > 2 * kMaxSlots) slots = 2 * kMaxSlots;
    if (slots < 4) return false;
    // a K slot is held until S is queued, a V slot until P V has completed: the odd slot goes to V
    plan->n_kslots = slots / 2;
    plan->n_vslots = slots - plan->n_kslots > kMaxSlots ? kMaxSlots : slots - plan->n_kslots;
    size_t bytes = qp + static_cast<size_t>(plan->n_kslots + plan->n_vslots) * slot;
    // after the pipeline the same memory stages partial rows ((head_dim + 4) floats each): 2 KB, then the 128
    // outgoing rows
    const size_t row_bytes = static_cast<size_t>(p.head_dim + 4) * 4;
    const size_t stage = 2048 + kBlockRows * row_bytes;
    if (stage > bytes) bytes = stage;
    plan->smem = bytes + 1024;
    // workspace: one partial row per (group, CTA of the group, row)
    plan->partial_bytes = c > 1 ? static_cast<size_t>(plan->groups) * c * kBlockRows * row_bytes : 0;
    return plan->smem <= static_cast<size_t>(kPairMaxDynSmem);
}

template <int HD>
static int32_t launch(const AttnArgs& args, const AttnPlan& plan, cudaStream_t stream) {
    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SS_ERR_CUDA;
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(msa_attention_kernel<HD, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairMaxDynSmem) !=
                cudaSuccess ||
            cudaFuncSetAttribute(msa_attention_kernel<HD, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairMaxDynSmem) !=
                cudaSuccess)
            return SS_ERR_CUDA;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(plan.groups * plan.cluster), 1, 1);
    cfg.blockDim = dim3(static_cast<unsigned>(Geo<HD>::kThreads), 1, 1);
    // always more than half of an SM's shared memory: one CTA per SM, so a CTA never queues for TMEM
    cfg.dynamicSmemBytes = plan.smem < 120 * 1024 ? 120 * 1024 : plan.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    // programmatic dependent launch: the CTAs may be scheduled while the previous kernel of the stream
    // drains; the kernel touches global memory only after its griddepcontrol.wait, so stream order holds
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t err = plan.cluster == 1 ? cudaLaunchKernelEx(&cfg, msa_attention_kernel<HD, true>, args)
                                              : cudaLaunchKernelEx(&cfg, msa_attention_kernel<HD, false>, args);
    return err == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}

template <int HD>
static int32_t launch_cols(const AttnArgs& args, const AttnPlan& plan, cudaStream_t stream) {
    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SS_ERR_CUDA;
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(msa_attention_small_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmDynSmem) != cudaSuccess ||
            cudaFuncSetAttribute(msa_attention_small_kernel<HD>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared) != cudaSuccess)
            return SS_ERR_CUDA;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(plan.groups * plan.cluster), 1, 1);
    cfg.blockDim = dim3(static_cast<unsigned>(kSmThreads), 1, 1);
    cfg.dynamicSmemBytes = plan.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, msa_attention_small_kernel<HD>, args) == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}

}  // namespace ss

extern "C" size_t ss_msa_attention_workspace_bytes(const ss_attn_params* p) {
    ss::AttnPlan plan;
    if (p == nullptr || !ss::make_plan(*p, &plan)) return 0;
    return ss::kWsHeaderBytes + plan.partial_bytes;
}

extern "C" int32_t ss_msa_attention(const ss_attn_params* p, void* stream) {
    if (p == nullptr) return SS_ERR_INVALID_ARG;
    if (p->batch < 1 || p->n_heads < 1 || p->max_nodes < 1 || p->gamma < 0) return SS_ERR_INVALID_ARG;
    if (p->head_dim != 64 && p->head_dim != 80 && p->head_dim != 128) return SS_ERR_UNSUPPORTED;
    if (p->max_nodes > SS_MAX_NODES || p->gamma > SS_MAX_GAMMA) return SS_ERR_UNSUPPORTED;
    ss::AttnPlan plan;
    if (!ss::make_plan(*p, &plan)) return SS_ERR_UNSUPPORTED;
    if (!p->q_main || !p->o_main || !p->k_cache || !p->v_cache || !p->kv_start || !p->kv_len || !p->trees ||
        !p->workspace)
        return SS_ERR_INVALID_ARG;
    if (p->gamma > 0 && (!p->q_spec || !p->k_spec || !p->v_spec || !p->o_spec)) return SS_ERR_INVALID_ARG;
    if (p->kv_slot_stride < p->head_dim || p->kv_head_stride < 0 || p->kv_total_slots < 1) return SS_ERR_INVALID_ARG;
    if ((p->kv_slot_stride & 7) || (p->kv_head_stride & 7)) return SS_ERR_INVALID_ARG;
    if (p->kv_total_slots > 0x7fffffffll) return SS_ERR_UNSUPPORTED;
    const long long rows_main = static_cast<long long>(p->batch) * p->max_nodes;
    if (rows_main * (p->gamma > 0 ? p->gamma : 1) > 0x7fffffffll) return SS_ERR_UNSUPPORTED;
    if (plan.groups * plan.cluster > 0x7fffffffll) return SS_ERR_UNSUPPORTED;
    const void* ptrs[] = {p->q_main, p->o_main, p->k_cache, p->v_cache, p->workspace,
                          p->gamma ? p->q_spec : nullptr, p->gamma ? p->k_spec : nullptr,
                          p->gamma ? p->v_spec : nullptr, p->gamma ? p->o_spec : nullptr};
    for (const void* q : ptrs)
        if (!ss::aligned16(q)) return SS_ERR_INVALID_ARG;
    if (!(p->sm_scale == p->sm_scale)) return SS_ERR_INVALID_ARG;
    if (p->workspace_bytes < ss_msa_attention_workspace_bytes(p)) return SS_ERR_WORKSPACE;

    ss::AttnArgs a;
    const int d = p->head_dim, H = p->n_heads, tk = ss::kTileKeys;
    const bool shared_heads = (p->kv_head_stride == 0);
    const long long kv_heads = shared_heads ? 1 : H;
    const long long kv_hstride = shared_heads ? d : p->kv_head_stride;
    bool ok = ss::make_map(&a.tm_k, p->k_cache, d, kv_heads, kv_hstride, p->kv_total_slots, p->kv_slot_stride, tk) &&
              ss::make_map(&a.tm_v, p->v_cache, d, kv_heads, kv_hstride, p->kv_total_slots, p->kv_slot_stride, tk) &&
              ss::make_map(&a.tm_qm, p->q_main, d, H, d, rows_main, static_cast<long long>(H) * d, plan.tmax8);
    if (ok && p->gamma > 0) {
        const long long rows_spec = rows_main * p->gamma;
        const long long hd = static_cast<long long>(H) * d;
        ok = ss::make_map(&a.tm_qs, p->q_spec, d, H, d, rows_spec, hd, plan.s0rows > 0 ? plan.s0rows : 8) &&
             ss::make_map(&a.tm_qs1, p->q_spec, d, H, d, rows_spec, hd, ss::kBlockRows) &&
             ss::make_map(&a.tm_ks, p->k_spec, d, H, d, rows_spec, hd, tk) &&
             ss::make_map(&a.tm_vs, p->v_spec, d, H, d, rows_spec, hd, tk);
    } else if (ok) {
        a.tm_qs = a.tm_qm; a.tm_qs1 = a.tm_qm; a.tm_ks = a.tm_k; a.tm_vs = a.tm_v;     // never used when gamma == 0
    }
    if (!ok) return SS_ERR_CUDA;
    a.batch = p->batch; a.n_heads = H; a.gamma = p->gamma; a.max_nodes = p->max_nodes;
    a.tmax8 = plan.tmax8; a.s0rows = plan.s0rows; a.n_blocks = plan.n_blocks;
    a.n_kslots = plan.n_kslots; a.n_vslots = plan.n_vslots;
    a.cluster = plan.cluster;
    a.cluster_shift = 0;
    while ((1 << a.cluster_shift) < plan.cluster) ++a.cluster_shift;
    a.head_coord = shared_heads ? 0 : 1;
    a.gamma_magic = p->gamma > 0 ? (65536 + p->gamma - 1) / p->gamma : 0;
    a.prefix_stable = (p->flags & SS_ATTN_PREFIX_STABLE) ? 1 : 0;
    a.scale_log2 = p->sm_scale * 1.4426950408889634f;
    a.o_main = static_cast<__nv_bfloat16*>(p->o_main);
    a.o_spec = static_cast<__nv_bfloat16*>(p->o_spec);
    a.lse_main = p->lse_main; a.lse_spec = p->lse_spec;
    a.kv_start = reinterpret_cast<const long long*>(p->kv_start);
    a.kv_len = p->kv_len; a.kv_capacity = p->kv_capacity; a.trees = p->trees;
    a.status = reinterpret_cast<int*>(p->workspace);
    a.partials = reinterpret_cast<float*>(static_cast<char*>(p->workspace) + ss::kWsHeaderBytes);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (plan.mode == ss::kCols) {
        switch (d) {
            case 64: return ss::launch_cols<64>(a, plan, s);
            case 80: return ss::launch_cols<80>(a, plan, s);
            default: return ss::launch_cols<128>(a, plan, s);
        }
    }
    switch (d) {
        case 64: return ss::launch<64>(a, plan, s);
        case 80: return ss::launch<80>(a, plan, s);
        default: return ss::launch<128>(a, plan, s);
    }
}

namespace ss {
// One warp runs the merge step of a head that is split two ways, as its CTA 0, for one row -- and no CTA 1 was
// launched, so the row it waits for never arrives: the wait runs out after its bound and the status word
// reports it.  Nothing else is read or written unless the area was not zero.
__global__ void wait_selftest_kernel(const __grid_constant__ AttnArgs a) {
    __shared__ __align__(16) float own_row[64 + 4];
    __shared__ int abort_flag;
    const int lane = threadIdx.x;
    for (int i = lane; i < 64 + 4; i += 32) own_row[i] = 1.f;
    if (lane == 0) abort_flag = 0;
    __syncwarp();
    int lim;
    asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(lim) : "l"(a.status + 1) : "memory");
    const long long limit = lim > 0 ? static_cast<long long>(lim) << 10 : kWaitCycles;
    Span sp;
    sp.L = 0; sp.T = 1; sp.gamma = 0; sp.tmax8 = 8; sp.n_stream = 0; sp.spec_end = 8;
    if (!merge_partial_rows<64>(a, sp, 0, 0, 0, 0, 2, 0, smem_u32(own_row), a.partials, static_cast<size_t>(64) * (64 + 4), 0, 1, lane, 32, limit,
                                &abort_flag))
        set_status(a.status, SS_ERR_DEVICE_TIMEOUT);
}
}  // namespace ss

extern "C" int32_t ss_wait_selftest(void* workspace, size_t workspace_bytes, void* stream) {
    const size_t need = ss::kWsHeaderBytes + static_cast<size_t>(2) * 64 * (64 + 4) * 4 + 256;
    if (workspace == nullptr) return SS_ERR_INVALID_ARG;
    if (workspace_bytes < need) return SS_ERR_WORKSPACE;
    ss::AttnArgs a{};
    a.status = static_cast<int*>(workspace);
    a.partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + ss::kWsHeaderBytes);
    a.o_main = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + need - 256);      // never reached on a zero area
    a.max_nodes = 1; a.n_heads = 1;
    ss::wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(a);
    return cudaGetLastError() == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}

#ifdef SS_TRACE
// developer build only: copies the timestamp buffer to the host / clears it
extern "C" int32_t ss_trace_read(long long* out) {
    return cudaMemcpyFromSymbol(out, ss::g_trace, sizeof(ss::g_trace)) == cudaSuccess ? 0 : -1;
}
extern "C" int32_t ss_trace_clear() {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, ss::g_trace) != cudaSuccess) return -1;
    if (cudaMemset(p, 0, sizeof(ss::g_trace)) != cudaSuccess) return -1;
    unsigned long long wall[8][6];
    for (int i = 0; i < 8; ++i) { wall[i][0] = ~0ull; wall[i][1] = 0ull; wall[i][2] = 0ull; wall[i][3] = ~0ull; wall[i][4] = 0ull; wall[i][5] = ~0ull; }
    unsigned long long keys[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (cudaMemcpyToSymbol(ss::g_wall, wall, sizeof(wall)) != cudaSuccess) return -1;
    return cudaMemcpyToSymbol(ss::g_key, keys, sizeof(keys)) == cudaSuccess ? 0 : -1;
}
extern "C" int32_t ss_trace_cta_wall(unsigned long long* out) {
    return cudaMemcpyFromSymbol(out, ss::g_cta_wall, sizeof(ss::g_cta_wall)) == cudaSuccess ? 0 : -1;
}
extern "C" int32_t ss_trace_base(int base) {
    return cudaMemcpyToSymbol(ss::g_trace_base, &base, sizeof(int)) == cudaSuccess ? 0 : -1;
}
extern "C" int32_t ss_trace_wall(unsigned long long* out) {
    return cudaMemcpyFromSymbol(out, ss::g_wall, sizeof(ss::g_wall)) == cudaSuccess ? 0 : -1;
}
#endif
