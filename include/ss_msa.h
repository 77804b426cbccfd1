/*
 * ss_msa.h -- C ABI of the Speculative-Streaming decode hot path on NVIDIA B200 (sm_100a).
 *
 * One decode step of Speculative Streaming verifies the tree draft of the previous pass and
 * speculates the next one in the same forward pass (Sec. 3.2.2).  This library implements the
 * attention of that pass, the verification and the cache backtracking:
 *
 *   ss_tree_build      parent array -> depth / ancestor-bitmask descriptor       (host, pure)
 *   ss_msa_attention   one layer of tree-masked multi-stream attention           (Eq. 1, Eq. 2)
 *   ss_tree_verify     greedy verification of the tree draft                     (Sec. 3.2.2, App. A.1)
 *   ss_kv_compact      lazy KV-cache backtracking of the accepted path           (App. A.1)
 *   ss_next_draft      next tree draft from the stream logits of the last accepted node (Sec. 3.2.2, App. A.1)
 *   ss_tree_prune      parallel tree pruning by early-exit transition probabilities  (Sec. 3.2.3)
 *   ss_tree_verify_soft / ss_tree_verify_sampled   soft matching, top-k sampling at T = 1  (App. A.2, App. B)
 *   ss_stream_insert   stream initialisation S = M + P_j                            (Eq. 3)
 *   ss_value_rotate    value-rotation stream variant                                (Eq. 7)
 *   ss_status          read back the device status word
 *   ss_wait_selftest   diagnostic: a device-side wait that runs out reports SS_ERR_DEVICE_TIMEOUT
 *
 * Conventions
 *   - Every call returns an int32 status: SS_OK or a negative SS_ERR_* code.  No exceptions.
 *   - All buffers are caller-owned.  Unless a parameter says "host", a pointer is a DEVICE pointer.
 *   - Device calls validate their host-visible arguments first (an error means nothing was
 *     launched), then enqueue kernels on `stream` (a cudaStream_t passed as void*; NULL = the
 *     default stream) and return without synchronising.  They never allocate or free memory and
 *     never read device memory back to the host, so they can be captured into a CUDA graph.
 *   - bf16 tensors are raw 16-bit patterns; the innermost (head_dim) axis is contiguous and every
 *     tensor base, and every K/V row, must be 16-byte aligned.
 *   - A workspace must be zero-filled once (cudaMemset) before its first use; each call leaves
 *     it ready for the next.  Word 0 of a workspace is the device status word: a kernel that
 *     detects a broken invariant (sequence over capacity, a wait that ran out) stores its
 *     SS_ERR_* code there and returns instead of faulting.  After SS_ERR_DEVICE_TIMEOUT the
 *     workspace's contents are undefined: zero-fill it again before reuse.
 *   - Two calls that share a workspace must not overlap on the device.
 */
#ifndef SS_MSA_H_
#define SS_MSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SS_MAX_NODES 64      /* tree nodes per sequence (one 64-bit ancestor word per node) */
#define SS_MAX_GAMMA 4       /* speculative streams per node */
#define SS_PATH_STRIDE SS_MAX_NODES /* entries per sequence in accept_path */
#define SS_MAX_TOPK 8        /* tokens taken per stream / per node by the top-k entry points */

enum {
    SS_OK = 0,
    SS_ERR_INVALID_ARG = -1,    /* null pointer, non-positive size, misaligned buffer */
    SS_ERR_BAD_TREE = -2,       /* parent[0] != -1 or parent[i] outside [0, i) */
    SS_ERR_UNSUPPORTED = -3,    /* head_dim not in {64, 80, 128}, too many nodes or streams */
    SS_ERR_WORKSPACE = -4,      /* workspace smaller than the *_workspace_bytes() answer */
    SS_ERR_CAPACITY = -5,       /* kv_len + n_nodes exceeds the sequence's slot capacity */
    SS_ERR_CUDA = -6,           /* a CUDA runtime/driver call failed (launch, tensor-map encode) */
    SS_ERR_DEVICE_TIMEOUT = -7  /* a bounded device-side wait ran out */
};

/* Tree / mask descriptor.  Plain data, identical on host and device.
 * Node 0 is the root (the correction token issued by the main stream in the previous pass,
 * App. A.1); nodes are flattened root-first so that parent[i] < i.  anc_mask[t] has bit a set
 * iff a is t or lies on the path from the root to t: a node attends to all its predecessors
 * starting from the root, and to itself (attention-mask figure of App. A). */
typedef struct ss_tree_desc {
    int32_t n_nodes;                 /* T, 1..SS_MAX_NODES */
    int32_t gamma;                   /* streams per node the tree was built for (informative) */
    int32_t max_depth;               /* depth(root) = 0 */
    int32_t reserved;
    int32_t parent[SS_MAX_NODES];    /* parent[0] = -1; entries >= n_nodes are -1 */
    int32_t depth[SS_MAX_NODES];
    uint64_t anc_mask[SS_MAX_NODES];
} ss_tree_desc;

/* Builds the descriptor of one tree on the HOST (all pointers are host pointers).
 * Errors: SS_ERR_INVALID_ARG (null), SS_ERR_UNSUPPORTED (n_nodes > SS_MAX_NODES or gamma outside
 * [0, SS_MAX_GAMMA]), SS_ERR_BAD_TREE (n_nodes < 1, parent[0] != -1, parent[i] not in [0, i)).
 * Pure and reentrant.  The mask is constant for a fixed tree shape (Sec. 3.2.2), so a caller
 * may build it once and reuse it. */
int32_t ss_tree_build(const int32_t* parent, int32_t n_nodes, int32_t gamma, ss_tree_desc* out);

/* One layer of attention for a batch of sequences, each with its own tree draft.
 *
 * Main-stream row of node t (Eq. 1): attends the sequence's cached prefix (slots 0..L-1) plus the
 * tree nodes on its root path, itself included.  Speculative-stream row (t, j), 1 <= j <= gamma
 * (Eq. 2): attends the same main-stream keys plus the stream keys (t,1)..(t,j) of the same node.
 * Only main-stream K/V live in the cache; stream K/V are transient inputs (Sec. 3.2.1).
 * gamma = 0 gives a plain tree-masked layer (the N - N_s lower layers); the *_spec pointers are
 * then ignored.
 *
 * Layouts (bf16, element strides):
 *   q_main, o_main                 [batch][max_nodes][n_heads][head_dim]
 *   q_spec, k_spec, v_spec, o_spec [batch][max_nodes][gamma][n_heads][head_dim]
 *   k_cache, v_cache               this layer's slab: slot s, head h at
 *                                  base + s*kv_slot_stride + h*kv_head_stride, kv_total_slots slots.
 *                                  Sequence b owns slots kv_start[b] .. ; its prefix sits at
 *                                  +0..L_b-1 and the caller has already written the K/V of tree node
 *                                  t at slot kv_start[b] + L_b + t.
 *   kv_start int64[batch], kv_len int32[batch] (= L_b), kv_capacity int32[batch] (may be NULL):
 *                                  device arrays, read by the kernel (the host never needs L_b).
 *   trees                          device array of `batch` descriptors; rows of nodes >= n_nodes of a
 *                                  sequence are neither read nor written.
 *   lse_main float[batch][max_nodes][n_heads], lse_spec float[batch][max_nodes][gamma][n_heads]:
 *                                  optional natural-log sum-exp of the scaled scores (NULL to skip).
 * Scores are sm_scale * <q, k>; softmax statistics and both products accumulate in fp32.
 * The workspace holds, after its 256-byte header, the partial rows (fp32 O, m, l per query row) of blocks
 * of 128 query rows whose keys are split over several CTAs (ss_msa_attention_workspace_bytes).  The rows are
 * their own arrival flags: between calls that area is all zero, a partial row is never stored with a +0
 * word (-0 is stored instead), a CTA waits for the words it combines to read non-zero and stores zeros over
 * them afterwards.  So calls of different shapes may share one workspace as long as they are ordered on one
 * stream and it is large enough for each.  Word 1 of the workspace, if positive, shortens the bound of the
 * device-side waits to that many units of 1024 cycles (default: about one second) for calls whose heads
 * have at most 64 query rows and for ss_wait_selftest; the library reads it and never writes it.
 * Word 2 counts, over all calls since the caller last cleared it, the CTAs of unsplit 128-row blocks that
 * started over: such a block first takes every row's exponentials against the maximum of the row's first
 * 128 keys, and if a later tile exceeds that reference by more than about 2^57 it runs its tiles again
 * with a running maximum (same result, about twice the time for that block).  Diagnostics only.
 * Precondition of a split (batch * n_heads * row blocks below the SM count): the CTAs that share a block's
 * keys wait for one another's partial rows at the end, so they must all be resident at once.  The call sizes the split from
 * the device's SM count; if other work holds SMs for the whole duration of the call (another stream, another
 * process, a partition of the GPU) the wait can run out: the CTAs then give up, the status word reads
 * SS_ERR_DEVICE_TIMEOUT and the outputs of the blocks concerned are not written.
 * Reads no K/V row past slot kv_start[b]+L_b+T_b-1 whose value can reach an output (a tile may touch
 * later slots of the slab; what it finds there is masked or cleared); writes only o_*, lse_* and the
 * workspace.
 * If kv_capacity is given and L_b + T_b > kv_capacity[b], sequence b is skipped and the status word
 * is set to SS_ERR_CAPACITY.
 * Errors (nothing launched): SS_ERR_INVALID_ARG, SS_ERR_UNSUPPORTED, SS_ERR_WORKSPACE, SS_ERR_CUDA. */
/* ss_attn_params.flags.
 * SS_ATTN_PREFIX_STABLE: the caller promises that no kernel that may still be running when this call's
 * kernel is scheduled writes the cached prefix (slots below kv_len of every sequence), kv_start, kv_len,
 * kv_capacity or the tree descriptors.  The call is launched so that it can be scheduled while the
 * previous kernel of the stream drains (programmatic dependent launch); with the promise it reads the
 * lengths and starts streaming the prefix during that time.  Queries, the tree nodes' K/V, the stream K/V
 * and every output keep plain stream order either way.  Inside a decode step the promise holds naturally:
 * the kernels before a layer's attention write this step's queries and tree-node K/V, never the prefix.
 * It does NOT hold for a call that directly follows ss_kv_compact on the same cache when that call writes
 * the kv_len array the attention reads (kv_len_out == kv_len) or when the attention's lengths already
 * include the compacted slots: compaction turns tree slots into prefix and writes the lengths.  Pass
 * flags = 0 to the first attention call after such a compaction, or put any other kernel between them. */
#define SS_ATTN_PREFIX_STABLE 1u

typedef struct ss_attn_params {
    int32_t batch, n_heads, head_dim, gamma;
    int32_t max_nodes;              /* row stride (in nodes) of the q/o/lse arrays, <= SS_MAX_NODES */
    float sm_scale;
    const void* q_main;
    void* o_main;
    const void* q_spec;
    const void* k_spec;
    const void* v_spec;
    void* o_spec;
    const void* k_cache;
    const void* v_cache;
    int64_t kv_slot_stride, kv_head_stride, kv_total_slots;
    const int64_t* kv_start;
    const int32_t* kv_len;
    const int32_t* kv_capacity;
    const ss_tree_desc* trees;
    float* lse_main;
    float* lse_spec;
    void* workspace;
    size_t workspace_bytes;
    uint32_t flags;                 /* SS_ATTN_* bits, 0 for none */
} ss_attn_params;

/* Bytes of workspace ss_msa_attention needs for these shapes (pointers in *p are not read). */
size_t ss_msa_attention_workspace_bytes(const ss_attn_params* p);
int32_t ss_msa_attention(const ss_attn_params* p, void* stream);

/* Greedy ("hard" matching, App. A.2) verification of each sequence's tree draft (Sec. 3.2.2,
 * App. A.1).  am[t] = lowest index maximising logits[b][t][.]; the root is always accepted; node c
 * is valid iff its parent is valid and draft_tokens[c] == am[parent[c]]; the deepest valid node
 * wins, the lowest node index among equally deep ones.
 *   logits        float [batch][max_nodes][vocab]   main-stream logits of every tree node
 *   draft_tokens  int32 [batch][max_nodes]
 *   accept_len    int32 [batch]      nodes on the accepted path, root included (1 .. max_depth+1)
 *   accept_path   int32 [batch][SS_PATH_STRIDE]  node indices root-first, padded with -1
 *   last_node     int32 [batch]      last accepted node
 *   bonus_token   int32 [batch]      am[last_node]: the correction token, root of the next draft
 *   node_argmax   int32 [batch][max_nodes] or NULL
 * Bit-exact by definition (comparisons of fp32 values only). */
size_t ss_tree_verify_workspace_bytes(int32_t batch, int32_t max_nodes, int32_t vocab);
int32_t ss_tree_verify(const float* logits, const int32_t* draft_tokens, const ss_tree_desc* trees,
                       int32_t batch, int32_t max_nodes, int32_t vocab, int32_t* accept_len,
                       int32_t* accept_path, int32_t* last_node, int32_t* bonus_token,
                       int32_t* node_argmax, void* workspace, size_t workspace_bytes, void* stream);

/* ss_tree_verify for callers that cannot provide scratch memory.  (The paper has no counterpart:
 * this is a property of the library, not of the method.)
 * Who needs it: code that must not allocate device memory where it calls this library, for example a
 * plug-in that owns no allocator, a serving loop whose memory was fixed at start-up, or a section in
 * which cudaMalloc is not permitted.  The scratch that ss_tree_verify takes as `workspace` lives here
 * in a fixed array of SS_VERIFY_STATIC_SCRATCH_BYTES bytes inside the library's device image; every
 * GPU that loads the library holds that array until the process exits.  The call allocates and frees
 * nothing.  Same arguments, outputs and results as ss_tree_verify, minus the workspace.
 *   - Sizes whose scratch need (ss_tree_verify_workspace_bytes) exceeds the fixed array are rejected
 *     with SS_ERR_WORKSPACE and nothing is launched.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current); make that first call before starting any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; each call
 *     clears the words that must start at zero (on `stream`, before its kernel).  Calls that overlap
 *     on the same device (different streams, or several host threads) race: serialise them. */
#define SS_VERIFY_STATIC_SCRATCH_BYTES (1u << 20)
int32_t ss_tree_verify_static(const float* logits, const int32_t* draft_tokens, const ss_tree_desc* trees,
                              int32_t batch, int32_t max_nodes, int32_t vocab, int32_t* accept_len,
                              int32_t* accept_path, int32_t* last_node, int32_t* bonus_token,
                              int32_t* node_argmax, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Order of logits used by every arg-max / top-k below and by ss_tree_verify: IEEE fp32 order with
 * -0 == +0, equal values by ascending index; a NaN ranks below every comparable value (inputs are
 * meant to be finite; a row without any comparable value reports index 0 first). */

/* Next tree draft (Sec. 3.2.2 "Parallel speculation and verification", App. A.1).  The correction token
 * is the root; the top_k best tokens of stream g's logits are the children of every node of level g - 1,
 * so that tokens drawn from stream n are the predecessors of those drawn from stream n + 1.  Nodes are
 * numbered level by level, the children of a node in rank order (parent[i] < i); the full tree has
 * 1 + sum_{g=1..gamma} top_k^g nodes (Sec. 3.2.3) and is cut after max_nodes nodes in that order.
 *   stream_logits float [batch][n_rows][gamma][vocab]   logits of the speculative streams
 *   row_index     int32 [batch] or NULL   which of the n_rows of each sequence to use: the last accepted
 *                                         node written by a verification call (NULL: row 0)
 *   bonus_token   int32 [batch]           the correction token (root of the new draft)
 *   draft_tokens  int32 [batch][max_nodes]  out: tokens of the new tree, -1 past its nodes
 *   trees         [batch]                 out: descriptors of the new trees, as ss_tree_build would give
 * All pointers are device pointers: a decode loop needs no host round trip between the verification of one
 * draft and the attention over the next.  Errors: SS_ERR_INVALID_ARG, SS_ERR_UNSUPPORTED (gamma >
 * SS_MAX_GAMMA, top_k > SS_MAX_TOPK or > vocab, max_nodes > SS_MAX_NODES), SS_ERR_WORKSPACE, SS_ERR_CUDA. */
size_t ss_next_draft_workspace_bytes(int32_t batch, int32_t gamma, int32_t vocab);
int32_t ss_next_draft(const float* stream_logits, int32_t n_rows, const int32_t* row_index, const int32_t* bonus_token,
                      int32_t batch, int32_t gamma, int32_t vocab, int32_t top_k, int32_t max_nodes,
                      int32_t* draft_tokens, ss_tree_desc* trees, void* workspace, size_t workspace_bytes, void* stream);

/* Parallel tree pruning (Sec. 3.2.3; pruning paragraph and figure of App. A.1).  The transition probability
 * of the edge parent -> child is the early-exit probability of the child's token at the parent,
 * softmax(exit_logits[parent])[draft_tokens[child]]; an edge below `threshold` drops the child's whole
 * sub-tree; the survivors keep their order and are re-indexed.  The root always survives.  The cache of
 * the layers below is not touched (backtracking is lazy: ss_kv_compact gathers by original node index, so
 * map a path of the pruned tree through kept_nodes first).
 *   exit_logits  float [batch][max_nodes][vocab]   early-exit logits of every node (the caller's H(o(M^l)))
 *   edge_prob    float [batch][max_nodes]  out: transition probability of each node's edge (root: 1)
 *   new_index    int32 [batch][max_nodes]  out: index in the pruned tree, -1 if dropped
 *   kept_nodes   int32 [batch][max_nodes]  out: original index of each surviving node, -1 past them
 *   kept_tokens  int32 [batch][max_nodes]  out: their draft tokens
 *   pruned_trees [batch]                   out: descriptors of the pruned trees
 * Probabilities are computed in fp32 (log-sum-exp of the row); a transition within rounding of the
 * threshold may fall on either side. */
size_t ss_tree_prune_workspace_bytes(int32_t batch, int32_t max_nodes, int32_t vocab);
int32_t ss_tree_prune(const float* exit_logits, const int32_t* draft_tokens, const ss_tree_desc* trees, int32_t batch,
                      int32_t max_nodes, int32_t vocab, float threshold, float* edge_prob, int32_t* new_index,
                      int32_t* kept_nodes, int32_t* kept_tokens, ss_tree_desc* pruned_trees, void* workspace,
                      size_t workspace_bytes, void* stream);

/* Verification with "soft" matching (App. A.2 names it as the relaxation of the hard criterion; the rule is
 * the typical acceptance of the work it cites): a draft token is accepted when the main stream gives it a
 * probability of at least min(eps, delta * exp(-H)), H the entropy of the main stream's distribution at the
 * parent.  Outputs as ss_tree_verify (bonus_token is the arg-max at the last accepted node), plus
 * edge_prob and node_entropy (float [batch][max_nodes], node_entropy may be NULL).  Workspace:
 * ss_tree_prune_workspace_bytes. */
int32_t ss_tree_verify_soft(const float* logits, const int32_t* draft_tokens, const ss_tree_desc* trees, int32_t batch,
                            int32_t max_nodes, int32_t vocab, float eps, float delta, int32_t* accept_len,
                            int32_t* accept_path, int32_t* last_node, int32_t* bonus_token, float* edge_prob,
                            float* node_entropy, void* workspace, size_t workspace_bytes, void* stream);

/* Verification under top-k sampling at temperature 1 (App. B "Top-k Sampling"): the main stream's token at
 * node t is drawn from the softmax over its top_k largest logits by inversion with uniforms[b][t] in [0, 1)
 * (the first rank whose cumulative probability exceeds it); a draft token is accepted when it equals the
 * token drawn at its parent; bonus_token is the token drawn at the last accepted node.  The caller owns
 * the random numbers.  node_token int32 [batch][max_nodes] (may be NULL) receives the drawn tokens. */
size_t ss_tree_verify_sampled_workspace_bytes(int32_t batch, int32_t max_nodes, int32_t vocab);
int32_t ss_tree_verify_sampled(const float* logits, const int32_t* draft_tokens, const ss_tree_desc* trees,
                               const float* uniforms, int32_t batch, int32_t max_nodes, int32_t vocab, int32_t top_k,
                               int32_t* accept_len, int32_t* accept_path, int32_t* last_node, int32_t* bonus_token,
                               int32_t* node_token, void* workspace, size_t workspace_bytes, void* stream);

/* Stream insertion (Eq. 3) with the identity for the transformation f, as in all of the paper's experiments
 * (App. A.2): S_tj = M_t + P_j.  bf16 in and out, one fp32 addition per element.
 *   main_hidden [rows][hidden], stream_emb [gamma][hidden], out [rows][gamma][hidden]; hidden % 8 == 0. */
int32_t ss_stream_insert(const void* main_hidden, const void* stream_emb, void* out, int64_t rows, int32_t gamma,
                         int32_t hidden, void* stream);

/* Value rotation (App. B, Eq. 7): V_tn = V_t e^{i epsilon n}, n = 1..gamma.  Consecutive pairs of a value
 * vector are the real and imaginary part of a complex number; stream n's value is the main stream's rotated
 * by the angle epsilon * n (cos and sin evaluated on the host in double, used as fp32).
 *   v_main [rows][width] bf16, v_streams [rows][gamma][width] bf16; width % 8 == 0. */
int32_t ss_value_rotate(const void* v_main, void* v_streams, int64_t rows, int32_t gamma, int32_t width, float epsilon,
                        void* stream);

/* Cache layout shared by all layers: layer l, slot s, head h, element c of K sits at
 * k_cache_all + l*layer_stride + s*slot_stride + h*head_stride + c (strides in elements). */
typedef struct ss_cache_layout {
    int32_t n_layers, n_heads, head_dim, reserved;
    int64_t layer_stride, slot_stride, head_stride;
} ss_cache_layout;

/* Lazy KV backtracking (App. A.1): in every layer and for every sequence b, the K and V of accepted
 * node accept_path[b][i] move from slot kv_start[b]+L_b+path[i] to slot kv_start[b]+L_b+i, in place,
 * for i < accept_len[b]; kv_len_out[b] = L_b + accept_len[b] (kv_len_out may alias kv_len_in).
 * Prefix slots are never written; slots at or past L_b + accept_len[b] are unspecified afterwards.
 * Stream K/V are never cached, so nothing else moves (Sec. 3.2.1).
 * accept_len / accept_path are the device outputs of ss_tree_verify: no host round trip. */
int32_t ss_kv_compact(void* k_cache_all, void* v_cache_all, const ss_cache_layout* layout, int32_t batch,
                      const int64_t* kv_start, const int32_t* kv_len_in, const int32_t* accept_len,
                      const int32_t* accept_path, int32_t* kv_len_out, void* stream);

/* Diagnostic of the bounded device-side waits.  Runs, as one warp, the step in which a CTA of a head split
 * two ways combines its share of the partial rows (the routine ss_msa_attention's kernels use), with no
 * second CTA launched: the row it waits for cannot arrive, the wait runs out after its bound (workspace
 * word 1, as for ss_msa_attention) and the kernel stores SS_ERR_DEVICE_TIMEOUT in the status word and
 * returns.  Nothing faults or hangs; the stream stays usable.  `workspace`: device, zero-filled (apart from
 * word 1), at least 64 KiB; it is left as found.  Errors (nothing launched): SS_ERR_INVALID_ARG,
 * SS_ERR_WORKSPACE, SS_ERR_CUDA. */
int32_t ss_wait_selftest(void* workspace, size_t workspace_bytes, void* stream);

/* Synchronises `stream`, copies the status word of `workspace` to *device_status_out (host) and
 * clears it.  Returns SS_ERR_CUDA if the stream reports an error. */
int32_t ss_status(void* workspace, void* stream, int32_t* device_status_out);

/* Library version (major*10000 + minor*100 + patch) and a short human-readable error string. */
int32_t ss_version(void);
const char* ss_error_string(int32_t status);

#ifdef __cplusplus
}
#endif
#endif /* SS_MSA_H_ */
