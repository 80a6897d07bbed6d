/*
 * mtv.h — C ABI of the static-tree verification library (Medusa-style
 * speculative decoding, one verification step on one NVIDIA B200, sm_100a).
 *
 * One decode step (Section 3.1 and Section 3.2 of the paper):
 *   medusa_heads_topk      K residual-MLP heads -> per-head top-k -> flat candidate
 *                          buffer -> tokens of the T static tree nodes
 *   tree_verify_attention  attention of all T tree nodes over [prefix ; tree] K/V under
 *                          the static visibility matrix (once per backbone layer)
 *   tree_accept            greedy longest-prefix acceptance + Gather of the accepted
 *                          tokens through retrieve_indices
 *   kv_compact_accepted    the same Gather applied to the accepted nodes' K/V rows,
 *                          in place, all layers; advances seq_lens
 * with the tree's static tensors built once by tree_build_static.  Beside the step proper:
 *   tree_kv_append_rope    K/V rows of the tree nodes into the cache, rotary embedding at
 *                          position seq_len + depth
 *   lm_head_argmax         the base model's LM head with the per-node argmax fused in, and
 *   tree_accept_keys       the acceptance that reads its result instead of stored logits
 *
 * Conventions
 *   - Every function returns an int: MTV_OK (0) or a negative MTV_ERR_* code.
 *   - "device" pointers are CUDA global-memory addresses valid on the current
 *     device; "host" pointers are ordinary process memory.  The caller owns every
 *     buffer; the library owns only mtv_tree_t objects.
 *   - Hot calls (the four step functions and mtv_verify_step) only enqueue work on
 *     `stream` (a cudaStream_t passed as void*; NULL = default stream).  They never
 *     allocate, never synchronise and never copy to the host.  Results are ready
 *     when the stream reaches the end of the enqueued work.
 *   - bf16 data is passed as raw 16-bit patterns (mtv_bf16).  Indices are int32.
 *   - Data-dependent faults (a sequence that does not fit its cache) are written to
 *     the caller's device `status[B]` (0 = ok, MTV_ERR_* otherwise); the outputs of
 *     that sequence are left untouched.  status may be NULL.
 *   - Supported shapes: D in {64, 128}; 1 <= T <= 128; 1 <= K <= 8; per-depth
 *     top-k <= 16; Hq a multiple of Hkv with Hq/Hkv <= 8; H a multiple of 8; at most
 *     16 batch rows in medusa_heads_topk.
 *     Anything else returns MTV_ERR_UNSUPPORTED_SHAPE.
 */
#ifndef MTV_H_
#define MTV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MTV_OK 0
#define MTV_ERR_INVALID_ARG (-1)
#define MTV_ERR_UNSUPPORTED_SHAPE (-2)
#define MTV_ERR_WORKSPACE (-3)
#define MTV_ERR_CUDA (-4)
#define MTV_ERR_TIMEOUT (-5)
#define MTV_ERR_CAPACITY (-6) /* status[b]: seq_lens[b] + T exceeds the cache capacity */
#define MTV_ERR_BOUNDS (-7)   /* device error word, -DMTV_DEBUG_BOUNDS builds only: an index read from device
                                 memory (a tree table, acc_nodes, accept_len, the sequence order) was out of
                                 range; the access was skipped */

#define MTV_MAX_K 8
#define MTV_MAX_T 128
#define MTV_MAX_TOPK 16

typedef uint16_t mtv_bf16;
typedef struct mtv_tree mtv_tree_t;

/* Host view of a tree's static tensors (pointers stay valid until tree_destroy). */
typedef struct {
    int32_t T;           /* nodes including the root */
    int32_t K;           /* heads = maximum depth */
    int32_t P;           /* N_paths = number of leaves */
    int32_t C;           /* flat candidate buffer length = 1 + sum k_d */
    int32_t anc_words;   /* 64-bit words per row of anc */
    int32_t on_device;   /* 1 if the tables were uploaded */
    int32_t k_d[MTV_MAX_K];         /* candidates taken from head d+1 */
    int32_t cand_offset[MTV_MAX_K]; /* first slot of head d+1 in the candidate buffer */
    const int32_t *node_ranks;       /* [T][K] rank tuple of each node, -1 padded */
    const int32_t *parent;           /* [T], -1 for the root */
    const int32_t *depth;            /* [T] */
    const int32_t *rank;             /* [T] rank within its head, -1 for the root */
    const int32_t *tree_indices;     /* [T] node -> slot of the candidate buffer */
    const int32_t *retrieve_indices; /* [P][K+1] node ids root..leaf, -1 padded */
    const uint64_t *anc;             /* [T][anc_words] ancestor-or-self bitmask */
    const uint8_t *medusa_attn_mask; /* [T][T] dense 0/1 form of anc */
} mtv_tree_info;

/* ---------------------------------------------------------------------------
 * Static tree tensors — Section 3.2, "Tensorization of Tree Topology" (the
 * visibility matrix medusa_attn_mask and tree_indices) and "Zero-Copy Retrieval"
 * (retrieve_indices [N_paths][K+1]).  Host-side, run once at initialisation.
 *
 * node_ranks: host, [n_nodes][K] int32.  Row = the per-depth ranks on the way from
 *   the root to the node (r_1..r_d), padded with -1.  The root is implicit.  Order is
 *   free; duplicates are an error; every node's parent must be present.
 * The flattened order is root first, then ascending (depth, rank tuple).  Node i's
 *   K/V row lives in cache slot seq_lens[b] + i; its token is candidate slot
 *   tree_indices[i]; paths are ordered by ascending leaf index.
 * upload != 0 copies the tables to the current CUDA device (needed by the hot
 *   calls); upload == 0 builds the host tables only (no CUDA call is made).
 * Errors: MTV_ERR_INVALID_ARG (bad ranks, orphan, duplicate), MTV_ERR_UNSUPPORTED_SHAPE
 *   (K, T or a top-k beyond the limits), MTV_ERR_CUDA (upload failed).
 */
int tree_build_static(int K, int n_nodes, const int32_t *node_ranks, int upload, mtv_tree_t **out);

/* Full Cartesian tree: every rank tuple with r_d < topk[d].  node_ranks: host
 * [capacity][K]; *n_nodes receives the node count (root excluded).  Returns
 * MTV_ERR_INVALID_ARG if capacity is too small (then *n_nodes = needed count). */
int tree_gen_cartesian(int K, const int32_t *topk, int capacity, int32_t *node_ranks, int *n_nodes);

/* Sparse tree: root plus the T_total-1 highest-scoring nodes of the full R_max-ary
 * depth-K tree, score = product over depths of p(r) = 1/((r+1) Z), Z = sum_{r<R_max} 1/(r+1);
 * ties by depth ascending then rank tuple ascending; scores compared exactly.
 * node_ranks: host [T_total-1][K].  R_max <= 16, K <= 7. */
int tree_gen_rank_prior(int K, int T_total, int R_max, int32_t *node_ranks, int *n_nodes);

int tree_query(const mtv_tree_t *tree, mtv_tree_info *info);
void tree_destroy(mtv_tree_t *tree);

/* Bytes of device scratch that any hot call below may need for these shapes.
 * Lcap = cache capacity in rows.  The same buffer may be reused by successive
 * calls on one stream; concurrent calls need separate buffers.  Returns 0 on
 * invalid arguments. */
size_t mtv_workspace_bytes(const mtv_tree_t *tree, int B, int H, int V, int Hq, int Hkv, int D, int Lcap);

/* ---------------------------------------------------------------------------
 * Medusa heads + per-head top-k + tree expansion — Section 3.1 (K parallel heads,
 * each an MLP with a residual connection, head k predicting token t+k+1) and the
 * candidate buffer of Section 3.2.
 *   y = W1_k h_b + b1_k;  h' = h_b + SiLU(y);  z_k = W2_k h'      (fp32, no rounding between)
 *   cand[b] = [root_tok[b] | ids of the k_1 largest z_1 | k_2 largest z_2 | ...]
 *             (descending logit, equal logits by ascending id)
 *   tree_tok[b][i] = cand[b][tree_indices[i]]
 * All pointers device.  hidden [B][H]; W1 [K][H][H] and W2 [K][V][H] row-major with
 * the output feature outermost; b1 [K][H] or NULL; root_tok [B]; cand [B][C];
 * cand_logit [B][C-1] fp32 or NULL; tree_tok [B][T].  1 <= B <= 16.
 */
int medusa_heads_topk(const mtv_tree_t *tree, int B, int H, int V,
                      const mtv_bf16 *hidden, const mtv_bf16 *W1, const mtv_bf16 *b1,
                      const mtv_bf16 *W2, const int32_t *root_tok,
                      int32_t *cand, float *cand_logit, int32_t *tree_tok,
                      void *ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------
 * Tree K/V append with rotary embedding — the step just before the tree attention; Section 3.2
 * ("Tensorization of Tree Topology": tree_indices maps the flattened nodes to their positions).
 * For sequence b and node i, position = seq_lens[b] + depth[i]:
 *   angle_d = position * theta^(-2d/D), d < D/2        (rotate-half pairing, a reading: the paper is silent)
 *   (x[d], x[d + D/2]) -> (x[d] cos - x[d + D/2] sin, x[d + D/2] cos + x[d] sin)
 * q [B][T][Hq][D] is rotated in place; k_new, v_new [B][T][Hkv][D]: the rotated K row and the V row
 * are written to cache row seq_lens[b] + i (cache layout and strides as in tree_verify_attention).
 * Angles in double precision, arithmetic in fp32, bf16 results (round to nearest even).
 * All pointers device.  rope_theta == 0 means 10000.  status[b] = MTV_ERR_CAPACITY (nothing
 * written for b) if seq_lens[b] + T > Lcap.  seq_lens is not changed.
 */
int tree_kv_append_rope(const mtv_tree_t *tree, int B, int Hq, int Hkv, int D, mtv_bf16 *q,
                        const mtv_bf16 *k_new, const mtv_bf16 *v_new, mtv_bf16 *k_cache, mtv_bf16 *v_cache,
                        int64_t stride_b, int64_t stride_h, int64_t stride_t, int Lcap,
                        const int32_t *seq_lens, float rope_theta, int32_t *status, void *stream);

/* The same for all n_layers caches of a step in one launch: q_layers [n_layers][B][T][Hq][D] (rotated
 * in place), k_new_layers, v_new_layers [n_layers][B][T][Hkv][D]; k_caches / v_caches: device arrays of
 * n_layers device pointers, as for kv_compact_accepted. */
int tree_kv_append_rope_layers(const mtv_tree_t *tree, int B, int Hq, int Hkv, int D, int n_layers,
                               mtv_bf16 *q_layers, const mtv_bf16 *k_new_layers, const mtv_bf16 *v_new_layers,
                               mtv_bf16 *const *k_caches, mtv_bf16 *const *v_caches,
                               int64_t stride_b, int64_t stride_h, int64_t stride_t, int Lcap,
                               const int32_t *seq_lens, float rope_theta, int32_t *status, void *stream);

/* ---------------------------------------------------------------------------
 * Tree attention — Section 3.2 / Fig. 2(b): the T tree nodes attend to the KV cache
 * under the static visibility matrix.  For sequence b, node i, query head h
 * (KV head g = h / (Hq/Hkv)):
 *   visible = [0, seq_lens[b])  U  { seq_lens[b] + a : a ancestor-or-self of i }
 *   out[b][i][h] = softmax_j(scale <q[b][i][h], k[b][g][j]>) . v[b][g][j]   over visible j
 * bf16 inputs, fp32 scores / softmax / accumulation, bf16 output (round to nearest even).
 * All pointers device.  q, out [B][T][Hq][D] contiguous.  k_cache / v_cache: element
 * (b, g, row, d) at b*stride_b + g*stride_h + row*stride_t + d (strides in elements,
 * multiples of 8; base 16-byte aligned); the caller has already written the tree
 * nodes' K/V to rows seq_lens[b] + i.  seq_lens [B] device int32 (0 is legal).
 * scale == 0 means 1/sqrt(D).  status[b] = MTV_ERR_CAPACITY if seq_lens[b] + T > Lcap.
 * Precondition at head size 128 when one sequence's keys are split over several thread-block
 * pairs (few, long sequences: B * Hkv * ceil(T*Hq/Hkv / 256) at most half the pairs the device
 * holds): the splits of a query block meet inside the launch through counters in the workspace,
 * so all blocks of the launch must be resident at once.  The grid is sized to fit an idle
 * device (one block per SM); do not run the call while another long-running kernel occupies
 * SMs of the same device (other streams, other processes under MPS).  If the blocks cannot
 * meet, the bounded waits run out after about a second, the tree's device error word reads
 * MTV_ERR_TIMEOUT and the output is undefined — the call never hangs.  Calls that share a
 * tree or a workspace must not overlap on the device.  The encoded tensor maps of (pointer,
 * shape, strides) are kept in a process-wide table; a mutex guards it, so calls from several
 * host threads are safe.
 * Development build option -DMTV_TRACE: the head-size-128 kernel stamps the cycle counter at
 * its phases into a buffer given by mtv_trace_set (absent from normal builds).
 */
int tree_verify_attention(const mtv_tree_t *tree, int B, int Hq, int Hkv, int D,
                          const mtv_bf16 *q, const mtv_bf16 *k_cache, const mtv_bf16 *v_cache,
                          int64_t stride_b, int64_t stride_h, int64_t stride_t, int Lcap,
                          const int32_t *seq_lens, float scale,
                          mtv_bf16 *out, int32_t *status,
                          void *ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------
 * Acceptance + token retrieval — Section 3.2, "Zero-Copy Retrieval": the best path
 * index is found by the acceptance criterion and the final token sequence is
 * gathered from the candidates through retrieve_indices, all on the device.
 *   am[b][i]  = argmax_v logits[b][i][v]                        (ties: lowest v)
 *   len_p     = number of leading j >= 1 with tree_tok[b][ri[p][j]] == am[b][ri[p][j-1]]
 *   best_path = argmax_p len_p (ties: lowest p);  accept_len = len_best in [0, K]
 *   acc_nodes[b][0..accept_len] = ri[best][..], acc_tok = tree_tok at those nodes, -1 padded
 *   next_root[b] = am[b][acc_nodes[b][accept_len]]
 * All pointers device.  logits [B][T][V] bf16 (base-model logits at every tree node), base
 * address 16-byte aligned (rows are scanned in 16-byte chunks; a misaligned base is refused
 * with MTV_ERR_INVALID_ARG and nothing is launched; V need not be a multiple of 8).
 * Outputs: accept_len, best_path, next_root [B]; acc_nodes, acc_tok [B][K+1].
 * Host threads: the per-device launch set-up is remembered in plain flags; two threads that
 * make their first call on a device at the same time both do the (idempotent) set-up.
 */
int tree_accept(const mtv_tree_t *tree, int B, int V, const mtv_bf16 *logits, const int32_t *tree_tok,
                int32_t *accept_len, int32_t *best_path, int32_t *acc_nodes, int32_t *acc_tok,
                int32_t *next_root, void *ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------
 * LM-head projection fused with the per-node argmax — the base model's last layer as the
 * acceptance of Section 3.2 consumes it: only the most likely token at every tree node is
 * needed, so the [B][T][V] logits are never written.
 *   am[b][i]     = argmax_v <x[b][i], W[v]>                      (ties: lowest v)
 *   am_val[b][i] = that maximum
 * bf16 inputs, products accumulated in fp32 on the tensor cores; the comparison is made on
 * the fp32 sums (no rounding to bf16 first, unlike tree_accept on stored bf16 logits).
 * All pointers device.  x [B][T][H] (final hidden state of the tree nodes, after the last
 * norm), W [V][H] row-major (the LM head), both bf16, 16-byte aligned; H a multiple of 64.
 * keys [B*T] uint64, written by the call (zeroed, then filled): per node the order-preserving
 * image of the maximum in the high word and 0xffffffff - argmax in the low word — the input of
 * tree_accept_keys.  am [B*T] int32 and am_val [B*T] float may be NULL (am_val only if am is).
 * No workspace.  A wait inside the kernel that runs out sets the tree's device error word
 * (mtv_device_error) to MTV_ERR_TIMEOUT; the outputs are then undefined.
 * Errors: MTV_ERR_INVALID_ARG (null / misaligned pointers, sizes < 1),
 * MTV_ERR_UNSUPPORTED_SHAPE (H), MTV_ERR_CUDA.
 */
int lm_head_argmax(const mtv_tree_t *tree, int B, int H, int V, const mtv_bf16 *x, const mtv_bf16 *W,
                   int32_t *am, float *am_val, unsigned long long *keys, void *stream);

/* tree_accept on the keys of lm_head_argmax instead of stored logits: same outputs, same
 * acceptance rule (Section 3.2), am[b][i] taken from keys[b*T + i].  All pointers device. */
int tree_accept_keys(const mtv_tree_t *tree, int B, const unsigned long long *keys, const int32_t *tree_tok,
                     int32_t *accept_len, int32_t *best_path, int32_t *acc_nodes, int32_t *acc_tok,
                     int32_t *next_root, void *stream);

/* ---------------------------------------------------------------------------
 * tree_accept without a workspace — the paper has no counterpart; this is a convenience of
 * the library.  Same inputs, outputs and results as tree_accept, but the scratch (the
 * per-chunk argmax keys) sits in a 64 KB array that is part of the library image, so the call
 * needs no buffer from the caller and the library never calls cudaMalloc / cudaFree for it.
 * It is meant for callers that are not allowed to allocate device memory: a plugin inside a
 * serving runtime that owns the whole device heap, a latency-critical decode loop in which an
 * allocator call (it may synchronise the device) is banned, a process whose memory budget was
 * fixed at start-up.
 *   - Limit: B * T * splits * 8 bytes <= tree_accept_static_scratch_capacity() (65536), i.e.
 *     up to 8192 logit rows; beyond that the call returns MTV_ERR_WORKSPACE, launches nothing,
 *     and mtv_last_error() says how much was needed.
 *   - The first call on a device looks up the array's device address (one runtime query, no
 *     allocation) and remembers it; make that first call outside any stream capture and with
 *     the device current that later calls will use.
 *   - Every GPU that loads the library holds the 64 KB until the process exits.
 *   - All calls on a device share the array and it keeps the previous call's contents; each call
 *     overwrites every entry it later reads, so nothing has to be cleared.  Two calls that
 *     overlap on the GPU (different streams) race on it: keep them stream-ordered.
 */
int tree_accept_static_scratch(const mtv_tree_t *tree, int B, int V, const mtv_bf16 *logits,
                               const int32_t *tree_tok, int32_t *accept_len, int32_t *best_path,
                               int32_t *acc_nodes, int32_t *acc_tok, int32_t *next_root, void *stream);
size_t tree_accept_static_scratch_capacity(void);

/* ---------------------------------------------------------------------------
 * KV compaction — Section 3.2, "Zero-Copy Retrieval" applied to K/V: for every layer,
 * sequence b, KV head g and j = 1..accept_len[b], row seq_lens[b] + acc_nodes[b][j]
 * moves to row seq_lens[b] + j, in place (all sources are read before any row is
 * written); then seq_lens[b] += accept_len[b] + 1.
 * k_caches / v_caches: device arrays of n_layers device pointers, every cache with
 * the strides of tree_verify_attention.  seq_lens is read and updated on the device.
 * status[b] = MTV_ERR_CAPACITY (and b is skipped) if seq_lens[b] + T > Lcap.
 */
int kv_compact_accepted(const mtv_tree_t *tree, int B, int Hkv, int D, int n_layers,
                        mtv_bf16 *const *k_caches, mtv_bf16 *const *v_caches,
                        int64_t stride_b, int64_t stride_h, int64_t stride_t, int Lcap,
                        int32_t *seq_lens, const int32_t *accept_len, const int32_t *acc_nodes,
                        int32_t *status, void *stream);

/* ---------------------------------------------------------------------------
 * One whole verification step (the order of Section 3.2's pipeline), enqueued on
 * one stream with no host involvement: heads -> attention for each of n_layers
 * caches -> acceptance -> compaction.  Device pointers throughout.
 * q_layers / out_layers: [n_layers][B][T][Hq][D] contiguous.
 */
typedef struct {
    int32_t B, H, V, Hq, Hkv, D, n_layers, Lcap;
    int64_t stride_b, stride_h, stride_t;
    float scale;
    const mtv_bf16 *hidden, *W1, *b1, *W2;
    const int32_t *root_tok;
    const mtv_bf16 *q_layers;
    mtv_bf16 *const *k_caches; /* device array [n_layers] */
    mtv_bf16 *const *v_caches; /* device array [n_layers] */
    mtv_bf16 *const *k_caches_host; /* host copy of the same pointer array */
    mtv_bf16 *const *v_caches_host;
    const mtv_bf16 *logits;    /* [B][T][V] */
    int32_t *seq_lens;         /* [B] in/out */
    int32_t *cand; float *cand_logit; int32_t *tree_tok;
    mtv_bf16 *out_layers;
    int32_t *accept_len, *best_path, *acc_nodes, *acc_tok, *next_root;
    int32_t *status;           /* [B] or NULL */
    void *ws; size_t ws_bytes;
    /* Optional: the acceptance takes the base model's argmax from the fused LM head instead of
     * stored logits.  If x_final ([B][T][H], final hidden state of the tree nodes) and W_lm
     * ([V][H]) are both non-NULL, the step runs lm_head_argmax on them followed by
     * tree_accept_keys and never reads `logits` (which may then be NULL); the keys live at the
     * start of ws.  The host variant uploads x_final instead of logits. */
    const mtv_bf16 *x_final, *W_lm;
} mtv_step_args;

int mtv_verify_step(const mtv_tree_t *tree, const mtv_step_args *args, void *stream);

/* ---------------------------------------------------------------------------
 * A chain of n_steps verification steps enqueued on one stream with no host decision between
 * them — Section 3.2: the step is one static graph without dynamic control flow, and nothing
 * the next step needs (the accepted length, the compacted cache, the next root token) passes
 * through the CPU.  steps[s] describes step s as for mtv_verify_step; within a chain
 *   - steps[s].root_tok == NULL (s >= 1) means "the previous step's next_root" (device pointer
 *     steps[s-1].next_root, read when step s runs);
 *   - all steps share one seq_lens array, advanced on the device by every step's compaction.
 * appends (NULL, or n_steps entries): where appends[s].k_new_layers / v_new_layers are given,
 * step s first writes its tree nodes' K/V rows into the caches — all layers in one launch of
 * tree_kv_append_rope's kernel, directly in front of the step's first attention call, which
 * starts its set-up under that kernel's tail (programmatic dependent launch) — and rotates
 * steps[s].q_layers in place (so that buffer must be writable although the struct says const).
 * k_new_layers, v_new_layers: [n_layers][B][T][Hkv][D] device, un-rotated K rows and V rows;
 * rope_theta == 0 means 10000.  Per-step inputs that a backbone would compute from the previous
 * step's tokens (hidden, q, k_new, v_new, logits / x_final) are the caller's, laid out per step
 * before the call: the backbone is outside this library.
 * Errors: as the calls it chains; MTV_ERR_INVALID_ARG for a first step without root_tok or
 * steps that name different seq_lens.  Nothing is rolled back when a later step is refused. */
typedef struct {
    const mtv_bf16 *k_new_layers, *v_new_layers;
    float rope_theta;
} mtv_append_args;

int mtv_verify_steps(const mtv_tree_t *tree, const mtv_step_args *steps, const mtv_append_args *appends,
                     int n_steps, void *stream);

/* The same step for a caller whose per-step tensors live in (pinned) host memory.
 * Copies hidden, root_tok, q_layers and logits host->device into the device
 * buffers named in `dev`, runs the step, copies tree_tok, out_layers,
 * accept_len, best_path, acc_nodes, acc_tok, next_root and seq_lens back to the
 * host buffers, and synchronises the stream before returning.  Weights, KV caches
 * and the tree stay resident on the device.  `host` uses the same struct: only
 * the fields listed above are read from it.
 * The transfers overlap the compute on two copy streams that the library creates
 * on first use: queries and logits go up while the heads run, the attention
 * outputs come down in groups of layers while later layers run.  Unlike the other
 * step calls this one is therefore neither allocation-free on its first call nor
 * capturable; use pinned host buffers, or the copies serialise. */
int mtv_verify_step_host(const mtv_tree_t *tree, const mtv_step_args *dev, const mtv_step_args *host,
                         void *stream);

/* ---------------------------------------------------------------------------
 * One sequence's step split over several GPUs (the paper runs on one device and has no counterpart; the
 * split follows its structure: the heads of Section 3.1 are independent over the vocabulary, the tree
 * attention of Section 3.2 over KV heads).  Each rank runs the ordinary calls on its slice — medusa_heads_topk
 * on the vocabulary slab [r * v_slab, min(V, (r+1) * v_slab)) of W2 (W1 replicated), tree_verify_attention on
 * its Hkv / n KV heads and their Hq / n query heads, lm_head_argmax on its slab of W_lm —, a collective outside
 * this library (NCCL all-gather) brings all ranks' results into LOCAL buffers, and the calls below merge them.
 * No kernel of this library is ever given another GPU's memory.  All pointers device.
 *
 * heads_merge_shards: cand_shards [n_shards][B][C] (ids local to the slab, slot 0 unused), logit_shards
 *   [n_shards][B][C-1] as medusa_heads_topk wrote them on each rank -> cand, cand_logit (may be NULL), tree_tok
 *   as medusa_heads_topk on the whole vocabulary writes them: per head the k_d best of the n_shards * k_d entries
 *   by (logit descending, global id ascending), the same order, so the ids are identical.  Every slab must hold
 *   at least max k_d rows.  ws: B * 4 bytes.  n_shards <= 16.
 * attn_interleave_shards: gathered [n_shards][rows][Hq_local][D] (rows = B * T) -> out [rows][n_shards * Hq_local][D].
 * keys_merge_shards: key_shards [n_shards][n] from lm_head_argmax on each slab (n = B * T) -> keys [n] for
 *   tree_accept_keys, the slab offsets folded into the index half; ties across slabs go to the lowest global id.
 */
/* Per-node argmax keys of stored logits [B][T][V] (16-byte aligned base, as for tree_accept), in the form
 * tree_accept_keys and keys_merge_shards read: keys [B*T]; ws as for tree_accept.  tree_accept(logits) equals
 * node_argmax_keys followed by tree_accept_keys; a rank that holds the vocabulary slab [B][T][v_local] of the logits
 * runs it on its slab, and keys_merge_shards over the gathered keys gives the keys of the whole vocabulary. */
int node_argmax_keys(const mtv_tree_t *tree, int B, int V, const mtv_bf16 *logits, unsigned long long *keys,
                     void *ws, size_t ws_bytes, void *stream);
int heads_merge_shards(const mtv_tree_t *tree, int B, int n_shards, int v_slab, const int32_t *cand_shards,
                       const float *logit_shards, const int32_t *root_tok, int32_t *cand, float *cand_logit,
                       int32_t *tree_tok, void *ws, size_t ws_bytes, void *stream);
int attn_interleave_shards(int rows, int n_shards, int Hq_local, int D, const mtv_bf16 *gathered, mtv_bf16 *out,
                           void *stream);
int keys_merge_shards(int n, int n_shards, int v_slab, const unsigned long long *key_shards,
                      unsigned long long *keys, void *stream);

/* ---------------------------------------------------------------------------
 * Measurement aid (the paper has no counterpart): per-kernel device timing.
 * While taps are set for a kernel id, every launch of that kernel by this library is
 * bracketed by cudaEventRecord(start[i]) / cudaEventRecord(stop[i]) on the launch
 * stream, i = 0, 1, ... until `capacity` launches have been recorded; later launches
 * are not recorded.  start/stop: host arrays of cudaEvent_t created by the caller and
 * kept alive until the taps are cleared (capacity = 0 or NULL arrays clears them).
 * Not thread-safe; do not use during stream capture.
 */
#define MTV_KERNEL_HEADS_RESBLOCK 0
#define MTV_KERNEL_HEADS_VOCAB_TOPK 1
#define MTV_KERNEL_HEADS_MERGE 2
#define MTV_KERNEL_ATTN_PARTIAL 3
#define MTV_KERNEL_ATTN_COMBINE 4
#define MTV_KERNEL_ARGMAX_PARTIAL 5
#define MTV_KERNEL_ACCEPT_FINISH 6
#define MTV_KERNEL_KV_COMPACT 7
#define MTV_KERNEL_SEQ_ADVANCE 8
#define MTV_KERNEL_COUNT 9
int mtv_set_kernel_taps(int kernel_id, void **start_events, void **stop_events, int capacity);
/* Number of launches recorded since the taps of kernel_id were set (-1: bad id). */
int mtv_kernel_taps_used(int kernel_id);

/* Sticky device-side error word of the device the tree was uploaded to (the paper has
 * no counterpart).  A kernel whose bounded wait ran out (a copy or a tensor-core
 * operation that never signalled completion) stores MTV_ERR_TIMEOUT there and unwinds
 * instead of spinning; the outputs of that call are then undefined.  *code receives
 * the word (0 = no error since it was last cleared); clear != 0 resets it.  This call
 * synchronises with the device: use it between steps, not inside one. */
int mtv_device_error(const mtv_tree_t *tree, int clear, int32_t *code);

/* Self-test of that mechanism (the paper has no counterpart): one warp waits, with the same
 * bounded wait the hot kernels use, on a shared-memory barrier that nothing ever arrives on.
 * After about a second of SM cycles the wait gives up, the kernel stores MTV_ERR_TIMEOUT in the
 * tree's device error word and returns normally: nothing faults, the context stays usable.
 * Only enqueues the kernel; read the word with mtv_device_error afterwards. */
int mtv_selftest_wait_timeout(const mtv_tree_t *tree, void *stream);

/* 1 if the library was compiled with -DMTV_DEBUG_BOUNDS, else 0 (the paper has no counterpart).  That build
 * checks every index that a kernel reads from device memory before it is used as an address — tree tables,
 * acc_nodes / accept_len handed to the compaction, the length-ranked sequence order — records MTV_ERR_BOUNDS in the
 * tree's device error word and skips the access instead of following it: a stand-in for a memory checker
 * where none can be run.  Results are otherwise identical; the checks cost a few instructions per index. */
int mtv_debug_bounds_enabled(void);

/* Human-readable text for the most recent MTV_ERR_CUDA (or refused size) on this thread (never NULL). */
const char *mtv_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* MTV_H_ */
