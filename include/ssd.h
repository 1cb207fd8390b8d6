/*
 * ssd.h - C ABI of the B200 (sm_100a) Self Speculative Decoding library.
 *
 * The library runs the hot path of SSD for masked-diffusion language models: per block of
 * the semi-autoregressive schedule (Eq. 3) it turns the model's own drafts for the masked
 * positions (Eq. 4) into the greedy verification chain of N+1 nodes (Section 3.2.3), runs all
 * nodes through the model in ONE forward against the cached prefix K/V (Eq. 5), and accepts
 * the longest draft prefix that one-token-per-step decoding would also have produced
 * (Section 3.2.4, Algorithm 1).  The tokens it returns are those of stepwise decoding.
 *
 * General rules
 *  - Every function returns SSD_OK (0) or a negative SSD_ERR_* code; ssd_last_error() gives a
 *    message.  Nothing aborts, traps or throws across this boundary.  Arguments are checked on
 *    the host before any kernel is launched.
 *  - "host" pointers are ordinary host memory owned by the caller and only used during the
 *    call.  "device" pointers are CUDA device memory of the current device.
 *  - All device work is enqueued on the stream given to ssd_create().  Calls that return
 *    results in host memory synchronise that stream before returning.
 *  - A context is not thread-safe; use one per host thread / GPU.
 *  - There is no CPU fallback: without a CUDA device ssd_create() fails with SSD_ERR_CUDA.
 */
#ifndef SSD_B200_H_
#define SSD_B200_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SSD_OK                0
#define SSD_ERR_INVALID_ARG  (-1)   /* null pointer, negative size, unknown name or enum          */
#define SSD_ERR_SHAPE        (-2)   /* a shape the kernels do not support, or a mismatching one   */
#define SSD_ERR_OOM          (-3)   /* device or host allocation failed                           */
#define SSD_ERR_CUDA         (-4)   /* a CUDA runtime / driver call failed                        */
#define SSD_ERR_OVERFLOW     (-5)   /* cached length + block would exceed max_seq, batch too big  */
#define SSD_ERR_TIMEOUT      (-6)   /* a bounded device-side wait expired (kernel bailed out)     */
#define SSD_ERR_STATE        (-7)   /* call out of order (weights missing, no prefill, ...)       */
#define SSD_ERR_NONFINITE    (-8)   /* a confidence came out NaN/Inf (non-finite weights?)        */

#define SSD_DTYPE_BF16 0
#define SSD_DTYPE_F32  1

#define SSD_MODE_STEPWISE 0   /* one token per forward (the lossless reference behaviour, Fig. 2)  */
#define SSD_MODE_SSD      1   /* self speculative decoding, greedy chain                           */

typedef struct ssd_ctx ssd_ctx;   /* opaque: owns weights copy, KV cache, workspaces, decode state */

/* Model f_theta (Eq. 2: a bidirectional transformer; pre-norm RMSNorm, rotary embedding with the
 * rotate-half pairing, grouped-query attention without mask, SwiGLU, untied LM head, no biases)
 * and decode limits. */
typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  int32_t mask_id;          /* id of the mask token m_i of Eq. 1; never predicted                  */
  float   rope_theta, rms_eps;
  int32_t max_batch;        /* sequences decoded in lockstep, each with its own tree               */
  int32_t max_seq;          /* P + L of Eq. 1: capacity of the KV cache per sequence               */
  int32_t block_len;        /* B of Eq. 3                                                          */
  int32_t max_drafts;       /* cap on the draft length N (Section 3.2.2); >= block_len-1 means the
                               chain may cover the whole block; 0 makes SSD mode equal stepwise    */
} ssd_config;

/* Supported shapes: head_dim 64 or 128; d_model, d_ffn, n_heads*head_dim multiples of 8;
 * n_heads a multiple of n_kv_heads; block_len <= 256.  `cuda_stream` is a cudaStream_t (NULL =
 * legacy default stream).  Allocates everything the context will ever need. */
int ssd_create(const ssd_config* cfg, void* cuda_stream, ssd_ctx** out);
void ssd_destroy(ssd_ctx* ctx);
const char* ssd_last_error(const ssd_ctx* ctx);   /* ctx may be NULL: message of a failed create */

/* Copy one weight tensor into the context (the library keeps its own bf16, re-laid-out copy; the
 * caller may free `dev_ptr` afterwards).  `dev_ptr` is DEVICE memory, row-major, `shape[ndim]`,
 * of type SSD_DTYPE_BF16 or SSD_DTYPE_F32 (fp32 matrices are rounded to bf16, the arithmetic
 * type of every contraction here; norm gains stay fp32).  Names: "embed" [V,d], "lm_head" [V,d],
 * "norm_final" [d], and for layer l "layers.l.wq" [H*hd,d], ".wk"/".wv" [Hkv*hd,d], ".wo"
 * [d,H*hd], ".w_gate"/".w_up" [ffn,d], ".w_down" [d,ffn], ".norm_attn"/".norm_ffn" [d]
 * (matrices are [out_features, in_features]).  Synchronises the stream. */
int ssd_load_weights(ssd_ctx* ctx, const char* tensor_name, const void* dev_ptr, int32_t dtype,
                     const int64_t* shape, int32_t ndim);

/* Eq. 1 initial state: forward of the prompts (each prompt attends to itself only) that fills
 * the prefix K/V cache.  `prompt_ids` HOST [batch, prompt_len], ids in [0, vocab), no mask id
 * required.  Resets the decode position to prompt_len.  1 <= batch <= max_batch.  The prompts of a batch
 * share forwards of up to 4096 rows (one stream of the weights for all of them); every sequence's cache is
 * bit for bit what prefilling it alone gives. */
int ssd_prefill(ssd_ctx* ctx, int32_t batch, int32_t prompt_len, const int32_t* prompt_ids);
/* Same with `prompt_ids` in DEVICE memory (no host->device copy of inputs). */
int ssd_prefill_dev(ssd_ctx* ctx, int32_t batch, int32_t prompt_len, const int32_t* prompt_ids_dev);

/* Decode the next block B_j (Eq. 3) for every sequence of the batch (Algorithm 1 restricted to
 * one block, or stepwise decoding), then commit it (see ssd_block_commit: the block's K/V reach
 * the cache with the first forward of the next call).
 *   mode           SSD_MODE_STEPWISE or SSD_MODE_SSD
 *   block_tokens   number of positions in this block: block_len, or less for a ragged last block
 *   out_tokens         HOST [batch, block_tokens]   decoded ids
 *   out_accept_counts  HOST [batch, block_tokens]   tokens accepted by forward 0,1,2,... of each
 *                      sequence, 0-terminated list; each entry in [1, N+1], sum = block_tokens
 *   out_n_forwards     HOST [batch]                 verification forwards the sequence took part in
 * Any out pointer may be NULL.  Errors: SSD_ERR_STATE before prefill, SSD_ERR_OVERFLOW if the
 * cache would exceed max_seq. */
int ssd_decode_block(ssd_ctx* ctx, int32_t mode, int32_t block_tokens, int32_t* out_tokens,
                     int32_t* out_accept_counts, int32_t* out_n_forwards);

/* ---- the same block, one step at a time (used by ssd_decode_block; exposed so that every
 * ---- forward can be checked against a reference with the state forced to the reference's) --- */

/* Start block B_j: all `block_tokens` positions masked, no drafts. */
int ssd_block_begin(ssd_ctx* ctx, int32_t block_tokens);
/* Overwrite the state of the current block.  HOST arrays [batch, block_tokens]: ids (value
 * ignored where masked), masked (0/1), and either both draft_tok/draft_conf (drafts for the
 * masked positions, Eq. 4) or both NULL (no drafts: next forward is root-only). */
int ssd_set_block_state(ssd_ctx* ctx, const int32_t* ids, const uint8_t* masked,
                        const int32_t* draft_tok, const float* draft_conf);
/* Read the state back; any pointer may be NULL.  draft arrays are zero where not masked. */
int ssd_get_block_state(ssd_ctx* ctx, int32_t* ids, uint8_t* masked, int32_t* draft_tok, float* draft_conf);
/* The same for the next block's half of the window (only for a block begun with option "cross_block" > 0):
 * HOST arrays [batch, cross_block].  ssd_set_block_state resets this half to "all masked, no drafts". */
int ssd_set_next_block_state(ssd_ctx* ctx, const int32_t* ids, const uint8_t* masked,
                             const int32_t* draft_tok, const float* draft_conf);
int ssd_get_next_block_state(ssd_ctx* ctx, int32_t* ids, uint8_t* masked, int32_t* draft_tok, float* draft_conf);
/* One iteration of Algorithm 1's loop for every unfinished sequence: candidate selection with
 * draft length N = min(max_drafts, masked-1) (0 if there are no drafts), chain of N+1 nodes,
 * one batched forward, traversal, state and draft update.  `max_drafts` < 0 uses the config's;
 * 0 gives a stepwise step.  accepted HOST [batch] (0 for finished sequences), n_nodes HOST
 * [batch]; both may be NULL. */
int ssd_block_step(ssd_ctx* ctx, int32_t max_drafts, int32_t* accepted, int32_t* n_nodes);
/* Dual cache (Section 4.1; option "dual_cache"): recompute the K/V of EVERY position of every sequence -
 * prompt, decoded blocks, the block in progress (MASK where still masked) and the still masked rest - by one
 * forward per sequence in which all positions see all positions.  ssd_block_step / ssd_decode_block call it
 * on their own at every block start and after every "refresh_interval" decoded tokens; exposed so that a
 * forward can be compared with a reference from a known cache.  ssd_refresh_count: refresh forwards so far. */
int ssd_refresh_cache(ssd_ctx* ctx);
int64_t ssd_refresh_count(const ssd_ctx* ctx);

/* Test hook: (token, confidence) of the first n_rows rows of the latest forward, in its row order
 * [sequence slot][node][rows of the node] (a node's rows: a finished block riding in front, if any, the
 * current block, the next block's half of a window, if any); -1 / 0 on rows nothing was asked of. */
int ssd_read_forward_outputs(ssd_ctx* ctx, int32_t n_rows, int32_t* out_tok, float* out_conf);
/* Commit the (fully unmasked) block: its K/V are appended to the prefix cache and
 * ssd_cache_length grows by the block.  The paper leaves open how a block's K/V reach the cache;
 * here it is one forward over the block's final tokens, and by default that forward is not run
 * by itself: the block waits and rides in front of the first ssd_block_step of the next block,
 * per sequence one causal chain [finished block | next block], which is the commit forward and
 * the next block's root forward in one weight stream.  A call that needs the complete cache
 * first (ssd_verify_forward, ssd_read_cache, ssd_set_block_state, a rewind into the waiting
 * block) runs the waiting commit on its own; a waiting block that is rewound away or followed
 * by a new prefill is never committed.  Option "fuse_commit" = 0 commits here, at once. */
int ssd_block_commit(ssd_ctx* ctx);

/* The verification forward alone (Eq. 5) on caller-given node rows, against the current cache;
 * the decode state is not touched.  HOST arrays: node_ids [batch, n_nodes, block_tokens],
 * node_masked same shape (1 = this row's prediction is wanted); out_tok / out_conf same shape
 * (token = argmax with the mask id excluded, lowest id on ties; conf = its softmax probability;
 * -1 / 0 on rows not masked); out_logits [batch, n_nodes, block_tokens, vocab] fp32 or NULL
 * (debug: materialises the logits, which the normal path never does). */
int ssd_verify_forward(ssd_ctx* ctx, int32_t batch, int32_t n_nodes, int32_t block_tokens,
                       const int32_t* node_ids, const uint8_t* node_masked,
                       int32_t* out_tok, float* out_conf, float* out_logits);

/* The verification forward with the `k` most probable tokens per wanted row instead of the single best
 * (Section 5.1: the candidates a k-ary verification tree would draw from).  1 <= k <= 8.  HOST outputs
 * out_tok / out_prob [batch, n_nodes, block_tokens, k]: tokens by descending softmax probability (mask id
 * excluded, lower id first among equals) and those probabilities; -1 / 0 on rows not masked.  out_tok[..., 0]
 * and out_prob[..., 0] are what ssd_verify_forward returns.  The logits still never reach HBM: the LM-head
 * epilogue ranks every 128-entry vocabulary tile on chip and a merge kernel ranks the tiles' lists. */
int ssd_verify_forward_topk(ssd_ctx* ctx, int32_t batch, int32_t n_nodes, int32_t block_tokens,
                            const int32_t* node_ids, const uint8_t* node_masked, int32_t k,
                            int32_t* out_tok, float* out_prob);

/* Acceptance-rate limit of self-drafting (Section 5.1, Table 2), measured on the next block: the block is
 * decoded stepwise (the tokens are those of SSD_MODE_STEPWISE) in rounds of draft_len + 1 forwards; the
 * forward that opens a round is the draft and its top-k_max tokens per position are kept on the device;
 * every later token of the round is looked up in them.  out_matched HOST [k_max]: tokens, summed over the
 * batch, that lay within the draft's top k for k = 1 .. k_max - tokens a verification tree over the top-k
 * candidates could have accepted without a forward of their own; out_steps HOST [1]: forwards x sequences
 * stepwise decoding took.  matched[k-1] / steps is Table 2's reduction ratio, bounded by
 * draft_len / (draft_len + 1).  out_tokens HOST [batch, block_tokens] or NULL.  Commits the block like
 * ssd_decode_block. */
int ssd_probe_acceptance_limit(ssd_ctx* ctx, int32_t block_tokens, int32_t draft_len, int32_t k_max,
                               int32_t* out_tokens, int64_t* out_matched, int64_t* out_steps);

/* Read cached K (post-rotary) and V of one layer and sequence: HOST fp32
 * [length, n_kv_heads, head_dim] each, positions [0, length).  Test hook for cache semantics. */
int ssd_read_cache(ssd_ctx* ctx, int32_t layer, int32_t seq, int32_t length, float* out_k, float* out_v);

/* The reverse: overwrite cached K (post-rotary) and V of one layer and sequence, positions
 * [0, length), from HOST fp32 [length, n_kv_heads, head_dim] (rounded to bf16, the cache's type).
 * Test hook: lets a reference supply the prefix of a layer-by-layer comparison.  Does not change
 * ssd_cache_length. */
int ssd_write_cache(ssd_ctx* ctx, int32_t layer, int32_t seq, int32_t length, const float* k, const float* v);

/* Layers [layer_begin, layer_end) of the verification forward (Eq. 5) on a caller-given residual
 * stream, against the current cache: `h_in` HOST fp32 [batch * n_nodes * block_tokens, d_model] is
 * the stream entering layer_begin, `h_out` (same shape, may be NULL) the stream leaving
 * layer_end - 1.  With layer_end == n_layers, out_tok / out_conf (HOST [batch, n_nodes,
 * block_tokens], may be NULL) receive the LM-head statistics of every row.  Test hook: each layer can
 * be checked against a reference from the reference's own input, so that rounding noise does not
 * compound over the depth.  The decode state is not touched. */
int ssd_verify_layers(ssd_ctx* ctx, int32_t batch, int32_t n_nodes, int32_t block_tokens,
                      int32_t layer_begin, int32_t layer_end, const float* h_in, float* h_out,
                      int32_t* out_tok, float* out_conf);

/* Cached prefix length S (prompt + committed blocks, a block that waits for its commit
 * included), or a negative error. */
int ssd_cache_length(const ssd_ctx* ctx);

/* Forget the blocks committed after position `length` (prompt_len <= length <= current length):
 * the next block is decoded at `length` again.  The prompt's K/V stay valid, so several
 * generations from one prefill cost one prefill.  Abandons a block in progress. */
int ssd_rewind(ssd_ctx* ctx, int32_t length);

/* The skinny projection kernel alone: out[r][n] = sum_k x[r][k] * w[n][k] with bf16 operands and
 * fp32 accumulation, split over `split_k` K ranges that are summed in order.  DEVICE pointers:
 * x [rows, k] bf16, w [n, k] bf16, out [rows, n] fp32.  k a multiple of 8.  Test / tuning hook. */
int ssd_gemm_bf16(ssd_ctx* ctx, const void* x_dev, const void* w_dev, float* out_dev,
                  int32_t rows, int32_t n, int32_t k, int32_t split_k);

/* The same projection for callers that cannot allocate device memory while they run (the paper has
 * no counterpart: this is a deployment aid).  Think of a server that handed the whole GPU to its own
 * arena at start-up, or of a latency-critical loop that may not make a call which can block on the
 * device or run out of memory: neither can use a context, whose creation allocates.  This entry point
 * needs no context and calls no cudaMalloc/cudaFree nor any allocating library routine: its split-K
 * scratch is a fixed 4 MiB array inside the library image (each GPU that loads the library holds it
 * until the process exits).
 *   x_dev [rows,k] bf16, w_dev [n,k] bf16, out_dev [rows,n] fp32: DEVICE memory of the current device,
 *   owned by the caller; k a multiple of 8; 1 <= split_k <= 8; `cuda_stream` a cudaStream_t.
 *   Limit: split_k * rows * n <= 1048512 floats (4 MiB minus a 256-byte flag area), else
 *   SSD_ERR_OVERFLOW; bad shapes SSD_ERR_SHAPE; null pointers SSD_ERR_INVALID_ARG.
 * The first call on each device looks up the array's device address (with that device current); under
 * the driver's lazy module loading that is also when the array and the kernels are placed on the device, so
 * make that first call early - before the host's arena takes the remaining memory and before starting any
 * stream capture.  Later calls take no device memory at all.  All calls share the one array, which
 * keeps the previous call's contents (the error word is cleared at the start of every call): two
 * calls whose GPU work overlaps - different streams or threads - race on it, so serialise them.
 * Synchronises the stream before returning; same result as ssd_gemm_bf16. */
int ssd_gemm_bf16_noalloc(const void* x_dev, const void* w_dev, float* out_dev, int32_t rows, int32_t n,
                          int32_t k, int32_t split_k, void* cuda_stream);

/* ---- measurement ---------------------------------------------------------------------------- */

/* Kernel launches issued by this context since creation (all streams of the context). */
int64_t ssd_launch_count(const ssd_ctx* ctx);

/* Per-kernel-family device time.  ssd_profile_enable(ctx, mode):
 *   0  off;
 *   1  every launch is bracketed by CUDA events on the context's stream: the kernel alone, without the
 *      overlap with its neighbours that dependent launches give it (this serialises the stream; do
 *      not time throughput in this mode);
 *   2  the live stream: a one-thread marker kernel behind every launch records the time that launch
 *      completed, and a launch is charged the time from its predecessor's completion to its own (so
 *      the charges add up to the wall time; each marker adds about a microsecond of dependency
 *      latency).
 * ssd_profile_read fills, for family f in [0, SSD_PROF_FAMILIES): launches[f], milliseconds[f],
 * algorithmic bytes[f] (operand bytes that must cross HBM once), and resets the counters. */
#define SSD_PROF_GEMM      0   /* QKV / O / gate-up / down projections                         */
#define SSD_PROF_LMHEAD    1   /* LM head fused with softmax statistics                        */
#define SSD_PROF_ATTN      2   /* shared-prefix attention (+ split merge)                      */
#define SSD_PROF_ELEMWISE  3   /* embedding, norms, residuals, rotary, reductions              */
#define SSD_PROF_TREE      4   /* tree build, acceptance                                       */
#define SSD_PROF_GEMM_QKV  5   /* families 5-8 break family 0 down by projection               */
#define SSD_PROF_GEMM_O    6
#define SSD_PROF_GEMM_GU   7
#define SSD_PROF_GEMM_DOWN 8
#define SSD_PROF_FAMILIES  9
int ssd_profile_enable(ssd_ctx* ctx, int32_t on);
int ssd_profile_read(ssd_ctx* ctx, int64_t* launches, double* milliseconds, double* bytes);

/* Tuning knobs (set before prefill).  key:
 *   "split_k_qkv", "split_k_o", "split_k_down"  split-K factor of a projection: 1..16 for QKV, 1..8 for
 *        the O and down projections (they reduce their splits inside a thread-block cluster), never
 *        more than the projection has 64-wide K blocks, bounded by the split-K workspace;
 *   "kv_split"   prefix keys per attention part, a multiple of 64; 0 = 128; raised automatically (in
 *        steps of 128) while a prefix would need more than 7 parts;
 *   "max_drafts" lower the draft-length cap below the capacity fixed at creation;
 *   "gemm_max_stages" tuning: cap on the depth of the projection kernel's shared-memory ring (0 = as deep as
 *        two CTAs per SM allow, the default); changes no result;
 *   "wait_limit_us" bound of every device-side barrier wait of the projection kernel in microseconds (0 = the
 *        default of 2 s): when it runs out the kernel raises an error word, lets its copies in flight land,
 *        frees its tensor memory and returns, and the call reports SSD_ERR_TIMEOUT; the context stays usable;
 *   "starve_gemm_kb" test hook for ssd_gemm_bf16 (split_k 1, up to 256 rows): > 0 makes the kernel's producer
 *        leave out the copies of that K block (1-based), so that the wait for it provably runs out; 0 = off;
 *   "dual_cache" P + L > 0 = the dual cache of the paper's set-up (Section 4.1) instead of the exact prefix
 *        cache: the K/V of all P + L positions are cached, a block forward attends to every position outside
 *        the block (prefix and still masked suffix) plus its own rows, and the cache is refreshed by a
 *        full-sequence forward at every block start and after every "refresh_interval" (default 8) decoded
 *        tokens.  Between refreshes the cached K/V are stale (an approximation), so stepwise decoding is
 *        defined with the schedule, and SSD caps every chain at refresh_interval - decoded - 1 drafts so that
 *        no forward accepts past a refresh point: the tokens stay those of stepwise decoding under the same
 *        schedule.  Blocks are not committed (the next refresh recomputes them).  Set after ssd_prefill,
 *        outside a block; 0 = off (default);
 *   "refresh_interval" decoded tokens between two refreshes of the dual cache, >= 1;
 *   "cross_block" T2 > 0 = candidates may come from the next block (Section 3.2.2): the block after the next
 *        one to be begun is T2 tokens long.  While a sequence's current block holds more masked positions
 *        than the draft length a forward is unchanged; once it cannot fill the chain (r <= max_drafts) the
 *        nodes of the forward span the window [current block | next block] (block-causal, like the whole
 *        sequence), the candidates are all masked positions of the current block followed by the next
 *        block's most confident drafts, and a node predicts in the next block only once its current block
 *        is full, so nothing of block j+1 is accepted before block j is complete (Section 3.1).  What the
 *        next block has accepted, and its drafts, are kept for its own ssd_block_begin / ssd_decode_block
 *        (same block_tokens); set the option again before every block and to 0 before the last.  The tokens
 *        are still those of stepwise decoding.  A finished block whose commit rides in front of such a
 *        block's first forward makes every node a chain [finished block | node].  0 = off (default);
 *   "mix_order"  1 = the verification tree is the greedy chain plus the mix-order branches of
 *        Section 5.2 (Table 3): every chain node that has a grandchild gets one more child, its state
 *        with candidate i+2 in place of candidate i+1; when a node predicts that candidate (right
 *        tokens, other order) it is accepted together with the branch's own prediction and the walk
 *        ends.  2N nodes instead of N+1; the tokens are still those of stepwise decoding.  The tree
 *        must fit the node capacity fixed at creation (max_drafts + 1 nodes): create the context with
 *        max_drafts >= 2N - 1, then set "max_drafts" to N.  0 = greedy chain (default);
 *   "attn_impl"  1 = attention of the verification forward on tcgen05 where the shape allows (head
 *        dimension 128, parts of whole 128-key tiles, block length dividing 128), the default; 0 = always the
 *        mma.sync form;
 *   "attn_pipe_ctas", "attn_pipe_keys" with attn_impl 1: a prefilled batch that gives at least attn_pipe_ctas
 *        (default 64) pairs (head, sequence) - batch * heads - takes the pipelined tcgen05 form, one CTA per pair
 *        walking all key tiles, instead of the cluster of key parts; one sequence is faster with its key parts
 *        side by side.  attn_pipe_keys (default 1; 0 = never) is the shortest prefix that may take it.
 *        The two forms sum in different orders, so a sequence's bits depend on the prefilled batch SIZE - never
 *        on the other sequences' contents, on the node count, or on which sequences are still unfinished;
 *   "two_sm_rows" the QKV, gate/up and LM-head projections run pairs of weight tiles as ONE tcgen05.mma
 *        with cta_group::2 (two CTAs of a cluster, M = 256, each SM holding half of the activation tile)
 *        from this many padded rows per launch on; 0 = never; default 128, where it starts to pay.  The results
 *        are bit-identical either way;
 *   "fuse_commit" 1 = a block's commit is folded into the next block's first forward (default); 0 = a
 *        commit forward of its own inside ssd_block_commit;
 * Unknown key: SSD_ERR_INVALID_ARG. */
int ssd_set_option(ssd_ctx* ctx, const char* key, int32_t value);

#ifdef __cplusplus
}
#endif
#endif  /* SSD_B200_H_ */
