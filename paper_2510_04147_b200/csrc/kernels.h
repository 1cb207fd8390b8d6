// Internal launcher declarations shared by the translation units of the library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;

namespace ssd {

// ---------------------------------------------------------------- programmatic dependent launch
// Every kernel of the forward is launched with the "programmatic stream serialization" attribute:
// it may become resident while its predecessor in the stream still runs.  A kernel first lets ITS
// successor be scheduled (pdl_launch_dependents), does whatever does not depend on earlier kernels
// (barrier set-up, weight prefetch), and calls pdl_wait() before it touches anything an earlier
// kernel wrote or still reads.  pdl_wait() returns once the predecessor grid has completed and its
// memory operations are visible, so completion is transitive along the stream.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// A cluster dimension > 1 additionally groups that many consecutive CTAs along x (or y) into a
// thread-block cluster.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster_xy(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                         unsigned cluster_x, unsigned cluster_y, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.numAttrs = 1;
  if (cluster_x > 1 || cluster_y > 1) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = cluster_y;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  cfg.attrs = attr;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                      unsigned cluster_x, Args... args) {
  return launch_pdl_cluster_xy(kernel, grid, block, smem, st, cluster_x, 1u, args...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
  return launch_pdl_cluster_xy(kernel, grid, block, smem, st, 1u, 1u, args...);
}
#endif

// ---------------------------------------------------------------- per-device set-up
// Function attributes (the opt-in to large dynamic shared memory) belong to a device, not to the
// process: launchers keep one flag per device ordinal and set the attribute on a device's first use.
constexpr int kMaxDevices = 64;
inline int device_slot() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

// ---------------------------------------------------------------- layout helpers (host+device)
// Rows of a forward are ordered [sequence slot a][node i][in-block index t].
struct RowMap {
  int rows_per_seq;    // n_nodes * T
  int T;               // rows per node (block tokens, or prompt length for prefill)
  int pos0;            // absolute position of t = 0 (= cached prefix length S)
  int seq_base;        // sequence id of slot 0 when seq_map == nullptr
  const int* seq_map;  // device [slots] slot -> sequence id, or nullptr (identity + seq_base)
  // The same map by value when the host knows it and it is short: a kernel may then use it before
  // its dependency wait (the device array is written by an earlier kernel of the same forward).
  int n_inline;        // 0: not given
  int inline_seq[8];
  // > 0: the rows of a sequence are ONE causal chain of two blocks - the first chain_T0 rows are a
  // finished block (they see the prefix and themselves, and their K/V go to the cache), the rest
  // is the next block, which also sees the finished one.  rows_per_seq == T then.
  int chain_T0;
};
__host__ __device__ inline int seq_of_slot(const RowMap& m, int slot) {
  if (m.n_inline > 0) return m.inline_seq[slot];
  return m.seq_map ? m.seq_map[slot] : m.seq_base + slot;
}

// ---------------------------------------------------------------- weight repacking
// dst[(j / group) * group_stride + group_offset + j % group][c] = bf16(src[j][c]),  j < rows, c < cols
void launch_convert_rows(cudaStream_t st, const void* src, int src_is_f32, bf16* dst, int rows, int cols,
                         int dst_pitch, int group, int group_stride, int group_offset);
// same row mapping, but dst is tile-contiguous: element (n, k) of the mapped matrix lives at
// (((n / 128) * kb_total + k / 64) * 128 + n % 128) * 64 + k % 64, kb_total = ceil(cols_padded / 64)
void launch_convert_tiled(cudaStream_t st, const void* src, int src_is_f32, bf16* dst, int rows, int cols,
                          int kb_total, int group, int group_stride, int group_offset);
inline size_t tiled_elems(int n, int k) { return (size_t)((n + 127) / 128) * ((k + 63) / 64) * 128 * 64; }
void launch_copy_f32(cudaStream_t st, const void* src, int src_is_f32, float* dst, int n);

// ---------------------------------------------------------------- elementwise / reductions
// producer side of the fused RMSNorm: h[r] = embed[ids[r]]; hb[r] = bf16(h[r] * gain);
// sq[r * sq_stride] = sum of squares of h[r]
// (ids outside [0, V) read row 0: the table is never indexed out of range)
void launch_embed_prep(cudaStream_t st, const int* ids, const bf16* embed, const float* gain, float* h, bf16* hb,
                       float* sq, int sq_stride, int R, int d, int V);
// the same producer step for a residual stream already in h: hb[r] = bf16(h[r] * gain), sq as above
void launch_stream_prep(cudaStream_t st, const float* h, const float* gain, bf16* hb, float* sq, int sq_stride, int R,
                        int d);
// sums the split-K partials of the fused QKV projection, rotates q and k, writes bf16.
// kv_to_cache: k/v rows go to cache[(seq*max_seq + pos)*Hkv*hd] else to local [r][Hkv][hd].
void launch_qkv_rope(cudaStream_t st, const float* partial, int splits, size_t split_stride, int R, int H,
                     int Hkv, int hd, const float2* rope_table, RowMap map, bf16* q, bf16* k_dst, bf16* v_dst,
                     int kv_to_cache, size_t cache_seq_stride, size_t kv_pos_stride, size_t kv_head_stride);
// per row: argmax / max-softmax-probability over the vocabulary with mask_id excluded
void launch_lm_stats_from_logits(cudaStream_t st, const float* logits, int R, int V, int mask_id,
                                 const uint8_t* row_wanted, int* tok, float* conf);
// merge per-tile (max, sumexp, argmax) in tile order; the token is always inside [0, V)
void launch_lm_merge(cudaStream_t st, const float* tile_max, const float* tile_sum, const int* tile_arg,
                     int tiles, int R, int V, const uint8_t* row_wanted, int* tok, float* conf);

// the k most probable tokens per row from the per-tile candidate lists (merged in tile order, lower index
// first among equals): topk_tok [R][kLmTopKMax], topk_prob likewise = exp(logit - max) * conf[row]
void launch_lm_merge_topk(cudaStream_t st, const float* tile_topv, const int* tile_topi, int tiles, int R, int V, int k,
                          const uint8_t* row_wanted, const float* conf, int* topk_tok, float* topk_prob);

// ---------------------------------------------------------------- attention
struct AttnArgs {
  // verification forward: Q and the node-local K/V come straight from the fp32 split-K partials
  // of the fused q|k|v projection ([splits][R][(H + 2 Hkv) * hd]) and are rotated in the prologue
  const float* qkv_partial;
  int qkv_splits;
  size_t qkv_split_stride;
  const float2* rope;         // [max_seq][hd/2] (cos, sin)
  // block commit through the verification form (one node per sequence, rows_per_seq == T): the
  // rotated K and the V of the rows are also written to the cache at their absolute positions
  bf16* cache_k_out;          // layer base like cache_k, or nullptr
  bf16* cache_v_out;
  int* err_flag;              // device int set non-zero when a bounded wait expires (tcgen05 form)
  const bf16* q;        // [R][H][hd], rotated
  const bf16* cache_k;  // layer base: [seq][max_seq][Hkv][hd]
  const bf16* cache_v;
  const bf16* local_k;  // [R][Hkv][hd] or nullptr (no node-local keys)
  const bf16* local_v;
  float* part_o;        // [n_parts][R][H][hd]
  float2* part_ml;      // [n_parts][R][H]  (running max in log2 domain, sum)
  bf16* out;            // [R][H*hd]
  int R, H, Hkv, hd;
  int S;                // keys read from the cache
  // Dual cache: the cached keys are the positions [0, hole_begin) and [hole_begin + hole_len, ...), i.e. key
  // index k >= hole_begin lives in cache row k + hole_len (the rows of the block being computed are skipped:
  // its own keys are the node-local ones).  hole_len = 0: the cached keys are the prefix [0, S).
  int hole_begin, hole_len;
  int kv_split;         // prefix keys per split (a function of S only)
  size_t cache_seq_stride;
  size_t cache_rows;                      // rows of hd elements in one layer's K (or V) cache: max_batch * Hkv * max_seq; 0: unknown
  size_t kv_pos_stride, kv_head_stride;   // element (sequence, position, kv head) of the cache lies at
                                          // seq * cache_seq_stride + head * kv_head_stride + pos * kv_pos_stride
  RowMap map;
  int n_seq_slots;
};
void launch_attention(cudaStream_t st, const AttnArgs& a, int* launches);
// Verification-forward form: one kernel; rotary embedding, node-local K/V and the merge of the
// key parts (through a thread-block cluster) inside.  Needs prefix parts + 1 <= kAttnMaxClusterParts.
// Returns 0 or a negative ssd error code.
int launch_attention_verify(cudaStream_t st, const AttnArgs& a);
// The same on the tcgen05 tensor cores, for head dimension 128, kv_split 128 (<= 7 prefix parts) and
// node-local keys that fit one 128-key tile; needs a.err_flag.  Returns 0 (launched), 1 (shape not
// covered: use launch_attention_verify) or a negative ssd error code.
int launch_attention_verify_tc(cudaStream_t st, const AttnArgs& a);
// The same for batches of sequences: one CTA per (query tile, head, sequence) with all key tiles in one software pipeline
// (no cluster, no merge).  Head dimension 128, node width dividing 128, any prefix length; needs a.err_flag.
// Same return codes.
int launch_attention_verify_pipe(cudaStream_t st, const AttnArgs& a);
constexpr int kAttnMaxClusterParts = 8;

// ---------------------------------------------------------------- projections
// EPI_RESIDUAL: the split-K CTAs of a tile form a cluster; they sum their accumulators through
// distributed shared memory in split order, add the residual stream, and write the new stream
// h (fp32), its bf16 copy times the next norm's gain (hb, the next projection's operand) and the
// tile's share of every row's sum of squares.  The RMSNorm itself is then applied by the consumer:
// rmsnorm(h) * g . W^T  ==  inv_rms(row) * ((h * g) . W^T), with inv_rms from the sums of squares.
enum { EPI_PARTIAL = 0, EPI_SWIGLU = 1, EPI_LMHEAD = 2, EPI_RESIDUAL = 3 };
constexpr int kGemmMaxClusterSplits = 8;
constexpr int kLmTopKMax = 8;   // most candidates per row the LM-head epilogue can rank
struct GemmArgs {
  const bf16* x;  // [R][x_pitch] activations (K-major)
  const bf16* w;  // [N][w_pitch] weights (K-major), or the tile-contiguous layout below when w_tiled
  int R, N, K, x_pitch, w_pitch;
  int w_tiled;           // 1: w is [ceil(N/128)][ceil(K/64)][128][64] (one 16 KB block per MMA tile, zero padded)
  int splits;            // split-K factor (EPI_PARTIAL only)
  int two_sm_min_rows;   // tensor-core kernel: pairs of tiles run as one cta_group::2 MMA from this many rows on; 0 = never
  int epi;
  float* out;            // EPI_PARTIAL: [splits][R][N] fp32
  bf16* act;             // EPI_SWIGLU: [R][act_pitch], N/2 features
  int act_pitch;
  float* tile_max;       // EPI_LMHEAD: [tiles][R]
  float* tile_sum;
  int* tile_arg;
  int topk;              // EPI_LMHEAD: 0, or how many of the tile's largest logits per row to write as well (<= kLmTopKMax)
  float* tile_topv;      // [tiles][R][kLmTopKMax] values, descending
  int* tile_topi;        // [tiles][R][kLmTopKMax] vocabulary indices (lower index first among equals)
  int mask_id;
  int* err_flag;         // device int set non-zero when a bounded wait expires
  unsigned long long wait_limit_ns;   // bound of every barrier wait in the kernel; 0 = the default (2 s)
  int max_stages;        // tuning: cap on the depth of the shared-memory ring (0: as deep as the budget allows)
  int starve_kb;         // test hook, 0 = off: leave out the copies of K block starve_kb - 1 (plain EPI_PARTIAL launches only)
  // consumer side of a fused RMSNorm: every output row r is multiplied by
  // rsqrt(sum_{t < sq_count} sq[r * sq_stride + t] / norm_dim + norm_eps); sq == nullptr: no scaling
  const float* sq;
  int sq_count, sq_stride, norm_dim;
  float norm_eps;
  // EPI_RESIDUAL: splits = cluster size (<= kGemmMaxClusterSplits)
  float* h;              // [R][N] fp32 residual stream, updated in place
  bf16* hb;              // [R][N] bf16(h * gain)
  const float* gain;     // [N]
  float* sq_out;         // [R][sq_out_stride]: slot `tile` of a row receives the tile's sum of squares
  int sq_out_stride;
};
int gemm_tiles(int N);
// tensor-core path (TMA + tcgen05). Returns 0 or a negative ssd error code.
int launch_gemm_tc(cudaStream_t st, const GemmArgs& g);
int gemm_tc_init();   // resolves the driver entry point for tensor-map encoding
// Tensor map (a CUtensorMap, 128 bytes, 64-byte aligned) over a row-major bf16 matrix [rows][cols] with `pitch_elems`
// elements between rows: boxes of 64 columns x box_rows rows, 128-byte swizzle.  Returns 0 or a negative ssd error code.
int encode_tmap_bf16_2d(void* map_out, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch_elems, uint32_t box_rows);

// ---------------------------------------------------------------- tree build / acceptance
struct BlockState {       // device arrays, [max_batch][stride] unless noted; a row holds [current block | next block]
  int* ids;
  uint8_t* masked;
  int* draft_tok;
  float* draft_conf;
  int* has_drafts;        // [max_batch] bit 0: the current block has drafts, bit 1: the next block has
  int* remaining;         // [max_batch] r of the current block
  int* remaining_nxt;     // [max_batch] masked positions of the next block
  const int* draft_cap;   // [max_batch] per-sequence cap on the draft length (INT_MAX: none)
  int* window;            // [max_batch] 1: the sequence takes candidates from the next block in the current forward
  int* cand_pos;          // [max_batch][block_len]
  int* cand_tok;
  int* n_cand;            // [max_batch] N of the current forward
  int* accept_log;        // [max_batch][block_len] accepted per forward, 0-terminated
  int* n_forwards;        // [max_batch]
  int* last_accept;       // [max_batch] accepted by the latest step (0 if not active)
  int* last_pos;          // [max_batch] position and token of the last token the latest step accepted
  int* last_tok;          //             (the last valid node's own prediction)
  int* seq_map;           // [max_batch] slot -> sequence of the current forward
  int stride;             // 2 * block_len (row pitch of the arrays above)
};
// Nodes of the verification tree for N candidates: the greedy chain has N + 1; the mix-order tree adds
// one branch for every chain node that has a grandchild (N - 1 of them): 2N nodes for N >= 1.
__host__ __device__ inline int tree_nodes(int N, int mix_order) { return N + 1 + ((mix_order && N >= 2) ? N - 1 : 0); }
// slot a (= rank among unfinished sequences): candidates, node rows [a][n_cap][prev_T + T + T2].  A node's rows
// are: the prev_T tokens of a finished block (prev_ids, device [batch][prev_stride]; nothing asked of them) when
// the forward also commits that block, then the T rows of the current block, then - in a forward whose window
// includes it - the T2 rows of the next block.
void launch_tree_build(cudaStream_t st, BlockState s, int batch, int T, int T2, int max_drafts, int n_cap, int mask_id,
                       int* node_ids, uint8_t* node_masked, const int* prev_ids, int prev_T, int prev_stride,
                       int mix_order);
// per slot: per-node best masked position, walk, state/draft update (same row layout)
void launch_accept(cudaStream_t st, BlockState s, int n_slots, int T, int T2, int n_cap, const int* tok, const float* conf,
                   const uint8_t* node_masked, int* nonfinite_flag, int prev_T, int mix_order);

}  // namespace ssd
