// Host side of the C ABI declared in include/ssd.h: context, weight repacking, the forward pass
// schedule (one launch sequence per layer), and the per-block decode loop of Algorithm 1.
#include "../../include/ssd.h"
#include "kernels.h"

#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <string>
#include <vector>

using namespace ssd;

namespace {

struct LayerW {
  bf16 *wqkv = nullptr, *wo = nullptr, *wgu = nullptr, *wd = nullptr;
  float *g_attn = nullptr, *g_ffn = nullptr;
  uint32_t loaded = 0;   // bit per tensor
};

struct ProfRec { int fam, sub; cudaEvent_t e0, e1; double bytes; };
struct MarkRec { int fam, sub; double bytes; };
constexpr int kMaxMarks = 16384;      // launches one in-stream measurement can hold

char g_create_error[256] = "";

}  // namespace

struct ssd_ctx {
  ssd_config cfg;
  cudaStream_t st = nullptr;
  int H = 0, Hkv = 0, hd = 0, d = 0, ffn = 0, ffn_pad = 0, V = 0, nqkv = 0, qdim = 0, kvdim = 0;
  std::vector<LayerW> L;
  bf16 *embed = nullptr, *lm_head = nullptr;
  float* g_final = nullptr;
  uint32_t loaded_globals = 0;

  bf16 *cacheK = nullptr, *cacheV = nullptr;
  size_t cache_seq_stride = 0, cache_layer_stride = 0;
  // The cache is head-major, [layer][sequence][kv head][position][hd]: the keys of one head - what an attention CTA
  // streams - are contiguous, a 128-key tile is one 32 KB run instead of 128 runs of 256 bytes a whole row apart.
  size_t kv_pos_stride = 0, kv_head_stride = 0;
  float2* rope = nullptr;

  int n_max = 1;         // nodes per sequence the buffers can hold
  int R_dec = 0;         // max rows of a verification forward
  int R_cap = 0;         // max rows of any forward
  size_t partial_elems = 0, part_rows_parts = 0;
  size_t partial_row_floats = 0;   // split-K workspace per row
  float* h = nullptr;
  bf16* xn = nullptr;
  float* sq = nullptr;           // [R_cap][sq_stride] per-tile sums of squares of h (fused RMSNorm)
  int sq_stride = 1;
  float* partial = nullptr;
  bf16 *q = nullptr, *att = nullptr, *act = nullptr;
  float* part_o = nullptr;
  float2* part_ml = nullptr;
  float *tile_max = nullptr, *tile_sum = nullptr;
  int* tile_arg = nullptr;
  int* tok = nullptr;
  float* conf = nullptr;
  int* node_ids = nullptr;
  uint8_t* node_masked = nullptr;
  float* logits = nullptr;
  size_t logits_elems = 0;
  // acceptance-limit probe (allocated on first use): per-tile candidate lists of the LM head, the merged
  // top-k per row, the draft forward's top-k per block position, match counters
  float* tile_topv = nullptr;
  int* tile_topi = nullptr;
  int* topk_tok = nullptr;       // [R_dec][kLmTopKMax]
  float* topk_prob = nullptr;
  int* draft_top = nullptr;      // [max_batch][block_len][kLmTopKMax]
  unsigned long long* probe_counts = nullptr;   // [kLmTopKMax] tokens matched at k = 1.., then [kLmTopKMax] = steps counted
  int* flags = nullptr;          // [0] bounded-wait expiry, [1] non-finite confidence
  int* h_pinned = nullptr;       // pinned host staging: [0..1] flags, then 3 * max_batch ints
  BlockState bs{};

  int batch = 0, prompt_len = 0, cache_len = -1, block_tokens = 0;
  bool in_block = false;
  // A finished block whose K/V are not in the cache yet: its commit is folded into the next block's
  // first forward (or run on its own when something else needs the cache first).
  int pending_T = 0;
  int* pending_ids = nullptr;    // [max_batch][stride] tokens of that block
  // Candidates from the next block (Section 3.2.2): the block after the current one is next_T tokens long
  // (option "cross_block", 0 = there is none / off); window_T2 is the value the block in progress was begun
  // with; when a block is committed its neighbour's state (tokens accepted across the boundary, drafts) is
  // carried over to the next ssd_block_begin.
  int next_T = 0, window_T2 = 0;
  bool carry = false;
  int carry_T = 0;
  std::vector<int> h_remaining_nxt;
  // Dual cache (Section 4.1): dual_total = P + L of the sequences being decoded (0 = off, the exact prefix
  // cache); the K/V of all positions are recomputed by a full-sequence forward at every block start and
  // after every refresh_interval decoded tokens; h_since = tokens decoded since a sequence's last refresh.
  int dual_total = 0, refresh_interval = 8;
  int64_t refreshes = 0;
  int* seq_ids = nullptr;        // [max_batch][max_seq] tokens known so far: prompt, then committed blocks
  int* refresh_rows = nullptr;   // [max_seq] ids of one refresh forward
  int* draft_cap_dev = nullptr;  // [max_batch] per-sequence cap on the draft length (dual cache), else INT_MAX
  std::vector<int> h_since, h_draft_cap;
  int* prompt_stage = nullptr;   // [max_batch][max_seq] device copy of a host prompt (ssd_prefill)
  int fuse_commit = 1;
  std::vector<int> h_remaining, h_has_drafts, h_nodes, h_max_accept;
  int mix_order = 0;             // 1: the verification tree gets the out-of-order branches of Section 5.2

  int split_qkv = 1, split_o = 1, split_down = 1, kv_split_opt = 0;
  int two_sm_rows = 128;                   // projections pair their tiles (two-SM MMA) from this many rows on; 0 = never
  int attn_impl = 1;                       // 1: tcgen05 attention where the shape allows; 0: mma.sync form only
  int64_t launches = 0;
  int gemm_max_stages = 0;       // tuning: cap on the projection kernel's ring depth (0: none)
  int attn_pipe_keys = 1;        // prefixes of at least this many keys take the pipelined attention form (0: never) ...
  int attn_pipe_ctas = 64;       // ... when the prefilled batch gives it at least this many (head, sequence) CTAs
  int wait_limit_us = 0;         // bound of the projection kernel's barrier waits (0: the kernel's default, 2 s)
  int starve_gemm_kb = 0;        // test hook for ssd_gemm_bf16: K block (1-based) whose copies are left out
  bool profiling = false;        // mode 1: CUDA events around every launch (serialises the stream)
  bool marking = false;          // mode 2: a marker kernel after every launch stamps the time it ended, in the live stream
  unsigned long long* marks = nullptr;   // device [kMaxMarks]
  std::vector<MarkRec> mark_rec;
  std::vector<ProfRec> prof;
  std::vector<void*> allocs;
  char err[256] = "";
};

namespace {

int fail(ssd_ctx* c, int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(c ? c->err : g_create_error, 256, fmt, ap);
  va_end(ap);
  return code;
}

#define CUDA_TRY(c, expr)                                                                          \
  do {                                                                                             \
    cudaError_t e_ = (expr);                                                                       \
    if (e_ != cudaSuccess)                                                                         \
      return fail((c), e_ == cudaErrorMemoryAllocation ? SSD_ERR_OOM : SSD_ERR_CUDA, "%s: %s", #expr, \
                  cudaGetErrorString(e_));                                                         \
  } while (0)

template <typename T>
int dev_alloc(ssd_ctx* c, T** p, size_t n, bool zero = true) {
  void* v = nullptr;
  if (n == 0) n = 1;
  cudaError_t e = cudaMalloc(&v, n * sizeof(T));
  if (e != cudaSuccess) return fail(c, SSD_ERR_OOM, "cudaMalloc of %zu bytes failed: %s", n * sizeof(T), cudaGetErrorString(e));
  if (zero) {
    e = cudaMemsetAsync(v, 0, n * sizeof(T), c->st);
    if (e != cudaSuccess) return fail(c, SSD_ERR_CUDA, "cudaMemset failed: %s", cudaGetErrorString(e));
  }
  c->allocs.push_back(v);
  *p = reinterpret_cast<T*>(v);
  return SSD_OK;
}
#define ALLOC(c, p, n)                               \
  do {                                               \
    int rc_ = dev_alloc((c), &(p), (size_t)(n));     \
    if (rc_ != SSD_OK) return rc_;                   \
  } while (0)

constexpr int kMaxSplit = 16;

constexpr int kPrefillRows = 4096;      // rows of one prefill forward when a batch's prompts are prefilled together

// Split-K factor that fills the machine: two CTAs per SM on 148 SMs, at least four K blocks each.
// A function of the matrix shape alone, so a row's summation order never depends on the row count.
int auto_split(int tiles, int k) {
  const int kb = (k + 63) / 64;
  int s = (2 * 148 + tiles / 2) / tiles;
  if (s > kb / 4) s = kb / 4;
  if (s > kMaxSplit) s = kMaxSplit;
  if (s < 1) s = 1;
  return s;
}

// Prefix keys per attention part: a function of the prefix length (and the option) only.  The
// verification forward merges the parts inside one cluster, so prefix parts + the local part <= 8.
int kv_split_for(const ssd_ctx* c, int S) {
  int ks = c->kv_split_opt > 0 ? c->kv_split_opt : 128;
  // raised in steps of 128 keys: whole tensor-core tiles whenever the starting value is one
  while ((S + ks - 1) / ks > kAttnMaxClusterParts - 1) ks += 128;
  return ks;
}

// ---- profiling / launch accounting --------------------------------------------------------
// Runs as one more dependent launch behind the kernel it measures: its dependency wait ends when that
// kernel has completed, and it writes the time.  The kernel after it still starts early and prefetches.
__global__ void mark_end_kernel(unsigned long long* slot) {
  pdl_launch_dependents();
  pdl_wait();
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  *slot = t;
}

struct Scope {
  ssd_ctx* c;
  int fam, sub;
  double bytes;
  int mark = -1;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  Scope(ssd_ctx* c_, int fam_, double bytes_, int n_launches = 1, int sub_ = -1)
      : c(c_), fam(fam_), sub(sub_), bytes(bytes_) {
    c->launches += n_launches;
    if (c->profiling) {
      cudaEventCreate(&e0);
      cudaEventCreate(&e1);
      cudaEventRecord(e0, c->st);
    }
    if (c->marking && (int)c->mark_rec.size() < kMaxMarks) {
      mark = (int)c->mark_rec.size();
      c->mark_rec.push_back({fam, sub, bytes});
    }
  }
  ~Scope() {
    if (mark >= 0) launch_pdl(mark_end_kernel, dim3(1), dim3(1), 0, c->st, c->marks + mark);
    if (c->profiling) {
      cudaEventRecord(e1, c->st);
      c->prof.push_back({fam, sub, e0, e1, bytes});
    }
  }
};

__global__ void sum_splits_kernel(const float* partial, int splits, size_t stride, float* out, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float v = 0.f;
  for (int s = 0; s < splits; ++s) v += partial[s * stride + i];
  out[i] = v;
}

// Fresh state: the current block (T positions) and the next one (T2, may be 0) all masked, no drafts.
__global__ void block_init_kernel(BlockState s, int batch, int max_batch, int T, int T2, int mask_id) {
  const int b = blockIdx.x;
  for (int t = threadIdx.x; t < s.stride; t += blockDim.x) {
    const size_t o = (size_t)b * s.stride + t;
    s.ids[o] = mask_id;
    s.masked[o] = (b < batch && t < T + T2) ? 1 : 0;
    s.draft_tok[o] = 0;
    s.draft_conf[o] = 0.f;
    s.cand_pos[o] = 0;
    s.cand_tok[o] = 0;
    s.accept_log[o] = 0;
  }
  if (threadIdx.x == 0) {
    s.has_drafts[b] = 0;
    s.remaining[b] = (b < batch) ? T : 0;
    s.remaining_nxt[b] = (b < batch) ? T2 : 0;
    s.window[b] = 0;
    s.n_cand[b] = 0;
    s.n_forwards[b] = 0;
    s.last_accept[b] = 0;
    s.seq_map[b] = b;
  }
}

// The next block (old_T .. old_T + T positions of the row) becomes the current one, with whatever was
// accepted into it and its drafts; behind it a fresh next block of T2 positions.
__global__ void block_shift_kernel(BlockState s, int batch, int old_T, int T, int T2, int mask_id) {
  __shared__ int ids[512];
  __shared__ int dt[512];
  __shared__ float dc[512];
  __shared__ uint8_t mk[512];
  const int b = blockIdx.x;
  for (int t = threadIdx.x; t < T; t += blockDim.x) {
    const size_t o = (size_t)b * s.stride + old_T + t;
    ids[t] = s.ids[o]; mk[t] = s.masked[o]; dt[t] = s.draft_tok[o]; dc[t] = s.draft_conf[o];
  }
  __syncthreads();
  for (int t = threadIdx.x; t < s.stride; t += blockDim.x) {
    const size_t o = (size_t)b * s.stride + t;
    const bool keep = t < T;
    s.ids[o] = keep ? ids[t] : mask_id;
    s.masked[o] = keep ? mk[t] : ((b < batch && t < T + T2) ? 1 : 0);
    s.draft_tok[o] = keep ? dt[t] : 0;
    s.draft_conf[o] = keep ? dc[t] : 0.f;
    s.cand_pos[o] = 0;
    s.cand_tok[o] = 0;
    s.accept_log[o] = 0;
  }
  if (threadIdx.x == 0) {
    s.has_drafts[b] = (s.has_drafts[b] >> 1) & 1;
    s.remaining[b] = s.remaining_nxt[b];
    s.remaining_nxt[b] = (b < batch) ? T2 : 0;
    s.window[b] = 0;
    s.n_cand[b] = 0;
    s.n_forwards[b] = 0;
    s.last_accept[b] = 0;
    s.seq_map[b] = b;
  }
}

// ---- projections ----------------------------------------------------------------------------
int run_gemm(ssd_ctx* c, GemmArgs g, int fam, int sub = -1) {
  Scope sc(c, fam, (double)g.N * g.K * 2.0, 1, sub);
  g.err_flag = c->flags;
  g.two_sm_min_rows = c->two_sm_rows;
  g.wait_limit_ns = (unsigned long long)c->wait_limit_us * 1000ull;
  g.max_stages = c->gemm_max_stages;
  const int rc = launch_gemm_tc(c->st, g);
  if (rc != 0) return fail(c, rc, "projection kernel rejected R=%d N=%d K=%d epi=%d splits=%d (code %d)", g.R, g.N, g.K, g.epi, g.splits, rc);
  return SSD_OK;
}

bool all_loaded(const ssd_ctx* c) {
  if (c->loaded_globals != 7u) return false;
  for (const LayerW& l : c->L)
    if (l.loaded != 0x1FFu) return false;
  return true;
}

enum { FWD_FILL = 0, FWD_VERIFY = 1 };

// Layers [begin, end) of a forward; from_stream: the residual stream entering `begin` is already in
// c->h (no embedding gather); lm_head: run the LM head after the last layer of the range.
struct LayerRange {
  int begin = 0, end = -1;       // end < 0: all layers
  bool from_stream = false;
  bool lm_head = true;
  int topk = 0;                  // > 0: the LM head also ranks the `topk` most probable tokens of every wanted row
  bool commit_chain = false;     // the rows before chain_T0 of every sequence's first node go to the K/V cache
  int keys_total = 0;            // dual cache: the cache holds positions [0, keys_total); all of them except the rows' own
                                 // block [pos0, pos0 + T) are attended to (0: the prefix [0, pos0) only)
};

// One forward over R rows.  FILL: K/V go to the cache at positions pos0.., attention over the cache
// only (which then contains the rows themselves), no LM head.  VERIFY: K/V stay node-local, attention
// over cached prefix + own node, LM head statistics into tok/conf (and logits if wanted).
int forward(ssd_ctx* c, int kind, const int* ids_dev, int R, RowMap map, int n_slots, bool want_logits,
            const uint8_t* row_wanted, LayerRange range = LayerRange()) {
  const int d = c->d, H = c->H, Hkv = c->Hkv, hd = c->hd;
  const int S = map.pos0;
  if (R > c->R_cap) return fail(c, SSD_ERR_OVERFLOW, "forward of %d rows exceeds capacity %d", R, c->R_cap);
  // A block commit is a one-node verification forward whose K/V also go to the cache: it takes the
  // verification attention kernel.  Only the prefill (many rows, empty cache) fills through the
  // rotary pass and the cache-reading attention.
  const bool commit_form = kind == FWD_FILL && S > 0 && map.rows_per_seq == map.T &&
                           map.T <= c->cfg.block_len;
  const bool via_cache = kind == FWD_FILL && !commit_form;
  const int hole_len = (!via_cache && range.keys_total > 0) ? map.T : 0;
  const int attn_S = via_cache ? S + map.T : (hole_len > 0 ? range.keys_total - hole_len : S);
  const int kv_split = via_cache ? attn_S : kv_split_for(c, attn_S);
  const int n_parts = (attn_S + kv_split - 1) / kv_split;
  if (via_cache && (size_t)n_parts * R > c->part_rows_parts)
    return fail(c, SSD_ERR_OVERFLOW, "attention workspace too small for %d parts x %d rows", n_parts, R);
  const int nl = range.end < 0 ? c->cfg.n_layers : range.end;
  // The RMSNorms have no kernel of their own: a producer (the embedding gather, the O and down
  // projections) writes the residual stream h, bf16(h * gain) in `xn` and per-tile sums of squares in
  // `sq`; the consuming projection scales its output rows by 1/rms.
  int sq_count = 1;                       // slots of `sq` the next consumer sums per row
  auto consume_norm = [&](GemmArgs& ga) {
    ga.sq = c->sq; ga.sq_count = sq_count; ga.sq_stride = c->sq_stride; ga.norm_dim = d; ga.norm_eps = c->cfg.rms_eps;
  };
  auto produce_norm = [&](GemmArgs& ga, const float* gain, int splits) {
    ga.epi = EPI_RESIDUAL; ga.splits = splits < kGemmMaxClusterSplits ? splits : kGemmMaxClusterSplits;
    ga.h = c->h; ga.hb = c->xn; ga.gain = gain; ga.sq_out = c->sq; ga.sq_out_stride = c->sq_stride;
  };
  {
    Scope sc(c, SSD_PROF_ELEMWISE, (double)R * d * 8);
    if (range.from_stream) launch_stream_prep(c->st, c->h, c->L[range.begin].g_attn, c->xn, c->sq, c->sq_stride, R, d);
    else launch_embed_prep(c->st, ids_dev, c->embed, c->L[0].g_attn, c->h, c->xn, c->sq, c->sq_stride, R, d, c->V);
  }
  for (int l = range.begin; l < nl; ++l) {
    const LayerW& w = c->L[l];
    // ---- QKV projection, rotary embedding
    GemmArgs g{};
    g.x = c->xn; g.w = w.wqkv; g.R = R; g.N = c->nqkv; g.K = d; g.x_pitch = d; g.w_pitch = d; g.w_tiled = 1;
    g.splits = c->split_qkv; g.epi = EPI_PARTIAL; g.out = c->partial;
    consume_norm(g);
    if ((size_t)g.splits * R * g.N > c->partial_elems) return fail(c, SSD_ERR_OVERFLOW, "split-K workspace too small");
    int rc = run_gemm(c, g, SSD_PROF_GEMM, SSD_PROF_GEMM_QKV);
    if (rc) return rc;
    AttnArgs a{};
    a.cache_k = c->cacheK + (size_t)l * c->cache_layer_stride;
    a.cache_v = c->cacheV + (size_t)l * c->cache_layer_stride;
    a.out = c->att;
    a.R = R; a.H = H; a.Hkv = Hkv; a.hd = hd; a.S = attn_S; a.kv_split = kv_split;
    a.hole_begin = hole_len > 0 ? S : 0; a.hole_len = hole_len;
    a.cache_rows = c->cache_layer_stride / (size_t)hd;
    a.cache_seq_stride = c->cache_seq_stride; a.kv_pos_stride = c->kv_pos_stride; a.kv_head_stride = c->kv_head_stride;
    a.map = map; a.n_seq_slots = n_slots;
    const double kvb = (double)n_slots * attn_S * Hkv * hd * 4.0 + (double)R * (H + 2 * Hkv) * hd * 2.0 + (double)R * H * hd * 2.0;
    if (via_cache) {
      // the rotary pass writes K/V into the cache; attention then reads the cache, which holds the rows themselves
      {
        Scope sc(c, SSD_PROF_ELEMWISE, (double)R * c->nqkv * (4.0 * g.splits + 2.0));
        launch_qkv_rope(c->st, c->partial, g.splits, (size_t)R * c->nqkv, R, H, Hkv, hd, c->rope, map, c->q,
                        c->cacheK + (size_t)l * c->cache_layer_stride, c->cacheV + (size_t)l * c->cache_layer_stride, 1,
                        c->cache_seq_stride, c->kv_pos_stride, c->kv_head_stride);
      }
      if (l == nl - 1) break;   // only this layer's K/V were still needed
      a.q = c->q; a.part_o = c->part_o; a.part_ml = c->part_ml;
      Scope sc(c, SSD_PROF_ATTN, kvb, 2);
      launch_attention(c->st, a, nullptr);
    } else {
      // rotary embedding, node-local K/V and the merge of the key parts happen inside the attention kernel
      a.qkv_partial = c->partial; a.qkv_splits = g.splits; a.qkv_split_stride = (size_t)R * c->nqkv; a.rope = c->rope;
      if (commit_form || (map.chain_T0 > 0 && range.commit_chain)) {
        a.cache_k_out = c->cacheK + (size_t)l * c->cache_layer_stride;
        a.cache_v_out = c->cacheV + (size_t)l * c->cache_layer_stride;
      }
      Scope sc(c, SSD_PROF_ATTN, kvb, 1);
      a.err_flag = c->flags;
      int arc = 1;
      // One pipelined CTA per (head, sequence) walks all key tiles - when there are enough of those to fill the machine
      // (a batch of two or more sequences at 32 heads); one sequence is faster with its key parts side by side.  A function of the prefix
      // length and of the PREFILLED batch size (not of the rows or of the sequences still unfinished), so stepwise and
      // SSD forwards of one generation always take the same form.
      if (c->attn_impl == 1 && c->attn_pipe_keys > 0 && attn_S >= c->attn_pipe_keys && c->batch * H >= c->attn_pipe_ctas)
        arc = launch_attention_verify_pipe(c->st, a);
      if (arc == 1 && c->attn_impl == 1) arc = launch_attention_verify_tc(c->st, a);   // 1: shape not covered by the tcgen05 form
      if (arc == 1) arc = launch_attention_verify(c->st, a);
      if (arc != 0) return fail(c, arc, "verification attention rejected S=%d kv_split=%d (code %d)", attn_S, kv_split, arc);
      if (commit_form && l == nl - 1) break;   // the last layer's K/V are in the cache; nothing reads its output
    }
    // ---- output projection + residual + norm
    g = GemmArgs{};
    g.x = c->att; g.w = w.wo; g.R = R; g.N = d; g.K = c->qdim; g.x_pitch = c->qdim; g.w_pitch = c->qdim; g.w_tiled = 1;
    g.splits = c->split_o; g.epi = EPI_PARTIAL; g.out = c->partial;
    produce_norm(g, w.g_ffn, c->split_o);
    rc = run_gemm(c, g, SSD_PROF_GEMM, SSD_PROF_GEMM_O);
    if (rc) return rc;
    sq_count = gemm_tiles(d);
    // ---- gate/up projection with SwiGLU
    g = GemmArgs{};
    g.x = c->xn; g.w = w.wgu; g.R = R; g.N = 2 * c->ffn_pad; g.K = d; g.x_pitch = d; g.w_pitch = d; g.w_tiled = 1;
    g.splits = 1;
    g.epi = EPI_SWIGLU; g.act = c->act; g.act_pitch = c->ffn_pad;
    consume_norm(g);
    rc = run_gemm(c, g, SSD_PROF_GEMM, SSD_PROF_GEMM_GU);
    if (rc) return rc;
    // ---- down projection + residual + next norm
    g = GemmArgs{};
    g.x = c->act; g.w = w.wd; g.R = R; g.N = d; g.K = c->ffn_pad; g.x_pitch = c->ffn_pad; g.w_pitch = c->ffn_pad; g.w_tiled = 1;
    g.splits = c->split_down; g.epi = EPI_PARTIAL; g.out = c->partial;
    const float* gain = (l + 1 < c->cfg.n_layers) ? c->L[l + 1].g_attn : c->g_final;
    produce_norm(g, gain, c->split_down);
    rc = run_gemm(c, g, SSD_PROF_GEMM, SSD_PROF_GEMM_DOWN);
    if (rc) return rc;
  }
  if (kind == FWD_VERIFY && range.lm_head && nl == c->cfg.n_layers) {
    GemmArgs g{};
    g.x = c->xn; g.w = c->lm_head; g.R = R; g.N = c->V; g.K = d; g.x_pitch = d; g.w_pitch = d; g.splits = 1; g.w_tiled = 1;
    g.mask_id = c->cfg.mask_id;
    consume_norm(g);
    if (want_logits) {
      const size_t need = (size_t)R * c->V;
      if (need > c->logits_elems) {
        float* p = nullptr;
        if (cudaMalloc(&p, need * sizeof(float)) != cudaSuccess)
          return fail(c, SSD_ERR_OOM, "cannot allocate %zu bytes for debug logits", need * sizeof(float));
        c->allocs.push_back(p);
        c->logits = p;
        c->logits_elems = need;
      }
      g.epi = EPI_PARTIAL; g.out = c->logits;
      int rc = run_gemm(c, g, SSD_PROF_LMHEAD);
      if (rc) return rc;
      Scope sc(c, SSD_PROF_LMHEAD, (double)R * c->V * 4.0);
      launch_lm_stats_from_logits(c->st, c->logits, R, c->V, c->cfg.mask_id, row_wanted, c->tok, c->conf);
    } else {
      g.epi = EPI_LMHEAD; g.tile_max = c->tile_max; g.tile_sum = c->tile_sum; g.tile_arg = c->tile_arg;
      if (range.topk > 0) { g.topk = range.topk; g.tile_topv = c->tile_topv; g.tile_topi = c->tile_topi; }
      int rc = run_gemm(c, g, SSD_PROF_LMHEAD);
      if (rc) return rc;
      Scope sc(c, SSD_PROF_LMHEAD, (double)gemm_tiles(c->V) * R * 12.0, range.topk > 0 ? 2 : 1);
      launch_lm_merge(c->st, c->tile_max, c->tile_sum, c->tile_arg, gemm_tiles(c->V), R, c->V, row_wanted, c->tok, c->conf);
      if (range.topk > 0)
        launch_lm_merge_topk(c->st, c->tile_topv, c->tile_topi, gemm_tiles(c->V), R, c->V, range.topk, row_wanted, c->conf,
                             c->topk_tok, c->topk_prob);
    }
  }
  CUDA_TRY(c, cudaGetLastError());
  return SSD_OK;
}

// ids of one refresh forward of sequence b: what is known ([0, known)), the block in progress (MASK where it is
// still masked), MASK beyond
__global__ void refresh_rows_kernel(const int* seq_ids, BlockState s, int b, int known, int T, int total, int mask_id,
                                    int* out) {
  const int p = blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= total) return;
  int id = mask_id;
  if (p < known) id = seq_ids[p];
  else if (p < known + T && !s.masked[(size_t)b * s.stride + p - known]) id = s.ids[(size_t)b * s.stride + p - known];
  out[p] = id;
}

// Buffers of the acceptance-limit probe; allocated the first time a top-k forward is asked for.
int ensure_topk_buffers(ssd_ctx* c) {
  if (c->tile_topv) return SSD_OK;
  const size_t tiles = gemm_tiles(c->V);
  ALLOC(c, c->tile_topv, tiles * c->R_dec * kLmTopKMax);
  ALLOC(c, c->tile_topi, tiles * c->R_dec * kLmTopKMax);
  ALLOC(c, c->topk_tok, (size_t)c->R_dec * kLmTopKMax);
  ALLOC(c, c->topk_prob, (size_t)c->R_dec * kLmTopKMax);
  ALLOC(c, c->draft_top, (size_t)c->cfg.max_batch * c->bs.stride * kLmTopKMax);
  ALLOC(c, c->probe_counts, kLmTopKMax + 1);
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  return SSD_OK;
}

// round opening: the draft forward's top-k of every block position of every sequence
__global__ void probe_store_kernel(const int* topk_tok, int* draft_top, const int* seq_map, int T, int stride,
                                   int slot_rows, int row_offset) {
  const int slot = blockIdx.x, b = seq_map[slot];
  for (int e = threadIdx.x; e < T * kLmTopKMax; e += blockDim.x)
    draft_top[(size_t)b * stride * kLmTopKMax + e] = topk_tok[((size_t)slot * slot_rows + row_offset) * kLmTopKMax + e];
}

// after a stepwise step: is the token just decoded among the draft's top k at its position?
__global__ void probe_count_kernel(BlockState s, const int* draft_top, int n_slots, int k_max, int count_matches,
                                   unsigned long long* counts) {
  const int slot = threadIdx.x;
  if (slot >= n_slots) return;
  const int b = s.seq_map[slot];
  atomicAdd(&counts[kLmTopKMax], 1ull);
  if (!count_matches) return;
  const int q = s.last_pos[b], t = s.last_tok[b];
  for (int r = 0; r < k_max; ++r) {
    if (draft_top[((size_t)b * s.stride + q) * kLmTopKMax + r] == t) {
      for (int k = r; k < k_max; ++k) atomicAdd(&counts[k], 1ull);      // matched at every k above its rank
      break;
    }
  }
}

int check_flags_after_sync(ssd_ctx* c) {
  if (c->h_pinned[0] != 0) return fail(c, SSD_ERR_TIMEOUT, "a bounded device-side wait expired (role %d)", c->h_pinned[0]);
  if (c->h_pinned[1] != 0) return fail(c, SSD_ERR_NONFINITE, "non-finite confidence in the verification forward");
  return SSD_OK;
}

int sync_and_check(ssd_ctx* c) {
  CUDA_TRY(c, cudaMemcpyAsync(c->h_pinned, c->flags, 2 * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  return check_flags_after_sync(c);
}

// The commit forward of a finished block on its own (Section 3.2.4 leaves open how a block's K/V
// reach the cache; here: one forward over its final tokens).  ids: device [batch][stride].
int commit_now(ssd_ctx* c, const int* ids, int stride, int T) {
  const int B = c->batch;
  CUDA_TRY(c, cudaMemcpy2DAsync(c->node_ids, T * sizeof(int), ids, stride * sizeof(int), T * sizeof(int), B, cudaMemcpyDeviceToDevice, c->st));
  CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  RowMap map{T, T, c->cache_len, 0, nullptr};
  int rc = forward(c, FWD_FILL, c->node_ids, B * T, map, B, false, nullptr);
  if (rc) return rc;
  rc = sync_and_check(c);
  if (rc) return rc;
  c->cache_len += T;
  return SSD_OK;
}

// Whatever needs the whole cache (a test hook, a read-back, a teacher-forced state) first runs the
// commit that was waiting for the next block's first forward.
int flush_pending(ssd_ctx* c) {
  if (c->pending_T <= 0) return SSD_OK;
  const int rc = commit_now(c, c->pending_ids, c->bs.stride, c->pending_T);
  if (rc) return rc;
  c->pending_T = 0;
  return SSD_OK;
}

// Dual cache: one forward over ALL positions of sequence b, every position seeing every position, rewrites
// the K/V of the whole sequence (Section 4.1).  T = tokens of the block in progress (0: none).
int refresh_sequence(ssd_ctx* c, int b, int T) {
  const int total = c->dual_total;
  refresh_rows_kernel<<<(total + 255) / 256, 256, 0, c->st>>>(c->seq_ids + (size_t)b * c->cfg.max_seq, c->bs, b, c->cache_len, T,
                                                           total, c->cfg.mask_id, c->refresh_rows);
  c->launches += 1;
  RowMap map{total, total, 0, b, nullptr};
  const int rc = forward(c, FWD_FILL, c->refresh_rows, total, map, 1, false, nullptr);
  if (rc) return rc;
  c->refreshes += 1;
  c->h_since[b] = 0;
  return SSD_OK;
}

int parse_layer_name(const char* name, int* layer, const char** rest) {
  if (strncmp(name, "layers.", 7) != 0) return 0;
  char* end = nullptr;
  long l = strtol(name + 7, &end, 10);
  if (end == name + 7 || *end != '.') return 0;
  *layer = (int)l;
  *rest = end + 1;
  return 1;
}

}  // namespace

// =============================================================================================
extern "C" {

const char* ssd_last_error(const ssd_ctx* ctx) { return ctx ? ctx->err : g_create_error; }

int ssd_create(const ssd_config* cfg, void* cuda_stream, ssd_ctx** out) {
  if (!cfg || !out) return fail(nullptr, SSD_ERR_INVALID_ARG, "null argument");
  *out = nullptr;
  const ssd_config& k = *cfg;
  if (k.n_layers < 1 || k.d_model < 8 || k.n_heads < 1 || k.n_kv_heads < 1 || k.d_ffn < 8 || k.vocab < 2 ||
      k.max_batch < 1 || k.max_seq < 1 || k.block_len < 1 || k.max_drafts < 0)
    return fail(nullptr, SSD_ERR_INVALID_ARG, "non-positive size in config");
  if (k.head_dim != 64 && k.head_dim != 128) return fail(nullptr, SSD_ERR_SHAPE, "head_dim must be 64 or 128");
  if (k.d_model % 8 || k.d_ffn % 8 || k.n_heads % k.n_kv_heads || k.block_len > 256)
    return fail(nullptr, SSD_ERR_SHAPE, "d_model, d_ffn must be multiples of 8, heads a multiple of kv heads, block_len <= 256");
  if (k.mask_id < 0 || k.mask_id >= k.vocab) return fail(nullptr, SSD_ERR_INVALID_ARG, "mask_id outside the vocabulary");
  if (k.block_len > k.max_seq) return fail(nullptr, SSD_ERR_INVALID_ARG, "block_len exceeds max_seq");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1)
    return fail(nullptr, SSD_ERR_CUDA, "no CUDA device: this library has no CPU path");
  if (gemm_tc_init() != 0) return fail(nullptr, SSD_ERR_CUDA, "cannot resolve the tensor-map encoder of the CUDA driver");

  ssd_ctx* c = new (std::nothrow) ssd_ctx();
  if (!c) return fail(nullptr, SSD_ERR_OOM, "host allocation failed");
  c->cfg = k;
  c->st = reinterpret_cast<cudaStream_t>(cuda_stream);
  c->H = k.n_heads; c->Hkv = k.n_kv_heads; c->hd = k.head_dim; c->d = k.d_model; c->ffn = k.d_ffn;
  c->ffn_pad = (k.d_ffn + 63) / 64 * 64; c->V = k.vocab;
  c->qdim = c->H * c->hd; c->kvdim = c->Hkv * c->hd; c->nqkv = c->qdim + 2 * c->kvdim;
  c->L.resize(k.n_layers);
  c->n_max = (k.max_drafts < k.block_len - 1 ? k.max_drafts : k.block_len - 1) + 1;
  // at least two blocks of rows per sequence: the forward that commits a block together with the
  // first step of the next one
  c->R_dec = k.max_batch * (c->n_max > 2 ? c->n_max : 2) * k.block_len;
  c->R_cap = c->R_dec > k.max_seq ? c->R_dec : k.max_seq;
  // room to prefill several sequences of a batch in one forward (one stream of the weights for all of them)
  const long long group_rows = std::min<long long>((long long)k.max_batch * k.max_seq, kPrefillRows);
  if (group_rows > c->R_cap) c->R_cap = (int)group_rows;
  c->split_qkv = auto_split(gemm_tiles(c->nqkv), c->d);
  c->split_o = auto_split(gemm_tiles(c->d), c->qdim);
  c->split_down = auto_split(gemm_tiles(c->d), c->ffn_pad);
  c->h_remaining.assign(k.max_batch, 0);
  c->h_has_drafts.assign(k.max_batch, 0);
  c->h_remaining_nxt.assign(k.max_batch, 0);
  c->h_since.assign(k.max_batch, 0);
  c->h_draft_cap.assign(k.max_batch, 0x7fffffff);
  c->h_nodes.assign(k.max_batch, 0);
  c->h_max_accept.assign(k.max_batch, 0);

  int rc = SSD_OK;
  auto build = [&]() -> int {
    const int d = c->d;
    for (LayerW& w : c->L) {
      // tile-contiguous, zero padded to whole 128 x 64 tiles
      ALLOC(c, w.wqkv, tiled_elems(c->nqkv, d));
      ALLOC(c, w.wo, tiled_elems(d, c->qdim));
      ALLOC(c, w.wgu, tiled_elems(2 * c->ffn_pad, d));
      ALLOC(c, w.wd, tiled_elems(d, c->ffn_pad));
      ALLOC(c, w.g_attn, d);
      ALLOC(c, w.g_ffn, d);
    }
    ALLOC(c, c->embed, (size_t)c->V * d);
    ALLOC(c, c->lm_head, tiled_elems(c->V, d));
    ALLOC(c, c->g_final, d);
    c->cache_seq_stride = (size_t)k.max_seq * c->kvdim;
    c->kv_pos_stride = (size_t)c->hd;
    c->kv_head_stride = (size_t)k.max_seq * c->hd;
    c->cache_layer_stride = c->cache_seq_stride * k.max_batch;
    ALLOC(c, c->cacheK, c->cache_layer_stride * k.n_layers);
    ALLOC(c, c->cacheV, c->cache_layer_stride * k.n_layers);
    // rotary table in double precision on the host
    {
      const int half = c->hd / 2;
      std::vector<float2> t((size_t)k.max_seq * half);
      for (int p = 0; p < k.max_seq; ++p)
        for (int i = 0; i < half; ++i) {
          const double inv = pow((double)k.rope_theta, -2.0 * i / (double)c->hd);
          const double a = (double)p * inv;
          t[(size_t)p * half + i] = make_float2((float)cos(a), (float)sin(a));
        }
      ALLOC(c, c->rope, t.size());
      CUDA_TRY(c, cudaMemcpyAsync(c->rope, t.data(), t.size() * sizeof(float2), cudaMemcpyHostToDevice, c->st));
      CUDA_TRY(c, cudaStreamSynchronize(c->st));
    }
    const size_t R = (size_t)c->R_cap;
    ALLOC(c, c->h, R * d);
    ALLOC(c, c->xn, R * d);
    c->sq_stride = gemm_tiles(d);
    ALLOC(c, c->sq, R * c->sq_stride);
    c->partial_row_floats = (size_t)kMaxSplit * d;
    if ((size_t)4 * c->nqkv > c->partial_row_floats) c->partial_row_floats = (size_t)4 * c->nqkv;
    if ((size_t)c->split_qkv * c->nqkv > c->partial_row_floats) c->partial_row_floats = (size_t)c->split_qkv * c->nqkv;
    if ((size_t)2 * c->ffn_pad > c->partial_row_floats) c->partial_row_floats = (size_t)2 * c->ffn_pad;
    c->partial_elems = R * c->partial_row_floats;
    ALLOC(c, c->partial, c->partial_elems);
    ALLOC(c, c->q, R * c->qdim);
    ALLOC(c, c->att, R * c->qdim);
    ALLOC(c, c->act, R * c->ffn_pad);
    c->part_rows_parts = R;      // the cache-fill attention runs one key part per query tile
    ALLOC(c, c->part_o, c->part_rows_parts * c->qdim);
    ALLOC(c, c->part_ml, c->part_rows_parts * c->H);
    const size_t tiles = gemm_tiles(c->V);
    ALLOC(c, c->tile_max, tiles * c->R_dec);
    ALLOC(c, c->tile_sum, tiles * c->R_dec);
    ALLOC(c, c->tile_arg, tiles * c->R_dec);
    ALLOC(c, c->tok, R);
    ALLOC(c, c->conf, R);
    ALLOC(c, c->node_ids, R);
    ALLOC(c, c->node_masked, R);
    ALLOC(c, c->flags, 4);
    ALLOC(c, c->marks, kMaxMarks);
    const size_t sb = (size_t)k.max_batch * 2 * k.block_len;      // a row holds [current block | next block]
    c->bs.stride = 2 * k.block_len;
    ALLOC(c, c->bs.ids, sb); ALLOC(c, c->bs.masked, sb); ALLOC(c, c->bs.draft_tok, sb); ALLOC(c, c->bs.draft_conf, sb);
    ALLOC(c, c->bs.cand_pos, sb); ALLOC(c, c->bs.cand_tok, sb); ALLOC(c, c->bs.accept_log, sb);
    ALLOC(c, c->pending_ids, sb);
    ALLOC(c, c->prompt_stage, (size_t)k.max_batch * k.max_seq);
    ALLOC(c, c->seq_ids, (size_t)k.max_batch * k.max_seq);
    ALLOC(c, c->refresh_rows, (size_t)k.max_seq);
    ALLOC(c, c->draft_cap_dev, k.max_batch);
    CUDA_TRY(c, cudaMemcpyAsync(c->draft_cap_dev, c->h_draft_cap.data(), k.max_batch * sizeof(int), cudaMemcpyHostToDevice, c->st));
    c->bs.draft_cap = c->draft_cap_dev;
    ALLOC(c, c->bs.has_drafts, k.max_batch); ALLOC(c, c->bs.remaining, k.max_batch); ALLOC(c, c->bs.n_cand, k.max_batch);
    ALLOC(c, c->bs.n_forwards, k.max_batch); ALLOC(c, c->bs.last_accept, k.max_batch); ALLOC(c, c->bs.seq_map, k.max_batch);
    ALLOC(c, c->bs.last_pos, k.max_batch); ALLOC(c, c->bs.last_tok, k.max_batch);
    ALLOC(c, c->bs.remaining_nxt, k.max_batch); ALLOC(c, c->bs.window, k.max_batch);
    CUDA_TRY(c, cudaMallocHost(&c->h_pinned, (2 + 5 * (size_t)k.max_batch) * sizeof(int)));
    CUDA_TRY(c, cudaStreamSynchronize(c->st));
    return SSD_OK;
  };
  rc = build();
  if (rc != SSD_OK) {
    snprintf(g_create_error, sizeof(g_create_error), "%s", c->err);
    ssd_destroy(c);
    return rc;
  }
  *out = c;
  return SSD_OK;
}

void ssd_destroy(ssd_ctx* c) {
  if (!c) return;
  cudaStreamSynchronize(c->st);
  for (ProfRec& r : c->prof) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
  for (void* p : c->allocs) cudaFree(p);
  if (c->h_pinned) cudaFreeHost(c->h_pinned);
  delete c;
}

int ssd_load_weights(ssd_ctx* c, const char* name, const void* dev_ptr, int32_t dtype, const int64_t* shape, int32_t ndim) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!name || !dev_ptr || !shape) return fail(c, SSD_ERR_INVALID_ARG, "null argument");
  if (dtype != SSD_DTYPE_BF16 && dtype != SSD_DTYPE_F32) return fail(c, SSD_ERR_INVALID_ARG, "unknown dtype %d", dtype);
  const int f32 = dtype == SSD_DTYPE_F32;
  const int d = c->d;
  auto want2 = [&](int64_t r, int64_t k) { return ndim == 2 && shape[0] == r && shape[1] == k; };
  auto want1 = [&](int64_t n) { return ndim == 1 && shape[0] == n; };
  int layer = -1;
  const char* rest = nullptr;
  bool ok_shape = true;
  if (!strcmp(name, "embed")) {
    if ((ok_shape = want2(c->V, d))) { launch_convert_rows(c->st, dev_ptr, f32, c->embed, c->V, d, d, c->V, 0, 0); c->loaded_globals |= 1u; }
  } else if (!strcmp(name, "lm_head")) {
    if ((ok_shape = want2(c->V, d))) { launch_convert_tiled(c->st, dev_ptr, f32, c->lm_head, c->V, d, (d + 63) / 64, c->V, 0, 0); c->loaded_globals |= 2u; }
  } else if (!strcmp(name, "norm_final")) {
    if ((ok_shape = want1(d))) { launch_copy_f32(c->st, dev_ptr, f32, c->g_final, d); c->loaded_globals |= 4u; }
  } else if (parse_layer_name(name, &layer, &rest)) {
    if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, SSD_ERR_INVALID_ARG, "layer %d out of range", layer);
    LayerW& w = c->L[layer];
    const int kbd = (d + 63) / 64;
    if (!strcmp(rest, "wq")) {
      if ((ok_shape = want2(c->qdim, d))) { launch_convert_tiled(c->st, dev_ptr, f32, w.wqkv, c->qdim, d, kbd, c->qdim, 0, 0); w.loaded |= 1u; }
    } else if (!strcmp(rest, "wk")) {
      if ((ok_shape = want2(c->kvdim, d))) { launch_convert_tiled(c->st, dev_ptr, f32, w.wqkv, c->kvdim, d, kbd, c->kvdim, 0, c->qdim); w.loaded |= 2u; }
    } else if (!strcmp(rest, "wv")) {
      if ((ok_shape = want2(c->kvdim, d))) { launch_convert_tiled(c->st, dev_ptr, f32, w.wqkv, c->kvdim, d, kbd, c->kvdim, 0, c->qdim + c->kvdim); w.loaded |= 4u; }
    } else if (!strcmp(rest, "wo")) {
      if ((ok_shape = want2(d, c->qdim))) { launch_convert_tiled(c->st, dev_ptr, f32, w.wo, d, c->qdim, (c->qdim + 63) / 64, d, 0, 0); w.loaded |= 8u; }
    } else if (!strcmp(rest, "w_gate")) {
      // 64 gate features then the 64 matching up features per 128-row tile
      if ((ok_shape = want2(c->ffn, d))) { launch_convert_tiled(c->st, dev_ptr, f32, w.wgu, c->ffn, d, kbd, 64, 128, 0); w.loaded |= 16u; }
    } else if (!strcmp(rest, "w_up")) {
      if ((ok_shape = want2(c->ffn, d))) { launch_convert_tiled(c->st, dev_ptr, f32, w.wgu, c->ffn, d, kbd, 64, 128, 64); w.loaded |= 32u; }
    } else if (!strcmp(rest, "w_down")) {
      if ((ok_shape = want2(d, c->ffn))) { launch_convert_tiled(c->st, dev_ptr, f32, w.wd, d, c->ffn, c->ffn_pad / 64, d, 0, 0); w.loaded |= 64u; }
    } else if (!strcmp(rest, "norm_attn")) {
      if ((ok_shape = want1(d))) { launch_copy_f32(c->st, dev_ptr, f32, w.g_attn, d); w.loaded |= 128u; }
    } else if (!strcmp(rest, "norm_ffn")) {
      if ((ok_shape = want1(d))) { launch_copy_f32(c->st, dev_ptr, f32, w.g_ffn, d); w.loaded |= 256u; }
    } else {
      return fail(c, SSD_ERR_INVALID_ARG, "unknown tensor '%s'", name);
    }
  } else {
    return fail(c, SSD_ERR_INVALID_ARG, "unknown tensor '%s'", name);
  }
  if (!ok_shape) return fail(c, SSD_ERR_SHAPE, "tensor '%s' has the wrong shape", name);
  c->launches += 1;
  CUDA_TRY(c, cudaGetLastError());
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  return SSD_OK;
}

int ssd_prefill_dev(ssd_ctx* c, int32_t batch, int32_t prompt_len, const int32_t* prompt_ids_dev) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!prompt_ids_dev) return fail(c, SSD_ERR_INVALID_ARG, "null prompt");
  if (batch < 1 || batch > c->cfg.max_batch) return fail(c, SSD_ERR_OVERFLOW, "batch %d outside [1, %d]", batch, c->cfg.max_batch);
  if (prompt_len < 1 || prompt_len > c->cfg.max_seq) return fail(c, SSD_ERR_OVERFLOW, "prompt_len %d outside [1, %d]", prompt_len, c->cfg.max_seq);
  if (!all_loaded(c)) return fail(c, SSD_ERR_STATE, "not every weight tensor has been loaded");
  CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  // as many sequences per forward as the row capacity holds: their rows share one stream of the weights
  const int group = std::max(1, c->R_cap / prompt_len);
  for (int b = 0; b < batch; b += group) {
    const int n = std::min(group, batch - b);
    RowMap map{prompt_len, prompt_len, 0, b, nullptr};
    const int rc = forward(c, FWD_FILL, prompt_ids_dev + (size_t)b * prompt_len, n * prompt_len, map, n, false, nullptr);
    if (rc) return rc;
  }
  // the tokens of every sequence as far as they are known (a refresh of the dual cache needs them all)
  CUDA_TRY(c, cudaMemcpy2DAsync(c->seq_ids, (size_t)c->cfg.max_seq * sizeof(int), prompt_ids_dev, (size_t)prompt_len * sizeof(int),
                                (size_t)prompt_len * sizeof(int), batch, cudaMemcpyDeviceToDevice, c->st));
  const int rc = sync_and_check(c);
  if (rc) return rc;
  c->batch = batch;
  c->prompt_len = prompt_len;
  c->cache_len = prompt_len;
  c->in_block = false;
  c->pending_T = 0;
  c->carry = false;
  return SSD_OK;
}

int ssd_prefill(ssd_ctx* c, int32_t batch, int32_t prompt_len, const int32_t* prompt_ids) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!prompt_ids) return fail(c, SSD_ERR_INVALID_ARG, "null prompt");
  if (batch < 1 || batch > c->cfg.max_batch) return fail(c, SSD_ERR_OVERFLOW, "batch %d outside [1, %d]", batch, c->cfg.max_batch);
  if (prompt_len < 1 || prompt_len > c->cfg.max_seq) return fail(c, SSD_ERR_OVERFLOW, "prompt_len %d outside [1, %d]", prompt_len, c->cfg.max_seq);
  for (size_t i = 0; i < (size_t)batch * prompt_len; ++i)
    if (prompt_ids[i] < 0 || prompt_ids[i] >= c->V) return fail(c, SSD_ERR_INVALID_ARG, "prompt id %d outside the vocabulary", prompt_ids[i]);
  // staged in the context's own buffer (sized max_batch x max_seq at creation): no allocation per call
  CUDA_TRY(c, cudaMemcpyAsync(c->prompt_stage, prompt_ids, (size_t)batch * prompt_len * sizeof(int), cudaMemcpyHostToDevice, c->st));
  return ssd_prefill_dev(c, batch, prompt_len, c->prompt_stage);
}

int ssd_cache_length(const ssd_ctx* c) {
  if (!c) return SSD_ERR_INVALID_ARG;
  return c->cache_len < 0 ? SSD_ERR_STATE : c->cache_len + c->pending_T;   // a block waiting for its commit counts
}

int ssd_rewind(ssd_ctx* c, int32_t length) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (c->cache_len < 0) return fail(c, SSD_ERR_STATE, "prefill first");
  if (length < c->prompt_len || length > c->cache_len + c->pending_T)
    return fail(c, SSD_ERR_INVALID_ARG, "rewind target %d outside [%d, %d]", length, c->prompt_len, c->cache_len + c->pending_T);
  if (length > c->cache_len) {          // part of the waiting block stays: its K/V are needed after all
    const int rc = flush_pending(c);
    if (rc) return rc;
  }
  c->pending_T = 0;                     // a block cut off entirely is never committed
  c->cache_len = length;
  c->in_block = false;
  c->carry = false;
  return SSD_OK;
}

int ssd_block_begin(ssd_ctx* c, int32_t T) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (c->cache_len < 0) return fail(c, SSD_ERR_STATE, "prefill first");
  if (T < 1 || T > c->cfg.block_len) return fail(c, SSD_ERR_INVALID_ARG, "block_tokens %d outside [1, %d]", T, c->cfg.block_len);
  if (c->cache_len + c->pending_T + T > c->cfg.max_seq)
    return fail(c, SSD_ERR_OVERFLOW, "cache %d + block %d exceeds max_seq %d", c->cache_len + c->pending_T, T, c->cfg.max_seq);
  // the block after this one takes part as the second half of the window while there is room for it
  int T2 = c->next_T;
  if (T2 > 0 && c->cache_len + c->pending_T + T + T2 > c->cfg.max_seq) T2 = 0;
  if (c->dual_total > 0) {
    if (c->cache_len + T > c->dual_total) return fail(c, SSD_ERR_OVERFLOW, "block ends at %d, beyond the dual cache's sequence length %d", c->cache_len + T, c->dual_total);
    T2 = 0;
    for (int b = 0; b < c->cfg.max_batch; ++b) c->h_since[b] = c->refresh_interval;      // refresh before the first forward
  }
  if (c->carry && c->carry_T == T) {
    // this block was the second half of the previous block's window: keep what it already holds
    block_shift_kernel<<<c->cfg.max_batch, 128, 0, c->st>>>(c->bs, c->batch, c->block_tokens, T, T2, c->cfg.mask_id);
    for (int b = 0; b < c->cfg.max_batch; ++b) {
      c->h_remaining[b] = b < c->batch ? c->h_remaining_nxt[b] : 0;
      c->h_has_drafts[b] = (c->h_has_drafts[b] >> 1) & 1;
      c->h_remaining_nxt[b] = b < c->batch ? T2 : 0;
    }
  } else {
    block_init_kernel<<<c->cfg.max_batch, 128, 0, c->st>>>(c->bs, c->batch, c->cfg.max_batch, T, T2, c->cfg.mask_id);
    for (int b = 0; b < c->cfg.max_batch; ++b) {
      c->h_remaining[b] = b < c->batch ? T : 0;
      c->h_has_drafts[b] = 0;
      c->h_remaining_nxt[b] = b < c->batch ? T2 : 0;
    }
  }
  c->launches += 1;
  CUDA_TRY(c, cudaGetLastError());
  c->carry = false;
  c->window_T2 = T2;
  c->block_tokens = T;
  c->in_block = true;
  return SSD_OK;
}

int ssd_set_block_state(ssd_ctx* c, const int32_t* ids, const uint8_t* masked, const int32_t* draft_tok, const float* draft_conf) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!c->in_block) return fail(c, SSD_ERR_STATE, "no block in progress");
  if (!ids || !masked || ((draft_tok == nullptr) != (draft_conf == nullptr))) return fail(c, SSD_ERR_INVALID_ARG, "null argument");
  {
    const int frc = flush_pending(c);   // an injected state continues from a complete cache
    if (frc) return frc;
  }
  const int T = c->block_tokens, st = c->bs.stride;
  // (the next block's half of the window starts afresh; ssd_set_next_block_state can fill it)
  block_init_kernel<<<c->cfg.max_batch, 128, 0, c->st>>>(c->bs, c->batch, c->cfg.max_batch, T, c->window_T2, c->cfg.mask_id);
  c->launches += 1;
  for (int b = 0; b < c->batch; ++b) c->h_remaining_nxt[b] = c->window_T2;
  for (int b = 0; b < c->batch; ++b) {
    int r = 0;
    for (int t = 0; t < T; ++t) {
      r += masked[b * T + t] ? 1 : 0;
      if (!masked[b * T + t] && (ids[b * T + t] < 0 || ids[b * T + t] >= c->V)) return fail(c, SSD_ERR_INVALID_ARG, "token id outside the vocabulary");
      if (draft_tok && masked[b * T + t] && (draft_tok[b * T + t] < 0 || draft_tok[b * T + t] >= c->V)) return fail(c, SSD_ERR_INVALID_ARG, "draft id outside the vocabulary");
    }
    c->h_remaining[b] = r;
    c->h_has_drafts[b] = draft_tok ? 1 : 0;
  }
  CUDA_TRY(c, cudaMemcpy2DAsync(c->bs.ids, st * sizeof(int), ids, T * sizeof(int), T * sizeof(int), c->batch, cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaMemcpy2DAsync(c->bs.masked, st, masked, T, T, c->batch, cudaMemcpyHostToDevice, c->st));
  if (draft_tok) {
    CUDA_TRY(c, cudaMemcpy2DAsync(c->bs.draft_tok, st * sizeof(int), draft_tok, T * sizeof(int), T * sizeof(int), c->batch, cudaMemcpyHostToDevice, c->st));
    CUDA_TRY(c, cudaMemcpy2DAsync(c->bs.draft_conf, st * sizeof(float), draft_conf, T * sizeof(float), T * sizeof(float), c->batch, cudaMemcpyHostToDevice, c->st));
  }
  CUDA_TRY(c, cudaMemcpyAsync(c->bs.remaining, c->h_remaining.data(), c->batch * sizeof(int), cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaMemcpyAsync(c->bs.has_drafts, c->h_has_drafts.data(), c->batch * sizeof(int), cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  return SSD_OK;
}

int ssd_get_block_state(ssd_ctx* c, int32_t* ids, uint8_t* masked, int32_t* draft_tok, float* draft_conf) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!c->in_block) return fail(c, SSD_ERR_STATE, "no block in progress");
  const int T = c->block_tokens, st = c->bs.stride;
  if (ids) CUDA_TRY(c, cudaMemcpy2DAsync(ids, T * sizeof(int), c->bs.ids, st * sizeof(int), T * sizeof(int), c->batch, cudaMemcpyDeviceToHost, c->st));
  if (masked) CUDA_TRY(c, cudaMemcpy2DAsync(masked, T, c->bs.masked, st, T, c->batch, cudaMemcpyDeviceToHost, c->st));
  if (draft_tok) CUDA_TRY(c, cudaMemcpy2DAsync(draft_tok, T * sizeof(int), c->bs.draft_tok, st * sizeof(int), T * sizeof(int), c->batch, cudaMemcpyDeviceToHost, c->st));
  if (draft_conf) CUDA_TRY(c, cudaMemcpy2DAsync(draft_conf, T * sizeof(float), c->bs.draft_conf, st * sizeof(float), T * sizeof(float), c->batch, cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  return SSD_OK;
}

namespace {

int resolve_drafts(const ssd_ctx* c, int max_drafts) {
  int md = max_drafts < 0 ? c->cfg.max_drafts : max_drafts;
  return md > c->cfg.max_drafts ? c->cfg.max_drafts : md;
}

// Enqueues one iteration of Algorithm 1's loop for every unfinished sequence - tree build, the batched
// forward, acceptance - without waiting for it.  The host's mirror of `remaining` / `has_drafts` decides
// the launch shape; h_nodes[b] receives the nodes sequence b gets (0: finished).  The error flags are
// sticky and are NOT cleared here.
struct ProbeStep { int k_max; bool open_round; };

int step_enqueue(ssd_ctx* c, int md, bool* launched, const ProbeStep* probe = nullptr) {
  const int T = c->block_tokens, B = c->batch;
  // chain length of sequence b; with `window` it may take candidates from the next block (Section 3.2.2)
  auto drafts_of = [&](int b, bool window) -> int {
    const int r = c->h_remaining[b];
    if (!(c->h_has_drafts[b] & 1)) return 0;
    if (window && r <= md) {
      int more = 0;
      if (c->h_has_drafts[b] & 2) more = std::max(0, std::min(md - r, c->h_remaining_nxt[b] - 1));
      return r + more;
    }
    const int cap = (c->dual_total > 0) ? std::min(md, c->h_draft_cap[b]) : md;
    return cap < r - 1 ? cap : r - 1;
  };
  auto shape = [&](bool window, int* active_out) -> int {
    int active = 0, n_cap = 1;
    for (int b = 0; b < B; ++b) {
      c->h_nodes[b] = 0;
      c->h_max_accept[b] = 0;
      if (c->h_remaining[b] <= 0) continue;
      ++active;
      const int N = drafts_of(b, window);
      c->h_nodes[b] = tree_nodes(N, c->mix_order);
      c->h_max_accept[b] = N + 1;            // (a branch ends the walk at most N tokens in)
      if (c->h_nodes[b] > n_cap) n_cap = c->h_nodes[b];
    }
    *active_out = active;
    return n_cap;
  };
  const bool dual = c->dual_total > 0;
  if (dual) {
    // refresh the sequences that are due, and cap every chain so that no forward accepts past the next
    // refresh point: the tokens stay those of stepwise decoding under the same schedule
    for (int b = 0; b < B; ++b) {
      c->h_draft_cap[b] = 0x7fffffff;
      if (c->h_remaining[b] <= 0) continue;
      if (c->h_since[b] >= c->refresh_interval) {
        const int rrc = refresh_sequence(c, b, T);
        if (rrc) return rrc;
      }
      c->h_draft_cap[b] = std::max(0, c->refresh_interval - c->h_since[b] - 1);
    }
    CUDA_TRY(c, cudaMemcpyAsync(c->draft_cap_dev, c->h_draft_cap.data(), B * sizeof(int), cudaMemcpyHostToDevice, c->st));
  }
  int active = 0;
  int n_cap = shape(false, &active);
  *launched = active > 0;
  if (active == 0) return SSD_OK;
  // A block waiting for its commit rides in front of this block's forward: every node is one causal chain
  // [finished block | this block's node state], and the first node's finished-block rows write the K/V.  All
  // sequences must take part (each has a block to commit); otherwise the commit runs on its own first.
  int Tp = 0;
  if (c->pending_T > 0) {
    if (!dual && active == B && active * n_cap * (c->pending_T + T) <= c->R_dec) {
      Tp = c->pending_T;
    } else {
      const int frc = flush_pending(c);
      if (frc) return frc;
      CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
    }
  }
  // The window [this block | next block]: whenever a sequence can no longer fill its chain from this block.
  int T2 = 0;
  if (Tp == 0 && c->window_T2 > 0 && !c->mix_order && !probe && !dual) {
    bool any = false;
    for (int b = 0; b < B; ++b) any = any || (c->h_remaining[b] > 0 && (c->h_has_drafts[b] & 1) && c->h_remaining[b] <= md);
    if (any) {
      int act2 = 0;
      const int cap2 = shape(true, &act2);
      if (cap2 <= c->n_max && active * cap2 * (T + c->window_T2) <= c->R_dec) {
        T2 = c->window_T2;
        n_cap = cap2;
      } else {
        n_cap = shape(false, &act2);         // no room for the window: single-block chains
      }
    }
  }
  if (n_cap > c->n_max) return fail(c, SSD_ERR_OVERFLOW, "a tree of %d nodes exceeds the capacity of %d nodes fixed at creation", n_cap, c->n_max);
  const int node_rows = Tp + T + T2;
  const int slot_rows = n_cap * node_rows;
  const int R = active * slot_rows;
  if (R > c->R_dec) return fail(c, SSD_ERR_OVERFLOW, "%d rows exceed the capacity %d set by max_batch/max_drafts/block_len", R, c->R_dec);
  {
    Scope sc(c, SSD_PROF_TREE, (double)R * 5);
    launch_tree_build(c->st, c->bs, B, T, T2, md, n_cap, c->cfg.mask_id, c->node_ids, c->node_masked,
                      Tp > 0 ? c->pending_ids : nullptr, Tp, c->bs.stride, c->mix_order);
  }
  RowMap map{slot_rows, node_rows, c->cache_len, 0, c->bs.seq_map};
  if (Tp > 0) map.chain_T0 = Tp;                // a node's rows: [finished block | this block]
  else if (T2 > 0) map.chain_T0 = T;            //                [this block | next block]
  if (active <= 8) {           // the host mirrors `remaining`, so it knows the slot -> sequence map too
    for (int b = 0; b < B; ++b)
      if (c->h_remaining[b] > 0) map.inline_seq[map.n_inline++] = b;
  }
  LayerRange range;
  if (probe && probe->open_round) range.topk = probe->k_max;
  range.commit_chain = Tp > 0;
  if (dual) range.keys_total = c->dual_total;
  int rc = forward(c, FWD_VERIFY, c->node_ids, R, map, active, false, c->node_masked, range);
  if (rc) return rc;
  {
    Scope sc(c, SSD_PROF_TREE, (double)R * 9);
    launch_accept(c->st, c->bs, active, T, T2, n_cap, c->tok, c->conf, c->node_masked, c->flags + 1, Tp, c->mix_order);
  }
  if (probe) {
    // the forward that opens a round is the draft: keep its top-k per block position; every later token of
    // the round is looked up in it
    Scope sc(c, SSD_PROF_TREE, (double)active * T * kLmTopKMax * 4, probe->open_round ? 2 : 1);
    if (probe->open_round)
      probe_store_kernel<<<active, 128, 0, c->st>>>(c->topk_tok, c->draft_top, c->bs.seq_map, T, c->bs.stride, slot_rows, Tp);
    probe_count_kernel<<<1, (active + 31) / 32 * 32, 0, c->st>>>(c->bs, c->draft_top, active, probe->k_max,
                                                               probe->open_round ? 0 : 1, c->probe_counts);
  }
  if (Tp > 0) {                // the finished block's K/V are in the cache once this forward has run
    c->cache_len += Tp;
    c->pending_T = 0;
  }
  for (int b = 0; b < B; ++b)
    if (c->h_nodes[b] > 0) c->h_has_drafts[b] |= 1 | ((T2 > 0 && c->h_remaining[b] <= md && (c->h_has_drafts[b] & 1)) ? 2 : 0);
  return SSD_OK;
}

// Waits for everything enqueued, checks the error flags and refreshes the host's mirror of `remaining`.
int step_collect(ssd_ctx* c, int32_t* accepted, int32_t* n_nodes) {
  const int B = c->batch;
  int* hp = c->h_pinned;
  const int mb = c->cfg.max_batch;
  CUDA_TRY(c, cudaMemcpyAsync(hp, c->flags, 2 * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(c, cudaMemcpyAsync(hp + 2, c->bs.remaining, B * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  if (accepted || c->dual_total > 0) CUDA_TRY(c, cudaMemcpyAsync(hp + 2 + mb, c->bs.last_accept, B * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  if (n_nodes) CUDA_TRY(c, cudaMemcpyAsync(hp + 2 + 2 * mb, c->bs.n_cand, B * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(c, cudaMemcpyAsync(hp + 2 + 3 * mb, c->bs.remaining_nxt, B * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(c, cudaMemcpyAsync(hp + 2 + 4 * mb, c->bs.has_drafts, B * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  const int rc = check_flags_after_sync(c);
  if (rc) return rc;
  for (int b = 0; b < B; ++b) {
    c->h_remaining[b] = hp[2 + b];
    c->h_remaining_nxt[b] = hp[2 + 3 * mb + b];
    if (c->dual_total > 0 && c->h_nodes[b] > 0) c->h_since[b] += hp[2 + mb + b];
    c->h_has_drafts[b] = hp[2 + 4 * mb + b];
    if (accepted) accepted[b] = hp[2 + mb + b];
    if (n_nodes) n_nodes[b] = c->h_nodes[b] > 0 ? tree_nodes(hp[2 + 2 * mb + b], c->mix_order) : 0;
  }
  return SSD_OK;
}

}  // namespace

int ssd_block_step(ssd_ctx* c, int32_t max_drafts, int32_t* accepted, int32_t* n_nodes) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!c->in_block) return fail(c, SSD_ERR_STATE, "no block in progress");
  const int md = resolve_drafts(c, max_drafts);
  const int B = c->batch;
  if (accepted) memset(accepted, 0, B * sizeof(int));
  if (n_nodes) memset(n_nodes, 0, B * sizeof(int));
  CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  bool launched = false;
  int rc = step_enqueue(c, md, &launched);
  if (rc) return rc;
  if (!launched) return SSD_OK;
  return step_collect(c, accepted, n_nodes);
}

int ssd_block_commit(ssd_ctx* c) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!c->in_block) return fail(c, SSD_ERR_STATE, "no block in progress");
  for (int b = 0; b < c->batch; ++b)
    if (c->h_remaining[b] > 0) return fail(c, SSD_ERR_STATE, "sequence %d still has %d masked positions", b, c->h_remaining[b]);
  const int T = c->block_tokens, B = c->batch;
  int rc = flush_pending(c);           // (a block that ended without a single forward of its own)
  if (rc) return rc;
  // the block's tokens join what is known of every sequence
  CUDA_TRY(c, cudaMemcpy2DAsync(c->seq_ids + c->cache_len, (size_t)c->cfg.max_seq * sizeof(int), c->bs.ids, c->bs.stride * sizeof(int),
                                T * sizeof(int), B, cudaMemcpyDeviceToDevice, c->st));
  if (c->dual_total > 0) {
    // dual cache: nothing to commit - the next block starts with a refresh of every position's K/V
    rc = sync_and_check(c);
    if (rc) return rc;
    c->cache_len += T;
  } else if (c->fuse_commit) {
    // keep the tokens; the next block's first forward (or whoever needs the cache first) commits them
    CUDA_TRY(c, cudaMemcpy2DAsync(c->pending_ids, c->bs.stride * sizeof(int), c->bs.ids, c->bs.stride * sizeof(int), T * sizeof(int), B,
                                  cudaMemcpyDeviceToDevice, c->st));
    rc = sync_and_check(c);
    if (rc) return rc;
    c->pending_T = T;
  } else {
    rc = commit_now(c, c->bs.ids, c->bs.stride, T);
    if (rc) return rc;
  }
  c->in_block = false;
  // what the window already holds of the next block is kept for its ssd_block_begin
  c->carry = c->window_T2 > 0;
  c->carry_T = c->window_T2;
  return SSD_OK;
}

int ssd_set_next_block_state(ssd_ctx* c, const int32_t* ids, const uint8_t* masked, const int32_t* draft_tok, const float* draft_conf) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!c->in_block) return fail(c, SSD_ERR_STATE, "no block in progress");
  if (c->window_T2 <= 0) return fail(c, SSD_ERR_STATE, "the block in progress was begun without a next block (option cross_block)");
  if (!ids || !masked || ((draft_tok == nullptr) != (draft_conf == nullptr))) return fail(c, SSD_ERR_INVALID_ARG, "null argument");
  const int T = c->block_tokens, T2 = c->window_T2, st = c->bs.stride;
  for (int b = 0; b < c->batch; ++b) {
    int r = 0;
    for (int t = 0; t < T2; ++t) {
      r += masked[b * T2 + t] ? 1 : 0;
      if (!masked[b * T2 + t] && (ids[b * T2 + t] < 0 || ids[b * T2 + t] >= c->V)) return fail(c, SSD_ERR_INVALID_ARG, "token id outside the vocabulary");
      if (draft_tok && masked[b * T2 + t] && (draft_tok[b * T2 + t] < 0 || draft_tok[b * T2 + t] >= c->V)) return fail(c, SSD_ERR_INVALID_ARG, "draft id outside the vocabulary");
    }
    c->h_remaining_nxt[b] = r;
    c->h_has_drafts[b] = (c->h_has_drafts[b] & 1) | (draft_tok ? 2 : 0);
  }
  CUDA_TRY(c, cudaMemcpy2DAsync(c->bs.ids + T, st * sizeof(int), ids, T2 * sizeof(int), T2 * sizeof(int), c->batch, cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaMemcpy2DAsync(c->bs.masked + T, st, masked, T2, T2, c->batch, cudaMemcpyHostToDevice, c->st));
  if (draft_tok) {
    CUDA_TRY(c, cudaMemcpy2DAsync(c->bs.draft_tok + T, st * sizeof(int), draft_tok, T2 * sizeof(int), T2 * sizeof(int), c->batch, cudaMemcpyHostToDevice, c->st));
    CUDA_TRY(c, cudaMemcpy2DAsync(c->bs.draft_conf + T, st * sizeof(float), draft_conf, T2 * sizeof(float), T2 * sizeof(float), c->batch, cudaMemcpyHostToDevice, c->st));
  }
  CUDA_TRY(c, cudaMemcpyAsync(c->bs.remaining_nxt, c->h_remaining_nxt.data(), c->batch * sizeof(int), cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaMemcpyAsync(c->bs.has_drafts, c->h_has_drafts.data(), c->batch * sizeof(int), cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  return SSD_OK;
}

int ssd_get_next_block_state(ssd_ctx* c, int32_t* ids, uint8_t* masked, int32_t* draft_tok, float* draft_conf) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!c->in_block) return fail(c, SSD_ERR_STATE, "no block in progress");
  if (c->window_T2 <= 0) return fail(c, SSD_ERR_STATE, "the block in progress was begun without a next block (option cross_block)");
  const int T = c->block_tokens, T2 = c->window_T2, st = c->bs.stride;
  if (ids) CUDA_TRY(c, cudaMemcpy2DAsync(ids, T2 * sizeof(int), c->bs.ids + T, st * sizeof(int), T2 * sizeof(int), c->batch, cudaMemcpyDeviceToHost, c->st));
  if (masked) CUDA_TRY(c, cudaMemcpy2DAsync(masked, T2, c->bs.masked + T, st, T2, c->batch, cudaMemcpyDeviceToHost, c->st));
  if (draft_tok) CUDA_TRY(c, cudaMemcpy2DAsync(draft_tok, T2 * sizeof(int), c->bs.draft_tok + T, st * sizeof(int), T2 * sizeof(int), c->batch, cudaMemcpyDeviceToHost, c->st));
  if (draft_conf) CUDA_TRY(c, cudaMemcpy2DAsync(draft_conf, T2 * sizeof(float), c->bs.draft_conf + T, st * sizeof(float), T2 * sizeof(float), c->batch, cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  return SSD_OK;
}

int ssd_decode_block(ssd_ctx* c, int32_t mode, int32_t T, int32_t* out_tokens, int32_t* out_accept_counts, int32_t* out_n_forwards) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (mode != SSD_MODE_STEPWISE && mode != SSD_MODE_SSD) return fail(c, SSD_ERR_INVALID_ARG, "unknown mode %d", mode);
  int rc = ssd_block_begin(c, T);
  if (rc) return rc;
  const int md = resolve_drafts(c, mode == SSD_MODE_STEPWISE ? 0 : -1);
  CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  // A forward accepts between 1 and nodes tokens per sequence, so after it at least remaining - nodes
  // positions are still masked.  While that bound leaves every sequence a full chain (>= md + 1), the
  // next forward's launch shape is known without its predecessor's result: it is enqueued at once and
  // the host mirror carries the bound.  The host waits (and learns the true counts) only when the bound
  // no longer decides the shape - a handful of times per block instead of once per forward.
  for (int guard = 0; guard <= T; ++guard) {
    bool any = false;
    for (int b = 0; b < c->batch; ++b) any = any || c->h_remaining[b] > 0;
    if (!any) break;
    bool launched = false;
    rc = step_enqueue(c, md, &launched);
    if (rc) return rc;
    bool decided = true;
    for (int b = 0; b < c->batch; ++b)
      if (c->h_nodes[b] > 0 && (c->h_remaining[b] - c->h_max_accept[b] < md + 1 || c->dual_total > 0)) decided = false;
    if (decided) {
      for (int b = 0; b < c->batch; ++b) c->h_remaining[b] -= c->h_max_accept[b];
      continue;
    }
    rc = step_collect(c, nullptr, nullptr);
    if (rc) return rc;
    CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  }
  const int st = c->bs.stride, B = c->batch;
  if (out_tokens) CUDA_TRY(c, cudaMemcpy2DAsync(out_tokens, T * sizeof(int), c->bs.ids, st * sizeof(int), T * sizeof(int), B, cudaMemcpyDeviceToHost, c->st));
  if (out_accept_counts) CUDA_TRY(c, cudaMemcpy2DAsync(out_accept_counts, T * sizeof(int), c->bs.accept_log, st * sizeof(int), T * sizeof(int), B, cudaMemcpyDeviceToHost, c->st));
  if (out_n_forwards) CUDA_TRY(c, cudaMemcpyAsync(out_n_forwards, c->bs.n_forwards, B * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  return ssd_block_commit(c);
}

int ssd_verify_forward(ssd_ctx* c, int32_t batch, int32_t n_nodes, int32_t T, const int32_t* node_ids, const uint8_t* node_masked,
                       int32_t* out_tok, float* out_conf, float* out_logits) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (c->cache_len < 0) return fail(c, SSD_ERR_STATE, "prefill first");
  if (!node_ids || !node_masked) return fail(c, SSD_ERR_INVALID_ARG, "null argument");
  if (batch < 1 || batch > c->batch) return fail(c, SSD_ERR_INVALID_ARG, "batch %d outside [1, %d]", batch, c->batch);
  if (T < 1 || T > c->cfg.block_len || n_nodes < 1) return fail(c, SSD_ERR_INVALID_ARG, "bad node shape");
  {
    const int frc = flush_pending(c);
    if (frc) return frc;
  }
  const size_t R = (size_t)batch * n_nodes * T;
  if (R > (size_t)c->R_dec) return fail(c, SSD_ERR_OVERFLOW, "%zu rows exceed the capacity %d set by max_batch/max_drafts/block_len", R, c->R_dec);
  if (c->cache_len + T > c->cfg.max_seq) return fail(c, SSD_ERR_OVERFLOW, "cache %d + block %d exceeds max_seq", c->cache_len, T);
  for (size_t i = 0; i < R; ++i)
    if (node_ids[i] < 0 || node_ids[i] >= c->V) return fail(c, SSD_ERR_INVALID_ARG, "node id outside the vocabulary");
  CUDA_TRY(c, cudaMemcpyAsync(c->node_ids, node_ids, R * sizeof(int), cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaMemcpyAsync(c->node_masked, node_masked, R, cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  RowMap map{n_nodes * T, T, c->cache_len, 0, nullptr};
  LayerRange range;
  if (c->dual_total > 0) {
    if (c->cache_len + T > c->dual_total) return fail(c, SSD_ERR_OVERFLOW, "block ends beyond the dual cache's sequence length %d", c->dual_total);
    range.keys_total = c->dual_total;
  }
  int rc = forward(c, FWD_VERIFY, c->node_ids, (int)R, map, batch, out_logits != nullptr, c->node_masked, range);
  if (rc) return rc;
  if (out_tok) CUDA_TRY(c, cudaMemcpyAsync(out_tok, c->tok, R * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  if (out_conf) CUDA_TRY(c, cudaMemcpyAsync(out_conf, c->conf, R * sizeof(float), cudaMemcpyDeviceToHost, c->st));
  if (out_logits) CUDA_TRY(c, cudaMemcpyAsync(out_logits, c->logits, R * (size_t)c->V * sizeof(float), cudaMemcpyDeviceToHost, c->st));
  return sync_and_check(c);
}

int ssd_read_cache(ssd_ctx* c, int32_t layer, int32_t seq, int32_t length, float* out_k, float* out_v) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= c->cfg.n_layers || seq < 0 || seq >= c->cfg.max_batch || length < 0 || length > c->cfg.max_seq)
    return fail(c, SSD_ERR_INVALID_ARG, "index out of range");
  {
    const int frc = flush_pending(c);
    if (frc) return frc;
  }
  const size_t n = (size_t)length * c->kvdim;
  std::vector<bf16> tmp(n);
  for (int which = 0; which < 2; ++which) {
    float* dst = which ? out_v : out_k;
    if (!dst) continue;
    const bf16* src = (which ? c->cacheV : c->cacheK) + (size_t)layer * c->cache_layer_stride + (size_t)seq * c->cache_seq_stride;
    // the interface's layout is [position][kv head][hd]: one strided copy per head of the head-major cache
    for (int j = 0; j < c->Hkv && length > 0; ++j)
      CUDA_TRY(c, cudaMemcpy2DAsync(tmp.data() + (size_t)j * c->hd, (size_t)c->kvdim * sizeof(bf16), src + (size_t)j * c->kv_head_stride,
                                    c->kv_pos_stride * sizeof(bf16), (size_t)c->hd * sizeof(bf16), (size_t)length,
                                    cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(c, cudaStreamSynchronize(c->st));
    for (size_t i = 0; i < n; ++i) dst[i] = __bfloat162float(tmp[i]);
  }
  return SSD_OK;
}

int ssd_write_cache(ssd_ctx* c, int32_t layer, int32_t seq, int32_t length, const float* k, const float* v) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!k || !v) return fail(c, SSD_ERR_INVALID_ARG, "null argument");
  if (c->cache_len < 0) return fail(c, SSD_ERR_STATE, "prefill first");
  if (layer < 0 || layer >= c->cfg.n_layers || seq < 0 || seq >= c->cfg.max_batch || length < 0 || length > c->cfg.max_seq)
    return fail(c, SSD_ERR_INVALID_ARG, "index out of range");
  {
    const int frc = flush_pending(c);
    if (frc) return frc;
  }
  const size_t n = (size_t)length * c->kvdim;
  std::vector<bf16> tmp(n);
  for (int which = 0; which < 2; ++which) {
    const float* src = which ? v : k;
    bf16* dst = (which ? c->cacheV : c->cacheK) + (size_t)layer * c->cache_layer_stride + (size_t)seq * c->cache_seq_stride;
    for (size_t i = 0; i < n; ++i) tmp[i] = __float2bfloat16_rn(src[i]);
    for (int j = 0; j < c->Hkv && length > 0; ++j)
      CUDA_TRY(c, cudaMemcpy2DAsync(dst + (size_t)j * c->kv_head_stride, c->kv_pos_stride * sizeof(bf16), tmp.data() + (size_t)j * c->hd,
                                    (size_t)c->kvdim * sizeof(bf16), (size_t)c->hd * sizeof(bf16), (size_t)length,
                                    cudaMemcpyHostToDevice, c->st));
    CUDA_TRY(c, cudaStreamSynchronize(c->st));
  }
  return SSD_OK;
}

int ssd_verify_layers(ssd_ctx* c, int32_t batch, int32_t n_nodes, int32_t T, int32_t layer_begin, int32_t layer_end,
                      const float* h_in, float* h_out, int32_t* out_tok, float* out_conf) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (c->cache_len < 0) return fail(c, SSD_ERR_STATE, "prefill first");
  if (!h_in) return fail(c, SSD_ERR_INVALID_ARG, "null argument");
  if (batch < 1 || batch > c->batch) return fail(c, SSD_ERR_INVALID_ARG, "batch %d outside [1, %d]", batch, c->batch);
  if (T < 1 || T > c->cfg.block_len || n_nodes < 1) return fail(c, SSD_ERR_INVALID_ARG, "bad node shape");
  if (layer_begin < 0 || layer_end <= layer_begin || layer_end > c->cfg.n_layers)
    return fail(c, SSD_ERR_INVALID_ARG, "layer range [%d, %d) outside [0, %d)", layer_begin, layer_end, c->cfg.n_layers);
  if ((out_tok || out_conf) && layer_end != c->cfg.n_layers)
    return fail(c, SSD_ERR_INVALID_ARG, "token statistics need the last layer in the range");
  {
    const int frc = flush_pending(c);
    if (frc) return frc;
  }
  const size_t R = (size_t)batch * n_nodes * T;
  if (R > (size_t)c->R_dec) return fail(c, SSD_ERR_OVERFLOW, "%zu rows exceed the capacity %d set by max_batch/max_drafts/block_len", R, c->R_dec);
  if (c->cache_len + T > c->cfg.max_seq) return fail(c, SSD_ERR_OVERFLOW, "cache %d + block %d exceeds max_seq", c->cache_len, T);
  CUDA_TRY(c, cudaMemcpyAsync(c->h, h_in, R * c->d * sizeof(float), cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  RowMap map{n_nodes * T, T, c->cache_len, 0, nullptr};
  LayerRange range;
  range.begin = layer_begin; range.end = layer_end; range.from_stream = true; range.lm_head = out_tok || out_conf;
  int rc = forward(c, FWD_VERIFY, nullptr, (int)R, map, batch, false, nullptr, range);
  if (rc) return rc;
  if (h_out) CUDA_TRY(c, cudaMemcpyAsync(h_out, c->h, R * c->d * sizeof(float), cudaMemcpyDeviceToHost, c->st));
  if (out_tok) CUDA_TRY(c, cudaMemcpyAsync(out_tok, c->tok, R * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  if (out_conf) CUDA_TRY(c, cudaMemcpyAsync(out_conf, c->conf, R * sizeof(float), cudaMemcpyDeviceToHost, c->st));
  return sync_and_check(c);
}

int ssd_verify_forward_topk(ssd_ctx* c, int32_t batch, int32_t n_nodes, int32_t T, const int32_t* node_ids,
                            const uint8_t* node_masked, int32_t k, int32_t* out_tok, float* out_prob) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (c->cache_len < 0) return fail(c, SSD_ERR_STATE, "prefill first");
  if (!node_ids || !node_masked || !out_tok || !out_prob) return fail(c, SSD_ERR_INVALID_ARG, "null argument");
  if (batch < 1 || batch > c->batch) return fail(c, SSD_ERR_INVALID_ARG, "batch %d outside [1, %d]", batch, c->batch);
  if (T < 1 || T > c->cfg.block_len || n_nodes < 1) return fail(c, SSD_ERR_INVALID_ARG, "bad node shape");
  if (k < 1 || k > kLmTopKMax) return fail(c, SSD_ERR_INVALID_ARG, "k %d outside [1, %d]", k, kLmTopKMax);
  int rc = flush_pending(c);
  if (rc) return rc;
  rc = ensure_topk_buffers(c);
  if (rc) return rc;
  const size_t R = (size_t)batch * n_nodes * T;
  if (R > (size_t)c->R_dec) return fail(c, SSD_ERR_OVERFLOW, "%zu rows exceed the capacity %d set by max_batch/max_drafts/block_len", R, c->R_dec);
  if (c->cache_len + T > c->cfg.max_seq) return fail(c, SSD_ERR_OVERFLOW, "cache %d + block %d exceeds max_seq", c->cache_len, T);
  for (size_t i = 0; i < R; ++i)
    if (node_ids[i] < 0 || node_ids[i] >= c->V) return fail(c, SSD_ERR_INVALID_ARG, "node id outside the vocabulary");
  CUDA_TRY(c, cudaMemcpyAsync(c->node_ids, node_ids, R * sizeof(int), cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaMemcpyAsync(c->node_masked, node_masked, R, cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  RowMap map{n_nodes * T, T, c->cache_len, 0, nullptr};
  LayerRange range;
  range.topk = k;
  rc = forward(c, FWD_VERIFY, c->node_ids, (int)R, map, batch, false, c->node_masked, range);
  if (rc) return rc;
  std::vector<int> tk(R * kLmTopKMax);
  std::vector<float> tp(R * kLmTopKMax);
  CUDA_TRY(c, cudaMemcpyAsync(tk.data(), c->topk_tok, tk.size() * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(c, cudaMemcpyAsync(tp.data(), c->topk_prob, tp.size() * sizeof(float), cudaMemcpyDeviceToHost, c->st));
  rc = sync_and_check(c);
  if (rc) return rc;
  for (size_t i = 0; i < R; ++i)
    for (int j = 0; j < k; ++j) {
      out_tok[i * k + j] = tk[i * kLmTopKMax + j];
      out_prob[i * k + j] = tp[i * kLmTopKMax + j];
    }
  return SSD_OK;
}

int ssd_probe_acceptance_limit(ssd_ctx* c, int32_t T, int32_t draft_len, int32_t k_max, int32_t* out_tokens,
                               int64_t* out_matched, int64_t* out_steps) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!out_matched || !out_steps) return fail(c, SSD_ERR_INVALID_ARG, "null argument");
  if (draft_len < 0 || k_max < 1 || k_max > kLmTopKMax) return fail(c, SSD_ERR_INVALID_ARG, "draft_len >= 0 and k_max in [1, %d]", kLmTopKMax);
  int rc = ensure_topk_buffers(c);
  if (rc) return rc;
  rc = ssd_block_begin(c, T);
  if (rc) return rc;
  CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  CUDA_TRY(c, cudaMemsetAsync(c->probe_counts, 0, (kLmTopKMax + 1) * sizeof(unsigned long long), c->st));
  // stepwise decoding (every sequence accepts exactly one token per forward, so all stay in lockstep) in rounds
  // of draft_len + 1 forwards; nothing depends on a forward's result, so the whole block is enqueued at once
  for (int step = 0; step < T; ++step) {
    ProbeStep ps{k_max, step % (draft_len + 1) == 0};
    bool launched = false;
    rc = step_enqueue(c, 0, &launched, &ps);
    if (rc) return rc;
    for (int b = 0; b < c->batch; ++b) c->h_remaining[b] -= 1;
  }
  rc = step_collect(c, nullptr, nullptr);
  if (rc) return rc;
  unsigned long long counts[kLmTopKMax + 1];
  CUDA_TRY(c, cudaMemcpyAsync(counts, c->probe_counts, sizeof(counts), cudaMemcpyDeviceToHost, c->st));
  if (out_tokens) CUDA_TRY(c, cudaMemcpy2DAsync(out_tokens, T * sizeof(int), c->bs.ids, c->bs.stride * sizeof(int), T * sizeof(int), c->batch, cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  for (int k = 0; k < k_max; ++k) out_matched[k] = (int64_t)counts[k];
  *out_steps = (int64_t)counts[kLmTopKMax];
  return ssd_block_commit(c);
}

int ssd_refresh_cache(ssd_ctx* c) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (c->cache_len < 0) return fail(c, SSD_ERR_STATE, "prefill first");
  if (c->dual_total <= 0) return fail(c, SSD_ERR_STATE, "the dual cache is off (option dual_cache)");
  const int T = c->in_block ? c->block_tokens : 0;
  if (c->cache_len + T > c->dual_total) return fail(c, SSD_ERR_OVERFLOW, "the sequence is longer than the dual cache's length %d", c->dual_total);
  CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  for (int b = 0; b < c->batch; ++b) {
    const int rc = refresh_sequence(c, b, T);
    if (rc) return rc;
  }
  return sync_and_check(c);
}

int64_t ssd_refresh_count(const ssd_ctx* c) { return c ? c->refreshes : -1; }

int ssd_read_forward_outputs(ssd_ctx* c, int32_t n_rows, int32_t* out_tok, float* out_conf) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (n_rows < 0 || n_rows > c->R_cap) return fail(c, SSD_ERR_INVALID_ARG, "row count outside [0, %d]", c->R_cap);
  if (out_tok) CUDA_TRY(c, cudaMemcpyAsync(out_tok, c->tok, (size_t)n_rows * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  if (out_conf) CUDA_TRY(c, cudaMemcpyAsync(out_conf, c->conf, (size_t)n_rows * sizeof(float), cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  return SSD_OK;
}

int ssd_gemm_bf16(ssd_ctx* c, const void* x_dev, const void* w_dev, float* out_dev, int32_t rows, int32_t n, int32_t k, int32_t split_k) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!x_dev || !w_dev || !out_dev) return fail(c, SSD_ERR_INVALID_ARG, "null argument");
  if (rows < 1 || n < 1 || k < 8 || (k % 8) || split_k < 1 || split_k > 8) return fail(c, SSD_ERR_SHAPE, "bad GEMM shape");
  if ((size_t)split_k * rows * n > c->partial_elems) return fail(c, SSD_ERR_OVERFLOW, "GEMM exceeds the workspace");
  CUDA_TRY(c, cudaMemsetAsync(c->flags, 0, 4 * sizeof(int), c->st));
  GemmArgs g{};
  g.x = (const bf16*)x_dev; g.w = (const bf16*)w_dev; g.R = rows; g.N = n; g.K = k; g.x_pitch = k; g.w_pitch = k;
  g.splits = split_k; g.epi = EPI_PARTIAL; g.out = c->partial;
  g.starve_kb = c->starve_gemm_kb;
  int rc = run_gemm(c, g, SSD_PROF_GEMM);
  if (rc) return rc;
  const size_t total = (size_t)rows * n;
  sum_splits_kernel<<<(unsigned)((total + 255) / 256), 256, 0, c->st>>>(c->partial, split_k, total, out_dev, total);
  c->launches += 1;
  CUDA_TRY(c, cudaGetLastError());
  return sync_and_check(c);
}

int64_t ssd_launch_count(const ssd_ctx* c) { return c ? c->launches : -1; }

int ssd_profile_enable(ssd_ctx* c, int32_t on) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (on < 0 || on > 2) return fail(c, SSD_ERR_INVALID_ARG, "profile mode is 0 (off), 1 (events around every launch) or 2 (end-of-launch marks in the live stream)");
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  c->profiling = on == 1;
  c->marking = on == 2;
  c->mark_rec.clear();
  if (c->marking) CUDA_TRY(c, cudaMemsetAsync(c->marks, 0, kMaxMarks * sizeof(unsigned long long), c->st));
  return SSD_OK;
}

int ssd_profile_read(ssd_ctx* c, int64_t* launches, double* ms, double* bytes) {
  if (!c) return SSD_ERR_INVALID_ARG;
  CUDA_TRY(c, cudaStreamSynchronize(c->st));
  for (int f = 0; f < SSD_PROF_FAMILIES; ++f) {
    if (launches) launches[f] = 0;
    if (ms) ms[f] = 0;
    if (bytes) bytes[f] = 0;
  }
  for (ProfRec& r : c->prof) {
    float t = 0.f;
    cudaEventElapsedTime(&t, r.e0, r.e1);
    for (int f : {r.fam, r.sub}) {
      if (f < 0) continue;
      if (launches) launches[f] += 1;
      if (ms) ms[f] += t;
      if (bytes) bytes[f] += r.bytes;
    }
    cudaEventDestroy(r.e0);
    cudaEventDestroy(r.e1);
  }
  c->prof.clear();
  // mode 2: a launch is charged the time from the end of its predecessor to its own end
  if (!c->mark_rec.empty()) {
    std::vector<unsigned long long> t(c->mark_rec.size());
    CUDA_TRY(c, cudaMemcpy(t.data(), c->marks, t.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
    for (size_t i = 1; i < t.size(); ++i) {
      if (t[i] == 0 || t[i - 1] == 0 || t[i] < t[i - 1]) continue;
      const double dt = (double)(t[i] - t[i - 1]) * 1e-6;
      const MarkRec& r = c->mark_rec[i];
      for (int f : {r.fam, r.sub}) {
        if (f < 0) continue;
        if (launches) launches[f] += 1;
        if (ms) ms[f] += dt;
        if (bytes) bytes[f] += r.bytes;
      }
    }
    c->mark_rec.clear();
    CUDA_TRY(c, cudaMemsetAsync(c->marks, 0, kMaxMarks * sizeof(unsigned long long), c->st));
  }
  return SSD_OK;
}

int ssd_set_option(ssd_ctx* c, const char* key, int32_t value) {
  if (!c) return SSD_ERR_INVALID_ARG;
  if (!key) return fail(c, SSD_ERR_INVALID_ARG, "null key");
  if (!strcmp(key, "split_k_qkv") || !strcmp(key, "split_k_o") || !strcmp(key, "split_k_down")) {
    const bool is_qkv = !strcmp(key, "split_k_qkv");
    const int width = is_qkv ? c->nqkv : c->d;
    const int kdim = is_qkv ? c->d : (!strcmp(key, "split_k_o") ? c->qdim : c->ffn_pad);
    int hi = kMaxSplit;                                   // every split owns at least one 64-wide K block
    if ((kdim + 63) / 64 < hi) hi = (kdim + 63) / 64;
    if (!is_qkv && kGemmMaxClusterSplits < hi) hi = kGemmMaxClusterSplits;   // these reduce inside a cluster
    if (c->partial_row_floats / width < (size_t)hi) hi = (int)(c->partial_row_floats / width);
    if (value < 1 || value > hi)
      return fail(c, SSD_ERR_INVALID_ARG, "split-K for this projection must be in [1, %d]", hi);
    if (!strcmp(key, "split_k_qkv")) c->split_qkv = value;
    else if (!strcmp(key, "split_k_o")) c->split_o = value;
    else c->split_down = value;
    return SSD_OK;
  }
  if (!strcmp(key, "kv_split")) {
    if (value != 0 && (value < 64 || value % 64)) return fail(c, SSD_ERR_INVALID_ARG, "kv_split must be 0 (automatic) or a multiple of 64");
    c->kv_split_opt = value;
    return SSD_OK;
  }
  if (!strcmp(key, "max_drafts")) {
    if (value < 0 || value + 1 > c->n_max) return fail(c, SSD_ERR_INVALID_ARG, "max_drafts must be in [0, %d] (the capacity fixed at creation)", c->n_max - 1);
    c->cfg.max_drafts = value;
    return SSD_OK;
  }
  if (!strcmp(key, "gemm_max_stages")) {
    if (value < 0 || value == 1) return fail(c, SSD_ERR_INVALID_ARG, "gemm_max_stages is 0 (no cap) or >= 2");
    c->gemm_max_stages = value;
    return SSD_OK;
  }
  if (!strcmp(key, "wait_limit_us")) {
    if (value < 0) return fail(c, SSD_ERR_INVALID_ARG, "wait_limit_us is 0 (default, 2 s) or a bound in microseconds");
    c->wait_limit_us = value;
    return SSD_OK;
  }
  if (!strcmp(key, "attn_pipe_ctas")) {
    if (value < 1) return fail(c, SSD_ERR_INVALID_ARG, "attn_pipe_ctas is a number of (head, sequence) pairs >= 1");
    c->attn_pipe_ctas = value;
    return SSD_OK;
  }
  if (!strcmp(key, "attn_pipe_keys")) {
    if (value < 0) return fail(c, SSD_ERR_INVALID_ARG, "attn_pipe_keys is 0 (never) or a prefix length in keys");
    c->attn_pipe_keys = value;
    return SSD_OK;
  }
  if (!strcmp(key, "starve_gemm_kb")) {
    if (value < 0) return fail(c, SSD_ERR_INVALID_ARG, "starve_gemm_kb is 0 (off) or a 1-based K block index");
    c->starve_gemm_kb = value;
    return SSD_OK;
  }
  if (!strcmp(key, "dual_cache")) {
    if (value != 0 && (value < 1 || value > c->cfg.max_seq)) return fail(c, SSD_ERR_INVALID_ARG, "dual_cache is 0 (off) or the sequence length P + L <= max_seq = %d", c->cfg.max_seq);
    if (c->in_block) return fail(c, SSD_ERR_STATE, "a block is in progress");
    if (value > 0) {
      const int frc = flush_pending(c);
      if (frc) return frc;
    }
    c->dual_total = value;
    c->carry = false;
    return SSD_OK;
  }
  if (!strcmp(key, "refresh_interval")) {
    if (value < 1) return fail(c, SSD_ERR_INVALID_ARG, "refresh_interval must be >= 1");
    c->refresh_interval = value;
    return SSD_OK;
  }
  if (!strcmp(key, "cross_block")) {
    if (value < 0 || value > c->cfg.block_len) return fail(c, SSD_ERR_INVALID_ARG, "cross_block is the length of the block after the next one to be begun: 0 (none) .. %d", c->cfg.block_len);
    c->next_T = value;
    return SSD_OK;
  }
  if (!strcmp(key, "mix_order")) {
    if (value != 0 && value != 1) return fail(c, SSD_ERR_INVALID_ARG, "mix_order is 0 (greedy chain) or 1 (chain plus out-of-order branches)");
    c->mix_order = value;
    return SSD_OK;
  }
  if (!strcmp(key, "attn_impl")) {
    if (value != 0 && value != 1) return fail(c, SSD_ERR_INVALID_ARG, "attn_impl is 0 (mma.sync) or 1 (tcgen05 where the shape allows)");
    c->attn_impl = value;
    return SSD_OK;
  }
  if (!strcmp(key, "two_sm_rows")) {
    if (value < 0 || value > 256) return fail(c, SSD_ERR_INVALID_ARG, "two_sm_rows is 0 (never) or a row count up to 256");
    c->two_sm_rows = value;
    return SSD_OK;
  }
  if (!strcmp(key, "fuse_commit")) {
    if (value != 0 && value != 1) return fail(c, SSD_ERR_INVALID_ARG, "fuse_commit is 0 (commit forward of its own) or 1 (folded into the next block's first forward)");
    if (value == 0) {
      const int frc = flush_pending(c);
      if (frc) return frc;
    }
    c->fuse_commit = value;
    return SSD_OK;
  }
  return fail(c, SSD_ERR_INVALID_ARG, "unknown option '%s'", key);
}

}  // extern "C"
