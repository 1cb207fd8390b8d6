// Tree build and acceptance for the greedy verification chain (Sections 3.2.2 - 3.2.4).
//
// tree_build: per unfinished sequence, order the stale drafts of the masked positions by
//   confidence (descending, lower position first on ties), keep N = min(max_drafts, r-1), and
//   write the N+1 node rows: node i = block state with candidates 1..i written in.
// accept: per node the position a stepwise step would fill (highest confidence among the node's
//   masked rows, lower position on ties) and its token; walk the chain while node i's prediction
//   equals candidate i+1 (position AND token); write the accepted tokens, the next drafts (the
//   last valid node's own predictions) and the bookkeeping.
// mix-order tree (Section 5.2): behind the chain nodes 0..N sit the branches of chain nodes 0..N-2 -
//   branch j = node j's state with candidate j+2 written in instead of candidate j+1 - and the walk
//   takes a branch when node j predicts candidate j+2: that candidate and the branch's own prediction
//   are accepted, and the walk ends (branches have no children).
// window over two blocks (Section 3.2.2, candidates from the next block): the state of a sequence is
//   [current block | next block]; a sequence whose current block cannot fill the chain (r <= max_drafts)
//   takes ALL masked positions of the current block as candidates, then the next block's most confident
//   drafts; a node predicts in the next block only once its current block is full (Section 3.1).
// All integer / comparison work; one CTA per sequence.
#include "kernels.h"

#include <math.h>

namespace ssd {

namespace {

constexpr int kMaxW = 512;       // positions of a window: two blocks of at most 256

// Does sequence b take candidates from the next block in a forward whose window has T2 > 0 next-block rows?
__device__ __forceinline__ bool spills(const BlockState& s, int b, int T2, int max_drafts) {
  return T2 > 0 && (s.has_drafts[b] & 1) && s.remaining[b] <= max_drafts;
}

__global__ void __launch_bounds__(256) tree_build_kernel(BlockState s, int batch, int T, int T2, int max_drafts, int n_cap,
                                                         int mask_id, int* node_ids, uint8_t* node_masked,
                                                         const int* prev_ids, int prev_T, int prev_stride, int mix_order) {
  __shared__ int rank[kMaxW];
  __shared__ float cf[kMaxW];
  __shared__ uint8_t mk[kMaxW];
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  if (threadIdx.x == 0) s.last_accept[b] = 0;
  const int r = s.remaining[b];
  if (r <= 0) return;
  max_drafts = min(max_drafts, s.draft_cap[b]);          // (a refresh schedule may shorten a sequence's chain)
  int slot = 0;
  for (int i = 0; i < b; ++i) slot += (s.remaining[i] > 0) ? 1 : 0;
  const int W = T + T2;
  const bool cur_has = (s.has_drafts[b] & 1) != 0, nxt_has = (s.has_drafts[b] & 2) != 0;
  const bool spill = spills(s, b, T2, max_drafts);
  int N = cur_has ? min(max_drafts, r - 1) : 0;
  int n_from_next = 0;
  if (spill) {                       // every masked position of the current block, then the next block's drafts
    if (nxt_has) n_from_next = max(0, min(max_drafts - r, s.remaining_nxt[b] - 1));
    N = r + n_from_next;
  }
  const int* ids = s.ids + (size_t)b * s.stride;
  const uint8_t* masked = s.masked + (size_t)b * s.stride;
  const int* dtok = s.draft_tok + (size_t)b * s.stride;
  const float* dconf = s.draft_conf + (size_t)b * s.stride;
  for (int t = threadIdx.x; t < W; t += blockDim.x) {
    mk[t] = masked[t];
    cf[t] = dconf[t];
  }
  __syncthreads();
  // rank among the masked positions of its own block: how many come strictly before in (confidence desc,
  // position asc); the next block's positions rank behind all of the current block's
  for (int t = threadIdx.x; t < W; t += blockDim.x) {
    int rk = 0x7fffffff;
    const bool in_next = t >= T;
    if (mk[t] && N > 0 && (!in_next || n_from_next > 0)) {
      rk = in_next ? r : 0;
      const float c = cf[t];
      const int lo = in_next ? T : 0, hi = in_next ? W : T;
      for (int u = lo; u < hi; ++u)
        if (mk[u] && (cf[u] > c || (cf[u] == c && u < t))) ++rk;
      if (rk < N) {
        s.cand_pos[(size_t)b * s.stride + rk] = t;
        s.cand_tok[(size_t)b * s.stride + rk] = dtok[t];
      }
    }
    rank[t] = rk;
  }
  if (threadIdx.x == 0) {
    s.n_cand[b] = N;
    s.window[b] = spill ? 1 : 0;
    s.seq_map[slot] = b;
  }
  __syncthreads();
  // rows of a slot: [node][a finished block in front (prev_T tokens, nothing asked) | the W state rows]
  const int node_rows = prev_T + W;
  const size_t base = (size_t)slot * n_cap * node_rows;
  const int n_nodes = tree_nodes(N, mix_order);
  for (int e = threadIdx.x; e < n_cap * node_rows; e += blockDim.x) {
    const int i = e / node_rows, t = e % node_rows - prev_T;
    int id;
    uint8_t m;
    if (t < 0) {
      id = prev_ids[(size_t)b * prev_stride + t + prev_T];
      m = 0;
    } else {
      // chain node i: candidates of rank < i written in; branch of chain node j = i - (N + 1): ranks < j and
      // rank j + 1; nodes beyond the tree repeat node N and ask for nothing.  Next-block rows of a sequence
      // that does not spill carry the next block's state and ask for nothing.
      const bool branch = i > N && i < n_nodes;
      const int depth = branch ? i - (N + 1) : min(i, N);
      if (!mk[t]) { id = ids[t]; m = 0; }
      else if (rank[t] < depth || (branch && rank[t] == depth + 1)) { id = dtok[t]; m = 0; }
      else { id = mask_id; m = (i < n_nodes && (t < T || spill)) ? 1 : 0; }
    }
    node_ids[base + e] = id;
    node_masked[base + e] = m;
  }
}

__global__ void __launch_bounds__(256) accept_kernel(BlockState s, int T, int T2, int n_cap, const int* tok, const float* conf,
                                                     const uint8_t* node_masked, int* nonfinite_flag, int prev_T,
                                                     int mix_order) {
  __shared__ int pred_q[kMaxW];
  __shared__ int pred_t[kMaxW];
  __shared__ int s_a, s_last, s_skip;
  pdl_launch_dependents();
  pdl_wait();
  const int slot = blockIdx.x;
  const int b = s.seq_map[slot];
  const int N = s.n_cand[b];
  const bool spill = s.window[b] != 0;
  const int W = T + T2, node_rows = prev_T + W;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const size_t base = (size_t)slot * n_cap * node_rows + prev_T;        // + i * node_rows: first state row of node i
  const int n_nodes = tree_nodes(N, mix_order);
  for (int i = warp; i < n_nodes; i += nw) {
    const size_t nb = base + (size_t)i * node_rows;
    // the current block while it has a masked position (block order, Section 3.1), else the next block
    bool any = false;
    for (int t = lane; t < T; t += 32) any = any || node_masked[nb + t] != 0;
    const bool in_cur = __any_sync(0xffffffffu, any);
    const int lo = in_cur ? 0 : T, hi = in_cur ? T : (spill ? W : T);
    float bc = -1.f;
    int bq = 0x7fffffff;
    for (int t = lo + lane; t < hi; t += 32) {
      if (node_masked[nb + t]) {
        const float c = conf[nb + t];
        if (c > bc) { bc = c; bq = t; }        // ascending t: strict > keeps the lower position
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float oc = __shfl_xor_sync(0xffffffffu, bc, o);
      const int oq = __shfl_xor_sync(0xffffffffu, bq, o);
      if (oc > bc || (oc == bc && oq < bq)) { bc = oc; bq = oq; }
    }
    if (lane == 0) {
      if (bq >= W) { bq = 0; atomicExch(nonfinite_flag, 1); }   // every confidence was NaN
      pred_q[i] = bq;
      pred_t[i] = tok[nb + bq];
      if (!isfinite(bc)) atomicExch(nonfinite_flag, 1);
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int* cp = s.cand_pos + (size_t)b * s.stride;
    const int* ct = s.cand_tok + (size_t)b * s.stride;
    int a = 0;
    while (a < N && pred_q[a] == cp[a] && pred_t[a] == ct[a]) ++a;
    // out of order: node a predicts candidate a + 2 - take it and move to node a's branch
    const bool skip = mix_order && a + 1 < N && pred_q[a] == cp[a + 1] && pred_t[a] == ct[a + 1];
    s_a = a;
    s_skip = skip ? 1 : 0;
    s_last = skip ? N + 1 + a : a;
  }
  __syncthreads();
  const int a = s_a, last = s_last, n_acc = a + 1 + s_skip;
  int* ids = s.ids + (size_t)b * s.stride;
  uint8_t* masked = s.masked + (size_t)b * s.stride;
  // accepted drafts (with the skipped-to candidate, if any), then the last valid node's own prediction
  for (int j = threadIdx.x; j < a + s_skip; j += blockDim.x) {
    const int c = j < a ? j : a + 1;
    const int p = s.cand_pos[(size_t)b * s.stride + c];
    ids[p] = s.cand_tok[(size_t)b * s.stride + c];
    masked[p] = 0;
  }
  if (threadIdx.x == 0) {
    ids[pred_q[last]] = pred_t[last];
    masked[pred_q[last]] = 0;
  }
  __syncthreads();
  // next drafts: the last valid node's predictions on what is still masked (the next block's too when the
  // sequence spilled into it)
  const size_t lb = base + (size_t)last * node_rows;
  for (int t = threadIdx.x; t < (spill ? W : T); t += blockDim.x) {
    const bool m = masked[t] != 0;
    s.draft_tok[(size_t)b * s.stride + t] = m ? tok[lb + t] : 0;
    s.draft_conf[(size_t)b * s.stride + t] = m ? conf[lb + t] : 0.f;
  }
  if (threadIdx.x == 0) {
    int in_next = 0;                             // accepted positions that lie in the next block
    for (int j = 0; j < a + s_skip; ++j) in_next += (s.cand_pos[(size_t)b * s.stride + (j < a ? j : a + 1)] >= T) ? 1 : 0;
    in_next += (pred_q[last] >= T) ? 1 : 0;
    s.remaining[b] -= n_acc - in_next;
    s.remaining_nxt[b] -= in_next;
    s.has_drafts[b] = 1 | (spill ? 2 : (s.has_drafts[b] & 2));
    const int f = s.n_forwards[b];
    s.accept_log[(size_t)b * s.stride + f] = n_acc;
    s.n_forwards[b] = f + 1;
    s.last_accept[b] = n_acc;
    s.last_pos[b] = pred_q[last];
    s.last_tok[b] = pred_t[last];
  }
}

}  // namespace

void launch_tree_build(cudaStream_t st, BlockState s, int batch, int T, int T2, int max_drafts, int n_cap, int mask_id,
                       int* node_ids, uint8_t* node_masked, const int* prev_ids, int prev_T, int prev_stride,
                       int mix_order) {
  if (!prev_ids) prev_T = 0;
  launch_pdl(tree_build_kernel, dim3(batch), dim3(256), 0, st, s, batch, T, T2, max_drafts, n_cap, mask_id, node_ids,
             node_masked, prev_ids, prev_T, prev_stride, mix_order);
}

void launch_accept(cudaStream_t st, BlockState s, int n_slots, int T, int T2, int n_cap, const int* tok, const float* conf,
                   const uint8_t* node_masked, int* nonfinite_flag, int prev_T, int mix_order) {
  launch_pdl(accept_kernel, dim3(n_slots), dim3(256), 0, st, s, T, T2, n_cap, tok, conf, node_masked, nonfinite_flag,
             prev_T, mix_order);
}

}  // namespace ssd
