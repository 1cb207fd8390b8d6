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
// All integer / comparison work; one CTA per sequence.
#include "kernels.h"

#include <math.h>

namespace ssd {

namespace {

constexpr int kMaxT = 256;

__global__ void __launch_bounds__(256) tree_build_kernel(BlockState s, int batch, int T, int max_drafts, int n_cap,
                                                         int mask_id, int* node_ids, uint8_t* node_masked,
                                                         const int* prev_ids, int prev_T, int prev_stride, int mix_order) {
  __shared__ int rank[kMaxT];
  __shared__ float cf[kMaxT];
  __shared__ uint8_t mk[kMaxT];
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  if (threadIdx.x == 0) s.last_accept[b] = 0;
  const int r = s.remaining[b];
  if (r <= 0) return;
  int slot = 0;
  for (int i = 0; i < b; ++i) slot += (s.remaining[i] > 0) ? 1 : 0;
  const int N = s.has_drafts[b] ? min(max_drafts, r - 1) : 0;
  const int* ids = s.ids + (size_t)b * s.stride;
  const uint8_t* masked = s.masked + (size_t)b * s.stride;
  const int* dtok = s.draft_tok + (size_t)b * s.stride;
  const float* dconf = s.draft_conf + (size_t)b * s.stride;
  for (int t = threadIdx.x; t < T; t += blockDim.x) {
    mk[t] = masked[t];
    cf[t] = dconf[t];
  }
  __syncthreads();
  // rank among the masked positions: how many come strictly before in (confidence desc, position asc)
  for (int t = threadIdx.x; t < T; t += blockDim.x) {
    int rk = 0x7fffffff;
    if (mk[t] && N > 0) {
      rk = 0;
      const float c = cf[t];
      for (int u = 0; u < T; ++u)
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
    s.seq_map[slot] = b;
  }
  __syncthreads();
  size_t base = (size_t)slot * (prev_T + n_cap * T);
  for (int e = threadIdx.x; e < prev_T; e += blockDim.x) {      // the finished block in front: tokens, nothing asked
    node_ids[base + e] = prev_ids[(size_t)b * prev_stride + e];
    node_masked[base + e] = 0;
  }
  base += prev_T;
  const int n_nodes = tree_nodes(N, mix_order);
  for (int e = threadIdx.x; e < n_cap * T; e += blockDim.x) {
    const int i = e / T, t = e % T;
    // chain node i: candidates of rank < i written in; branch of chain node j = i - (N + 1): ranks < j and
    // rank j + 1; nodes beyond the tree repeat node N and ask for nothing
    const bool branch = i > N && i < n_nodes;
    const int depth = branch ? i - (N + 1) : min(i, N);
    int id;
    uint8_t m;
    if (!mk[t]) { id = ids[t]; m = 0; }
    else if (rank[t] < depth || (branch && rank[t] == depth + 1)) { id = dtok[t]; m = 0; }
    else { id = mask_id; m = (i < n_nodes) ? 1 : 0; }
    node_ids[base + e] = id;
    node_masked[base + e] = m;
  }
}

__global__ void __launch_bounds__(256) accept_kernel(BlockState s, int T, int n_cap, const int* tok, const float* conf,
                                                     const uint8_t* node_masked, int* nonfinite_flag, int slot_rows,
                                                     int row_offset, int mix_order) {
  __shared__ int pred_q[2 * kMaxT];
  __shared__ int pred_t[2 * kMaxT];
  __shared__ int s_a, s_last, s_skip;
  pdl_launch_dependents();
  pdl_wait();
  const int slot = blockIdx.x;
  const int b = s.seq_map[slot];
  const int N = s.n_cand[b];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const size_t base = (size_t)slot * slot_rows + row_offset;
  const int n_nodes = tree_nodes(N, mix_order);
  for (int i = warp; i < n_nodes; i += nw) {
    float bc = -1.f;
    int bq = 0x7fffffff;
    for (int t = lane; t < T; t += 32) {
      if (node_masked[base + (size_t)i * T + t]) {
        const float c = conf[base + (size_t)i * T + t];
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
      if (bq >= T) { bq = 0; atomicExch(nonfinite_flag, 1); }   // every confidence was NaN
      pred_q[i] = bq;
      pred_t[i] = tok[base + (size_t)i * T + bq];
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
  // next drafts: the last valid node's predictions on what is still masked
  for (int t = threadIdx.x; t < T; t += blockDim.x) {
    const bool m = masked[t] != 0;
    s.draft_tok[(size_t)b * s.stride + t] = m ? tok[base + (size_t)last * T + t] : 0;
    s.draft_conf[(size_t)b * s.stride + t] = m ? conf[base + (size_t)last * T + t] : 0.f;
  }
  if (threadIdx.x == 0) {
    s.remaining[b] -= n_acc;
    s.has_drafts[b] = 1;
    const int f = s.n_forwards[b];
    s.accept_log[(size_t)b * s.stride + f] = n_acc;
    s.n_forwards[b] = f + 1;
    s.last_accept[b] = n_acc;
    s.last_pos[b] = pred_q[last];
    s.last_tok[b] = pred_t[last];
  }
}

}  // namespace

void launch_tree_build(cudaStream_t st, BlockState s, int batch, int T, int max_drafts, int n_cap, int mask_id,
                       int* node_ids, uint8_t* node_masked, const int* prev_ids, int prev_T, int prev_stride,
                       int mix_order) {
  if (!prev_ids) prev_T = 0;
  launch_pdl(tree_build_kernel, dim3(batch), dim3(256), 0, st, s, batch, T, max_drafts, n_cap, mask_id, node_ids,
             node_masked, prev_ids, prev_T, prev_stride, mix_order);
}

void launch_accept(cudaStream_t st, BlockState s, int n_slots, int T, int n_cap, const int* tok, const float* conf,
                   const uint8_t* node_masked, int* nonfinite_flag, int slot_rows, int row_offset, int mix_order) {
  if (slot_rows <= 0) { slot_rows = n_cap * T; row_offset = 0; }
  launch_pdl(accept_kernel, dim3(n_slots), dim3(256), 0, st, s, T, n_cap, tok, conf, node_masked, nonfinite_flag,
             slot_rows, row_offset, mix_order);
}

}  // namespace ssd
