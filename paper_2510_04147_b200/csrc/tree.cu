// Tree build and acceptance for the greedy verification chain (Sections 3.2.2 - 3.2.4).
//
// tree_build: per unfinished sequence, order the stale drafts of the masked positions by
//   confidence (descending, lower position first on ties), keep N = min(max_drafts, r-1), and
//   write the N+1 node rows: node i = block state with candidates 1..i written in.
// accept: per node the position a stepwise step would fill (highest confidence among the node's
//   masked rows, lower position on ties) and its token; walk the chain while node i's prediction
//   equals candidate i+1 (position AND token); write the accepted tokens, the next drafts (the
//   last valid node's own predictions) and the bookkeeping.
// All integer / comparison work; one CTA per sequence.
#include "kernels.h"

#include <math.h>

namespace ssd {

namespace {

constexpr int kMaxT = 256;

__global__ void __launch_bounds__(256) tree_build_kernel(BlockState s, int batch, int T, int max_drafts, int n_cap,
                                                         int mask_id, int* node_ids, uint8_t* node_masked,
                                                         const int* prev_ids, int prev_T, int prev_stride) {
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
  for (int e = threadIdx.x; e < n_cap * T; e += blockDim.x) {
    const int i = e / T, t = e % T;
    const int depth = min(i, N);                 // nodes beyond N repeat node N and ask for nothing
    int id;
    uint8_t m;
    if (!mk[t]) { id = ids[t]; m = 0; }
    else if (rank[t] < depth) { id = dtok[t]; m = 0; }
    else { id = mask_id; m = (i <= N) ? 1 : 0; }
    node_ids[base + e] = id;
    node_masked[base + e] = m;
  }
}

__global__ void __launch_bounds__(256) accept_kernel(BlockState s, int T, int n_cap, const int* tok, const float* conf,
                                                     const uint8_t* node_masked, int* nonfinite_flag, int slot_rows,
                                                     int row_offset) {
  __shared__ int pred_q[kMaxT];
  __shared__ int pred_t[kMaxT];
  __shared__ int s_a;
  pdl_launch_dependents();
  pdl_wait();
  const int slot = blockIdx.x;
  const int b = s.seq_map[slot];
  const int N = s.n_cand[b];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const size_t base = (size_t)slot * slot_rows + row_offset;
  for (int i = warp; i <= N; i += nw) {
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
    int a = 0;
    while (a < N && pred_q[a] == s.cand_pos[(size_t)b * s.stride + a] &&
           pred_t[a] == s.cand_tok[(size_t)b * s.stride + a])
      ++a;
    s_a = a;
  }
  __syncthreads();
  const int a = s_a;
  int* ids = s.ids + (size_t)b * s.stride;
  uint8_t* masked = s.masked + (size_t)b * s.stride;
  // accepted drafts, then the last valid node's own prediction
  for (int j = threadIdx.x; j < a; j += blockDim.x) {
    const int p = s.cand_pos[(size_t)b * s.stride + j];
    ids[p] = s.cand_tok[(size_t)b * s.stride + j];
    masked[p] = 0;
  }
  if (threadIdx.x == 0) {
    ids[pred_q[a]] = pred_t[a];
    masked[pred_q[a]] = 0;
  }
  __syncthreads();
  // next drafts: node a's predictions on what is still masked
  for (int t = threadIdx.x; t < T; t += blockDim.x) {
    const bool m = masked[t] != 0;
    s.draft_tok[(size_t)b * s.stride + t] = m ? tok[base + (size_t)a * T + t] : 0;
    s.draft_conf[(size_t)b * s.stride + t] = m ? conf[base + (size_t)a * T + t] : 0.f;
  }
  if (threadIdx.x == 0) {
    s.remaining[b] -= a + 1;
    s.has_drafts[b] = 1;
    const int f = s.n_forwards[b];
    s.accept_log[(size_t)b * s.stride + f] = a + 1;
    s.n_forwards[b] = f + 1;
    s.last_accept[b] = a + 1;
  }
}

}  // namespace

void launch_tree_build(cudaStream_t st, BlockState s, int batch, int T, int max_drafts, int n_cap, int mask_id,
                       int* node_ids, uint8_t* node_masked, const int* prev_ids, int prev_T, int prev_stride) {
  if (!prev_ids) prev_T = 0;
  launch_pdl(tree_build_kernel, dim3(batch), dim3(256), 0, st, s, batch, T, max_drafts, n_cap, mask_id, node_ids,
             node_masked, prev_ids, prev_T, prev_stride);
}

void launch_accept(cudaStream_t st, BlockState s, int n_slots, int T, int n_cap, const int* tok, const float* conf,
                   const uint8_t* node_masked, int* nonfinite_flag, int slot_rows, int row_offset) {
  if (slot_rows <= 0) { slot_rows = n_cap * T; row_offset = 0; }
  launch_pdl(accept_kernel, dim3(n_slots), dim3(256), 0, st, s, T, n_cap, tok, conf, node_masked, nonfinite_flag,
             slot_rows, row_offset);
}

}  // namespace ssd
