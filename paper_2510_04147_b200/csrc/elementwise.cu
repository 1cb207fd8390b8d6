// Small memory-bound kernels around the projections: weight repacking, embedding gather, QKV
// finalisation with rotary embedding (cache-fill forward), softmax statistics.
// Every reduction has a fixed order that depends on the row alone, so a row's result does not
// depend on how many other rows share the launch.
#include "kernels.h"

#include <math.h>

namespace ssd {

namespace {

constexpr int kThreads = 256;

// Deterministic block-wide sum (xor butterfly inside warps, then warp partials in warp order).
__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = 0.f;
  const int nw = blockDim.x >> 5;
  for (int i = 0; i < nw; ++i) t += red[i];
  return t;
}

__global__ void convert_rows_kernel(const void* src, int src_is_f32, bf16* dst, int rows, int cols, int dst_pitch,
                                    int group, int group_stride, int group_offset) {
  const size_t total = (size_t)rows * cols;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int j = (int)(i / cols), c = (int)(i % cols);
    const float v = src_is_f32 ? ((const float*)src)[i] : __bfloat162float(((const bf16*)src)[i]);
    const size_t dr = (size_t)(j / group) * group_stride + group_offset + (j % group);
    dst[dr * dst_pitch + c] = __float2bfloat16_rn(v);
  }
}

__global__ void convert_tiled_kernel(const void* src, int src_is_f32, bf16* dst, int rows, int cols, int kb_total,
                                     int group, int group_stride, int group_offset) {
  const size_t total = (size_t)rows * cols;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int j = (int)(i / cols), c = (int)(i % cols);
    const float v = src_is_f32 ? ((const float*)src)[i] : __bfloat162float(((const bf16*)src)[i]);
    const size_t n = (size_t)(j / group) * group_stride + group_offset + (j % group);
    dst[(((n >> 7) * kb_total + (c >> 6)) * 128 + (n & 127)) * 64 + (c & 63)] = __float2bfloat16_rn(v);
  }
}

__global__ void copy_f32_kernel(const void* src, int src_is_f32, float* dst, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src_is_f32 ? ((const float*)src)[i] : __bfloat162float(((const bf16*)src)[i]);
}

constexpr int kRowThreadsMax = 1024;   // one float4 per thread up to d = 4096

__global__ void __launch_bounds__(kRowThreadsMax) embed_prep_kernel(const int* ids, const bf16* embed, const float* gain,
                                                                    float* h, bf16* hb, float* sq, int sq_stride, int d,
                                                                    int V) {
  __shared__ float red[kRowThreadsMax / 32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  // ids come from the device-side decode state: never index the table with one outside the vocabulary
  int id = ids[r];
  if ((unsigned)id >= (unsigned)V) id = 0;
  const bf16* e = embed + (size_t)id * d;
  float ss = 0.f;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(e + c);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(e + c + 2);
    const float4 g = *reinterpret_cast<const float4*>(gain + c);
    const float4 v = make_float4(__low2float(a), __high2float(a), __low2float(b), __high2float(b));
    *reinterpret_cast<float4*>(h + (size_t)r * d + c) = v;
    *reinterpret_cast<__nv_bfloat162*>(hb + (size_t)r * d + c) = __floats2bfloat162_rn(v.x * g.x, v.y * g.y);
    *reinterpret_cast<__nv_bfloat162*>(hb + (size_t)r * d + c + 2) = __floats2bfloat162_rn(v.z * g.z, v.w * g.w);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = block_sum(ss, red);
  if (threadIdx.x == 0) sq[(size_t)r * sq_stride] = ss;
}

// The same producer step for a residual stream that is already in h (a forward entered at a
// later layer): hb[r] = bf16(h[r] * gain); sq[r * sq_stride] = sum of squares of h[r]
__global__ void __launch_bounds__(kRowThreadsMax) stream_prep_kernel(const float* h, const float* gain, bf16* hb,
                                                                     float* sq, int sq_stride, int d) {
  __shared__ float red[kRowThreadsMax / 32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  float ss = 0.f;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(h + (size_t)r * d + c);
    const float4 g = *reinterpret_cast<const float4*>(gain + c);
    *reinterpret_cast<__nv_bfloat162*>(hb + (size_t)r * d + c) = __floats2bfloat162_rn(v.x * g.x, v.y * g.y);
    *reinterpret_cast<__nv_bfloat162*>(hb + (size_t)r * d + c + 2) = __floats2bfloat162_rn(v.z * g.z, v.w * g.w);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = block_sum(ss, red);
  if (threadIdx.x == 0) sq[(size_t)r * sq_stride] = ss;
}

// One CTA per (row, group of 8 heads of the fused q|k|v output); a warp per head.
constexpr int kRopeHeadsPerBlock = 8;
__global__ void __launch_bounds__(kRopeHeadsPerBlock * 32) qkv_rope_kernel(const float* partial, int splits,
                                                                            size_t split_stride, int H, int Hkv, int hd,
                                                                            const float2* rope_table, RowMap map,
                                                                            bf16* q, bf16* k_dst, bf16* v_dst,
                                                                            int kv_to_cache, size_t cache_seq_stride,
                                                                            size_t kv_pos_stride, size_t kv_head_stride) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  const int head = blockIdx.y * kRopeHeadsPerBlock + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (head >= H + 2 * Hkv) return;
  const int half = hd >> 1;
  const int nqkv = (H + 2 * Hkv) * hd;
  const int slot = r / map.rows_per_seq;
  const int t = r % map.T;
  const int pos = map.pos0 + t;
  const int seq = map.seq_map ? map.seq_map[slot] : map.seq_base + slot;
  const float* prow = partial + (size_t)r * nqkv + (size_t)head * hd;
  // destination of KV head j of this row: the cache, or a plain [row][Hkv][hd] buffer
  const size_t kv_row = kv_to_cache ? ((size_t)seq * cache_seq_stride + (size_t)pos * kv_pos_stride) : (size_t)r * Hkv * hd;
  const size_t kv_head = kv_to_cache ? kv_head_stride : (size_t)hd;
  if (head < H + Hkv) {
    const float2* rt = rope_table + (size_t)pos * half;
    bf16* dst = head < H ? q + ((size_t)r * H + head) * hd : k_dst + kv_row + (size_t)(head - H) * kv_head;
    for (int i = lane; i < half; i += 32) {
      float x1 = 0.f, x2 = 0.f;
      for (int s = 0; s < splits; ++s) {
        x1 += prow[s * split_stride + i];
        x2 += prow[s * split_stride + i + half];
      }
      const float2 cs = rt[i];
      dst[i] = __float2bfloat16_rn(x1 * cs.x - x2 * cs.y);
      dst[i + half] = __float2bfloat16_rn(x2 * cs.x + x1 * cs.y);
    }
  } else {
    bf16* dst = v_dst + kv_row + (size_t)(head - H - Hkv) * kv_head;
    for (int e = lane; e < hd; e += 32) {
      float x = 0.f;
      for (int s = 0; s < splits; ++s) x += prow[s * split_stride + e];
      dst[e] = __float2bfloat16_rn(x);
    }
  }
}

__global__ void __launch_bounds__(kThreads) lm_stats_from_logits_kernel(const float* logits, int V, int mask_id,
                                                                        const uint8_t* row_wanted, int* tok,
                                                                        float* conf) {
  __shared__ float red[kThreads / 32];
  __shared__ float s_m[kThreads / 32];
  __shared__ int s_a[kThreads / 32];
  const int r = blockIdx.x;
  if (row_wanted && !row_wanted[r]) {
    if (threadIdx.x == 0) { tok[r] = -1; conf[r] = 0.f; }
    return;
  }
  const float* l = logits + (size_t)r * V;
  float m = -INFINITY;
  int a = 0x7fffffff;
  for (int v = threadIdx.x; v < V; v += kThreads) {
    const float x = (v == mask_id) ? -INFINITY : l[v];
    if (x > m) { m = x; a = v; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o);
    const int oa = __shfl_xor_sync(0xffffffffu, a, o);
    if (om > m || (om == m && oa < a)) { m = om; a = oa; }
  }
  if ((threadIdx.x & 31) == 0) { s_m[threadIdx.x >> 5] = m; s_a[threadIdx.x >> 5] = a; }
  __syncthreads();
  m = s_m[0]; a = s_a[0];
  for (int i = 1; i < kThreads / 32; ++i)
    if (s_m[i] > m || (s_m[i] == m && s_a[i] < a)) { m = s_m[i]; a = s_a[i]; }
  float s = 0.f;
  for (int v = threadIdx.x; v < V; v += kThreads)
    if (v != mask_id) s += expf(l[v] - m);
  s = block_sum(s, red);
  // non-finite logits leave no valid argmax: the token stays inside the vocabulary, the confidence says so
  if (threadIdx.x == 0) { tok[r] = ((unsigned)a >= (unsigned)V) ? 0 : a; conf[r] = 1.f / s; }
}

// Symmetric merge of two (max, sum-exp, argmax) triples: both partners of a butterfly step compute
// bit-identical results, and ties keep the lower token id.
__device__ __forceinline__ void stat_merge(float& m, float& s, int& a, float om, float os, int oa) {
  const float nm = fmaxf(m, om);
  if (nm == -INFINITY) return;
  const float lo_m = fminf(m, om);
  const float hi_s = (m >= om) ? s : os;
  const float lo_s = (m >= om) ? os : s;
  const float ns = (m == om) ? (s + os) : (hi_s + lo_s * expf(lo_m - nm));
  int na;
  if (m == om) na = min(a, oa); else na = (m > om) ? a : oa;
  m = nm; s = ns; a = na;
}

// One CTA per row: threads stride over the vocabulary tiles, butterfly inside each warp, then the
// warp results in warp order.  The order depends on the tile count alone.
__global__ void __launch_bounds__(kThreads) lm_merge_kernel(const float* tile_max, const float* tile_sum,
                                                            const int* tile_arg, int tiles, int R, int V,
                                                            const uint8_t* row_wanted, int* tok, float* conf) {
  __shared__ float w_m[kThreads / 32], w_s[kThreads / 32];
  __shared__ int w_a[kThreads / 32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (row_wanted && !row_wanted[r]) {
    if (threadIdx.x == 0) { tok[r] = -1; conf[r] = 0.f; }
    return;
  }
  float m = -INFINITY, s = 0.f;
  int a = 0x7fffffff;
  for (int t = threadIdx.x; t < tiles; t += kThreads) {
    const float tm = tile_max[(size_t)t * R + r];
    if (tm == -INFINITY) continue;
    const float ts = tile_sum[(size_t)t * R + r];
    const int ta = tile_arg[(size_t)t * R + r];
    if (tm > m) { s = s * expf(m - tm) + ts; m = tm; a = ta; }   // expf(-inf) = 0 on the first hit
    else { s += ts * expf(tm - m); if (tm == m && ta < a) a = ta; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o);
    const float os = __shfl_xor_sync(0xffffffffu, s, o);
    const int oa = __shfl_xor_sync(0xffffffffu, a, o);
    stat_merge(m, s, a, om, os, oa);
  }
  if (lane == 0) { w_m[warp] = m; w_s[warp] = s; w_a[warp] = a; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < kThreads / 32; ++i) stat_merge(m, s, a, w_m[i], w_s[i], w_a[i]);
    // non-finite logits leave no valid argmax: the token stays inside the vocabulary, the confidence says so
    tok[r] = ((unsigned)a >= (unsigned)V) ? 0 : a;
    conf[r] = 1.f / s;
  }
}

// The k most probable tokens of a row from the per-tile candidate lists.  One CTA per row: a thread
// keeps the best k of the tiles it strides over (tile order, so equal values keep the lower index), the
// threads' sorted lists are merged per warp by k rounds of a warp-wide argmax over the list heads, and
// thread 0 merges the warps' lists the same way.  prob = exp(logit - max) * conf, conf = 1 / sum-exp.
__global__ void __launch_bounds__(kThreads) lm_merge_topk_kernel(const float* tile_topv, const int* tile_topi, int tiles,
                                                                 int R, int V, int k, const uint8_t* row_wanted,
                                                                 const float* conf, int* topk_tok, float* topk_prob) {
  __shared__ float w_v[kThreads / 32][kLmTopKMax];
  __shared__ int w_i[kThreads / 32][kLmTopKMax];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (row_wanted && !row_wanted[r]) {
    for (int j = threadIdx.x; j < kLmTopKMax; j += kThreads) { topk_tok[(size_t)r * kLmTopKMax + j] = -1; topk_prob[(size_t)r * kLmTopKMax + j] = 0.f; }
    return;
  }
  float bv[kLmTopKMax];
  int bi[kLmTopKMax];
#pragma unroll
  for (int j = 0; j < kLmTopKMax; ++j) { bv[j] = -INFINITY; bi[j] = 0x7fffffff; }
  for (int t = threadIdx.x; t < tiles; t += kThreads) {
    const size_t o = ((size_t)t * R + r) * kLmTopKMax;
    for (int c = 0; c < k; ++c) {
      float v = tile_topv[o + c];
      int i = tile_topi[o + c];
      if (!(v > bv[k - 1] || (v == bv[k - 1] && i < bi[k - 1]))) break;      // a tile's list is sorted: the rest is worse
#pragma unroll
      for (int j = 0; j < kLmTopKMax; ++j) {                                   // insert, keeping (value desc, index asc)
        if (j < k && (v > bv[j] || (v == bv[j] && i < bi[j]))) {
          const float tv = bv[j]; const int ti = bi[j];
          bv[j] = v; bi[j] = i; v = tv; i = ti;
        }
      }
    }
  }
  // warp merge: k rounds over the heads of the 32 sorted lists
  int head = 0;
  for (int c = 0; c < k; ++c) {
    float m = -INFINITY;
    int a = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < kLmTopKMax; ++j)
      if (j == head) { m = bv[j]; a = bi[j]; }
    float wm = m;
    int wa = a;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, wm, o);
      const int oa = __shfl_xor_sync(0xffffffffu, wa, o);
      if (om > wm || (om == wm && oa < wa)) { wm = om; wa = oa; }
    }
    if (wm == m && wa == a && a != 0x7fffffff) ++head;      // (indices are unique: exactly one lane advances)
    if (lane == 0) { w_v[warp][c] = wm; w_i[warp][c] = wa; }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int hd[kThreads / 32];
    for (int q = 0; q < kThreads / 32; ++q) hd[q] = 0;
    float top = -INFINITY;
    for (int c = 0; c < k; ++c) {
      float bm = -INFINITY;
      int ba = 0x7fffffff, bq = 0;
      for (int q = 0; q < kThreads / 32; ++q) {
        if (hd[q] < k) {
          const float m = w_v[q][hd[q]];
          const int a = w_i[q][hd[q]];
          if (m > bm || (m == bm && a < ba)) { bm = m; ba = a; bq = q; }
        }
      }
      ++hd[bq];
      if (c == 0) top = bm;
      const bool valid = (unsigned)ba < (unsigned)V && bm != -INFINITY;
      topk_tok[(size_t)r * kLmTopKMax + c] = valid ? ba : -1;
      topk_prob[(size_t)r * kLmTopKMax + c] = valid ? expf(bm - top) * conf[r] : 0.f;
    }
    for (int c = k; c < kLmTopKMax; ++c) { topk_tok[(size_t)r * kLmTopKMax + c] = -1; topk_prob[(size_t)r * kLmTopKMax + c] = 0.f; }
  }
}


}  // namespace

void launch_convert_rows(cudaStream_t st, const void* src, int src_is_f32, bf16* dst, int rows, int cols, int dst_pitch,
                         int group, int group_stride, int group_offset) {
  const size_t total = (size_t)rows * cols;
  int blocks = (int)((total + 255) / 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  convert_rows_kernel<<<blocks, 256, 0, st>>>(src, src_is_f32, dst, rows, cols, dst_pitch, group, group_stride,
                                              group_offset);
}

void launch_convert_tiled(cudaStream_t st, const void* src, int src_is_f32, bf16* dst, int rows, int cols, int kb_total,
                          int group, int group_stride, int group_offset) {
  const size_t total = (size_t)rows * cols;
  int blocks = (int)((total + 255) / 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  convert_tiled_kernel<<<blocks, 256, 0, st>>>(src, src_is_f32, dst, rows, cols, kb_total, group, group_stride,
                                               group_offset);
}

void launch_copy_f32(cudaStream_t st, const void* src, int src_is_f32, float* dst, int n) {
  copy_f32_kernel<<<(n + 255) / 256, 256, 0, st>>>(src, src_is_f32, dst, n);
}

static int row_threads(int d) {
  int t = ((d / 4 + 31) / 32) * 32;
  if (t > kRowThreadsMax) t = kRowThreadsMax;
  if (t < 32) t = 32;
  return t;
}

void launch_embed_prep(cudaStream_t st, const int* ids, const bf16* embed, const float* gain, float* h, bf16* hb,
                       float* sq, int sq_stride, int R, int d, int V) {
  launch_pdl(embed_prep_kernel, dim3(R), dim3(row_threads(d)), 0, st, ids, embed, gain, h, hb, sq, sq_stride, d, V);
}

void launch_stream_prep(cudaStream_t st, const float* h, const float* gain, bf16* hb, float* sq, int sq_stride, int R,
                        int d) {
  launch_pdl(stream_prep_kernel, dim3(R), dim3(row_threads(d)), 0, st, h, gain, hb, sq, sq_stride, d);
}

void launch_qkv_rope(cudaStream_t st, const float* partial, int splits, size_t split_stride, int R, int H, int Hkv,
                     int hd, const float2* rope_table, RowMap map, bf16* q, bf16* k_dst, bf16* v_dst, int kv_to_cache,
                     size_t cache_seq_stride, size_t kv_pos_stride, size_t kv_head_stride) {
  const int heads = H + 2 * Hkv;
  dim3 grid(R, (heads + kRopeHeadsPerBlock - 1) / kRopeHeadsPerBlock);
  launch_pdl(qkv_rope_kernel, grid, dim3(kRopeHeadsPerBlock * 32), 0, st, partial, splits, split_stride, H, Hkv, hd,
             rope_table, map, q, k_dst, v_dst, kv_to_cache, cache_seq_stride, kv_pos_stride, kv_head_stride);
}

void launch_lm_stats_from_logits(cudaStream_t st, const float* logits, int R, int V, int mask_id,
                                 const uint8_t* row_wanted, int* tok, float* conf) {
  lm_stats_from_logits_kernel<<<R, kThreads, 0, st>>>(logits, V, mask_id, row_wanted, tok, conf);
}

void launch_lm_merge(cudaStream_t st, const float* tile_max, const float* tile_sum, const int* tile_arg, int tiles,
                     int R, int V, const uint8_t* row_wanted, int* tok, float* conf) {
  launch_pdl(lm_merge_kernel, dim3(R), dim3(kThreads), 0, st, tile_max, tile_sum, tile_arg, tiles, R, V, row_wanted,
             tok, conf);
}

void launch_lm_merge_topk(cudaStream_t st, const float* tile_topv, const int* tile_topi, int tiles, int R, int V, int k,
                          const uint8_t* row_wanted, const float* conf, int* topk_tok, float* topk_prob) {
  launch_pdl(lm_merge_topk_kernel, dim3(R), dim3(kThreads), 0, st, tile_topv, tile_topi, tiles, R, V, k, row_wanted,
             conf, topk_tok, topk_prob);
}

}  // namespace ssd
