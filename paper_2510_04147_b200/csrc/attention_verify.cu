// Shared-prefix bidirectional attention of the verification forward (Eq. 5), one kernel.
//
// Rows are ordered [sequence slot][node][in-block index].  A query row attends, without a causal
// mask, to the cached prefix keys of its sequence and to the keys of ITS OWN node's block.  The
// keys are cut into parts: prefix parts whose boundaries depend on the prefix length only, plus one
// node-local part (masked block-diagonally: key and query must belong to the same node).  The
// parts of one (64-row query tile, head) form a thread-block cluster, one CTA per part, so a
// prefix K/V tile is read once for all tree nodes of the tile.
//
// Prologue: the rotated Q tile - and, in the CTA of the local part, the rotated K and the V of the
// tile's own nodes - are built straight from the fp32 split-K partials of the QKV projection
// (sum over splits in split order, rotary embedding at the absolute position), so there is no
// separate rotary pass and no q/k/v round trip through HBM.  The cached prefix does not depend on
// any earlier kernel of the forward: its first tiles are requested before the dependency wait.
//
// Main loop: eight warps = four groups of 16 query rows x two key sets; key set s takes the
// 64-key tiles with (tile & 1) == s of the part.  Online softmax in the log2 domain, mma.sync
// (bf16 in, fp32 accumulate): attention is < 3 % of the forward's flops and latency-bound.
//
// Epilogue: every warp publishes (max, sum, unnormalised output) of its (rows, key set) in shared
// memory; after a cluster barrier CTA p normalises the rows r with r % parts == p, reading all
// 2 * parts sub-parts through distributed shared memory and merging them in (part, key set) order.
// Every reduction order depends on the row and the prefix length alone, never on the row count.
#include "attn_common.cuh"

namespace ssd {

namespace {

using namespace attn;

constexpr int kPairKeys = 2 * kKTile;      // keys per loop step: one tile per key set

__device__ __forceinline__ void cluster_arrive() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
}
// per-thread form for code where the threads of a warp may have diverged
__device__ __forceinline__ void cluster_arrive_thread() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
__device__ __forceinline__ void st_cluster_u4(uint32_t addr, uint4 v) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release;\nbarrier.cluster.wait.acquire;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_rank(const void* p, uint32_t rank) {
  uint32_t out;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(smem_u32(p)), "r"(rank));
  return out;
}
// volatile keeps these after the cluster barrier; no memory clobber, so several can be in flight
__device__ __forceinline__ float2 ld_cluster_f32x2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}

// MINB: CTAs per SM the register allocation must allow (3 trades a few spills for one wave at 64 rows)
template <int HD, int QT, int MINB>
__global__ void __launch_bounds__(QT * 4, MINB) attn_verify_kernel(AttnArgs a, int n_prefix_parts, int nbuf,
                                                                     float scale_log2) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  constexpr int kQTile = QT;                                    // query rows per CTA: 32 or 64
  constexpr int kVerifyThreads = QT * 4;                        // (QT / 16 row groups) x 2 key sets, one warp each
  bf16* sQ = reinterpret_cast<bf16*>(smem_raw);                 // [QT][HD]
  bf16* sKV = sQ + kQTile * HD;                                 // nbuf x { K [128][HD], V [128][HD] }
  constexpr int CH = HD / 8;                                    // 16-byte chunks per row
  constexpr int HALF = HD / 2;
  constexpr int kBufElems = 2 * kPairKeys * HD;

  pdl_launch_dependents();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gq = lane >> 2, tq = lane & 3;
  const int rg = warp % (QT / 16), kset = warp / (QT / 16);
  const int n_parts = n_prefix_parts + 1;
  const int part = blockIdx.x, h = blockIdx.y;                  // the cluster spans x
  const int q_tiles = (a.map.rows_per_seq + kQTile - 1) / kQTile;
  const int qt = blockIdx.z % q_tiles, slot = blockIdx.z / q_tiles;
  const int kvh = h / (a.H / a.Hkv);
  const int rps = a.map.rows_per_seq, T = a.map.T;
  const int lr0 = qt * kQTile;                                  // first sequence-local query row
  const size_t grow0 = (size_t)slot * rps + lr0;                // first global row
  const bool local = part == n_prefix_parts;
  const int nqkv = (a.H + 2 * a.Hkv) * HD;

  int k_begin, k_end;
  if (!local) {
    k_begin = part * a.kv_split;
    k_end = min(a.S, k_begin + a.kv_split);
  } else {
    const int last = min(lr0 + kQTile - 1, rps - 1);
    k_begin = (lr0 / T) * T;
    k_end = (last / T + 1) * T;
  }
  const int n_tiles = (k_end - k_begin + kKTile - 1) / kKTile;
  const int n_pairs = (n_tiles + 1) / 2;

  // ---- prefix K/V: asynchronous copies from the cache, 128 keys per step
  auto load_prefix = [&](int pair, int buf) {
    const int seq = seq_of_slot(a.map, slot);
    const bf16* kbase = a.cache_k + (size_t)seq * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride;
    const bf16* vbase = a.cache_v + (size_t)seq * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride;
    const size_t krow_stride = a.kv_pos_stride;
    const int key0 = k_begin + pair * kPairKeys;
    bf16* dK = sKV + (size_t)buf * kBufElems;
    bf16* dV = dK + kPairKeys * HD;
    for (int idx = tid; idx < kPairKeys * CH; idx += kVerifyThreads) {
      const int row = idx / CH, ch = idx % CH;
      const int key = key0 + row;
      const bool valid = key < k_end;
      int crow = valid ? key : k_begin;                       // cache row of the key (a hole skips the block's own rows)
      if (crow >= a.hole_begin) crow += a.hole_len;
      const size_t off = (size_t)crow * krow_stride + ch * 8;
      cp_async16(dK + swz<HD>(row, ch), kbase + off, valid);
      cp_async16(dV + swz<HD>(row, ch), vbase + off, valid);
    }
  };
  // block commit: the first query head of a KV group also stores the rows' K/V into the cache.
  // Sequence-local row lr is in-block index lr (one node per sequence) at position pos0 + lr.
  const bool commit_kv = a.cache_k_out != nullptr && (h % (a.H / a.Hkv)) == 0;
  const int commit_rows = a.map.chain_T0 > 0 ? a.map.chain_T0 : rps;   // sequence-local rows whose K/V are cached
  auto cache_row = [&](int lr) -> size_t {
    return (size_t)seq_of_slot(a.map, slot) * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride + (size_t)(a.map.pos0 + lr) * a.kv_pos_stride;
  };
  // ---- one chunk (8 rotation pairs) of one row of a head of the fused projection: sum over the
  //      splits in split order (four splits' loads in flight at a time), rotary embedding, bf16
  auto rot_item = [&](int lr, int c, int col0, uint4& lo, uint4& hi) {
    float x1[8], x2[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { x1[j] = 0.f; x2[j] = 0.f; }
    const float* pr = a.qkv_partial + ((size_t)slot * rps + lr) * nqkv + col0 + c * 8;
    const float4* cs4 = reinterpret_cast<const float4*>(a.rope + (size_t)(a.map.pos0 + lr % T) * HALF + c * 8);
    float4 cs[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) cs[j] = cs4[j];              // (cos, sin) of pairs 2j and 2j+1
    for (int s0 = 0; s0 < a.qkv_splits; s0 += 4) {
      float4 a0[4], a1[4], b0[4], b1[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        a0[u] = a1[u] = b0[u] = b1[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (s0 + u < a.qkv_splits) {
          const float* ps = pr + (size_t)(s0 + u) * a.qkv_split_stride;
          a0[u] = *reinterpret_cast<const float4*>(ps);
          a1[u] = *reinterpret_cast<const float4*>(ps + 4);
          b0[u] = *reinterpret_cast<const float4*>(ps + HALF);
          b1[u] = *reinterpret_cast<const float4*>(ps + HALF + 4);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (s0 + u < a.qkv_splits) {
          x1[0] += a0[u].x; x1[1] += a0[u].y; x1[2] += a0[u].z; x1[3] += a0[u].w;
          x1[4] += a1[u].x; x1[5] += a1[u].y; x1[6] += a1[u].z; x1[7] += a1[u].w;
          x2[0] += b0[u].x; x2[1] += b0[u].y; x2[2] += b0[u].z; x2[3] += b0[u].w;
          x2[4] += b1[u].x; x2[5] += b1[u].y; x2[6] += b1[u].z; x2[7] += b1[u].w;
        }
      }
    }
    float y1[8], y2[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      y1[2 * j] = x1[2 * j] * cs[j].x - x2[2 * j] * cs[j].y;
      y2[2 * j] = x2[2 * j] * cs[j].x + x1[2 * j] * cs[j].y;
      y1[2 * j + 1] = x1[2 * j + 1] * cs[j].z - x2[2 * j + 1] * cs[j].w;
      y2[2 * j + 1] = x2[2 * j + 1] * cs[j].z + x1[2 * j + 1] * cs[j].w;
    }
    lo = make_uint4(pack_bf16(y1[0], y1[1]), pack_bf16(y1[2], y1[3]), pack_bf16(y1[4], y1[5]), pack_bf16(y1[6], y1[7]));
    hi = make_uint4(pack_bf16(y2[0], y2[1]), pack_bf16(y2[2], y2[3]), pack_bf16(y2[4], y2[5]), pack_bf16(y2[6], y2[7]));
  };
  // ---- one 16-byte chunk (8 columns) of one row, summed over the splits, bf16 (for V)
  auto plain_item = [&](int lr, int c, int col0) -> uint4 {
    float x[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) x[j] = 0.f;
    const float* pr = a.qkv_partial + ((size_t)slot * rps + lr) * nqkv + col0 + c * 8;
    for (int s0 = 0; s0 < a.qkv_splits; s0 += 4) {
      float4 a0[4], a1[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        a0[u] = a1[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (s0 + u < a.qkv_splits) {
          const float* ps = pr + (size_t)(s0 + u) * a.qkv_split_stride;
          a0[u] = *reinterpret_cast<const float4*>(ps);
          a1[u] = *reinterpret_cast<const float4*>(ps + 4);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (s0 + u < a.qkv_splits) {
          x[0] += a0[u].x; x[1] += a0[u].y; x[2] += a0[u].z; x[3] += a0[u].w;
          x[4] += a1[u].x; x[5] += a1[u].y; x[6] += a1[u].z; x[7] += a1[u].w;
        }
      }
    }
    return make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
  };
  // later 128-key steps of a long local part (block length > 32): built by the local CTA alone
  auto fill_local = [&](int pair, int buf) {
    constexpr int CPR = HALF / 8;
    const int key0 = k_begin + pair * kPairKeys;
    bf16* dK = sKV + (size_t)buf * kBufElems;
    bf16* dV = dK + kPairKeys * HD;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    for (int idx = tid; idx < kPairKeys * CPR; idx += kVerifyThreads) {
      const int row = idx / CPR, c = idx % CPR;
      uint4 lo = zero, hi = zero;
      if (key0 + row < k_end) rot_item(key0 + row, c, (a.H + kvh) * HD, lo, hi);
      *reinterpret_cast<uint4*>(dK + swz<HD>(row, c)) = lo;
      *reinterpret_cast<uint4*>(dK + swz<HD>(row, c + CPR)) = hi;
      if (commit_kv && key0 + row < k_end && key0 + row < commit_rows) {
        bf16* dst = a.cache_k_out + cache_row(key0 + row) + c * 8;
        *reinterpret_cast<uint4*>(dst) = lo;
        *reinterpret_cast<uint4*>(dst + HALF) = hi;
      }
    }
    for (int idx = tid; idx < kPairKeys * CH; idx += kVerifyThreads) {
      const int row = idx / CH, c = idx % CH;
      const uint4 v = (key0 + row < k_end) ? plain_item(key0 + row, c, (a.H + a.Hkv + kvh) * HD) : zero;
      *reinterpret_cast<uint4*>(dV + swz<HD>(row, c)) = v;
      if (commit_kv && key0 + row < k_end && key0 + row < commit_rows) *reinterpret_cast<uint4*>(a.cache_v_out + cache_row(key0 + row) + c * 8) = v;
    }
  };

  // The cache is not written by any kernel of this forward, so its first tiles may be requested
  // before the dependency wait - unless the slot -> sequence map is only known on the device.
  const bool early = a.map.n_inline > 0 || a.map.seq_map == nullptr;
  if (!local && early) load_prefix(0, 0);
  cluster_arrive();                        // every CTA of the cluster runs before shared memory is written remotely
  pdl_wait();                              // the QKV projection's partials are complete from here on
  if (!local && !early) load_prefix(0, 0);
  cp_async_commit();

  // ---- cooperative prologue: the cluster's threads share the rotary work.  The Q tile is needed by
  //      every CTA (each chunk is built once and stored into all of them), the first 128 local keys
  //      only by the CTA of the local part.  Rows past the end are zero (a masked key's V row must
  //      not hold stale shared memory: 0 * NaN would poison the output).
  {
    constexpr int CPR = HALF / 8;
    const int last = min(lr0 + kQTile - 1, rps - 1);
    const int lk_begin = (lr0 / T) * T;
    const int lk_rows = min((last / T + 1) * T - lk_begin, kPairKeys);       // valid local keys of step 0
    const int lk_fill = min(((lk_rows + kKTile - 1) / kKTile) * kKTile, kPairKeys);   // rows of the tiles in use
    const int n_q = kQTile * CPR, n_k = lk_fill * CPR, n_v = lk_fill * CH;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    bf16* lK = sKV;                          // buffer 0 of the local CTA
    bf16* lV = sKV + kPairKeys * HD;
    cluster_wait();
    for (int it = part * kVerifyThreads + tid; it < n_q + n_k + n_v; it += n_parts * kVerifyThreads) {
      if (it < n_q) {
        const int row = it / CPR, c = it % CPR;
        uint4 lo = zero, hi = zero;
        if (lr0 + row < rps) rot_item(lr0 + row, c, h * HD, lo, hi);
        for (int r = 0; r < n_parts; ++r) {
          st_cluster_u4(map_to_rank(sQ + swz<HD>(row, c), (uint32_t)r), lo);
          st_cluster_u4(map_to_rank(sQ + swz<HD>(row, c + CPR), (uint32_t)r), hi);
        }
      } else if (it < n_q + n_k) {
        const int row = (it - n_q) / CPR, c = (it - n_q) % CPR;
        uint4 lo = zero, hi = zero;
        if (row < lk_rows) rot_item(lk_begin + row, c, (a.H + kvh) * HD, lo, hi);
        st_cluster_u4(map_to_rank(lK + swz<HD>(row, c), (uint32_t)n_prefix_parts), lo);
        st_cluster_u4(map_to_rank(lK + swz<HD>(row, c + CPR), (uint32_t)n_prefix_parts), hi);
        if (commit_kv && row < lk_rows && lk_begin + row < commit_rows) {
          bf16* dst = a.cache_k_out + cache_row(lk_begin + row) + c * 8;
          *reinterpret_cast<uint4*>(dst) = lo;
          *reinterpret_cast<uint4*>(dst + HALF) = hi;
        }
      } else {
        const int row = (it - n_q - n_k) / CH, c = (it - n_q - n_k) % CH;
        const uint4 v = (row < lk_rows) ? plain_item(lk_begin + row, c, (a.H + a.Hkv + kvh) * HD) : zero;
        st_cluster_u4(map_to_rank(lV + swz<HD>(row, c), (uint32_t)n_prefix_parts), v);
        if (commit_kv && row < lk_rows && lk_begin + row < commit_rows) *reinterpret_cast<uint4*>(a.cache_v_out + cache_row(lk_begin + row) + c * 8) = v;
      }
    }
    cluster_sync_all();
  }

  float o[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};
  uint32_t qf[HD / 16][4];
  const int qrow_w = rg * 16;                          // the warp's first row inside the query tile
  // keys a query row may see in this part (no division in the inner loop): everything up to k_end for a
  // prefix part, the row's own node for the local part
  int node_lo[2], node_hi[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int qlr = lr0 + qrow_w + gq + i * 8;
    node_lo[i] = local ? (qlr / T) * T : 0;
    node_hi[i] = local ? min(node_lo[i] + T, k_end) : k_end;
    // causal chain of two blocks: a row of the finished block does not see the next block
    if (local && a.map.chain_T0 > 0 && qlr - node_lo[i] < a.map.chain_T0) node_hi[i] = min(node_hi[i], node_lo[i] + a.map.chain_T0);
  }
  const bool rows_live = lr0 + qrow_w < rps;           // otherwise the warp only keeps the barriers

  for (int pair = 0; pair < n_pairs; ++pair) {
    const int buf = pair % nbuf;
    if (pair + 1 < n_pairs) {                          // nbuf == 2 whenever a part has several steps
      if (local) fill_local(pair + 1, (pair + 1) % nbuf);
      else load_prefix(pair + 1, (pair + 1) % nbuf);
    }
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (pair == 0 && rows_live) {
#pragma unroll
      for (int kk = 0; kk < HD / 16; ++kk) {
        const int row = qrow_w + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int ch = kk * 2 + (lane >> 4);
        ldmatrix_x4(qf[kk], sQ + swz<HD>(row, ch));
      }
    }
    const int tile = 2 * pair + kset;
    if (rows_live && tile < n_tiles) {
      const bf16* tK = sKV + (size_t)buf * kBufElems + (size_t)kset * kKTile * HD;
      const bf16* tV = tK + kPairKeys * HD;
      float s[kKTile / 8][4];
#pragma unroll
      for (int j = 0; j < kKTile / 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
      // k outer, key group inner: consecutive MMAs update different accumulators
#pragma unroll
      for (int k2 = 0; k2 < HD / 32; ++k2) {
        uint32_t b[kKTile / 8][4];
#pragma unroll
        for (int j = 0; j < kKTile / 8; ++j) ldmatrix_x4(b[j], tK + swz<HD>(j * 8 + (lane & 7), k2 * 4 + (lane >> 3)));
#pragma unroll
        for (int j = 0; j < kKTile / 8; ++j) mma_bf16(s[j], qf[2 * k2], b[j][0], b[j][1]);
#pragma unroll
        for (int j = 0; j < kKTile / 8; ++j) mma_bf16(s[j], qf[2 * k2 + 1], b[j][2], b[j][3]);
      }
      // ---- scale, mask, online softmax (log2 domain)
      const int key0 = k_begin + tile * kKTile;
      float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
      for (int j = 0; j < kKTile / 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = key0 + j * 8 + 2 * tq + (e & 1);
          // local part: the key must lie in the query row's own node [node_lo, node_hi)
          const bool ok = key >= node_lo[e >> 1] && key < node_hi[e >> 1];
          const float v = ok ? s[j][e] * scale_log2 : -INFINITY;
          s[j][e] = v;
          mx[e >> 1] = fmaxf(mx[e >> 1], v);
        }
      }
      float corr[2], m_use[2];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 1));
        mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 2));
        const float m_new = fmaxf(m_run[i], mx[i]);
        m_use[i] = (m_new == -INFINITY) ? 0.f : m_new;
        corr[i] = exp2f(m_run[i] - m_use[i]);          // exp2(-inf) = 0 while nothing was seen
        m_run[i] = m_new;
        l_run[i] *= corr[i];
      }
#pragma unroll
      for (int nb = 0; nb < HD / 8; ++nb) {
        o[nb][0] *= corr[0]; o[nb][1] *= corr[0];
        o[nb][2] *= corr[1]; o[nb][3] *= corr[1];
      }
#pragma unroll
      for (int j = 0; j < kKTile / 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float p = exp2f(s[j][e] - m_use[e >> 1]);
          s[j][e] = p;
          l_run[e >> 1] += p;
        }
      }
      // ---- O += P V
#pragma unroll
      for (int jj = 0; jj < kKTile / 16; ++jj) {
        uint32_t pa[4];
        pa[0] = pack_bf16(s[2 * jj][0], s[2 * jj][1]);
        pa[1] = pack_bf16(s[2 * jj][2], s[2 * jj][3]);
        pa[2] = pack_bf16(s[2 * jj + 1][0], s[2 * jj + 1][1]);
        pa[3] = pack_bf16(s[2 * jj + 1][2], s[2 * jj + 1][3]);
#pragma unroll
        for (int n2 = 0; n2 < HD / 16; ++n2) {
          uint32_t vb[4];
          const int mtx = lane >> 3;
          const int krow = jj * 16 + (mtx & 1) * 8 + (lane & 7);
          ldmatrix_x4_trans(vb, tV + swz<HD>(krow, n2 * 2 + (mtx >> 1)));
          mma_bf16(o[2 * n2], pa, vb[0], vb[1]);
          mma_bf16(o[2 * n2 + 1], pa, vb[2], vb[3]);
        }
      }
    }
    __syncthreads();   // everyone is done with buf before it is refilled
  }
  cp_async_wait<0>();

  // ---- publish (max, sum, unnormalised output) of this warp's (rows, key set)
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    l_run[i] += __shfl_xor_sync(0xffffffffu, l_run[i], 1);
    l_run[i] += __shfl_xor_sync(0xffffffffu, l_run[i], 2);
  }
  float* sO = reinterpret_cast<float*>(sKV);            // [2 key sets][64][HD] fp32 (K/V buffers are free now)
  float2* sML = reinterpret_cast<float2*>(sQ);          // [2 key sets][64] (the Q fragments live in registers)
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int row = qrow_w + gq + i * 8;
    if (tq == 0) sML[kset * kQTile + row] = make_float2(m_run[i], l_run[i]);
    float* dst = sO + ((size_t)kset * kQTile + row) * HD + 2 * tq;
#pragma unroll
    for (int nb = 0; nb < HD / 8; ++nb) *reinterpret_cast<float2*>(dst + nb * 8) = make_float2(o[nb][2 * i], o[nb][2 * i + 1]);
  }
  __syncthreads();
  // ---- the two key sets of this CTA are merged first (set 0, then set 1), in place
  float2* sML2 = sML + 2 * kQTile;                      // [QT] merged (max, sum)
#pragma unroll
  for (int it = tid; it < kQTile * (HD / 4); it += kVerifyThreads) {   // HD / 16 iterations, independent
    const int row = it / (HD / 4), c4 = (it % (HD / 4)) * 4;
    const float2 ml0 = sML[row], ml1 = sML[kQTile + row];
    const float M = fmaxf(ml0.x, ml1.x);
    const float w0 = (ml0.x == -INFINITY) ? 0.f : exp2f(ml0.x - M);
    const float w1 = (ml1.x == -INFINITY) ? 0.f : exp2f(ml1.x - M);
    float4* p0 = reinterpret_cast<float4*>(sO + (size_t)row * HD + c4);
    const float4 v0 = *p0;
    const float4 v1 = *reinterpret_cast<const float4*>(sO + ((size_t)kQTile + row) * HD + c4);
    *p0 = make_float4(v0.x * w0 + v1.x * w1, v0.y * w0 + v1.y * w1, v0.z * w0 + v1.z * w1, v0.w * w0 + v1.w * w1);
    if (c4 == 0) sML2[row] = make_float2(M, ml0.y * w0 + ml1.y * w1);
  }
  cluster_sync_all();

  // ---- CTA `part` normalises the rows r with r % n_parts == part: all remote loads of a row are
  //      issued before the first use, the parts are merged in part order
  constexpr int TPR = HD / 8;                           // threads per row, eight columns each
  const int col = (tid % TPR) * 8;
  bool arrived = false;     // final barrier: arrive once the last remote read has landed, wait before leaving
  constexpr int kRowStepUnits = kVerifyThreads / TPR;
  for (int row = part + (tid / TPR) * n_parts; row < kQTile; row += kRowStepUnits * n_parts) {
    if (lr0 + row >= rps) break;
    const int next_row = row + kRowStepUnits * n_parts;
    const bool last_row = next_row >= kQTile || lr0 + next_row >= rps;
    float2 ml[kAttnMaxClusterParts];
    float4 va[kAttnMaxClusterParts], vb[kAttnMaxClusterParts];
#pragma unroll
    for (int pp = 0; pp < kAttnMaxClusterParts; ++pp) {
      ml[pp] = make_float2(-INFINITY, 0.f);
      va[pp] = vb[pp] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (pp < n_parts) {
        ml[pp] = ld_cluster_f32x2(map_to_rank(sML2 + row, (uint32_t)pp));
        const uint32_t base = map_to_rank(sO + (size_t)row * HD + col, (uint32_t)pp);
        va[pp] = ld_cluster_f32x4(base);
        vb[pp] = ld_cluster_f32x4(base + 16);
      }
    }
    float M = -INFINITY;
#pragma unroll
    for (int pp = 0; pp < kAttnMaxClusterParts; ++pp) M = fmaxf(M, ml[pp].x);
    float L = 0.f;
    float4 acc0 = make_float4(0.f, 0.f, 0.f, 0.f), acc1 = acc0;
#pragma unroll
    for (int pp = 0; pp < kAttnMaxClusterParts; ++pp) {
      if (ml[pp].x == -INFINITY) continue;
      const float w = exp2f(ml[pp].x - M);
      L += ml[pp].y * w;
      acc0.x += va[pp].x * w; acc0.y += va[pp].y * w; acc0.z += va[pp].z * w; acc0.w += va[pp].w * w;
      acc1.x += vb[pp].x * w; acc1.y += vb[pp].y * w; acc1.z += vb[pp].z * w; acc1.w += vb[pp].w * w;
    }
    if (last_row) { cluster_arrive_thread(); arrived = true; }
    const float inv = 1.f / L;
    *reinterpret_cast<uint4*>(a.out + ((grow0 + row) * a.H + h) * HD + col) =
        make_uint4(pack_bf16(acc0.x * inv, acc0.y * inv), pack_bf16(acc0.z * inv, acc0.w * inv),
                   pack_bf16(acc1.x * inv, acc1.y * inv), pack_bf16(acc1.z * inv, acc1.w * inv));
  }
  if (!arrived) cluster_arrive_thread();
  cluster_wait();        // nobody leaves while its shared memory may still be read
}

}  // namespace

int launch_attention_verify(cudaStream_t st, const AttnArgs& a) {
  if (a.hd != 64 && a.hd != 128) return -2;
  if (!a.qkv_partial || !a.rope || a.kv_split < kKTile || (a.kv_split % kKTile)) return -1;
  if ((a.cache_k_out != nullptr) != (a.cache_v_out != nullptr)) return -1;
  // a commit writes the K/V of one node per sequence, or of the rows before chain_T0 of the first node
  if (a.cache_k_out != nullptr && a.map.rows_per_seq != a.map.T && a.map.chain_T0 <= 0) return -1;
  const int n_prefix = (a.S + a.kv_split - 1) / a.kv_split;
  const int n_parts = n_prefix + 1;
  if (n_parts > kAttnMaxClusterParts) return -2;
  const float scale_log2 = (1.0f / sqrtf((float)a.hd)) * 1.4426950408889634f;
  // 32-row query tiles (128 threads) while that still fits the machine in one wave, else 64-row tiles
  const int tiles32 = (a.map.rows_per_seq + 31) / 32;
  const int qt_rows = ((long long)a.n_seq_slots * tiles32 * n_parts * a.H <= 3 * 148) ? 32 : 64;
  const int q_tiles = (a.map.rows_per_seq + qt_rows - 1) / qt_rows;
  // one 128-key step per part needs one K/V buffer; longer parts double-buffer
  const int nbuf = (a.kv_split > kPairKeys || a.map.T > 32) ? 2 : 1;
  const size_t smem = (size_t)(qt_rows + nbuf * 2 * kPairKeys) * a.hd * 2;
  // two CTAs per SM by default; three (register-capped build) when only that keeps the grid in one wave
  const long long n_ctas = (long long)a.n_seq_slots * q_tiles * n_parts * a.H;
  const bool dense = qt_rows == 32 && n_ctas > 2 * 148;
  static bool attr_set[kMaxDevices] = {};        // the shared-memory opt-in is per device
  const int dev = device_slot();
  if (dev < 0) return -4;
  if (!attr_set[dev]) {
    const int max_smem = (64 + 2 * 2 * kPairKeys) * 128 * 2;
    if (cudaFuncSetAttribute(attn_verify_kernel<128, 32, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess ||
        cudaFuncSetAttribute(attn_verify_kernel<128, 32, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess ||
        cudaFuncSetAttribute(attn_verify_kernel<128, 64, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess ||
        cudaFuncSetAttribute(attn_verify_kernel<64, 32, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem / 2) != cudaSuccess ||
        cudaFuncSetAttribute(attn_verify_kernel<64, 32, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem / 2) != cudaSuccess ||
        cudaFuncSetAttribute(attn_verify_kernel<64, 64, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem / 2) != cudaSuccess)
      return -4;
    attr_set[dev] = true;
  }
  dim3 grid(n_parts, a.H, a.n_seq_slots * q_tiles);
  dim3 block(qt_rows * 4);
  const unsigned cl = (unsigned)n_parts;
  cudaError_t e;
#define SSD_LAUNCH_VERIFY(HD_, QT_, MB_) \
  e = launch_pdl_cluster(attn_verify_kernel<HD_, QT_, MB_>, grid, block, smem, st, cl, a, n_prefix, nbuf, scale_log2)
  if (a.hd == 128) {
    if (qt_rows == 64) SSD_LAUNCH_VERIFY(128, 64, 1);
    else if (dense) SSD_LAUNCH_VERIFY(128, 32, 3);
    else SSD_LAUNCH_VERIFY(128, 32, 2);
  } else {
    if (qt_rows == 64) SSD_LAUNCH_VERIFY(64, 64, 1);
    else if (dense) SSD_LAUNCH_VERIFY(64, 32, 3);
    else SSD_LAUNCH_VERIFY(64, 32, 2);
  }
#undef SSD_LAUNCH_VERIFY
  return e == cudaSuccess ? 0 : -4;
}

}  // namespace ssd
