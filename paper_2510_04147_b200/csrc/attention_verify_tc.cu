// Shared-prefix bidirectional attention of the verification forward (Eq. 5) on the tcgen05 tensor
// cores: the form for head dimension 128 and key parts that are whole 128-key tiles.
//
// Same decomposition as attention_verify.cu - the key parts of one (query tile, head) form a cluster,
// one CTA per part, rotary prologue shared by the cluster's threads, parts merged through
// distributed shared memory in part order - but a CTA owns up to 128 query rows and both
// contractions run as tcgen05.mma with the accumulators in tensor memory:
//     S[row, key] = Q[row, :] . K[key, :]        (A = Q, B = K, both K-major over the head dimension)
//     O[row, :]   = P[row, :] . V[:, :]          (A = P, K-major over the keys; B = V as stored,
//                                                 [key][hd]: the MN-major operand form)
// A query row is one TMEM lane, shared by two threads (warps w and w + 4 read the same lane quadrant),
// each owning half of the lane's columns: the softmax needs no shuffles, only one exchange of the row
// maximum through shared memory, and no accumulator lives in registers, so 32, 64 or 128 rows per CTA
// cost the same 256 threads and the grid stays at parts x heads CTAs per 128 rows - one wave for the
// chains SSD runs.
//
// Shared-memory tiles are [64-column half][128 rows][64 columns] bf16 with the 128-byte swizzle the
// tensor core expects (16-byte chunk c of row r at chunk c ^ (r & 7)).  A query tile of 32 or 64
// rows is replicated to 128, so that 4 or 2 threads share a row's softmax (each takes a slice of
// the keys) and the read-out of its output row.  P overwrites the K tile once S is complete.  A part
// of several tiles runs them in order with a running (max, sum) per row; the output accumulator in
// tensor memory is rescaled in place before a later tile is added (online softmax).
#include "attn_common.cuh"

#include <cuda.h>

namespace ssd {

namespace {

using namespace attn;

constexpr int kHD = 128;
constexpr int kKeys = 128;                  // keys per MMA tile
constexpr int kTcAttnThreads = 256;       // two threads per TMEM lane (= query row copy): each takes half of the lane's columns
constexpr int kHalfBytesKV = kKeys * 128;   // one 64-column half of a 128-row tile
constexpr unsigned long long kAttnWaitLimitNs = 2000000000ull;

__device__ __forceinline__ unsigned long long gtimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// bounded: false when the limit expired
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  unsigned long long t0 = 0;
  for (uint32_t spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 255u) == 0) {
      const unsigned long long now = gtimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kAttnWaitLimitNs) return false;
    }
  }
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Operand tile with 128-byte swizzle: rows 128 B apart inside an 8-row group, groups `sbo` bytes apart
// (1024 for both forms used here); `lbo` is the distance between the two 64-element halves of the
// contiguous dimension for the MN-major form and unused for the K-major form.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;                 // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                 // 128-byte swizzle
  return d;
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// 16 consecutive columns of the thread's lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
  uint32_t r[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(v[i]);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_arrive() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
}
__device__ __forceinline__ void cluster_arrive_thread() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync_all() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release;\nbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(const void* p, uint32_t rank) {
  uint32_t out;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(smem_u32(p)), "r"(rank));
  return out;
}
__device__ __forceinline__ void st_cluster_u4(uint32_t addr, uint4 v) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
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
// byte offset of 16-byte chunk `ch` (0..15 over 128 columns) of row `row` in a [half][rows][64] tile
__device__ __forceinline__ uint32_t tile_off(int row, int ch, int rows) {
  return (uint32_t)((ch >> 3) * rows * 128 + row * 128 + (((ch & 7) ^ (row & 7)) << 4));
}

template <int QT>
__global__ void __launch_bounds__(kTcAttnThreads, 2) attn_verify_tc_kernel(AttnArgs a, int n_prefix_parts, float scale_log2) {
  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                                   // [2][128][64] bf16
  uint8_t* sK = sQ + 2 * kHalfBytesKV;                  // [2][128][64]; P overwrites it once S is complete
  uint8_t* sV = sK + 2 * kHalfBytesKV;                  // [2][128][64]
  float* sMax = reinterpret_cast<float*>(sV + 2 * kHalfBytesKV);         // [2 halves x 4 copies][128 rows]
  float* sSum = sMax + 8 * 128;                                          // [8 chunks of 16 keys][128 rows]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sSum + 8 * 128);          // [0] S ready, [1] O ready
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
  constexpr int HALF = kHD / 2, CPR = HALF / 8, CH = kHD / 8;

  pdl_launch_dependents();
  const int tid = threadIdx.x, warp = tid >> 5;
  const int n_parts = n_prefix_parts + 1;
  const int part = blockIdx.x, h = blockIdx.y;          // the cluster spans x
  const int q_tiles = (a.map.rows_per_seq + QT - 1) / QT;
  const int qt = blockIdx.z % q_tiles, slot = blockIdx.z / q_tiles;
  const int kvh = h / (a.H / a.Hkv);
  const int rps = a.map.rows_per_seq, T = a.map.T;
  const int lr0 = qt * QT;
  const size_t grow0 = (size_t)slot * rps + lr0;
  const bool local = part == n_prefix_parts;
  const int nqkv = (a.H + 2 * a.Hkv) * kHD;

  int k_begin, k_end;
  if (!local) {
    k_begin = part * a.kv_split;                        // a multiple of 128 keys per part
    k_end = min(a.S, k_begin + a.kv_split);
  } else {
    const int last = min(lr0 + QT - 1, rps - 1);
    k_begin = (lr0 / T) * T;
    k_end = (last / T + 1) * T;                         // the launcher guarantees k_end - k_begin <= 128
  }
  const int n_tiles = (k_end - k_begin + kKeys - 1) / kKeys;

  if (tid == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }

  // ---- prefix K/V straight from the cache (zero rows past the end of the part)
  auto load_prefix = [&](int tile, bool want_k = true, bool want_v = true) {
    const int seq = seq_of_slot(a.map, slot);
    const int kb = k_begin + tile * kKeys;
    const bf16* kbase = a.cache_k + (size_t)seq * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride;
    const bf16* vbase = a.cache_v + (size_t)seq * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride;
    const size_t krow_stride = a.kv_pos_stride;
    for (int idx = tid; idx < kKeys * CH; idx += kTcAttnThreads) {
      const int row = idx / CH, ch = idx % CH;
      const int key = kb + row;
      const bool valid = key < k_end;
      int crow = valid ? key : kb;                            // cache row of the key (a hole skips the block's own rows)
      if (crow >= a.hole_begin) crow += a.hole_len;
      const size_t off = (size_t)crow * krow_stride + ch * 8;
      if (want_k) cp_async16(sK + tile_off(row, ch, kKeys), kbase + off, valid);
      if (want_v) cp_async16(sV + tile_off(row, ch, kKeys), vbase + off, valid);
    }
  };
  const bool commit_kv = a.cache_k_out != nullptr && (h % (a.H / a.Hkv)) == 0;
  const int commit_rows = a.map.chain_T0 > 0 ? a.map.chain_T0 : rps;   // sequence-local rows whose K/V are cached
  auto cache_row = [&](int lr) -> size_t {
    return (size_t)seq_of_slot(a.map, slot) * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride + (size_t)(a.map.pos0 + lr) * a.kv_pos_stride;
  };
  // The cache is not written by any kernel of this forward, so its tiles may be requested before the
  // dependency wait - unless the slot -> sequence map is only known on the device.
  const bool early = a.map.n_inline > 0 || a.map.seq_map == nullptr;
  if (!local && early) load_prefix(0);
  cluster_arrive();                        // every CTA of the cluster runs before shared memory is written remotely
  pdl_wait();                              // the QKV projection's partials are complete from here on
  if (!local && !early) load_prefix(0);
  cp_async_commit();

  // ---- cooperative prologue: the cluster's threads share the rotary work.  Each chunk of the Q tile
  //      is built once and stored into every CTA; the local part's K (rotated) and V go to its CTA.
  //      Rows past the end are zero (a masked key's V row must be finite: 0 * NaN would poison O).
  {
    const int last = min(lr0 + QT - 1, rps - 1);
    const int lk_begin = (lr0 / T) * T;
    const int lk_rows = min((last / T + 1) * T - lk_begin, kKeys);
    const int n_q = QT * CPR, n_k = lk_rows * CPR, n_v = lk_rows * CH;    // shared work: valid rows only
    const uint4 zero = make_uint4(0, 0, 0, 0);
    if (local) {
      // rows of the 128-key tile past the local keys: zero, written by their own CTA
      for (int idx = lk_rows * CH + tid; idx < kKeys * CH; idx += kTcAttnThreads) {
        const int row = idx / CH, ch = idx % CH;
        *reinterpret_cast<uint4*>(sK + tile_off(row, ch, kKeys)) = zero;
        *reinterpret_cast<uint4*>(sV + tile_off(row, ch, kKeys)) = zero;
      }
    }
    // A work item = one 16-byte chunk of a row (with its rotation partner for Q and K).  All split-K
    // partials of an item are requested before the first is used, so their L2 round trips overlap.
    struct Item { int kind, row, c; const float* pr; const float4* cs4; };   // kind 0 Q, 1 K, 2 V, -1 none
    auto decode = [&](int it) -> Item {
      Item w{-1, 0, 0, nullptr, nullptr};
      if (it >= n_q + n_k + n_v) return w;
      int lr, col0;
      if (it < n_q) {
        w.kind = 0; w.row = it / CPR; w.c = it % CPR;
        lr = lr0 + w.row; col0 = h * kHD;
        if (lr >= rps) return w;                         // rows past the end of the sequence stay zero
      } else if (it < n_q + n_k) {
        w.kind = 1; w.row = (it - n_q) / CPR; w.c = (it - n_q) % CPR;
        lr = lk_begin + w.row; col0 = (a.H + kvh) * kHD;
      } else {
        w.kind = 2; w.row = (it - n_q - n_k) / CH; w.c = (it - n_q - n_k) % CH;
        lr = lk_begin + w.row; col0 = (a.H + a.Hkv + kvh) * kHD;
      }
      w.pr = a.qkv_partial + ((size_t)slot * rps + lr) * nqkv + col0 + w.c * 8;
      if (w.kind != 2) w.cs4 = reinterpret_cast<const float4*>(a.rope + (size_t)(a.map.pos0 + lr % T) * HALF + w.c * 8);
      return w;
    };
    // sums over the splits in split order: x1 = the chunk itself, x2 = its rotation partner (rotary items)
    auto gather = [&](const Item& A, float (&x1)[8], float (&x2)[8]) {
#pragma unroll
      for (int j = 0; j < 8; ++j) { x1[j] = x2[j] = 0.f; }
      const bool la = A.pr != nullptr;
      const bool ra = la && A.kind != 2;
      for (int s0 = 0; s0 < a.qkv_splits; s0 += 4) {
        float4 a0[4], a1[4], a2[4], a3[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          a0[u] = a1[u] = a2[u] = a3[u] = make_float4(0.f, 0.f, 0.f, 0.f);
          const bool on = s0 + u < a.qkv_splits;
          const size_t off = (size_t)(s0 + u) * a.qkv_split_stride;
          if (on && la) { a0[u] = *reinterpret_cast<const float4*>(A.pr + off); a1[u] = *reinterpret_cast<const float4*>(A.pr + off + 4); }
          if (on && ra) { a2[u] = *reinterpret_cast<const float4*>(A.pr + off + HALF); a3[u] = *reinterpret_cast<const float4*>(A.pr + off + HALF + 4); }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (s0 + u < a.qkv_splits) {
            x1[0] += a0[u].x; x1[1] += a0[u].y; x1[2] += a0[u].z; x1[3] += a0[u].w;
            x1[4] += a1[u].x; x1[5] += a1[u].y; x1[6] += a1[u].z; x1[7] += a1[u].w;
            x2[0] += a2[u].x; x2[1] += a2[u].y; x2[2] += a2[u].z; x2[3] += a2[u].w;
            x2[4] += a3[u].x; x2[5] += a3[u].y; x2[6] += a3[u].z; x2[7] += a3[u].w;
          }
        }
      }
    };
    // rotary embedding (Q, K) or plain rounding (V), then the stores of the item
    auto finish = [&](const Item& w, const float (&x1)[8], const float (&x2)[8]) {
      if (w.kind < 0) return;
      uint4 lo = zero, hi = zero;
      if (w.pr != nullptr) {
        if (w.kind == 2) {
          lo = make_uint4(pack_bf16(x1[0], x1[1]), pack_bf16(x1[2], x1[3]), pack_bf16(x1[4], x1[5]), pack_bf16(x1[6], x1[7]));
        } else {
          float4 cs[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) cs[j] = w.cs4[j];
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
        }
      }
      if (w.kind == 0) {
        for (int r = 0; r < n_parts; ++r) {
          st_cluster_u4(map_to_rank(sQ + tile_off(w.row, w.c, 128), (uint32_t)r), lo);
          st_cluster_u4(map_to_rank(sQ + tile_off(w.row, w.c + 8, 128), (uint32_t)r), hi);
        }
      } else if (w.kind == 1) {
        st_cluster_u4(map_to_rank(sK + tile_off(w.row, w.c, kKeys), (uint32_t)n_prefix_parts), lo);
        st_cluster_u4(map_to_rank(sK + tile_off(w.row, w.c + 8, kKeys), (uint32_t)n_prefix_parts), hi);
        if (commit_kv && lk_begin + w.row < commit_rows) {
          bf16* dst = a.cache_k_out + cache_row(lk_begin + w.row) + w.c * 8;
          *reinterpret_cast<uint4*>(dst) = lo;
          *reinterpret_cast<uint4*>(dst + HALF) = hi;
        }
      } else {
        st_cluster_u4(map_to_rank(sV + tile_off(w.row, w.c, kKeys), (uint32_t)n_prefix_parts), lo);
        if (commit_kv && lk_begin + w.row < commit_rows) *reinterpret_cast<uint4*>(a.cache_v_out + cache_row(lk_begin + w.row) + w.c * 8) = lo;
      }
    };
    const int stride = n_parts * kTcAttnThreads;
    bool waited = false;
    for (int it = part * kTcAttnThreads + tid; it < n_q + n_k + n_v; it += stride) {
      const Item A = decode(it);
      float x1[8], x2[8];
      gather(A, x1, x2);
      if (!waited) { cluster_wait(); waited = true; }      // remote stores only once every CTA of the cluster runs
      finish(A, x1, x2);
    }
    if (!waited) cluster_wait();
    asm volatile("fence.proxy.async.shared::cluster;" ::: "memory");  // these stores (into other CTAs too) are read by the tensor core
    cluster_sync_all();
  }
  // The MMA always works on 128 query rows (= 128 TMEM lanes, one per thread).  A tile of QT < 128
  // rows is replicated REP = 128 / QT times, so that REP threads share the softmax of a row: copy w
  // (lanes w * QT ..) takes the keys [w * QT, (w + 1) * QT) of the part.
  constexpr int REP = 128 / QT;
  if (REP > 1) {
    for (int idx = tid; idx < QT * CH * (REP - 1); idx += kTcAttnThreads) {
      const int k = idx / (QT * CH) + 1, rem = idx % (QT * CH);
      const int r = rem / CH, ch = rem % CH;
      *reinterpret_cast<uint4*>(sQ + tile_off(k * QT + r, ch, 128)) = *reinterpret_cast<const uint4*>(sQ + tile_off(r, ch, 128));
    }
  }
  cp_async_wait<0>();
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_S = tmem_base, tmem_O = tmem_base + 128;
  // f32 accumulate, bf16 operands, N = 128, M = 128; bit 16: B is MN-major (V as stored, [key][hd])
  const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

  // ---- softmax, log2 domain.  TMEM lane lt = copy `cw` of query row `row`; a copy covers the keys
  //      [cw * QT, +QT) of a tile and the lane's two threads (hw = 0, 1) half of those each, in 16-key
  //      chunks.  The row maximum is exchanged through shared memory; a tile's row sum is ALWAYS formed
  //      from its eight 16-key chunks as (((c0 + c1) + (c2 + c3)) + (c4 + c5)) + (c6 + c7), each chunk
  //      summed in key order, whatever QT is - a row's bits do not depend on how many rows share the forward.
  constexpr int KPT = QT / 2;                           // keys of a tile per thread
  constexpr int NCH = KPT / 16;                         // 16-key chunks per thread
  const int lt = tid & 127, hw = tid >> 7;
  const int cw = lt / QT, row = lt % QT;
  const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;   // warps w and w + 4 read TMEM lanes 32 (w & 3) ...
  const int col0 = cw * QT + hw * KPT;                  // first column (key of a tile) of this thread
  const int lr = lr0 + row;
  const bool row_live = lr < rps;
  int key_lo = k_begin, key_hi = k_end;                 // keys this row may see in this part
  if (local) {
    key_lo = (lr / T) * T;
    key_hi = min(key_lo + T, k_end);
    // causal chain of two blocks: a row of the finished block does not see the next block
    if (a.map.chain_T0 > 0 && lr - key_lo < a.map.chain_T0) key_hi = min(key_hi, key_lo + a.map.chain_T0);
  }
  float m_row = -INFINITY, l_row = 0.f;                 // running maximum and sum over the tiles so far
  bool ok = true;
#pragma unroll 1
  for (int t = 0; t < n_tiles; ++t) {
    const int kb = k_begin + t * kKeys;                 // first key of the tile
    const uint32_t phase = (uint32_t)(t & 1);
    if (t > 0) {
      // the previous tile's MMAs are complete: K (holding P) and V are free
      // (K and V as two groups: S = Q K^T starts when K has landed, V may take until P is ready)
      load_prefix(t, true, false);
      cp_async_commit();
      load_prefix(t, false, true);
      cp_async_commit();
      cp_async_wait<1>();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      __syncthreads();
      tc_fence_after();
    }
    if (tid == 0) {
      // ---- S = Q . K^T: eight k16 steps over the head dimension (four per 64-column half)
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint32_t qa = smem_u32(sQ) + (uint32_t)((k >> 2) * kHalfBytesKV + (k & 3) * 32);
        const uint32_t ka = smem_u32(sK) + (uint32_t)((k >> 2) * kHalfBytesKV + (k & 3) * 32);
        tc_mma_bf16(tmem_S, make_desc(qa, 16, 1024), make_desc(ka, 16, 1024), idesc, (uint32_t)(k != 0));
      }
      tc_commit(smem_u32(&bars[0]));
    }
    ok = mbar_wait(smem_u32(&bars[0]), phase);
    tc_fence_after();
    ok = __syncthreads_and(ok ? 1 : 0) != 0;              // one decision for the CTA (barriers follow)
    if (!ok) break;

    float m_loc = -INFINITY;
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
      const int c0 = col0 + ch * 16;
      float v[16];
      tmem_ld16(tmem_S + lane_addr + c0, v);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int key = kb + c0 + j;
        if (key >= key_lo && key < key_hi) m_loc = fmaxf(m_loc, v[j] * scale_log2);
      }
    }
    sMax[(hw * 4 + cw) * 128 + row] = m_loc;
    __syncthreads();
    float m_tile = -INFINITY;
#pragma unroll
    for (int k = 0; k < REP; ++k) m_tile = fmaxf(m_tile, fmaxf(sMax[k * 128 + row], sMax[(4 + k) * 128 + row]));
    const float m_new = fmaxf(m_row, m_tile);
    const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
    const float corr = exp2f(m_row - m_use);              // 0 for the first tile that holds a visible key
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
      const int c0 = col0 + ch * 16;
      float v[16];
      tmem_ld16(tmem_S + lane_addr + c0, v);
      uint32_t packed[8];
      float csum = 0.f;
#pragma unroll
      for (int j = 0; j < 16; j += 2) {
        const int key = kb + c0 + j;
        const float p0 = (key >= key_lo && key < key_hi) ? exp2f(v[j] * scale_log2 - m_use) : 0.f;
        const float p1 = (key + 1 >= key_lo && key + 1 < key_hi) ? exp2f(v[j + 1] * scale_log2 - m_use) : 0.f;
        csum += p0;
        csum += p1;
        packed[j >> 1] = pack_bf16(p0, p1);
      }
      sSum[(c0 >> 4) * 128 + row] = csum;               // chunk index = c0 / 16
      // P overwrites K, in every copy of the row
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const uint4 val = row_live ? make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3])
                                   : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int k = 0; k < REP; ++k)
          *reinterpret_cast<uint4*>(sK + tile_off(k * QT + row, (c0 >> 3) + q, 128)) = val;
      }
    }
    if (t > 0) {
      // the output so far was accumulated against the old maximum: rescale this thread's columns of its
      // lane (the columns it reads out at the end; the rest of a copy's lane is never read)
#pragma unroll
      for (int ch = 0; ch < NCH; ++ch) {
        float v[16];
        const uint32_t ta = tmem_O + lane_addr + col0 + ch * 16;
        tmem_ld16(ta, v);
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] *= corr;
        tmem_st16(ta, v);
      }
    }
    cp_async_wait<0>();                                   // V of a later tile
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // P (and V) are read by the tensor core
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      // ---- O (+)= P . V: eight k16 steps over the keys.  P is K-major (keys contiguous); V is used as
      //      stored, [key][hd] = MN-major: 8-key groups 1024 B apart, the two 64-column halves 16 KB apart.
      const uint32_t idesc_pv = idesc | (1u << 16);
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint32_t pa = smem_u32(sK) + (uint32_t)((k >> 2) * kHalfBytesKV + (k & 3) * 32);
        const uint32_t va = smem_u32(sV) + (uint32_t)(2 * k * 1024);
        tc_mma_bf16(tmem_O, make_desc(pa, 16, 1024), make_desc(va, kHalfBytesKV, 1024), idesc_pv, (uint32_t)((t | k) != 0));
      }
      tc_commit(smem_u32(&bars[1]));
    }
    ok = mbar_wait(smem_u32(&bars[1]), phase);
    tc_fence_after();
    ok = __syncthreads_and(ok ? 1 : 0) != 0;              // every MMA is complete: shared memory is free
    if (!ok) break;
    const float l_tile = (((sSum[0 * 128 + row] + sSum[1 * 128 + row]) + (sSum[2 * 128 + row] + sSum[3 * 128 + row])) +
                          (sSum[4 * 128 + row] + sSum[5 * 128 + row])) + (sSum[6 * 128 + row] + sSum[7 * 128 + row]);
    l_row = l_row * corr + l_tile;
    m_row = m_new;
  }

  // ---- publish (max, sum, unnormalised output) of the rows
  constexpr int kPitch = kHD + 4;                         // floats per staged row
  float* sO = reinterpret_cast<float*>(smem);             // [QT][kPitch]
  float2* sML = reinterpret_cast<float2*>(sO + QT * kPitch);
  if (ok) {
    // every copy of a row holds the same O row: a thread stages the columns it owns, [col0, +KPT)
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
      float v[16];
      tmem_ld16(tmem_O + lane_addr + col0 + ch * 16, v);
#pragma unroll
      for (int j = 0; j < 16; j += 4)
        *reinterpret_cast<float4*>(sO + row * kPitch + col0 + ch * 16 + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
    }
    if (cw == 0 && hw == 0) sML[row] = row_live ? make_float2(m_row, l_row) : make_float2(-INFINITY, 0.f);
  } else if (tid == 0) {
    atomicExch(a.err_flag, 4);
  }
  tc_fence_before();
  cluster_sync_all();

  // ---- CTA `part` normalises the rows r with r % n_parts == part: all remote loads of a row are
  //      issued before the first use, the parts are merged in part order
  constexpr int TPR = kHD / 8;                            // threads per row, eight columns each
  constexpr int kRowStep = kTcAttnThreads / TPR;
  const int col = (tid % TPR) * 8;
  bool arrived = false;
  for (int r = part + (tid / TPR) * n_parts; r < QT; r += kRowStep * n_parts) {
    if (lr0 + r >= rps) break;
    const int next_r = r + kRowStep * n_parts;
    const bool last_r = next_r >= QT || lr0 + next_r >= rps;
    float2 ml[kAttnMaxClusterParts];
    float4 va[kAttnMaxClusterParts], vb[kAttnMaxClusterParts];
#pragma unroll
    for (int pp = 0; pp < kAttnMaxClusterParts; ++pp) {
      ml[pp] = make_float2(-INFINITY, 0.f);
      va[pp] = vb[pp] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (pp < n_parts) {
        ml[pp] = ld_cluster_f32x2(map_to_rank(sML + r, (uint32_t)pp));
        const uint32_t base = map_to_rank(sO + (size_t)r * kPitch + col, (uint32_t)pp);
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
    if (last_r) { cluster_arrive_thread(); arrived = true; }
    const float inv = 1.f / L;
    *reinterpret_cast<uint4*>(a.out + ((grow0 + r) * a.H + h) * kHD + col) =
        make_uint4(pack_bf16(acc0.x * inv, acc0.y * inv), pack_bf16(acc0.z * inv, acc0.w * inv),
                   pack_bf16(acc1.x * inv, acc1.y * inv), pack_bf16(acc1.z * inv, acc1.w * inv));
  }
  if (!arrived) cluster_arrive_thread();
  __syncwarp();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  }
  cluster_wait();        // nobody leaves while its shared memory may still be read
}

}  // namespace

int launch_attention_verify_tc(cudaStream_t st, const AttnArgs& a) {
  if (a.hd != kHD || !a.qkv_partial || !a.rope || !a.err_flag) return 1;
  if (a.kv_split < kKeys || (a.kv_split % kKeys) != 0) return 1;
  if ((a.cache_k_out != nullptr) != (a.cache_v_out != nullptr)) return -1;
  const int rps = a.map.rows_per_seq, T = a.map.T;
  // a commit writes the K/V of one node per sequence, or of the rows before chain_T0 of the first node
  if (a.cache_k_out != nullptr && rps != T && a.map.chain_T0 <= 0) return -1;
  const int n_prefix = (a.S + a.kv_split - 1) / a.kv_split;
  const int n_parts = n_prefix + 1;
  if (n_parts > kAttnMaxClusterParts) return 1;
  // Eligibility depends on the head dimension, the prefix length and the block length only - never on
  // the number of rows - so that a node meets the same arithmetic alone and among other nodes.
  // Blocks that divide 128 keep every query tile's node-local keys inside one 128-key tile.
  if (T < 1 || (kKeys % T) != 0) return 1;
  const int qt_rows = rps <= 32 ? 32 : (rps <= 64 ? 64 : 128);
  const int q_tiles = (rps + qt_rows - 1) / qt_rows;
  const float scale_log2 = (1.0f / sqrtf((float)a.hd)) * 1.4426950408889634f;
  // 101 KB: never more than two CTAs per SM, so that two 256-column TMEM allocations always fit
  const size_t smem = 6 * (size_t)kHalfBytesKV + 8192 + 64 + 1024;   // Q, K/P, V tiles of 128 rows + the softmax exchange
  static bool attr_set[kMaxDevices] = {};        // the shared-memory opt-in is per device
  const int dev = device_slot();
  if (dev < 0) return -4;
  if (!attr_set[dev]) {
    const int max_smem = 6 * kHalfBytesKV + 8192 + 64 + 1024;
    if (cudaFuncSetAttribute(attn_verify_tc_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess ||
        cudaFuncSetAttribute(attn_verify_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess ||
        cudaFuncSetAttribute(attn_verify_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess)
      return -4;
    attr_set[dev] = true;
  }
  dim3 grid(n_parts, a.H, a.n_seq_slots * q_tiles);
  dim3 block(kTcAttnThreads);
  cudaError_t e;
  if (qt_rows == 32)
    e = launch_pdl_cluster(attn_verify_tc_kernel<32>, grid, block, smem, st, (unsigned)n_parts, a, n_prefix, scale_log2);
  else if (qt_rows == 64)
    e = launch_pdl_cluster(attn_verify_tc_kernel<64>, grid, block, smem, st, (unsigned)n_parts, a, n_prefix, scale_log2);
  else
    e = launch_pdl_cluster(attn_verify_tc_kernel<128>, grid, block, smem, st, (unsigned)n_parts, a, n_prefix, scale_log2);
  return e == cudaSuccess ? 0 : -4;
}

}  // namespace ssd
