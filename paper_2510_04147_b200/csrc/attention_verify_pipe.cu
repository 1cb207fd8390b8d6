// Shared-prefix bidirectional attention of the verification forward (Eq. 5) on the tcgen05 tensor cores for
// BATCHES: one CTA per (query tile, head, sequence) walks all key tiles of the head in one software pipeline.  It
// wins once there are about as many such CTAs as SMs; one sequence takes the cluster form, which runs the key parts
// of a head side by side.
//
// A query tile is up to 128 rows of one sequence (nodes side by side); its keys are the node-local keys (tile
// 0, visibility per row: the row's own node, block-causal inside a chain of two blocks) followed by the cached
// keys in 128-key tiles.  The prologue builds the query tile and the node-local K/V from the fp32 split-K
// partials of the fused q|k|v projection (summed in split order, rotary embedding, bf16) and writes the cache
// rows of a commit.  Every cached K/V tile is read once per (query tile, head) and serves all nodes.
//
// Pipeline (two K stages, one P tile and two V stages in shared memory, two S accumulators and one O accumulator
// in tensor memory): while the threads run the softmax of tile u - row maximum, running (max, sum), P written to
// its tile - the tensor core already computes S = Q K^T of tile u+1.  K of tile u+2 is requested as soon as S of
// tile u is complete (its stage is free then), V of tile u+1 as soon as O += P V of tile u-1 is: both a whole
// iteration before they are needed.  O += P V of tile u is issued when P is complete and finishes under the next
// tile's
// softmax.  O is rescaled in tensor memory when a row's maximum grows.  A query row is one TMEM lane shared by
// two threads (warps w and w+4), each owning half of the lane's columns; a tile of 32 or 64 rows is replicated
// to 128 lanes so that more threads share a row.  The order of the tiles and of every sum is fixed by the shapes
// alone, so a row's bits do not depend on what shares the forward with it.
#include "attn_common.cuh"

#include <cuda.h>
#include <string.h>

namespace ssd {

namespace {

using namespace attn;

constexpr int kHD = 128;
constexpr int kKeys = 128;                  // keys per tile
constexpr int kPipeThreads = 256;           // softmax threads: two per TMEM lane
constexpr int kPipeBlock = kPipeThreads + 64;   // + one warp that issues the MMAs + one that asks for the bulk tile copies
constexpr int kHalfBytes = kKeys * 128;     // one 64-column half of a 128-row tile
constexpr int kTileBytes = 2 * kHalfBytes;  // a [128][128] bf16 tile
constexpr int kStagesK = 2, kStagesV = 2;      // + one P tile
constexpr unsigned long long kPipeWaitLimitNs = 2000000000ull;

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
// bounded: false when the limit expired or another thread of the CTA gave up (`abort` set)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort) {
  unsigned long long t0 = 0;
  for (uint32_t spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 255u) == 0) {
      if (*abort) return false;
      const unsigned long long now = gtimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kPipeWaitLimitNs) { *abort = 1; return false; }
    }
  }
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// one box of a 2-D tensor map into shared memory; its bytes count on the mbarrier
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"((unsigned long long)map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// barrier 1 of the softmax threads (the MMA warp does not take part); returns the AND of `v` over them
__device__ __forceinline__ bool softmax_barrier_and(bool v) {
  uint32_t r;
  asm volatile(
      "{\n.reg .pred p, q;\n"
      "setp.ne.b32 q, %1, 0;\n"
      "bar.red.and.pred p, 1, 256, q;\n"
      "selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(r) : "r"((uint32_t)(v ? 1 : 0)) : "memory");
  return r != 0;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Operand tile with 128-byte swizzle: rows 128 B apart inside an 8-row group, groups `sbo` bytes apart;
// `lbo` is the distance between the two 64-element halves of the contiguous dimension for the MN-major form.
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
// 16 consecutive columns of the thread's lane, requested only: several requests share one wait, and no register of
// a request may be read before tmem_ld_wait() and keep16() on it
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// (keeps the compiler from reading the registers of a request above the wait)
__device__ __forceinline__ void keep16(uint32_t* r) {
  asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                    "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]));
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
// 2^x on the special-function unit (the one form used everywhere in this kernel, so that a key's probability has the
// same bits on every code path)
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// byte offset of 16-byte chunk `ch` (0..15 over 128 columns) of row `row` in a [half][128 rows][64] tile
__device__ __forceinline__ uint32_t tile_off(int row, int ch) {
  return (uint32_t)((ch >> 3) * kHalfBytes + row * 128 + (((ch & 7) ^ (row & 7)) << 4));
}

template <int QT>
__global__ void __launch_bounds__(kPipeBlock, 1) attn_verify_pipe_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                               const __grid_constant__ CUtensorMap tmV, AttnArgs a,
                                                                               float scale_log2, int use_tma) {
  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                                   // [2][128][64] bf16
  uint8_t* sKs = sQ + kTileBytes;                       // kStagesK K tiles: a stage is free as soon as its S = Q K^T is complete
  uint8_t* sP = sKs + kStagesK * kTileBytes;            // P of the tile in work (bf16, the A operand of O += P V)
  uint8_t* sVs = sP + kTileBytes;                       // kStagesV V tiles
  float* sMax = reinterpret_cast<float*>(sVs + kStagesV * kTileBytes);      // 2 x [2 halves x 4 copies][128 rows] (tiles alternate)
  float* sSum = sMax + 2 * 8 * 128;                                         // 2 x [8 chunks of 16 keys][128 rows]
  // [0], [1] S ready (two accumulators), [2] O += P V complete, [3], [4] K stage landed, [5] P written and V landed
  uint64_t* bars = reinterpret_cast<uint64_t*>(sSum + 2 * 8 * 128);
  // ... [6], [7] V stage landed (bulk copies only)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  constexpr int CH = kHD / 8;                            // 16-byte chunks per row

  pdl_launch_dependents();
  const int tid = threadIdx.x, warp = tid >> 5;
  const int h = blockIdx.x;
  const int rps = a.map.rows_per_seq, T = a.map.T;
  const int q_tiles = (rps + QT - 1) / QT;
  const int qt = blockIdx.y % q_tiles, slot = blockIdx.y / q_tiles;
  const int kvh = h / (a.H / a.Hkv);
  const int lr0 = qt * QT;
  const size_t grow0 = (size_t)slot * rps + lr0;
  const int nqkv = (a.H + 2 * a.Hkv) * kHD;
  // node-local keys of this query tile: the rows of the nodes it touches (the launcher keeps them within one tile)
  const int last_row = min(lr0 + QT - 1, rps - 1);
  const int lk_begin = (lr0 / T) * T;
  const int lk_rows = min((last_row / T + 1) * T - lk_begin, kKeys);
  const int n_cached_tiles = (a.S + kKeys - 1) / kKeys;
  const int n_tiles = 1 + n_cached_tiles;               // tile 0: node-local keys; tile u >= 1: cached keys [(u-1) * 128, ...)

  if (tid == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    mbar_init(smem_u32(&bars[2]), 1);
    mbar_init(smem_u32(&bars[3]), kPipeThreads + 1);        // every softmax thread (it has read S of the tile whose accumulator
    mbar_init(smem_u32(&bars[4]), kPipeThreads + 1);        // is reused; its own copies have landed) + the copy thread
    mbar_init(smem_u32(&bars[5]), kPipeThreads);
    mbar_init(smem_u32(&bars[6]), 1);
    mbar_init(smem_u32(&bars[7]), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  __syncthreads();                          // the barriers exist before the copy thread uses them

  // ---- copies into a stage: cached K/V (zero rows past the end), or the node-local rows of the projection
  // A thread copies the same 16-byte column chunk of the rows ld_row0, ld_row0 + 16, ...: the swizzle term of its
  // shared-memory address and its byte offset inside a cache row are constants, so a copy costs a few instructions.
  const bool softmax_thread = tid < kPipeThreads;        // warps 0-7; warp 8 issues the MMAs, warp 9 asks for the bulk copies
  // Whole tiles of cached keys are copied by the tensor-map engine (one thread asks, the bytes count on an mbarrier);
  // a last, partial tile is copied by the softmax threads, which fill the rows past the end with zeros.
  auto bulk = [&](int u) { return use_tma != 0 && u >= 1 && u * kKeys <= a.S; };
  const int ld_ch = tid % CH, ld_row0 = tid / CH;
  const uint32_t ld_soff = tile_off(ld_row0, ld_ch);      // + 16 * 128 bytes per step (16 rows: the same swizzle phase)
  auto load_cached = [&](int u, bool want_k, bool want_v) {
    const uint32_t dK = smem_u32(sKs + (size_t)(u % kStagesK) * kTileBytes) + ld_soff;
    const uint32_t dV = smem_u32(sVs + (size_t)(u % kStagesV) * kTileBytes) + ld_soff;
    const int seq = seq_of_slot(a.map, slot);
    const int kb = (u - 1) * kKeys;
    const size_t base = (size_t)seq * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride + ld_ch * 8;
    const bf16* kbase = a.cache_k + base;
    const bf16* vbase = a.cache_v + base;
    if (kb + kKeys <= a.S && (a.hole_len == 0 || kb + kKeys <= a.hole_begin)) {
      // a whole tile of consecutive cache rows: 16 rows further per step
      const size_t off0 = (size_t)(kb + ld_row0) * a.kv_pos_stride, step = (size_t)(kPipeThreads / CH) * a.kv_pos_stride;
#pragma unroll
      for (int it = 0; it < kKeys * CH / kPipeThreads; ++it) {
        const uint32_t so = (uint32_t)it * (kPipeThreads / CH) * 128u;
        if (want_k) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dK + so), "l"(kbase + off0 + it * step));
        if (want_v) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dV + so), "l"(vbase + off0 + it * step));
      }
      return;
    }
#pragma unroll
    for (int it = 0; it < kKeys * CH / kPipeThreads; ++it) {
      const int key = kb + ld_row0 + it * (kPipeThreads / CH);
      const bool valid = key < a.S;
      int crow = valid ? key : kb;                            // cache row of the key (a hole skips the block's own rows)
      if (crow >= a.hole_begin) crow += a.hole_len;
      const size_t off = (size_t)crow * a.kv_pos_stride;
      const int sz = valid ? 16 : 0;                          // 0: the chunk is filled with zeros
      const uint32_t so = (uint32_t)it * (kPipeThreads / CH) * 128u;
      if (want_k) asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dK + so), "l"(kbase + off), "r"(sz));
      if (want_v) asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dV + so), "l"(vbase + off), "r"(sz));
    }
  };
  const bool commit_kv = a.cache_k_out != nullptr && (h % (a.H / a.Hkv)) == 0;
  const int commit_rows = a.map.chain_T0 > 0 ? a.map.chain_T0 : rps;   // sequence-local rows whose K/V are cached
  // The cache is not written below the rows' own positions by any kernel of this forward, so its first tile may be
  // requested before the dependency wait - unless the slot -> sequence map is only known on the device.
  const bool early = a.map.n_inline > 0 || a.map.seq_map == nullptr;
  if (softmax_thread && early && n_tiles > 1 && !bulk(1)) load_cached(1, true, false);
  auto ask_tile1 = [&]() {                 // copy warp, lanes 0 (K) and 1 (V): both stages 1 are free from the start
    const int lane = tid & 31;
    if (warp != kPipeThreads / 32 + 1 || lane >= 2 || n_tiles < 2) return;
    const uint32_t kb_ = smem_u32(&bars[3]) + 8u, vb_ = smem_u32(&bars[6]) + 8u;
    if (!bulk(1)) { if (lane == 0) mbar_arrive(kb_); return; }
    const int seq = seq_of_slot(a.map, slot);
    const int r0 = (int)(((size_t)seq * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride) / kHD);
    const uint32_t dst = smem_u32((lane == 0 ? sKs : sVs) + kTileBytes);
    const uint32_t bar = lane == 0 ? kb_ : vb_;
    mbar_arrive_expect_tx(bar, (uint32_t)kTileBytes);
    tma_load_2d(dst, lane == 0 ? &tmK : &tmV, bar, 0, r0);
    tma_load_2d(dst + kHalfBytes, lane == 0 ? &tmK : &tmV, bar, 64, r0);
  };
  if (early) ask_tile1();
  pdl_wait();                              // the QKV projection's partials are complete from here on
  if (!early) ask_tile1();
  if (softmax_thread && !early && n_tiles > 1 && !bulk(1)) load_cached(1, true, false);
  cp_async_commit();

  // ---- prologue: the query tile and the node-local K/V from the fp32 split-K partials of the fused q|k|v
  //      projection.  A work item = one 16-byte chunk of a row (with its rotation partner for Q and K): the
  //      partials are summed in split order, q and k rotated, everything rounded to bf16.  Rows past the end are
  //      zero (a masked key's V row must be finite: 0 * NaN would poison O).  Two items per thread in flight.
  if (softmax_thread) {
    constexpr int HALF = kHD / 2, CPR = HALF / 8;
    uint8_t* dK = sKs, *dV = sVs;                        // tile 0 lives in the stages 0
    const uint4 zero = make_uint4(0, 0, 0, 0);
    for (int idx = lk_rows * CH + tid; idx < kKeys * CH; idx += kPipeThreads) {
      const int row = idx / CH, ch = idx % CH;
      *reinterpret_cast<uint4*>(dK + tile_off(row, ch)) = zero;
      *reinterpret_cast<uint4*>(dV + tile_off(row, ch)) = zero;
    }
    const int n_q = QT * CPR, n_k = lk_rows * CPR, n_v = lk_rows * CH;
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
        // the query tile is replicated to 128 lanes: lane k * QT + row holds query row `row`
#pragma unroll
        for (int k = 0; k < 128 / QT; ++k) {
          *reinterpret_cast<uint4*>(sQ + tile_off(k * QT + w.row, w.c)) = lo;
          *reinterpret_cast<uint4*>(sQ + tile_off(k * QT + w.row, w.c + 8)) = hi;
        }
      } else if (w.kind == 1) {
        *reinterpret_cast<uint4*>(dK + tile_off(w.row, w.c)) = lo;
        *reinterpret_cast<uint4*>(dK + tile_off(w.row, w.c + 8)) = hi;
        if (commit_kv && lk_begin + w.row < commit_rows) {
          bf16* dst = a.cache_k_out + (size_t)seq_of_slot(a.map, slot) * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride +
                      (size_t)(a.map.pos0 + lk_begin + w.row) * a.kv_pos_stride + w.c * 8;
          *reinterpret_cast<uint4*>(dst) = lo;
          *reinterpret_cast<uint4*>(dst + HALF) = hi;
        }
      } else {
        *reinterpret_cast<uint4*>(dV + tile_off(w.row, w.c)) = lo;
        if (commit_kv && lk_begin + w.row < commit_rows)
          *reinterpret_cast<uint4*>(a.cache_v_out + (size_t)seq_of_slot(a.map, slot) * a.cache_seq_stride +
                                    (size_t)kvh * a.kv_head_stride + (size_t)(a.map.pos0 + lk_begin + w.row) * a.kv_pos_stride + w.c * 8) = lo;
      }
    };
    for (int it = tid; it < n_q + n_k + n_v; it += 2 * kPipeThreads) {
      const Item A = decode(it), B = decode(it + kPipeThreads);
      float x1[8], x2[8], z1[8], z2[8];
      gather(A, x1, x2);
      gather(B, z1, z2);
      finish(A, x1, x2);
      finish(B, z1, z2);
    }
  }
  cp_async_wait<0>();
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_O = tmem_base + 256;
  const uint32_t bar_s0 = smem_u32(&bars[0]), bar_o = smem_u32(&bars[2]), bar_k0 = smem_u32(&bars[3]), bar_p = smem_u32(&bars[5]);
  const uint32_t bar_v0 = smem_u32(&bars[6]);
  bool ok = true;

  if (warp == kPipeThreads / 32) {
    // ================================================================== MMA warp
    // Per tile u: S(u+1) = Q K(u+1)^T as soon as the softmax threads report K(u+1) landed (they do so when they
    // enter tile u, i.e. after they have read S(u-1), whose accumulator S(u+1) overwrites), then O += P(u) V(u) as
    // soon as they report P(u) written and V(u) landed.  The tensor core runs the MMAs in issue order.
    if ((tid & 31) == 0) {
      // f32 accumulate, bf16 operands, N = 128, M = 128; bit 16: B is MN-major (V as stored, [key][hd])
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      const uint32_t idesc_pv = idesc | (1u << 16);
      auto issue_s = [&](int u) {                        // S[u & 1] = Q . K(u)^T: eight k16 steps over the head dimension
        const uint32_t kbase = smem_u32(sKs + (size_t)(u % kStagesK) * kTileBytes);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t qa = smem_u32(sQ) + (uint32_t)((k >> 2) * kHalfBytes + (k & 3) * 32);
          const uint32_t ka = kbase + (uint32_t)((k >> 2) * kHalfBytes + (k & 3) * 32);
          tc_mma_bf16(tmem_base + (uint32_t)(u & 1) * 128u, make_desc(qa, 16, 1024), make_desc(ka, 16, 1024), idesc, (uint32_t)(k != 0));
        }
        tc_commit(bar_s0 + 8u * (uint32_t)(u & 1));
      };
      issue_s(0);
#pragma unroll 1
      for (int u = 0; u < n_tiles && ok; ++u) {
        if (u + 1 < n_tiles) {
          ok = mbar_wait(bar_k0 + 8u * (uint32_t)((u + 1) & 1), (uint32_t)((u >> 1) & 1), abort_flag);
          if (!ok) break;
          tc_fence_after();
          issue_s(u + 1);
        }
        ok = mbar_wait(bar_p, (uint32_t)(u & 1), abort_flag);
        if (ok && bulk(u)) ok = mbar_wait(bar_v0 + 8u * (uint32_t)(u & 1), (uint32_t)(((u - 1) >> 1) & 1), abort_flag);
        if (!ok) break;
        tc_fence_after();
        // O (+)= P . V: eight k16 steps over the keys.  P is K-major (keys contiguous); V is used as stored,
        // [key][hd] = MN-major: 8-key groups 1024 B apart, the two 64-column halves 16 KB apart.
        const uint32_t vbase = smem_u32(sVs + (size_t)(u % kStagesV) * kTileBytes);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t pa = smem_u32(sP) + (uint32_t)((k >> 2) * kHalfBytes + (k & 3) * 32);
          const uint32_t va = vbase + (uint32_t)(2 * k * 1024);
          tc_mma_bf16(tmem_O, make_desc(pa, 16, 1024), make_desc(va, kHalfBytes, 1024), idesc_pv, (uint32_t)((u | k) != 0));
        }
        tc_commit(bar_o);
      }
      if (!ok) atomicExch(a.err_flag, 6);
    }
  } else if (!softmax_thread) {
    // ================================================================== copy warp (bulk tiles)
    // Lane 0 asks for K of tile t once S of tile t-2 is complete (its stage is free then), lane 1 for V of tile t once
    // O += P V of tile t-2 is.  A tile the softmax threads copy themselves only gets lane 0's arrival on its K barrier.
    const int lane = tid & 31;
    if (lane < 2 && n_tiles > 1) {
      const int seq = seq_of_slot(a.map, slot);
      const int row_base = (int)(((size_t)seq * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride) / kHD);   // row of key 0 in the [rows][128] view
#pragma unroll 1
      for (int t = 2; t < n_tiles && ok; ++t) {          // (tile 1 was asked for before the prologue)
        const int r0 = row_base + (t - 1) * kKeys;
        if (lane == 0) {
          if (t >= 2) ok = mbar_wait(bar_s0 + 8u * (uint32_t)(t & 1), (uint32_t)(((t - 2) >> 1) & 1), abort_flag);
          if (!ok) break;
          const uint32_t kb_ = bar_k0 + 8u * (uint32_t)(t & 1);
          if (bulk(t)) {
            const uint32_t dst = smem_u32(sKs + (size_t)(t % kStagesK) * kTileBytes);
            mbar_arrive_expect_tx(kb_, (uint32_t)kTileBytes);
            tma_load_2d(dst, &tmK, kb_, 0, r0);
            tma_load_2d(dst + kHalfBytes, &tmK, kb_, 64, r0);
          } else {
            mbar_arrive(kb_);
          }
        } else if (bulk(t)) {
          if (t >= 2) ok = mbar_wait(bar_o, (uint32_t)((t - 2) & 1), abort_flag);
          if (!ok) break;
          const uint32_t vb_ = bar_v0 + 8u * (uint32_t)(t & 1);
          const uint32_t dst = smem_u32(sVs + (size_t)(t % kStagesV) * kTileBytes);
          mbar_arrive_expect_tx(vb_, (uint32_t)kTileBytes);
          tma_load_2d(dst, &tmV, vb_, 0, r0);
          tma_load_2d(dst + kHalfBytes, &tmV, vb_, 64, r0);
        }
      }
      if (!ok) atomicExch(a.err_flag, 6);
    }
  } else {
    // ================================================================== softmax threads (log2 domain)
    // TMEM lane lt = copy `cw` of query row `row`; a copy covers the keys [cw * QT, +QT) of a tile and the lane's
    // two threads (hw = 0, 1) half of those each, in 16-key chunks.  A tile's row sum is ALWAYS formed from its
    // eight 16-key chunks as (((c0 + c1) + (c2 + c3)) + (c4 + c5)) + (c6 + c7), each chunk summed in key order,
    // whatever QT is.  The threads meet once per tile (exchange of the row maxima); everything else is handed
    // over through mbarriers, so that no thread waits for the MMA issue.
    constexpr int REP = 128 / QT;
    constexpr int KPT = QT / 2;                           // keys of a tile per thread
    constexpr int NCH = KPT / 16;                         // 16-key chunks per thread
    // A thread takes its keys in passes of at most 32 (its scores then fit in registers): one pass for tiles of 32
    // or 64 rows, whose scores stay in registers from the maximum to the exponentials; two for 128 rows, read again.
    constexpr int HK = KPT < 32 ? KPT : 32, NP = KPT / HK, NCP = HK / 16;
    const int lt = tid & 127, hw = tid >> 7;
    const int cw = lt / QT, row = lt % QT;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;   // warps w and w + 4 read TMEM lanes 32 (w & 3) ...
    const int col0 = cw * QT + hw * KPT;                  // first column (key of a tile) of this thread
    const int lr = lr0 + row;
    const bool row_live = lr < rps;
    // node-local keys this row may see, as key indices of tile 0 (key j = sequence row lk_begin + j)
    int loc_lo = (lr / T) * T - lk_begin, loc_hi = loc_lo + T;
    if (a.map.chain_T0 > 0 && lr % T < a.map.chain_T0) loc_hi = loc_lo + a.map.chain_T0;   // finished block: not the next block
    loc_hi = min(loc_hi, lk_rows);
    float m_row = -INFINITY, l_row = 0.f;                 // running maximum; running sum up to the tile before the last one met
    bool broke = false;                                   // the loop ended at the meeting point, for all threads alike
    float corr_prev = 1.f;                                // rescale factor of the tile whose sum is still to be added
    auto tile_sum = [&](int u) -> float {                 // the row's sum over tile u, from the eight chunk sums
      const float* q = sSum + (u & 1) * 8 * 128 + row;
      return (((q[0 * 128] + q[1 * 128]) + (q[2 * 128] + q[3 * 128])) + (q[4 * 128] + q[5 * 128])) + (q[6 * 128] + q[7 * 128]);
    };
#pragma unroll 1
    for (int u = 0; u < n_tiles; ++u) {
      // ---- K of the next tile (requested a whole iteration ago) has landed for this thread: tell the MMA warp.
      //      Copy groups are committed in the order K(u+1), V(u), K(u+2), V(u+1), ...
      if (u + 1 < n_tiles) {
        if (!bulk(u + 1)) {                                 // (a tile this thread helped to copy)
          cp_async_wait<1>();                               // everything but V(u), which has until O += P V
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        tc_fence_before();                                  // (this thread's reads of S(u-1) are complete)
        mbar_arrive(bar_k0 + 8u * (uint32_t)((u + 1) & 1));
      }
      ok = mbar_wait(bar_s0 + 8u * (uint32_t)(u & 1), (uint32_t)((u >> 1) & 1), abort_flag);
      tc_fence_after();
      ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;        // the tensor-memory accesses below are warp-wide
      // S of tile u is complete: its K stage takes K of tile u + 2
      if (ok && u + 2 < n_tiles && !bulk(u + 2)) load_cached(u + 2, true, false);
      cp_async_commit();
      const uint32_t tmem_S = tmem_base + (uint32_t)(u & 1) * 128u;
      const int key_lo = u == 0 ? loc_lo : 0;
      const int key_hi = u == 0 ? loc_hi : min(kKeys, a.S - (u - 1) * kKeys);
      const bool all_vis = key_lo <= col0 && key_hi >= col0 + KPT;   // every key of this thread's columns is visible
      // this thread's scores of the tile, a pass at a time: one round trip to tensor memory per pass
      uint32_t sv[HK];
      auto load_scores = [&](int pass) {
#pragma unroll
        for (int ch = 0; ch < NCP; ++ch) tmem_ld16_issue(tmem_S + lane_addr + col0 + pass * HK + ch * 16, &sv[ch * 16]);
        tmem_ld_wait();
#pragma unroll
        for (int ch = 0; ch < NCP; ++ch) keep16(&sv[ch * 16]);
      };
      float m_loc = -INFINITY;
      if (ok) {
#pragma unroll
        for (int pass = 0; pass < NP; ++pass) {
          load_scores(pass);
          if (all_vis) {                                    // (scale > 0: the maximum of the products is the product of the maximum)
            float m = __uint_as_float(sv[0]);
#pragma unroll
            for (int j = 1; j < HK; ++j) m = fmaxf(m, __uint_as_float(sv[j]));
            m_loc = fmaxf(m_loc, __fmul_rn(m, scale_log2));
          } else {
#pragma unroll
            for (int j = 0; j < HK; ++j) {
              const int key = col0 + pass * HK + j;
              if (key >= key_lo && key < key_hi) m_loc = fmaxf(m_loc, __fmul_rn(__uint_as_float(sv[j]), scale_log2));
            }
          }
        }
      } else {
#pragma unroll
        for (int j = 0; j < HK; ++j) sv[j] = 0u;
      }
      float* sMaxU = sMax + (u & 1) * 8 * 128;
      sMaxU[(hw * 4 + cw) * 128 + row] = m_loc;
      ok = softmax_barrier_and(ok);                         // the one meeting of a tile; also one decision for all
      if (!ok) { broke = true; break; }
      if (u > 0) {                                          // (every chunk sum of the previous tile is visible now)
        l_row = l_row * corr_prev + tile_sum(u - 1);
      }
      float m_tile = -INFINITY;
#pragma unroll
      for (int k = 0; k < REP; ++k) m_tile = fmaxf(m_tile, fmaxf(sMaxU[k * 128 + row], sMaxU[(4 + k) * 128 + row]));
      const float m_new = fmaxf(m_row, m_tile);
      const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
      const float corr = ex2(m_row - m_use);                // 0 while no visible key has been met
      if (u > 0) {
        // O += P V of the previous tile is complete: the P tile may be rewritten, its V stage takes V of tile u + 1,
        // and the output so far may be rescaled
        ok = mbar_wait(bar_o, (uint32_t)((u - 1) & 1), abort_flag);
        tc_fence_after();
        ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
      }
      if (ok && u + 1 < n_tiles && !bulk(u + 1)) load_cached(u + 1, false, true);
      cp_async_commit();
      // the output so far was accumulated against the old maximum: rescale this thread's columns of its lane - unless
      // no row of the warp moved its maximum (a factor of exactly 1 changes nothing)
      if (ok && u > 0 && __any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
        for (int pass = 0; pass < NP; ++pass) {
          uint32_t ov[HK];
#pragma unroll
          for (int ch = 0; ch < NCP; ++ch) tmem_ld16_issue(tmem_O + lane_addr + col0 + pass * HK + ch * 16, &ov[ch * 16]);
          tmem_ld_wait();
#pragma unroll
          for (int ch = 0; ch < NCP; ++ch) keep16(&ov[ch * 16]);
#pragma unroll
          for (int ch = 0; ch < NCP; ++ch) {
            float v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(ov[ch * 16 + j]) * corr;
            tmem_st16(tmem_O + lane_addr + col0 + pass * HK + ch * 16, v);
          }
        }
      }
      float* sSumU = sSum + (u & 1) * 8 * 128;
#pragma unroll
      for (int ch = 0; ch < NCH; ++ch) {
        if (NP > 1 && ch % NCP == 0 && ok) load_scores(ch / NCP);     // (one pass: the scores are still in registers)
        const int c0 = col0 + ch * 16;
        uint32_t packed[8];
        float csum = 0.f;
#pragma unroll
        for (int j = 0; j < 16; j += 2) {
          const int key = c0 + j;
          const float s0 = __uint_as_float(sv[(ch % NCP) * 16 + j]), s1 = __uint_as_float(sv[(ch % NCP) * 16 + j + 1]);
          // (the same arithmetic whether or not the visibility test is needed)
          float p0 = ex2(__fmaf_rn(s0, scale_log2, -m_use)), p1 = ex2(__fmaf_rn(s1, scale_log2, -m_use));
          if (!all_vis) {
            p0 = (key >= key_lo && key < key_hi) ? p0 : 0.f;
            p1 = (key + 1 >= key_lo && key + 1 < key_hi) ? p1 : 0.f;
          }
          csum += p0;
          csum += p1;
          packed[j >> 1] = pack_bf16(p0, p1);
        }
        sSumU[(c0 >> 4) * 128 + row] = csum;              // chunk index = c0 / 16
        // P, in every copy of the row
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const uint4 val = row_live ? make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3])
                                     : make_uint4(0, 0, 0, 0);
#pragma unroll
          for (int k = 0; k < REP; ++k)
            *reinterpret_cast<uint4*>(sP + tile_off(k * QT + row, (c0 >> 3) + q)) = val;
        }
      }
      // ---- this thread's part of P is written, its part of V(u) has landed, its rescale of O is complete: the MMA
      //      warp issues O += P V once every softmax thread has said so
      cp_async_wait<2>();                                   // V of this tile (two younger groups may still be in flight)
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // P and V are read by the tensor core
      tc_fence_before();
      mbar_arrive(bar_p);
      corr_prev = corr;
      m_row = m_new;
    }
    cp_async_wait<0>();                                     // nothing of this thread's copies is left in flight
    if (!broke) ok = softmax_barrier_and(ok);               // the last tile's chunk sums are visible
    if (ok) {
      l_row = l_row * corr_prev + tile_sum(n_tiles - 1);
      ok = mbar_wait(bar_o, (uint32_t)((n_tiles - 1) & 1), abort_flag);
      tc_fence_after();
    }
    ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
    if (ok) {
      // every copy of a row holds the same O row: a thread normalises and stores the columns it owns, [col0, +KPT)
      const float inv = 1.f / l_row;
      bf16* dst = a.out + ((grow0 + row) * a.H + h) * kHD + col0;
#pragma unroll
      for (int ch = 0; ch < NCH; ++ch) {
        float v[16];
        tmem_ld16(tmem_O + lane_addr + col0 + ch * 16, v);
        if (!row_live) continue;
        uint4 lo = make_uint4(pack_bf16(v[0] * inv, v[1] * inv), pack_bf16(v[2] * inv, v[3] * inv),
                              pack_bf16(v[4] * inv, v[5] * inv), pack_bf16(v[6] * inv, v[7] * inv));
        uint4 hi = make_uint4(pack_bf16(v[8] * inv, v[9] * inv), pack_bf16(v[10] * inv, v[11] * inv),
                              pack_bf16(v[12] * inv, v[13] * inv), pack_bf16(v[14] * inv, v[15] * inv));
        *reinterpret_cast<uint4*>(dst + ch * 16) = lo;
        *reinterpret_cast<uint4*>(dst + ch * 16 + 8) = hi;
      }
    } else if ((tid & 31) == 0) {
      atomicExch(a.err_flag, 6);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace

int launch_attention_verify_pipe(cudaStream_t st, const AttnArgs& a) {
  if (a.hd != kHD || !a.qkv_partial || !a.rope || !a.err_flag) return 1;
  if ((a.cache_k_out != nullptr) != (a.cache_v_out != nullptr)) return -1;
  const int rps = a.map.rows_per_seq, T = a.map.T;
  // Eligibility depends on the head dimension and the node width only - never on the number of rows - so that a
  // node meets the same arithmetic alone and among other nodes.  Node widths that divide 128 keep every query
  // tile's node-local keys inside one 128-key tile.
  if (T < 1 || (kKeys % T) != 0) return 1;
  const int qt_rows = rps <= 32 ? 32 : (rps <= 64 ? 64 : 128);
  const int q_tiles = (rps + qt_rows - 1) / qt_rows;
  const float scale_log2 = (1.0f / sqrtf((float)a.hd)) * 1.4426950408889634f;
  const size_t smem = (size_t)kTileBytes * (2 + kStagesK + kStagesV) + 16384 + 128 + 1024;   // Q, P, K and V stages, softmax exchange
  static bool attr_set[kMaxDevices] = {};        // the shared-memory opt-in is per device
  const int dev = device_slot();
  if (dev < 0) return -4;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(attn_verify_pipe_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(attn_verify_pipe_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(attn_verify_pipe_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return -4;
    attr_set[dev] = true;
  }
  // Whole tiles of cached keys go through the tensor-map engine when a head's keys are contiguous rows of the cache
  // viewed as [rows][128] (head-major layout, no hole in the key range); otherwise every tile is copied by the threads.
  alignas(64) CUtensorMap tmK, tmV;
  memset(&tmK, 0, sizeof(tmK));
  memset(&tmV, 0, sizeof(tmV));
  int use_tma = 0;
  if (a.cache_rows > 0 && a.kv_pos_stride == (size_t)kHD && a.hole_len == 0 && (a.cache_seq_stride % kHD) == 0 &&
      (a.kv_head_stride % kHD) == 0 && a.cache_rows < (size_t)0x7fffffff) {
    if (encode_tmap_bf16_2d(&tmK, a.cache_k, a.cache_rows, kHD, kHD, kKeys) != 0 ||
        encode_tmap_bf16_2d(&tmV, a.cache_v, a.cache_rows, kHD, kHD, kKeys) != 0)
      return -4;
    use_tma = 1;
  }
  dim3 grid(a.H, a.n_seq_slots * q_tiles);
  dim3 block(kPipeBlock);
  cudaError_t e;
  if (qt_rows == 32) e = launch_pdl(attn_verify_pipe_kernel<32>, grid, block, smem, st, tmK, tmV, a, scale_log2, use_tma);
  else if (qt_rows == 64) e = launch_pdl(attn_verify_pipe_kernel<64>, grid, block, smem, st, tmK, tmV, a, scale_log2, use_tma);
  else e = launch_pdl(attn_verify_pipe_kernel<128>, grid, block, smem, st, tmK, tmV, a, scale_log2, use_tma);
  return e == cudaSuccess ? 0 : -4;
}

}  // namespace ssd
