// Weight-streaming skinny GEMM for the projections of the verification forward:
//     out[r][n] = sum_k x[r][k] * w[n][k]      (bf16 operands, fp32 accumulation)
// with r = rows of ALL tree nodes (tens to a few hundred) and n = output features (thousands).
// The weight matrix is the big operand and is read from HBM exactly once per forward; the
// activations are small and stay in L2.
//
// Tensor-core kernel (sm_100a): "swap-AB" mapping.  A CTA owns 128 output features: the weight
// tile [128 x 64] is the M x K operand of tcgen05.mma, the activation tile [rows x 64] is the
// N x K operand, the fp32 accumulator [128 lanes x rows columns] lives in tensor memory.  Both
// tiles are staged by TMA (128-byte swizzle) through an mbarrier ring; one thread issues the
// MMAs; four warps read the accumulator back with tcgen05.ld and run the epilogue:
//   EPI_PARTIAL  fp32 partial sums per K split (summed later in split order),
//   EPI_SWIGLU   weight rows interleaved as 64 gate + 64 up features per tile -> silu(g)*u in bf16,
//   EPI_LMHEAD   per-row max / argmax / sum-exp over the tile's 128 vocabulary entries, so the
//                logits never leave the SM.
// Every wait is bounded: on expiry the kernel raises an error word and unwinds.
#include "kernels.h"

#include <cuda.h>
#include <math.h>
#include <stdio.h>

namespace ssd {

int gemm_tiles(int N) { return (N + 127) / 128; }

// =====================================================================================
// Tensor-core kernel
// =====================================================================================
namespace {

constexpr int kTileM = 128;          // output features per CTA (MMA M)
constexpr int kBlockK = 64;          // bf16 elements per stage along K = one 128-byte swizzle row
constexpr int kTcThreads = 192;      // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-5: epilogue
constexpr int kMaxStages = 8;
constexpr int kWTileBytes = kTileM * kBlockK * 2;
constexpr int kEpiPitch = 132;       // floats per row of the epilogue's transpose buffer (128 + padding)
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // default bound of a wait, 2 s: far beyond any legitimate one

struct TcParams {
  int R, N, K;
  int npad;        // MMA N: rows of one row chunk rounded up to 16 (<= 256)
  int splits;
  int stages;
  int epi;
  int w_tiled;     // weights in the tile-contiguous layout: one 16 KB block per (tile, K block)
  int two_sm;      // the CTAs of tiles 2i, 2i + 1 issue ONE tcgen05.mma.cta_group::2 (M = 256): each holds half of the activation tile
  uint32_t tmem_cols;
  float* out;
  bf16* act;
  int act_pitch;
  float* tile_max;
  float* tile_sum;
  int* tile_arg;
  unsigned long long wait_limit_ns;   // bound of every barrier wait
  int starve_kb;   // test hook, 0 = off: the producer leaves out the copies of K block starve_kb - 1, so the wait for it runs out
  int topk;        // EPI_LMHEAD: > 0 also writes the tile's `topk` largest logits per row (value, vocabulary index)
  float* tile_topv;
  int* tile_topi;
  int mask_id;
  int* err_flag;
  const float* sq;
  int sq_count, sq_stride, norm_dim;
  float norm_eps;
  float* h;
  bf16* hb;
  const float* gain;
  float* sq_out;
  int sq_out_stride;
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// Bounded wait.  Returns false when the limit expired or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63) == 0) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > limit_ns) return false;
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"((unsigned long long)map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// ---- forms for a pair of CTAs working as one MMA (cta_group::2).  The even CTA of the pair leads: it
// owns the "full" barriers (both CTAs' copies count their bytes there - the barrier address with the
// pair bit cleared), issues the MMAs, and its commits arrive on both CTAs' barriers.
constexpr uint32_t kPairLeaderMask = 0xFEFFFFFFu;       // shared::cluster address of the same offset in the even CTA
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"((unsigned long long)map), "r"(bar & kPairLeaderMask), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
  const uint32_t z = 0;
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n}\n"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(z) : "memory");
}
// K-major operand tile in shared memory, 128-byte swizzle, rows 128 B apart, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                 // leading-dimension byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;       // stride-dimension byte offset: 8 rows * 128 B
  d |= (uint64_t)1 << 46;                 // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                 // 128-byte swizzle
  return d;
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Cluster-wide barrier in two halves.  All 192 threads of every CTA of the cluster arrive once per
// phase; only threads that go on to touch remote shared memory need to wait.
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_rank(const void* p, uint32_t rank) {
  uint32_t out;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(smem_addr(p)), "r"(rank));
  return out;
}
// x^2 + y^2 + z^2 + w^2 with the roundings spelled out, so that the value does not depend on what the
// compiler contracts around it
__device__ __forceinline__ float sumsq4(const float4& a) {
  return __fmaf_rn(a.w, a.w, __fmaf_rn(a.z, a.z, __fmaf_rn(a.y, a.y, __fmul_rn(a.x, a.x))));
}
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}

// kTwoSm: the instantiation whose CTAs work in pairs (cluster of two along x); the single-CTA
// instantiation contains none of the pair instructions.
template <bool kTwoSm>
__global__ void __launch_bounds__(kTcThreads, 2)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const TcParams p) {
  extern __shared__ uint8_t smem_dyn[];
  // 1024-byte alignment for the swizzled tiles
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  constexpr bool ts = kTwoSm;
  const int x_tile_bytes = (ts ? p.npad / 2 : p.npad) * kBlockK * 2;    // a pair holds half of the rows each
  uint8_t* sW = smem;
  uint8_t* sX = smem + (size_t)p.stages * kWTileBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sX + (size_t)p.stages * x_tile_bytes);
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = bars + kMaxStages;
  uint64_t* acc_bar = bars + 2 * kMaxStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* s_inv = reinterpret_cast<float*>(bars + 32);           // [256] per-row 1/rms of the consumer side

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, split = blockIdx.y, row0 = blockIdx.z * 256;
  const int kb_total = (p.K + kBlockK - 1) / kBlockK;
  const int kb_begin = (int)((long long)split * kb_total / p.splits);
  const int kb_end = (int)((long long)(split + 1) * kb_total / p.splits);
  const int n_kb = kb_end - kb_begin;
  uint32_t crank = 0u;
  if constexpr (ts) crank = cluster_ctarank() & 1u;
  const bool leader = crank == 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_addr(&full_bar[s]), 1);
      mbar_init(smem_addr(&empty_bar[s]), 1);
    }
    mbar_init(smem_addr(acc_bar), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tmW) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tmX) : "memory");
  }
  if (warp == 1) {
    if constexpr (ts) {        // the same warp of both CTAs: the columns are taken in both SMs
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)),
                   "r"(p.tmem_cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)),
                   "r"(p.tmem_cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (ts) {                    // the peer's barriers exist before anything arrives on them
    cluster_arrive_release();
    cluster_wait_acquire();
  }
  const uint32_t tmem_base = *tmem_slot;

  bool epi_ok = false;       // epilogue threads: the accumulator is complete
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const uint32_t stage_bytes = (uint32_t)(kWTileBytes + x_tile_bytes);
      int issued = 0;
      bool ok = true;
      // In a pair only the leader's barrier counts: it expects both CTAs' bytes, and both CTAs' copies
      // complete on it.
      auto expect = [&](uint32_t fb) {
        if (!ts) mbar_expect_tx(fb, stage_bytes);
        else if (leader) mbar_expect_tx(fb, 2u * stage_bytes);
      };
      auto load_w = [&](int it, int s, uint32_t fb) {
        const int kb = kb_begin + it;
        const uint32_t dst = smem_addr(sW + (size_t)s * kWTileBytes);
        const int c0 = p.w_tiled ? 0 : kb * kBlockK, c1 = p.w_tiled ? (tile * kb_total + kb) * kTileM : tile * kTileM;
        if constexpr (ts) tma_load_2d_pair(dst, &tmW, fb, c0, c1);
        else tma_load_2d(dst, &tmW, fb, c0, c1);
      };
      auto load_x = [&](int it, int s, uint32_t fb) {
        const uint32_t dst = smem_addr(sX + (size_t)s * x_tile_bytes);
        if constexpr (ts) tma_load_2d_pair(dst, &tmX, fb, (kb_begin + it) * kBlockK, row0 + (int)crank * (p.npad / 2));
        else tma_load_2d(dst, &tmX, fb, (kb_begin + it) * kBlockK, row0);
      };
      // The weights do not depend on any earlier kernel: fill the ring with weight tiles first, and
      // only then wait for the kernel that produces the activations.
      const int pre = n_kb < p.stages ? n_kb : p.stages;
      // (test hook: a starved K block gets neither its byte count nor its copies - its barrier never completes)
      auto starved = [&](int it) { return p.starve_kb > 0 && kb_begin + it == p.starve_kb - 1; };
      for (int it = 0; it < pre; ++it) {
        if (starved(it)) continue;
        const uint32_t fb = smem_addr(&full_bar[it]);
        expect(fb);
        load_w(it, it, fb);
      }
      pdl_wait();
      for (int it = 0; it < pre; ++it) {
        if (starved(it)) continue;
        load_x(it, it, smem_addr(&full_bar[it]));
        ++issued;
      }
      for (int it = pre; it < n_kb; ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (uint32_t)((it / p.stages) & 1);
        if (!mbar_wait(smem_addr(&empty_bar[s]), ph ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
        if (starved(it)) continue;
        const uint32_t fb = smem_addr(&full_bar[s]);
        expect(fb);
        load_w(it, s, fb);
        load_x(it, s, fb);
        ++issued;
      }
      if (!ok) {
        *abort_flag = 1;
        atomicExch(p.err_flag, 1);
        // let the copies already in flight land before the CTA's shared memory goes away
        const int first = issued > p.stages ? issued - p.stages : 0;
        for (int j = first; j < issued && (!ts || leader); ++j) {
          const unsigned long long t0 = globaltimer_ns();
          while (!mbar_try_wait(smem_addr(&full_bar[j % p.stages]), (uint32_t)((j / p.stages) & 1)))
            if (globaltimer_ns() - t0 > p.wait_limit_ns) break;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && leader) {        // (in a pair the even CTA issues for both)
      // M = 128 features of this CTA, or 256 = the pair's two weight tiles; N = the padded rows
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.npad >> 3) << 17) |
                             ((uint32_t)((ts ? 2 * kTileM : kTileM) >> 4) << 24);
      bool ok = true;
      for (int it = 0; it < n_kb; ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (uint32_t)((it / p.stages) & 1);
        if (!mbar_wait(smem_addr(&full_bar[s]), ph, abort_flag, p.wait_limit_ns)) { ok = false; break; }
        tc_fence_after();
        const uint32_t wa = smem_addr(sW + (size_t)s * kWTileBytes);
        const uint32_t xa = smem_addr(sX + (size_t)s * x_tile_bytes);
#pragma unroll
        for (int k = 0; k < kBlockK / 16; ++k) {
          if constexpr (ts) tc_mma_bf16_pair(tmem_base, make_smem_desc(wa + k * 32), make_smem_desc(xa + k * 32), idesc,
                                   (uint32_t)((it | k) != 0));
          else tc_mma_bf16(tmem_base, make_smem_desc(wa + k * 32), make_smem_desc(xa + k * 32), idesc,
                           (uint32_t)((it | k) != 0));
        }
        // a pair's commits arrive on both CTAs' barriers; only stages that will be refilled need one
        if constexpr (!ts) tc_commit(smem_addr(&empty_bar[s]));
        else if (it + p.stages < n_kb) tc_commit_pair(smem_addr(&empty_bar[s]));
      }
      if (ok) {
        if constexpr (ts) tc_commit_pair(smem_addr(acc_bar));
        else tc_commit(smem_addr(acc_bar));
      } else {
        *abort_flag = 1;
        atomicExch(p.err_flag, 2);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (4 warps)
    const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
    const int lrow = quad * 32 + lane;         // accumulator lane = feature inside the tile
    pdl_wait();                                // outputs may still be read by the predecessor
    const int et = threadIdx.x - 64;           // 0..127 among the epilogue threads
    if (p.sq != nullptr) {
      // fused RMSNorm, consumer side: 1/rms of every row from the producers' per-tile sums of squares
      // (summed in slot order), computed while the main loop still runs
      for (int rr = et; rr < p.npad; rr += 128) {
        float inv = 0.f;
        if (row0 + rr < p.R) {
          const float* q = p.sq + (size_t)(row0 + rr) * p.sq_stride;
          float ss = 0.f;
          for (int t = 0; t < p.sq_count; ++t) ss += q[t];
          inv = rsqrtf(ss / (float)p.norm_dim + p.norm_eps);
        }
        s_inv[rr] = inv;
      }
      epi_bar_sync();
    }
    bool ok = true;
    if (n_kb > 0) ok = mbar_wait(smem_addr(acc_bar), 0u, abort_flag, p.wait_limit_ns);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const int rows_here = min(p.R - row0, 256);
    float* scratch = reinterpret_cast<float*>(sW);   // stage 0 of the ring is free once acc_bar fired
    epi_ok = ok;
    if (!ok) {
      if (lane == 0) { *abort_flag = 1; atomicExch(p.err_flag, 3); }
    } else if (p.epi == EPI_RESIDUAL) {
      // after the role branches: every thread of the CTA takes part in the cluster barriers
    } else if (p.epi == EPI_PARTIAL) {
      // Transpose 32 rows x 128 features through shared memory so that a thread stores four
      // consecutive features of one row: 8 vector stores per thread and chunk instead of 32 scalars.
      const int n_base = tile * kTileM;
      const bool vec_ok = ((p.N & 3) == 0) && (n_base + kTileM <= p.N);
      for (int c0 = 0; c0 < p.npad; c0 += 32) {
        float v[32];
        if (n_kb > 0) tmem_ld32(taddr + c0, v);
        else {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0.f;
        }
        if (p.sq != nullptr) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] *= s_inv[c0 + j];
        }
        if (vec_ok) {
#pragma unroll
          for (int j = 0; j < 32; ++j) scratch[j * kEpiPitch + lrow] = v[j];
          epi_bar_sync();
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int rr = i * 4 + (et >> 5);          // row inside the chunk
            const int f4 = (et & 31) * 4;              // first of four features
            if (c0 + rr < rows_here) {
              const float4 val = *reinterpret_cast<const float4*>(scratch + rr * kEpiPitch + f4);
              *reinterpret_cast<float4*>(p.out + ((size_t)split * p.R + row0 + c0 + rr) * p.N + n_base + f4) = val;
            }
          }
          epi_bar_sync();
        } else {
          const int n = n_base + lrow;
          if (n < p.N) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int rr = c0 + j;
              if (rr < rows_here) p.out[((size_t)split * p.R + row0 + rr) * p.N + n] = v[j];
            }
          }
        }
      }
    } else if (p.epi == EPI_SWIGLU) {
      // lanes 0-63 hold gate features, lanes 64-127 the matching up features.  After the transpose a
      // thread owns 16 consecutive features of one row: silu(gate) * up, 32 bytes of bf16 per thread.
      const int rr = et >> 2, fg = (et & 3) * 16;
      for (int c0 = 0; c0 < p.npad; c0 += 32) {
        float v[32];
        tmem_ld32(taddr + c0, v);
        if (p.sq != nullptr) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] *= s_inv[c0 + j];
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) scratch[j * kEpiPitch + lrow] = v[j];
        epi_bar_sync();
        if (c0 + rr < rows_here) {
          uint32_t packed[8];
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const float4 g = *reinterpret_cast<const float4*>(scratch + rr * kEpiPitch + fg + q4 * 4);
            const float4 u = *reinterpret_cast<const float4*>(scratch + rr * kEpiPitch + 64 + fg + q4 * 4);
            const float a0 = g.x / (1.f + expf(-g.x)) * u.x, a1 = g.y / (1.f + expf(-g.y)) * u.y;
            const float a2 = g.z / (1.f + expf(-g.z)) * u.z, a3 = g.w / (1.f + expf(-g.w)) * u.w;
            __nv_bfloat162 lo = __floats2bfloat162_rn(a0, a1), hi = __floats2bfloat162_rn(a2, a3);
            packed[q4 * 2] = *reinterpret_cast<uint32_t*>(&lo);
            packed[q4 * 2 + 1] = *reinterpret_cast<uint32_t*>(&hi);
          }
          uint4* dst = reinterpret_cast<uint4*>(p.act + (size_t)(row0 + c0 + rr) * p.act_pitch + tile * 64 + fg);
          dst[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
          dst[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
        }
        epi_bar_sync();
      }
    } else {
      // EPI_LMHEAD: lane = vocabulary entry; reduce over the 128 lanes per row (= column)
      const int n = tile * kTileM + lrow;
      const bool live = (n < p.N) && (n != p.mask_id);
      {
        // Statistics.  32 rows at a time are transposed through shared memory (dead entries as -inf); four threads
        // then share a row: each scans a quarter of the tile's 128 entries in index order - maximum with the lowest
        // index among equals, sum of exp(x - its maximum) - and the quarters are merged (0 + 1) + (2 + 3).  The order
        // depends on the tile alone.
        const int rr = et >> 2, qf = (et & 3) * 32;
        for (int c0 = 0; c0 < p.npad; c0 += 32) {
          float v[32];
          tmem_ld32(taddr + c0, v);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float x = p.sq != nullptr ? v[j] * s_inv[c0 + j] : v[j];
            scratch[j * kEpiPitch + lrow] = live ? x : -INFINITY;
          }
          epi_bar_sync();
          float m = -INFINITY, sum = 0.f;
          int arg = 0x7fffffff;
          {
            float x[32];
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4) {
              const float4 t4 = *reinterpret_cast<const float4*>(scratch + rr * kEpiPitch + qf + q4 * 4);
              x[q4 * 4] = t4.x; x[q4 * 4 + 1] = t4.y; x[q4 * 4 + 2] = t4.z; x[q4 * 4 + 3] = t4.w;
            }
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (x[j] > m) { m = x[j]; arg = tile * kTileM + qf + j; }
            if (m != -INFINITY) {
#pragma unroll
              for (int j = 0; j < 32; ++j) sum += expf(x[j] - m);          // (exp(-inf) = 0 for dead entries)
            }
          }
#pragma unroll
          for (int o = 1; o <= 2; o <<= 1) {                               // quarters: (0 + 1), (2 + 3), then the pairs
            const float om = __shfl_xor_sync(0xffffffffu, m, o);
            const float os = __shfl_xor_sync(0xffffffffu, sum, o);
            const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
            // the same value from both partners: the lower quarter's (maximum, index) wins a tie
            const bool lower = (et & o) == 0;
            const float m_lo = lower ? m : om, s_lo = lower ? sum : os, m_hi = lower ? om : m, s_hi = lower ? os : sum;
            const int a_lo = lower ? arg : oa, a_hi = lower ? oa : arg;
            const float M = fmaxf(m_lo, m_hi);
            float S = 0.f;
            if (m_lo != -INFINITY) S += s_lo * expf(m_lo - M);
            if (m_hi != -INFINITY) S += s_hi * expf(m_hi - M);
            arg = (m_hi > m_lo) ? a_hi : a_lo;
            m = M;
            sum = S;
          }
          if ((et & 3) == 0 && c0 + rr < rows_here) {
            const size_t o = (size_t)tile * p.R + row0 + c0 + rr;
            p.tile_max[o] = m;
            p.tile_sum[o] = sum;
            p.tile_arg[o] = arg;
          }
          epi_bar_sync();
        }
      }
      if (p.topk > 0) {
        // The tile's largest logits on top of the statistics above (the acceptance-limit probe)
      for (int c0 = 0; c0 < p.npad; c0 += 32) {
        {
          // The tile's `topk` largest logits of every row of the chunk (value descending, lower index first):
          // per warp by repeated warp-wide argmax with the winner struck out, then the four warps' sorted
          // lists are merged by one thread per row.
          float* s_tv = scratch + 12 * 256;              // [4 warps][kLmTopKMax][32 rows]
          int* s_ti = reinterpret_cast<int*>(s_tv + 4 * kLmTopKMax * 32);
          float tv[kLmTopKMax];
          int ti[kLmTopKMax];
#pragma unroll
          for (int r = 0; r < kLmTopKMax; ++r) { tv[r] = -INFINITY; ti[r] = 0x7fffffff; }
          float w[32];                                   // a copy of its own: indexed by a loop variable below
          tmem_ld32(taddr + c0, w);
#pragma unroll 1
          for (int j = 0; j < 32; ++j) {
            float x = live ? (p.sq != nullptr ? w[j] * s_inv[c0 + j] : w[j]) : -INFINITY;
#pragma unroll
            for (int r = 0; r < kLmTopKMax; ++r) {
              if (r < p.topk) {
                float m = x;
                int a = n;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                  const float om = __shfl_xor_sync(0xffffffffu, m, o);
                  const int oa = __shfl_xor_sync(0xffffffffu, a, o);
                  if (om > m || (om == m && oa < a)) { m = om; a = oa; }
                }
                if (a == n) x = -INFINITY;               // struck out for the next round
                if (lane == j) { tv[r] = m; ti[r] = (m == -INFINITY) ? 0x7fffffff : a; }
              }
            }
          }
#pragma unroll
          for (int r = 0; r < kLmTopKMax; ++r) {
            s_tv[(quad * kLmTopKMax + r) * 32 + lane] = tv[r];
            s_ti[(quad * kLmTopKMax + r) * 32 + lane] = ti[r];
          }
          epi_bar_sync();
          if (warp == 2 && c0 + lane < rows_here) {
            int head[4] = {0, 0, 0, 0};
            const size_t o = ((size_t)tile * p.R + row0 + c0 + lane) * kLmTopKMax;
            for (int r = 0; r < p.topk; ++r) {
              float bm = -INFINITY;
              int ba = 0x7fffffff, bq = 0;
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                if (head[q] < p.topk) {
                  const float m = s_tv[(q * kLmTopKMax + head[q]) * 32 + lane];
                  const int a = s_ti[(q * kLmTopKMax + head[q]) * 32 + lane];
                  if (m > bm || (m == bm && a < ba)) { bm = m; ba = a; bq = q; }
                }
              }
              ++head[bq];
              p.tile_topv[o + r] = bm;
              p.tile_topi[o + r] = ba;
            }
          }
          epi_bar_sync();
        }
      }
      }
    }
  }
  if (p.epi == EPI_RESIDUAL) {
    // ---- split-K reduction inside the cluster + residual + operand of the next projection.
    // Per pass (all rows when the tile ring can hold them): every CTA stages its partial [rows][128
    // features] in shared memory;
    // after a cluster barrier CTA `rank` owns the rows rank, rank + splits, ... (one warp per row, a
    // lane per four features): it adds the partials in split order to the residual stream, writes h,
    // bf16(h * gain) and the tile's sum of squares of the row.  A second barrier frees the staging
    // buffer.  Every thread of every CTA passes both barriers of every pass, also after an error.
    const bool epi_warp = warp >= 2;
    const int quad = warp & 3;
    const int lrow = quad * 32 + lane;
    const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const int rows_here = min(p.R - row0, 256);
    float* scratch = reinterpret_cast<float*>(sW);
    const uint32_t n_ranks = (uint32_t)p.splits, rank = cluster_ctarank();
    const int n_base = tile * kTileM;
    const int f4 = lane * 4;
    const bool col_ok = n_base + f4 < p.N;
    float4 g4 = make_float4(0.f, 0.f, 0.f, 0.f);
    if (epi_warp && col_ok) g4 = *reinterpret_cast<const float4*>(p.gain + n_base + f4);
    // as many 32-row chunks per pass as the (now idle) tile ring can stage
    int pass_rows = (p.stages * (kWTileBytes + x_tile_bytes)) / (kEpiPitch * 4) / 32 * 32;
    const int npad32 = (p.npad + 31) & ~31;               // whole chunks (TMEM holds a power of two >= 32 columns)
    if (pass_rows > npad32) pass_rows = npad32;
    for (int g0 = 0; g0 < npad32; g0 += pass_rows) {
      const int pass_cnt = min(pass_rows, npad32 - g0);
      if (epi_warp && epi_ok) {
        for (int c0 = 0; c0 < pass_cnt; c0 += 32) {
          float v[32];
          if (n_kb > 0) tmem_ld32(taddr + g0 + c0, v);       // a split without K blocks issued no MMA: it adds zeros
          else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0.f;
          }
#pragma unroll
          for (int j = 0; j < 32; ++j) scratch[(c0 + j) * kEpiPitch + lrow] = v[j];
        }
      }
      __syncwarp();
      cluster_arrive_release();
      cluster_wait_acquire();
      bool arrived = false;
      if (epi_warp && epi_ok) {
        // a warp takes its rows two at a time: the remote reads of both are in flight together
        const int step = 4 * (int)n_ranks;
        auto pull = [&](int rr, bool on, float4 (&part)[kGemmMaxClusterSplits]) {
#pragma unroll
          for (int q = 0; q < kGemmMaxClusterSplits; ++q) {
            part[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (on && (uint32_t)q < n_ranks) part[q] = ld_cluster_f32x4(map_to_rank(scratch + rr * kEpiPitch + f4, (uint32_t)q));
          }
        };
        // residual + partials in split order
        auto reduce = [&](float4 acc, const float4 (&part)[kGemmMaxClusterSplits]) -> float4 {
#pragma unroll
          for (int q = 0; q < kGemmMaxClusterSplits; ++q) {
            if ((uint32_t)q < n_ranks) { acc.x += part[q].x; acc.y += part[q].y; acc.z += part[q].z; acc.w += part[q].w; }
          }
          return acc;
        };
        // h, bf16(h * gain) and the tile's sum of squares of the row
        auto store = [&](int row, const float4& acc) {
          float ss = 0.f;
          if (col_ok) {
            *reinterpret_cast<float4*>(p.h + (size_t)(row0 + row) * p.N + n_base + f4) = acc;
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * g4.x, acc.y * g4.y);
            __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * g4.z, acc.w * g4.w);
            *reinterpret_cast<uint2*>(p.hb + (size_t)(row0 + row) * p.N + n_base + f4) =
                make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
            ss = sumsq4(acc);
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
          if (lane == 0) p.sq_out[(size_t)(row0 + row) * p.sq_out_stride + tile] = ss;
        };
        for (int rrA = (int)rank + (warp - 2) * (int)n_ranks; rrA < pass_cnt; rrA += 2 * step) {
          if (g0 + rrA >= rows_here) break;
          const int rrB = rrA + step;
          const bool onB = rrB < pass_cnt && g0 + rrB < rows_here;
          float4 partA[kGemmMaxClusterSplits], partB[kGemmMaxClusterSplits];
          pull(rrA, true, partA);
          pull(rrB, onB, partB);
          float4 hA = make_float4(0.f, 0.f, 0.f, 0.f), hB = hA;
          if (col_ok) hA = *reinterpret_cast<const float4*>(p.h + (size_t)(row0 + g0 + rrA) * p.N + n_base + f4);
          if (col_ok && onB) hB = *reinterpret_cast<const float4*>(p.h + (size_t)(row0 + g0 + rrB) * p.N + n_base + f4);
          const float4 accA = reduce(hA, partA), accB = reduce(hB, partB);   // (uses every value read remotely)
          // this warp's last remote read of the pass has landed: arrive now, the stores overlap the barrier
          const int nextA = rrA + 2 * step;
          if (nextA >= pass_cnt || g0 + nextA >= rows_here) {
            __syncwarp();
            cluster_arrive_release();
            arrived = true;
          }
          store(g0 + rrA, accA);
          if (onB) store(g0 + rrB, accB);
        }
      }
      if (!arrived) { __syncwarp(); cluster_arrive_release(); }
      cluster_wait_acquire();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (ts) {                    // both CTAs have read their accumulators; nothing is on its way between them
    cluster_arrive_release();
    cluster_wait_acquire();
  }
  if (warp == 1) {
    if constexpr (ts) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// [rows][pitch] bf16, K contiguous; box = 64 x box_rows; out-of-range elements read as zero
bool make_tmap(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint64_t pitch_elems, uint32_t box_rows) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {pitch_elems * 2};
  cuuint32_t box[2] = {(cuuint32_t)kBlockK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

// (for other kernels of the library that copy bf16 tiles with the tensor-map engine: boxes of 64 columns x box_rows rows,
// 128-byte swizzle)
int encode_tmap_bf16_2d(void* map_out, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch_elems, uint32_t box_rows) {
  if (!g_encode && gemm_tc_init() != 0) return -4;
  return make_tmap(reinterpret_cast<CUtensorMap*>(map_out), base, rows, cols, pitch_elems, box_rows) ? 0 : -4;
}

int gemm_tc_init() {
  if (g_encode) return 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
      q != cudaDriverEntryPointSuccess)
    return -4;
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return 0;
}

int launch_gemm_tc(cudaStream_t st, const GemmArgs& g) {
  if (!g_encode) return -4;
  if ((g.x_pitch % 8) || (!g.w_tiled && (g.w_pitch % 8)) || (((uintptr_t)g.x) & 15) || (((uintptr_t)g.w) & 15)) return -2;
  if (g.R < 1 || g.N < 1 || g.K < 1) return -2;
  if (g.splits < 1 || g.splits > (g.K + kBlockK - 1) / kBlockK) return -2;   // every split owns at least one K block
  if (g.epi != EPI_PARTIAL && g.epi != EPI_RESIDUAL && g.splits != 1) return -2;
  if (g.epi == EPI_RESIDUAL &&
      (g.splits < 1 || g.splits > kGemmMaxClusterSplits || (g.N & 3) || !g.h || !g.hb || !g.gain || !g.sq_out)) return -2;
  if (g.sq != nullptr && (g.sq_count < 1 || g.norm_dim < 1)) return -2;
  if (g.epi == EPI_SWIGLU && (g.N % 128)) return -2;
  TcParams p;
  p.R = g.R; p.N = g.N; p.K = g.K;
  const int rows_chunk = g.R < 256 ? g.R : 256;
  p.npad = (rows_chunk + 15) & ~15;
  p.splits = g.splits;
  p.epi = g.epi;
  p.w_tiled = g.w_tiled;
  // Pairs of tiles as one two-SM MMA from `two_sm_min_rows` padded rows on (0: never): every SM then takes
  // in half of the activation tile.  The accumulation order is the same, so the row count may decide.
  p.two_sm = (g.two_sm_min_rows > 0 && p.npad >= g.two_sm_min_rows && g.epi != EPI_RESIDUAL && (gemm_tiles(g.N) % 2) == 0) ? 1 : 0;
  uint32_t cols = 32;
  while ((int)cols < p.npad) cols <<= 1;
  p.tmem_cols = cols;
  const int stage_bytes = kWTileBytes + (p.two_sm ? p.npad / 2 : p.npad) * kBlockK * 2;
  // two CTAs per SM while the activation tile is small, one deep pipeline otherwise
  const int budget = 108 * 1024;
  int stages = budget / stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (g.max_stages > 0 && stages > g.max_stages) stages = g.max_stages;
  if (stages < 2) stages = 2;
  p.stages = stages;
  p.out = g.out; p.act = g.act; p.act_pitch = g.act_pitch;
  p.tile_max = g.tile_max; p.tile_sum = g.tile_sum; p.tile_arg = g.tile_arg;
  p.wait_limit_ns = g.wait_limit_ns > 0 ? g.wait_limit_ns : kWaitLimitNs;
  p.starve_kb = g.starve_kb;
  // the starvation hook is for the plain single-CTA launch only (no cluster partner waits on this CTA)
  if (g.starve_kb != 0 && (g.epi != EPI_PARTIAL || g.splits != 1 || g.R > 256)) return -2;
  p.topk = g.topk; p.tile_topv = g.tile_topv; p.tile_topi = g.tile_topi;
  if (g.topk < 0 || g.topk > kLmTopKMax || (g.topk > 0 && (g.epi != EPI_LMHEAD || !g.tile_topv || !g.tile_topi))) return -2;
  p.mask_id = g.mask_id; p.err_flag = g.err_flag;
  p.sq = g.sq; p.sq_count = g.sq_count; p.sq_stride = g.sq_stride; p.norm_dim = g.norm_dim; p.norm_eps = g.norm_eps;
  p.h = g.h; p.hb = g.hb; p.gain = g.gain; p.sq_out = g.sq_out; p.sq_out_stride = g.sq_out_stride;
  const int smem = stages * stage_bytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + 1024 /*per-row 1/rms*/;
  // tensor-memory safety: CTAs that fit by shared memory must also fit by TMEM columns
  if ((227 * 1024 / smem) * (int)cols > 512) return -2;
  CUtensorMap tmW, tmX;
  if (g.w_tiled) {
    // [tiles * K blocks * 128 rows][64]: every box is one contiguous 16 KB block
    const uint64_t rows = (uint64_t)gemm_tiles(g.N) * ((g.K + kBlockK - 1) / kBlockK) * kTileM;
    if (!make_tmap(&tmW, g.w, rows, kBlockK, kBlockK, kTileM)) return -4;
  } else if (!make_tmap(&tmW, g.w, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.w_pitch, kTileM)) {
    return -4;
  }
  if (!make_tmap(&tmX, g.x, (uint64_t)g.R, (uint64_t)g.K, (uint64_t)g.x_pitch, (uint32_t)(p.two_sm ? p.npad / 2 : p.npad))) return -4;
  // the opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of the function
  static bool smem_set[kMaxDevices] = {};
  const int dev = device_slot();
  if (dev < 0) return -4;
  if (!smem_set[dev]) {
    if (cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
      return -4;
    smem_set[dev] = true;
  }
  dim3 grid(gemm_tiles(g.N), g.splits, (g.R + 255) / 256);
  const unsigned cluster_y = (g.epi == EPI_RESIDUAL) ? (unsigned)g.splits : 1u;
  const cudaError_t le = p.two_sm
      ? launch_pdl_cluster_xy(gemm_tc_kernel<true>, grid, dim3(kTcThreads), (size_t)smem, st, 2u, cluster_y, tmW, tmX, p)
      : launch_pdl_cluster_xy(gemm_tc_kernel<false>, grid, dim3(kTcThreads), (size_t)smem, st, 1u, cluster_y, tmW, tmX, p);
  if (le != cudaSuccess)
    return -4;
  return 0;
}

}  // namespace ssd
