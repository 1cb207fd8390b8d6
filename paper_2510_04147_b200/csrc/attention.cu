// Bidirectional attention of the cache-fill forward (prefill of the prompt, and any forward whose
// rows were first written to the KV cache by the rotary pass): every query row attends, without a
// causal mask, to the cached keys of its sequence, which include the rows themselves.
//
// Rows are ordered [sequence slot][node][in-block index].  The keys are cut into parts whose
// boundaries depend on the key count only; a CTA owns (64 query rows of one sequence, one head, one
// part) and streams the part's K/V tiles through shared memory once for all of those rows.  An
// optional node-local part (keys given outside the cache, masked block-diagonally) is supported
// for cross-checks.  Parts are merged in part order by a second kernel (log-sum-exp, fixed order).
// The verification forward and the block commit use attention_verify.cu instead.
//
// Tensor-core work uses warp-level mma.sync (bf16 in, fp32 accumulate): attention is < 3 % of the
// forward's flops and is bound by the K/V stream and by latency, not by the tensor pipe.
#include "attn_common.cuh"

namespace ssd {

namespace {

using namespace attn;

template <int HD>
__global__ void __launch_bounds__(kAttnThreads) attn_split_kernel(AttnArgs a, int n_prefix_parts, int has_local,
                                                                  float scale_log2) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  bf16* sQ = reinterpret_cast<bf16*>(smem_raw);
  bf16* sK = sQ + kQTile * HD;
  bf16* sV = sK + 2 * kKTile * HD;
  constexpr int CH = HD / 8;   // 16-byte chunks per row

  pdl_launch_dependents();
  pdl_wait();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gq = lane >> 2, tq = lane & 3;
  const int qt = blockIdx.x, h = blockIdx.y;
  const int n_parts = n_prefix_parts + has_local;
  const int slot = blockIdx.z / n_parts, part = blockIdx.z % n_parts;
  const int kvh = h / (a.H / a.Hkv);
  const int seq = a.map.seq_map ? a.map.seq_map[slot] : a.map.seq_base + slot;
  const int rps = a.map.rows_per_seq, T = a.map.T;
  const int lr0 = qt * kQTile;                       // first sequence-local query row
  const size_t grow0 = (size_t)slot * rps + lr0;     // first global row
  const bool local = has_local && part == n_prefix_parts;

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

  const bf16* kbase;
  const bf16* vbase;
  size_t krow_stride = (size_t)a.Hkv * HD;
  if (!local) {
    kbase = a.cache_k + (size_t)seq * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride;
    vbase = a.cache_v + (size_t)seq * a.cache_seq_stride + (size_t)kvh * a.kv_head_stride;
    krow_stride = a.kv_pos_stride;
  } else {
    kbase = a.local_k + ((size_t)slot * rps * a.Hkv + kvh) * HD;
    vbase = a.local_v + ((size_t)slot * rps * a.Hkv + kvh) * HD;
  }

  // ---- Q tile
  for (int idx = tid; idx < kQTile * CH; idx += kAttnThreads) {
    const int row = idx / CH, ch = idx % CH;
    const bool valid = (lr0 + row) < rps;
    const bf16* src = a.q + ((grow0 + (valid ? row : 0)) * a.H + h) * HD + ch * 8;
    cp_async16(sQ + swz<HD>(row, ch), src, valid);
  }
  auto load_kv = [&](int tile, int buf) {
    const int key0 = k_begin + tile * kKTile;
    bf16* dK = sK + buf * kKTile * HD;
    bf16* dV = sV + buf * kKTile * HD;
    for (int idx = tid; idx < kKTile * CH; idx += kAttnThreads) {
      const int row = idx / CH, ch = idx % CH;
      const int key = key0 + row;
      const bool valid = key < k_end;
      const size_t off = (size_t)(valid ? key : k_begin) * krow_stride + ch * 8;
      cp_async16(dK + swz<HD>(row, ch), kbase + off, valid);
      cp_async16(dV + swz<HD>(row, ch), vbase + off, valid);
    }
  };
  if (n_tiles > 0) load_kv(0, 0);
  cp_async_commit();

  float o[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};
  uint32_t qf[HD / 16][4];

  const int qrow_w = warp * 16;   // warp's first row inside the tile
  for (int tile = 0; tile < n_tiles; ++tile) {
    const int buf = tile & 1;
    if (tile + 1 < n_tiles) load_kv(tile + 1, buf ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (tile == 0) {
#pragma unroll
      for (int kk = 0; kk < HD / 16; ++kk) {
        const int row = qrow_w + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int ch = kk * 2 + (lane >> 4);
        ldmatrix_x4(qf[kk], sQ + swz<HD>(row, ch));
      }
    }
    const bf16* tK = sK + buf * kKTile * HD;
    const bf16* tV = sV + buf * kKTile * HD;
    float s[kKTile / 8][4];
#pragma unroll
    for (int j = 0; j < kKTile / 8; ++j) {
      s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
      for (int k2 = 0; k2 < HD / 32; ++k2) {
        uint32_t b[4];
        ldmatrix_x4(b, tK + swz<HD>(j * 8 + (lane & 7), k2 * 4 + (lane >> 3)));
        mma_bf16(s[j], qf[2 * k2], b[0], b[1]);
        mma_bf16(s[j], qf[2 * k2 + 1], b[2], b[3]);
      }
    }
    // ---- scale, mask, online softmax (log2 domain)
    const int key0 = k_begin + tile * kKTile;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < kKTile / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = key0 + j * 8 + 2 * tq + (e & 1);
        bool ok = key < k_end;
        if (local) {
          const int qlr = lr0 + qrow_w + gq + (e >> 1) * 8;
          ok = ok && (key / T == qlr / T);
        }
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
      corr[i] = exp2f(m_run[i] - m_use[i]);       // exp2(-inf) = 0 while nothing was seen
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
    __syncthreads();   // everyone is done with buf before it is refilled
  }
  cp_async_wait<0>();

  // ---- write the unnormalised partial
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    l_run[i] += __shfl_xor_sync(0xffffffffu, l_run[i], 1);
    l_run[i] += __shfl_xor_sync(0xffffffffu, l_run[i], 2);
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int row = qrow_w + gq + i * 8;
    if (lr0 + row >= rps) continue;
    const size_t grow = grow0 + row;
    const size_t base = ((size_t)part * a.R + grow) * a.H + h;
    if (tq == 0) a.part_ml[base] = make_float2(m_run[i], l_run[i]);
    float* dst = a.part_o + base * HD;
#pragma unroll
    for (int nb = 0; nb < HD / 8; ++nb)
      *reinterpret_cast<float2*>(dst + nb * 8 + 2 * tq) = make_float2(o[nb][2 * i], o[nb][2 * i + 1]);
  }
}

// One CTA per (row, group of heads): 256 threads, two output elements each.  Parts are merged in
// part order with weights 2^(m_p - M).
__global__ void __launch_bounds__(256) attn_merge_kernel(const float* part_o, const float2* part_ml, bf16* out, int R,
                                                         int H, int hd, int n_parts) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  const int width = H * hd;
  const int e = (blockIdx.y * 256 + threadIdx.x) * 2;
  if (e >= width) return;
  const int h = e / hd;
  float M = -INFINITY;
  for (int p = 0; p < n_parts; ++p) M = fmaxf(M, part_ml[((size_t)p * R + r) * H + h].x);
  float L = 0.f, ax = 0.f, ay = 0.f;
  for (int p = 0; p < n_parts; ++p) {
    const float2 ml = part_ml[((size_t)p * R + r) * H + h];
    if (ml.x == -INFINITY) continue;
    const float w = exp2f(ml.x - M);
    const float2 v = *reinterpret_cast<const float2*>(part_o + ((size_t)p * R + r) * width + e);
    L += ml.y * w;
    ax += v.x * w;
    ay += v.y * w;
  }
  const float inv = 1.f / L;
  *reinterpret_cast<__nv_bfloat162*>(out + (size_t)r * width + e) = __floats2bfloat162_rn(ax * inv, ay * inv);
}

}  // namespace

void launch_attention(cudaStream_t st, const AttnArgs& a, int* launches) {
  const int n_prefix = (a.S + a.kv_split - 1) / a.kv_split;
  const int has_local = a.local_k != nullptr ? 1 : 0;
  const int n_parts = n_prefix + has_local;
  const float scale_log2 = (1.0f / sqrtf((float)a.hd)) * 1.4426950408889634f;
  const int q_tiles = (a.map.rows_per_seq + kQTile - 1) / kQTile;
  dim3 grid(q_tiles, a.H, a.n_seq_slots * n_parts);
  if (a.hd == 128) {
    const int smem = (kQTile + 4 * kKTile) * 128 * 2;
    static bool attr_set[kMaxDevices] = {};      // the shared-memory opt-in is per device
    const int dev = device_slot();
    if (dev >= 0 && !attr_set[dev]) {
      cudaFuncSetAttribute(attn_split_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      attr_set[dev] = true;
    }
    launch_pdl(attn_split_kernel<128>, grid, dim3(kAttnThreads), (size_t)smem, st, a, n_prefix, has_local, scale_log2);
  } else {
    const int smem = (kQTile + 4 * kKTile) * 64 * 2;
    launch_pdl(attn_split_kernel<64>, grid, dim3(kAttnThreads), (size_t)smem, st, a, n_prefix, has_local, scale_log2);
  }
  dim3 mgrid(a.R, (a.H * a.hd / 2 + 255) / 256);
  launch_pdl(attn_merge_kernel, mgrid, dim3(256), 0, st, (const float*)a.part_o, (const float2*)a.part_ml, a.out, a.R,
             a.H, a.hd, n_parts);
  if (launches) *launches += 2;
}

}  // namespace ssd
