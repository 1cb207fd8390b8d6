// ssd_gemm_bf16_noalloc: the skinny projection GEMM for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc while they run: a serving process that gave the
// whole device to its own memory arena at start-up has nothing left for the driver to hand out, and a
// latency-critical loop cannot afford a call that may block on the device or fail for lack of memory.
// For them the split-K scratch of the projection kernel lives in a fixed array that is part of the
// library image: every GPU that loads the library holds these 4 MiB until the process exits.
//
// The array's name is a device symbol.  In host code the name stands for a host-side shadow, not for
// device memory, so the host never passes it to a kernel: once per device, with that device current,
// it asks the runtime for the real address (cudaGetSymbolAddress) and passes that pointer on.
#include "../../include/ssd.h"
#include "kernels.h"

#include <mutex>

namespace {

constexpr size_t kScratchFloats = (size_t)1 << 20;   // 4 MiB in total
constexpr size_t kFlagFloats = 64;                   // first 256 bytes: the kernel's error word
constexpr size_t kPartialFloats = kScratchFloats - kFlagFloats;
constexpr int kMaxDevices = 64;

static __device__ __align__(256) float g_noalloc_scratch[kScratchFloats];

std::mutex g_setup_mutex;
float* g_scratch_addr[kMaxDevices] = {};

__global__ void noalloc_sum_kernel(const float* partial, int splits, size_t stride, float* out, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float v = 0.f;
  for (int s = 0; s < splits; ++s) v += partial[s * stride + i];
  out[i] = v;
}

// Device address of the scratch array on the current device; resolved on the first call per device.
int scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SSD_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    if (ssd::gemm_tc_init() != 0) return SSD_ERR_CUDA;
    float* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
    if (e != cudaSuccess || p == nullptr) return SSD_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return SSD_OK;
}

}  // namespace

extern "C" int ssd_gemm_bf16_noalloc(const void* x_dev, const void* w_dev, float* out_dev, int32_t rows, int32_t n,
                                     int32_t k, int32_t split_k, void* cuda_stream) {
  if (!x_dev || !w_dev || !out_dev) return SSD_ERR_INVALID_ARG;
  if (rows < 1 || n < 1 || k < 8 || (k % 8) || split_k < 1 || split_k > 8) return SSD_ERR_SHAPE;
  if ((size_t)split_k * (size_t)rows * (size_t)n > kPartialFloats) return SSD_ERR_OVERFLOW;
  float* scratch = nullptr;
  int rc = scratch_for_current_device(&scratch);
  if (rc != SSD_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  int* flag = reinterpret_cast<int*>(scratch);
  float* partial = scratch + kFlagFloats;
  // the array keeps the previous call's contents: the error word must start at zero
  if (cudaMemsetAsync(flag, 0, kFlagFloats * sizeof(float), st) != cudaSuccess) return SSD_ERR_CUDA;
  ssd::GemmArgs g{};
  g.x = (const bf16*)x_dev; g.w = (const bf16*)w_dev; g.R = rows; g.N = n; g.K = k; g.x_pitch = k; g.w_pitch = k;
  g.splits = split_k; g.epi = ssd::EPI_PARTIAL; g.out = partial; g.err_flag = flag;
  rc = ssd::launch_gemm_tc(st, g);
  if (rc != 0) return rc;
  const size_t total = (size_t)rows * n;
  noalloc_sum_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(partial, split_k, total, out_dev, total);
  if (cudaGetLastError() != cudaSuccess) return SSD_ERR_CUDA;
  int h_flag = 0;
  if (cudaMemcpyAsync(&h_flag, flag, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SSD_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SSD_ERR_CUDA;
  return h_flag ? SSD_ERR_TIMEOUT : SSD_OK;
}
