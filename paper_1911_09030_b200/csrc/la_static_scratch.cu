// la_replica_means_static: the replica average of the synchronisation step, for callers that
// must not allocate device memory.
//
// The by-worker synchronisation keeps its intermediate sums in an exchange buffer that
// la_comm_create obtains with cudaMalloc.  Some users of this library cannot do that: a process
// that handed the whole device to its own allocator at start-up (the caller-arena mode of
// la_create_ex exists for exactly those), or a service that bans cudaMalloc/cudaFree after
// initialisation because both synchronise the device.  For them this file keeps the
// intermediate sums in a fixed array that is part of the library image.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/local_adaalter.h"
#include "la_sweep.cuh"

namespace {

constexpr uint64_t kMaxCoords = LA_STATIC_SCRATCH_MAX_COORDS;  // per-replica stride limit
constexpr int kMaxDevices = 64;

// [2][kMaxCoords] floats: tree sums of x, then of B^2.  8 MiB on every GPU that loads the
// library, held until the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress; kernels receive the device address obtained from it.
static __device__ __align__(256) float g_static_sums[2 * kMaxCoords];

std::mutex g_mutex;
float* g_scratch_addr[kMaxDevices] = {};  // device address of g_static_sums, per device ordinal

__global__ void __launch_bounds__(LA_BLOCK) la_scale_sums(const float* __restrict__ sums, uint64_t sums_stride,
                                                          float* __restrict__ x_mean, float* __restrict__ b2_mean,
                                                          uint64_t n, uint32_t W) {
  const uint64_t nthreads = (uint64_t)gridDim.x * blockDim.x;
  const float w = __uint2float_rn(W);
  for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += nthreads) {
    x_mean[j] = __fdiv_rn(sums[j], w);
    b2_mean[j] = __fdiv_rn(sums[sums_stride + j], w);
  }
}

}  // namespace

extern "C" int la_replica_means_static(const float* x_dev, const float* b2_dev, uint32_t W, uint64_t n,
                                       uint64_t stride, float* x_mean_dev, float* b2_mean_dev, void* stream) {
  if (!x_dev || !b2_dev || !x_mean_dev || !b2_mean_dev) return LA_EINVAL;
  if (W == 0 || W > LA_MAX_WORKERS || n == 0 || stride < n || stride % 4 != 0) return LA_EINVAL;
  if (stride > kMaxCoords) return LA_ETOOBIG;  // the fixed scratch holds 2 * LA_STATIC_SCRATCH_MAX_COORDS floats
  if ((reinterpret_cast<uintptr_t>(x_dev) | reinterpret_cast<uintptr_t>(b2_dev)) & 15u) return LA_EINVAL;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LA_ECUDA;
  float* scratch = nullptr;
  {
    // once per device, with that device current: resolve the array's device address
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
      // With lazy module loading (CUDA's default) this is also the moment the driver reserves the
      // array's 8 MiB on this device.  On failure nothing is cached, so a later call tries again.
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_sums) != cudaSuccess || !p) {
        cudaGetLastError();  // clear the error so that it does not surface in the caller's next CUDA call
        return LA_ECUDA;
      }
      g_scratch_addr[dev] = static_cast<float*>(p);
    }
    scratch = g_scratch_addr[dev];
  }

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the export pass of the by-worker synchronisation: tree sums over the replicas -> scratch
  const la::SweepKernel k = la::lookup_sweep((int)W, 0, la::kGradNoise, false, true, false, false, 1);
  if (!k.fn) return LA_ESTATE;
  la::SweepParams p{};
  p.X = const_cast<float*>(x_dev);  // the export pass only reads the replicas
  p.B2 = const_cast<float*>(b2_dev);
  p.xch = scratch;
  p.xch_b_off = stride;
  p.n = n; p.stride = stride;
  p.W = W; p.W_total = W;
  const unsigned block = la::kBlockThreads;
  uint64_t blocks = ((n + (uint64_t)k.vec - 1) / (uint64_t)k.vec + block - 1) / block;
  if (blocks > (1u << 20)) blocks = 1u << 20;
  k.fn<<<(unsigned)blocks, block, 0, st>>>(p);   // sums -> scratch[0..n), scratch[stride..stride+n)
  if (cudaGetLastError() != cudaSuccess) return LA_ECUDA;
  uint64_t blocks2 = (n + block - 1) / block;
  if (blocks2 > (1u << 20)) blocks2 = 1u << 20;
  la_scale_sums<<<(unsigned)blocks2, block, 0, st>>>(scratch, stride, x_mean_dev, b2_mean_dev, n, W);
  if (cudaGetLastError() != cudaSuccess) return LA_ECUDA;
  return LA_OK;
}
