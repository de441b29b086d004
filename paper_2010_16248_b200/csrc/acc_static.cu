// acc_sumsq_static: squared L2 norm of one flat buffer, with its scratch in a file-scope device array.
//
// For callers that must not allocate device memory at the time of the call and have no workspace to
// hand over: code running inside another framework's memory budget, a plugin that only receives
// tensors, a latency-critical loop in which cudaMalloc's implicit device synchronisation is not
// acceptable.  The two-stage reduction is the one acc_layer_norms uses (fixed-order fp64 partial
// per 8192-element tile, then a fixed-order sum of the partials), but the partials live in the
// array below instead of a caller-provided workspace.
#include <mutex>

#include "acc_internal.cuh"

namespace acc {

constexpr int kStaticMaxTiles = ACC_STATIC_NORM_MAX_ELEMS / kTile;  // 32768 partials = 256 KB per GPU

// Held by every GPU that loads the library, until the process exits.  In host code this name is only
// a stand-in for the symbol: the device address comes from cudaGetSymbolAddress (static_scratch()).
static __device__ __align__(256) double g_static_partials[kStaticMaxTiles];

constexpr int kMaxDevices = 64;
static double* g_scratch_ptr[kMaxDevices] = {nullptr};
static std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device; resolved once per device.
static cudaError_t static_scratch(double** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    double* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_partials);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

// One block per 8192-element tile: fp64 sum of squares in a fixed order.
__global__ void __launch_bounds__(256)
static_sumsq_partial_kernel(const float* __restrict__ x, long long n, double* __restrict__ part) {
  __shared__ double sm[8];
  const long long e0 = (long long)blockIdx.x * kTile;
  const int nelem = (int)(n - e0 < kTile ? n - e0 : kTile);
  const float* p = x + e0;
  double acc = 0.0;
  const int n4 = nelem >> 2;
  for (int i = threadIdx.x; i < n4; i += blockDim.x) {
    const float4 v = ld_stream4(p + 4 * i);
    acc += (double)v.x * v.x;
    acc += (double)v.y * v.y;
    acc += (double)v.z * v.z;
    acc += (double)v.w * v.w;
  }
  for (int i = 4 * n4 + threadIdx.x; i < nelem; i += blockDim.x) acc += (double)p[i] * p[i];
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int i = 0; i < 8; ++i) s += sm[i];
    part[blockIdx.x] = s;
  }
}

// One warp: sums the first n_tiles partials in a fixed order.
__global__ void static_sumsq_final_kernel(const double* __restrict__ part, int n_tiles, double* __restrict__ out) {
  double acc = 0.0;
  for (int i = threadIdx.x; i < n_tiles; i += 32) acc += part[i];
  acc = warp_sum(acc);
  if (threadIdx.x == 0) *out = acc;
}

}  // namespace acc

extern "C" int acc_sumsq_static(const float* buf, int64_t n, double* norm2, void* stream) {
  using namespace acc;
  if (!buf || !norm2 || n < 1) return ACC_EINVAL;
  if (n > (int64_t)ACC_STATIC_NORM_MAX_ELEMS) return ACC_ETOOBIG;
  if ((reinterpret_cast<uintptr_t>(buf) & 15u) || (reinterpret_cast<uintptr_t>(norm2) & 7u)) return ACC_EALIGN;
  double* scratch = nullptr;
  if (static_scratch(&scratch) != cudaSuccess) return ACC_ECUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int n_tiles = (int)((n + kTile - 1) / kTile);
  // every partial that the second kernel reads is written by the first: nothing has to start at zero
  static_sumsq_partial_kernel<<<n_tiles, 256, 0, s>>>(buf, n, scratch);
  static_sumsq_final_kernel<<<1, 32, 0, s>>>(scratch, n_tiles, norm2);
  return cudaGetLastError() == cudaSuccess ? ACC_OK : ACC_ECUDA;
}
