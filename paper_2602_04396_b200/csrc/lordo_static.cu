// Clip coefficient of one gradient array with all scratch in a static device array: the one entry
// point of the library that needs neither a context nor a caller-provided workspace, for callers
// that are not in a position to allocate device memory (see lordo_clip_coefficient_static in lordo.h).
#include <mutex>

#include "lordo_common.cuh"

namespace lordo {
namespace {

constexpr long long kStaticChunk = 32768;  // elements per partial sum
constexpr int kStaticMaxChunks = 16384;    // 128 KiB of partial sums per device
constexpr int kMaxDevices = 64;

// Partial sums of squares of the call in flight. Lives in every device that loads the library.
static __device__ __align__(256) double g_static_partials[kStaticMaxChunks];

__global__ void __launch_bounds__(256) static_sumsq_kernel(const void* __restrict__ g, int dt, long long count,
                                                          double* __restrict__ partial) {
  const long long begin = (long long)blockIdx.x * kStaticChunk;
  long long end = begin + kStaticChunk;
  if (end > count) end = count;
  float acc = 0.f;
  for (long long e = begin + 4ll * threadIdx.x; e < end; e += 4ll * 256) {  // count is a multiple of 8
    const float4 x = load4(g, dt, e);
    acc += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
  }
  double d = (double)acc;
  for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
  __shared__ double warp_sum[8];
  if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = d;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < 8; ++w) s += warp_sum[w];
    partial[blockIdx.x] = s;  // every slot a call reads was written by that call: nothing to clear
  }
}

__global__ void __launch_bounds__(256) static_finalize_kernel(const double* __restrict__ partial, int chunks, float rho,
                                                             float* __restrict__ coef) {
  __shared__ double red[256];
  double a = 0.0;
  for (int c = threadIdx.x; c < chunks; c += 256) a += partial[c];
  red[threadIdx.x] = a;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    // a NaN or infinite sum of squares has no coefficient: report NaN instead of fminf's silent 1
    const double ss = red[0];
    const bool finite = ss == ss && ss < 1.7e308;
    coef[0] = !finite ? __int_as_float(0x7fc00000) : (rho > 0.f ? fminf(1.f, rho / ((float)sqrt(ss) + 1e-6f)) : 1.f);
  }
}

std::mutex g_setup_mutex;
double* g_partials_addr[kMaxDevices] = {nullptr};

// Device address of the static array on the current device, looked up once per device.
// (In host code the array's name is only a handle for this lookup, never a device pointer.)
// The address is cached for the life of the process: it does not survive a cudaDeviceReset.
int static_scratch(double** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LORDO_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_partials_addr[dev]) {
    double* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_partials) != cudaSuccess || !p) {
      cudaGetLastError();
      return LORDO_ERR_CUDA;
    }
    g_partials_addr[dev] = p;
  }
  *out = g_partials_addr[dev];
  return LORDO_OK;
}

}  // namespace
}  // namespace lordo

extern "C" {

int64_t lordo_clip_coefficient_static_max_count(void) { return (int64_t)lordo::kStaticMaxChunks * lordo::kStaticChunk; }

int lordo_clip_coefficient_static(const void* G_dev, int g_dtype, int64_t count, float rho, float* coef_out_dev, void* stream) {
  using namespace lordo;
  if (!G_dev || !coef_out_dev || count < 8 || (count & 7) != 0) return LORDO_ERR_INVALID_ARG;
  if (g_dtype != LORDO_F32 && g_dtype != LORDO_BF16) return LORDO_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(G_dev) & 15u) != 0) return LORDO_ERR_ALIGN;
  if (count > lordo_clip_coefficient_static_max_count()) return LORDO_ERR_UNSUPPORTED;  // beyond the static scratch
  double* partial = nullptr;
  const int rc = static_scratch(&partial);
  if (rc != LORDO_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int chunks = (int)((count + kStaticChunk - 1) / kStaticChunk);
  if (cudaPeekAtLastError() != cudaSuccess) return LORDO_ERR_CUDA;  // an earlier, unrelated error: not reported as this call's
  static_sumsq_kernel<<<chunks, 256, 0, st>>>(G_dev, g_dtype, count, partial);
  static_finalize_kernel<<<1, 256, 0, st>>>(partial, chunks, rho, coef_out_dev);
  return cudaPeekAtLastError() == cudaSuccess ? LORDO_OK : LORDO_ERR_CUDA;
}

}  // extern "C"
