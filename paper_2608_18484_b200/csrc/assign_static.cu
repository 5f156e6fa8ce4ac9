// sparsepr_stage_assign_static: the k-means assignment stage for callers that cannot
// allocate device memory.  Same kernels and same result as sparsepr_stage_assign, but
// the scratch (zero-padded copies of X and mu, the centroid norms) lives in a
// file-scope device array that is part of the library image instead of a workspace
// supplied by the caller.
#include <mutex>
#include "kernels.cuh"

using namespace spr;

namespace {

constexpr int kStaticMaxRows = 16384;      // n
constexpr int kStaticMaxCentroids = 1024;  // C
// padded X [n][64] + padded mu [C][64] + ||mu||^2 [C] + max norm, each 256-byte aligned
constexpr size_t kOffMu = (size_t)kStaticMaxRows * kMaxRank * sizeof(float);
constexpr size_t kOffMu2 = kOffMu + (size_t)kStaticMaxCentroids * kMaxRank * sizeof(float);
constexpr size_t kOffMax = kOffMu2 + (size_t)kStaticMaxCentroids * sizeof(float);
constexpr size_t kStaticBytes = kOffMax + 256;

// About 4.3 MB of every GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_assign_scratch[kStaticBytes];

// In host code `g_assign_scratch` is only a handle for the runtime, not a device
// address; the address a kernel may use comes from cudaGetSymbolAddress, once per device.
constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned char* g_scratch_ptr[kMaxDevices] = {};

cudaError_t scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_assign_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

// out[i][k] = in[i][k] for k < r, 0 for r <= k < R: every element of the padded copy is
// rewritten on every call, so nothing left behind by an earlier call is ever read.
__global__ void k_pad_rows_static(const float* __restrict__ in, int n, int r, int R, float* __restrict__ out) {
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < (i64)n * R; e += (i64)gridDim.x * blockDim.x) {
    const int k = (int)(e % R);
    out[e] = k < r ? in[(e / R) * r + k] : 0.f;
  }
}

}  // namespace

extern "C" sparsepr_status_t sparsepr_stage_assign_static(int32_t n, int32_t C, int32_t r, const float* X,
                                                          const float* mu, int32_t* a, void* cuda_stream) {
  if (n < 1 || C < 1 || r < 1 || !X || !mu || !a) return SPARSEPR_ERR_INVALID_ARG;
  if (n > kStaticMaxRows || C > kStaticMaxCentroids || r > kMaxRank) return SPARSEPR_ERR_UNSUPPORTED;
  unsigned char* base = nullptr;
  if (scratch_for_current_device(&base) != cudaSuccess) return SPARSEPR_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int R = r <= 16 ? 16 : r <= 32 ? 32 : r <= 48 ? 48 : 64;
  float* Xp = reinterpret_cast<float*>(base);
  float* mup = reinterpret_cast<float*>(base + kOffMu);
  float* mu2 = reinterpret_cast<float*>(base + kOffMu2);
  float* mumax = reinterpret_cast<float*>(base + kOffMax);
  cudaGetLastError();
  k_pad_rows_static<<<(unsigned)(((i64)n * R + 255) / 256), 256, 0, st>>>(X, n, r, R, Xp);
  k_pad_rows_static<<<(unsigned)(((i64)C * R + 255) / 256), 256, 0, st>>>(mu, C, r, R, mup);
  launch_kmeans_finalize(mup, mu2, mumax, nullptr, nullptr, nullptr, 1, C, r, 0, st);   // writes ||mu||^2 and the max norm
  launch_kmeans_assign(Xp, R, 1, n, r, mup, mu2, mumax, C, a, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, st);
  return cudaGetLastError() == cudaSuccess ? SPARSEPR_OK : SPARSEPR_ERR_CUDA;
}
