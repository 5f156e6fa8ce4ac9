// Shared device/host helpers of the SparsePR CUDA library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "sparsepr.h"

namespace spr {

typedef long long i64;
typedef unsigned long long u64;

constexpr int kMaxGroups = 2048;     // C_k, C_q limit (shared-memory histograms)
constexpr int kMaxProbes = 1024;     // M limit
constexpr int kMaxRank = 64;         // r_K, r_Q limit
// row length of a feature buffer that holds r columns (zero padded): 16, 32, 48, 64, or 128 for the raw
// activations of the semantic partition
__host__ __device__ __forceinline__ int feature_ld(int r) { return r <= 16 ? 16 : r <= 32 ? 32 : r <= 48 ? 48 : r <= 64 ? 64 : 128; }

// ---- device error word -------------------------------------------------------
__device__ __forceinline__ void set_error(int* err, int code) {
  if (err) atomicCAS(err, 0, code);
}

// ---- element access ----------------------------------------------------------
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// 8 consecutive elements starting at p (16-byte aligned for bf16, 32 for f32 halves)
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  float4 a = *reinterpret_cast<const float4*>(p);
  float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
  uint4 u = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void store8(float* p, const float (&v)[8]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&v)[8]) {
  uint4 u;
  uint32_t* w = reinterpret_cast<uint32_t*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  *reinterpret_cast<uint4*>(p) = u;
}

// ---- deterministic row sample (Appendix B.1: "a deterministic sample") --------
__host__ __device__ __forceinline__ u64 splitmix64(u64 x) {
  u64 z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
enum { kTagQuerySample = 1, kTagKvInit = 2, kTagQInit = 3 };
// Programmatic dependent launch: a kernel launched with launch_pdl may be scheduled while the kernel before it in
// the stream still runs; pdl_wait() returns once that kernel has completed and its writes are visible, and must come
// before the first access to anything it wrote.  pdl_launch_dependents() lets the kernel behind this one be scheduled
// (its blocks wait in their own pdl_wait()), which takes the launch latency off a chain of short dependent kernels.
// Both are no-ops for a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#ifdef __CUDACC__
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

__host__ __device__ __forceinline__ u64 sample_offset(u64 seed, int tag, int bh) {
  return splitmix64(seed * 0x100000001B3ull + (u64)tag * 0x10001ull + (u64)bh) >> 40;
}
// s-th of n evenly strided rows out of N with the 24-bit offset U
__host__ __device__ __forceinline__ int strided_row(int s, int n, int N, u64 U) {
  return (int)(((((u64)s) << 24) + U) * (u64)N / (((u64)n) << 24));
}

// ---- warp / block reductions ----------------------------------------------------
template <typename T> __device__ __forceinline__ T warp_sum(T v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <typename T> __device__ __forceinline__ T warp_max(T v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { T w = __shfl_xor_sync(0xffffffffu, v, o); v = w > v ? w : v; }
  return v;
}
// block-wide sum; `scratch` holds >= 33 elements; every thread gets the result
template <typename T> __device__ __forceinline__ T block_sum(T v, T* scratch) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) scratch[w] = v;
  __syncthreads();
  if (w == 0) {
    T t = lane < nw ? scratch[lane] : T(0);
    t = warp_sum(t);
    if (lane == 0) scratch[32] = t;
  }
  __syncthreads();
  return scratch[32];
}
template <typename T> __device__ __forceinline__ T block_max(T v, T* scratch) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_max(v);
  __syncthreads();
  if (lane == 0) scratch[w] = v;
  __syncthreads();
  if (w == 0) {
    T t = scratch[lane < nw ? lane : 0];
    t = warp_max(t);
    if (lane == 0) scratch[32] = t;
  }
  __syncthreads();
  return scratch[32];
}

// exclusive prefix sum over n <= 4 * blockDim.x ints held in shared memory, in place;
// returns the total.  `scratch` >= 33 ints.
__device__ __forceinline__ int block_exclusive_scan(int* data, int n, int* scratch) {
  const int per = (n + blockDim.x - 1) / blockDim.x;
  const int lo = min((int)threadIdx.x * per, n), hi = min(lo + per, n);
  int s = 0;
  for (int i = lo; i < hi; ++i) s += data[i];
  // scan of the per-thread sums
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  int inc = s;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
  __syncthreads();
  if (lane == 31) scratch[w] = inc;
  __syncthreads();
  if (w == 0) {
    int t = lane < nw ? scratch[lane] : 0;
    int ti = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int u = __shfl_up_sync(0xffffffffu, ti, o); if (lane >= o) ti += u; }
    scratch[lane] = ti - t;
    if (lane == 31) scratch[32] = ti;
  }
  __syncthreads();
  int run = scratch[w] + inc - s;
  for (int i = lo; i < hi; ++i) { int t = data[i]; data[i] = run; run += t; }
  __syncthreads();
  return scratch[32];
}

}  // namespace spr
