// Response projections on the sm_100a tensor cores (bf16 tensors, d = 128):
//   phi_K = K F_K (Eq. 6),  phi_Q = RMS-normalised Q F_Q (Eq. 7).
// X is bf16 and enters the MMA unchanged; the float32 feature map F is split into three bf16
// terms (F = F1 + F2 + F3 up to 2^-24), so the three accumulated products reproduce the float32
// projection.  The pass is bandwidth bound: X is read once by TMA, phi written once.
// Persistent CTAs own contiguous row tiles of one head; F^T (3 x [64 x 128] bf16) stays in
// shared memory.  Roles: warps 0-3 epilogue (one row per thread: normalisation, store, max |phi|),
// warp 4 (one lane) TMA loads and tcgen05.mma, TMEM owner.  Two X stages and two accumulators
// let the loads, the MMAs and the epilogue of consecutive tiles overlap.
// Every mbarrier wait is bounded; on expiry the CTA records SPARSEPR_ERR_TIMEOUT and leaves.
#include <cuda.h>
#include <algorithm>
#include "kernels.cuh"
#include "tc_common.cuh"

namespace spr {
namespace tc {

constexpr int kPjThreads = 160;
constexpr uint32_t kPjXHalf = 128 * 128;            // [128 rows x 64 bf16]
constexpr uint32_t kPjXBytes = 2 * kPjXHalf;
constexpr uint32_t kPjFHalf = 64 * 128;             // [64 rows x 64 bf16]
constexpr uint32_t kPjFBytes = 2 * kPjFHalf;
struct PjSmem {
  static constexpr uint32_t x = 0;                              // 2 stages
  static constexpr uint32_t f = x + 2 * kPjXBytes;              // 3 terms
  static constexpr uint32_t bars = f + 3 * kPjFBytes;           // F_FULL, X_FULL[2], X_EMPTY[2], ACC_FULL[2], ACC_EMPTY[2]
  static constexpr uint32_t misc = bars + 16 * 8;
  static constexpr uint32_t total = misc + 16;
};
enum PjBar { PF_FULL = 0, PX_FULL = 1, PX_EMPTY = 3, PACC_FULL = 5, PACC_EMPTY = 7 };

struct PjParams {
  int H, N, r, ldphi, ctas_per_head, rms;
  float eps;
  float* phi;
  unsigned* maxabs_bits;
  int* err;
};

__global__ void __launch_bounds__(kPjThreads)
k_project_tc(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapF, PjParams prm) {
  pdl_wait();                                                   // the split feature map comes from the kernel before
  pdl_launch_dependents();
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  volatile int* misc = reinterpret_cast<volatile int*>(smem_raw + PjSmem::misc);   // [0] tmem base, [1] abort, [2] skip
  const uint32_t bars = base + PjSmem::bars;
  auto bar = [&](int i) { return bars + 8u * i; };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y, b = bh / prm.H, h = bh % prm.H;
  const int row_tiles = (prm.N + 127) / 128;
  const int per_cta = (row_tiles + prm.ctas_per_head - 1) / prm.ctas_per_head;
  const int tile0 = blockIdx.x * per_cta;
  const int my_tiles = max(0, min(per_cta, row_tiles - tile0));
  if (tid == 0) {
    misc[2] = (prm.err != nullptr && *reinterpret_cast<volatile int*>(prm.err) == SPARSEPR_ERR_TIMEOUT) || (base & 1023u) != 0;
    if ((base & 1023u) != 0) set_error(prm.err, SPARSEPR_ERR_CUDA);
    for (int i = 0; i < 9; ++i) mbar_init(bar(i), (i == PACC_EMPTY || i == PACC_EMPTY + 1) ? 128 : 1);
    misc[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (misc[2] || my_tiles == 0) return;
  if (warp == 4) tmem_alloc(base + PjSmem::misc, 128);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = (uint32_t)misc[0];
  volatile int* abort_flag = &misc[1];

  if (warp == 4) {
    if (lane == 0) {
      auto load_x = [&](int t) {
        const int s = t & 1;
        const int row0 = (tile0 + t) * 128;
        mbar_expect_tx(bar(PX_FULL + s), kPjXBytes);
        tma_load_4d(base + PjSmem::x + s * kPjXBytes, &mapX, bar(PX_FULL + s), 0, row0, h, b);
        tma_load_4d(base + PjSmem::x + s * kPjXBytes + kPjXHalf, &mapX, bar(PX_FULL + s), 64, row0, h, b);
      };
      mbar_expect_tx(bar(PF_FULL), 3 * kPjFBytes);
#pragma unroll
      for (int t = 0; t < 3; ++t) {
        tma_load_4d(base + PjSmem::f + t * kPjFBytes, &mapF, bar(PF_FULL), 0, 0, t, bh);
        tma_load_4d(base + PjSmem::f + t * kPjFBytes + kPjFHalf, &mapF, bar(PF_FULL), 64, 0, t, bh);
      }
      load_x(0);
      bool ok = mbar_wait(bar(PF_FULL), 0, abort_flag);
      const uint32_t idesc = idesc_bf16(0, 64);
      for (int t = 0; t < my_tiles && ok; ++t) {
        const int s = t & 1;
        if (t + 1 < my_tiles) {
          // stage (t+1)&1 was last read by the MMAs of tile t-1
          if (t >= 1 && !mbar_wait(bar(PX_EMPTY + ((t + 1) & 1)), ((t - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
          load_x(t + 1);
        }
        if (!mbar_wait(bar(PX_FULL + s), (t >> 1) & 1, abort_flag)) { ok = false; break; }
        if (t >= 2 && !mbar_wait(bar(PACC_EMPTY + s), ((t - 2) >> 1) & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint64_t xd = smem_desc(base + PjSmem::x + s * kPjXBytes, 16);
        const uint32_t d = tmem + (uint32_t)s * 64u;
#pragma unroll
        for (int term = 0; term < 3; ++term) {
          const uint64_t fd = smem_desc(base + PjSmem::f + term * kPjFBytes, 16);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t xoff = (uint64_t)((kk >> 2) * (kPjXHalf >> 4) + (kk & 3) * 2);
            const uint64_t foff = (uint64_t)((kk >> 2) * (kPjFHalf >> 4) + (kk & 3) * 2);
            umma_bf16(d, xd + xoff, fd + foff, idesc, (term > 0 || kk > 0) ? 1u : 0u);
          }
        }
        umma_commit(bar(PX_EMPTY + s));
        umma_commit(bar(PACC_FULL + s));
      }
    }
  } else {
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    float m = 0.f;
    bool bad = false, ok = true;
    for (int t = 0; t < my_tiles; ++t) {
      const int s = t & 1;
      ok = __all_sync(0xffffffffu, ok && mbar_wait(bar(PACC_FULL + s), (t >> 1) & 1, abort_flag));
      if (!ok) continue;
      tc_fence_after();
      float v[64];
      tmem_ld32_nowait(tmem + lane_addr + s * 64, *reinterpret_cast<float(*)[32]>(&v[0]));
      tmem_ld32_nowait(tmem + lane_addr + s * 64 + 32, *reinterpret_cast<float(*)[32]>(&v[32]));
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive(bar(PACC_EMPTY + s));                       // the accumulator is in registers
      const int row = (tile0 + t) * 128 + warp * 32 + lane;
      if (prm.rms) {
        float ss = 0.f;
#pragma unroll
        for (int c = 0; c < 64; ++c) ss = fmaf(v[c], v[c], ss);    // columns r..63 are exact zeros
        const float inv = 1.f / fmaxf(sqrtf(ss / (float)prm.r), prm.eps);
#pragma unroll
        for (int c = 0; c < 64; ++c) v[c] *= inv;
      }
      if (row < prm.N) {
        float* out = prm.phi + ((i64)bh * prm.N + row) * prm.ldphi;
#pragma unroll
        for (int c = 0; c < 64; c += 4)
          if (c < prm.ldphi) *reinterpret_cast<float4*>(out + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
#pragma unroll
        for (int c = 0; c < 64; ++c) {
          m = fmaxf(m, fabsf(v[c]));
          bad |= !(fabsf(v[c]) <= 3.0e38f);
        }
      }
    }
    m = warp_max(m);
    if (lane == 0) atomicMax(prm.maxabs_bits + bh, __float_as_uint(m));
    if (bad) set_error(prm.err, SPARSEPR_ERR_NUMERIC);
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int k = 0; k < 64; ++k) __nanosleep(1000);      // let copies that may still be in flight land
    if (tid == 0) set_error(prm.err, SPARSEPR_ERR_TIMEOUT);
    __syncthreads();
  }
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem, 128);
  }
}

// F [BH][128][r] float32 -> Ft [BH][3][64][128] bf16: term t, row j (output column, zero beyond r), column k
// (f_div heads share one feature map: the query heads of a K/V head under grouped-query attention)
__global__ void k_split_feature_map(const float* __restrict__ F, int r, __nv_bfloat16* __restrict__ Ft, int f_div) {
  pdl_wait();                                                   // the feature map comes from the kernels before
  pdl_launch_dependents();
  const int bh = blockIdx.y;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < 64 * 128; e += gridDim.x * blockDim.x) {
    const int j = e / 128, k = e % 128;
    float x = j < r ? F[((i64)(bh / f_div) * 128 + k) * r + j] : 0.f;
    __nv_bfloat16* out = Ft + (i64)bh * 3 * 64 * 128 + e;
#pragma unroll
    for (int t = 0; t < 3; ++t) {
      const __nv_bfloat16 hb = __float2bfloat16_rn(x);
      out[(i64)t * 64 * 128] = hb;
      x -= __bfloat162float(hb);
    }
  }
}

}  // namespace tc

cudaError_t init_project_tc() {
  return cudaFuncSetAttribute(tc::k_project_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::PjSmem::total);
}
bool project_tc_supported(int dtype, int d, int r, const i64* xs) {
  return dtype == SPARSEPR_BF16 && d == 128 && r <= 64 && xs[2] % 8 == 0 && xs[1] % 8 == 0 && xs[0] % 8 == 0 && tc::tma_available();
}

// Ft: bf16 scratch [BH][3][64][128]
bool launch_project_tc(const void* X, const i64* xs, int BH, int H, int N, int r, const float* F, bool rms, float eps,
                       float* phi, int ldphi, unsigned* maxabs, __nv_bfloat16* Ft, int* err, cudaStream_t st, int f_div) {
  using namespace tc;
  CUtensorMap mx, mf;
  launch_pdl(tc::k_split_feature_map, dim3(8, BH), dim3(256), 0, st, F, r, Ft, f_div < 1 ? 1 : f_div);
  if (!make_map(&mx, X, 128, N, H, BH / H, xs[0], xs[1], xs[2], 128) ||
      !make_map(&mf, Ft, 128, 64, 3, BH, (i64)3 * 64 * 128, (i64)64 * 128, 128, 64))
    return false;
  PjParams p{};
  p.H = H; p.N = N; p.r = r; p.ldphi = ldphi; p.rms = rms; p.eps = eps; p.phi = phi; p.maxabs_bits = maxabs; p.err = err;
  const int row_tiles = (N + 127) / 128;
  p.ctas_per_head = std::max(1, std::min(row_tiles, (2 * sm_count()) / BH));
  launch_pdl(k_project_tc, dim3(p.ctas_per_head, BH), dim3(kPjThreads), PjSmem::total, st, mx, mf, p);
  return true;
}

}  // namespace spr
