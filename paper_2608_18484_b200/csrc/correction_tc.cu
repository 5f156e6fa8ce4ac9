// Residual correction of Eq. 9 as a pass of its own on the sm_100a tensor cores:
//   O <- X + X A + c     (in place, bf16, d_v = 128; A, c = composed affine map of one head)
// It runs after the block-sparse kernels, so that the probe rows and the fit (which produce A and c) can execute
// on a second stream while those kernels are busy.  The block-sparse kernels hand over the hard-drop rows X = O^sp
// as two bf16 words, X = X_h + X_l: X_h is what they stored in O, X_l the part that rounding dropped (2^-17
// relative together), so that the corrected output is rounded to bf16 once -- a one-word hand-over rounds twice,
// which shows in the largest elements.  A enters the product as two bf16 words as well, A = A_h + A_l: with few probes
// (M < d_v) and a small ridge the fitted map can have a norm of ~10, and one word of A then costs up to 0.012 of
// the 0.02 that the output may differ from the oracle (the products are X_h A_h + X_l A_h + X_h A_l; X_l A_l is
// below 2^-17 of the result).
// The pass is bandwidth bound: each 128-row tile is read once (2 x 256 B per row) and written once (256 B per row).
// A CTA takes TWO consecutive row tiles of a head (the map's 64 KB are loaded once for both, and all loads of the CTA
// are issued up front: 192 KB in flight per SM).
//   warps 0-3  one thread per row of tile 0: X A from TMEM, X from the two swizzled tiles, + c, store; warps 4-7: tile 1
//   warp  8    TMA loads (2 x (X_h, X_l), A_h^T, A_l^T), twenty-four tcgen05.mma per tile, TMEM owner
// Every mbarrier wait is bounded; on expiry the CTA records SPARSEPR_ERR_TIMEOUT and leaves.
#include <cuda.h>
#include "kernels.cuh"
#include "tc_common.cuh"

namespace spr {
namespace tc {

constexpr int kCorrThreads = 288;
constexpr int kCorrTile = 128;
constexpr uint32_t kCorrHalf = kCorrTile * 128;      // one [128 rows x 64 bf16] swizzled block
constexpr uint32_t kCorrTileBytes = 2 * kCorrHalf;
struct CorrSmem {
  static constexpr uint32_t xh = 0;                        // tile u at xh + 2 u kCorrTileBytes, its second words one tile further
  static constexpr uint32_t xl = xh + kCorrTileBytes;
  static constexpr uint32_t a = xh + 4 * kCorrTileBytes;
  static constexpr uint32_t al = a + kCorrTileBytes;
  static constexpr uint32_t bars = al + kCorrTileBytes;    // full[2], done[2]
  static constexpr uint32_t misc = bars + 32;
  static constexpr uint32_t total = misc + 16;
};
static_assert(CorrSmem::total <= 227 * 1024, "shared memory");

struct CorrParams {
  int H, N;
  const float* c;                  // [BH][128]
  __nv_bfloat16* O; i64 os[3];
  int* err;
};

__global__ void __launch_bounds__(kCorrThreads)
k_correction_tc(const __grid_constant__ CUtensorMap mapO, const __grid_constant__ CUtensorMap mapL,
                const __grid_constant__ CUtensorMap mapA, CorrParams prm) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  volatile int* misc = reinterpret_cast<volatile int*>(smem_raw + CorrSmem::misc);   // [0] tmem base, [1] abort, [2] skip
  const uint32_t bar_full = base + CorrSmem::bars, bar_done = bar_full + 16;       // [2] each
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y, b = bh / prm.H, h = bh % prm.H;
  const int n_tiles = (prm.N + kCorrTile - 1) / kCorrTile;
  const int tile0 = blockIdx.x * 2;
  const int nt = min(2, n_tiles - tile0);
  if (tid == 0) {
    misc[2] = (prm.err != nullptr && *reinterpret_cast<volatile int*>(prm.err) == SPARSEPR_ERR_TIMEOUT) || (base & 1023u) != 0;
    if ((base & 1023u) != 0) set_error(prm.err, SPARSEPR_ERR_CUDA);
    for (int i = 0; i < 2; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_done + 8 * i, 1); }
    misc[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (misc[2]) return;
  if (warp == 8) tmem_alloc(base + CorrSmem::misc, 256);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = (uint32_t)misc[0];
  volatile int* abort_flag = &misc[1];

  if (warp == 8) {
    if (lane == 0) {
      // every load of the CTA first: tile 0 with the map, then tile 1
      for (int u = 0; u < nt; ++u) {
        const uint32_t bf = bar_full + 8 * u, xb = base + CorrSmem::xh + u * 2 * kCorrTileBytes;
        const int row0 = (tile0 + u) * kCorrTile;
        mbar_expect_tx(bf, (u == 0 ? 4 : 2) * kCorrTileBytes);
        tma_load_4d(xb, &mapO, bf, 0, row0, h, b);
        tma_load_4d(xb + kCorrHalf, &mapO, bf, 64, row0, h, b);
        tma_load_4d(xb + kCorrTileBytes, &mapL, bf, 0, row0, bh, 0);
        tma_load_4d(xb + kCorrTileBytes + kCorrHalf, &mapL, bf, 64, row0, bh, 0);
        if (u == 0) {
          tma_load_4d(base + CorrSmem::a, &mapA, bf, 0, 0, bh, 0);
          tma_load_4d(base + CorrSmem::a + kCorrHalf, &mapA, bf, 64, 0, bh, 0);
          tma_load_4d(base + CorrSmem::al, &mapA, bf, 0, 0, gridDim.y + bh, 0);          // the second words follow the first ones
          tma_load_4d(base + CorrSmem::al + kCorrHalf, &mapA, bf, 64, 0, gridDim.y + bh, 0);
        }
      }
      const uint64_t ad = smem_desc(base + CorrSmem::a, 16), ald = smem_desc(base + CorrSmem::al, 16);
      const uint32_t idesc = idesc_bf16(0, 128);
      for (int u = 0; u < nt; ++u) {
        if (!mbar_wait(bar_full + 8 * u, 0, abort_flag)) break;
        tc_fence_after();
        const uint64_t hd = smem_desc(base + CorrSmem::xh + u * 2 * kCorrTileBytes, 16);
        const uint64_t ld = smem_desc(base + CorrSmem::xl + u * 2 * kCorrTileBytes, 16);
        const uint32_t d = tmem + 128u * u;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t koff = (uint64_t)((kk >> 2) * (kCorrHalf >> 4) + (kk & 3) * 2);
          umma_bf16(d, hd + koff, ad + koff, idesc, kk > 0);             // (X A)[m][n] = sum_k X[m][k] At[n][k]
        }
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t koff = (uint64_t)((kk >> 2) * (kCorrHalf >> 4) + (kk & 3) * 2);
          umma_bf16(d, ld + koff, ad + koff, idesc, 1);
        }
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t koff = (uint64_t)((kk >> 2) * (kCorrHalf >> 4) + (kk & 3) * 2);
          umma_bf16(d, hd + koff, ald + koff, idesc, 1);
        }
        umma_commit(bar_done + 8 * u);
      }
    }
  } else {
    // ---- epilogue: one thread per row; warps 0-3 take tile 0, warps 4-7 tile 1 ---------------------------------
    const int row = (warp & 3) * 32 + lane;
    const float* cv = prm.c + (i64)bh * 128;
    for (int u = warp >> 2; u < nt; u += 2) {
      const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_done + 8 * u, 0, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const int row0 = (tile0 + u) * kCorrTile;
      __nv_bfloat16* op = prm.O + b * prm.os[0] + h * prm.os[1] + (i64)(row0 + row) * prm.os[2];
      const unsigned char* hrow = smem_raw + CorrSmem::xh + u * 2 * kCorrTileBytes + row * 128;
      const unsigned char* lrow = smem_raw + CorrSmem::xl + u * 2 * kCorrTileBytes + row * 128;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float t[32];
        tmem_ld32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + 128u * u + q * 32, t);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          const int j = (q & 1) * 4 + ch;                                // 16-byte chunk of the 128-byte row
          const uint32_t so = (q >> 1) * kCorrHalf + ((j ^ (row & 7)) << 4);
          const uint4 rh = *reinterpret_cast<const uint4*>(hrow + so);
          const uint4 rl = *reinterpret_cast<const uint4*>(lrow + so);
          const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&rh);
          const __nv_bfloat162* lp = reinterpret_cast<const __nv_bfloat162*>(&rl);
          float v8[8];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float2 fh = __bfloat1622float2(hp[k]), fl = __bfloat1622float2(lp[k]);
            const int col = q * 32 + ch * 8 + 2 * k;
            v8[2 * k] = (fh.x + fl.x) + t[ch * 8 + 2 * k] + cv[col];
            v8[2 * k + 1] = (fh.y + fl.y) + t[ch * 8 + 2 * k + 1] + cv[col + 1];
          }
          if (row0 + row < prm.N) store8(op + q * 32 + ch * 8, v8);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int k = 0; k < 64; ++k) __nanosleep(1000);      // let copies that may still be in flight land
    if (tid == 0) set_error(prm.err, SPARSEPR_ERR_TIMEOUT);
    __syncthreads();
  }
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

// A [BH][128][128] float32 (row k, column n) -> At [2][BH][n][k] bf16: first words, then what their rounding dropped
__global__ void k_transpose_correction(const float* __restrict__ A, __nv_bfloat16* __restrict__ At) {
  __shared__ float tile[32][33];
  const int bh = blockIdx.z;
  const float* a = A + (i64)bh * 128 * 128;
  __nv_bfloat16* t = At + (i64)bh * 128 * 128;
  const int k0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  for (int r = threadIdx.y; r < 32; r += 8) tile[r][threadIdx.x] = a[(k0 + r) * 128 + n0 + threadIdx.x];
  __syncthreads();
  __nv_bfloat16* tl = At + ((i64)gridDim.z + bh) * 128 * 128;
  for (int r = threadIdx.y; r < 32; r += 8) {
    const float x = tile[threadIdx.x][r];
    const __nv_bfloat16 hb = __float2bfloat16_rn(x);
    t[(n0 + r) * 128 + k0 + threadIdx.x] = hb;
    tl[(n0 + r) * 128 + k0 + threadIdx.x] = __float2bfloat16_rn(x - __bfloat162float(hb));
  }
}

// Self-test of the bounded wait: one warp waits on an mbarrier that nobody arrives at (no copy in flight, no
// tensor memory held), with a limit of 2^16 cycles; the wait gives up, the error word receives
// SPARSEPR_ERR_TIMEOUT, the kernel returns normally and the context stays usable.
__global__ void k_selftest_bounded_wait(int* err, long long limit) {
  __shared__ __align__(8) unsigned long long sbar;
  __shared__ int abort_flag;
  const uint32_t bar = smem_u32(&sbar);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool ok = mbar_wait_limit(bar, 0, &abort_flag, limit);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || abort_flag)) set_error(err, SPARSEPR_ERR_TIMEOUT);
}

}  // namespace tc

void launch_selftest_bounded_wait(int* err, cudaStream_t st) { tc::k_selftest_bounded_wait<<<1, 32, 0, st>>>(err, 1ll << 16); }

cudaError_t init_correction_tc() {
  return cudaFuncSetAttribute(tc::k_correction_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::CorrSmem::total);
}

bool launch_correction_tc(const float* A, const float* c, __nv_bfloat16* At, const void* O_lo, void* O, const i64* os, int BH,
                          int H, int N, int* err, cudaStream_t st) {
  using namespace tc;
  CUtensorMap mo, ml, ma;
  k_transpose_correction<<<dim3(4, 4, BH), dim3(32, 8), 0, st>>>(A, At);
  if (!make_map(&mo, O, 128, N, H, BH / H, os[0], os[1], os[2], kCorrTile) ||
      !make_map(&ml, O_lo, 128, N, BH, 1, 0, (i64)N * 128, 128, kCorrTile) ||
      !make_map(&ma, At, 128, 128, 2 * BH, 1, 0, (i64)128 * 128, 128, kCorrTile))
    return false;
  CorrParams p{};
  p.H = H; p.N = N; p.c = c; p.O = (__nv_bfloat16*)O; p.err = err;
  for (int i = 0; i < 3; ++i) p.os[i] = os[i];
  k_correction_tc<<<dim3(((N + kCorrTile - 1) / kCorrTile + 1) / 2, BH), kCorrThreads, CorrSmem::total, st>>>(mo, ml, ma, p);
  return true;
}

}  // namespace spr
