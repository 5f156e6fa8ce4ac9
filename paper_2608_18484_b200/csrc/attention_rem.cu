// Block-sparse attention (Eq. 3) for the short remainder of a query group: at most 64 query rows
// that are left after the group's full 128-row tiles (bf16, d = d_v = 128).
//
// A 128-row tile would spend a full tile of tensor and softmax work on a handful of rows.  Here the
// product is transposed, so that the cost follows the number of rows nq (rounded up to 16):
//   S^T [128 keys x nq] = K_i Q^T        tcgen05.mma, M = 128 keys, N = nq
//   P^T                 = exp2(.)        one thread per KEY (TMEM lane); bf16 P^T goes to shared memory
//   O^T [128 d_v x nq] += V_i^T P^T      tcgen05.mma, A = V tile read M-major, B = P^T from shared memory
// Per-query statistics run across the TMEM lanes.  The reference maximum of a query moves only when some
// score of a tile exceeds it by more than 2^8; that is detected with one warp vote per query and one
// 128-thread barrier per tile.  Only then the exact tile maximum is formed (warp reduction plus a four-way
// combine through shared memory) and O^T and the partial row sums are rescaled.  The row sums are kept
// per lane and reduced once at the end.
// Roles and streaming are those of the 128-row kernel: warps 0-3 / 4-7 softmax groups on even / odd key
// tiles, warp 8 K producer (+Q, tile meta ring), warp 9 MMA issuer and TMEM owner, warp 10 V producer;
// routed K/V groups arrive as one concatenated key sequence in 16-row TMA boxes.
// Every mbarrier wait is bounded; on expiry the CTA records SPARSEPR_ERR_TIMEOUT and leaves.
#include <cuda.h>
#include <cstdio>
#include "kernels.cuh"
#include "tc_common.cuh"

namespace spr {
namespace tc {

namespace rem {

constexpr int kThreads = 352;
constexpr int kKeys = 128;             // keys per tile (TMEM lanes)
constexpr int kD = 128;
constexpr int kMaxQ = 64;              // query rows per CTA at most
constexpr int kSub = 16;
constexpr int kSubPerTile = kKeys / kSub;
constexpr uint32_t kHalfBytes = kKeys * 128;          // [128 rows x 64 bf16]
constexpr uint32_t kTileBytes = 2 * kHalfBytes;       // 32 KB
constexpr uint32_t kSubBytes = kSub * 128;
// Shared memory and barriers of the instantiation for NQ = 16 NQC query rows.  The Q tile and the two P^T
// buffers are [NQ rows x 128 bytes] x 2 halves; the bytes they do not need at small NQ go into deeper K and V
// rings, because with few rows per tile the kernel is bound by the latency of the K/V stream (bytes in flight).
template <int NQC> struct Cfg {
  static constexpr int NQ = 16 * NQC;
  static constexpr uint32_t kQHalf = NQ * 128;
  static constexpr uint32_t kQBytes = 2 * kQHalf;
  static constexpr int kStages = NQC == 1 ? 3 : 2;                  // per ring
  static constexpr uint32_t q = 0;
  static constexpr uint32_t p = q + ((kQBytes + 1023u) & ~1023u);                    // 2 groups
  static constexpr uint32_t k = p + ((2 * kQBytes + 1023u) & ~1023u);
  static constexpr uint32_t v = k + kStages * kTileBytes;
  static constexpr uint32_t ranges = v + kStages * kTileBytes;
  static constexpr uint32_t wmax = ranges + kMaxGroups * 8;        // float [2][4][64] per-warp tile maxima
  static constexpr uint32_t mref = wmax + 2 * 4 * 64 * 4;          // float [2][64] reference maximum (log2 domain)
  static constexpr uint32_t corr = mref + 2 * 64 * 4;              // float [2][64] rescale factor of the current tile
  static constexpr uint32_t lsum = corr + 2 * 64 * 4;              // float [2][4][64] per-warp row sums (end)
  static constexpr uint32_t fin = lsum + 2 * 4 * 64 * 4;           // float [2][64] final weights of the two groups
  static constexpr uint32_t gmask = fin + 3 * 64 * 4;              // unsigned [2][4][2] per-warp masks of queries whose maximum grew
  static constexpr uint32_t meta = gmask + 64;                     // uint2[8]
  static constexpr uint32_t bars = meta + 8 * 8;
  static constexpr uint32_t misc = bars + 32 * 8;                  // tmem base, abort, boxes, skip, moved[2]
  static constexpr uint32_t total = misc + 64;
  enum { Q_FULL = 0, K_FULL = 1, K_EMPTY = K_FULL + kStages, V_FULL = K_EMPTY + kStages, V_EMPTY = V_FULL + kStages,
         S_FULL = V_EMPTY + kStages, P_FULL = S_FULL + 2, P_EMPTY = P_FULL + 2, O_DONE = P_EMPTY + 2, META_FULL,
         kNumBars = META_FULL + 8 };
  static_assert(kNumBars <= 32, "barrier area");
  static_assert(total <= 227 * 1024, "shared memory");
};

struct Params {
  int BH, N, Cq, Ck;
  float scale_log2;
  const int *q_off, *kv_off, *route_ptr, *route_idx, *q_perm;
  __nv_bfloat16* O; i64 os[3]; int H;
  float* O_sparse;
  int* err;
};

// instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = n; a_mn / b_mn = 1 when the operand is stored
// with its M / N index contiguous
__device__ __forceinline__ constexpr uint32_t idesc(int a_mn, int b_mn, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) | (((uint32_t)n >> 3) << 17) |
         ((128u >> 4) << 24);
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                 "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
  uint32_t w[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) w[i] = __float_as_uint(v[i]);
  tmem_st16u(taddr, w);
}
// order-preserving map float -> int (for finite values and infinities), so that an integer warp
// reduction gives the float maximum
__device__ __forceinline__ int ord(float x) { const int i = __float_as_int(x); return i ^ ((i >> 31) & 0x7fffffff); }
__device__ __forceinline__ float unord(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

// NQC = query rows / 16 (1..4)
template <int NQC>
__global__ void __launch_bounds__(kThreads, 1)
k_attention_rem(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                const __grid_constant__ CUtensorMap mapV, Params prm) {
  using Smem = Cfg<NQC>;
  using C = Cfg<NQC>;
  constexpr int NQ = C::NQ;
  constexpr int kStages = C::kStages;
  constexpr uint32_t kQHalf = C::kQHalf, kQBytes = C::kQBytes;
  constexpr int Q_FULL = C::Q_FULL, K_FULL = C::K_FULL, K_EMPTY = C::K_EMPTY, V_FULL = C::V_FULL, V_EMPTY = C::V_EMPTY, S_FULL = C::S_FULL,
                P_FULL = C::P_FULL, P_EMPTY = C::P_EMPTY, O_DONE = C::O_DONE, META_FULL = C::META_FULL, kNumBars = C::kNumBars;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char* sm = smem_raw;
  int2* ranges = reinterpret_cast<int2*>(sm + Smem::ranges);
  float* wmax = reinterpret_cast<float*>(sm + Smem::wmax);
  float* mref = reinterpret_cast<float*>(sm + Smem::mref);
  float* corr = reinterpret_cast<float*>(sm + Smem::corr);
  float* lsum = reinterpret_cast<float*>(sm + Smem::lsum);
  float* fin = reinterpret_cast<float*>(sm + Smem::fin);
  uint2* meta = reinterpret_cast<uint2*>(sm + Smem::meta);
  volatile int* misc = reinterpret_cast<volatile int*>(sm + Smem::misc);   // [0] tmem, [1] abort, [2] boxes, [3] skip, [4..5] moved
  const uint32_t bars = base + Smem::bars;
  auto bar = [&](int i) { return bars + 8u * i; };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y, g_q = blockIdx.x;

  // ---- which rows: the remainder of query group g_q, if it has 1..64 rows and this instantiation's size ----
  const int* qoff = prm.q_off + (i64)bh * (prm.Cq + 1);
  const int gsize = qoff[g_q + 1] - qoff[g_q];
  const int nq = gsize % 128;
  if (nq == 0 || nq > kMaxQ || (nq + 15) / 16 != NQC) return;
  const int row0 = qoff[g_q + 1] - nq;
  if (tid == 0) {
    misc[3] = (prm.err != nullptr && *reinterpret_cast<volatile int*>(prm.err) == SPARSEPR_ERR_TIMEOUT) || (base & 1023u) != 0;
    if ((base & 1023u) != 0) set_error(prm.err, SPARSEPR_ERR_CUDA);
  }
  __syncthreads();
  if (misc[3]) return;
  const int* rp = prm.route_ptr + (i64)bh * (prm.Cq + 1);
  const int* ridx = prm.route_idx + (i64)bh * prm.Cq * prm.Ck + rp[g_q];
  const int nroute = rp[g_q + 1] - rp[g_q];
  const int* kvoff = prm.kv_off + (i64)bh * (prm.Ck + 1);

  if (tid == 0) {
    for (int i = 0; i < kNumBars; ++i) mbar_init(bar(i), (i == P_FULL || i == P_FULL + 1) ? 128 : 1);
    misc[1] = 0; misc[2] = 0; misc[4] = 0; misc[5] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) tmem_alloc(base + Smem::misc, 256);
  __syncthreads();
  {
    int boxes = 0;
    for (int t = tid; t < nroute; t += kThreads) {
      const int g = ridx[t];
      const int start = kvoff[g], len = kvoff[g + 1] - start;
      ranges[t] = make_int2(start, len);
      boxes += (len + kSub - 1) / kSub;
    }
    boxes = warp_sum(boxes);
    if (lane == 0 && boxes) atomicAdd((int*)&misc[2], boxes);
    if (tid < 2 * 64) { mref[tid] = -INFINITY; corr[tid] = 1.f; }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = (uint32_t)misc[0];
  const int total_boxes = misc[2];
  const int n_tiles = (total_boxes + kSubPerTile - 1) / kSubPerTile;
  volatile int* abort_flag = &misc[1];
  // TMEM columns: S_A [0,64), S_B [64,128), O_A [128,192), O_B [192,256)

  if (warp == 8 || warp == 10) {
    // =========================== TMA producers (as in the 128-row kernel) ================================
    if (n_tiles > 0) {
      const bool is_k = warp == 8;
      if (is_k && lane == 0) {
        mbar_expect_tx(bar(Q_FULL), kQBytes);
        tma_load_4d(base + Smem::q, &mapQ, bar(Q_FULL), 0, row0, bh, 0);               // NQ-row box; rows past nq are never used
        tma_load_4d(base + Smem::q + kQHalf, &mapQ, bar(Q_FULL), 64, row0, bh, 0);
      }
      const int full0 = is_k ? K_FULL : V_FULL, empty0 = is_k ? K_EMPTY : V_EMPTY;
      const uint32_t buf0 = base + (is_k ? Smem::k : Smem::v);
      const CUtensorMap* map = is_k ? &mapK : &mapV;
      int ri = 0, off = 0;
      bool ok = true;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int s = i % kStages;
        const uint32_t ph = ((i / kStages) & 1) ^ 1;
        int my_start = 0;
        uint32_t cnt_bits = 0;
        int nsub = 0;
#pragma unroll
        for (int j = 0; j < kSubPerTile; ++j) {
          if (ri < nroute) {
            const int2 rg = ranges[ri];
            if (j == lane) my_start = rg.x + off;
            const int cnt = min(kSub, rg.y - off);
            cnt_bits |= (uint32_t)(cnt - 1) << (4 * j);
            nsub = j + 1;
            off += kSub;
            if (off >= rg.y) { ++ri; off = 0; }
          }
        }
        ok = __all_sync(0xffffffffu, mbar_wait(bar(empty0 + s), ph, abort_flag));
        if (!ok) break;
        if (lane == 0) {
          if (is_k) {
            meta[i & 7] = make_uint2(cnt_bits, (uint32_t)nsub);
            mbar_arrive(bar(META_FULL + (i & 7)));
          }
          mbar_expect_tx(bar(full0 + s), nsub * 2 * kSubBytes);
        }
        __syncwarp();
        if (lane < nsub) {
          const uint32_t dst = buf0 + s * kTileBytes + lane * kSubBytes;
          tma_load_4d(dst, map, bar(full0 + s), 0, my_start, bh, 0);
          tma_load_4d(dst + kHalfBytes, map, bar(full0 + s), 64, my_start, bh, 0);
        }
      }
    }
  } else if (warp == 9) {
    // =========================== MMA issuer ===========================================================
    if (lane == 0 && n_tiles > 0) {
      const uint32_t idesc_qk = idesc(0, 0, NQ);                  // A = K tile (K-major), B = Q (K-major)
      const uint32_t idesc_pv = idesc(1, 0, NQ);                  // A = V tile read M-major (d_v contiguous), B = P^T (K-major)
      const uint64_t q_desc = smem_desc(base + Smem::q, 16);
      const uint64_t k_desc0 = smem_desc(base + Smem::k, 16);
      const uint64_t v_desc0 = smem_desc(base + Smem::v, kHalfBytes);
      bool ok = mbar_wait(bar(Q_FULL), 0, abort_flag);
      auto issue_qk = [&](int i) -> bool {
        const int s = i % kStages;
        if (!mbar_wait(bar(K_FULL + s), (i / kStages) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint32_t d = tmem + (uint32_t)(i & 1) * 64u;
        const uint64_t kd = k_desc0 + (uint64_t)(s * (kTileBytes >> 4));
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint64_t koff = (uint64_t)((kk >> 2) * (kHalfBytes >> 4) + (kk & 3) * 2);
          const uint64_t qoffd = (uint64_t)((kk >> 2) * (kQHalf >> 4) + (kk & 3) * 2);
          umma_bf16(d, kd + koff, q_desc + qoffd, idesc_qk, kk > 0);
        }
        umma_commit(bar(K_EMPTY + s));
        umma_commit(bar(S_FULL + (i & 1)));
        return true;
      };
      if (ok) ok = issue_qk(0);
      if (ok && n_tiles > 1) ok = issue_qk(1);
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int g = i & 1, j = i >> 1, s = i % kStages;
        const uint2 mt = meta[i & 7];
        if (!mbar_wait(bar(V_FULL + s), (i / kStages) & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(bar(P_FULL + g), j & 1, abort_flag)) { ok = false; break; }   // P^T(i) in shared memory, O_g rescaled if needed
        tc_fence_after();
        const uint32_t d = tmem + 128u + (uint32_t)g * 64u;
        const uint64_t pd = smem_desc(base + Smem::p + g * kQBytes, 16);
        const uint64_t vd = v_desc0 + (uint64_t)(s * (kTileBytes >> 4));
        const int nsub = (int)mt.y;
#pragma unroll
        for (int kk = 0; kk < kSubPerTile; ++kk)
          if (kk < nsub) {
            // K step kk = keys [16 kk, 16 kk + 16): rows of the V tile, columns of P^T
            const uint64_t poff = (uint64_t)((kk >> 2) * (kQHalf >> 4) + (kk & 3) * 2);
            umma_bf16(d, vd + (uint64_t)(kk * (kSubBytes >> 4)), pd + poff, idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
          }
        umma_commit(bar(V_EMPTY + s));
        umma_commit(bar(P_EMPTY + g));
        if (i + 2 < n_tiles) ok = issue_qk(i + 2);
      }
      if (ok) umma_commit(bar(O_DONE));
    }
  } else {
    // =========================== softmax (warps 0-7): one thread per key ==================================
    const int g = warp >> 2, wq = warp & 3;
    const int key = wq * 32 + lane;                               // TMEM lane = key of the tile
    const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
    const uint32_t FULL = 0xffffffffu;
    const uint32_t s_addr = tmem + lane_addr + (uint32_t)g * 64u;
    const uint32_t o_addr = tmem + lane_addr + 128u + (uint32_t)g * 64u;
    float* wmax_g = wmax + g * 4 * 64;
    float* mref_g = mref + g * 64;
    float* corr_g = corr + g * 64;
    unsigned char* pbuf = sm + Smem::p + g * kQBytes;
    const float sc = prm.scale_log2;
    float lpart[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) lpart[q] = 0.f;
    bool ok = true;
#ifdef SPR_REM_TIMING
    long long tA = 0, tB = 0, tC = 0, tD = 0, tE = 0, tF = 0, t0;
    const long long tstart = clock64();
#define SPR_RT0() t0 = clock64()
#define SPR_RT(v) do { const long long t1 = clock64(); v += t1 - t0; t0 = t1; } while (0)
#else
#define SPR_RT0()
#define SPR_RT(v)
#endif
    for (int i = g, j = 0; i < n_tiles; i += 2, ++j) {
      SPR_RT0();
      ok = __all_sync(FULL, ok && mbar_wait(bar(S_FULL + g), j & 1, abort_flag) &&
                                mbar_wait(bar(META_FULL + (i & 7)), (i >> 3) & 1, abort_flag));
      if (ok) tc_fence_after();
      SPR_RT(tA);
      const uint2 mt = meta[i & 7];
      const int box = key >> 4;
      const bool valid = ok && box < (int)mt.y && (key & 15) <= (int)((mt.x >> (4 * box)) & 15u);
      float s[NQ];
      if (ok) {
#pragma unroll
        for (int c = 0; c < NQC; ++c) tmem_ld16(s_addr + c * 16, *reinterpret_cast<float(*)[16]>(&s[c * 16]));
      } else {
#pragma unroll
        for (int q = 0; q < NQ; ++q) s[q] = 0.f;
      }
      SPR_RT(tB);
      // scores go to the log2 domain; a query whose score exceeds the reference maximum by more than 8 for some
      // valid key of the tile makes the reference move (always on the group's first tile, where it is -inf)
      unsigned grew_lo = 0, grew_hi = 0;
      {
        float4 m4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
          if ((q & 3) == 0) m4 = reinterpret_cast<const float4*>(mref_g)[q >> 2];
          const float mr = (q & 3) == 0 ? m4.x : (q & 3) == 1 ? m4.y : (q & 3) == 2 ? m4.z : m4.w;
          s[q] *= sc;
          const bool gq = __any_sync(FULL, valid && s[q] - mr > 8.f);
          if (q < 32) grew_lo |= (unsigned)gq << q; else grew_hi |= (unsigned)gq << (q - 32);
        }
      }
      unsigned* gmask = reinterpret_cast<unsigned*>(sm + Smem::gmask) + g * 8;
      if (lane == 0) { gmask[wq * 2] = grew_lo; gmask[wq * 2 + 1] = grew_hi; }
      asm volatile("bar.sync %0, 128;" ::"r"(1 + g) : "memory");
      const unsigned all_lo = gmask[0] | gmask[2] | gmask[4] | gmask[6], all_hi = gmask[1] | gmask[3] | gmask[5] | gmask[7];
      const bool moved = (all_lo | all_hi) != 0;                    // uniform over the group
      if (moved) {
        // exact tile maximum of the flagged queries: warp reduction, four-way combine by warp 0 of the group
        float keep0 = -INFINITY, keep1 = -INFINITY;
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
          const bool fl = ((q < 32 ? all_lo >> q : all_hi >> (q - 32)) & 1u) != 0;   // uniform
          if (fl) {
            const int m = __reduce_max_sync(FULL, valid ? ord(s[q]) : ord(-INFINITY));
            if (q < 32) { if (lane == q) keep0 = unord(m); } else { if (lane == q - 32) keep1 = unord(m); }
          }
        }
        if (lane < NQ) wmax_g[wq * 64 + lane] = keep0;
        if (NQ > 32 && lane + 32 < NQ) wmax_g[wq * 64 + lane + 32] = keep1;
        asm volatile("bar.sync %0, 128;" ::"r"(1 + g) : "memory");
        if (wq == 0) {
#pragma unroll
          for (int hq = 0; hq < (NQ + 31) / 32; ++hq) {
            const int q = lane + 32 * hq;
            if (q < NQ) {
              const bool fl = (((hq == 0 ? all_lo : all_hi) >> lane) & 1u) != 0;
              const float tm = fmaxf(fmaxf(wmax_g[q], wmax_g[64 + q]), fmaxf(wmax_g[128 + q], wmax_g[192 + q]));
              const float old = mref_g[q];
              corr_g[q] = fl ? ex2(old - tm) : 1.f;                // 0 on the first tile
              if (fl) mref_g[q] = tm;
            }
          }
        }
        asm volatile("bar.sync %0, 128;" ::"r"(1 + g) : "memory");
      }
      SPR_RT(tC);
      // the previous P^T of this group must have been consumed (and O_g is then complete up to tile i - 2)
      if (j > 0) ok = __all_sync(FULL, ok && mbar_wait(bar(P_EMPTY + g), (j - 1) & 1, abort_flag));
      if (ok) tc_fence_after();
      SPR_RT(tD);
      if (moved && j > 0 && ok) {
        // rescale this thread's TMEM lane (= one output dimension) of O_g, column q by corr[q]
#pragma unroll
        for (int c = 0; c < NQC; ++c) {
          float t[16];
          tmem_ld16(o_addr + c * 16, t);
#pragma unroll
          for (int q = 0; q < 16; ++q) t[q] *= corr_g[c * 16 + q];
          tmem_st16(o_addr + c * 16, t);
        }
      }
      SPR_RT(tE);
      // P^T: element (query q, key) of the K-major [NQ x 128] tile, 128-byte swizzle, two halves of 64 keys
      {
        unsigned char* prow = pbuf + (key >> 6) * kQHalf;
        const uint32_t kc = (uint32_t)key & 63u;
        const uint32_t kchunk = kc >> 3, kin = (kc & 7u) << 1;
        float4 m4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (!moved) {
#pragma unroll
          for (int q = 0; q < NQ; ++q) {
            if ((q & 3) == 0) m4 = reinterpret_cast<const float4*>(mref_g)[q >> 2];
            const float mr = (q & 3) == 0 ? m4.x : (q & 3) == 1 ? m4.y : (q & 3) == 2 ? m4.z : m4.w;
            const float pq = valid ? ex2(s[q] - mr) : 0.f;
            lpart[q] += pq;
            *reinterpret_cast<__nv_bfloat16*>(prow + q * 128 + ((kchunk ^ (uint32_t)(q & 7)) << 4) + kin) = __float2bfloat16_rn(pq);
          }
        } else {
#pragma unroll
          for (int q = 0; q < NQ; ++q) {
            if ((q & 3) == 0) m4 = reinterpret_cast<const float4*>(mref_g)[q >> 2];
            const float mr = (q & 3) == 0 ? m4.x : (q & 3) == 1 ? m4.y : (q & 3) == 2 ? m4.z : m4.w;
            const float pq = valid ? ex2(s[q] - mr) : 0.f;
            lpart[q] = fmaf(lpart[q], corr_g[q], pq);
            *reinterpret_cast<__nv_bfloat16*>(prow + q * 128 + ((kchunk ^ (uint32_t)(q & 7)) << 4) + kin) = __float2bfloat16_rn(pq);
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      mbar_arrive(bar(P_FULL + g));
      SPR_RT(tF);
    }
#ifdef SPR_REM_TIMING
    if (blockIdx.x < 40 && blockIdx.y == 0 && lane == 0 && warp == 0 && n_tiles > 8) {
      const int nt = (n_tiles + 1) / 2;
      printf("rem NQ=%d tiles %d (group %d): wait S %lld  tmem ld %lld  max+combine %lld  wait P_EMPTY %lld  rescale %lld  P loop %lld | total per tile %lld\n",
             NQ, n_tiles, nt, tA / nt, tB / nt, tC / nt, tD / nt, tE / nt, tF / nt, (clock64() - tstart) / n_tiles);
    }
#endif
    // ---- row sums of the group, merge of the two groups ------------------------------------------------
    if (n_tiles > 0) ok = __all_sync(FULL, ok && mbar_wait(bar(O_DONE), 0, abort_flag));
    {
      float keep0 = 0.f, keep1 = 0.f;
#pragma unroll
      for (int q = 0; q < NQ; ++q) {
        const float t = warp_sum(lpart[q]);
        if (q < 32) { if (lane == q) keep0 = t; } else { if (lane == q - 32) keep1 = t; }
      }
      float* ls = lsum + (g * 4 + wq) * 64;
      if (lane < NQ) ls[lane] = keep0;
      if (NQ > 32 && lane + 32 < NQ) ls[lane + 32] = keep1;
    }
    asm volatile("bar.sync 3, 256;" ::: "memory");
    if (warp == 0) {
#pragma unroll
      for (int hq = 0; hq < (NQ + 31) / 32; ++hq) {
        const int q = lane + 32 * hq;
        if (q < NQ) {
          const float la = lsum[q] + lsum[64 + q] + lsum[128 + q] + lsum[192 + q];
          const float lb = lsum[256 + q] + lsum[320 + q] + lsum[384 + q] + lsum[448 + q];
          const float ma = mref[q], mb = mref[64 + q];
          const float mm = fmaxf(ma, mb);
          const float wa = la > 0.f ? ex2(ma - mm) : 0.f, wb = lb > 0.f ? ex2(mb - mm) : 0.f;
          const float lt = la * wa + lb * wb;
          const float inv = lt > 0.f ? 1.f / lt : 0.f;
          fin[q] = wa * inv; fin[64 + q] = wb * inv;
        }
      }
    }
    asm volatile("bar.sync 3, 256;" ::: "memory");
    // group A finishes queries [0, NQ/2), group B the rest; this thread's TMEM lane is output dimension `key`
    if (ok) {
      tc_fence_after();
      constexpr int HC = NQC > 1 ? NQC / 2 : 1;                    // 16-column chunks per group (NQC = 3: group A one, group B two)
      const int c0 = NQC == 1 ? 0 : (g == 0 ? 0 : HC);
      const int c1 = NQC == 1 ? (g == 0 ? 1 : 0) : (g == 0 ? HC : NQC);
      for (int c = c0; c < c1; ++c) {
        float ta[16], tb[16];
        if (n_tiles > 0) tmem_ld16(tmem + lane_addr + 128u + c * 16, ta);
        if (n_tiles > 1) tmem_ld16(tmem + lane_addr + 192u + c * 16, tb);
#pragma unroll
        for (int qq = 0; qq < 16; ++qq) {
          const int q = c * 16 + qq;
          if (q < nq) {
            const float fa = fin[q], fb = fin[64 + q];
            float o = 0.f;
            if (n_tiles > 0 && fa != 0.f) o = ta[qq] * fa;
            if (n_tiles > 1 && fb != 0.f) o += tb[qq] * fb;
            const int dst = prm.q_perm[(i64)bh * prm.N + row0 + q];
            const int b = bh / prm.H, h = bh % prm.H;
            prm.O[b * prm.os[0] + h * prm.os[1] + (i64)dst * prm.os[2] + key] = __float2bfloat16_rn(o);
            if (prm.O_sparse) prm.O_sparse[((i64)bh * prm.N + dst) * kD + key] = o;
          }
        }
      }
    }
  }
  // ---- teardown ----------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int k = 0; k < 64; ++k) __nanosleep(1000);
    if (tid == 0) set_error(prm.err, SPARSEPR_ERR_TIMEOUT);
    __syncthreads();
  }
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

}  // namespace rem
}  // namespace tc

cudaError_t init_attention_rem() {
  using namespace tc::rem;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k_attention_rem<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<1>::total)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(k_attention_rem<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<2>::total)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(k_attention_rem<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<3>::total)) != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_attention_rem<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<4>::total);
}

// Remainders of 1..64 rows of every query group (the 128-row kernel must have been given tile offsets
// that leave them out).  Q, K, V group-major [BH][N][128] bf16.
bool launch_attention_rem(const AttnArgs& a, cudaStream_t st) {
  using namespace tc;
  using namespace tc::rem;
  CUtensorMap mq[4], mk, mv;
  for (int z = 0; z < 4; ++z)
    if (!make_map(&mq[z], a.Q, kD, a.N, a.BH, 1, 0, (i64)a.N * kD, kD, 16 * (z + 1))) return false;
  if (!make_map(&mk, a.K, kD, a.N, a.BH, 1, 0, (i64)a.N * kD, kD, kSub) || !make_map(&mv, a.V, kD, a.N, a.BH, 1, 0, (i64)a.N * kD, kD, kSub))
    return false;
  Params p{};
  p.BH = a.BH; p.N = a.N; p.Cq = a.Cq; p.Ck = a.Ck; p.scale_log2 = a.scale * 1.4426950408889634f;
  p.q_off = a.q_off; p.kv_off = a.kv_off; p.route_ptr = a.route_ptr; p.route_idx = a.route_idx; p.q_perm = a.q_perm;
  p.O = (__nv_bfloat16*)a.O; for (int i = 0; i < 3; ++i) p.os[i] = a.os[i];
  p.H = a.H; p.O_sparse = a.O_sparse; p.err = a.err;
  const dim3 grid(a.Cq, a.BH);
  k_attention_rem<1><<<grid, kThreads, Cfg<1>::total, st>>>(mq[0], mk, mv, p);
  k_attention_rem<2><<<grid, kThreads, Cfg<2>::total, st>>>(mq[1], mk, mv, p);
  k_attention_rem<3><<<grid, kThreads, Cfg<3>::total, st>>>(mq[2], mk, mv, p);
  k_attention_rem<4><<<grid, kThreads, Cfg<4>::total, st>>>(mq[3], mk, mv, p);
  return true;
}

}  // namespace spr
