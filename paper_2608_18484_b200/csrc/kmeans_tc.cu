// k-means assignment (Section 4.1) with the score contraction on the tensor cores.
//
// score(x, c) = ||mu_c||^2 - 2 x.mu_c.  The dot products run on tcgen05.mma with both
// operands split into two bf16 words (x = xh + xl, mu = mh + ml; the products xh.mh,
// xh.ml, xl.mh are accumulated in fp32 in TMEM; the dropped term is ~2^-18 relative).
// Each row keeps its best and second-best score; a row whose gap is not larger than a
// conservative bound on the score error is NOT decided here but handed to the exact
// recheck (per-head row lists; float64 with the operation order of the definition for every
// centroid that a float32 filter cannot rule out), so the final assignment always equals the
// exact float64 decision with ties to the lowest id.
//
// Persistent CTAs: each owns row tiles (128 rows) of one head; centroid chunks of 256
// stream through shared memory (resident when C <= 256).  Roles: warps 0-3 and 6-9 are two
// epilogue groups on alternate row tiles (one row per thread: tcgen05.ld, best/second,
// fixed-point centroid sums with warp-level pre-aggregation), warp 4 TMA producer, warp 5
// MMA issuer.
#include "kernels.cuh"
#include "tc_common.cuh"

namespace spr {
namespace tc {

constexpr int kKmThreads = 320;
constexpr int kKmChunk = 256;                         // centroids per MMA (N)
constexpr uint32_t kXBytes = 128 * 128;               // one [128 rows x 64 bf16] block
constexpr uint32_t kMuBytes = kKmChunk * 128;         // one [256 x 64 bf16] block

struct KmSmem {
  static constexpr uint32_t x = 0;                              // 2 stages x (hi, lo)
  static constexpr uint32_t mu = x + 2 * 2 * kXBytes;           // 2 stages x (hi, lo)
  static constexpr uint32_t bars = mu + 2 * 2 * kMuBytes;       // 12 mbarriers
  static constexpr uint32_t misc = bars + 12 * 8;
  static constexpr uint32_t total = misc + 32;
};
constexpr size_t kKmSmemBytes = KmSmem::total + 1024;
enum KmBar { X_FULL = 0, X_EMPTY = 2, MU_FULL = 4, MU_EMPTY = 6, ACC_FULL = 8, ACC_EMPTY = 10 };

struct KmParams {
  int N, C, r, R, n_chunks, ctas_per_head;
  const float* phi; int ldphi;          // fp32 features (for the centroid sums)
  const float* xnorm;                   // [BH][N]
  const float* mu2;                     // [BH][C]
  int* assign;
  i64* sums; int* counts; const int* fx_shift;
  int* flagged; int* flag_count;        // rows left to the exact recheck: [BH][N] row indices, [BH] their number
  int* flag_count_next;                 // [BH] or null: the counters of the next pass, zeroed here
  int* err;
  const int* prev_changed; int* cur_changed;   // [BH] or null: rows whose assignment changed in the previous / this pass
};

__global__ void __launch_bounds__(kKmThreads, 1)
k_kmeans_assign_tc(const __grid_constant__ CUtensorMap mapXh, const __grid_constant__ CUtensorMap mapXl,
                   const __grid_constant__ CUtensorMap mapMh, const __grid_constant__ CUtensorMap mapMl, KmParams prm) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw);
  volatile int* misc = reinterpret_cast<volatile int*>(sm + KmSmem::misc);   // [0] tmem base, [1] abort
  const uint32_t bars = base + KmSmem::bars;
  auto bar = [&](int i) { return bars + 8u * i; };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y, cta = blockIdx.x;

  __shared__ __align__(16) float mu2s[kMaxGroups];          // ||mu_c||^2, +inf beyond C
  __shared__ int s_skip;
  __shared__ float s_red[34];
  pdl_wait();                                               // the centroids of this pass come from the kernel before
  pdl_launch_dependents();
  if (cta == 0 && tid == 0 && prm.flag_count_next) prm.flag_count_next[bh] = 0;   // last read by the recheck two kernels back
  float mu2max = 0.f;
  for (int c = tid; c < kMaxGroups; c += kKmThreads) {
    const float v = c < prm.C ? prm.mu2[(i64)bh * prm.C + c] : INFINITY;
    mu2s[c] = v;
    if (c < prm.C) mu2max = fmaxf(mu2max, v);
  }
  // a head whose previous pass changed no assignment has reached the fixed point of the iteration: skipped
  if (tid == 0) s_skip = (prm.err != nullptr && *reinterpret_cast<volatile int*>(prm.err) == SPARSEPR_ERR_TIMEOUT) ||
                         (prm.prev_changed != nullptr && prm.prev_changed[bh] == 0);
  // largest centroid norm of the head, rounded up: it enters the bound on the score error only
  const float mm_head = sqrtf(block_max(mu2max, s_red)) * 1.000001f;
  __syncthreads();
  if (s_skip) return;

  const int row_tiles = (prm.N + 127) / 128;
  // contiguous chunk of row tiles per CTA: CTAs that run at the same time then work on distant
  // tokens, i.e. on different clusters, and do not contend for the same centroid sums
  const int per_cta = (row_tiles + prm.ctas_per_head - 1) / prm.ctas_per_head;
  const int tile0 = cta * per_cta;
  const int my_tiles = max(0, min(per_cta, row_tiles - tile0));
  const int n_chunks = prm.n_chunks;
  const int steps = my_tiles * n_chunks;
  const int n_pairs = (my_tiles + 1) / 2;
  if (tid == 0) {
    for (int i = 0; i < 12; ++i) mbar_init(bar(i), (i == ACC_EMPTY || i == ACC_EMPTY + 1) ? 128 : 1);
    misc[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(base + KmSmem::misc, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = (uint32_t)misc[0];
  volatile int* abort_flag = &misc[1];

  if (warp == 4) {
    // =========================== TMA producer ============================================
    if (lane == 0) {
      // Step order: the row tiles are taken in pairs, and inside a pair the centroid chunks are interleaved
      // (tile 0 chunk 0, tile 1 chunk 0, tile 0 chunk 1, ...): score buffer b then only ever holds tiles of parity b,
      // i.e. belongs to one epilogue group, whose waits follow the buffer's phases in order.  (With the chunks of a
      // tile back to back both groups would share both buffers, and a group waiting for a phase that lies two ahead
      // of the barrier's current one takes the parity test for passed.)  v counts the steps that exist.
      int v = 0;
      int pair = 0, r2 = 0;                                    // sidx = pair * 2 n_chunks + r2
      for (int sidx = 0; sidx < n_pairs * 2 * n_chunks; ++sidx) {
        const int tl = 2 * pair + (r2 & 1), ch = r2 >> 1;
        if (++r2 == 2 * n_chunks) { r2 = 0; ++pair; }
        if (tl >= my_tiles) continue;
        if (n_chunks > 1 || v == 0) {
          const int ms = n_chunks > 1 ? (v & 1) : 0;
          if (n_chunks > 1 && !mbar_wait(bar(MU_EMPTY + ms), ((v >> 1) & 1) ^ 1, abort_flag)) break;
          mbar_expect_tx(bar(MU_FULL + ms), 2 * kMuBytes);
          tma_load_4d(base + KmSmem::mu + ms * 2 * kMuBytes, &mapMh, bar(MU_FULL + ms), 0, ch * kKmChunk, bh, 0);
          tma_load_4d(base + KmSmem::mu + ms * 2 * kMuBytes + kMuBytes, &mapMl, bar(MU_FULL + ms), 0, ch * kKmChunk, bh, 0);
        }
        if (ch == 0) {
          const int xs = tl & 1;
          if (!mbar_wait(bar(X_EMPTY + xs), ((tl >> 1) & 1) ^ 1, abort_flag)) break;
          const int row0 = (tile0 + tl) * 128;
          mbar_expect_tx(bar(X_FULL + xs), 2 * kXBytes);
          tma_load_4d(base + KmSmem::x + xs * 2 * kXBytes, &mapXh, bar(X_FULL + xs), 0, row0, bh, 0);
          tma_load_4d(base + KmSmem::x + xs * 2 * kXBytes + kXBytes, &mapXl, bar(X_FULL + xs), 0, row0, bh, 0);
        }
        ++v;
      }
    }
  } else if (warp == 5) {
    // =========================== MMA issuer ================================================
    if (lane == 0) {
      // The issuing thread shares its warp scheduler with epilogue warps that leave it few issue slots, and the next
      // product of a score buffer can only be issued once the epilogue has released it: every instruction of this
      // loop is on the critical path.  Descriptors are therefore built once (only their 16-byte address field moves),
      // the step order is tracked with counters instead of divisions, and the k-steps are unrolled.
      const uint32_t idesc = idesc_bf16(0, kKmChunk);
      const int ksteps = prm.R / 16;
      const uint64_t x_desc0 = smem_desc(base + KmSmem::x, 16), m_desc0 = smem_desc(base + KmSmem::mu, 16);
      int v = 0;                                               // same step order as the producer
      int pair = 0, r2 = 0;                                    // sidx = pair * 2 n_chunks + r2
      for (int sidx = 0; sidx < n_pairs * 2 * n_chunks; ++sidx) {
        const int tl = 2 * pair + (r2 & 1), ch = r2 >> 1;
        if (++r2 == 2 * n_chunks) { r2 = 0; ++pair; }
        if (tl >= my_tiles) continue;
        const int xs = tl & 1, ms = n_chunks > 1 ? (v & 1) : 0;
        const int ab = tl & 1, au = (tl >> 1) * n_chunks + ch;   // score buffer and how often it has been used before
        if (ch == 0 && !mbar_wait(bar(X_FULL + xs), (tl >> 1) & 1, abort_flag)) break;
        if ((n_chunks > 1 || v == 0) && !mbar_wait(bar(MU_FULL + ms), n_chunks > 1 ? ((v >> 1) & 1) : 0, abort_flag)) break;
        if (!mbar_wait(bar(ACC_EMPTY + ab), (au & 1) ^ 1, abort_flag)) break;
        tc_fence_after();
        const uint32_t d = tmem + (uint32_t)ab * 256u;
        const uint64_t xh = x_desc0 + (uint64_t)((xs * 2 * kXBytes) >> 4), xl = xh + (uint64_t)(kXBytes >> 4);
        const uint64_t mh = m_desc0 + (uint64_t)((ms * 2 * kMuBytes) >> 4), ml = mh + (uint64_t)(kMuBytes >> 4);
        // x_h mu_h + x_h mu_l + x_l mu_h; one k-step = 16 columns = 32 bytes = 2 address units
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) if (kk < ksteps) umma_bf16(d, xh + 2 * kk, mh + 2 * kk, idesc, kk > 0);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) if (kk < ksteps) umma_bf16(d, xh + 2 * kk, ml + 2 * kk, idesc, 1);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) if (kk < ksteps) umma_bf16(d, xl + 2 * kk, mh + 2 * kk, idesc, 1);
        if (ch == n_chunks - 1) umma_commit(bar(X_EMPTY + xs));
        if (n_chunks > 1) umma_commit(bar(MU_EMPTY + ms));
        umma_commit(bar(ACC_FULL + ab));
        ++v;
      }
    }
  } else {
    // =========================== epilogue: argmin, sums =====================================
    // two groups of four warps (warps 0-3 and 6-9) take alternate row tiles
    const uint32_t FULL = 0xffffffffu;
    const int grp = warp < 4 ? 0 : 1, wq = warp & 3;
    const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
    const float mm = mm_head;
    bool ok = true;
    for (int tl = grp; tl < my_tiles; tl += 2) {
      const int row = (tile0 + tl) * 128 + wq * 32 + lane;
      float best = 3.0e38f, second = 3.0e38f;
      int bi = 0;
      // features of the warp's 32 rows for this lane's two columns (used by the centroid sums);
      // issued before the score wait so that the loads overlap it
      float pv0[32], pv1[32];
      const float xn = row < prm.N ? prm.xnorm[(i64)bh * prm.N + row] : 0.f;   // needed after the scores: fetched now
      // the row's group of the previous pass, for the count of rows that move (same reason: its latency is hidden here)
      const int old_a = (prm.prev_changed != nullptr && row < prm.N) ? prm.assign[(i64)bh * prm.N + row] : -1;
      if (prm.sums) {
        const int rowbase = (tile0 + tl) * 128 + wq * 32;
        // this lane's columns are (2 lane, 2 lane + 1): one 8-byte load per row (ldphi is a multiple of 16, and
        // columns r..ldphi-1 hold zeros, so a pair that straddles r reads a zero)
        const bool cok = 2 * lane < prm.r;
        if (rowbase + 31 < prm.N) {                            // every tile but the last of a head (uniform)
          const float* xb = prm.phi + ((i64)bh * prm.N + rowbase) * prm.ldphi + 2 * lane;
#pragma unroll
          for (int rr = 0; rr < 32; ++rr) {
            const float2 x2 = cok ? *reinterpret_cast<const float2*>(xb + rr * prm.ldphi) : make_float2(0.f, 0.f);
            pv0[rr] = x2.x; pv1[rr] = x2.y;
          }
        } else {
#pragma unroll
          for (int rr = 0; rr < 32; ++rr) {
            const int rw = min(rowbase + rr, prm.N - 1);
            const float* xr = prm.phi + ((i64)bh * prm.N + rw) * prm.ldphi + 2 * lane;
            const float2 x2 = cok ? *reinterpret_cast<const float2*>(xr) : make_float2(0.f, 0.f);
            pv0[rr] = x2.x; pv1[rr] = x2.y;
          }
        }
      }
      for (int ch = 0; ch < n_chunks; ++ch) {
        const int ab = tl & 1, au = (tl >> 1) * n_chunks + ch;   // this group's score buffer and its phase
        ok = __all_sync(FULL, ok && mbar_wait(bar(ACC_FULL + ab), au & 1, abort_flag));
        if (!ok) continue;
        tc_fence_after();
        const int c0 = ch * kKmChunk;
        const int nvalid = min(kKmChunk, prm.C - c0);
#pragma unroll 1
        for (int g = 0; g < kKmChunk / 32; ++g) {
          if (g * 32 >= nvalid) break;                       // uniform: whole column groups beyond C
          float t[32];
          tmem_ld32(tmem + lane_addr + (uint32_t)ab * 256u + g * 32, t);
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const int c = c0 + g * 32 + j;
            const float4 m4 = *reinterpret_cast<const float4*>(mu2s + c);
            const float mv[4] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const float s = fmaf(-2.f, t[j + u], mv[u]);
              second = fminf(second, fmaxf(s, best));
              bi = s < best ? c + u : bi;
              best = fminf(best, s);
            }
          }
        }
        tc_fence_before();
        mbar_arrive(bar(ACC_EMPTY + ab));
      }
      // decide, or hand the row to the exact recheck
      const bool valid = ok && row < prm.N;
      bool decided = false, moved = false;
      if (valid) {
        // bound on |computed score - true score|: split-operand products (2^-13 relative with
        // margin), fp32 accumulation and the final combination
        const float E = 2.5e-4f * xn * mm + 1.0e-6f * (mm * mm + xn * mm);
        decided = second - best > 2.f * E;
        if (decided) {
          moved = old_a != bi;
          prm.assign[(i64)bh * prm.N + row] = bi;
        } else {                                             // the recheck writes (and compares) this row's assignment
          const int pos = atomicAdd(prm.flag_count + bh, 1);
          prm.flagged[(i64)bh * prm.N + pos] = row;
        }
      }
      if (prm.cur_changed != nullptr) {
        const int nmoved = __popc(__ballot_sync(FULL, moved));
        if (lane == 0 && nmoved) atomicAdd(prm.cur_changed + bh, nmoved);
      }
      if (prm.sums) {
        // warp-level pre-aggregation: lanes = feature columns (2 lane, 2 lane + 1); the 32 rows of the
        // warp were prefetched above; one fixed-point atomic per (cluster, column)
        unsigned todo = __ballot_sync(FULL, decided);
        // 2^shift as a float: scaling a float32 partial sum by a power of two is exact, so the conversion below
        // gives the same integer as a float64 product would
        const float scl = __int_as_float((127 + prm.fx_shift[bh]) << 23);
        while (todo) {
          const int leader = __ffs(todo) - 1;
          const int cl = __shfl_sync(FULL, bi, leader);
          const unsigned members = __ballot_sync(FULL, decided && bi == cl) & todo;
          todo &= ~members;
          // float32 partial sums in a fixed order (hence reproducible), one
          // conversion to fixed point per (cluster, column)
          // (four interleaved partial sums: one chain of 32 dependent additions would set the pace of this loop)
          float2 a2[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
          for (int rr = 0; rr < 32; ++rr)
            if ((members >> rr) & 1u) a2[rr & 3] = __fadd2_rn(a2[rr & 3], make_float2(pv0[rr], pv1[rr]));   // one packed add per member row
          const float2 a01 = __fadd2_rn(__fadd2_rn(a2[0], a2[1]), __fadd2_rn(a2[2], a2[3]));
          const float a0 = a01.x, a1 = a01.y;
          const i64 acc0 = __float2ll_rn(a0 * scl), acc1 = __float2ll_rn(a1 * scl);
          i64* s = prm.sums + ((i64)bh * prm.C + cl) * prm.R;
          if (2 * lane < prm.r) atomicAdd(reinterpret_cast<u64*>(s + 2 * lane), (u64)acc0);
          if (2 * lane + 1 < prm.r) atomicAdd(reinterpret_cast<u64*>(s + 2 * lane + 1), (u64)acc1);
          if (lane == 0) atomicAdd(prm.counts + (i64)bh * prm.C + cl, __popc(members));
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int k = 0; k < 64; ++k) __nanosleep(1000);
    if (tid == 0) set_error(prm.err, SPARSEPR_ERR_TIMEOUT);
    __syncthreads();
  }
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// Exact decision for the rows the fast path could not prove (a few thousand per pass at N = 32760 and 24 heads).
// The definition is the squared distance in float64 with the terms added in order of k (the zero padding of columns
// r..R-1 adds exact zeros), ties to the lowest id.  Every such row needs all C centroids of its head, so the rows of a
// head share them: grid (G, BH); a CTA brings the head's centroids to shared memory once and its eight warps take the
// head's flagged rows in turn.  Per row:
//   1. float32 distances to all centroids (lane = centroid, 8 at a time; rows of mu padded by 4 floats, so that the
//      16-byte reads of consecutive centroids fall into different banks).  Every term is non-negative, hence the
//      float32 value is within (R + 3) 2^-24 of the true distance, relatively;
//   2. only centroids within 4 (R + 4) 2^-24 of the float32 minimum (relative, plus a denormal's worth) can hold the
//      float64 minimum: those few (normally one or two) are evaluated by the definition, one lane each.
__global__ void __launch_bounds__(256) k_assign_recheck_staged(const int* __restrict__ flagged, const int* __restrict__ flag_count,
                                                               const float* __restrict__ phi, int ldphi, int N, int r, int R,
                                                               const float* __restrict__ mu, int C, int* __restrict__ assign,
                                                               i64* __restrict__ sums, int* __restrict__ counts,
                                                               const int* __restrict__ fx_shift, int* __restrict__ recheck_total,
                                                               int first_pass, int* __restrict__ cur_changed) {
  extern __shared__ __align__(16) float rs_smem[];
  const unsigned FULL = 0xffffffffu;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.y;
  pdl_wait();                                                  // the row lists come from the assignment kernel before
  pdl_launch_dependents();
  const int n = flag_count[bh];
  if (blockIdx.x == 0 && bh == 0 && tid == 0 && recheck_total) {
    int total = 0;
    for (int h = 0; h < (int)gridDim.y; ++h) total += flag_count[h];
    *recheck_total = total;
  }
  if ((int)blockIdx.x * 8 >= n) return;                        // no row for this CTA
  const int LDM = R + 4, Cp = (C + 31) & ~31;
  float* mu_s = rs_smem;                                       // [C][R + 4]
  float* d32_all = mu_s + (size_t)C * LDM;                     // [8 warps][Cp]
  float* xs_all = d32_all + 8 * Cp;                            // [8 warps][R]
  {
    const float4* src = reinterpret_cast<const float4*>(mu + (i64)bh * C * R);
    const int q = R / 4;
    for (int e = tid; e < C * q; e += 256) {
      const int c = e / q, k4 = e - c * q;
      *reinterpret_cast<float4*>(mu_s + (size_t)c * LDM + 4 * k4) = src[e];
    }
  }
  __syncthreads();
  float* d32 = d32_all + warp * Cp;
  float* xs = xs_all + warp * R;
  for (int i = blockIdx.x * 8 + warp; i < n; i += gridDim.x * 8) {
    const int row = flagged[(i64)bh * N + i];
    const i64 gr = (i64)bh * N + row;
    const float* x = phi + gr * ldphi;
    __syncwarp();
    for (int k = lane; k < R; k += 32) xs[k] = x[k];
    __syncwarp();
    float best32 = INFINITY;
    for (int c0 = 0; c0 < C; c0 += 256) {
      // packed float32 arithmetic, two columns per instruction: (m - x)^2 summed in two partial sums per centroid
      float2 acc[8];
      const float* mrow[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) { acc[j] = make_float2(0.f, 0.f); mrow[j] = mu_s + (size_t)min(c0 + 32 * j + lane, C - 1) * LDM; }
#pragma unroll 2
      for (int k = 0; k < R; k += 4) {
        const float4 xv = *reinterpret_cast<const float4*>(xs + k);
        const float2 nx0 = make_float2(-xv.x, -xv.y), nx1 = make_float2(-xv.z, -xv.w);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float4 mv = *reinterpret_cast<const float4*>(mrow[j] + k);
          const float2 d0 = __fadd2_rn(make_float2(mv.x, mv.y), nx0), d1 = __fadd2_rn(make_float2(mv.z, mv.w), nx1);
          acc[j] = __ffma2_rn(d0, d0, acc[j]);
          acc[j] = __ffma2_rn(d1, d1, acc[j]);
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int c = c0 + 32 * j + lane;
        if (c < Cp) {
          const float d = c < C ? acc[j].x + acc[j].y : INFINITY;
          d32[c] = d;
          best32 = fminf(best32, d);
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best32 = fminf(best32, __shfl_xor_sync(FULL, best32, o));
    const float thr = best32 * (1.f + 4.f * (float)(R + 4) * 5.9604645e-8f) + 1e-30f;
    // candidates: normally one, and then the decision is made (float64 arithmetic is slow on this GPU: about 16
    // cycles per warp instruction, 5 instructions per term)
    int ncand = 0, cand = -1;
    for (int c = lane; c < C; c += 32)                         // (never past C: with a NaN row thr is +inf, and so are the pad entries)
      if (d32[c] <= thr) { ++ncand; cand = c; }
    const int total_cand = __reduce_add_sync(FULL, ncand);
    int bi;
    if (total_cand == 1) {
      bi = __reduce_max_sync(FULL, cand);
    } else if (total_cand == 0) {
      bi = 0;                                                  // every distance is NaN (non-finite input, reported elsewhere): group 0
    } else {
      double best = 0.0;
      bi = -1;
      for (int c = lane; c < C; c += 32) {
        if (d32[c] <= thr) {
          const float* m = mu_s + (size_t)c * LDM;
          double dsum = 0.0;
#pragma unroll 8
          for (int k = 0; k < R; ++k) {
            const double diff = __dsub_rn((double)xs[k], (double)m[k]);
            dsum = __dadd_rn(dsum, __dmul_rn(diff, diff));
          }
          if (bi < 0 || dsum < best) { best = dsum; bi = c; }    // a lane meets its centroids in increasing order
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const double ob = __shfl_xor_sync(FULL, best, o);
        const int oi = __shfl_xor_sync(FULL, bi, o);
        if (oi >= 0 && (bi < 0 || ob < best || (ob == best && oi < bi))) { best = ob; bi = oi; }
      }
    }
    bi = min(max(bi, 0), C - 1);
    if (lane == 0) {
      if (cur_changed != nullptr && (first_pass || assign[gr] != bi)) atomicAdd(cur_changed + bh, 1);
      assign[gr] = bi;
    }
    if (sums) {
      // 2^shift as a float: scaling a float32 value by a power of two is exact, so the conversion gives the same
      // integer as the float64 product
      const float scl = __int_as_float((127 + fx_shift[bh]) << 23);
      i64* sp = sums + ((i64)bh * C + bi) * R;
      for (int t = lane; t < r; t += 32) atomicAdd(reinterpret_cast<u64*>(sp + t), (u64)__float2ll_rn(xs[t] * scl));
      if (lane == 0) atomicAdd(counts + (i64)bh * C + bi, 1);
    }
  }
}
// shared memory of the kernel above
static size_t recheck_staged_smem(int C, int R) { return ((size_t)C * (R + 4) + 8 * (size_t)((C + 31) & ~31) + 8 * (size_t)R) * sizeof(float); }

// The same decision without staging, for centroid tables that do not fit into shared memory: grid (X, BH), one CTA per
// row, one thread per centroid, float64 throughout.
__global__ void __launch_bounds__(256) k_assign_recheck(const int* __restrict__ flagged, const int* __restrict__ flag_count,
                                                        const float* __restrict__ phi, int ldphi, int N, int r, int R,
                                                        const float* __restrict__ mu, int C, int* __restrict__ assign,
                                                        i64* __restrict__ sums, int* __restrict__ counts,
                                                        const int* __restrict__ fx_shift, int* __restrict__ recheck_total,
                                                        int first_pass, int* __restrict__ cur_changed) {
  __shared__ double s_best[8];
  __shared__ int s_bi[8];
  const unsigned FULL = 0xffffffffu;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.y;
  const int n = flag_count[bh];
  if (blockIdx.x == 0 && bh == 0 && tid == 0 && recheck_total) {
    int total = 0;
    for (int h = 0; h < (int)gridDim.y; ++h) total += flag_count[h];
    *recheck_total = total;
  }
  for (int i = blockIdx.x; i < n; i += gridDim.x) {
    const i64 gr = (i64)bh * N + flagged[(i64)bh * N + i];
    const float4* x4 = reinterpret_cast<const float4*>(phi + gr * ldphi);
    const float* muh = mu + (i64)bh * C * R;
    double best = 0.0;
    int bi = -1;
    for (int c = tid; c < C; c += 256) {
      const float4* m4 = reinterpret_cast<const float4*>(muh + (i64)c * R);
      double dsum = 0.0;
      for (int k4 = 0; k4 < R / 4; k4 += 4) {               // R is a multiple of 16: four vector loads in flight
        float4 xv[4], mv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { xv[u] = x4[k4 + u]; mv[u] = m4[k4 + u]; }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float xs[4] = {xv[u].x, xv[u].y, xv[u].z, xv[u].w}, ms[4] = {mv[u].x, mv[u].y, mv[u].z, mv[u].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const double diff = __dsub_rn((double)xs[e], (double)ms[e]);
            dsum = __dadd_rn(dsum, __dmul_rn(diff, diff));
          }
        }
      }
      if (bi < 0 || dsum < best) { best = dsum; bi = c; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ob = __shfl_xor_sync(FULL, best, o);
      const int oi = __shfl_xor_sync(FULL, bi, o);
      if (oi >= 0 && (bi < 0 || ob < best || (ob == best && oi < bi))) { best = ob; bi = oi; }
    }
    if (lane == 0) { s_best[warp] = best; s_bi[warp] = bi; }
    __syncthreads();
    best = s_best[0]; bi = s_bi[0];
#pragma unroll
    for (int w = 1; w < 8; ++w) {
      const double ob = s_best[w];
      const int oi = s_bi[w];
      if (oi >= 0 && (bi < 0 || ob < best || (ob == best && oi < bi))) { best = ob; bi = oi; }
    }
    if (tid == 0) {
      if (cur_changed != nullptr && (first_pass || assign[gr] != bi)) atomicAdd(cur_changed + bh, 1);
      assign[gr] = bi;
    }
    if (sums) {
      const float* x = phi + gr * ldphi;
      const double scl = ldexp(1.0, fx_shift[bh]);
      i64* sp = sums + ((i64)bh * C + bi) * R;
      if (tid < r) atomicAdd(reinterpret_cast<u64*>(sp + tid), (u64)__double2ll_rn((double)x[tid] * scl));
      if (tid == 0) atomicAdd(counts + (i64)bh * C + bi, 1);
    }
    __syncthreads();
  }
}

// phi fp32 [rows][ld] -> hi/lo bf16 [rows][64] (zero padded) and the row norms
__global__ void __launch_bounds__(256) k_split_bf16(const float* __restrict__ x, int ld, i64 rows, int r,
                                                    __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                    float* __restrict__ norm) {
  pdl_wait();                                                   // the features come from the kernels before
  pdl_launch_dependents();
  const i64 t = (i64)blockIdx.x * 256 + threadIdx.x;
  const i64 row = t >> 3;
  const int c0 = (int)(t & 7) * 8;
  if (row >= rows) return;
  float v[8], h[8], l[8];
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    v[k] = c0 + k < r ? x[row * ld + c0 + k] : 0.f;
    const __nv_bfloat16 hb = __float2bfloat16_rn(v[k]);
    h[k] = __bfloat162float(hb);
    l[k] = v[k] - h[k];
    ss = fmaf(v[k], v[k], ss);
  }
  store8(hi + row * 64 + c0, h);
  store8(lo + row * 64 + c0, l);
  if (norm) {
    ss += __shfl_xor_sync(0xffffffffu, ss, 1);
    ss += __shfl_xor_sync(0xffffffffu, ss, 2);
    ss += __shfl_xor_sync(0xffffffffu, ss, 4);
    if ((t & 7) == 0) norm[row] = sqrtf(ss) * 1.000001f;
  }
}

}  // namespace tc

constexpr size_t kRecheckSmemMax = 200 * 1024;
cudaError_t init_kmeans_tc() {
  const cudaError_t e = cudaFuncSetAttribute(tc::k_assign_recheck_staged, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRecheckSmemMax);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(tc::k_kmeans_assign_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kKmSmemBytes);
}
bool kmeans_tc_supported() { return tc::tma_available(); }

void launch_split_bf16(const float* x, int ld, i64 rows, int r, __nv_bfloat16* hi, __nv_bfloat16* lo, float* norm,
                       cudaStream_t st) {
  launch_pdl(tc::k_split_bf16, dim3((unsigned)((rows * 8 + 255) / 256)), dim3(256), 0, st, x, ld, rows, r, hi, lo, norm);
}

// One assignment pass.  xh/xl: bf16 [BH][N][64]; mh/ml: bf16 [BH][C][64]; sums may be null (no update wanted).
bool launch_kmeans_assign_tc(const KmeansTcArgs& a, cudaStream_t st) {
  using namespace tc;
  CUtensorMap mxh, mxl, mmh, mml;
  if (!make_map(&mxh, a.xh, 64, a.N, a.BH, 1, 0, (i64)a.N * 64, 64, 128) || !make_map(&mxl, a.xl, 64, a.N, a.BH, 1, 0, (i64)a.N * 64, 64, 128) ||
      !make_map(&mmh, a.mh, 64, a.C, a.BH, 1, 0, (i64)a.C * 64, 64, kKmChunk) || !make_map(&mml, a.ml, 64, a.C, a.BH, 1, 0, (i64)a.C * 64, 64, kKmChunk))
    return false;
  KmParams p{};
  p.N = a.N; p.C = a.C; p.r = a.r; p.R = a.R; p.n_chunks = (a.C + kKmChunk - 1) / kKmChunk;
  const int row_tiles = (a.N + 127) / 128;
  // CTAs per head: one CTA fills an SM and works through its row tiles one after the other, so the launch takes
  // (rounds of CTAs over the SMs) x (tiles per CTA, plus about three tiles' worth of set-up).  With heads x CTAs below
  // the SM count a single round can leave many SMs idle (40 heads x 3 CTAs on 148 SMs); several rounds of shorter
  // CTAs are then faster, as long as a chunk keeps 24 tiles or more so that the set-up remains small.
  {
    const int sms = sm_count();
    int best_k = 1;
    long best_cost = -1;
    for (int k = 1; k <= row_tiles; ++k) {
      const int per = (row_tiles + k - 1) / k;
      if ((long)k * a.BH > sms && per < 24) break;          // several rounds only with chunks of 24 tiles or more
      const long rounds = ((long)k * a.BH + sms - 1) / sms;
      const long cost = rounds * (per + 3);
      if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_k = k; }
    }
    p.ctas_per_head = best_k;
  }
  p.phi = a.phi; p.ldphi = a.ldphi; p.xnorm = a.xnorm; p.mu2 = a.mu2; p.assign = a.assign;
  p.sums = a.sums; p.counts = a.counts; p.fx_shift = a.fx_shift; p.flagged = a.flagged; p.flag_count = a.flag_count; p.err = a.err;
  p.prev_changed = a.prev_changed; p.cur_changed = a.cur_changed; p.flag_count_next = a.flag_count_next;
  // the three kernels of a pass (assignment, exact recheck, new centroids) follow each other with programmatic
  // dependent launches: 48 short dependent launches per k-means run otherwise pay their launch latency one by one
  launch_pdl(k_kmeans_assign_tc, dim3(p.ctas_per_head, a.BH), dim3(kKmThreads), kKmSmemBytes, st, mxh, mxl, mmh, mml, p);
  const size_t rs = recheck_staged_smem(a.C, a.R);
  const int per_head = std::max(1, 2 * sm_count() / a.BH);
  if (rs <= kRecheckSmemMax)
    launch_pdl(k_assign_recheck_staged, dim3(per_head, a.BH), dim3(256), rs, st, a.flagged, a.flag_count, a.phi, a.ldphi, a.N, a.r, a.R, a.mu, a.C,
               a.assign, a.sums, a.counts, a.fx_shift, a.recheck_total, (int)(a.prev_changed == nullptr), a.cur_changed);
  else
    k_assign_recheck<<<dim3(std::max(1, 4 * sm_count() / a.BH), a.BH), 256, 0, st>>>(a.flagged, a.flag_count, a.phi, a.ldphi, a.N, a.r, a.R, a.mu, a.C,
                                                                                     a.assign, a.sums, a.counts, a.fx_shift, a.recheck_total,
                                                                                     a.prev_changed == nullptr, a.cur_changed);
  return true;
}

}  // namespace spr
