// Block-sparse attention (Eq. 3) for the short remainders of the query groups (bf16, d = d_v = 128).
//
// A query group of n rows gives floor(n / 128) full tiles to the 128-row kernel; when the n mod 128 rows
// that are left are at most kRemRows they come here.  An M = 128 tensor-core tile for a handful of rows
// costs as much as a full one, and rows of different groups attend to different keys, so the
// remainders of MANY groups are packed into common 128-row tiles instead: such a tile walks over the keys of
// every K/V group that any of its rows routes to (group-major order) and every row masks the groups that its
// own query group does not route to.  At a routed density of 25 % and 16-row remainders that is about a third of the
// tile passes that one tile per remainder needs.
//
//   warps 0-7  softmax: warps w and w+4 share the 32 rows of TMEM quadrant w and split the 128 scores
//              of a row in two halves; they also bring the query rows into tensor memory (the rows of a
//              packed tile are scattered, so there is no TMA box for them)
//   warp  8    K producer: streams the K/V groups that some row of the tile routes to, as one sequence of 16-row
//              boxes (tiles of 128 keys, every box inside one group), and publishes the group of every box;
//   warp  10   V producer
//   warp  9    issues Q K^T (one thread); owns the TMEM allocation;  warp 11 issues P V (one thread)
// TMEM: S_0 [0,128), S_1 [128,256), P [256,320), O [320,448), Q [448,512); both products take their A
// operand from tensor memory.  Reference maxima move lazily (growth beyond 2^8), as in the 128-row kernel.
// Every mbarrier wait is bounded; on expiry the CTA records SPARSEPR_ERR_TIMEOUT and leaves.
#include <cuda.h>
#include "kernels.cuh"
#include "tc_common.cuh"

namespace spr {
namespace tc {
namespace packed {

constexpr int kThreads = 384;
constexpr int kPolyOf8 = 3;                           // pairs of every 8 whose exponential is a polynomial on the FMA pipe
constexpr int kTile = 128;
constexpr int kD = 128;
constexpr int kSub = 16;                               // rows per TMA box of the K/V stream
constexpr int kSubPerTile = kTile / kSub;
constexpr uint32_t kHalfBytes = kTile * 128;          // [128 rows x 64 bf16]
constexpr uint32_t kTileBytes = 2 * kHalfBytes;       // 32 KB
constexpr uint32_t kSubBytes = kSub * 128;
constexpr int kStages = 2;

// per key tile: number of boxes, valid rows of every box (4 bits each, minus one), K/V group of every box
struct Meta { uint32_t cnt_bits, nsub; unsigned short grp[kSubPerTile]; uint32_t pad[2]; };   // 32 bytes

struct Smem {
  static constexpr uint32_t k = 0;
  static constexpr uint32_t v = k + kStages * kTileBytes;
  static constexpr uint32_t bitmap = v + kStages * kTileBytes;           // [kMaxGroups/32 words][128 rows]
  static constexpr uint32_t uni = bitmap + (kMaxGroups / 32) * 128 * 4;  // [kMaxGroups/32] union of the rows' route bitmaps
  static constexpr uint32_t ranges = uni + (kMaxGroups / 32) * 4;        // int2[kMaxGroups] (start, length) of the wanted K/V groups
  static constexpr uint32_t gid = ranges + kMaxGroups * 8;               // unsigned short[kMaxGroups] their group ids
  static constexpr uint32_t idx = gid + kMaxGroups * 2;                  // int[kMaxGroups] scan scratch
  static constexpr uint32_t xchg = idx + kMaxGroups * 4;                 // float [2][2][128] half-row maxima, [2][128] half-row sums
  static constexpr uint32_t meta = xchg + 6 * 128 * 4;                   // Meta[8]
  static constexpr uint32_t bars = meta + 8 * 32;
  static constexpr uint32_t misc = bars + 32 * 8;
  static constexpr uint32_t total = misc + 256;
};
static_assert(Smem::total <= 227 * 1024, "shared memory");
enum Bar { Q_FULL = 0, K_FULL = 1, K_EMPTY = K_FULL + kStages, V_FULL = K_EMPTY + kStages, V_EMPTY = V_FULL + kStages,
           S_FULL = V_EMPTY + kStages, S_FREE = S_FULL + 2, P_FULL = S_FREE + 2, P_EMPTY, O_DONE, META_FULL, kNumBars = META_FULL + 8 };
static_assert(kNumBars <= 32, "barrier area");

struct Maps { CUtensorMap m[4]; };      // the same tensor with boxes of 16, 32, 64 and 128 rows

struct Params {
  int BH, H, N, Cq, Ck;
  int kv_div;                                  // query heads per K/V head: Kg, Vg and kv_off are indexed by bh / kv_div
  float scale_log2;
  const int *rem_pos, *rem_grp, *rem_cnt;      // [BH][N] group-major position and query group of every packed row; [BH] their number
  const int *kv_off, *route_ptr, *route_idx, *q_perm;
  const __nv_bfloat16* Qg;                     // [BH][N][128] group-major
  __nv_bfloat16* O; i64 os[3];
  float* O_sparse;
  __nv_bfloat16* O_lo;             // optional [BH][N][128]: o - bf16(o), original order (second word for the correction pass)
  int* err;
};

__global__ void __launch_bounds__(kThreads, 1)
k_attention_packed(const __grid_constant__ Maps mapsK, const __grid_constant__ Maps mapsV, Params prm) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char* sm = smem_raw;
  unsigned* bitmap = reinterpret_cast<unsigned*>(sm + Smem::bitmap);
  unsigned* uni = reinterpret_cast<unsigned*>(sm + Smem::uni);
  int2* ranges = reinterpret_cast<int2*>(sm + Smem::ranges);
  unsigned short* gid = reinterpret_cast<unsigned short*>(sm + Smem::gid);
  int* idx = reinterpret_cast<int*>(sm + Smem::idx);
  float* xmax = reinterpret_cast<float*>(sm + Smem::xchg);
  float* xsum = xmax + 4 * 128;
  Meta* meta = reinterpret_cast<Meta*>(sm + Smem::meta);
  volatile int* misc = reinterpret_cast<volatile int*>(sm + Smem::misc);   // [0] tmem, [1] abort, [2] boxes, [3] skip, [8..41] scan scratch
  const uint32_t bars = base + Smem::bars;
  auto bar = [&](int i) { return bars + 8u * i; };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y, m0 = blockIdx.x * kTile;
  const int cnt = prm.rem_cnt[bh];
  if (m0 >= cnt) return;
  const int nrows = min(kTile, cnt - m0);
  if (tid == 0) {
    misc[3] = (prm.err != nullptr && *reinterpret_cast<volatile int*>(prm.err) == SPARSEPR_ERR_TIMEOUT) || (base & 1023u) != 0;
    if ((base & 1023u) != 0) set_error(prm.err, SPARSEPR_ERR_CUDA);
  }
  __syncthreads();
  if (misc[3]) return;
  const int words = (prm.Ck + 31) / 32;
  const int* rpos = prm.rem_pos + (i64)bh * prm.N + m0;
  const int* rgrp = prm.rem_grp + (i64)bh * prm.N + m0;
  const int kvh = bh / prm.kv_div;
  const int* kvoff = prm.kv_off + (i64)kvh * (prm.Ck + 1);

  if (tid == 0) {
    for (int i = 0; i < kNumBars; ++i) mbar_init(bar(i), (i == P_FULL || i == Q_FULL || i == S_FREE || i == S_FREE + 1) ? 256 : 1);
    misc[1] = 0; misc[2] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) tmem_alloc(base + Smem::misc, 512);
  // route bitmap of every row of the tile, transposed: bitmap[word][row]
  for (int e = tid; e < words * 128; e += kThreads) bitmap[e] = 0u;
  __syncthreads();
  for (int r = tid >> 1; r < nrows; r += kThreads / 2) {
    const int g = rgrp[r];
    const int* rp = prm.route_ptr + (i64)bh * (prm.Cq + 1);
    const int* ri = prm.route_idx + (i64)bh * prm.Cq * prm.Ck;
    for (int t = rp[g] + (tid & 1); t < rp[g + 1]; t += 2) atomicOr(&bitmap[(ri[t] >> 5) * 128 + r], 1u << (ri[t] & 31));
  }
  __syncthreads();
  // the K/V groups that some row routes to, in order: they are streamed, the others are not even loaded
  for (int w = tid; w < words; w += kThreads) {
    unsigned u = 0u;
    for (int r = 0; r < nrows; ++r) u |= bitmap[w * 128 + r];
    uni[w] = u;
  }
  __syncthreads();
  for (int g = tid; g < prm.Ck; g += kThreads) idx[g] = (((uni[g >> 5] >> (g & 31)) & 1u) && kvoff[g + 1] > kvoff[g]) ? 1 : 0;
  __syncthreads();
  const int nroute = block_exclusive_scan(idx, prm.Ck, const_cast<int*>(misc + 8));
  __syncthreads();
  {
    int boxes = 0;
    for (int g = tid; g < prm.Ck; g += kThreads) {
      const int start = kvoff[g], len = kvoff[g + 1] - start;
      if (((uni[g >> 5] >> (g & 31)) & 1u) && len > 0) {
        ranges[idx[g]] = make_int2(start, len);
        gid[idx[g]] = (unsigned short)g;
        boxes += (len + kSub - 1) / kSub;
      }
    }
    boxes = warp_sum(boxes);
    if (lane == 0 && boxes) atomicAdd((int*)&misc[2], boxes);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = (uint32_t)misc[0];
  const int total_boxes = misc[2];
  const int n_tiles = (total_boxes + kSubPerTile - 1) / kSubPerTile;
  volatile int* abort_flag = &misc[1];

  if (warp == 8 || warp == 10) {
    // =========================== TMA producers ==========================================
    // All lanes of a producer walk the wanted key ranges together (uniform); lane j issues the copies of box j.
    if (n_tiles > 0) {
      const bool is_k = warp == 8;
      const int full0 = is_k ? K_FULL : V_FULL, empty0 = is_k ? K_EMPTY : V_EMPTY;
      const uint32_t buf0 = base + (is_k ? Smem::k : Smem::v);
      const Maps* maps = is_k ? &mapsK : &mapsV;
      int ri = 0, off = 0;
      bool ok = true;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int s = i % kStages;
        const uint32_t ph = ((i / kStages) & 1) ^ 1;         // empty barriers: the first pass completes immediately
        // up to 8 boxes of 16 rows; consecutive boxes of one group form a segment, fetched by one copy per set bit
        // of its box count (128, 64, 32 or 16 rows), largest first
        int my_start = 0, my_gid = 0, my_t = 0, my_n = 0, nsub = 0;
        uint32_t cnt_bits = 0;
        while (nsub < kSubPerTile && ri < nroute) {
          const int2 rg = ranges[ri];
          const int left = rg.y - off, nb = (left + kSub - 1) / kSub;
          const int n = min(kSubPerTile - nsub, nb);
          if (lane >= nsub && lane < nsub + n) { my_t = lane - nsub; my_n = n; my_start = rg.x + off + my_t * kSub; my_gid = gid[ri]; }
          uint32_t bits = n == 8 ? 0xFFFFFFFFu : ((1u << (4 * n)) - 1u);
          if (n == nb) {
            const int sh = 4 * (n - 1);
            bits = (bits & ~(0xFu << sh)) | ((uint32_t)(left - (n - 1) * kSub - 1) << sh);
            ++ri; off = 0;
          } else {
            off += n * kSub;
          }
          cnt_bits |= bits << (4 * nsub);
          nsub += n;
        }
        int my_k = -1;
#pragma unroll
        for (int kb = 0; kb < 4; ++kb)
          if (lane < nsub && ((my_n >> kb) & 1) && my_t == ((my_n >> (kb + 1)) << (kb + 1))) my_k = kb;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(empty0 + s), ph, abort_flag));
        if (!ok) break;
        if (is_k) {
          if (lane < kSubPerTile) meta[i & 7].grp[lane] = (unsigned short)my_gid;
          if (lane == 0) { meta[i & 7].cnt_bits = cnt_bits; meta[i & 7].nsub = (uint32_t)nsub; }
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(META_FULL + (i & 7)));
        }
        if (lane == 0) mbar_expect_tx(bar(full0 + s), nsub * 2 * kSubBytes);
        __syncwarp();
        if (my_k >= 0) {
          const uint32_t dst = buf0 + s * kTileBytes + lane * kSubBytes;
          tma_load_4d(dst, &maps->m[my_k], bar(full0 + s), 0, my_start, kvh, 0);
          tma_load_4d(dst + kHalfBytes, &maps->m[my_k], bar(full0 + s), 64, my_start, kvh, 0);
        }
      }
    }
  } else if (warp == 9) {
    // =========================== Q K^T issuer (the two products are issued by two threads) ====
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_bf16(0, 128);
      const uint64_t k_desc0 = smem_desc(base + Smem::k, 16);
      bool ok = mbar_wait(bar(Q_FULL), 0, abort_flag);
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int s = i % kStages;
        // score buffer i mod 2 is free once every softmax thread holds tile i - 2 in registers
        if (i >= 2 && !mbar_wait(bar(S_FREE + (i & 1)), ((i - 2) >> 1) & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(bar(K_FULL + s), (i / kStages) & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d = tmem + (uint32_t)(i & 1) * 128u;
        const uint64_t kd = k_desc0 + (uint64_t)(s * (kTileBytes >> 4));
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint64_t koff = (uint64_t)((kk >> 2) * (kHalfBytes >> 4) + (kk & 3) * 2);
          umma_bf16_ts(d, tmem + 448u + kk * 8, kd + koff, idesc_qk, kk > 0);
        }
        umma_commit(bar(K_EMPTY + s));
        umma_commit(bar(S_FULL + (i & 1)));
      }
    }
  } else if (warp == 11) {
    // =========================== P V issuer ==================================================
    if (lane == 0) {
      const uint32_t idesc_pv = idesc_bf16(1, 128);
      const uint64_t v_desc0 = smem_desc(base + Smem::v, kHalfBytes);
      bool ok = true;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int s = i % kStages;
        if (!mbar_wait(bar(META_FULL + (i & 7)), (i >> 3) & 1, abort_flag)) { ok = false; break; }
        const int nsub = (int)meta[i & 7].nsub;
        if (!mbar_wait(bar(V_FULL + s), (i / kStages) & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(bar(P_FULL), i & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint64_t vd = v_desc0 + (uint64_t)(s * (kTileBytes >> 4));
#pragma unroll
        for (int kk = 0; kk < kSubPerTile; ++kk)
          if (kk < nsub)
            umma_bf16_ts(tmem + 320u, tmem + 256u + kk * 8, vd + (uint64_t)(kk * (kSubBytes >> 4)), idesc_pv, (i > 0 || kk > 0) ? 1u : 0u);
        umma_commit(bar(V_EMPTY + s));
        umma_commit(bar(P_EMPTY));
      }
      if (ok) umma_commit(bar(O_DONE));                        // completes at once when there was no tile
    }
  } else if (warp < 8) {
    // =========================== softmax (warps 0-7) =======================================
    const int hh = warp >> 2, wq = warp & 3;
    const int row = wq * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
    const uint32_t FULL = 0xffffffffu;
    const uint32_t p_addr = tmem + lane_addr + 256u + (uint32_t)hh * 32u;
    const uint32_t o_addr = tmem + lane_addr + 320u + (uint32_t)hh * 64u;
    const float sc = prm.scale_log2;
    const int my_pos = row < nrows ? rpos[row] : -1;
    // this thread's half (64 of 128 dimensions) of its query row goes to tensor memory, two bf16 per column
    {
      uint32_t qw[32];
      if (my_pos >= 0) {
        const uint4* qp = reinterpret_cast<const uint4*>(prm.Qg + ((i64)bh * prm.N + my_pos) * kD + hh * 64);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint4 u = qp[c];
          qw[4 * c] = u.x; qw[4 * c + 1] = u.y; qw[4 * c + 2] = u.z; qw[4 * c + 3] = u.w;
        }
      } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) qw[c] = 0u;
      }
      tmem_st32u(tmem + lane_addr + 448u + (uint32_t)hh * 32u, qw);
      tc_fence_before();
      mbar_arrive(bar(Q_FULL));
    }
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int i = 0; i < n_tiles; ++i) {
      // the barriers of this tile are polled back to back (their shared-memory round trips overlap)
      const bool t_meta = mbar_try(bar(META_FULL + (i & 7)), (i >> 3) & 1);
      const bool t_s = mbar_try(bar(S_FULL + (i & 1)), (i >> 1) & 1);
      {
        bool w = ok;
        if (!t_meta) w = w && mbar_wait(bar(META_FULL + (i & 7)), (i >> 3) & 1, abort_flag);
        if (!t_s) w = w && mbar_wait(bar(S_FULL + (i & 1)), (i >> 1) & 1, abort_flag);
        ok = __all_sync(FULL, w);
      }
      float s[64];
      float mx = -INFINITY;
      bool lim_neg[4] = {true, true, true, true};              // box bx holds no key that this row may see
      if (ok) {
        tc_fence_after();
        const Meta& mt = meta[i & 7];
        const uint32_t cnt_bits = mt.cnt_bits;
        const int nsub = (int)mt.nsub;
        const uint32_t s_addr = tmem + lane_addr + (uint32_t)(i & 1) * 128u + (uint32_t)hh * 64u;
        tmem_ld32_nowait(s_addr, *reinterpret_cast<float(*)[32]>(&s[0]));
        tmem_ld32_nowait(s_addr + 32, *reinterpret_cast<float(*)[32]>(&s[32]));
        // a box counts for this row when its K/V group is routed by the row's query group; lim = its last valid column
        int lim[4];
#pragma unroll
        for (int bx = 0; bx < 4; ++bx) {
          const int box = hh * 4 + bx;
          lim[bx] = -1;
          if (box < nsub) {
            const int g = mt.grp[box];
            if ((bitmap[(g >> 5) * 128 + row] >> (g & 31)) & 1u) lim[bx] = (int)((cnt_bits >> (4 * box)) & 15u);
          }
        }
        tmem_ld_wait();
        tc_fence_before();
        mbar_arrive(bar(S_FREE + (i & 1)));                         // the scores are in registers
#pragma unroll
        for (int bx = 0; bx < 4; ++bx) {
          lim_neg[bx] = lim[bx] < 0;
#pragma unroll
          for (int c = 0; c < 16; ++c) s[bx * 16 + c] = (c <= lim[bx]) ? s[bx * 16 + c] : -INFINITY;
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int c = 0; c < 64; c += 8) {
          mx4[0] = max3(mx4[0], s[c], s[c + 1]); mx4[1] = max3(mx4[1], s[c + 2], s[c + 3]);
          mx4[2] = max3(mx4[2], s[c + 4], s[c + 5]); mx4[3] = max3(mx4[3], s[c + 6], s[c + 7]);
        }
        mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      }
      // the two halves of the row exchange their maxima (buffer of this tile's parity; executed whatever happened)
      float* xm = xmax + (i & 1) * 256;
      xm[hh * 128 + row] = mx;
      asm volatile("bar.sync %0, 64;" ::"r"(1 + wq) : "memory");
      mx = fmaxf(mx, xm[(hh ^ 1) * 128 + row]);
      const bool move = mx > -INFINITY && (mx - m_ref) * sc > 8.f;     // a row without any routed key so far keeps -inf
      const float m_new = move ? mx : m_ref;
      const float corr = move ? ex2((m_ref - m_new) * sc) : 1.f;      // 0 when the reference was -inf
      const float mneg = m_new > -INFINITY ? -m_new * sc : 0.f;
      // O has to be rescaled only for a row that already holds something: a row that meets its first routed key in
      // this tile (rows of a packed tile do so at different tiles) still has an all-zero accumulator
      const bool rescale = move && m_ref > -INFINITY;
      m_ref = m_new;
      // The product P V of the previous tile must be complete before P (a single buffer) is overwritten, and before O
      // is rescaled.  The rescale is rare, so the wait normally comes after the exponentials, which then run while
      // the tensor cores still work on the previous tile.
      bool p_free = i == 0;
      if (!__all_sync(FULL, ok)) { ok = false; continue; }
      if (i > 0 && __any_sync(FULL, rescale)) {
        ok = __all_sync(FULL, mbar_wait(bar(P_EMPTY), (i - 1) & 1, abort_flag));
        if (!ok) continue;
        p_free = true;
        tc_fence_after();
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float t[32];
          tmem_ld32(o_addr + q * 32, t);
#pragma unroll
          for (int c = 0; c < 32; ++c) t[c] *= corr;
          tmem_st32(o_addr + q * 32, t);
        }
      }
      // exponentials: kPolyOf8 of every 8 pairs on the FMA pipe, the others on the special-function unit;
      // masked columns give exactly 0 on both.  A box that no row of this warp routes to (a warp holds the
      // remainders of few query groups, and a group routes to a fraction of the K/V groups) is all zeros:
      // its exponentials are skipped for the whole warp.
      float2 ps2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      const float2 sc2 = make_float2(sc, sc), mneg2 = make_float2(mneg, mneg);
#pragma unroll
      for (int bx = 0; bx < 4; ++bx) {
        if (__all_sync(FULL, lim_neg[bx])) {
#pragma unroll
          for (int c = 0; c < 16; ++c) s[bx * 16 + c] = 0.f;
        } else {
#pragma unroll
          for (int q = bx * 8; q < bx * 8 + 8; ++q) {
            float2 x = __ffma2_rn(make_float2(s[2 * q], s[2 * q + 1]), sc2, mneg2);
            if ((q & 7) < kPolyOf8) x = ex2_poly2(x);
            else { x.x = ex2(x.x); x.y = ex2(x.y); }
            s[2 * q] = x.x; s[2 * q + 1] = x.y;
            ps2[q & 1] = __fadd2_rn(ps2[q & 1], x);
          }
        }
      }
      l = l * corr + ((ps2[0].x + ps2[0].y) + (ps2[1].x + ps2[1].y));
      {
        uint32_t w[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) w[c] = pack_bf16x2(s[2 * c], s[2 * c + 1]);
        if (!p_free) {
          ok = __all_sync(FULL, mbar_wait(bar(P_EMPTY), (i - 1) & 1, abort_flag));
          if (!ok) continue;
          tc_fence_after();
        }
        tmem_st32u(p_addr, w);
      }
      tc_fence_before();
      mbar_arrive(bar(P_FULL));
    }
    // ---- row sums of the two halves, normalise, store ------------------------------------------
    ok = __all_sync(FULL, ok && mbar_wait(bar(O_DONE), 0, abort_flag));
    xsum[hh * 128 + row] = l;
    asm volatile("bar.sync %0, 64;" ::"r"(1 + wq) : "memory");
    const float ltot = l + xsum[(hh ^ 1) * 128 + row];
    const float inv = ltot > 0.f ? 1.f / ltot : 0.f;
    if (ok) {
      tc_fence_after();
      float o[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) o[c] = 0.f;
      if (n_tiles > 0) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float t[32];
          tmem_ld32(o_addr + q * 32, t);
#pragma unroll
          for (int c = 0; c < 32; ++c) o[q * 32 + c] = inv != 0.f ? t[c] * inv : 0.f;
        }
      }
      if (my_pos >= 0) {
        const int dst = prm.q_perm[(i64)bh * prm.N + my_pos];
        const int b = bh / prm.H, h = bh % prm.H;
        __nv_bfloat16* op = prm.O + b * prm.os[0] + h * prm.os[1] + (i64)dst * prm.os[2] + hh * 64;
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          float v8[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) v8[k] = o[ch * 8 + k];
          store8(op + ch * 8, v8);
        }
        if (prm.O_lo) {                                        // what the bf16 rounding above dropped
          __nv_bfloat16* lp = prm.O_lo + ((i64)bh * prm.N + dst) * kD + hh * 64;
#pragma unroll
          for (int ch = 0; ch < 8; ++ch) {
            float v8[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) v8[k] = o[ch * 8 + k] - __bfloat162float(__float2bfloat16_rn(o[ch * 8 + k]));
            store8(lp + ch * 8, v8);
          }
        }
        if (prm.O_sparse) {
          float* sp = prm.O_sparse + ((i64)bh * prm.N + dst) * kD + hh * 64;
#pragma unroll
          for (int ch = 0; ch < 8; ++ch) {
            float v8[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) v8[k] = o[ch * 8 + k];
            store8(sp + ch * 8, v8);
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
    tmem_dealloc(tmem, 512);
  }
}

// The rows of the short remainders of one head: rem_pos = group-major position, rem_grp = query group; rem_cnt =
// their number.  One CTA per head.  The groups are taken in the order (number of routed K/V groups descending, first
// routed K/V group ascending, id): a packed tile streams the union of the routes of the ~8 groups it holds, and groups
// that route alike then share a tile (about a third fewer key tiles than in id order on the benchmark workloads).
__global__ void __launch_bounds__(1024) k_remainder_rows(const int* __restrict__ q_off, const int* __restrict__ route_ptr,
                                                         const int* __restrict__ route_idx, int Cq, int Ck, int N, int rem_rows,
                                                         int* __restrict__ rem_pos, int* __restrict__ rem_grp,
                                                         int* __restrict__ rem_cnt) {
  __shared__ unsigned long long key[kMaxGroups];
  __shared__ int cnt[kMaxGroups];
  __shared__ int scratch[34];
  const int bh = blockIdx.x;
  const int* qo = q_off + (i64)bh * (Cq + 1);
  const int* rp = route_ptr + (i64)bh * (Cq + 1);
  const int* ri = route_idx + (i64)bh * Cq * Ck;
  int P = 1;
  while (P < Cq) P <<= 1;
  for (int a = threadIdx.x; a < P; a += blockDim.x) {
    unsigned long long k = ~0ull;                               // groups without a short remainder sort to the end
    if (a < Cq) {
      const int rem = (qo[a + 1] - qo[a]) % 128;
      if (rem > 0 && rem <= rem_rows) {
        const int n = rp[a + 1] - rp[a];
        const int first = n > 0 ? ri[rp[a]] : 0;
        k = ((unsigned long long)(Ck - n) << 24) | ((unsigned long long)first << 12) | (unsigned long long)a;
      }
    }
    key[a] = k;
  }
  __syncthreads();
  // bitonic sort, ascending
  for (int size = 2; size <= P; size <<= 1)
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = threadIdx.x; t < P / 2; t += blockDim.x) {
        const int lo = 2 * t - (t & (stride - 1)), hi = lo + stride;
        const bool up = (lo & size) == 0;
        const unsigned long long x = key[lo], y = key[hi];
        if ((x > y) == up) { key[lo] = y; key[hi] = x; }
      }
      __syncthreads();
    }
  for (int s = threadIdx.x; s < Cq; s += blockDim.x) {
    const unsigned long long k = key[s];
    int c = 0;
    if (k != ~0ull) { const int a = (int)(k & 0xFFFull); c = (qo[a + 1] - qo[a]) % 128; }
    cnt[s] = c;
  }
  __syncthreads();
  const int total = block_exclusive_scan(cnt, Cq, scratch);
  __syncthreads();
  for (int s = threadIdx.x >> 5; s < Cq; s += blockDim.x >> 5) {
    const unsigned long long k = key[s];
    if (k == ~0ull) continue;
    const int a = (int)(k & 0xFFFull);
    const int rem = (qo[a + 1] - qo[a]) % 128;
    for (int j = threadIdx.x & 31; j < rem; j += 32) {
      rem_pos[(i64)bh * N + cnt[s] + j] = qo[a + 1] - rem + j;
      rem_grp[(i64)bh * N + cnt[s] + j] = a;
    }
  }
  if (threadIdx.x == 0) rem_cnt[bh] = total;
}

}  // namespace packed
}  // namespace tc

cudaError_t init_attention_packed() {
  return cudaFuncSetAttribute(tc::packed::k_attention_packed, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::packed::Smem::total);
}

void launch_remainder_rows(const int* q_off, const int* route_ptr, const int* route_idx, int BH, int Cq, int Ck, int N, int* rem_pos,
                           int* rem_grp, int* rem_cnt, cudaStream_t st) {
  tc::packed::k_remainder_rows<<<BH, 1024, 0, st>>>(q_off, route_ptr, route_idx, Cq, Ck, N, kRemRows, rem_pos, rem_grp, rem_cnt);
}

// Short remainders of every query group, packed (the 128-row kernel must have been given tile offsets that leave
// them out).  Q, K, V group-major [BH][N][128] bf16; rem_* from launch_remainder_rows.
bool launch_attention_packed(const AttnArgs& a, const int* rem_pos, const int* rem_grp, const int* rem_cnt, cudaStream_t st) {
  using namespace tc;
  using namespace tc::packed;
  Maps mk, mv;
  const int kvd = a.kv_div < 1 ? 1 : a.kv_div;
  for (int k = 0; k < 4; ++k)
    if (!make_map(&mk.m[k], a.K, kD, a.N, a.BH / kvd, 1, 0, (i64)a.N * kD, kD, kSub << k) ||
        !make_map(&mv.m[k], a.V, kD, a.N, a.BH / kvd, 1, 0, (i64)a.N * kD, kD, kSub << k))
      return false;
  Params p{};
  p.kv_div = kvd;
  p.BH = a.BH; p.H = a.H; p.N = a.N; p.Cq = a.Cq; p.Ck = a.Ck; p.scale_log2 = a.scale * 1.4426950408889634f;
  p.rem_pos = rem_pos; p.rem_grp = rem_grp; p.rem_cnt = rem_cnt;
  p.kv_off = a.kv_off; p.route_ptr = a.route_ptr; p.route_idx = a.route_idx; p.q_perm = a.q_perm;
  p.Qg = (const __nv_bfloat16*)a.Q;
  p.O = (__nv_bfloat16*)a.O; for (int i = 0; i < 3; ++i) p.os[i] = a.os[i];
  p.O_sparse = a.O_sparse; p.O_lo = (__nv_bfloat16*)a.O_lo; p.err = a.err;
  // a group contributes at most kRemRows of every 128 rows it has beyond a multiple of 128, so the packed rows of a
  // head never exceed N; CTAs past the head's count return at once
  const int tiles = (a.N + kTile - 1) / kTile;
  k_attention_packed<<<dim3(tiles, a.BH), kThreads, Smem::total, st>>>(mk, mv, p);
  return true;
}

}  // namespace spr
