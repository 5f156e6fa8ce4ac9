// Exact probe rows on the tensor cores (Appendix A.1-A.2; bf16, d = d_v = 128).
//
// For every probe row one pass over ALL keys (group-major order) maintains two
// online-softmax states: the keys retained by the probe's query group (Z_S, N_S) and the
// omitted ones (Z_U, N_U).  From them O_sp = N_S / Z_S and
// O_dense = (N_S + N_U) / (Z_S + Z_U).  A CTA owns 128 probe rows and one slice of the key
// range; partial states are merged by k_probe_merge.
//   warps 0-7  softmax: warps w and w + 4 share the 32 probe rows of TMEM quadrant w and split the 128 scores of a
//              row in two halves (every score belongs to one of the two states, so a half costs half the work;
//              with one warp per scheduler the loop ran at the latency of its instructions)
//   warp  8    K producer (also builds the per-tile list of K/V-group runs), warp 9 V producer
//   warp  10   tcgen05.mma issuer, owns TMEM
// TMEM: S0 [0,128), S1 [128,256), O_S [256,384), O_U [384,512).  The exponentials of a tile
// are written back over its score buffer as bf16: retained weights in columns [0,64),
// omitted weights in [64,128); the two P V products read them from TMEM.
#include "kernels.cuh"
#include "tc_common.cuh"

namespace spr {
namespace tc {

constexpr int kPbThreads = 352;
constexpr int kPbWarpK = 8, kPbWarpV = 9, kPbWarpMma = 10;
constexpr int kPbTile = 128;
constexpr uint32_t kPbHalf = 128 * 128;              // [128 rows x 64 bf16] swizzled block
constexpr uint32_t kPbTileBytes = 2 * kPbHalf;
constexpr int kPbKStages = 2, kPbVStages = 2;
constexpr int kPbMaxRuns = 8;                        // K/V-group runs per key tile

struct PbMeta { int ncols, nruns; unsigned short grp[kPbMaxRuns]; unsigned char end[kPbMaxRuns]; };   // 32 bytes

struct PbSmem {
  static constexpr uint32_t q = 0;
  static constexpr uint32_t k = q + kPbTileBytes;
  static constexpr uint32_t v = k + kPbKStages * kPbTileBytes;
  static constexpr uint32_t bitmap = v + kPbVStages * kPbTileBytes;        // [kMaxGroups/32 words][128 rows]
  static constexpr uint32_t meta = bitmap + (kMaxGroups / 32) * 128 * 4;   // PbMeta[8]
  static constexpr uint32_t xchg = meta + 8 * 32;                          // float [2][2][2][128] half-row maxima of both states, [2][2][128] sums
  static constexpr uint32_t bars = xchg + 12 * 128 * 4;
  static constexpr uint32_t misc = bars + 32 * 8;
  static constexpr uint32_t total = misc + 64;
};
enum PbBar { PQ_FULL = 0, PK_FULL = 1, PK_EMPTY = PK_FULL + kPbKStages, PV_FULL = PK_EMPTY + kPbKStages,
             PV_EMPTY = PV_FULL + kPbVStages, PS_FULL = PV_EMPTY + kPbVStages, PP_FULL = PS_FULL + 2, PT_DONE = PP_FULL + 2,
             PMETA_FULL, kPbNumBars = PMETA_FULL + 8 };
static_assert(kPbNumBars <= 32, "barrier area");

struct PbParams {
  int BH, N, M, Ck, Cq, n_split;
  int kv_div;                     // query heads per K/V head: the K/V maps and kv_off are indexed by bh / kv_div
  float scale_log2;
  const int *probe_idx, *q_assign, *kv_off, *route_ptr, *route_idx;
  float* partial;                 // [BH][n_split][M][2][130]
  int* err;
};

__global__ void __launch_bounds__(kPbThreads, 1)
k_probe_rows_tc(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                const __grid_constant__ CUtensorMap mapV, PbParams prm) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char* sm = smem_raw;
  unsigned* bitmap = reinterpret_cast<unsigned*>(sm + PbSmem::bitmap);
  PbMeta* meta = reinterpret_cast<PbMeta*>(sm + PbSmem::meta);
  volatile int* misc = reinterpret_cast<volatile int*>(sm + PbSmem::misc);   // [0] tmem, [1] abort, [3] skip
  const uint32_t bars = base + PbSmem::bars;
  auto bar = [&](int i) { return bars + 8u * i; };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, m0 = blockIdx.y * kPbTile, bh = blockIdx.z;
  if (tid == 0) {
    misc[3] = (prm.err != nullptr && *reinterpret_cast<volatile int*>(prm.err) == SPARSEPR_ERR_TIMEOUT) || (base & 1023u) != 0;
    if ((base & 1023u) != 0) set_error(prm.err, SPARSEPR_ERR_CUDA);
  }
  __syncthreads();
  if (misc[3]) return;

  // key positions of this slice (whole tiles of 128)
  const int tiles_all = (prm.N + kPbTile - 1) / kPbTile;
  const int per = (tiles_all + prm.n_split - 1) / prm.n_split;
  const int p_begin = min(prm.N, split * per * kPbTile), p_end = min(prm.N, (split + 1) * per * kPbTile);
  const int nrows = min(kPbTile, prm.M - m0);
  const int words = (prm.Ck + 31) / 32;

  if (tid == 0) {
    for (int i = 0; i < kPbNumBars; ++i) mbar_init(bar(i), (i == PP_FULL || i == PP_FULL + 1) ? 256 : 1);
    misc[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kPbWarpMma) tmem_alloc(base + PbSmem::misc, 512);
  // route bitmap of every probe row, transposed: bitmap[word][row]
  for (int e = tid; e < words * 128; e += kPbThreads) bitmap[e] = 0u;
  __syncthreads();
  for (int r = tid >> 1; r < nrows; r += kPbThreads / 2) {
    const int pi = prm.probe_idx[(i64)bh * prm.M + m0 + r];
    if (pi < 0) continue;
    const int g = prm.q_assign[(i64)bh * prm.N + pi];
    const int* rp = prm.route_ptr + (i64)bh * (prm.Cq + 1);
    const int* ri = prm.route_idx + (i64)bh * prm.Cq * prm.Ck;
    for (int t = rp[g] + (tid & 1); t < rp[g + 1]; t += 2) atomicOr(&bitmap[(ri[t] >> 5) * 128 + r], 1u << (ri[t] & 31));
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = (uint32_t)misc[0];
  volatile int* abort_flag = &misc[1];
  const int kvh = bh / prm.kv_div;
  const int* kvoff = prm.kv_off + (i64)kvh * (prm.Ck + 1);

  // Tiles are cut so that none spans more than kPbMaxRuns K/V groups; every role walks the same
  // sequence of (start position, columns) with this function.  `g` = group that contains `pos`.
  auto next_tile = [&](int pos, int& g, PbMeta* out) -> int {
    int runs = 0, c = 0;
    while (c < kPbTile && pos + c < p_end && runs < kPbMaxRuns) {
      while (kvoff[g + 1] <= pos + c) ++g;                        // skip empty groups
      const int e = min(min(kvoff[g + 1], p_end) - pos, kPbTile);
      if (out) { out->grp[runs] = (unsigned short)g; out->end[runs] = (unsigned char)(e - 1); }
      c = e;
      ++runs;
    }
    if (out) { out->ncols = c; out->nruns = runs; }
    return c;
  };

  if (warp == kPbWarpK || warp == kPbWarpV) {
    // =========================== producers ==================================================
    if (lane == 0 && p_begin < p_end) {
      const bool is_k = warp == kPbWarpK;
      if (is_k) {
        mbar_expect_tx(bar(PQ_FULL), kPbTileBytes);
        tma_load_4d(base + PbSmem::q, &mapQ, bar(PQ_FULL), 0, m0, bh, 0);
        tma_load_4d(base + PbSmem::q + kPbHalf, &mapQ, bar(PQ_FULL), 64, m0, bh, 0);
      }
      const int nst = is_k ? kPbKStages : kPbVStages;
      const int full0 = is_k ? PK_FULL : PV_FULL, empty0 = is_k ? PK_EMPTY : PV_EMPTY;
      const uint32_t buf0 = base + (is_k ? PbSmem::k : PbSmem::v);
      const CUtensorMap* map = is_k ? &mapK : &mapV;
      int g = 0;
      { int lo = 0, hi = prm.Ck - 1; while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (kvoff[mid] <= p_begin) lo = mid; else hi = mid - 1; } g = lo; }
      int pos = p_begin;
      for (int i = 0; pos < p_end; ++i) {
        const int s = i % nst;
        PbMeta mt;
        const int nc = next_tile(pos, g, &mt);
        if (!mbar_wait(bar(empty0 + s), ((i / nst) & 1) ^ 1, abort_flag)) break;
        if (is_k) {
          meta[i & 7] = mt;
          mbar_arrive(bar(PMETA_FULL + (i & 7)));
        }
        mbar_expect_tx(bar(full0 + s), kPbTileBytes);
        tma_load_4d(buf0 + s * kPbTileBytes, map, bar(full0 + s), 0, pos, kvh, 0);
        tma_load_4d(buf0 + s * kPbTileBytes + kPbHalf, map, bar(full0 + s), 64, pos, kvh, 0);
        pos += nc;
      }
    }
  } else if (warp == kPbWarpMma) {
    // =========================== MMA issuer ==================================================
    if (lane == 0 && p_begin < p_end) {
      const uint32_t idesc_qk = idesc_bf16(0, 128), idesc_pv = idesc_bf16(1, 128);
      bool ok = mbar_wait(bar(PQ_FULL), 0, abort_flag);
      auto issue_qk = [&](int i) -> bool {
        const int s = i % kPbKStages;
        if (!mbar_wait(bar(PK_FULL + s), (i / kPbKStages) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint32_t d = tmem + (uint32_t)(i & 1) * 128u;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t koff = (kk >> 2) * kPbHalf + (kk & 3) * 32;
          umma_bf16(d, smem_desc(base + PbSmem::q + koff, 16), smem_desc(base + PbSmem::k + s * kPbTileBytes + koff, 16), idesc_qk, kk > 0);
        }
        umma_commit(bar(PK_EMPTY + s));
        umma_commit(bar(PS_FULL + (i & 1)));
        return true;
      };
      // number of tiles of this slice (same walk as the producers)
      int n_tiles = 0;
      {
        int g = 0;
        { int lo = 0, hi = prm.Ck - 1; while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (kvoff[mid] <= p_begin) lo = mid; else hi = mid - 1; } g = lo; }
        for (int pos = p_begin; pos < p_end; ++n_tiles) pos += next_tile(pos, g, nullptr);
      }
      if (ok) ok = issue_qk(0);
      for (int i = 0; i < n_tiles && ok; ++i) {
        if (i + 1 < n_tiles) { ok = issue_qk(i + 1); if (!ok) break; }    // the other score buffer
        const int s = i % kPbVStages;
        if (!mbar_wait(bar(PV_FULL + s), (i / kPbVStages) & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(bar(PP_FULL + (i & 1)), (i >> 1) & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t pbuf = tmem + (uint32_t)(i & 1) * 128u;
#pragma unroll
        for (int which = 0; which < 2; ++which)                 // retained weights -> O_S, omitted -> O_U
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t bdesc = smem_desc(base + PbSmem::v + s * kPbTileBytes + kk * 2048, kPbHalf);
            umma_bf16_ts(tmem + 256u + which * 128u, pbuf + which * 64u + kk * 8, bdesc, idesc_pv, (i > 0 || kk > 0) ? 1u : 0u);
          }
        umma_commit(bar(PV_EMPTY + s));
        umma_commit(bar(PT_DONE));                              // O_S / O_U hold every tile up to i
      }
    }
  } else if (warp < 8) {
    // =========================== softmax ========================================================
    // Thread (half hh, quadrant wq, lane) owns the scores of keys [64 hh, 64 hh + 64) of probe row 32 wq + lane; the
    // two halves of a row meet at the named barrier 1 + wq to agree on the two maxima of the tile.
    const int hh = warp >> 2, wq = warp & 3;
    const int row = wq * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
    const uint32_t FULL = 0xffffffffu;
    const float sc = prm.scale_log2;
    float* xmax = reinterpret_cast<float*>(sm + PbSmem::xchg);             // [parity][half][state][row]
    float* xsum = xmax + 8 * 128;                                          // [half][state][row]
    float mS = -INFINITY, mU = -INFINITY, lS = 0.f, lU = 0.f;
    bool ok = true;
    int pos = p_begin, i = 0;
    for (; pos < p_end; ++i) {
      ok = __all_sync(FULL, ok && mbar_wait(bar(PS_FULL + (i & 1)), (i >> 1) & 1, abort_flag) &&
                                mbar_wait(bar(PMETA_FULL + (i & 7)), (i >> 3) & 1, abort_flag));
      if (!ok) break;                                           // uniform over the CTA: every softmax warp waits on the same barriers
      tc_fence_after();
      const PbMeta mt = meta[i & 7];
      pos += mt.ncols;
      // column masks of this half (two words of 32): valid (inside the tile) and retained (K/V group routed to this
      // row's query group)
      unsigned ret[2] = {0u, 0u}, val[2];
      {
        int beg = 0;
        for (int r = 0; r < mt.nruns; ++r) {
          const int g = mt.grp[r], e = mt.end[r] + 1;
          const bool on = (bitmap[(g >> 5) * 128 + row] >> (g & 31)) & 1u;
          if (on) {
#pragma unroll
            for (int w = 0; w < 2; ++w) {
              const int w0 = 32 * (2 * hh + w);
              const int lo = max(beg - w0, 0), hi = min(e - w0, 32);
              if (hi > lo) ret[w] |= (hi - lo == 32 ? 0xFFFFFFFFu : ((1u << (hi - lo)) - 1u) << lo);
            }
          }
          beg = e;
        }
#pragma unroll
        for (int w = 0; w < 2; ++w) {
          const int hi = min(mt.ncols - 32 * (2 * hh + w), 32);
          val[w] = hi <= 0 ? 0u : hi == 32 ? 0xFFFFFFFFu : (1u << hi) - 1u;
        }
      }
      const uint32_t s_addr = tmem + lane_addr + (uint32_t)(i & 1) * 128u;
      float s[64];
      tmem_ld32_nowait(s_addr + 64 * hh, *reinterpret_cast<float(*)[32]>(&s[0]));
      tmem_ld32_nowait(s_addr + 64 * hh + 32, *reinterpret_cast<float(*)[32]>(&s[32]));
      tmem_ld_wait();
      float mxS = -INFINITY, mxU = -INFINITY;
#pragma unroll
      for (int c = 0; c < 64; ++c) {
        const bool v = (val[c >> 5] >> (c & 31)) & 1u, r = (ret[c >> 5] >> (c & 31)) & 1u;
        s[c] = v ? s[c] : -INFINITY;
        mxS = fmaxf(mxS, r ? s[c] : -INFINITY);
        mxU = fmaxf(mxU, r ? -INFINITY : s[c]);
      }
      // the halves exchange their maxima; past this barrier both hold their scores in registers, so the weights
      // may be written over the score buffer
      {
        float* xm = xmax + (i & 1) * 512;
        xm[(hh * 2 + 0) * 128 + row] = mxS;
        xm[(hh * 2 + 1) * 128 + row] = mxU;
        asm volatile("bar.sync %0, 64;" ::"r"(1 + wq) : "memory");
        mxS = fmaxf(mxS, xm[((hh ^ 1) * 2 + 0) * 128 + row]);
        mxU = fmaxf(mxU, xm[((hh ^ 1) * 2 + 1) * 128 + row]);
      }
      // lazily moved reference maxima (see the attention kernel); a state without any key yet keeps -inf
      const bool moveS = mxS > -INFINITY && (mxS - mS) * sc > 8.f, moveU = mxU > -INFINITY && (mxU - mU) * sc > 8.f;
      const float cS = moveS ? ex2((mS - mxS) * sc) : 1.f, cU = moveU ? ex2((mU - mxU) * sc) : 1.f;
      if (moveS) mS = mxS;
      if (moveU) mU = mxU;
      // the accumulators are stable once the previous P V products have completed
      if (i > 0) ok = __all_sync(FULL, ok && mbar_wait(bar(PT_DONE), (i - 1) & 1, abort_flag));
      if (!ok) break;
      if (i > 0 && __any_sync(FULL, moveS || moveU)) {           // rescale this half of the O_S / O_U rows (rare)
        tc_fence_after();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float t[32];
          const float f = q < 2 ? cS : cU;
          const uint32_t a = tmem + lane_addr + 256u + (uint32_t)(q >> 1) * 128u + (uint32_t)hh * 64u + (uint32_t)(q & 1) * 32u;
          tmem_ld32(a, t);
#pragma unroll
          for (int c = 0; c < 32; ++c) t[c] *= f;
          tmem_st32(a, t);
        }
      }
      const float nS = mS > -INFINITY ? -mS * sc : 0.f, nU = mU > -INFINITY ? -mU * sc : 0.f;
      float sumS = 0.f, sumU = 0.f;
      // exponentials, packed in place: afterwards s[2j] holds the bf16 pair of retained weights of
      // columns (2j, 2j+1) of this half and s[2j+1] the pair of omitted weights
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        float eS[2], eU[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int c = 2 * j + u;
          const bool r = (ret[c >> 5] >> (c & 31)) & 1u;
          const float e = ex2(fmaf(s[c], sc, r ? nS : nU));     // masked columns: exp2(-inf) = 0
          eS[u] = r ? e : 0.f;
          eU[u] = r ? 0.f : e;
          sumS += eS[u];
          sumU += eU[u];
        }
        s[2 * j] = __uint_as_float(pack_bf16x2(eS[0], eS[1]));
        s[2 * j + 1] = __uint_as_float(pack_bf16x2(eU[0], eU[1]));
      }
      lS = lS * cS + sumS;
      lU = lU * cU + sumU;
      {
        uint32_t w[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) w[c] = __float_as_uint(s[2 * c]);
        tmem_st32u(s_addr + 32 * hh, w);                        // retained weights of keys [64 hh, 64 hh + 64)
#pragma unroll
        for (int c = 0; c < 32; ++c) w[c] = __float_as_uint(s[2 * c + 1]);
        tmem_st32u(s_addr + 64 + 32 * hh, w);                   // omitted weights
      }
      tc_fence_before();
      mbar_arrive(bar(PP_FULL + (i & 1)));
    }
    // ---- partial states of this slice -----------------------------------------------------------
    const bool any = p_begin < p_end;
    if (any) ok = __all_sync(FULL, ok && i > 0 && mbar_wait(bar(PT_DONE), (i - 1) & 1, abort_flag));
    xsum[(hh * 2 + 0) * 128 + row] = lS;
    xsum[(hh * 2 + 1) * 128 + row] = lU;
    asm volatile("bar.sync %0, 64;" ::"r"(1 + wq) : "memory");
    lS += xsum[((hh ^ 1) * 2 + 0) * 128 + row];
    lU += xsum[((hh ^ 1) * 2 + 1) * 128 + row];
    if (row < nrows && hh == 0) {
      float* out = prm.partial + ((((i64)bh * prm.n_split + split) * prm.M + m0 + row) * 2) * 130;
      const bool good = ok && any;
      out[0] = (good && lS > 0.f) ? mS * sc : -INFINITY; out[1] = good ? lS : 0.f;
      out[130] = (good && lU > 0.f) ? mU * sc : -INFINITY; out[131] = good ? lU : 0.f;
    }
    if (ok && any) {
      tc_fence_after();
#pragma unroll
      for (int q = 0; q < 4; ++q) {                             // this half's 64 columns of O_S, then of O_U
        float t[32];
        tmem_ld32(tmem + lane_addr + 256u + (uint32_t)(q >> 1) * 128u + (uint32_t)hh * 64u + (uint32_t)(q & 1) * 32u, t);
        if (row < nrows) {
          float* out = prm.partial + ((((i64)bh * prm.n_split + split) * prm.M + m0 + row) * 2 + (q >> 1)) * 130 + 2 + hh * 64 + (q & 1) * 32;
#pragma unroll
          for (int c = 0; c < 32; ++c) out[c] = t[c];
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
  if (warp == kPbWarpMma) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// probe rows of Q gathered into a dense [BH][M][128] bf16 buffer (rows of missing probes are zero)
__global__ void k_gather_probe_q(const __nv_bfloat16* __restrict__ Q, i64 sb, i64 sh, i64 sn, int H,
                                 const int* __restrict__ probe_idx, int M, __nv_bfloat16* __restrict__ out) {
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;          // 16 threads per row
  const int m = t >> 4, c = (t & 15) * 8;
  if (m >= M) return;
  const int pi = probe_idx[(i64)bh * M + m];
  uint4 v = make_uint4(0, 0, 0, 0);
  if (pi >= 0) v = *reinterpret_cast<const uint4*>(Q + b * sb + h * sh + (i64)pi * sn + c);
  *reinterpret_cast<uint4*>(out + ((i64)bh * M + m) * 128 + c) = v;
}

}  // namespace tc

cudaError_t init_probe_tc() {
  return cudaFuncSetAttribute(tc::k_probe_rows_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::PbSmem::total);
}
bool probe_tc_supported(const ProbeArgs& a) { return a.dtype == SPARSEPR_BF16 && a.d == 128 && tc::tma_available(); }

// Qp: scratch [BH][M][128] bf16.  Writes a.partial in the layout k_probe_merge reads.
bool launch_probe_rows_tc(const ProbeArgs& a, __nv_bfloat16* Qp, int* err, cudaStream_t st) {
  const int kvd = a.kv_div < 1 ? 1 : a.kv_div;
  using namespace tc;
  k_gather_probe_q<<<dim3((a.M * 16 + 255) / 256, a.BH), 256, 0, st>>>((const __nv_bfloat16*)a.Q, a.qs[0], a.qs[1], a.qs[2], a.H,
                                                                     a.probe_idx, a.M, Qp);
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, Qp, 128, a.M, a.BH, 1, 0, (i64)a.M * 128, 128, 128) ||
      !make_map(&mk, a.Kg, 128, a.N, a.BH / kvd, 1, 0, (i64)a.N * 128, 128, 128) ||
      !make_map(&mv, a.Vg, 128, a.N, a.BH / kvd, 1, 0, (i64)a.N * 128, 128, 128))
    return false;
  PbParams p{};
  p.BH = a.BH; p.N = a.N; p.M = a.M; p.Ck = a.Ck; p.Cq = a.Cq; p.n_split = a.n_split;
  p.scale_log2 = a.scale * 1.4426950408889634f;
  p.kv_div = kvd;
  p.probe_idx = a.probe_idx; p.q_assign = a.q_assign; p.kv_off = a.kv_off; p.route_ptr = a.route_ptr; p.route_idx = a.route_idx;
  p.partial = a.partial; p.err = err;
  k_probe_rows_tc<<<dim3(a.n_split, (a.M + 127) / 128, a.BH), kPbThreads, PbSmem::total, st>>>(mq, mk, mv, p);
  return true;
}

}  // namespace spr
