// float32 attention kernels on the CUDA cores: block-sparse attention with
// renormalised hard drop (Eq. 3) over the group-major layout, dense attention
// (Eq. 1), and the exact probe rows with their retained/omitted statistics
// (Appendix A.1).  These are the kernels of the float32 configuration (whose
// 1e-5 tolerance rules out reduced-precision tensor-core inputs) and the
// fallback shapes of the bf16 path.
#include "kernels.cuh"

namespace spr {

constexpr int BM = 64;     // query rows per CTA
constexpr int BN = 64;     // keys per tile
constexpr float kLog2e = 1.4426950408889634f;

template <int D> struct SimtSmem {
  static constexpr int q = D * BM, k = D * BN, v = BN * D, p = BN * BM;
  static constexpr size_t bytes = (size_t)(q + k + v + p) * sizeof(float) + 64 * sizeof(int);
};

// Transposed tile load: dst[(c)*64 + r] = src_row_r[c]; rows given by a row-pointer functor.
template <typename T, int D, typename RowPtr>
__device__ __forceinline__ void load_tile_transposed(float* dst, RowPtr rowptr) {
  const int r = threadIdx.x & 63;
  const T* p = rowptr(r);
#pragma unroll
  for (int pass = 0; pass < D / 32; ++pass) {
    const int c = ((threadIdx.x >> 6) + 4 * pass) * 8;
    float v[8];
    if (p) load8(p + c, v);
    else {
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = 0.f;
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) dst[(c + k) * 64 + r] = v[k];
  }
}
template <typename T, int D, typename RowPtr>
__device__ __forceinline__ void load_tile_natural(float* dst, RowPtr rowptr) {
  // 64 rows x D: thread handles 8 consecutive elements; consecutive threads -> consecutive chunks of a row
  constexpr int CPR = D / 8;
#pragma unroll
  for (int e = threadIdx.x; e < 64 * CPR; e += 256) {
    const int r = e / CPR, c = (e % CPR) * 8;
    const T* p = rowptr(r);
    float v[8];
    if (p) load8(p + c, v);
    else {
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = 0.f;
    }
    *reinterpret_cast<float4*>(dst + r * D + c) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(dst + r * D + c + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
}

// S[4][4] = Q_tile (rows ty*4..) . K_tile^T (cols tx*4..)
template <int D>
__device__ __forceinline__ void qk_tile(const float* Qs, const float* Ks, int ty, int tx, float (&s)[4][4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
#pragma unroll 8
  for (int k = 0; k < D; ++k) {
    const float4 a = *reinterpret_cast<const float4*>(Qs + k * BM + ty * 4);
    const float4 b = *reinterpret_cast<const float4*>(Ks + k * BN + tx * 4);
    const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) s[i][j] = fmaf(av[i], bv[j], s[i][j]);
  }
}

// O[4][D/16] += P^T-tile (Ps[j][rows]) . V_tile
template <int D>
__device__ __forceinline__ void pv_tile(const float* Ps, const float* Vs, int ty, int tx, int ncols, float (&o)[4][D / 16]) {
  constexpr int OC = D / 16;
  for (int j = 0; j < ncols; ++j) {
    const float4 p = *reinterpret_cast<const float4*>(Ps + j * BM + ty * 4);
    const float pv[4] = {p.x, p.y, p.z, p.w};
    float vv[OC];
#pragma unroll
    for (int c = 0; c < OC; c += 4) {
      const float4 v = *reinterpret_cast<const float4*>(Vs + j * D + tx * OC + c);
      vv[c] = v.x; vv[c + 1] = v.y; vv[c + 2] = v.z; vv[c + 3] = v.w;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int c = 0; c < OC; ++c) o[i][c] = fmaf(pv[i], vv[c], o[i][c]);
  }
}

__device__ __forceinline__ float row16_max(float v) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float row16_sum(float v) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// =============================================================================
// Main kernel.  SPARSE: one CTA per 64-row tile of one query group; the keys of
// the routed K/V groups are streamed as one concatenated sequence (every tile is
// full except the last).  Dense: one CTA per 64 rows over all keys.  Epilogue:
// O_hat = O_sp + (O_sp A + c) (the affine map of Eq. 9 composed into one matrix),
// stored at the original token index.
// =============================================================================
template <typename T, int D, bool SPARSE>
__global__ void __launch_bounds__(256) k_attention_simt(AttnArgs a) {
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;
  float* Ks = Qs + SimtSmem<D>::q;
  float* Vs = Ks + SimtSmem<D>::k;
  float* Ps = Vs + SimtSmem<D>::v;
  int* krow = reinterpret_cast<int*>(Ps + SimtSmem<D>::p);     // [64] source row of every tile key
  __shared__ int cum[SPARSE ? kMaxGroups + 1 : 1];
  __shared__ int scratch[34];
  constexpr int OC = D / 16;
  const int bh = blockIdx.y, b = bh / a.H, h = bh % a.H;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;

  int row0, nrows, nroute = 0, L;
  const int* ridx = nullptr;
  const int* kvoff = nullptr;
  const T *Qb, *Kb, *Vb;
  i64 qsn, ksn, vsn;
  if (SPARSE) {
    const int* toff = a.tile_off + (i64)bh * (a.Cq + 1);
    if ((int)blockIdx.x >= toff[a.Cq]) return;
    int lo = 0, hi = a.Cq - 1;                      // last group g with toff[g] <= blockIdx.x
    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (toff[mid] <= (int)blockIdx.x) lo = mid; else hi = mid - 1; }
    const int g = lo;
    const int* qoff = a.q_off + (i64)bh * (a.Cq + 1);
    row0 = qoff[g] + ((int)blockIdx.x - toff[g]) * BM;
    nrows = min(BM, qoff[g + 1] - row0);
    const int* rp = a.route_ptr + (i64)bh * (a.Cq + 1);
    ridx = a.route_idx + (i64)bh * a.Cq * a.Ck + rp[g];
    nroute = rp[g + 1] - rp[g];
    kvoff = a.kv_off + (i64)bh * (a.Ck + 1);
    for (int t = tid; t < nroute; t += 256) { const int bb = ridx[t]; cum[t] = kvoff[bb + 1] - kvoff[bb]; }
    __syncthreads();
    L = block_exclusive_scan(cum, nroute, scratch);
    if (tid == 0) cum[nroute] = L;
    Qb = (const T*)a.Q + (i64)bh * a.N * D; Kb = (const T*)a.K + (i64)bh * a.N * D; Vb = (const T*)a.V + (i64)bh * a.N * D;
    qsn = ksn = vsn = D;
  } else {
    row0 = blockIdx.x * BM;
    nrows = min(BM, a.N - row0);
    L = a.N;
    Qb = (const T*)a.Q + b * a.qs[0] + h * a.qs[1]; Kb = (const T*)a.K + b * a.ks[0] + h * a.ks[1];
    Vb = (const T*)a.V + b * a.vs[0] + h * a.vs[1];
    qsn = a.qs[2]; ksn = a.ks[2]; vsn = a.vs[2];
  }
  load_tile_transposed<T, D>(Qs, [&](int r) { return r < nrows ? Qb + (i64)(row0 + r) * qsn : (const T*)nullptr; });

  float o[4][OC], m[4], l[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m[i] = -INFINITY; l[i] = 0.f;
#pragma unroll
    for (int c = 0; c < OC; ++c) o[i][c] = 0.f;
  }
  const float sc = a.scale * kLog2e;
  for (int t0 = 0; t0 < L; t0 += BN) {
    const int ncols = min(BN, L - t0);
    __syncthreads();                                   // previous tile fully consumed
    if (tid < BN) {
      int src = -1;
      if (tid < ncols) {
        if (SPARSE) {
          const int pos = t0 + tid;
          int lo = 0, hi = nroute - 1;                 // last range with cum[range] <= pos
          while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (cum[mid] <= pos) lo = mid; else hi = mid - 1; }
          src = kvoff[ridx[lo]] + (pos - cum[lo]);
        } else src = t0 + tid;
      }
      krow[tid] = src;
    }
    __syncthreads();
    load_tile_transposed<T, D>(Ks, [&](int r) { return krow[r] >= 0 ? Kb + (i64)krow[r] * ksn : (const T*)nullptr; });
    load_tile_natural<T, D>(Vs, [&](int r) { return krow[r] >= 0 ? Vb + (i64)krow[r] * vsn : (const T*)nullptr; });
    __syncthreads();
    float s[4][4];
    qk_tile<D>(Qs, Ks, ty, tx, s);
    float corr[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        s[i][j] = (tx * 4 + j < ncols) ? s[i][j] * sc : -INFINITY;
        mx = fmaxf(mx, s[i][j]);
      }
      mx = row16_max(mx);
      const float mn = fmaxf(m[i], mx);
      corr[i] = exp2f(m[i] - mn);                      // 0 on the first tile (m = -inf)
      m[i] = mn;
      float ps = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) { s[i][j] = exp2f(s[i][j] - mn); ps += s[i][j]; }
      l[i] = l[i] * corr[i] + ps;
#pragma unroll
      for (int c = 0; c < OC; ++c) o[i][c] *= corr[i];
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
      *reinterpret_cast<float4*>(Ps + (tx * 4 + j) * BM + ty * 4) = make_float4(s[0][j], s[1][j], s[2][j], s[3][j]);
    __syncthreads();
    pv_tile<D>(Ps, Vs, ty, tx, ncols, o);
  }
  // ---- epilogue -------------------------------------------------------------------
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float tot = row16_sum(l[i]);
    const float inv = tot > 0.f ? 1.f / tot : 0.f;
#pragma unroll
    for (int c = 0; c < OC; ++c) o[i][c] *= inv;
  }
  float res[4][OC];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int c = 0; c < OC; ++c) res[i][c] = o[i][c];
  if (a.A != nullptr) {
    __syncthreads();
    float* Os = Qs;                                    // [BM][D]
    float* As = Ks;                                    // [D][D] spans the K and V tiles
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int c = 0; c < OC; ++c) Os[(ty * 4 + i) * D + tx * OC + c] = o[i][c];
    const float* Ah = a.A + (i64)bh * D * D;
    for (int e = tid * 4; e < D * D; e += 1024) *reinterpret_cast<float4*>(As + e) = *reinterpret_cast<const float4*>(Ah + e);
    __syncthreads();
    const float* ch = a.c + (i64)bh * D;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int c = 0; c < OC; ++c) res[i][c] += ch[tx * OC + c];
    for (int k = 0; k < D; ++k) {
      float av[OC];
#pragma unroll
      for (int c = 0; c < OC; c += 4) {
        const float4 v = *reinterpret_cast<const float4*>(As + k * D + tx * OC + c);
        av[c] = v.x; av[c + 1] = v.y; av[c + 2] = v.z; av[c + 3] = v.w;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float x = Os[(ty * 4 + i) * D + k];
#pragma unroll
        for (int c = 0; c < OC; ++c) res[i][c] = fmaf(x, av[c], res[i][c]);
      }
    }
  }
  T* Ob = (T*)a.O + b * a.os[0] + h * a.os[1];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = ty * 4 + i;
    if (r >= nrows) continue;
    const int dst = SPARSE ? a.q_perm[(i64)bh * a.N + row0 + r] : row0 + r;
    T* op = Ob + (i64)dst * a.os[2] + tx * OC;
#pragma unroll
    for (int c = 0; c < OC; ++c) op[c] = from_f32<T>(res[i][c]);
    if (a.O_sparse) {
      float* sp = a.O_sparse + ((i64)bh * a.N + dst) * D + tx * OC;
#pragma unroll
      for (int c = 0; c < OC; ++c) sp[c] = o[i][c];
    }
  }
}

// tiles per query group: ceil(n / tile_rows), or, with small_rem > 0, without the last tile when it
// would hold at most small_rem rows (those rows belong to the remainder kernel)
__global__ void __launch_bounds__(1024) k_tile_offsets(const int* __restrict__ q_off, int Cq, int tile_rows, int small_rem,
                                                       int* __restrict__ tile_off) {
  __shared__ int cnt[kMaxGroups];
  __shared__ int scratch[34];
  const int bh = blockIdx.x;
  const int* qo = q_off + (i64)bh * (Cq + 1);
  for (int a = threadIdx.x; a < Cq; a += blockDim.x) {
    const int n = qo[a + 1] - qo[a], rem = n % tile_rows;
    cnt[a] = n / tile_rows + (rem > small_rem ? 1 : 0);
  }
  __syncthreads();
  const int total = block_exclusive_scan(cnt, Cq, scratch);
  for (int a = threadIdx.x; a < Cq; a += blockDim.x) tile_off[(i64)bh * (Cq + 1) + a] = cnt[a];
  if (threadIdx.x == 0) tile_off[(i64)bh * (Cq + 1) + Cq] = total;
}
void launch_tile_offsets(const int* q_off, int BH, int Cq, int tile_rows, int small_rem, int* tile_off, cudaStream_t st) {
  k_tile_offsets<<<BH, 1024, 0, st>>>(q_off, Cq, tile_rows, small_rem, tile_off);
}

template <typename T, int D>
static void attention_dispatch(const AttnArgs& a, cudaStream_t st) {
  if (a.route_ptr) {
    dim3 grid((a.N + BM - 1) / BM + a.Cq, a.BH);
    k_attention_simt<T, D, true><<<grid, 256, SimtSmem<D>::bytes, st>>>(a);
  } else {
    dim3 grid((a.N + BM - 1) / BM, a.BH);
    k_attention_simt<T, D, false><<<grid, 256, SimtSmem<D>::bytes, st>>>(a);
  }
}
void launch_attention_simt(const AttnArgs& a, cudaStream_t st) {
  if (a.dtype == SPARSEPR_BF16) { if (a.d == 128) attention_dispatch<__nv_bfloat16, 128>(a, st); else attention_dispatch<__nv_bfloat16, 64>(a, st); }
  else { if (a.d == 128) attention_dispatch<float, 128>(a, st); else attention_dispatch<float, 64>(a, st); }
}

// =============================================================================
// Probe rows (Appendix A.1-A.2).  For each probe p one pass over ALL keys keeps two
// online-softmax states: the keys retained by p's query group (Z_S, N_S) and the
// omitted ones (Z_U, N_U).  Then O_sp = N_S/Z_S and O_dense = (N_S+N_U)/(Z_S+Z_U).
// The key range is split across CTAs; partial states are merged afterwards.
// partial layout: [BH][n_split][M][2][D+2] = (m, l, N[D]) for the S and the U state.
// =============================================================================
template <typename T, int D>
__global__ void __launch_bounds__(256) k_probe_rows(ProbeArgs a) {
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;
  float* Ks = Qs + SimtSmem<D>::q;
  float* Vs = Ks + SimtSmem<D>::k;
  float* Ps = Vs + SimtSmem<D>::v;                           // retained weights
  float* Pu = Ps + SimtSmem<D>::p;                           // omitted weights
  unsigned* bitmap = reinterpret_cast<unsigned*>(Pu + SimtSmem<D>::p);   // [64][words]
  const int words = (a.Ck + 31) / 32;
  int* kgrp = reinterpret_cast<int*>(bitmap + 64 * words);   // [64] K/V group of every tile key
  constexpr int OC = D / 16;
  const int bh = blockIdx.z, b = bh / a.H, h = bh % a.H;
  const int m0 = blockIdx.y * BM, nrows = min(BM, a.M - m0);
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int* pidx = a.probe_idx + (i64)bh * a.M + m0;
  const T* Qb = (const T*)a.Q + b * a.qs[0] + h * a.qs[1];
  const T* Kb = (const T*)a.Kg + (i64)bh * a.N * D;
  const T* Vb = (const T*)a.Vg + (i64)bh * a.N * D;
  const int* kvoff = a.kv_off + (i64)bh * (a.Ck + 1);

  for (int e = tid; e < 64 * words; e += 256) bitmap[e] = 0u;
  __syncthreads();
  for (int r = tid >> 2; r < nrows; r += 64) {               // 4 threads per probe row
    const int pi = pidx[r];
    if (pi < 0) continue;
    const int g = a.q_assign[(i64)bh * a.N + pi];
    const int* rp = a.route_ptr + (i64)bh * (a.Cq + 1);
    const int* ri = a.route_idx + (i64)bh * a.Cq * a.Ck;
    for (int t = rp[g] + (tid & 3); t < rp[g + 1]; t += 4) atomicOr(&bitmap[r * words + (ri[t] >> 5)], 1u << (ri[t] & 31));
  }
  load_tile_transposed<T, D>(Qs, [&](int r) { return (r < nrows && pidx[r] >= 0) ? Qb + (i64)pidx[r] * a.qs[2] : (const T*)nullptr; });

  // key positions of this split, in whole tiles
  const int tiles = (a.N + BN - 1) / BN;
  const int per = (tiles + a.n_split - 1) / a.n_split;
  const int k_begin = min(a.N, (int)blockIdx.x * per * BN), k_end = min(a.N, ((int)blockIdx.x + 1) * per * BN);

  float oS[4][OC], oU[4][OC], mS[4], lS[4], mU[4], lU[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    mS[i] = mU[i] = -INFINITY; lS[i] = lU[i] = 0.f;
#pragma unroll
    for (int c = 0; c < OC; ++c) oS[i][c] = oU[i][c] = 0.f;
  }
  const float sc = a.scale * kLog2e;
  for (int t0 = k_begin; t0 < k_end; t0 += BN) {
    const int ncols = min(BN, k_end - t0);
    __syncthreads();
    if (tid < BN) {
      int g = 0;
      if (tid < ncols) {
        const int pos = t0 + tid;
        int lo = 0, hi = a.Ck - 1;                     // last group with kvoff[g] <= pos
        while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (kvoff[mid] <= pos) lo = mid; else hi = mid - 1; }
        g = lo;
      }
      kgrp[tid] = g;
    }
    load_tile_transposed<T, D>(Ks, [&](int r) { return r < ncols ? Kb + (i64)(t0 + r) * D : (const T*)nullptr; });
    load_tile_natural<T, D>(Vs, [&](int r) { return r < ncols ? Vb + (i64)(t0 + r) * D : (const T*)nullptr; });
    __syncthreads();
    float s[4][4];
    qk_tile<D>(Qs, Ks, ty, tx, s);
    int grp[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) grp[j] = kgrp[tx * 4 + j];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const unsigned* bm = bitmap + (ty * 4 + i) * words;
      bool ret[4];
      float mxS = -INFINITY, mxU = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool valid = tx * 4 + j < ncols;
        ret[j] = (bm[grp[j] >> 5] >> (grp[j] & 31)) & 1u;
        s[i][j] = valid ? s[i][j] * sc : -INFINITY;
        if (ret[j]) mxS = fmaxf(mxS, s[i][j]); else mxU = fmaxf(mxU, s[i][j]);
      }
      mxS = row16_max(mxS); mxU = row16_max(mxU);
      const float nS = fmaxf(mS[i], mxS), nU = fmaxf(mU[i], mxU);
      const float cS = nS == -INFINITY ? 1.f : exp2f(mS[i] - nS), cU = nU == -INFINITY ? 1.f : exp2f(mU[i] - nU);
      mS[i] = nS; mU[i] = nU;
      float pS[4], pU[4], sS = 0.f, sU = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float e = exp2f(s[i][j] - (ret[j] ? nS : nU));       // -inf logit -> 0
        const bool live = s[i][j] > -INFINITY;
        pS[j] = (live && ret[j]) ? e : 0.f;
        pU[j] = (live && !ret[j]) ? e : 0.f;
        sS += pS[j]; sU += pU[j];
      }
      lS[i] = lS[i] * cS + sS; lU[i] = lU[i] * cU + sU;
#pragma unroll
      for (int c = 0; c < OC; ++c) { oS[i][c] *= cS; oU[i][c] *= cU; }
#pragma unroll
      for (int j = 0; j < 4; ++j) { Ps[(tx * 4 + j) * BM + ty * 4 + i] = pS[j]; Pu[(tx * 4 + j) * BM + ty * 4 + i] = pU[j]; }
    }
    __syncthreads();
    pv_tile<D>(Ps, Vs, ty, tx, ncols, oS);
    pv_tile<D>(Pu, Vs, ty, tx, ncols, oU);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = ty * 4 + i;
    const float tS = row16_sum(lS[i]), tU = row16_sum(lU[i]);
    if (r >= nrows) continue;
    float* out = a.partial + ((((i64)bh * a.n_split + blockIdx.x) * a.M + m0 + r) * 2) * (D + 2);
    if (tx == 0) { out[0] = mS[i]; out[1] = tS; out[D + 2] = mU[i]; out[D + 3] = tU; }
#pragma unroll
    for (int c = 0; c < OC; ++c) { out[2 + tx * OC + c] = oS[i][c]; out[D + 4 + tx * OC + c] = oU[i][c]; }
  }
}

// merge the split states; one warp per probe row
template <int D>
__global__ void __launch_bounds__(256) k_probe_merge(const float* __restrict__ partial, int n_split, int M,
                                                     float* __restrict__ X, float* __restrict__ Dn) {
  const int bh = blockIdx.y;
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (r >= M) return;
  const int lane = threadIdx.x & 31;
  constexpr int PL = D / 32;
  float mS = -INFINITY, mU = -INFINITY;
  for (int s = 0; s < n_split; ++s) {
    const float* p = partial + ((((i64)bh * n_split + s) * M + r) * 2) * (D + 2);
    mS = fmaxf(mS, p[0]); mU = fmaxf(mU, p[D + 2]);
  }
  float lS = 0.f, lU = 0.f, nS[PL], nU[PL];
#pragma unroll
  for (int c = 0; c < PL; ++c) nS[c] = nU[c] = 0.f;
  for (int s = 0; s < n_split; ++s) {
    const float* p = partial + ((((i64)bh * n_split + s) * M + r) * 2) * (D + 2);
    const float wS = p[0] == -INFINITY ? 0.f : exp2f(p[0] - mS), wU = p[D + 2] == -INFINITY ? 0.f : exp2f(p[D + 2] - mU);
    // a state without any key (empty key slice, or no retained / omitted key inside it) has weight 0 and its
    // numerator may never have been written: it is skipped, not multiplied by 0
    if (wS != 0.f) {
      lS += p[1] * wS;
#pragma unroll
      for (int c = 0; c < PL; ++c) nS[c] += p[2 + lane + 32 * c] * wS;
    }
    if (wU != 0.f) {
      lU += p[D + 3] * wU;
#pragma unroll
      for (int c = 0; c < PL; ++c) nU[c] += p[D + 4 + lane + 32 * c] * wU;
    }
  }
  const float mD = fmaxf(mS, mU);
  const float eS = mS == -INFINITY ? 0.f : exp2f(mS - mD), eU = mU == -INFINITY ? 0.f : exp2f(mU - mD);
  const float zD = lS * eS + lU * eU;
#pragma unroll
  for (int c = 0; c < PL; ++c) {
    X[((i64)bh * M + r) * D + lane + 32 * c] = lS > 0.f ? nS[c] / lS : 0.f;
    Dn[((i64)bh * M + r) * D + lane + 32 * c] = zD > 0.f ? (nS[c] * eS + nU[c] * eU) / zD : 0.f;
  }
}

template <int D> static size_t probe_smem_bytes(int Ck) {
  return (size_t)(SimtSmem<D>::q + SimtSmem<D>::k + SimtSmem<D>::v + 2 * SimtSmem<D>::p) * sizeof(float) +
         (size_t)64 * ((Ck + 31) / 32) * sizeof(unsigned) + 64 * sizeof(int);
}
size_t probe_partial_floats(int BH, int n_split, int M, int d) { return (size_t)BH * n_split * M * 2 * (d + 2); }

template <typename T, int D>
static void probe_dispatch(const ProbeArgs& a, cudaStream_t st) {
  dim3 grid(a.n_split, (a.M + BM - 1) / BM, a.BH);
  k_probe_rows<T, D><<<grid, 256, probe_smem_bytes<D>(a.Ck), st>>>(a);
  dim3 g2((a.M + 7) / 8, a.BH);
  k_probe_merge<D><<<g2, 256, 0, st>>>(a.partial, a.n_split, a.M, a.X, a.Dn);
}
void launch_probe_merge(const ProbeArgs& a, cudaStream_t st) {
  dim3 g2((a.M + 7) / 8, a.BH);
  if (a.d == 128) k_probe_merge<128><<<g2, 256, 0, st>>>(a.partial, a.n_split, a.M, a.X, a.Dn);
  else k_probe_merge<64><<<g2, 256, 0, st>>>(a.partial, a.n_split, a.M, a.X, a.Dn);
}
void launch_probe_rows(const ProbeArgs& a, cudaStream_t st) {
  if (a.dtype == SPARSEPR_BF16) { if (a.d == 128) probe_dispatch<__nv_bfloat16, 128>(a, st); else probe_dispatch<__nv_bfloat16, 64>(a, st); }
  else { if (a.d == 128) probe_dispatch<float, 128>(a, st); else probe_dispatch<float, 64>(a, st); }
}

// O[b,h,probe_idx[m],:] = O_dense of the probe (Eq. 10, first case)
template <typename T>
__global__ void k_write_probe_rows(const float* __restrict__ Dn, const int* __restrict__ probe_idx, int H, int M, int d,
                                   T* __restrict__ O, i64 ob, i64 oh, i64 on) {
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < M * d; e += gridDim.x * blockDim.x) {
    const int m = e / d, c = e % d;
    const int pi = probe_idx[(i64)bh * M + m];
    if (pi >= 0) O[b * ob + h * oh + (i64)pi * on + c] = from_f32<T>(Dn[((i64)bh * M + m) * d + c]);
  }
}
void launch_write_probe_rows(int dtype, const float* Dn, const int* probe_idx, int BH, int H, int M, int d, void* O,
                             const i64* os, cudaStream_t st) {
  dim3 grid((M * d + 255) / 256, BH);
  if (dtype == SPARSEPR_BF16) k_write_probe_rows<__nv_bfloat16><<<grid, 256, 0, st>>>(Dn, probe_idx, H, M, d, (__nv_bfloat16*)O, os[0], os[1], os[2]);
  else k_write_probe_rows<float><<<grid, 256, 0, st>>>(Dn, probe_idx, H, M, d, (float*)O, os[0], os[1], os[2]);
}

cudaError_t init_attention_simt() {
  cudaError_t e;
#define SPR_ATTR(KERN, BYTES) if ((e = cudaFuncSetAttribute(KERN, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(BYTES))) != cudaSuccess) return e
  SPR_ATTR((k_attention_simt<float, 128, true>), SimtSmem<128>::bytes);
  SPR_ATTR((k_attention_simt<float, 128, false>), SimtSmem<128>::bytes);
  SPR_ATTR((k_attention_simt<float, 64, true>), SimtSmem<64>::bytes);
  SPR_ATTR((k_attention_simt<float, 64, false>), SimtSmem<64>::bytes);
  SPR_ATTR((k_attention_simt<__nv_bfloat16, 128, true>), SimtSmem<128>::bytes);
  SPR_ATTR((k_attention_simt<__nv_bfloat16, 128, false>), SimtSmem<128>::bytes);
  SPR_ATTR((k_attention_simt<__nv_bfloat16, 64, true>), SimtSmem<64>::bytes);
  SPR_ATTR((k_attention_simt<__nv_bfloat16, 64, false>), SimtSmem<64>::bytes);
  SPR_ATTR((k_probe_rows<float, 128>), probe_smem_bytes<128>(kMaxGroups));
  SPR_ATTR((k_probe_rows<float, 64>), probe_smem_bytes<64>(kMaxGroups));
  SPR_ATTR((k_probe_rows<__nv_bfloat16, 128>), probe_smem_bytes<128>(kMaxGroups));
  SPR_ATTR((k_probe_rows<__nv_bfloat16, 64>), probe_smem_bytes<64>(kMaxGroups));
#undef SPR_ATTR
  return cudaSuccess;
}

}  // namespace spr
