// Response-Coupled Partitioning kernels (Section 4.1, Appendix B): sampled-query
// Gram matrix, batched Jacobi eigen-decomposition -> feature maps, response
// projections, k-means assignment/update, stable counting sort, group means.
#include <algorithm>
#include "kernels.cuh"

namespace spr {

// =============================================================================
// Gram matrices: M_K = Q_s^T Q_s / M_s (Appendix B.1) and
// M_Q = Ktilde^T Ktilde / (C_k^+ d) (Appendix B.2), float64 accumulation.
// Grid (D/16, heads): a CTA owns 16 rows of the D x D result; thread t owns column
// t % D and 8 consecutive rows.  Input rows are staged in shared memory as doubles.
// =============================================================================
constexpr int kGramChunk = 32;
constexpr int kGramSlab = 16;

template <int D>
__device__ __forceinline__ void gram_accumulate(const double* rows, int nrows, int i0, int j, double (&acc)[8]) {
  for (int s = 0; s < nrows; ++s) {
    const double xj = rows[s * D + j];
    const double* xi = rows + s * D + i0;                 // the same 8 values for the whole half-block: broadcast
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = fma(xi[k], xj, acc[k]);
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(256) k_sample_gram(const T* __restrict__ Q, i64 sb, i64 sh, i64 sn, int H, int N,
                                                     int Ms, u64 seed, int head0, double* __restrict__ Mout) {
  pdl_launch_dependents();                                     // (inputs of this kernel are the caller's)
  __shared__ __align__(16) double rows[kGramChunk * D];
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const T* base = Q + b * sb + h * sh;
  const u64 U = sample_offset(seed, kTagQuerySample, head0 + bh);
  const int j = threadIdx.x % D, i0 = blockIdx.x * kGramSlab + (threadIdx.x / D) * 8;
  const bool active = threadIdx.x < 2 * D;
  double acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  for (int s0 = 0; s0 < Ms; s0 += kGramChunk) {
    const int nr = min(kGramChunk, Ms - s0);
    __syncthreads();
    for (int t = threadIdx.x; t < nr * (D / 8); t += 256) {
      const int s = t / (D / 8), c = t % (D / 8);
      float v[8];
      load8(base + (i64)strided_row(s0 + s, Ms, N, U) * sn + c * 8, v);
#pragma unroll
      for (int k = 0; k < 8; ++k) rows[s * D + c * 8 + k] = (double)v[k];
    }
    __syncthreads();
    if (active) gram_accumulate<D>(rows, nr, i0, j, acc);
  }
  if (active) {
#pragma unroll
    for (int k = 0; k < 8; ++k) Mout[(i64)bh * D * D + (i64)(i0 + k) * D + j] = acc[k] / (double)Ms;
  }
}

// kappa [BH][C][D] float32, n [BH][C] group sizes.  Empty groups are skipped and the
// remaining centroids are centred by their uniform mean.
template <int D>
__global__ void __launch_bounds__(256) k_centroid_gram(const float* __restrict__ kappa, const int* __restrict__ n, int C,
                                                       double* __restrict__ Mout) {
  pdl_wait();                                                   // the group means come from the kernel before
  pdl_launch_dependents();
  __shared__ __align__(16) double rows[kGramChunk * D];
  __shared__ double mean[D];
  __shared__ int s_cnt;
  const int bh = blockIdx.y;
  const float* kp = kappa + (i64)bh * C * D;
  const int* nn = n + (i64)bh * C;
  if (threadIdx.x == 0) s_cnt = 0;
  __syncthreads();
  {
    int c = 0;
    for (int g = threadIdx.x; g < C; g += 256) c += nn[g] > 0;
    c = warp_sum(c);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(&s_cnt, c);
  }
  __syncthreads();
  const int cplus = s_cnt;
  if (threadIdx.x < D) {
    double m = 0.0;
    for (int g = 0; g < C; ++g)
      if (nn[g] > 0) m += (double)kp[(i64)g * D + threadIdx.x];
    mean[threadIdx.x] = cplus > 0 ? m / cplus : 0.0;
  }
  const int j = threadIdx.x % D, i0 = blockIdx.x * kGramSlab + (threadIdx.x / D) * 8;
  const bool active = threadIdx.x < 2 * D;
  double acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  for (int g0 = 0; g0 < C; g0 += kGramChunk) {
    const int nr = min(kGramChunk, C - g0);
    __syncthreads();
    for (int t = threadIdx.x; t < nr * D; t += 256) {
      const int s = t / D, jj = t % D;
      rows[t] = nn[g0 + s] > 0 ? (double)kp[(i64)(g0 + s) * D + jj] - mean[jj] : 0.0;
    }
    __syncthreads();
    if (active) gram_accumulate<D>(rows, nr, i0, j, acc);
  }
  const double denom = cplus > 0 ? (double)cplus * (double)D : 1.0;
  if (active) {
#pragma unroll
    for (int k = 0; k < 8; ++k) Mout[(i64)bh * D * D + (i64)(i0 + k) * D + j] = acc[k] / denom;
  }
}

void launch_sample_gram(int dtype, const void* Q, const i64* qs, int BH, int H, int N, int d, int Ms, u64 seed, int head0,
                        double* Mout, cudaStream_t st) {
  if (dtype == SPARSEPR_BF16) {
    if (d == 128) k_sample_gram<__nv_bfloat16, 128><<<dim3(d / kGramSlab, BH), 256, 0, st>>>((const __nv_bfloat16*)Q, qs[0], qs[1], qs[2], H, N, Ms, seed, head0, Mout);
    else k_sample_gram<__nv_bfloat16, 64><<<dim3(d / kGramSlab, BH), 256, 0, st>>>((const __nv_bfloat16*)Q, qs[0], qs[1], qs[2], H, N, Ms, seed, head0, Mout);
  } else {
    if (d == 128) k_sample_gram<float, 128><<<dim3(d / kGramSlab, BH), 256, 0, st>>>((const float*)Q, qs[0], qs[1], qs[2], H, N, Ms, seed, head0, Mout);
    else k_sample_gram<float, 64><<<dim3(d / kGramSlab, BH), 256, 0, st>>>((const float*)Q, qs[0], qs[1], qs[2], H, N, Ms, seed, head0, Mout);
  }
}
void launch_centroid_gram(const float* kappa, const int* n, int BH, int C, int d, double* Mout, cudaStream_t st) {
  if (d == 128) launch_pdl(k_centroid_gram<128>, dim3(128 / kGramSlab, BH), dim3(256), 0, st, kappa, n, C, Mout);
  else launch_pdl(k_centroid_gram<64>, dim3(64 / kGramSlab, BH), dim3(256), 0, st, kappa, n, C, Mout);
}

// =============================================================================
// Response projections: phi_K = K F_K (Eq. 6) and phi_Q = RMS-normalised Q F_Q
// (Eq. 7).  Each thread produces two rows of R outputs; F is staged in shared
// memory and read by broadcast.  Also tracks max |phi| per head (for the
// fixed-point centroid sums) and flags non-finite values.
// =============================================================================
template <typename T, int D, int R, bool RMS>
__global__ void __launch_bounds__(128) k_project(const T* __restrict__ X, i64 sb, i64 sh, i64 sn, int H, int N, int r,
                                                 const float* __restrict__ F, float eps, float* __restrict__ phi,
                                                 int ldphi, unsigned* __restrict__ maxabs_bits, int* err) {
  __shared__ __align__(16) float Fs[D * R];
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const float* Fh = F + (i64)bh * D * r;
  for (int e = threadIdx.x; e < D * R; e += 128) {
    const int k = e / R, c = e % R;
    Fs[e] = c < r ? Fh[k * r + c] : 0.f;
  }
  __syncthreads();
  const T* base = X + b * sb + h * sh;
  const int row0 = blockIdx.x * 256 + threadIdx.x, row1 = row0 + 128;
  const bool v0 = row0 < N, v1 = row1 < N;
  const T* p0 = base + (i64)(v0 ? row0 : 0) * sn;
  const T* p1 = base + (i64)(v1 ? row1 : 0) * sn;
  float acc0[R], acc1[R];
#pragma unroll
  for (int c = 0; c < R; ++c) { acc0[c] = 0.f; acc1[c] = 0.f; }
  for (int k0 = 0; k0 < D; k0 += 8) {
    float x0[8], x1[8];
    load8(p0 + k0, x0);
    load8(p1 + k0, x1);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      const float4* f4 = reinterpret_cast<const float4*>(Fs + (k0 + kk) * R);
#pragma unroll
      for (int c = 0; c < R / 4; ++c) {
        const float4 f = f4[c];
        acc0[4 * c] = fmaf(x0[kk], f.x, acc0[4 * c]); acc0[4 * c + 1] = fmaf(x0[kk], f.y, acc0[4 * c + 1]);
        acc0[4 * c + 2] = fmaf(x0[kk], f.z, acc0[4 * c + 2]); acc0[4 * c + 3] = fmaf(x0[kk], f.w, acc0[4 * c + 3]);
        acc1[4 * c] = fmaf(x1[kk], f.x, acc1[4 * c]); acc1[4 * c + 1] = fmaf(x1[kk], f.y, acc1[4 * c + 1]);
        acc1[4 * c + 2] = fmaf(x1[kk], f.z, acc1[4 * c + 2]); acc1[4 * c + 3] = fmaf(x1[kk], f.w, acc1[4 * c + 3]);
      }
    }
  }
  float m = 0.f;
  bool bad = false;
  auto finish = [&](float (&acc)[R], int row, bool valid) {
    if (!valid) return;
    if (RMS) {
      float ss = 0.f;
#pragma unroll
      for (int c = 0; c < R; ++c) ss = fmaf(acc[c], acc[c], ss);
      const float inv = 1.f / fmaxf(sqrtf(ss / (float)r), eps);
#pragma unroll
      for (int c = 0; c < R; ++c) acc[c] *= inv;
    }
    float* out = phi + ((i64)bh * N + row) * ldphi;
#pragma unroll
    for (int c = 0; c < R; c += 4)      // columns r..R-1 are written as zeros (ldphi >= R)
      *reinterpret_cast<float4*>(out + c) = make_float4(acc[c], acc[c + 1], acc[c + 2], acc[c + 3]);
#pragma unroll
    for (int c = 0; c < R; ++c) {
      m = fmaxf(m, fabsf(acc[c]));
      bad |= !(fabsf(acc[c]) <= 3.0e38f);
    }
  };
  finish(acc0, row0, v0);
  finish(acc1, row1, v1);
  m = warp_max(m);
  if ((threadIdx.x & 31) == 0) atomicMax(maxabs_bits + bh, __float_as_uint(m));
  if (bad) set_error(err, SPARSEPR_ERR_NUMERIC);
}

template <typename T, int D, bool RMS>
static void project_dispatch_r(const T* X, const i64* xs, int BH, int H, int N, int r, const float* F, float eps,
                               float* phi, int ldphi, unsigned* maxabs, int* err, cudaStream_t st) {
  dim3 grid((N + 255) / 256, BH);
  if (r <= 16) k_project<T, D, 16, RMS><<<grid, 128, 0, st>>>(X, xs[0], xs[1], xs[2], H, N, r, F, eps, phi, ldphi, maxabs, err);
  else if (r <= 32) k_project<T, D, 32, RMS><<<grid, 128, 0, st>>>(X, xs[0], xs[1], xs[2], H, N, r, F, eps, phi, ldphi, maxabs, err);
  else if (r <= 48) k_project<T, D, 48, RMS><<<grid, 128, 0, st>>>(X, xs[0], xs[1], xs[2], H, N, r, F, eps, phi, ldphi, maxabs, err);
  else k_project<T, D, 64, RMS><<<grid, 128, 0, st>>>(X, xs[0], xs[1], xs[2], H, N, r, F, eps, phi, ldphi, maxabs, err);
}
void launch_project(int dtype, const void* X, const i64* xs, int BH, int H, int N, int d, int r, const float* F,
                    bool rms, float eps, float* phi, int ldphi, unsigned* maxabs, int* err, cudaStream_t st) {
#define SPR_PROJ(TT, DD)                                                                                        \
  do {                                                                                                          \
    if (rms) project_dispatch_r<TT, DD, true>((const TT*)X, xs, BH, H, N, r, F, eps, phi, ldphi, maxabs, err, st); \
    else project_dispatch_r<TT, DD, false>((const TT*)X, xs, BH, H, N, r, F, eps, phi, ldphi, maxabs, err, st);    \
  } while (0)
  if (dtype == SPARSEPR_BF16) { if (d == 128) SPR_PROJ(__nv_bfloat16, 128); else SPR_PROJ(__nv_bfloat16, 64); }
  else { if (d == 128) SPR_PROJ(float, 128); else SPR_PROJ(float, 64); }
#undef SPR_PROJ
}

// Features of the semantic reference partition (Section 3.1): the activations themselves, as float32 rows
// [BH][N][d]; also the largest magnitude per head (for the fixed-point sums) and the non-finite check.
template <typename T>
__global__ void __launch_bounds__(256) k_raw_features(const T* __restrict__ X, i64 sb, i64 sh, i64 sn, int H, int N, int d,
                                                      float* __restrict__ phi, unsigned* __restrict__ maxabs, int* __restrict__ err) {
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const int per_row = d / 8;
  float mx = 0.f;
  bool bad = false;
  for (i64 e = (i64)blockIdx.x * 256 + threadIdx.x; e < (i64)N * per_row; e += (i64)gridDim.x * 256) {
    const int row = (int)(e / per_row), c8 = (int)(e % per_row) * 8;
    float v[8];
    load8(X + b * sb + h * sh + (i64)row * sn + c8, v);
#pragma unroll
    for (int k = 0; k < 8; ++k) { mx = fmaxf(mx, fabsf(v[k])); bad |= !isfinite(v[k]); }
    store8(phi + ((i64)bh * N + row) * d + c8, v);
  }
  mx = warp_max(mx);
  if ((threadIdx.x & 31) == 0 && mx > 0.f) atomicMax(maxabs + bh, __float_as_uint(mx));
  if (bad) set_error(err, SPARSEPR_ERR_NUMERIC);
}
void launch_raw_features(int dtype, const void* X, const i64* xs, int BH, int H, int N, int d, float* phi, unsigned* maxabs,
                         int* err, cudaStream_t st) {
  dim3 grid((unsigned)std::min<i64>(((i64)N * (d / 8) + 255) / 256, 1024), BH);
  if (dtype == SPARSEPR_BF16) k_raw_features<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)X, xs[0], xs[1], xs[2], H, N, d, phi, maxabs, err);
  else k_raw_features<float><<<grid, 256, 0, st>>>((const float*)X, xs[0], xs[1], xs[2], H, N, d, phi, maxabs, err);
}

// =============================================================================
// k-means (Section 4.1).  Assignment: a[j] = argmin_c ||x_j - mu_c||^2, ties to the
// lowest c.  Fast path in float32 via s_c = ||mu_c||^2 - 2 x.mu_c; whenever the
// gap between the best and the second-best score is inside a proven rounding
// bound the row is decided by the exact float64 evaluation (terms added in order
// of k, one multiply and one add each), so the decision always equals that
// evaluation.  Optionally accumulates order-independent fixed-point centroid sums.
// =============================================================================
__device__ __noinline__ int exact_assign(const float* __restrict__ x, const float* __restrict__ mu, int C, int r, int ldmu) {
  double best = 0.0;
  int bi = 0;
  for (int c = 0; c < C; ++c) {
    const float* m = mu + (i64)c * ldmu;
    double dsum = 0.0;
    for (int k = 0; k < r; ++k) {
      const double diff = __dsub_rn((double)x[k], (double)m[k]);
      dsum = __dadd_rn(dsum, __dmul_rn(diff, diff));
    }
    if (c == 0 || dsum < best) { best = dsum; bi = c; }
  }
  return bi;
}

constexpr int kAssignChunk = 64;   // centroids staged per shared-memory chunk

// R = padded feature width (16..128), ROWS = rows per thread (two up to 64 columns; one for the 128 columns of the
// semantic partition's raw activations, whose row already fills the registers)
template <int R, int ROWS>
__global__ void __launch_bounds__(128) k_kmeans_assign(const float* __restrict__ phi, int ldphi, int N, int r,
                                                       const float* __restrict__ mu, const float* __restrict__ mu2,
                                                       const float* __restrict__ mumax, int C, int* __restrict__ assign,
                                                       i64* __restrict__ sums, int* __restrict__ counts,
                                                       const int* __restrict__ fx_shift, int* __restrict__ recheck_count,
                                                       const int* __restrict__ prev_changed, int* __restrict__ cur_changed) {
  constexpr int kChunk = R > 64 ? 32 : kAssignChunk;
  __shared__ __align__(16) float mus[kChunk * R];
  __shared__ float mu2s[kChunk];
  const int bh = blockIdx.y;
  if (prev_changed != nullptr && prev_changed[bh] == 0) return;      // fixed point reached in the previous pass
  const float* ph = phi + (i64)bh * N * ldphi;
  const float* muh = mu + (i64)bh * C * R;
  int rows[ROWS];
  float x[ROWS][R];
  float xn2[ROWS];
#pragma unroll
  for (int t = 0; t < ROWS; ++t) {
    rows[t] = (int)(blockIdx.x * (128 * ROWS) + threadIdx.x + 128 * t);
    xn2[t] = 0.f;
    const float* p = ph + (i64)min(rows[t], N - 1) * ldphi;
#pragma unroll
    for (int k = 0; k < R; k += 4) {
      const float4 v = *reinterpret_cast<const float4*>(p + k);      // columns r..R-1 hold zeros
      x[t][k] = v.x; x[t][k + 1] = v.y; x[t][k + 2] = v.z; x[t][k + 3] = v.w;
    }
#pragma unroll
    for (int k = 0; k < R; ++k) xn2[t] = fmaf(x[t][k], x[t][k], xn2[t]);
  }
  float best[ROWS], second[ROWS];
  int bi[ROWS];
#pragma unroll
  for (int t = 0; t < ROWS; ++t) { best[t] = 3.0e38f; second[t] = 3.0e38f; bi[t] = 0; }
  for (int c0 = 0; c0 < C; c0 += kChunk) {
    const int nc = min(kChunk, C - c0);
    __syncthreads();
    for (int e = threadIdx.x; e < nc * R; e += 128) mus[e] = muh[(i64)c0 * R + e];
    if (threadIdx.x < nc) mu2s[threadIdx.x] = mu2[(i64)bh * C + c0 + threadIdx.x];
    __syncthreads();
    for (int c = 0; c < nc; ++c) {
      const float4* m4 = reinterpret_cast<const float4*>(mus + c * R);
      float dot[ROWS];
#pragma unroll
      for (int t = 0; t < ROWS; ++t) dot[t] = 0.f;
#pragma unroll
      for (int k = 0; k < R / 4; ++k) {
        const float4 m = m4[k];
#pragma unroll
        for (int t = 0; t < ROWS; ++t) {
          dot[t] = fmaf(x[t][4 * k], m.x, dot[t]); dot[t] = fmaf(x[t][4 * k + 1], m.y, dot[t]);
          dot[t] = fmaf(x[t][4 * k + 2], m.z, dot[t]); dot[t] = fmaf(x[t][4 * k + 3], m.w, dot[t]);
        }
      }
#pragma unroll
      for (int t = 0; t < ROWS; ++t) {
        const float sc = fmaf(-2.f, dot[t], mu2s[c]);
        if (sc < best[t]) { second[t] = best[t]; best[t] = sc; bi[t] = c0 + c; } else if (sc < second[t]) second[t] = sc;
      }
    }
  }
  const float mm = mumax[bh];
  const int shift = fx_shift ? fx_shift[bh] : 0;
#pragma unroll
  for (int t = 0; t < ROWS; ++t) {
    if (rows[t] >= N) continue;
    // |computed score - true score| <= E for every centroid (float32 rounding of the
    // dot product, of ||mu||^2 and of the final combination)
    const float E = 1.5f * 5.9604645e-8f * (2.f * mm * mm + (2.f * r + 2.f) * sqrtf(xn2[t]) * mm);
    int a = bi[t];
    if (!(second[t] - best[t] > 2.f * E)) {
      a = exact_assign(ph + (i64)rows[t] * ldphi, muh, C, r, R);
      if (recheck_count) atomicAdd(recheck_count, 1);
    }
    if (cur_changed != nullptr && (prev_changed == nullptr || assign[(i64)bh * N + rows[t]] != a)) atomicAdd(cur_changed + bh, 1);
    assign[(i64)bh * N + rows[t]] = a;
    if (sums) {
      i64* s = sums + ((i64)bh * C + a) * R;
      const double sc = ldexp(1.0, shift);
#pragma unroll
      for (int k = 0; k < R; ++k)
        if (k < r) atomicAdd(reinterpret_cast<u64*>(s + k), (u64)__double2ll_rn((double)x[t][k] * sc));
      atomicAdd(counts + (i64)bh * C + a, 1);
    }
  }
}

void launch_kmeans_assign(const float* phi, int ldphi, int BH, int N, int r, const float* mu, const float* mu2,
                          const float* mumax, int C, int* assign, i64* sums, int* counts, const int* fx_shift,
                          int* recheck_count, const int* prev_changed, int* cur_changed, cudaStream_t st) {
  const int R = feature_ld(r);
#define SPR_ASSIGN(RR, ROWS) k_kmeans_assign<RR, ROWS><<<dim3((N + 128 * ROWS - 1) / (128 * ROWS), BH), 128, 0, st>>>(phi, ldphi, N, r, mu, mu2, mumax, C, assign, sums, counts, fx_shift, recheck_count, prev_changed, cur_changed)
  if (R == 16) SPR_ASSIGN(16, 2); else if (R == 32) SPR_ASSIGN(32, 2); else if (R == 48) SPR_ASSIGN(48, 2);
  else if (R == 64) SPR_ASSIGN(64, 2); else SPR_ASSIGN(128, 1);
#undef SPR_ASSIGN
}

// Initial centroids = feature rows of the strided init sample; also clears the sums
// and derives the fixed-point shift of the head from max |phi|.
__global__ void k_kmeans_init(const float* __restrict__ phi, int ldphi, int N, int r, int R, int C, u64 seed, int tag, int head0,
                              float* __restrict__ mu, i64* __restrict__ sums, int* __restrict__ counts,
                              const unsigned* __restrict__ maxabs_bits, int* __restrict__ fx_shift) {
  pdl_wait();                                                   // the features come from the kernel before
  pdl_launch_dependents();
  const int bh = blockIdx.y;
  const u64 U = sample_offset(seed, tag, head0 + bh);
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < C * R; e += gridDim.x * blockDim.x) {
    const int c = e / R, k = e % R;
    const int row = strided_row(c, C, N, U);
    mu[(i64)bh * C * R + e] = k < r ? phi[((i64)bh * N + row) * ldphi + k] : 0.f;
    sums[(i64)bh * C * R + e] = 0;
    if (k == 0) counts[(i64)bh * C + c] = 0;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    // sums of up to N values of magnitude <= maxabs must stay below 2^62
    const float m = fmaxf(__uint_as_float(maxabs_bits[bh]), 1e-30f);
    int e2;
    frexpf(m, &e2);                                  // m < 2^e2
    int nb = 0;
    while ((1ll << nb) < (i64)N) ++nb;
    int sh = 61 - nb - e2;
    fx_shift[bh] = max(-60, min(sh, 60));
  }
}

// mu <- sums / counts for non-empty clusters (empty ones keep their centroid), then
// ||mu_c||^2 (float64 -> float32) and the largest centroid norm of the head.
// gridDim.y CTAs per head share the centroids (warp w of part y takes c = y nw + w, + nw gridDim.y, ...); the
// largest norm needs all of them and is written only when one CTA holds the whole head (mumax may be null otherwise:
// the tensor-core assignment derives the bound from ||mu_c||^2 itself).
__global__ void __launch_bounds__(1024) k_kmeans_finalize(float* __restrict__ mu, float* __restrict__ mu2,
                                                          float* __restrict__ mumax, i64* __restrict__ sums,
                                                          int* __restrict__ counts, const int* __restrict__ fx_shift,
                                                          int C, int r, int R, int update,
                                                          __nv_bfloat16* __restrict__ mh, __nv_bfloat16* __restrict__ ml) {
  __shared__ float red[34];
  const int bh = blockIdx.x;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  pdl_wait();                                                   // the sums come from the kernels before
  pdl_launch_dependents();
  const double inv_sc = update ? ldexp(1.0, -fx_shift[bh]) : 0.0;
  float mx = 0.f;
  for (int c = blockIdx.y * nw + w; c < C; c += nw * gridDim.y) {
    float* m = mu + ((i64)bh * C + c) * R;
    i64* s = sums + ((i64)bh * C + c) * R;
    const int cnt = update ? counts[(i64)bh * C + c] : 0;
    double n2 = 0.0;
    for (int k = lane; k < max(R, 64); k += 32) {
      float v = 0.f;
      if (k < R) {
        v = m[k];
        if (update) {
          if (cnt > 0 && k < r) { v = (float)((double)s[k] * inv_sc / (double)cnt); m[k] = v; }
          s[k] = 0;
        }
        n2 += (double)v * (double)v;
      }
      if (mh != nullptr && k < 64) {
        // the two bf16 words of the centroid for the tensor-core assignment, [C][64] with zeros beyond r
        const float x = k < r ? v : 0.f;
        const __nv_bfloat16 hb = __float2bfloat16_rn(x);
        mh[((i64)bh * C + c) * 64 + k] = hb;
        ml[((i64)bh * C + c) * 64 + k] = __float2bfloat16_rn(x - __bfloat162float(hb));
      }
    }
    n2 = warp_sum(n2);
    __syncwarp();
    if (lane == 0) {
      mu2[(i64)bh * C + c] = (float)n2;
      if (update) counts[(i64)bh * C + c] = 0;
      mx = fmaxf(mx, (float)sqrt(n2) * 1.0000002f);
    }
  }
  if (gridDim.y == 1 && mumax != nullptr) {
    mx = block_max(mx, red);
    if (threadIdx.x == 0) mumax[bh] = mx;
  }
}

// Warm start (Appendix C.1): fixed-point sums and counts of the CURRENT features over the groups of a previous
// partition `prev` [BH][N]; the update step that follows turns them into the initial centroids (a group that the
// previous partition left empty keeps the strided row k_kmeans_init gave it).  One warp per 32 consecutive rows,
// lanes = feature columns (2 lane, 2 lane + 1), one atomic per (cluster present in the warp, column).  Entries of
// `prev` outside [0, C) are ignored.
__global__ void __launch_bounds__(256) k_kmeans_warm_sums(const float* __restrict__ phi, int ldphi, int N, int r, int R, int C,
                                                          const int* __restrict__ prev, i64* __restrict__ sums,
                                                          int* __restrict__ counts, const int* __restrict__ fx_shift) {
  const unsigned FULL = 0xffffffffu;
  const int bh = blockIdx.y, lane = threadIdx.x & 31;
  const int rowbase = (blockIdx.x * 8 + (threadIdx.x >> 5)) * 32;
  if (rowbase >= N) return;
  const int row = rowbase + lane;
  int cl_mine = -1;
  if (row < N) { const int c = prev[(i64)bh * N + row]; if (c >= 0 && c < C) cl_mine = c; }
  const float scl = __int_as_float((127 + fx_shift[bh]) << 23);
  for (int cb = 0; cb < R; cb += 64) {                         // 64 columns at a time (two passes for raw activations)
    const int col = cb + 2 * lane;
    const bool cok = col < r;
    float pv0[32], pv1[32];
#pragma unroll
    for (int rr = 0; rr < 32; ++rr) {
      const int rw = min(rowbase + rr, N - 1);
      const float2 x2 = cok ? *reinterpret_cast<const float2*>(phi + ((i64)bh * N + rw) * ldphi + col) : make_float2(0.f, 0.f);
      pv0[rr] = x2.x; pv1[rr] = x2.y;
    }
    unsigned todo = __ballot_sync(FULL, cl_mine >= 0);
    while (todo) {
      const int leader = __ffs(todo) - 1;
      const int cl = __shfl_sync(FULL, cl_mine, leader);
      const unsigned members = __ballot_sync(FULL, cl_mine == cl) & todo;
      todo &= ~members;
      float a0 = 0.f, a1 = 0.f;
#pragma unroll
      for (int rr = 0; rr < 32; ++rr)
        if ((members >> rr) & 1u) { a0 += pv0[rr]; a1 += pv1[rr]; }
      i64* sp = sums + ((i64)bh * C + cl) * R;
      if (col < r) atomicAdd(reinterpret_cast<u64*>(sp + col), (u64)__float2ll_rn(a0 * scl));
      if (col + 1 < r) atomicAdd(reinterpret_cast<u64*>(sp + col + 1), (u64)__float2ll_rn(a1 * scl));
      if (lane == 0 && cb == 0) atomicAdd(counts + (i64)bh * C + cl, __popc(members));
    }
  }
}
void launch_kmeans_warm_sums(const float* phi, int ldphi, int BH, int N, int r, int C, const int* prev, i64* sums,
                             int* counts, const int* fx_shift, cudaStream_t st) {
  const int R = feature_ld(r);
  k_kmeans_warm_sums<<<dim3((N + 255) / 256, BH), 256, 0, st>>>(phi, ldphi, N, r, R, C, prev, sums, counts, fx_shift);
}

void launch_kmeans_init(const float* phi, int ldphi, int BH, int N, int r, int C, u64 seed, int tag, int head0, float* mu,
                        i64* sums, int* counts, const unsigned* maxabs_bits, int* fx_shift, cudaStream_t st) {
  const int R = feature_ld(r);
  dim3 grid((C * R + 255) / 256, BH);
  launch_pdl(k_kmeans_init, grid, dim3(256), 0, st, phi, ldphi, N, r, R, C, seed, tag, head0, mu, sums, counts, maxabs_bits, fx_shift);
}
void launch_kmeans_finalize(float* mu, float* mu2, float* mumax, i64* sums, int* counts, const int* fx_shift, int BH,
                            int C, int r, int update, cudaStream_t st, __nv_bfloat16* mh, __nv_bfloat16* ml) {
  const int R = feature_ld(r);
  if (mumax != nullptr) {
    k_kmeans_finalize<<<BH, 1024, 0, st>>>(mu, mu2, mumax, sums, counts, fx_shift, C, r, R, update, mh, ml);
  } else {
    // one warp per centroid, spread over enough CTAs to fill the GPU
    const int parts = std::max(1, std::min(32, (C + 7) / 8));
    launch_pdl(k_kmeans_finalize, dim3(BH, parts), dim3(256), 0, st, mu, mu2, (float*)nullptr, sums, counts, fx_shift, C, r, R, update, mh, ml);
  }
}

// =============================================================================
// Stable counting sort by group id (Section 4.3, group-major layout).  One CTA of
// 16 warps per head; warp w owns a contiguous segment of tokens, so that ranks
// inside a group follow the original token order.
// =============================================================================
constexpr int kSortWarps = 16;

__global__ void __launch_bounds__(kSortWarps * 32) k_group_sort(const int* __restrict__ assign, int N, int C,
                                                                 int* __restrict__ perm, int* __restrict__ inv,
                                                                 int* __restrict__ off, int* err) {
  pdl_wait();                                                   // the assignment comes from the kernels before
  pdl_launch_dependents();
  extern __shared__ int sm_sort[];
  int* hist = sm_sort;                    // [kSortWarps][C]
  int* tot = hist + kSortWarps * C;       // [C]
  __shared__ int scratch[34];
  const int bh = blockIdx.x;
  const int* a = assign + (i64)bh * N;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  for (int e = threadIdx.x; e < kSortWarps * C; e += blockDim.x) hist[e] = 0;
  __syncthreads();
  const int L = (((N + kSortWarps - 1) / kSortWarps) + 31) / 32 * 32;
  const int s0 = w * L, s1 = min(N, s0 + L);
  for (int i = s0 + lane; i < s1; i += 32) {
    int key = a[i];
    // an id out of range (only possible after an earlier stage gave up) is recorded and counted as group 0, so that
    // the permutation stays a permutation and nothing downstream indexes out of bounds
    if (key < 0 || key >= C) { set_error(err, SPARSEPR_ERR_INVALID_ARG); key = 0; }
    atomicAdd(&hist[w * C + key], 1);
  }
  __syncthreads();
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    int t = 0;
    for (int ww = 0; ww < kSortWarps; ++ww) t += hist[ww * C + c];
    tot[c] = t;
  }
  __syncthreads();
  const int total = block_exclusive_scan(tot, C, scratch);
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    int run = tot[c];
    off[(i64)bh * (C + 1) + c] = run;
    for (int ww = 0; ww < kSortWarps; ++ww) { const int t = hist[ww * C + c]; hist[ww * C + c] = run; run += t; }
  }
  if (threadIdx.x == 0) off[(i64)bh * (C + 1) + C] = total;
  __syncthreads();
  for (int i0 = s0; i0 < s1; i0 += 32) {
    const int i = i0 + lane;
    int key = i < s1 ? a[i] : -1;
    if (i < s1 && (key < 0 || key >= C)) key = 0;
    const unsigned same = __match_any_sync(0xffffffffu, key);
    const int rank = __popc(same & ((1u << lane) - 1));
    int pos = -1;
    if (key >= 0) pos = hist[w * C + key] + rank;
    __syncwarp();
    if (key >= 0 && rank == 0) hist[w * C + key] += __popc(same);
    __syncwarp();
    if (key >= 0) { perm[(i64)bh * N + pos] = i; inv[(i64)bh * N + i] = pos; }
  }
}

void launch_group_sort(const int* assign, int BH, int N, int C, int* perm, int* inv, int* off, int* err, cudaStream_t st) {
  launch_pdl(k_group_sort, dim3(BH), dim3(kSortWarps * 32), (size_t)(kSortWarps + 1) * C * sizeof(int), st, assign, N, C, perm, inv, off, err);
}
cudaError_t init_group_sort() {
  return cudaFuncSetAttribute(k_group_sort, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)((kSortWarps + 1) * kMaxGroups * sizeof(int)));
}

// =============================================================================
// Group means in the original activation space: kappa_b (Appendix B.2) and
// theta_a (router).  One CTA per group walks its members in group-major order, eight warps on
// interleaved blocks of rows; the float32 sums have a fixed order.
// =============================================================================
template <typename T, int D>
__global__ void __launch_bounds__(256) k_group_means(const T* __restrict__ X, i64 sb, i64 sh, i64 sn, int H,
                                                     const int* __restrict__ perm, const int* __restrict__ off, int N,
                                                     int C, float* __restrict__ out, int* __restrict__ sizes) {
  pdl_wait();                                                   // the permutation comes from the kernel before
  pdl_launch_dependents();
  constexpr int LPR = D / 8;                 // lanes per row (8 elements each)
  constexpr int RPW = 32 / LPR;              // rows per warp step
  __shared__ float part[8][D];
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const int g = blockIdx.x, w = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31, sub = lane / LPR, col = (lane % LPR) * 8;
  const T* base = X + b * sb + h * sh;
  const int* pm = perm + (i64)bh * N;
  const int p0 = off[(i64)bh * (C + 1) + g], p1 = off[(i64)bh * (C + 1) + g + 1];
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  // One CTA per group (group sizes spread over two orders of magnitude: with a warp per group the largest group set
  // the duration of the launch): warp w takes the blocks of 8 RPW rows number w, w + 8, ...; eight row loads in
  // flight per lane (the walk is bound by the latency of the index -> row chain); every sum has a fixed order, and
  // a slot beyond the group adds exact zeros
  for (int p = p0 + w * RPW * 8 + sub; p < p1; p += RPW * 8 * 8) {
    int src[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) src[j] = p + j * RPW < p1 ? pm[p + j * RPW] : -1;
    float v[8][8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (src[j] >= 0) {
        load8(base + (i64)src[j] * sn + col, v[j]);
      } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) v[j][k] = 0.f;
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[k] += v[j][k];
  }
  // combine the RPW interleaved partial sums of the warp, then the eight warps, in a fixed order
#pragma unroll
  for (int k = 0; k < 8; ++k)
    for (int o = LPR; o < 32; o <<= 1) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], o);
  if (sub == 0) {
#pragma unroll
    for (int k = 0; k < 8; ++k) part[w][col + k] = acc[k];
  }
  __syncthreads();
  const int n = p1 - p0;
  if (threadIdx.x < D) {
    float t = part[0][threadIdx.x];
#pragma unroll
    for (int ww = 1; ww < 8; ++ww) t += part[ww][threadIdx.x];
    out[((i64)bh * C + g) * D + threadIdx.x] = n > 0 ? t * (1.f / (float)n) : 0.f;
  }
  if (threadIdx.x == 0 && sizes) sizes[(i64)bh * C + g] = n;
}

void launch_group_means(int dtype, const void* X, const i64* xs, int BH, int H, const int* perm, const int* off, int N,
                        int C, int d, float* out, int* sizes, cudaStream_t st) {
  dim3 grid(C, BH);
#define SPR_GM(TT, DD) launch_pdl(k_group_means<TT, DD>, grid, dim3(256), 0, st, (const TT*)X, xs[0], xs[1], xs[2], H, perm, off, N, C, out, sizes)
  if (dtype == SPARSEPR_BF16) { if (d == 128) SPR_GM(__nv_bfloat16, 128); else SPR_GM(__nv_bfloat16, 64); }
  else { if (d == 128) SPR_GM(float, 128); else SPR_GM(float, 64); }
#undef SPR_GM
}

// =============================================================================
// Row gather into the group-major layout: out[bh][p][:] = in[b,h,perm[p],:].
// =============================================================================
template <typename T, int D>
__global__ void __launch_bounds__(256) k_gather_rows(const T* __restrict__ X, i64 sb, i64 sh, i64 sn, int H,
                                                     const int* __restrict__ perm, int N, T* __restrict__ out) {
  constexpr int VEC = 16 / sizeof(T);
  constexpr int TPR = D / VEC;               // threads per row
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const T* base = X + b * sb + h * sh;
  const i64 t = (i64)blockIdx.x * 256 + threadIdx.x;
  const int p = (int)(t / TPR), c = (int)(t % TPR) * VEC;
  if (p >= N) return;
  const int src = perm[(i64)bh * N + p];
  *reinterpret_cast<uint4*>(out + ((i64)bh * N + p) * D + c) = *reinterpret_cast<const uint4*>(base + (i64)src * sn + c);
}

void launch_gather_rows(int dtype, const void* X, const i64* xs, int BH, int H, const int* perm, int N, int d, void* out,
                        cudaStream_t st) {
  const int es = dtype == SPARSEPR_BF16 ? 2 : 4;
  const int tpr = d * es / 16;
  dim3 grid((unsigned)(((i64)N * tpr + 255) / 256), BH);
#define SPR_GA(TT, DD) k_gather_rows<TT, DD><<<grid, 256, 0, st>>>((const TT*)X, xs[0], xs[1], xs[2], H, perm, N, (TT*)out)
  if (dtype == SPARSEPR_BF16) { if (d == 128) SPR_GA(__nv_bfloat16, 128); else SPR_GA(__nv_bfloat16, 64); }
  else { if (d == 128) SPR_GA(float, 128); else SPR_GA(float, 64); }
#undef SPR_GA
}

}  // namespace spr
