// Probe-Fitted Residual Reconstruction, the per-head fit (Appendix A.3): weighted
// standardisation, weighted ridge normal equations solved by Cholesky, the
// probe-residual output subspace, and the composed affine map
//   R_hat_i = c + x_i A,  A = diag(1/s_x) B_lambda Psi_r Psi_r^T,  c = mu_R - mu_x A,
// which is algebraically Eq. 9.  Standardisation and composition are float64; the Gram matrices and the Cholesky
// solve are float64 for float32 tensors and float32 for 16-bit tensors; one CTA per head.
#include "kernels.cuh"

namespace spr {

// scratch per head (doubles): Xb[M*d] Rb[M*d] G[d*d] B[d*d] S[d*d] T[d*d] mu_x[d] mu_R[d] s_x[d] wt[M] flag[1]
struct FitLayout {
  size_t Xb, Rb, G, B, S, T, mu_x, mu_R, s_x, wt, flag, total;
  __host__ __device__ FitLayout(int M, int d) {
    size_t o = 0;
    Xb = o; o += (size_t)M * d;
    Rb = o; o += (size_t)M * d;
    G = o; o += (size_t)d * d;
    B = o; o += (size_t)d * d;
    S = o; o += (size_t)d * d;
    T = o; o += (size_t)d * d;
    mu_x = o; o += d; mu_R = o; o += d; s_x = o; o += d;
    wt = o; o += M;
    flag = o; o += 1;
    total = (o + 31) / 32 * 32;
  }
};
size_t fit_scratch_doubles(int BH, int M, int d) { return FitLayout(M, d).total * BH; }

// alpha, weighted means, feature scale, standardised probes, unit-mean weights
__global__ void __launch_bounds__(256) k_fit_prepare(FitArgs a) {
  __shared__ double red[34];
  const int bh = blockIdx.x, M = a.M, d = a.d;
  const FitLayout L(M, d);
  double* sc = a.scratch + (size_t)bh * L.total;
  const float* X = a.X + (i64)bh * M * d;
  const float* Dn = a.Dn + (i64)bh * M * d;
  const float* w = a.w + (i64)bh * M;
  double sw = 0.0, cnt = 0.0;
  for (int p = threadIdx.x; p < M; p += 256) { sw += (double)w[p]; cnt += w[p] > 0.f ? 1.0 : 0.0; }
  sw = block_sum(sw, red);
  cnt = block_sum(cnt, red);
  if (threadIdx.x == 0) sc[L.flag] = (sw > 0.0 && cnt > 0.0) ? 0.0 : 1.0;
  if (!(sw > 0.0)) sw = 1.0;
  // alpha_p = w_p / sum w once per probe (float64 divisions are expensive on this part), kept in the weight slot
  // until the unit-mean weights replace it at the end
  for (int p = threadIdx.x; p < M; p += 256) sc[L.wt + p] = (double)w[p] / sw;
  __syncthreads();
  for (int j = threadIdx.x; j < d; j += 256) {
    double mx = 0.0, mr = 0.0;
    for (int p = 0; p < M; ++p) {
      const double al = sc[L.wt + p], x = (double)X[p * d + j];
      mx += al * x;
      mr += al * ((double)Dn[p * d + j] - x);
    }
    double var = 0.0;
    for (int p = 0; p < M; ++p) { const double t = (double)X[p * d + j] - mx; var += sc[L.wt + p] * t * t; }
    const double s = sqrt(var + (double)a.eps_std), inv_s = 1.0 / s;
    sc[L.mu_x + j] = mx; sc[L.mu_R + j] = mr; sc[L.s_x + j] = s;
    for (int p = 0; p < M; ++p) {
      const double x = (double)X[p * d + j];
      sc[L.Xb + (size_t)p * d + j] = (x - mx) * inv_s;
      sc[L.Rb + (size_t)p * d + j] = ((double)Dn[p * d + j] - x) - mr;
    }
  }
  __syncthreads();
  for (int p = threadIdx.x; p < M; p += 256) sc[L.wt + p] = (double)M * (double)w[p] / sw;   // unit-mean weights M w_p / sum w (Appendix A.3)
}

// blockIdx.x selects G = Xb^T W Xb + lam I, B(rhs) = Xb^T W Rb, S = Rb^T W Rb.
// T = float for 16-bit tensors (the float64 pipe of this part is narrow: a float64 Gram is bound by it), double otherwise.
template <typename T>
__global__ void __launch_bounds__(256) k_fit_gram(FitArgs a) {
  extern __shared__ unsigned char sm_gram_raw[];   // [2][32][d] row chunks of the left and right factor
  T* sm_gram = reinterpret_cast<T*>(sm_gram_raw);
  const int bh = blockIdx.y, which = blockIdx.x, M = a.M, d = a.d;
  const FitLayout L(M, d);
  double* sc = a.scratch + (size_t)bh * L.total;
  const double* Lm = sc + (which == 2 ? L.Rb : L.Xb);
  const double* Rm = sc + (which == 0 ? L.Xb : L.Rb);
  double* out = sc + (which == 0 ? L.G : which == 1 ? L.B : L.S);
  T* ls = sm_gram;
  T* rs = sm_gram + 32 * d;
  const int per = d * d / 256;             // entries per thread (d = 64 or 128)
  T acc[64];
#pragma unroll
  for (int e = 0; e < 64; ++e) acc[e] = T(0);
  for (int p0 = 0; p0 < M; p0 += 32) {
    const int nr = min(32, M - p0);
    __syncthreads();
    for (int t = threadIdx.x; t < nr * d; t += 256) {
      const int p = t / d;
      ls[t] = (T)(Lm[(size_t)(p0 + p) * d + t % d] * sc[L.wt + p0 + p]);
      rs[t] = (T)Rm[(size_t)(p0 + p) * d + t % d];
    }
    __syncthreads();
#pragma unroll
    for (int e = 0; e < 64; ++e) {
      if (e < per) {
        const int idx = threadIdx.x + e * 256, i = idx / d, j = idx % d;
        T s = acc[e];
        for (int p = 0; p < nr; ++p) s += ls[p * d + i] * rs[p * d + j];
        acc[e] = s;
      }
    }
  }
#pragma unroll
  for (int e = 0; e < 64; ++e) {
    if (e < per) {
      const int idx = threadIdx.x + e * 256, i = idx / d, j = idx % d;
      out[idx] = (double)acc[e] + ((which == 0 && i == j) ? (double)a.lambda : 0.0);
    }
  }
}

// Cholesky G = L L^T in shared memory, then L Y = RHS and L^T B = Y.  T as in k_fit_gram.
template <typename T>
__global__ void __launch_bounds__(1024) k_fit_solve(FitArgs a) {
  extern __shared__ unsigned char Gs_raw[];  // [d][d+1]
  T* Gs = reinterpret_cast<T*>(Gs_raw);
  const int bh = blockIdx.x, d = a.d, ld = d + 1;
  const FitLayout L(a.M, d);
  double* sc = a.scratch + (size_t)bh * L.total;
  __shared__ int bad;
  // (square roots and divisions are expensive in float64 on this part: one thread forms 1/sqrt(pivot), and the
  // reciprocals of the diagonal are kept for the triangular solves)
  __shared__ T s_inv;
  __shared__ T dinv[128];
  if (threadIdx.x == 0) bad = sc[L.flag] != 0.0;
  for (int e = threadIdx.x; e < d * d; e += blockDim.x) Gs[(e / d) * ld + e % d] = (T)sc[L.G + e];
  __syncthreads();
  for (int k = 0; k < d; ++k) {
    if (threadIdx.x == 0) {
      const T piv = Gs[k * ld + k];
      if (!(piv > T(0))) bad = 1;
      else { s_inv = T(1) / sqrt(piv); dinv[k] = s_inv; }       // 1 / L_kk
    }
    __syncthreads();
    if (bad) break;                                               // uniform
    const T inv = s_inv;
    for (int i = k + threadIdx.x; i < d; i += blockDim.x) Gs[i * ld + k] *= inv;   // includes the diagonal: L_kk = sqrt(piv)
    __syncthreads();
    // trailing update of the lower triangle: eight threads per row, columns k+1+q, k+1+q+8, ... up to the diagonal
    for (int i = k + 1 + (int)(threadIdx.x >> 3); i < d; i += (int)(blockDim.x >> 3)) {
      const T lik = Gs[i * ld + k];
      for (int j = k + 1 + (int)(threadIdx.x & 7); j <= i; j += 8) Gs[i * ld + j] -= lik * Gs[j * ld + k];
    }
    __syncthreads();
  }
  __syncthreads();
  if (bad) {
    if (threadIdx.x == 0) { sc[L.flag] = 1.0; set_error(a.err, SPARSEPR_ERR_NUMERIC); }
    return;
  }
  // Triangular solves: eight threads per right-hand-side column.  Thread (c, q) keeps the entries i = q, q + 8, ...
  // of its column in registers; row i of the solve is a dot product over the entries already known, split over the
  // eight threads and added up by shuffles (fixed order).
  double* Bm = sc + L.B;
  constexpr int kTq = 8, kMaxPer = 128 / kTq;
  const int c = threadIdx.x / kTq, q = threadIdx.x % kTq;
  const int per = d / kTq;                                   // d = 64 or 128
  if (c < d) {
    T y[kMaxPer];
#pragma unroll
    for (int t = 0; t < kMaxPer; ++t) y[t] = t < per ? (T)Bm[(size_t)(q + kTq * t) * d + c] : T(0);
    for (int i = 0; i < d; ++i) {                            // forward: y_i = (b_i - sum_{j<i} L_ij y_j) / L_ii
      T s = T(0);
#pragma unroll
      for (int t = 0; t < kMaxPer; ++t) {
        const int j = q + kTq * t;
        if (t < per && j < i) s += Gs[i * ld + j] * y[t];
      }
#pragma unroll
      for (int o = 1; o < kTq; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      const T inv = dinv[i];
#pragma unroll
      for (int t = 0; t < kMaxPer; ++t)
        if (q + kTq * t == i) y[t] = (y[t] - s) * inv;
    }
    for (int i = d - 1; i >= 0; --i) {                       // backward: b_i = (y_i - sum_{j>i} L_ji b_j) / L_ii
      T s = T(0);
#pragma unroll
      for (int t = 0; t < kMaxPer; ++t) {
        const int j = q + kTq * t;
        if (t < per && j > i) s += Gs[j * ld + i] * y[t];
      }
#pragma unroll
      for (int o = 1; o < kTq; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      const T inv = dinv[i];
#pragma unroll
      for (int t = 0; t < kMaxPer; ++t)
        if (q + kTq * t == i) y[t] = (y[t] - s) * inv;
    }
#pragma unroll
    for (int t = 0; t < kMaxPer; ++t)
      if (t < per) Bm[(size_t)(q + kTq * t) * d + c] = (double)y[t];
  }
}

// T = B Psi (d x r); A = diag(1/s_x) T Psi^T; c = mu_R - mu_x A
__global__ void __launch_bounds__(256) k_fit_compose(FitArgs a, int r) {
  const int bh = blockIdx.x, d = a.d;
  const FitLayout L(a.M, d);
  double* sc = a.scratch + (size_t)bh * L.total;
  float* A = a.A + (i64)bh * d * d;
  float* c = a.c + (i64)bh * d;
  if (sc[L.flag] != 0.0) {                 // no usable fit: the head falls back to hard drop
    for (int e = threadIdx.x; e < d * d; e += 256) A[e] = 0.f;
    for (int j = threadIdx.x; j < d; j += 256) c[j] = 0.f;
    return;
  }
  const float* Psi = a.Psi + (i64)bh * d * r;
  const double* Bm = sc + L.B;
  double* T = sc + L.T;
  for (int e = threadIdx.x; e < d * r && !a.full_rank; e += 256) {
    const int i = e / r, t = e % r;
    double s = 0.0;
    for (int k = 0; k < d; ++k) s += Bm[(size_t)i * d + k] * (double)Psi[k * r + t];
    T[e] = s;
  }
  __shared__ double rs_x[128];             // 1 / s_x
  for (int i = threadIdx.x; i < d; i += 256) rs_x[i] = 1.0 / sc[L.s_x + i];
  __syncthreads();
  double* Ad = sc + L.G;                   // G is no longer needed
  for (int e = threadIdx.x; e < d * d; e += 256) {
    const int i = e / d, j = e % d;
    double s = 0.0;
    if (a.full_rank) {
      s = Bm[e];                           // every row of B lies in the row space of the probe residuals: B Psi Psi^T = B
    } else {
      for (int t = 0; t < r; ++t) s += T[i * r + t] * (double)Psi[j * r + t];
    }
    s *= rs_x[i];
    Ad[e] = s;
    A[e] = (float)s;
  }
  __syncthreads();
  for (int j = threadIdx.x; j < d; j += 256) {
    double s = sc[L.mu_R + j];
    for (int i = 0; i < d; ++i) s -= sc[L.mu_x + i] * Ad[(size_t)i * d + j];
    c[j] = (float)s;
  }
}

cudaError_t init_fit() {
  cudaError_t e = cudaFuncSetAttribute(k_fit_solve<double>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 129 * 8);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_fit_solve<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 129 * 4);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_fit_gram<double>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 32 * 128 * 8);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_fit_gram<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 32 * 128 * 4);
  return e;
}

void launch_fit(const FitArgs& a, cudaStream_t st) {
  const int d = a.d;
  const int r = min(a.r_out, min(a.M, d));
  const FitLayout L(a.M, d);
  k_fit_prepare<<<a.BH, 256, 0, st>>>(a);
  if (a.precise) {
    k_fit_gram<double><<<dim3(3, a.BH), 256, (size_t)2 * 32 * d * 8, st>>>(a);
    k_fit_solve<double><<<a.BH, 1024, (size_t)d * (d + 1) * 8, st>>>(a);
  } else {
    k_fit_gram<float><<<dim3(3, a.BH), 256, (size_t)2 * 32 * d * 4, st>>>(a);
    k_fit_solve<float><<<a.BH, 1024, (size_t)d * (d + 1) * 4, st>>>(a);
  }
  // Psi_r: leading eigenvectors of S = Rb^T W Rb, i.e. right singular vectors of W^(1/2) Rb.
  if (!a.full_rank) launch_eig_top(a.scratch + L.S, (i64)L.total, a.BH, d, r, 1, a.precise, a.Psi, nullptr, a.eig_ws, st);
  k_fit_compose<<<a.BH, 256, 0, st>>>(a, r);
}

}  // namespace spr
