// Leading eigenpairs of batched symmetric matrices (n = 64 or 128), one CTA per matrix:
// the feature maps F_K, F_Q of Section 4.1 and the probe-residual basis Psi_r of Eq. 9.
//
// Float64 for float32 tensors, float32 for bf16 tensors.  Two kernels: k_householder (step 1, 2 n threads, matrix in
// registers) hands the tridiagonal form and the reflectors to k_eig_tridiag (steps 2-6, 1024 threads) through a
// scratch buffer:
//   1. Householder reduction to tridiagonal form T (reflectors kept)
//   2. the r largest eigenvalues of T by Sturm-count bisection, one thread per eigenvalue
//   3. their eigenvectors by inverse iteration on T - lambda I (Gaussian elimination with
//      partial pivoting, factored once per eigenvalue), one thread per eigenvector
//   4. Gram-Schmidt with re-orthogonalisation inside groups of close eigenvalues
//   5. Rayleigh quotients, residuals ||T z - lambda z|| and all pairwise inner products are
//      checked; a matrix that fails the check is marked (NaN in its first output element)
//      and left to the cyclic Jacobi kernel, which is launched behind this one and returns
//      at once for unmarked matrices
//   6. back-transformation with the reflectors, scaling, output
// The work per matrix is O(n^3) for step 1 and O(r n^2) for step 6, each spread over the CTA;
// steps 2-3 are O(n) recurrences per thread.  Step 1 is a chain of n - 2 dependent steps, so it runs on few threads
// with many matrix entries each (64 registers of matrix per thread at n = 128) rather than on all 1024.
#include "kernels.cuh"

namespace spr {

namespace {

constexpr int kEigThreads = 1024;
constexpr int kEigMaxR = 64;
constexpr int kZld = kEigMaxR + 1;
constexpr int kTpr = 8;                                            // threads per matrix row in the Householder steps

__device__ __forceinline__ float hash_unit(int i, int j) {         // deterministic start vector entries in [0.5, 1.5)
  u64 x = (u64)(i + 1) * 0x9E3779B97F4A7C15ull + (u64)(j + 1) * 0xBF58476D1CE4E5B9ull;
  x ^= x >> 31; x *= 0x94D049BB133111EBull; x ^= x >> 29;
  return 0.5f + (float)(unsigned)(x >> 40) * (1.0f / 16777216.0f);
}

// Precision-dependent constants.  Float64 serves float32 tensors (whose output tolerance leaves no
// room for a float32 eigen-basis); float32 serves bf16 tensors, where float64 arithmetic would
// dominate the run time of the whole plan.
template <typename T> struct EigNum;
template <> struct EigNum<double> {
  static constexpr double pivot = 1.0e-15, res_tol = 1.0e-7, orth_tol = 1.0e-7, group_gap = 1.0e-8, polish_tol = 1.0e-12;
  static constexpr double e2_min = 1.0e-280;
  static constexpr int passes = 15;
};
template <> struct EigNum<float> {
  static constexpr float pivot = 1.0e-7f, res_tol = 1.0e-4f, orth_tol = 1.0e-3f, group_gap = 1.0e-5f, polish_tol = 1.0e-5f;
  static constexpr float e2_min = 1.0e-30f;
  static constexpr int passes = 9;
};

// kN consecutive elements (a multiple of 16 bytes, 16-byte aligned) between shared memory and registers
template <typename T, int kN> __device__ __forceinline__ void ld_vec(const T* p, T (&o)[kN]) {
  constexpr int kV = 16 / sizeof(T);
#pragma unroll
  for (int i = 0; i < kN / kV; ++i) {
    const uint4 raw = reinterpret_cast<const uint4*>(p)[i];
    T tmp[kV];
    *reinterpret_cast<uint4*>(tmp) = raw;
#pragma unroll
    for (int e = 0; e < kV; ++e) o[i * kV + e] = tmp[e];
  }
}
template <typename T, int kN> __device__ __forceinline__ void st_vec(T* p, const T (&o)[kN]) {
  constexpr int kV = 16 / sizeof(T);
#pragma unroll
  for (int i = 0; i < kN / kV; ++i) {
    T tmp[kV];
#pragma unroll
    for (int e = 0; e < kV; ++e) tmp[e] = o[i * kV + e];
    reinterpret_cast<uint4*>(p)[i] = *reinterpret_cast<const uint4*>(tmp);
  }
}

// sum over the 32 warps of the CTA with one barrier: partial sums go to one of two buffers in turn,
// every warp then adds the 32 partials itself (same order everywhere, so all threads agree bit for bit)
template <typename T> __device__ __forceinline__ T cta_sum(T v, T* red, int& turn) {
  v = warp_sum(v);
  T* buf = red + (turn & 1) * 32;
  ++turn;
  if ((threadIdx.x & 31) == 0) buf[threadIdx.x >> 5] = v;
  __syncthreads();
  return warp_sum(buf[threadIdx.x & 31]);
}
template <typename T> __device__ __forceinline__ T cta_max(T v, T* red, int& turn) {
  v = warp_max(v);
  T* buf = red + (turn & 1) * 32;
  ++turn;
  if ((threadIdx.x & 31) == 0) buf[threadIdx.x >> 5] = v;
  __syncthreads();
  return warp_max(buf[threadIdx.x & 31]);
}

constexpr size_t cmax3(size_t x, size_t y, size_t w) { return x > y ? (x > w ? x : w) : (y > w ? y : w); }

template <int NN, typename T> struct EigSmem {
  // a vector of NN entries is stored as kTpr segments of NN / kTpr entries, each followed by 16 bytes of
  // padding: the eight threads of a row then read their segments with conflict-free 16-byte accesses
  static constexpr int kPad = 16 / (int)sizeof(T);
  static constexpr int LD = NN + kTpr * kPad;
  // The factors of the inverse iteration (four numbers per row and vector) share the space of the reflectors, which
  // are fetched only for the back-transformation; float64 at n = 128 has no room for them (they stay in local memory).
  static constexpr size_t fac_bytes = sizeof(T) * 4 * NN * kEigMaxR;
  static constexpr bool fac_in_smem = fac_bytes <= 131072;
  static constexpr size_t a_bytes = sizeof(T) * NN * LD;
  // One region serves in turn the factors, the partial Gram matrices of the polish step ([4][64][64]) and the
  // reflectors.  Where the reflectors fit behind the Gram matrices they are fetched asynchronously while the polish
  // step runs (a_off > 0); otherwise they are fetched right before the back-transformation.
  static constexpr size_t g_bytes = sizeof(T) * 4 * 64 * 64;
  static constexpr size_t rest = sizeof(T) * (NN * kZld + 2 * LD + 6 * NN + kEigMaxR + 64) + sizeof(int) * (kEigMaxR + 4);
  static constexpr size_t a_off = g_bytes + a_bytes + rest <= 227 * 1024 ? g_bytes : 0;
  static constexpr size_t a = 0;                                           // region start
  static constexpr size_t region = cmax3(fac_in_smem ? fac_bytes : 0, a_off + a_bytes, g_bytes);
  static constexpr size_t z = a + region;                                  // T [NN][kZld]
  static constexpr size_t pb = z + sizeof(T) * NN * kZld;                  // T [2][LD]: p of two consecutive steps
  static constexpr size_t vec = pb + sizeof(T) * 2 * LD;                   // (2 spare), d, e, e2, beta: 6 x T[NN]
  static constexpr size_t lam = vec + sizeof(T) * 6 * NN;             // T [kEigMaxR]
  static constexpr size_t red = lam + sizeof(T) * kEigMaxR;           // T [2][32]
  static constexpr size_t cst = red + sizeof(T) * 64;                 // int [kEigMaxR] group start; int flags[4]
  static constexpr size_t total = cst + sizeof(int) * (kEigMaxR + 4);
};

// Reciprocal on the dependent chains of the Sturm count and of the factorisation: float32 takes the hardware
// approximation (the chains are perturbed at the level of their own rounding), float64 the division.
__device__ __forceinline__ float chain_rcp(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ double chain_rcp(double x) { return 1.0 / x; }

// eigenvalues of T below x (Sturm count): the pivots q_i = (d_i - x) - e_{i-1}^2 / q_{i-1} of the factorisation
// T - x I = L D L^T, one negative pivot per eigenvalue below x.  A zero pivot needs no test: its reciprocal is an
// infinity, the next pivot -infinity (counted; e2[] is kept strictly positive for this), whose reciprocal is zero.
template <int NN, typename T>
__device__ __forceinline__ int sturm_count(const T* __restrict__ dd, const T* __restrict__ e2, T x) {
  T q = dd[0] - x;
  int cnt = q < T(0.0);
#pragma unroll 8
  for (int i = 1; i < NN; ++i) {
    q = fma(-e2[i - 1], chain_rcp(q), dd[i] - x);
    cnt += q < T(0.0);
  }
  return cnt;
}

// What k_householder leaves per matrix for k_eig_tridiag (units of T): reflector k in row k of v (zero up to entry
// k), diagonal, subdiagonal, the factors b_k of H_k = I - b_k v_k v_k^T, and the scale max |a_ij| of the input.
template <int NN> struct HhLayout {
  static constexpr int v = 0, dd = NN * NN, ee = dd + NN, beta = ee + NN, scale = beta + NN, stride = scale + 4;
};

// Householder reduction of a symmetric matrix to tridiagonal form, matrix in registers: thread (row, h) owns the
// 16-column chunks h, h + 2, ... of its row (a CTA is 2 NN threads).  Step k: x = A[k+1.., k]; v = x + sgn(x_0) alpha e_1;
// p = b A22 v; w = p - (b/2)(p.v) v; A22 <- A22 - v w^T - w v^T.  Every row keeps its own entries of the next two
// columns (its entries of rows k+1 and k+2, by symmetry): the first becomes its entry of x, the second the term that
// turns A x into A v, so nobody has to publish a whole row.  x and p are zero outside the trailing block, which lets
// the inner loops run over all chunks without column tests.  Two barriers per step: one after x and the partial
// sums of its squares are in shared memory, one after p and the partial sums of p.v are.
template <int NN, typename T>
__global__ void __launch_bounds__(2 * NN) k_householder(const double* __restrict__ Min, i64 stride, T* __restrict__ ws) {
  pdl_wait();                                                   // the matrices come from the kernel before
  pdl_launch_dependents();
  using HL = HhLayout<NN>;
  constexpr int kCh = 16, kNc = NN / (2 * kCh), kWarps = 2 * NN / 32;
  constexpr int kScrLd = kCh + 16 / (int)sizeof(T);             // padded chunk: 16-byte aligned, spreads the banks
  constexpr unsigned FULL = 0xffffffffu;
  __shared__ __align__(16) T xs[2][NN];                         // x of two consecutive steps (zero at entries <= k)
  __shared__ __align__(16) T ps[NN];                            // p (zero at entries <= k)
  __shared__ __align__(16) T sqp[2][kWarps];                    // per-warp sums of x_i^2, i > k + 1
  __shared__ __align__(16) T pvp[kWarps];                       // per-warp parts of p.v
  __shared__ __align__(16) T scr[2 * NN * kScrLd];              // one chunk per thread: picks a column out of the registers
  __shared__ T dd_s[NN], ee_s[NN], beta_s[NN];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row = tid >> 1, h = tid & 1;
  const double* Mi = Min + (i64)blockIdx.x * stride;
  T* out = ws + (i64)blockIdx.x * HL::stride;

  // load, symmetrise, scale to max |a_ij| = 1
  T a[kNc * kCh];
  T amax = T(0.0);
#pragma unroll
  for (int i = 0; i < kNc; ++i) {
#pragma unroll
    for (int t = 0; t < kCh; ++t) {
      const int c = (2 * i + h) * kCh + t;
      a[i * kCh + t] = T(0.5 * (Mi[row * NN + c] + Mi[c * NN + row]));
      amax = fmax(amax, fabs(a[i * kCh + t]));
    }
  }
  amax = warp_max(amax);
  if (lane == 0) pvp[warp] = amax;
  __syncthreads();
  T scale = pvp[0];
#pragma unroll
  for (int wi = 1; wi < kWarps; ++wi) scale = fmax(scale, pvp[wi]);
  if (!(scale > T(0.0)) || !(scale * T(0.0) == T(0.0))) {       // zero or non-finite: the caller's kernel handles it
    if (tid == 0) out[HL::scale] = scale;
    return;
  }
  const T inv_scale = T(1.0) / scale;
#pragma unroll
  for (int e = 0; e < kNc * kCh; ++e) a[e] *= inv_scale;
  __syncthreads();                                              // pvp[] is reused below

  // A[row][j] for a column j that is uniform over the CTA (zero for j >= NN): the thread of the row that owns the
  // chunk of j copies it to shared memory, both threads of the row read entry j back
  auto column = [&](int j) -> T {
    const int ch = j >> 4, ip = ch >> 1, hp = ch & 1;
#pragma unroll
    for (int i = 0; i < kNc; ++i) {
      if (i == ip && h == hp) {
        T tmp[kCh];
#pragma unroll
        for (int t = 0; t < kCh; ++t) tmp[t] = a[i * kCh + t];
        st_vec<T, kCh>(scr + tid * kScrLd, tmp);
      }
    }
    __syncwarp();
    const T val = j < NN ? scr[(2 * row + hp) * kScrLd + (j & 15)] : T(0.0);
    __syncwarp();
    return val;
  };
  // x of step kn from this row's entry c0 = A[row][kn]
  T xk_row = T(0.0);
  auto publish = [&](int kn, T c0) {
    const T xr = row > kn ? c0 : T(0.0);
    T sq = (row > kn + 1 && h == 0) ? c0 * c0 : T(0.0);
#pragma unroll
    for (int o = 2; o < 32; o <<= 1) sq += __shfl_xor_sync(FULL, sq, o);
    if (h == 0) {
      xs[kn & 1][row] = xr;
      if (row == kn) dd_s[kn] = c0;                             // the diagonal entry is final once row kn leaves the block
    }
    if (lane == 0) sqp[kn & 1][warp] = sq;
    xk_row = xr;
  };
  T col1 = column(1);                                           // A[row][k + 1] at the start of step k
  publish(0, column(0));

  for (int k = 0; k < NN - 2; ++k) {
    const int kb = k & 1;
    __syncthreads();                                            // x and its partial sums are in place
    T below2 = sqp[kb][0];                                      // squares beyond the subdiagonal entry
#pragma unroll
    for (int wi = 1; wi < kWarps; ++wi) below2 += sqp[kb][wi];
    const T x0 = xs[kb][k + 1];
    if (!(below2 > T(0.0))) {                                   // uniform: already reduced, A stays as it is
      if (tid == 0) { ee_s[k] = x0; beta_s[k] = T(0.0); }
      if (h == 0) out[HL::v + k * NN + row] = T(0.0);
      const T c0 = col1;
      col1 = column(k + 2);
      publish(k + 1, c0);
      continue;
    }
    const T alpha = sqrt(below2 + x0 * x0);
    const T sa = x0 >= T(0.0) ? alpha : -alpha;
    const T b = T(1.0) / (alpha * (alpha + fabs(x0)));
    if (tid == 0) { ee_s[k] = -sa; beta_s[k] = b; }
    const T v_row = xk_row + (row == k + 1 ? sa : T(0.0));      // zero in the rows <= k
    if (h == 0) out[HL::v + k * NN + row] = v_row;
    const bool warp_live = warp * 16 + 15 > k;                  // some row of this warp is in the trailing block
    const T* xk = xs[kb];
    T p_row = T(0.0);
    if (warp_live) {
      T acc[4] = {T(0.0), T(0.0), T(0.0), T(0.0)};
#pragma unroll
      for (int i = 0; i < kNc; ++i) {
        T xv[kCh];
        ld_vec<T, kCh>(xk + (2 * i + h) * kCh, xv);
#pragma unroll
        for (int t = 0; t < kCh; ++t) acc[t & 3] = fma(a[i * kCh + t], xv[t], acc[t & 3]);
      }
      T s = (acc[0] + acc[1]) + (acc[2] + acc[3]);
      s += __shfl_xor_sync(FULL, s, 1);
      p_row = row > k ? b * fma(sa, col1, s) : T(0.0);          // x holds x_0 where v holds x_0 + sa: add sa A[row][k+1]
      T pv = h == 0 ? p_row * v_row : T(0.0);
#pragma unroll
      for (int o = 2; o < 32; o <<= 1) pv += __shfl_xor_sync(FULL, pv, o);
      if (lane == 0) pvp[warp] = pv;
    } else if (lane == 0) {
      pvp[warp] = T(0.0);
    }
    if (h == 0) ps[row] = p_row;
    __syncthreads();                                            // p and the parts of p.v are in place
    T c0 = col1;                                                // becomes A[row][k + 1] after the update
    if (warp_live) {
      T pvs = pvp[0];
#pragma unroll
      for (int wi = 1; wi < kWarps; ++wi) pvs += pvp[wi];
      const T hb = T(0.5) * b * pvs;
      const T w_row = p_row - hb * v_row;
      // a - v_row (p_c - hb v_c) - w_row v_c = a - v_row p_c + (v_row hb - w_row) v_c, with x in the place of v: the
      // entry of column k + 1, where the two differ, is never read from the registers again
      const T g = v_row * hb - w_row, nv = -v_row;
#pragma unroll
      for (int i = 0; i < kNc; ++i) {
        T xv[kCh], pc[kCh];
        ld_vec<T, kCh>(xk + (2 * i + h) * kCh, xv);
        ld_vec<T, kCh>(ps + (2 * i + h) * kCh, pc);
#pragma unroll
        for (int t = 0; t < kCh; ++t) a[i * kCh + t] = fma(g, xv[t], fma(nv, pc[t], a[i * kCh + t]));
      }
      const T vk1 = x0 + sa, wk1 = ps[k + 1] - hb * vk1;        // column k + 1 from its value before the update
      c0 = col1 - (v_row * wk1 + w_row * vk1);
    }
    col1 = column(k + 2);
    publish(k + 1, c0);
  }
  // the last 2 x 2 block: subdiagonal entry and last diagonal entry from row NN - 1
  if (row == NN - 1 && h == 0) { ee_s[NN - 2] = xk_row; dd_s[NN - 1] = col1; }
  if (tid == 0) { ee_s[NN - 1] = T(0.0); beta_s[NN - 2] = T(0.0); beta_s[NN - 1] = T(0.0); out[HL::scale] = scale; }
  __syncthreads();
  if (tid < NN) { out[HL::dd + tid] = dd_s[tid]; out[HL::ee + tid] = ee_s[tid]; out[HL::beta + tid] = beta_s[tid]; }
}

template <int NN, typename T>
__global__ void __launch_bounds__(kEigThreads) k_eig_tridiag(const T* __restrict__ ws, int r, int scale_mode,
                                                             float* __restrict__ Fout, double* __restrict__ lam_out) {
  pdl_wait();                                                   // T and the reflectors come from the kernel before
  pdl_launch_dependents();
  using S = EigSmem<NN, T>;
  constexpr int LD = S::LD;
  auto pos = [](int c) { return c + (c / (NN / kTpr)) * (16 / (int)sizeof(T)); };
  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* A = reinterpret_cast<T*>(smem_raw + S::a + S::a_off);      // T [NN][LD]: reflector k in row k
  T* pbuf = reinterpret_cast<T*>(smem_raw + S::pb);
  T* Z = reinterpret_cast<T*>(smem_raw + S::z);
  T* v = reinterpret_cast<T*>(smem_raw + S::vec);
  T* w = v + NN;
  T* dd = w + NN;
  T* ee = dd + NN;
  T* e2 = ee + NN;
  T* beta = e2 + NN;
  T* lam = reinterpret_cast<T*>(smem_raw + S::lam);
  T* red = reinterpret_cast<T*>(smem_raw + S::red);
  int* cstart = reinterpret_cast<int*>(smem_raw + S::cst);
  int* flags = cstart + kEigMaxR;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float* Fo = Fout + (i64)blockIdx.x * NN * r;
  int turn = 0;

  // ---- 1. the tridiagonal form and the reflectors come from k_householder -----------------------------------
  using HL = HhLayout<NN>;
  const T* hh = ws + (i64)blockIdx.x * HL::stride;
  const T scale = hh[HL::scale];
  if (!(scale > T(0.0)) || !(scale * T(0.0) == T(0.0))) {
    // zero matrix: eigenvalues 0, unit vectors; anything non-finite is left to the error checks downstream
    for (int e = tid; e < NN * r; e += kEigThreads) Fo[e] = (scale_mode == 1 && e / r == e % r) ? 1.f : 0.f;
    if (lam_out) for (int j = tid; j < NN; j += kEigThreads) lam_out[(i64)blockIdx.x * NN + j] = 0.0;
    return;
  }
  if (tid < NN) { dd[tid] = hh[HL::dd + tid]; ee[tid] = hh[HL::ee + tid]; beta[tid] = hh[HL::beta + tid]; }
  __syncthreads();
  if (tid < NN) e2[tid] = fmax(ee[tid] * ee[tid], EigNum<T>::e2_min);   // strictly positive: see sturm_count
  T g = T(0.0);
  if (tid < NN) g = fabs(dd[tid]) + fabs(ee[tid]) + (tid > 0 ? fabs(ee[tid - 1]) : T(0.0));
  const T tnorm = cta_max(g, red, turn);                   // Gershgorin bound on |lambda|; also makes e2[] visible

  // ---- 2. multi-section: 8 threads per eigenvalue, 9-fold interval reduction per pass -----------------
  // (the Sturm count is a chain of dependent reciprocals and multiply-adds: 16 warps of such chains keep the
  // schedulers busy, more probes per eigenvalue would only queue)
  {
    constexpr int kProbes = 8;
    if (tid < kProbes * kEigMaxR) {                             // whole warps: 4 eigenvalues per warp
      const int j = tid / kProbes, t = tid % kProbes;           // eigenvalue (j+1)-th largest, probe point t
      const bool active = j < r;
      const int kth = NN - 1 - j;                               // ascending index
      T lo = -tnorm, hi = tnorm;
      for (int it = 0; it < EigNum<T>::passes; ++it) {
        const T wdt = (hi - lo) * (T(1.0) / T(kProbes + 1));
        const T x = lo + wdt * (T)(t + 1);
        const bool below = active && sturm_count<NN, T>(dd, e2, x) <= kth;   // eigenvalue kth is >= x
        const unsigned bal = __ballot_sync(0xffffffffu, below);
        const int s = __popc((bal >> (lane & ~(kProbes - 1))) & ((1u << kProbes) - 1u));   // probes of this group still below the eigenvalue
        const T nlo = lo + wdt * (T)s;
        hi = s < kProbes ? lo + wdt * (T)(s + 1) : hi;
        lo = nlo;
      }
      if (active && t == 0) lam[j] = T(0.5) * (lo + hi);
    }
  }
  __syncthreads();

  // ---- 3. inverse iteration: thread j computes eigenvector j of T ------------------------------------
  if (tid < r) {
    const T shift = lam[tid];
    const T tiny = tnorm * EigNum<T>::pivot;
    // per row of U: 1 / pivot, the two superdiagonal entries times 1 / pivot, and the multiplier of the elimination
    struct alignas(16) Fac { T ip, u1, u2, m; };
    constexpr int fs = S::fac_in_smem ? kEigMaxR : 1;       // stride between consecutive rows of one vector's factors
    Fac fac_local[S::fac_in_smem ? 1 : NN];
    Fac* fac = fac_local;
    if constexpr (S::fac_in_smem) fac = reinterpret_cast<Fac*>(smem_raw + S::a) + tid;
    unsigned swp[NN / 32];                                  // bit i: rows i and i + 1 were swapped
    T acur = dd[0] - shift, ucur = ee[0];                 // current row i: diagonal and superdiagonal entries
#pragma unroll
    for (int q = 0; q < NN / 32; ++q) {
      unsigned w = 0u;
      for (int b0 = 0; b0 < 32; b0 += 4) {
        // rows i0 .. i0 + 3 (row NN - 1 has no successor: its step is masked out); operands first, then the chain
        const int i0 = 32 * q + b0;
        T dv[4], ev[5];
#pragma unroll
        for (int u = 0; u < 4; ++u) dv[u] = i0 + u + 1 < NN ? dd[i0 + u + 1] : T(0.0);
#pragma unroll
        for (int u = 0; u < 5; ++u) ev[u] = i0 + u < NN ? ee[i0 + u] : T(0.0);
        Fac fo[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          // row i against row i + 1 = (sub, anext, unext): the larger leading entry becomes the pivot; both cases run
          // the same instructions (selects), so the lanes of a warp stay together
          const bool on = i0 + u < NN - 1;
          const T sub = ev[u];
          const T anext = dv[u] - shift, unext = ev[u + 1];       // ee[NN-1] = 0
          const bool sw = !(fabs(acur) >= fabs(sub));
          T piv = sw ? sub : acur;
          if (fabs(piv) <= tiny) piv = piv >= T(0.0) ? tiny : -tiny;
          const T ip = chain_rcp(piv);
          const T m = (sw ? acur : sub) * ip;
          w |= (unsigned)(sw && on) << (b0 + u);
          fo[u] = Fac{ip, (sw ? anext : ucur) * ip, sw ? unext * ip : T(0.0), m};
          const T top = sw ? ucur : anext, und = sw ? anext : ucur;
          acur = on ? fma(-m, und, top) : acur;
          ucur = on ? (sw ? -m * unext : unext) : ucur;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (i0 + u < NN - 1) fac[(i0 + u) * fs] = fo[u];
      }
      swp[q] = w;
    }
    {
      T piv = acur;
      if (fabs(piv) <= tiny) piv = piv >= T(0.0) ? tiny : -tiny;
      fac[(NN - 1) * fs] = Fac{T(1.0) / piv, T(0.0), T(0.0), T(0.0)};
    }
    T* z = Z + tid;                                        // z_i = z[i * kZld]
    for (int i = 0; i < NN; ++i) z[i * kZld] = hash_unit(i, tid);
    // Both sweeps run in blocks of four rows whose operands are fetched before the dependent chain starts (the
    // compiler keeps every load behind the previous store to shared memory otherwise).
    unsigned* swp_s = reinterpret_cast<unsigned*>(pbuf) + tid;      // [NN / 32][kEigMaxR]; pbuf is idle until step 4
#pragma unroll
    for (int q = 0; q < NN / 32; ++q) swp_s[q * kEigMaxR] = swp[q];
    constexpr int kBlk = 4, kFull = (NN - 1) / kBlk * kBlk;        // rows 0 .. kFull - 1 in blocks, the rest one by one
    for (int it = 0; it < 3; ++it) {
      T zi = z[0];
      for (int i0 = 0; i0 < kFull; i0 += kBlk) {                    // forward elimination
        T zn[kBlk], mm[kBlk], kp[kBlk];
        const unsigned bits = swp_s[(i0 >> 5) * kEigMaxR] >> (i0 & 31);
#pragma unroll
        for (int u = 0; u < kBlk; ++u) { zn[u] = z[(i0 + u + 1) * kZld]; mm[u] = fac[(i0 + u) * fs].m; }
#pragma unroll
        for (int u = 0; u < kBlk; ++u) {
          const bool sw = (bits >> u) & 1u;
          kp[u] = sw ? zn[u] : zi;
          zi = fma(-mm[u], kp[u], sw ? zi : zn[u]);
        }
#pragma unroll
        for (int u = 0; u < kBlk; ++u) z[(i0 + u) * kZld] = kp[u];
      }
      for (int i = kFull; i < NN - 1; ++i) {
        const T zn = z[(i + 1) * kZld];
        const bool sw = (swp_s[(i >> 5) * kEigMaxR] >> (i & 31)) & 1u;
        const T keep = sw ? zn : zi, other = sw ? zi : zn;
        z[i * kZld] = keep;
        zi = fma(-fac[i * fs].m, keep, other);
      }
      T z1 = zi * fac[(NN - 1) * fs].ip, z2 = T(0.0);                // back substitution
      z[(NN - 1) * kZld] = z1;
      T big = fabs(z1);
      for (int i = NN - 2; i >= kFull; --i) {
        const Fac f = fac[i * fs];
        const T zz = fma(-f.u1, z1, fma(-f.u2, z2, z[i * kZld] * f.ip));
        z[i * kZld] = zz;
        big = fmax(big, fabs(zz));
        z2 = z1; z1 = zz;
      }
      for (int i0 = kFull - kBlk; i0 >= 0; i0 -= kBlk) {
        Fac f[kBlk];
        T zv[kBlk];
#pragma unroll
        for (int u = 0; u < kBlk; ++u) { f[u] = fac[(i0 + u) * fs]; zv[u] = z[(i0 + u) * kZld] * f[u].ip; }
#pragma unroll
        for (int u = kBlk - 1; u >= 0; --u) {
          const T zz = fma(-f[u].u1, z1, fma(-f[u].u2, z2, zv[u]));
          zv[u] = zz;
          big = fmax(big, fabs(zz));
          z2 = z1; z1 = zz;
        }
#pragma unroll
        for (int u = 0; u < kBlk; ++u) z[(i0 + u) * kZld] = zv[u];
      }
      const T sc = big > T(0.0) ? T(1.0) / big : T(1.0);
      for (int i = 0; i < NN; ++i) z[i * kZld] *= sc;
    }
    T nn = T(0.0);
    for (int i = 0; i < NN; ++i) nn = fma(z[i * kZld], z[i * kZld], nn);
    const T sc = nn > T(0.0) ? rsqrt(nn) : T(0.0);
    for (int i = 0; i < NN; ++i) z[i * kZld] *= sc;
  }
  __syncthreads();

  if constexpr (S::a_off != 0) {
    // the factors are dead: start fetching the reflectors (16 bytes per copy) for step 6
    constexpr int kV = 16 / (int)sizeof(T);
    for (int c = tid; c < (NN - 2) * NN / kV; c += kEigThreads) {
      const int e = c * kV;
      const unsigned dst = (unsigned)__cvta_generic_to_shared(A + (e / NN) * LD + pos(e % NN));
      asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(hh + HL::v + e) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  // ---- 4. groups of close eigenvalues: Gram-Schmidt inside each group ---------------------------------
  if (tid == 0) {
    const T gap = EigNum<T>::group_gap * tnorm;
    int start = 0;
    for (int j = 0; j < r; ++j) {
      if (j > 0 && fabs(lam[j - 1] - lam[j]) >= gap) start = j;
      cstart[j] = start;
    }
    flags[0] = 0;
  }
  __syncthreads();
  // vector a of a group is orthogonalised against all earlier vectors of the group at once: every warp
  // forms some of the inner products, then every thread subtracts its share; two passes per vector
  // (classical Gram-Schmidt with re-orthogonalisation)
  for (int j0 = 0; j0 < r;) {
    int j1 = j0;
    while (j1 + 1 < r && cstart[j1 + 1] == j0) ++j1;
    for (int a = j0 + 1; a <= j1; ++a) {
      for (int pass = 0; pass < 2; ++pass) {
        for (int bq = j0 + warp; bq < a; bq += 32) {
          T dot = T(0.0);
          for (int i = lane; i < NN; i += 32) dot = fma(Z[i * kZld + bq], Z[i * kZld + a], dot);
          dot = warp_sum(dot);
          if (lane == 0) pbuf[bq] = dot;
        }
        __syncthreads();
        if (tid < NN) {
          T acc = Z[tid * kZld + a];
          for (int bq = j0; bq < a; ++bq) acc = fma(-pbuf[bq], Z[tid * kZld + bq], acc);
          Z[tid * kZld + a] = acc;
        }
        __syncthreads();
      }
      T nn = T(0.0);
      if (tid < NN) nn = Z[tid * kZld + a] * Z[tid * kZld + a];
      nn = cta_sum(nn, red, turn);
      const T sc = nn > T(0.0) ? rsqrt(nn) : T(0.0);
      if (tid < NN) Z[tid * kZld + a] *= sc;
      __syncthreads();
    }
    j0 = j1 + 1;
  }
  // Polish: outside those (rare) tight groups the vectors of close eigenvalues are orthogonal only to about
  // eps ||T|| / gap.  One step Z <- Z (3 I - Z^T Z) / 2 squares the deviation of Z^T Z from the identity; steps are
  // taken until it is below polish_tol (normally one), and a basis that does not get there is left to the fallback.
  // Everything here is spread over the whole CTA, where the Gram-Schmidt loop above is sequential in the vectors.
  for (int i = tid; i < NN * (kEigMaxR - r); i += kEigThreads)    // unused columns read as zero below
    Z[(i / (kEigMaxR - r)) * kZld + r + i % (kEigMaxR - r)] = T(0.0);
  T* Gs = reinterpret_cast<T*>(smem_raw + S::a);                   // [4][64][64]: partial Gram matrices, then W
  bool polished = false;
  for (int step = 0; step < 4 && !polished; ++step) {
    {
      // Z^T Z in 4 x 4 tiles; the rows of Z are split over the four quarters of the CTA
      const int quarter = tid >> 8, t = tid & 255, a0 = 4 * (t >> 4), b0 = 4 * (t & 15);
      T acc[4][4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = T(0.0);
      if (a0 < r && b0 < r) {
        for (int i = quarter * (NN / 4); i < (quarter + 1) * (NN / 4); ++i) {
          T za[4], zb[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) { za[u] = Z[i * kZld + a0 + u]; zb[u] = Z[i * kZld + b0 + u]; }
#pragma unroll
          for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[u][v] = fma(za[u], zb[v], acc[u][v]);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) Gs[quarter * 4096 + (a0 + u) * 64 + b0 + v] = acc[u][v];
      if (tid == 0) flags[1] = 0;
    }
    __syncthreads();
    {
      // sum of the four parts; W = (3 I - G) / 2 takes the place of G
      T dev = T(0.0);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int e = 4 * tid + q, row = e >> 6, col = e & 63;
        const T g = (Gs[e] + Gs[4096 + e]) + (Gs[8192 + e] + Gs[12288 + e]);
        const T id = row == col ? T(1.0) : T(0.0);
        if (row < r && col < r) dev = fmax(dev, fabs(g - id));
        Gs[e] = T(1.5) * id - T(0.5) * g;
      }
      if (!(dev <= EigNum<T>::polish_tol)) flags[1] = 1;
    }
    __syncthreads();
    polished = flags[1] == 0;                                      // uniform
    if (!polished && step < 3) {
      const int i0 = 2 * (tid >> 4), j0 = 4 * (tid & 15);
      T o[2][4];
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) o[u][v] = T(0.0);
      if (i0 < NN) {
        for (int bq = 0; bq < r; ++bq) {
          const T z0 = Z[i0 * kZld + bq], z1 = Z[(i0 + 1) * kZld + bq];
          T wv[4];
          ld_vec<T, 4>(Gs + bq * 64 + j0, wv);
#pragma unroll
          for (int v = 0; v < 4; ++v) { o[0][v] = fma(z0, wv[v], o[0][v]); o[1][v] = fma(z1, wv[v], o[1][v]); }
        }
      }
      __syncthreads();
      if (i0 < NN) {
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
          for (int v = 0; v < 4; ++v) Z[(i0 + u) * kZld + j0 + v] = o[u][v];
      }
      __syncthreads();
    }
  }

  // ---- 5. Rayleigh quotients, residuals, orthogonality -------------------------------------------------
  bool bad = false;
  if (tid < r) {
    const T* z = Z + tid;
    T num = T(0.0), den = T(0.0);
    for (int i = 0; i < NN; ++i) {
      const T zi = z[i * kZld];
      T t = dd[i] * zi;
      if (i > 0) t = fma(ee[i - 1], z[(i - 1) * kZld], t);
      if (i + 1 < NN) t = fma(ee[i], z[(i + 1) * kZld], t);
      num = fma(zi, t, num);
      den = fma(zi, zi, den);
    }
    const T rq = den > T(0.0) ? num / den : T(0.0);
    T res = T(0.0);
    for (int i = 0; i < NN; ++i) {
      const T zi = z[i * kZld];
      T t = (dd[i] - rq) * zi;
      if (i > 0) t = fma(ee[i - 1], z[(i - 1) * kZld], t);
      if (i + 1 < NN) t = fma(ee[i], z[(i + 1) * kZld], t);
      res = fmax(res, fabs(t));
    }
    lam[tid] = rq;
    bad = !(res <= EigNum<T>::res_tol * tnorm) || !(fabs(den - T(1.0)) <= EigNum<T>::orth_tol);
  }
  bad |= !polished;                                             // all pairwise inner products were checked above
  if (bad) flags[0] = 1;
  __syncthreads();
  if (flags[0]) {
    if (tid == 0) Fo[0] = __int_as_float(0x7fc00000);           // marked for the Jacobi kernel
    return;
  }

  // ---- 6. back-transformation z <- H_0 ... H_{n-3} z, scaling, output -------------------------------------
  if constexpr (S::a_off != 0) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  } else {
    for (int e = tid; e < (NN - 2) * NN; e += kEigThreads) A[(e / NN) * LD + pos(e % NN)] = hh[HL::v + e];
  }
  __syncthreads();
  {
    constexpr int tpv = 16;                                      // threads per vector (1024 threads cover 64 vectors)
    constexpr int npt = NN / tpv;                                // entries of the vector per thread, kept in registers
    const int j = tid / tpv, q = tid % tpv;
    // thread q holds entries i = q, q + 16, ...; the reflector is stored with exact zeros up to entry k, so no entry
    // needs a test.  The reflector of the next step is fetched while the sum of the current one travels through the
    // shuffles.
    if ((tid >> 5) * (32 / tpv) < r) {                           // whole warps (two vectors each)
      const bool active = j < r;
      T zr[npt];
#pragma unroll
      for (int t = 0; t < npt; ++t) zr[t] = active ? Z[(q + tpv * t) * kZld + j] : T(0.0);
      T av[npt], an[npt];
      T bk = beta[NN - 3];
#pragma unroll
      for (int t = 0; t < npt; ++t) av[t] = A[(NN - 3) * LD + pos(q + tpv * t)];
      for (int k = NN - 3; k >= 0; --k) {
        const int kn = k > 0 ? k - 1 : 0;
        const T bn = beta[kn];
#pragma unroll
        for (int t = 0; t < npt; ++t) an[t] = A[kn * LD + pos(q + tpv * t)];
        T d0 = T(0.0), d1 = T(0.0);
#pragma unroll
        for (int t = 0; t < npt; t += 2) { d0 = fma(av[t], zr[t], d0); d1 = fma(av[t + 1], zr[t + 1], d1); }
        T dot = d0 + d1;
#pragma unroll
        for (int o = 1; o < tpv; o <<= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        const T f = bk * dot;                                        // b_k = 0 marks a step without reflector
#pragma unroll
        for (int t = 0; t < npt; ++t) { zr[t] = fma(-f, av[t], zr[t]); av[t] = an[t]; }
        bk = bn;
      }
      if (active) {
#pragma unroll
        for (int t = 0; t < npt; ++t) Z[(q + tpv * t) * kZld + j] = zr[t];
      }
    }
  }
  __syncthreads();
  T part = tid < r ? fmax(lam[tid], T(0.0)) : T(0.0);
  const T mean = cta_sum(part, red, turn) / (T)r;
  if (lam_out)
    for (int j = tid; j < NN; j += kEigThreads) lam_out[(i64)blockIdx.x * NN + j] = j < r ? (double)(lam[j] * scale) : 0.0;
  for (int e = tid; e < NN * r; e += kEigThreads) {
    const int rw = e / r, j = e % r;
    T sc = T(1.0);
    if (scale_mode == 0) sc = mean > T(0.0) ? sqrt(fmax(lam[j], T(0.0)) / mean) : T(0.0);
    Fo[e] = (float)(Z[rw * kZld + j] * sc);
  }
}

// Cyclic Jacobi in float64 (A in shared memory, one CTA per matrix, in-place 2x2 block updates):
// slow and unconditionally robust; processes only the matrices that the kernel above marked.
template <int NN>
__global__ void __launch_bounds__(1024) k_jacobi_eig_f64(const double* __restrict__ Min, i64 stride, int r, int scale_mode,
                                                         float* __restrict__ Fout, double* __restrict__ lam_out) {
  pdl_wait();                                                   // the marks come from the kernel before
  pdl_launch_dependents();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* A = reinterpret_cast<double*>(smem_raw);                 // [NN][NN+1]
  float* V = reinterpret_cast<float*>(A + NN * (NN + 1));          // [NN][NN+1]
  double* cs = reinterpret_cast<double*>(V + NN * (NN + 1) + (NN & 1));   // [NN/2][2]
  int* pq = reinterpret_cast<int*>(cs + NN);                        // [NN/2][2]
  double* red = reinterpret_cast<double*>(pq + NN);                 // [34]
  __shared__ int s_rank[NN];
  __shared__ int s_marked;
  constexpr int LD = NN + 1;
  const int tid = threadIdx.x, nt = blockDim.x;
  if (tid == 0) s_marked = isnan(Fout[(i64)blockIdx.x * NN * r]);
  __syncthreads();
  if (!s_marked) return;
  const double* Mi = Min + (i64)blockIdx.x * stride;
  for (int e = tid; e < NN * NN; e += nt) {
    const int i = e / NN, j = e % NN;
    A[i * LD + j] = 0.5 * (Mi[e] + Mi[j * NN + i]);
    V[i * LD + j] = i == j ? 1.f : 0.f;
  }
  __syncthreads();
  double fro = 0.0;
  for (int e = tid; e < NN * NN; e += nt) { const double a = A[(e / NN) * LD + e % NN]; fro += a * a; }
  fro = block_sum(fro, red);
  const double tol = fro * 1e-26;
  for (int sweep = 0; sweep < 20; ++sweep) {
    double off = 0.0;
    for (int e = tid; e < NN * NN; e += nt) {
      const int i = e / NN, j = e % NN;
      if (i != j) { const double a = A[i * LD + j]; off += a * a; }
    }
    off = block_sum(off, red);
    if (!(off > tol)) break;
    for (int round = 0; round < NN - 1; ++round) {
      if (tid < NN / 2) {
        int p, q;
        if (tid == 0) { p = NN - 1; q = round; }
        else { p = (round + tid) % (NN - 1); q = (round - tid + (NN - 1)) % (NN - 1); }
        if (p > q) { const int t = p; p = q; q = t; }
        const double app = A[p * LD + p], aqq = A[q * LD + q], apq = A[p * LD + q];
        double c = 1.0, s = 0.0;
        if (fabs(apq) > 1e-300 && apq * apq > 1e-34 * fabs(app * aqq) ) {
          const double tau = (aqq - app) / (2.0 * apq);
          const double t = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
          c = 1.0 / sqrt(1.0 + t * t);
          s = t * c;
        }
        pq[2 * tid] = p; pq[2 * tid + 1] = q;
        cs[2 * tid] = c; cs[2 * tid + 1] = s;
      }
      __syncthreads();
      for (int e = tid; e < (NN / 2) * (NN / 2); e += nt) {
        const int ki = e / (NN / 2), kj = e % (NN / 2);
        const int pi = pq[2 * ki], qi = pq[2 * ki + 1], pj = pq[2 * kj], qj = pq[2 * kj + 1];
        const double ci = cs[2 * ki], si = cs[2 * ki + 1], cj = cs[2 * kj], sj = cs[2 * kj + 1];
        const double a00 = A[pi * LD + pj], a01 = A[pi * LD + qj], a10 = A[qi * LD + pj], a11 = A[qi * LD + qj];
        // rows: J_i^T from the left
        const double b00 = ci * a00 - si * a10, b01 = ci * a01 - si * a11;
        const double b10 = si * a00 + ci * a10, b11 = si * a01 + ci * a11;
        // columns: J_j from the right
        A[pi * LD + pj] = cj * b00 - sj * b01; A[pi * LD + qj] = sj * b00 + cj * b01;
        A[qi * LD + pj] = cj * b10 - sj * b11; A[qi * LD + qj] = sj * b10 + cj * b11;
      }
      for (int e = tid; e < NN * (NN / 2); e += nt) {
        const int i = e / (NN / 2), kj = e % (NN / 2);
        const int pj = pq[2 * kj], qj = pq[2 * kj + 1];
        const float cj = (float)cs[2 * kj], sj = (float)cs[2 * kj + 1];
        const float vp = V[i * LD + pj], vq = V[i * LD + qj];
        V[i * LD + pj] = cj * vp - sj * vq;
        V[i * LD + qj] = sj * vp + cj * vq;
      }
      __syncthreads();
    }
  }
  // rank eigenvalues descending (ties by index), scale and emit the leading r
  if (tid < NN) {
    const double li = A[tid * LD + tid];
    int rank = 0;
    for (int j = 0; j < NN; ++j) {
      const double lj = A[j * LD + j];
      rank += (lj > li) || (lj == li && j < tid);
    }
    s_rank[tid] = rank;
    if (lam_out) lam_out[(i64)blockIdx.x * NN + rank] = li;
  }
  __syncthreads();
  double part = 0.0;
  if (tid < NN && s_rank[tid] < r) part = fmax(A[tid * LD + tid], 0.0);
  const double mean = block_sum(part, red) / (double)r;
  for (int e = tid; e < NN * NN; e += nt) {
    const int i = e / NN, col = e % NN;     // column `col` of V is the eigenvector of A[col][col]
    const int rank = s_rank[col];
    if (rank < r) {
      float sc = 1.f;
      if (scale_mode == 0) sc = mean > 0.0 ? (float)sqrt(fmax(A[col * LD + col], 0.0) / mean) : 0.f;
      Fout[(i64)blockIdx.x * NN * r + (i64)i * r + rank] = V[i * LD + col] * sc;
    }
  }
}

size_t jacobi64_smem(int n) {
  return (size_t)n * (n + 1) * 8 + (size_t)(n * (n + 1) + (n & 1)) * 4 + n * 8 + n * 4 + 34 * 8 + 16;
}

}  // namespace

cudaError_t init_eigen() {
  cudaError_t e = cudaFuncSetAttribute(k_eig_tridiag<128, double>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)EigSmem<128, double>::total);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_eig_tridiag<64, double>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)EigSmem<64, double>::total);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_eig_tridiag<128, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)EigSmem<128, float>::total);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_eig_tridiag<64, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)EigSmem<64, float>::total);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_jacobi_eig_f64<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)jacobi64_smem(128));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_jacobi_eig_f64<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)jacobi64_smem(64));
}

size_t eig_scratch_doubles(int batch, int n) { return (size_t)batch * ((size_t)n * n + 3 * n + 4); }

// Min: `batch` symmetric n x n matrices (n = 64 or 128), `stride` doubles apart; r <= 64 leading pairs.
// scale_mode 0: columns scaled by sqrt(lambda_j / mean retained lambda) (feature map of Section 4.1);
// 1: orthonormal columns (basis of Eq. 9).  precise: float64 arithmetic.  Fout [batch][n][r];
// lam_out [batch][n] or null (entries >= r are 0).  ws: eig_scratch_doubles(batch, n) doubles.
void launch_eig_top(const double* Min, i64 stride, int batch, int n, int r, int scale_mode, bool precise, float* Fout,
                    double* lam_out, double* ws, cudaStream_t st) {
#define SPR_EIG(NN, TT)                                                                                        \
  do {                                                                                                         \
    launch_pdl(k_householder<NN, TT>, dim3(batch), dim3(2 * NN), 0, st, Min, stride, reinterpret_cast<TT*>(ws));  \
    launch_pdl(k_eig_tridiag<NN, TT>, dim3(batch), dim3(kEigThreads), EigSmem<NN, TT>::total, st,               \
               reinterpret_cast<const TT*>(ws), r, scale_mode, Fout, lam_out);                                   \
  } while (0)
  if (n == 128) {
    if (precise) SPR_EIG(128, double); else SPR_EIG(128, float);
    launch_pdl(k_jacobi_eig_f64<128>, dim3(batch), dim3(1024), jacobi64_smem(128), st, Min, stride, r, scale_mode, Fout, lam_out);
  } else {
    if (precise) SPR_EIG(64, double); else SPR_EIG(64, float);
    launch_pdl(k_jacobi_eig_f64<64>, dim3(batch), dim3(1024), jacobi64_smem(64), st, Min, stride, r, scale_mode, Fout, lam_out);
  }
#undef SPR_EIG
}

}  // namespace spr
