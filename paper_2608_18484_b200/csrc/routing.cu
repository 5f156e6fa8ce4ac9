// Shared routing (Section 4.3) and query-group-stratified probe selection
// (Algorithm A.1, Appendix A.2).
#include "kernels.cuh"

namespace spr {

// =============================================================================
// Cell scores.  The paper fixes the pair budget and the cost model but no score;
// this library scores cell (a,b) by the attention weight a query at the centroid
// theta_a would give ONE key at the centroid kappa_b:
//   p_ab = exp(l_ab - LSE_a),  l_ab = s theta_a.kappa_b,
//   LSE_a = log sum_{b non-empty} n_b exp(l_ab).
// One CTA per eight query groups: the kappa slabs staged through shared memory are reused by all eight.
// Inner products and exponentials in float32, the weighted sum of the exponentials in float64, scores stored as float32.
// =============================================================================
constexpr int kCsRows = 8;     // query groups per CTA

__global__ void __launch_bounds__(256) k_cell_scores(const float* __restrict__ theta, const float* __restrict__ kappa,
                                                     const int* __restrict__ nq, const int* __restrict__ nk, int Cq,
                                                     int Ck, int d, float scale, float* __restrict__ score, int kv_div) {
  pdl_wait();                                                   // the group means come from the kernels before
  pdl_launch_dependents();
  __shared__ float th[kCsRows][128];
  __shared__ float kt[32][257];                              // a [256 groups x 32 dims] slab of kappa, transposed
  const int bh = blockIdx.y, a0 = blockIdx.x * kCsRows;
  const int kvh = bh / kv_div;                               // K/V head of this query head
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int e = tid; e < kCsRows * d; e += 256) {
    const int r = e / d, k = e % d;
    th[r][k] = a0 + r < Cq ? theta[((i64)bh * Cq + a0 + r) * d + k] : 0.f;
  }
  // phase 1: logits l_ab = s theta_a . kappa_b of eight query groups against all K/V groups
  for (int b0 = 0; b0 < Ck; b0 += 256) {
    float acc[kCsRows];
#pragma unroll
    for (int r = 0; r < kCsRows; ++r) acc[r] = 0.f;
    for (int k0 = 0; k0 < d; k0 += 32) {
      __syncthreads();
#pragma unroll 8
      for (int r = 0; r < 32; ++r) {
        const int b = b0 + warp * 32 + r;
        kt[lane][warp * 32 + r] = (b < Ck && k0 + lane < d) ? kappa[((i64)kvh * Ck + b) * d + k0 + lane] : 0.f;
      }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < 32; ++k) {
        const float kv = kt[k][tid];
#pragma unroll
        for (int r = 0; r < kCsRows; ++r) acc[r] = fmaf(th[r][k0 + k], kv, acc[r]);
      }
    }
    const int b = b0 + tid;
    if (b < Ck) {
#pragma unroll
      for (int r = 0; r < kCsRows; ++r)
        if (a0 + r < Cq) score[((i64)bh * Cq + a0 + r) * Ck + b] = acc[r] * scale;
    }
  }
  __syncthreads();                                           // the block's logits are visible to the block
  // phase 2: one warp per query group: weighted log-sum-exp over the non-empty K/V groups, scores in place
  const int a = a0 + warp;
  if (a >= Cq) return;
  float* out = score + ((i64)bh * Cq + a) * Ck;
  const int* nkh = nk + (i64)kvh * Ck;
  if (nq[(i64)bh * Cq + a] == 0) {
    for (int b = lane; b < Ck; b += 32) out[b] = 0.f;
    return;
  }
  float mx = -3.0e38f;
  for (int b = lane; b < Ck; b += 32)
    if (nkh[b] > 0) mx = fmaxf(mx, out[b]);
  mx = warp_max(mx);
  double z = 0.0;
  for (int b = lane; b < Ck; b += 32)
    if (nkh[b] > 0) z += (double)nkh[b] * (double)expf(out[b] - mx);
  z = warp_sum(z);
  const float lse = mx + (float)log(z);
  for (int b = lane; b < Ck; b += 32) out[b] = nkh[b] > 0 ? expf(out[b] - lse) : 0.f;
}

void launch_cell_scores(const float* theta, const float* kappa, const int* nq, const int* nk, int BH, int Cq, int Ck,
                        int d, float scale, float* score, int kv_div, cudaStream_t st) {
  dim3 grid((Cq + kCsRows - 1) / kCsRows, BH);
  launch_pdl(k_cell_scores, grid, dim3(256), 0, st, theta, kappa, nq, nk, Cq, Ck, d, scale, score, kv_div < 1 ? 1 : kv_div);
}

// =============================================================================
// Cell selection under the pair budget, one CTA per head.
//   1. forced cell per non-empty query group: its best non-empty cell (ties -> lowest b);
//   2. the remaining cells are taken in the order (score desc, a asc, b asc) while the
//      cumulative cost n_a n_b stays within the budget; the first cell that does not
//      fit ends the selection.  Instead of sorting, the cut is located by a binary
//      search over the 32-bit pattern of the (non-negative) float32 scores: the
//      smallest threshold t with cost{cells with bits >= t} <= remaining budget, and
//      the cells whose bits equal t-1 are then walked in (a,b) order.
//   3. CSR emission with ascending b inside a row.
// Everything is integer arithmetic on the given score bits.
// =============================================================================
__device__ __forceinline__ i64 block_sum_i64(i64 v, i64* scratch) { return block_sum<i64>(v, scratch); }

// Eight 32-cell chunks of one score row, loaded together: the scans below are bound by the latency of these reads
__device__ __forceinline__ void load_row_chunks(const unsigned* __restrict__ row, int b00, int Ck, int lane, unsigned (&ub)[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int b = b00 + 32 * j + lane;
    ub[j] = b < Ck ? row[b] : 0u;
  }
}

__global__ void __launch_bounds__(1024) k_route_select(const float* __restrict__ score, const int* __restrict__ nq,
                                                       const int* __restrict__ nk, int Cq, int Ck, i64 budget,
                                                       int select_all, int* __restrict__ route_ptr,
                                                       int* __restrict__ route_idx, RouteState* __restrict__ state,
                                                       i64* __restrict__ pairs_out, int kv_div) {
  pdl_wait();                                                   // the scores come from the kernel before
  pdl_launch_dependents();
  extern __shared__ int sm_route[];
  int* forced = sm_route;            // [Cq]
  int* cnt = forced + Cq;            // [Cq]
  int* nks = cnt + Cq;               // [Ck]
  int* nqs = nks + Ck;               // [Cq]
  __shared__ i64 red[34];
  __shared__ int scratch[34];
  __shared__ i64 s_last_tie;
  const int bh = blockIdx.x;
  const unsigned* u = reinterpret_cast<const unsigned*>(score) + (i64)bh * Cq * Ck;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  for (int b = threadIdx.x; b < Ck; b += blockDim.x) nks[b] = nk[(i64)(bh / kv_div) * Ck + b];
  for (int a = threadIdx.x; a < Cq; a += blockDim.x) nqs[a] = nq[(i64)bh * Cq + a];
  __syncthreads();

  // 1. forced cells
  i64 fcost = 0;
  for (int a = w; a < Cq; a += nw) {
    u64 best = 0;      // (bits+1) << 32 | (0xFFFFFFFF - b): larger = better score, then lower b
    if (nqs[a] > 0)
      for (int b00 = 0; b00 < Ck; b00 += 256) {
        unsigned ub[8];
        load_row_chunks(u + (i64)a * Ck, b00, Ck, lane, ub);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int b = b00 + 32 * j + lane;
          if (b < Ck && nks[b] > 0) {
            const u64 key = (((u64)ub[j] + 1ull) << 32) | (u64)(0xFFFFFFFFu - (unsigned)b);
            best = key > best ? key : best;
          }
        }
      }
    best = warp_max(best);
    const int fb = best ? (int)(0xFFFFFFFFu - (unsigned)(best & 0xFFFFFFFFull)) : -1;
    if (lane == 0) {
      forced[a] = fb;
      if (fb >= 0) fcost += (i64)nqs[a] * nks[fb];
    }
  }
  fcost = block_sum_i64(fcost, red);     // contains a __syncthreads: forced[] visible below
  const i64 rem = budget - fcost;

  // 2. threshold search: S(t) = cost of live, non-forced cells with bits >= t; find the smallest t with
  //    S(t) <= rem.  Radix descent, one byte of the bit pattern per pass: per-warp cost histograms over
  //    the next byte of the cells that share the prefix found so far, then the bucket that contains the
  //    threshold is the first one whose suffix cost fits.
  u64 tstar;
  i64 taken = 0;                        // cost of the cells with bits >= tstar
  if (select_all) tstar = 0;
  else if (rem < 0) tstar = 1ull << 32;
  else {
    i64* whist = reinterpret_cast<i64*>(nqs + Cq + ((Cq + Ck) & 1));   // [nw][256], 8-byte aligned (see route_smem)
    __shared__ i64 s_above;
    __shared__ int s_dstar;
    unsigned prefix = 0;
    i64 above = 0;                      // cost of the cells above the current bucket
    bool all_fit = false;
    for (int level = 0; level < 4; ++level) {
      const int shift = 24 - 8 * level;
      for (int e = threadIdx.x; e < nw * 256; e += blockDim.x) whist[e] = 0;
      __syncthreads();
      i64* myh = whist + w * 256;
      int* hk = reinterpret_cast<int*>(whist + nw * 256) + w * 256;   // per-row key counts by digit, zero between rows
      for (int k = lane; k < 256; k += 32) hk[k] = 0;
      __syncwarp();
      for (int a = w; a < Cq; a += nw) {
        if (nqs[a] == 0) continue;
        const int fb = forced[a];
        const i64 na = nqs[a];
        for (int b00 = 0; b00 < Ck; b00 += 256) {
          unsigned ub[8];
          load_row_chunks(u + (i64)a * Ck, b00, Ck, lane, ub);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int b = b00 + 32 * j + lane;
            if (b00 + 32 * j >= Ck) break;                           // uniform
            const unsigned bits = ub[j];
            const bool in = b < Ck && b != fb && nks[b] > 0 && (level == 0 || (bits >> (shift + 8)) == (prefix >> (shift + 8)));
            // key counts of the row per digit, in the warp's 32-bit histogram: the lanes that share the first
            // lane's digit add up together (the upper bytes of the scores take few values), the others add their own
            const unsigned todo = __ballot_sync(0xffffffffu, in);
            if (todo) {
              const int digit = (bits >> shift) & 255;
              const int dl = __shfl_sync(0xffffffffu, digit, __ffs(todo) - 1);
              const bool mine = in && digit == dl;
              const int keys = __reduce_add_sync(0xffffffffu, mine ? nks[b] : 0);
              if (lane == 0) hk[dl] += keys;
              __syncwarp();
              if (in && !mine) atomicAdd(&hk[digit], nks[b]);
            }
          }
        }
        // the row's counts times its number of queries go to the 64-bit cost histogram
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int d = lane + 32 * k;
          const int v = hk[d];
          if (v) { myh[d] += na * v; hk[d] = 0; }
        }
        __syncwarp();
      }
      __syncthreads();
      if (w == 0) {
        // lane l owns digits 8l .. 8l+7
        i64 loc[8], lsum = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          i64 t = 0;
          for (int ww = 0; ww < nw; ++ww) t += whist[ww * 256 + lane * 8 + k];
          loc[k] = t; lsum += t;
        }
        i64 suf = lsum;                                          // sum over lanes >= this lane
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const i64 t = __shfl_down_sync(0xffffffffu, suf, o); if (lane + o < 32) suf += t; }
        i64 run = suf;                                           // suffix cost from digit 8l
        int first = -1;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          if (first < 0 && above + run <= rem) first = lane * 8 + k;
          run -= loc[k];
        }
        const unsigned have = __ballot_sync(0xffffffffu, first >= 0);
        int dstar = 256;
        if (have) dstar = __shfl_sync(0xffffffffu, first, __ffs(have) - 1);
        // cost of the digits >= dstar
        i64 sfx = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) if (lane * 8 + k >= dstar) sfx += loc[k];
        sfx = warp_sum(sfx);
        if (lane == 0) { s_dstar = dstar; s_above = above + sfx; }
      }
      __syncthreads();
      const int dstar = s_dstar;
      above = s_above;
      if (dstar == 0) { all_fit = true; break; }                 // the whole bucket fits (only possible at the top level)
      prefix |= (unsigned)(dstar - 1) << shift;
    }
    tstar = all_fit ? (u64)prefix : (u64)prefix + 1ull;
    taken = above;
  }
  // tie tier: cells with bits == tstar-1, in (a,b) order, longest prefix that fits
  __shared__ int s_tie_cnt, s_tie_idx[32];
  if (threadIdx.x == 0) { s_last_tie = -1; s_tie_cnt = 0; }
  __syncthreads();
  const bool tie_tier = !select_all && rem >= 0 && tstar > 0 && tstar <= 0xFFFFFFFFull + 1ull;
  // The tier usually holds a single cell: collect its cells in parallel; up to 32 are ordered and
  // cut by one warp, larger tiers (many equal scores) take the sequential walk below.
  if (tie_tier) {
    const unsigned tv = (unsigned)(tstar - 1);
    for (int a = w; a < Cq; a += nw) {
      if (nqs[a] == 0) continue;
      const int fb = forced[a];
      for (int b00 = 0; b00 < Ck; b00 += 256) {
        unsigned ub[8];
        load_row_chunks(u + (i64)a * Ck, b00, Ck, lane, ub);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int b = b00 + 32 * j + lane;
          if (b < Ck && nks[b] > 0 && b != fb && ub[j] == tv) {
            const int pos = atomicAdd(&s_tie_cnt, 1);
            if (pos < 32) s_tie_idx[pos] = a * Ck + b;
          }
        }
      }
    }
  }
  __syncthreads();
  const int tie_cnt = s_tie_cnt;
  if (tie_tier && tie_cnt <= 32 && w == 0) {
    const int idx = lane < tie_cnt ? s_tie_idx[lane] : 0x7fffffff;
    const i64 cost = lane < tie_cnt ? (i64)nqs[idx / Ck] * nks[idx % Ck] : 0;
    i64 cum = taken;                                     // cost of the tier cells up to and including this one, in (a,b) order
    for (int j = 0; j < tie_cnt; ++j) {
      const int oj = __shfl_sync(0xffffffffu, idx, j);
      const i64 cj = __shfl_sync(0xffffffffu, cost, j);
      if (oj <= idx) cum += cj;
    }
    const bool fits = lane < tie_cnt && cum <= rem;      // monotone along the order: costs are positive
    int best = fits ? idx : -1;
    best = warp_max(best);
    if (lane == 0) s_last_tie = best;
  }
  if (tie_tier && tie_cnt > 32 && w == 0) {
    const unsigned tv = (unsigned)(tstar - 1);
    i64 cum = taken, last = -1;
    bool stop = false;
    for (int a = 0; a < Cq && !stop; ++a) {
      if (nqs[a] == 0) continue;
      const int fb = forced[a];
      for (int b0 = 0; b0 < Ck && !stop; b0 += 32) {
        const int b = b0 + lane;
        const bool is = b < Ck && nks[b] > 0 && b != fb && u[(i64)a * Ck + b] == tv;
        i64 c = is ? (i64)nqs[a] * nks[b] : 0;
        i64 inc = c;                                        // inclusive scan over the lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const i64 t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
        const bool over = is && (cum + inc > rem);
        const unsigned om = __ballot_sync(0xffffffffu, over);
        const unsigned im = __ballot_sync(0xffffffffu, is);
        if (om) {
          const unsigned before = im & ((1u << (__ffs(om) - 1)) - 1u);
          if (before) last = (i64)a * Ck + b0 + (31 - __clz(before));
          stop = true;
        } else {
          if (im) last = (i64)a * Ck + b0 + (31 - __clz(im));
          cum += __shfl_sync(0xffffffffu, inc, 31);
        }
      }
    }
    if (lane == 0) s_last_tie = last;
  }
  __syncthreads();
  const i64 last_tie = s_last_tie;
  const unsigned tvv = tie_tier ? (unsigned)(tstar - 1) : 0u;

  auto selected = [&](int a, int b, unsigned bits) -> bool {       // bits = the cell's score word
    if (nqs[a] == 0 || nks[b] == 0) return false;
    if (forced[a] == b) return true;
    if ((u64)bits >= tstar) return true;
    return tie_tier && bits == tvv && (i64)a * Ck + b <= last_tie;
  };

  // 3. counts, offsets, lists
  i64 pairs = 0;
  for (int a = w; a < Cq; a += nw) {
    int c = 0;
    i64 rs = 0;
    for (int b00 = 0; b00 < Ck; b00 += 256) {
      unsigned ub[8];
      load_row_chunks(u + (i64)a * Ck, b00, Ck, lane, ub);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int b = b00 + 32 * j + lane;
        const bool s = b < Ck && selected(a, b, ub[j]);
        c += __popc(__ballot_sync(0xffffffffu, s));
        if (s) rs += nks[b];
      }
    }
    pairs += rs * nqs[a];
    if (lane == 0) cnt[a] = c;
  }
  pairs = block_sum_i64(pairs, red);
  const int total = block_exclusive_scan(cnt, Cq, scratch);
  int* rp = route_ptr + (i64)bh * (Cq + 1);
  int* ri = route_idx + (i64)bh * Cq * Ck;
  for (int a = threadIdx.x; a < Cq; a += blockDim.x) rp[a] = cnt[a];
  if (threadIdx.x == 0) {
    rp[Cq] = total;
    if (state) { state[bh].pairs = pairs; state[bh].cells = total; }
    if (pairs_out) pairs_out[bh] = pairs;
  }
  for (int a = w; a < Cq; a += nw) {
    int pos = cnt[a];
    for (int b00 = 0; b00 < Ck; b00 += 256) {
      unsigned ub[8];
      load_row_chunks(u + (i64)a * Ck, b00, Ck, lane, ub);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int b = b00 + 32 * j + lane;
        const bool s = b < Ck && selected(a, b, ub[j]);
        const unsigned m = __ballot_sync(0xffffffffu, s);
        if (s) ri[pos + __popc(m & ((1u << lane) - 1u))] = b;
        pos += __popc(m);
      }
    }
  }
}

static size_t route_smem(int Cq, int Ck) {      // forced, cnt, nqs [Cq], nks [Ck] ints, then 32 x 256 int64 cost and int32 key histograms
  return (size_t)(3 * Cq + Ck + ((Cq + Ck) & 1)) * sizeof(int) + (size_t)32 * 256 * (sizeof(long long) + sizeof(int));
}
// routed pairs and cells of given routes (used when a plan is imported)
__global__ void __launch_bounds__(256) k_count_pairs(const int* __restrict__ q_off, const int* __restrict__ kv_off,
                                                     const int* __restrict__ route_ptr, const int* __restrict__ route_idx,
                                                     int Cq, int Ck, RouteState* __restrict__ state, int kv_div) {
  __shared__ i64 red[34];
  const int bh = blockIdx.x;
  const int* qo = q_off + (i64)bh * (Cq + 1);
  const int* ko = kv_off + (i64)(bh / kv_div) * (Ck + 1);
  const int* rp = route_ptr + (i64)bh * (Cq + 1);
  const int* ri = route_idx + (i64)bh * Cq * Ck;
  i64 pairs = 0;
  for (int a = threadIdx.x; a < Cq; a += 256) {
    i64 keys = 0;
    for (int t = rp[a]; t < rp[a + 1]; ++t) keys += ko[ri[t] + 1] - ko[ri[t]];
    pairs += keys * (qo[a + 1] - qo[a]);
  }
  pairs = block_sum<i64>(pairs, red);
  if (threadIdx.x == 0) { state[bh].pairs = pairs; state[bh].cells = rp[Cq]; }
}
void launch_count_pairs(const int* q_off, const int* kv_off, const int* route_ptr, const int* route_idx, int BH, int Cq,
                        int Ck, RouteState* state, int kv_div, cudaStream_t st) {
  k_count_pairs<<<BH, 256, 0, st>>>(q_off, kv_off, route_ptr, route_idx, Cq, Ck, state, kv_div < 1 ? 1 : kv_div);
}
void launch_route_select(const float* score, const int* nq, const int* nk, int BH, int Cq, int Ck, i64 budget,
                         int select_all, int* route_ptr, int* route_idx, RouteState* state, i64* pairs_out,
                         int kv_div, cudaStream_t st) {
  launch_pdl(k_route_select, dim3(BH), dim3(1024), route_smem(Cq, Ck), st, score, nq, nk, Cq, Ck, budget, select_all, route_ptr, route_idx,
             state, pairs_out, kv_div < 1 ? 1 : kv_div);
}

// =============================================================================
// Probe selection, Algorithm A.1.  Kernel 1 (one warp per query group): centroid
// c_a of the group in phi_Q space and the distance d_i of every member, stored at
// the member's group-major position.  Kernel 2 (one CTA per head): round t takes,
// from every group that still has rows, the unpicked row with the smallest
// (d_i, i); groups are visited in ascending id; stops at M rows.  Then the
// coverage weights w_p = |G_a| / m_a (Appendix A.2).
// =============================================================================
__global__ void __launch_bounds__(256) k_probe_dist(const float* __restrict__ phi, int ldphi, int r,
                                                    const int* __restrict__ perm, const int* __restrict__ off, int N,
                                                    int C, double* __restrict__ dist) {
  const int bh = blockIdx.y;
  const int g = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (g >= C) return;
  const int lane = threadIdx.x & 31;
  const int p0 = off[(i64)bh * (C + 1) + g], p1 = off[(i64)bh * (C + 1) + g + 1];
  if (p1 <= p0) return;
  const float* ph = phi + (i64)bh * N * ldphi;
  const int* pm = perm + (i64)bh * N;
  // lane owns columns lane, lane + 32, ... (up to four: 128 columns for a semantic query partition); the rows are
  // read eight at a time (the loads are independent, the sums keep their order)
  constexpr int kCols = 4;
  bool has[kCols];
  double cen[kCols];
#pragma unroll
  for (int j = 0; j < kCols; ++j) { has[j] = lane + 32 * j < r; cen[j] = 0.0; }
  for (int p = p0; p < p1; p += 8) {
    float x[8][kCols];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float* row = ph + (i64)pm[min(p + q, p1 - 1)] * ldphi;
#pragma unroll
      for (int j = 0; j < kCols; ++j) x[q][j] = has[j] ? row[lane + 32 * j] : 0.f;
    }
#pragma unroll
    for (int q = 0; q < 8; ++q)
      if (p + q < p1) {
#pragma unroll
        for (int j = 0; j < kCols; ++j) if (has[j]) cen[j] += (double)x[q][j];
      }
  }
#pragma unroll
  for (int j = 0; j < kCols; ++j) cen[j] /= (double)(p1 - p0);
  for (int p = p0; p < p1; p += 8) {
    float x[8][kCols];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float* row = ph + (i64)pm[min(p + q, p1 - 1)] * ldphi;
#pragma unroll
      for (int j = 0; j < kCols; ++j) x[q][j] = has[j] ? row[lane + 32 * j] : 0.f;
    }
    double s[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      s[q] = 0.0;
#pragma unroll
      for (int j = 0; j < kCols; ++j)
        if (has[j]) { const double t = (double)x[q][j] - cen[j]; s[q] += t * t; }
    }
    // eight independent butterflies
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
      for (int q = 0; q < 8; ++q) s[q] += __shfl_xor_sync(0xffffffffu, s[q], o);
    }
#pragma unroll
    for (int q = 0; q < 8; ++q)
      if (lane == q && p + q < p1) dist[(i64)bh * N + p + q] = sqrt(s[q]);
  }
}

__global__ void __launch_bounds__(1024) k_probe_pick(const double* __restrict__ dist, const int* __restrict__ perm,
                                                     const int* __restrict__ off, int N, int C, int M,
                                                     int* __restrict__ probe_idx, float* __restrict__ probe_w) {
  extern __shared__ unsigned char sm_probe[];
  double* prev_d = reinterpret_cast<double*>(sm_probe);       // [C] last picked distance per group
  int* prev_i = reinterpret_cast<int*>(prev_d + C);           // [C] last picked row
  int* pick = prev_i + C;                                     // [C] row picked this round or -1
  int* flag = pick + C;                                       // [C] scan buffer
  int* m_a = flag + C;                                        // [C] probes per group
  int* pgrp = m_a + C;                                        // [M] group of every probe
  __shared__ int scratch[34];
  const int bh = blockIdx.x;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int* of = off + (i64)bh * (C + 1);
  const int* pm = perm + (i64)bh * N;
  const double* ds = dist + (i64)bh * N;
  for (int a = threadIdx.x; a < C; a += blockDim.x) { prev_d[a] = -1.0; prev_i[a] = -1; m_a[a] = 0; }
  __syncthreads();
  int count = 0;
  for (int t = 0; count < M; ++t) {
    for (int a = w; a < C; a += nw) {
      const int p0 = of[a], p1 = of[a + 1];
      int bi = -1;
      double bd = 0.0;
      if (p1 - p0 > t) {
        const double pd = prev_d[a];
        const int pi = prev_i[a];
        for (int p = p0 + lane; p < p1; p += 32) {
          const double dd = ds[p];
          const int i = pm[p];
          const bool after = dd > pd || (dd == pd && i > pi);            // not yet picked
          if (after && (bi < 0 || dd < bd || (dd == bd && i < bi))) { bd = dd; bi = i; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const double od = __shfl_xor_sync(0xffffffffu, bd, o);
          const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (oi >= 0 && (bi < 0 || od < bd || (od == bd && oi < bi))) { bd = od; bi = oi; }
        }
      }
      if (lane == 0) {
        pick[a] = bi;
        flag[a] = bi >= 0;
        if (bi >= 0) { prev_d[a] = bd; prev_i[a] = bi; }
      }
    }
    __syncthreads();
    const int got = block_exclusive_scan(flag, C, scratch);
    for (int a = threadIdx.x; a < C; a += blockDim.x) {
      const int pos = count + flag[a];
      if (pick[a] >= 0 && pos < M) {
        probe_idx[(i64)bh * M + pos] = pick[a];
        pgrp[pos] = a;
        atomicAdd(&m_a[a], 1);
      }
    }
    __syncthreads();
    count += got;
    if (got == 0) break;                       // fewer than M rows exist
  }
  __syncthreads();
  for (int p = threadIdx.x; p < M; p += blockDim.x) {
    if (p < count) {
      const int a = pgrp[p];
      probe_w[(i64)bh * M + p] = (float)(of[a + 1] - of[a]) / (float)m_a[a];
    } else {
      probe_idx[(i64)bh * M + p] = -1;
      probe_w[(i64)bh * M + p] = 0.f;
    }
  }
}

static size_t probe_smem(int C, int M) { return (size_t)C * (8 + 5 * 4) + (size_t)M * 4 + 16; }
cudaError_t init_routing() {
  cudaError_t e = cudaFuncSetAttribute(k_route_select, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)route_smem(kMaxGroups, kMaxGroups));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_probe_pick, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)probe_smem(kMaxGroups, kMaxProbes));
}
void launch_probe_select(const float* phiQ, int ldphi, int r, const int* q_perm, const int* q_off, const int* nq, int BH,
                         int N, int Cq, int M, double* dist_scratch, int* probe_idx, float* probe_w, cudaStream_t st) {
  (void)nq;
  dim3 grid((Cq + 7) / 8, BH);
  k_probe_dist<<<grid, 256, 0, st>>>(phiQ, ldphi, r, q_perm, q_off, N, Cq, dist_scratch);
  k_probe_pick<<<BH, 1024, probe_smem(Cq, M), st>>>(dist_scratch, q_perm, q_off, N, Cq, M, probe_idx, probe_w);
}

}  // namespace spr
