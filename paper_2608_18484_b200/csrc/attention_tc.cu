// Block-sparse / dense attention on the sm_100a tensor cores (bf16, d = d_v = 128).
//
// One CTA processes one 128-row query tile (of one query group, Eq. 3; or of the whole
// head for dense attention, Eq. 1).  Roles:
//   warps 0-7  softmax: two threads per query row (64 score columns each)
//   warp  8    TMA producer: streams the routed keys/values as one concatenated
//              sequence in 16-row boxes (tiles of 128 keys, only range ends are ragged)
//   warp  9    tcgen05.mma issuer; owns the TMEM allocation
// Data path per key tile i:
//   S_i = Q K_i^T      tcgen05.mma (smem x smem -> TMEM, fp32), two S buffers
//   P_i = exp2(.)      softmax threads: tcgen05.ld S, running max / sum, bf16 P -> smem
//   T_i = P_i V_i      tcgen05.mma -> TMEM, accumulated into registers o = (o + T_{i-1}) * corr_i
// Epilogue: O_sp = o / l; correction O_sp A on the tensor cores (A = composed affine map
// of Eq. 9, bf16), + c, store at the original token index (inverse permutation).
// Every mbarrier wait is bounded; on expiry the CTA records SPARSEPR_ERR_TIMEOUT and leaves.
#include <cuda.h>
#include <mutex>
#include "kernels.cuh"
#include "tc_common.cuh"

namespace spr {

namespace tc {

constexpr int kThreads = 320;
constexpr int kTile = 128;            // query rows per CTA, keys per tile
constexpr int kD = 128;
constexpr int kSub = 16;              // rows per TMA box of the K/V stream
constexpr int kSubPerTile = kTile / kSub;
constexpr uint32_t kHalfBytes = kTile * 128;          // one [128 rows x 64 bf16] swizzled block
constexpr uint32_t kTileBytes = 2 * kHalfBytes;       // 32 KB
constexpr uint32_t kSubBytes = kSub * 128;            // 2 KB per box
constexpr int kStages = 2;

struct Smem {                          // offsets from a 1024-byte aligned base
  static constexpr uint32_t q = 0;
  static constexpr uint32_t k = q + kTileBytes;                   // kStages tiles
  static constexpr uint32_t v = k + kStages * kTileBytes;
  static constexpr uint32_t p = v + kStages * kTileBytes;
  static constexpr uint32_t ranges = p + kTileBytes;              // int2[kMaxGroups]: (start row, length)
  static constexpr uint32_t xchg = ranges + kMaxGroups * 8;       // float[2][2][128]
  static constexpr uint32_t meta = xchg + 4 * 128 * 4;            // uint2[4]
  static constexpr uint32_t bars = meta + 4 * 8;                  // 20 mbarriers
  static constexpr uint32_t misc = bars + 20 * 8;                 // tmem base, abort flag, counters
  static constexpr uint32_t total = misc + 64;
};
constexpr size_t kSmemBytes = Smem::total + 1024;                 // slack for manual alignment

enum Bar { Q_FULL = 0, K_FULL = 1, K_EMPTY = 3, V_FULL = 5, V_EMPTY = 7, S_FULL = 9, P_FULL = 11, T_FULL = 12,
           T_EMPTY = 13, C_FULL = 14, META_FULL = 15 };


struct Params {
  int BH, H, N, Cq, Ck, sparse;
  float scale_log2;
  const int *q_off, *kv_off, *route_ptr, *route_idx, *q_perm, *tile_off;
  const float* c;                 // [BH][128] or null
  int has_corr;
  __nv_bfloat16* O; i64 os[3];
  float* O_sparse;
  int* err;
};

// write 8 consecutive bf16 (one 16-byte chunk) of row `row`, chunk index `chunk` (0..15 over 128 columns)
__device__ __forceinline__ void store_p_chunk(uint32_t p_base, int row, int chunk, const float* v8) {
  const uint32_t half = chunk >> 3, c = chunk & 7;
  const uint32_t addr = p_base + half * kHalfBytes + row * 128 + ((c ^ (row & 7)) << 4);
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(v8[2 * i], v8[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
k_attention_tc(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
               const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapA, Params prm) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw);
  int2* ranges = reinterpret_cast<int2*>(sm + Smem::ranges);
  float* xchg = reinterpret_cast<float*>(sm + Smem::xchg);
  uint2* meta = reinterpret_cast<uint2*>(sm + Smem::meta);
  volatile int* misc = reinterpret_cast<volatile int*>(sm + Smem::misc);   // [0] tmem base, [1] abort, [2] total boxes
  const uint32_t bars = base + Smem::bars;
  auto bar = [&](int i) { return bars + 8u * i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y, b = bh / prm.H, h = bh % prm.H;
  // once any CTA has recorded a timeout the remaining CTAs of the launch leave at once
  __shared__ int s_skip;
  if (tid == 0) s_skip = prm.err != nullptr && *reinterpret_cast<volatile int*>(prm.err) == SPARSEPR_ERR_TIMEOUT;
  __syncthreads();
  if (s_skip) return;

  // ---- which query tile ---------------------------------------------------------------
  int row0, nrows, nroute;
  const int* ridx = nullptr;
  const int* kvoff = nullptr;
  if (prm.sparse) {
    const int* toff = prm.tile_off + (i64)bh * (prm.Cq + 1);
    if ((int)blockIdx.x >= toff[prm.Cq]) return;
    int lo = 0, hi = prm.Cq - 1;
    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (toff[mid] <= (int)blockIdx.x) lo = mid; else hi = mid - 1; }
    const int g = lo;
    const int* qoff = prm.q_off + (i64)bh * (prm.Cq + 1);
    row0 = qoff[g] + ((int)blockIdx.x - toff[g]) * kTile;
    nrows = min(kTile, qoff[g + 1] - row0);
    const int* rp = prm.route_ptr + (i64)bh * (prm.Cq + 1);
    ridx = prm.route_idx + (i64)bh * prm.Cq * prm.Ck + rp[g];
    nroute = rp[g + 1] - rp[g];
    kvoff = prm.kv_off + (i64)bh * (prm.Ck + 1);
  } else {
    row0 = blockIdx.x * kTile;
    nrows = min(kTile, prm.N - row0);
    nroute = 1;
  }

  // ---- set-up: barriers, TMEM, key ranges ---------------------------------------------------
  if (tid == 0) {
    mbar_init(bar(Q_FULL), 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar(K_FULL + s), 1); mbar_init(bar(K_EMPTY + s), 1);
      mbar_init(bar(V_FULL + s), 1); mbar_init(bar(V_EMPTY + s), 1);
      mbar_init(bar(S_FULL + s), 1);
    }
    mbar_init(bar(P_FULL), 256); mbar_init(bar(T_FULL), 1); mbar_init(bar(T_EMPTY), 1); mbar_init(bar(C_FULL), 1);
    for (int s = 0; s < 4; ++s) mbar_init(bar(META_FULL + s), 1);
    misc[1] = 0; misc[2] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) tmem_alloc(base + Smem::misc, 512);
  __syncthreads();
  {
    int boxes = 0;
    for (int t = tid; t < nroute; t += kThreads) {
      int start = 0, len = prm.N;
      if (prm.sparse) { const int g = ridx[t]; start = kvoff[g]; len = kvoff[g + 1] - start; }
      ranges[t] = make_int2(start, len);
      boxes += (len + kSub - 1) / kSub;
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

  if (warp == 8) {
    // =========================== TMA producer ===========================================
    if (lane == 0 && n_tiles > 0) {
      mbar_expect_tx(bar(Q_FULL), kTileBytes);
      tma_load_4d(base + Smem::q, &mapQ, bar(Q_FULL), 0, row0, prm.sparse ? bh : h, prm.sparse ? 0 : b);
      tma_load_4d(base + Smem::q + kHalfBytes, &mapQ, bar(Q_FULL), 64, row0, prm.sparse ? bh : h, prm.sparse ? 0 : b);
      const int c2 = prm.sparse ? bh : h, c3 = prm.sparse ? 0 : b;
      int ri = 0, off = 0;                       // walk state shared by the K and the V stream of a tile
      for (int i = 0; i < n_tiles; ++i) {
        const int s = i % kStages;
        const uint32_t ph = ((i / kStages) & 1) ^ 1;         // empty barriers: first pass completes immediately
        // box list of this tile
        int starts[kSubPerTile];
        uint32_t cnt_bits = 0;
        int nsub = 0, ri2 = ri, off2 = off;
#pragma unroll
        for (int j = 0; j < kSubPerTile; ++j) {
          starts[j] = 0;
          if (ri2 < nroute) {
            const int2 rg = ranges[ri2];
            starts[j] = rg.x + off2;
            const int cnt = min(kSub, rg.y - off2);
            cnt_bits |= (uint32_t)(cnt - 1) << (4 * j);
            nsub = j + 1;
            off2 += kSub;
            if (off2 >= rg.y) { ++ri2; off2 = 0; }
          }
        }
        ri = ri2; off = off2;
        if (!mbar_wait(bar(K_EMPTY + s), ph, abort_flag)) break;
        meta[i & 3] = make_uint2(cnt_bits, (uint32_t)nsub);
        mbar_arrive(bar(META_FULL + (i & 3)));
        mbar_expect_tx(bar(K_FULL + s), nsub * 2 * kSubBytes);
#pragma unroll
        for (int j = 0; j < kSubPerTile; ++j)
          if (j < nsub) {
            const uint32_t dst = base + Smem::k + s * kTileBytes + j * kSubBytes;
            tma_load_4d(dst, &mapK, bar(K_FULL + s), 0, starts[j], c2, c3);
            tma_load_4d(dst + kHalfBytes, &mapK, bar(K_FULL + s), 64, starts[j], c2, c3);
          }
        if (!mbar_wait(bar(V_EMPTY + s), ph, abort_flag)) break;
        mbar_expect_tx(bar(V_FULL + s), nsub * 2 * kSubBytes);
#pragma unroll
        for (int j = 0; j < kSubPerTile; ++j)
          if (j < nsub) {
            const uint32_t dst = base + Smem::v + s * kTileBytes + j * kSubBytes;
            tma_load_4d(dst, &mapV, bar(V_FULL + s), 0, starts[j], c2, c3);
            tma_load_4d(dst + kHalfBytes, &mapV, bar(V_FULL + s), 64, starts[j], c2, c3);
          }
      }
      if (prm.has_corr && !*abort_flag) {
        // the composed correction matrix (transposed, bf16) goes into K stage 0 once every QK^T is done
        const int uses0 = (n_tiles + kStages - 1) / kStages;       // completed phases of K_EMPTY[0]
        if (mbar_wait(bar(K_EMPTY + 0), (uint32_t)((uses0 - 1) & 1), abort_flag)) {
          mbar_expect_tx(bar(C_FULL), kTileBytes);
          tma_load_4d(base + Smem::k, &mapA, bar(C_FULL), 0, 0, bh, 0);
          tma_load_4d(base + Smem::k + kHalfBytes, &mapA, bar(C_FULL), 64, 0, bh, 0);
        }
      }
    }
  } else if (warp == 9) {
    // =========================== MMA issuer ==============================================
    if (lane == 0 && n_tiles > 0) {
      const uint32_t idesc_qk = idesc_bf16(0, 128), idesc_pv = idesc_bf16(1, 128);
      bool ok = mbar_wait(bar(Q_FULL), 0, abort_flag);
      auto issue_qk = [&](int i) -> bool {
        const int s = i % kStages;
        if (!mbar_wait(bar(K_FULL + s), (i / kStages) & 1, abort_flag)) return false;
        // S buffer i&1 was last read by softmax(i-2); the P_FULL wait of P V (i-2) below already covers that
        tc_fence_after();
        const uint32_t d = tmem + (uint32_t)(i & 1) * 128u;
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint32_t koff = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
          umma_bf16(d, smem_desc(base + Smem::q + koff, 16), smem_desc(base + Smem::k + s * kTileBytes + koff, 16), idesc_qk, kk > 0);
        }
        umma_commit(bar(K_EMPTY + s));
        umma_commit(bar(S_FULL + (i & 1)));
        return true;
      };
      if (ok) ok = issue_qk(0);
      for (int i = 0; i < n_tiles && ok; ++i) {
        if (i + 1 < n_tiles) { ok = issue_qk(i + 1); if (!ok) break; }
        const int s = i % kStages;
        const uint2 mt = meta[i & 3];
        if (!mbar_wait(bar(V_FULL + s), (i / kStages) & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(bar(P_FULL), i & 1, abort_flag)) { ok = false; break; }   // P(i) stored, O rescaled if needed
        tc_fence_after();
        const uint32_t d = tmem + 256u;
        const int nsub = (int)mt.y;
        for (int kk = 0; kk < nsub; ++kk) {
          const uint64_t a = smem_desc(base + Smem::p + (kk >> 2) * kHalfBytes + (kk & 3) * 32, 16);
          const uint64_t bdesc = smem_desc(base + Smem::v + s * kTileBytes + kk * kSubBytes, kHalfBytes);
          umma_bf16(d, a, bdesc, idesc_pv, (i > 0 || kk > 0) ? 1u : 0u);          // O accumulates over all tiles
        }
        umma_commit(bar(V_EMPTY + s));
        umma_commit(bar(T_FULL));
      }
      if (ok && prm.has_corr) {
        // correction product: bf16(O_sp) (in the P buffer) times A (in K stage 0) -> S buffer 0
        if (mbar_wait(bar(C_FULL), 0, abort_flag) && mbar_wait(bar(P_FULL), n_tiles & 1, abort_flag)) {
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < kD / 16; ++kk) {
            const uint32_t koff = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
            umma_bf16(tmem, smem_desc(base + Smem::p + koff, 16), smem_desc(base + Smem::k + koff, 16), idesc_qk, kk > 0);
          }
          umma_commit(bar(S_FULL + 0));
        }
      }
    }
  } else {
    // =========================== softmax (warps 0-7) =======================================
    // Two threads per query row (64 score columns each).  The output accumulator O stays in
    // TMEM for the whole key stream: P V products accumulate into it, and it is rescaled only
    // when the running row maximum has grown by more than 2^8 since the reference maximum
    // m_ref was fixed (the exponentials then stay below 2^8 and nothing overflows); the final
    // normalisation by the row sum removes the stale factor exactly.
    // Control flow stays uniform inside a warp (`ok` is voted) and the pair barriers are executed
    // by both warps of a row quad whatever happened, so a timed-out wait cannot strand a partner.
    const int wq = warp & 3, half = warp >> 2;
    const int row = wq * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
    const uint32_t FULL = 0xffffffffu;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    const float sc = prm.scale_log2;
    for (int i = 0; i < n_tiles; ++i) {
      ok = __all_sync(FULL, ok && mbar_wait(bar(S_FULL + (i & 1)), (i >> 1) & 1, abort_flag) &&
                                mbar_wait(bar(META_FULL + (i & 3)), (i >> 2) & 1, abort_flag));
      float s[64];
      float mx = -INFINITY;
      if (ok) {
        tc_fence_after();
        const uint2 mt = meta[i & 3];
        {
          float t[32];
          tmem_ld32(tmem + lane_addr + (uint32_t)(i & 1) * 128u + half * 64, t);
#pragma unroll
          for (int c = 0; c < 32; ++c) s[c] = t[c];
          tmem_ld32(tmem + lane_addr + (uint32_t)(i & 1) * 128u + half * 64 + 32, t);
#pragma unroll
          for (int c = 0; c < 32; ++c) s[32 + c] = t[c];
        }
        if (!(mt.x == 0xFFFFFFFFu && mt.y == 8u)) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int box = half * 4 + g;
            const int lim = box < (int)mt.y ? (int)((mt.x >> (4 * box)) & 15u) : -1;    // last valid column of the box
#pragma unroll
            for (int c = 0; c < 16; ++c) s[g * 16 + c] = (c <= lim) ? s[g * 16 + c] : -INFINITY;
          }
        }
#pragma unroll
        for (int c = 0; c < 64; ++c) mx = fmaxf(mx, s[c]);
      } else {
#pragma unroll
        for (int c = 0; c < 64; ++c) s[c] = 0.f;
      }
      float* xb = xchg + (i & 1) * 256;                                    // double buffered: one pair barrier per tile
      xb[half * 128 + row] = mx;
      asm volatile("bar.sync %0, 64;" ::"r"(1 + wq) : "memory");           // the two warps that share these rows
      mx = fmaxf(mx, xb[(half ^ 1) * 128 + row]);
      // reference maximum: moved only when the tile maximum exceeds it by more than 8 (log2 units)
      const bool move = (mx - m_ref) * sc > 8.f;                           // true on the first tile (m_ref = -inf)
      const float m_new = move ? mx : m_ref;
      const float corr = move ? ex2((m_ref - m_new) * sc) : 1.f;           // 0 on the first tile
      const float mneg = -m_new * sc;
      m_ref = m_new;
      float psum = 0.f;
#pragma unroll
      for (int c = 0; c < 64; ++c) { s[c] = ex2(fmaf(s[c], sc, mneg)); psum += s[c]; }
      l = l * corr + psum;
      // P buffer and O are free once the previous P V product has completed
      if (i >= 1) ok = __all_sync(FULL, ok && mbar_wait(bar(T_FULL), (i - 1) & 1, abort_flag));
      if (ok) {
        tc_fence_after();
        if (i >= 1 && __any_sync(FULL, move)) {                            // rescale this warp's O rows (rare)
#pragma unroll
          for (int hblk = 0; hblk < 2; ++hblk) {
            float t[32];
            tmem_ld32(tmem + lane_addr + 256u + half * 64 + hblk * 32, t);
#pragma unroll
            for (int c = 0; c < 32; ++c) t[c] *= corr;
            tmem_st32(tmem + lane_addr + 256u + half * 64 + hblk * 32, t);
          }
        }
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) store_p_chunk(base + Smem::p, row, half * 8 + ch, &s[ch * 8]);
        fence_async_smem();
        tc_fence_before();
        mbar_arrive(bar(P_FULL));
      }
    }
    float o[64];
#pragma unroll
    for (int c = 0; c < 64; ++c) o[c] = 0.f;
    if (n_tiles > 0) {
      ok = __all_sync(FULL, ok && mbar_wait(bar(T_FULL), (n_tiles - 1) & 1, abort_flag));
      if (ok) {
        tc_fence_after();
        float t[32];
        tmem_ld32(tmem + lane_addr + 256u + half * 64, t);
#pragma unroll
        for (int c = 0; c < 32; ++c) o[c] = t[c];
        tmem_ld32(tmem + lane_addr + 256u + half * 64 + 32, t);
#pragma unroll
        for (int c = 0; c < 32; ++c) o[32 + c] = t[c];
      }
    }
    // total row sum from both halves
    float* xe = xchg + (n_tiles & 1) * 256;
    xe[half * 128 + row] = l;
    asm volatile("bar.sync %0, 64;" ::"r"(1 + wq) : "memory");
    const float ltot = l + xe[(half ^ 1) * 128 + row];
    const float inv = ltot > 0.f ? 1.f / ltot : 0.f;
#pragma unroll
    for (int c = 0; c < 64; ++c) o[c] *= inv;
    float res[64];
#pragma unroll
    for (int c = 0; c < 64; ++c) res[c] = o[c];
    if (prm.has_corr && n_tiles > 0) {
      if (ok) {
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) store_p_chunk(base + Smem::p, row, half * 8 + ch, &o[ch * 8]);
        fence_async_smem();
        tc_fence_before();
        mbar_arrive(bar(P_FULL));
      }
      // S buffer 0 completes once more: its phase index = number of earlier completions
      const int prev = (n_tiles + 1) / 2;
      ok = __all_sync(FULL, ok && mbar_wait(bar(S_FULL + 0), prev & 1, abort_flag));
      if (ok) {
        tc_fence_after();
        const float* cv = prm.c + (i64)bh * kD + half * 64;
        float t[32];
        tmem_ld32(tmem + lane_addr + half * 64, t);
#pragma unroll
        for (int c = 0; c < 32; ++c) res[c] = o[c] + t[c] + cv[c];
        tmem_ld32(tmem + lane_addr + half * 64 + 32, t);
#pragma unroll
        for (int c = 0; c < 32; ++c) res[32 + c] = o[32 + c] + t[c] + cv[32 + c];
      }
    } else if (prm.has_corr) {
      const float* cv = prm.c + (i64)bh * kD + half * 64;
#pragma unroll
      for (int c = 0; c < 64; ++c) res[c] = cv[c];
    }
    if (ok && row < nrows) {
      const int dst = prm.sparse ? prm.q_perm[(i64)bh * prm.N + row0 + row] : row0 + row;
      __nv_bfloat16* op = prm.O + b * prm.os[0] + h * prm.os[1] + (i64)dst * prm.os[2] + half * 64;
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        float v8[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v8[k] = res[ch * 8 + k];
        store8(op + ch * 8, v8);
      }
      if (prm.O_sparse) {
        float* sp = prm.O_sparse + ((i64)bh * prm.N + dst) * kD + half * 64;
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
  // ---- teardown ----------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the shared memory is released
    for (int k = 0; k < 64; ++k) __nanosleep(1000);
    if (tid == 0) set_error(prm.err, SPARSEPR_ERR_TIMEOUT);
    __syncthreads();
  }
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// A [BH][128][128] float32 (row k, column n) -> At [BH][n][k] bf16
__global__ void k_transpose_correction(const float* __restrict__ A, __nv_bfloat16* __restrict__ At) {
  __shared__ float tile[32][33];
  const int bh = blockIdx.z;
  const float* a = A + (i64)bh * kD * kD;
  __nv_bfloat16* t = At + (i64)bh * kD * kD;
  const int k0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  for (int r = threadIdx.y; r < 32; r += 8) tile[r][threadIdx.x] = a[(k0 + r) * kD + n0 + threadIdx.x];
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += 8) t[(n0 + r) * kD + k0 + threadIdx.x] = __float2bfloat16_rn(tile[threadIdx.x][r]);
}

// ---- tensor maps (driver entry point fetched through the runtime; libcuda is not linked) -------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
std::once_flag g_encode_once;

EncodeTiledFn encode_fn() {
  std::call_once(g_encode_once, [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  });
  return g_encode;
}

bool tma_available() { return encode_fn() != nullptr; }

bool make_map(CUtensorMap* m, const void* ptr, int cols, int rows, int H, int B, i64 sb, i64 sh, i64 sn, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const i64 hstride = H > 1 ? sh : (i64)rows * sn;
  const i64 bstride = B > 1 ? sb : (i64)H * hstride;
  const cuuint64_t dims[4] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)H, (cuuint64_t)B};
  const cuuint64_t strides[3] = {(cuuint64_t)sn * 2, (cuuint64_t)hstride * 2, (cuuint64_t)bstride * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc

cudaError_t init_attention_tc() {
  return cudaFuncSetAttribute(tc::k_attention_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes);
}

bool attention_tc_supported(const AttnArgs& a) {
  return a.dtype == SPARSEPR_BF16 && a.d == 128 && tc::tma_available();
}

// `At` is scratch for the transposed bf16 correction matrix [BH][128][128] (only with a.A != null)
bool launch_attention_tc(const AttnArgs& a, __nv_bfloat16* At, cudaStream_t st) {
  using namespace tc;
  CUtensorMap mq, mk, mv, ma;
  const bool sparse = a.route_ptr != nullptr;
  const int B = a.BH / a.H;
  bool ok;
  if (sparse) {
    ok = make_map(&mq, a.Q, kD, a.N, a.BH, 1, 0, (i64)a.N * kD, kD, kTile) && make_map(&mk, a.K, kD, a.N, a.BH, 1, 0, (i64)a.N * kD, kD, kSub) &&
         make_map(&mv, a.V, kD, a.N, a.BH, 1, 0, (i64)a.N * kD, kD, kSub);
  } else {
    ok = make_map(&mq, a.Q, kD, a.N, a.H, B, a.qs[0], a.qs[1], a.qs[2], kTile) && make_map(&mk, a.K, kD, a.N, a.H, B, a.ks[0], a.ks[1], a.ks[2], kSub) &&
         make_map(&mv, a.V, kD, a.N, a.H, B, a.vs[0], a.vs[1], a.vs[2], kSub);
  }
  if (!ok) return false;
  if (a.A) {
    k_transpose_correction<<<dim3(kD / 32, kD / 32, a.BH), dim3(32, 8), 0, st>>>(a.A, At);
    if (!make_map(&ma, At, kD, kD, a.BH, 1, 0, (i64)kD * kD, kD, kTile)) return false;
  } else ma = mq;
  Params p{};
  p.BH = a.BH; p.H = a.H; p.N = a.N; p.Cq = a.Cq; p.Ck = a.Ck; p.sparse = sparse;
  p.scale_log2 = a.scale * 1.4426950408889634f;
  p.q_off = a.q_off; p.kv_off = a.kv_off; p.route_ptr = a.route_ptr; p.route_idx = a.route_idx; p.q_perm = a.q_perm;
  p.tile_off = a.tile_off; p.c = a.c; p.has_corr = a.A != nullptr;
  p.O = (__nv_bfloat16*)a.O; for (int i = 0; i < 3; ++i) p.os[i] = a.os[i];
  p.O_sparse = a.O_sparse; p.err = a.err;
  const int tiles = (a.N + kTile - 1) / kTile + (sparse ? a.Cq : 0);
  k_attention_tc<<<dim3(tiles, a.BH), kThreads, kSmemBytes, st>>>(mq, mk, mv, ma, p);
  return true;
}

}  // namespace spr
