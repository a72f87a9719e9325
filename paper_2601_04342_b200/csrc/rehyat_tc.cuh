// Tensor-core (tcgen05 / TMEM / TMA) path of the operator for bf16, head_dim 128: the softmax-window kernel and
// the host-side launchers of all three tensor-core kernels.
//
// window_tc: softmax window of Eq. 6 and 8 plus the joint normalisation of Eq. 5.
//   Persistent: one CTA per SM walks work items (batch*head, chunk, pair of 128-row query tiles); barriers, TMEM
//   and the K/V rings live across items.  An item walks the chunk's key window in tiles of 128 keys.
//   Roles (384 threads):
//     warp 0        TMA producer: Q per item, K and V tiles through two-stage rings
//     warp 1        UMMA issuer: S_i = Q_i K^T into TMEM, O_i += P_i V with P_i read from TMEM (in two halves)
//     warps 4-7     softmax and epilogue of query tile 0 (one thread per row), warps 8-11 of query tile 1
//   TMEM (512 columns): S_0 [0,128) S_1 [128,256) O_0 [256,384) O_1 [384,512); P_i (bf16) overwrites
//   the first 64 columns of S_i.  While one tile's softmax runs on the ALUs the tensor core works on
//   the other tile.  The running maximum is applied lazily: O and l are rescaled only when the row
//   maximum grew by more than 2^8 since the last rescale; the true maximum is tracked separately and
//   applied once after the last key tile, so that O and l end up relative to c_i = final row maximum
//   before the un-rescaled linear terms are added (Eq. 5-9).
#pragma once

#include <cuda.h>

#include "../../include/rehyat.h"
#include "rehyat_common.cuh"
#include "rehyat_ptx.cuh"
#include "rehyat_phi_tc.cuh"
#include "rehyat_readout_tc.cuh"

namespace rehyat {

constexpr int TC_BM = 128;            // rows per query tile
constexpr int TC_QT = 2;              // query tiles per CTA
constexpr int TC_BN = 128;            // keys per tile
constexpr int TC_STAGES = 2;          // K ring and V ring depth
constexpr int TC_THREADS = 384;
constexpr int TC_REGS_SOFTMAX = 200;   // registers per thread of the softmax warps (setmaxnreg)
constexpr int TC_REGS_OTHER = 96;       // ... of the producer / issuer warpgroup
// Sizes that follow from the head dimension D (128 or 64).  A Q, K or V tile of 128 rows is D/64 swizzled
// [128 x 64] sub-tiles of 16 KB.  TMEM keeps the map of D = 128 for both: S slots at columns 0 and 128, O slots at
// 256 and 384 (D = 64 uses the first 64 columns of each O slot).
template <int D>
struct WinShape {
  static_assert(D == 64 || D == 128, "head_dim of the tensor-core window kernels");
  static constexpr int SUBS = D / 64;
  static constexpr int SUB_BYTES = TC_BN * 64 * 2;
  static constexpr int TILE_BYTES = SUBS * SUB_BYTES;
  static constexpr int SMEM = (TC_QT + 2 * TC_STAGES) * TILE_BYTES + 1024 /*barriers*/ + 1024 /*align*/;      // window_tc
  static constexpr int SMEM1 = (1 + 2 * TC_STAGES) * TILE_BYTES + 8192 /*barriers, merge buffer*/ + 1024;   // window_tc1
};

enum TcErr : int { TC_ERR_LOAD = 1, TC_ERR_MMA = 2, TC_ERR_SOFTMAX = 4 };
// One 32-byte store (a whole sector) of sixteen bf16; the address must be 32-byte aligned.
__device__ __forceinline__ void st_global_32B(void* p, uint4 a, uint4 b) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}
// Suspend-time hints (ns) of the waits of the TMA producer, of the MMA issuer and of the softmax warps.  The first
// two roles wait most of the time; without a hint their polling takes issue slots from the softmax warps that share
// their schedulers, whose tiles then end 140 - 210 cycles after those of the other two schedulers (measured with
// clock64 stamps), and the hand-over waits for the slowest warp.  With the hints the window kernel is 1.5 % faster;
// longer hints (10, 100 us) and a hint on the softmax warps' own waits change nothing more.
constexpr uint32_t TC_HINT_P = 1000, TC_HINT_I = 1000, TC_HINT_S = 0;

struct WinBars {   // offsets (bytes) inside the barrier block
  uint64_t q_full, q_empty;
  uint64_t k_full[TC_STAGES], k_empty[TC_STAGES], v_full[TC_STAGES], v_empty[TC_STAGES];
  uint64_t s_ready[TC_QT], p_half[TC_QT][2], pv_done[TC_QT], o_free[TC_QT];
  uint64_t drained;
  uint32_t tmem_base;
  ptx::WaitCtx wctx;
};

// One work item of window_tc: two query tiles of one (chunk, batch*head).
struct WinItem {
  int bh, b_idx, h_idx, ci;
  int q0, q1, lo, hi;      // chunk queries [q0, q1), softmax window [lo, hi)
  int row_base, ntiles, n_kv;
  bool linear;             // the chunk has a non-empty linear set
};
// Items are numbered (batch*head, chunk, tile pair), tile pair fastest, so that the CTAs running at one
// time share few K/V windows in L2.  Returns false for pairs beyond the end of a short last chunk.
__device__ __forceinline__ bool win_item(const Geo& g, int item, int pairs, WinItem& w) {
  const int pair = item % pairs, rest = item / pairs, ci = rest % g.G;
  w.bh = rest / g.G;
  w.ci = ci;
  const int t = g.t0 + ci;
  w.q0 = geo_q0(g, t); w.q1 = geo_q1(g, t); w.lo = geo_lo(g, t); w.hi = w.q1;
  w.linear = geo_linear(g, t);
  w.row_base = w.q0 + pair * (TC_QT * TC_BM);
  if (w.row_base >= w.q1) return false;
  w.ntiles = (w.row_base + TC_BM < w.q1) ? 2 : 1;                  // query tiles with at least one valid row
  w.n_kv = (w.hi - w.lo + TC_BN - 1) / TC_BN;
  w.b_idx = w.bh / g.n_heads; w.h_idx = w.bh % g.n_heads;
  return true;
}

// The MMAs of both window kernels, issued by one thread.  TMEM: S slots at columns 0 and 128, O slots at 256 and
// 384.  Descriptors differ only in the start-address field (low word): built once, offsets added per MMA.
template <int D>
struct WinMma {
  using SH = WinShape<D>;
  static constexpr uint32_t idesc_qk = ptx::idesc_bf16(TC_BM, TC_BN, 0, 0);   // A = Q (K-major), B = K (K-major)
  static constexpr uint32_t idesc_pv = ptx::idesc_bf16(TC_BM, D, 0, 1);       // A = P (TMEM),    B = V (MN-major)
  uint32_t tmem, q_lo, q_hi, k_lo, k_hi, v_lo, v_hi;
  __device__ __forceinline__ WinMma(uint32_t tmem_base, uint32_t sQ, uint32_t sK, uint32_t sV) : tmem(tmem_base) {
    ptx::upk2u(ptx::smem_desc_sw128(sQ, 16, 1024), q_lo, q_hi);
    ptx::upk2u(ptx::smem_desc_sw128(sK, 16, 1024), k_lo, k_hi);
    ptx::upk2u(ptx::smem_desc_sw128(sV, SH::SUB_BYTES, 1024), v_lo, v_hi);
  }
  // S[slot] = Q[q_tile] K[stage]^T
  __device__ __forceinline__ void qk(int slot, int q_tile, int stage) const {
    const uint32_t a0 = q_lo + q_tile * (SH::TILE_BYTES >> 4), b0 = k_lo + stage * (SH::TILE_BYTES >> 4);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      const uint32_t off = ((kk >> 2) * SH::SUB_BYTES + (kk & 3) * 32) >> 4;
      ptx::umma_ss(tmem + slot * TC_BN, ptx::pk2u(a0 + off, q_hi), ptx::pk2u(b0 + off, k_hi), idesc_qk, kk > 0);
    }
  }
  // O[slot] (+)= P[slot][:, keys 64*half .. +64) V[stage][those keys, :]
  __device__ __forceinline__ void pv(int slot, int stage, int half, bool acc) const {
    const uint32_t b0 = v_lo + stage * (SH::TILE_BYTES >> 4);
#pragma unroll
    for (int kk = half * 4; kk < half * 4 + 4; ++kk)
      ptx::umma_ts(tmem + 256 + slot * 128, tmem + slot * TC_BN + kk * 8, ptx::pk2u(b0 + kk * (16 * 128 >> 4), v_hi), idesc_pv,
                   (acc || kk > half * 4) ? 1u : 0u);
  }
};

// Running softmax state of one query row over the key tiles of a TMEM slot: the true maximum so far, the
// reference the exponentials are taken against (it follows the maximum lazily), four partial row sums.
struct SoftmaxRow {
  float m_true = -INFINITY, m_used = -INFINITY;
  uint64_t l2a = 0ull, l2b = 0ull;
  __device__ __forceinline__ float sum() const {
    float a0, a1, b0, b1;
    ptx::upk2(l2a, a0, a1);
    ptx::upk2(l2b, b0, b1);
    return (a0 + a1) + (b0 + b1);
  }
};

// One 128-key tile of one query row (this thread's TMEM lane), shared by both window kernels (Eq. 6, 8): S is
// read from the 128 columns at tS, keys beyond n_valid are masked, the reference maximum is moved (and O at tO and
// the row sums rescaled) only when the maximum grew by more than 2^8, P = 2^((s - m_used) c) goes back to the
// first 64 columns of S as bf16 in two halves, each announced on its barrier.  `has_previous`: the slot already
// holds a P V of this item (O may then need the rescale); `wait_previous_pv()` waits for it and returns false if
// the wait was given up, which is also what this function then returns.
// EMU: of every four pairs of exponentials, how many are evaluated on the FMA pipe.
template <int EMU, int D, typename WaitPv>
__device__ __forceinline__ bool softmax_key_tile(uint32_t tS, uint32_t tO, int n_valid, float c, bool has_previous,
                                                 SoftmaxRow& st, uint32_t bar_half0, uint32_t bar_half1, int lane,
                                                 WaitPv&& wait_previous_pv) {
  using namespace ptx;
  uint32_t sr[4][32];
#pragma unroll
  for (int cc = 0; cc < 4; ++cc) tmem_ld32(tS + cc * 32, sr[cc]);
  tmem_wait_ld();
  if (n_valid < TC_BN) {
#pragma unroll
    for (int cc = 0; cc < 4; ++cc)
#pragma unroll
      for (int e = 0; e < 32; ++e)
        if (cc * 32 + e >= n_valid) sr[cc][e] = 0xff800000u;   // -inf
  }
  // row maximum: four independent chains of three-input max
  float mx[8] = {st.m_true, st.m_true, st.m_true, st.m_true, st.m_true, st.m_true, st.m_true, st.m_true};
#pragma unroll
  for (int cc = 0; cc < 4; ++cc)
#pragma unroll
    for (int e = 0; e < 32; e += 2)
      mx[cc * 2 + ((e >> 1) & 1)] = fmax3(mx[cc * 2 + ((e >> 1) & 1)], __uint_as_float(sr[cc][e]), __uint_as_float(sr[cc][e + 1]));
  st.m_true = fmaxf(fmax3(mx[0], mx[1], mx[2]), fmax3(fmaxf(mx[3], mx[4]), fmaxf(mx[5], mx[6]), mx[7]));
  const bool need = (st.m_true - st.m_used) * c > 8.f;               // true on the first tile (m_used = -inf)
  if (__any_sync(0xffffffffu, need)) {
    const float m_new = need ? st.m_true : st.m_used;
    if (has_previous) {
      // S of this tile follows the completion of the slot's previous P V, so O may be touched
      if (!wait_previous_pv()) return false;
      tc_fence_after();
      const float f = ex2((st.m_used - m_new) * c);                  // 1 for lanes that keep their reference
      const uint64_t f2 = pk2(f, f);
      st.l2a = mul2(st.l2a, f2);
      st.l2b = mul2(st.l2b, f2);
#pragma unroll 1
      for (int cc = 0; cc < D / 8; ++cc) {                           // rare: small pieces keep the register peak low
        uint32_t o[8];
        tmem_ld8(tO + cc * 8, o);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * f);
        tmem_st8(tO + cc * 8, o);
      }
    }
    st.m_used = m_new;
  }
  const float mc = -st.m_used * c;
  const uint64_t c2 = pk2(c, c), mc2 = pk2(mc, mc);
#pragma unroll
  for (int cc = 0; cc < 4; ++cc) {
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
      float t0, t1, p0, p1;
      upk2(fma2(pk2u(sr[cc][e], sr[cc][e + 1]), c2, mc2), t0, t1);
      if (((e >> 1) & 3) < EMU) {                                    // EMU of every 4 pairs on the FMA pipe
        ex2_poly2(t0, t1, p0, p1);
      } else {
        p0 = ex2(t0);
        p1 = ex2(t1);
      }
      if ((e >> 1) & 1) st.l2b = add2(st.l2b, pk2(p0, p1)); else st.l2a = add2(st.l2a, pk2(p0, p1));
      sr[cc >> 1][(cc & 1) * 16 + (e >> 1)] = pack_bf16(p0, p1);
    }
    if (cc & 1) {
      tmem_st32(tS + (cc >> 1) * 32, sr[cc >> 1]);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive_warp((cc >> 1) ? bar_half1 : bar_half0, lane);     // P of 64 keys is in place
    }
  }
  return true;
}

// Persistent: gridDim.x CTAs (one per SM) walk the items blockIdx.x, blockIdx.x + gridDim.x, ...  Barriers,
// TMEM and the K/V rings live across items; every role keeps running counts of the phases it has used.
// EMU: of every four pairs of exponentials, how many are evaluated on the FMA pipe.  D: head_dim.
template <int EMU, int D>
__global__ void __launch_bounds__(TC_THREADS, 1)
window_tc(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
          const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ out, Geo g,
          const float* __restrict__ rd, int rd_rows, float scale, int c_mode, ptx::WaitArgs wa,
          int n_items, int pairs, float* __restrict__ share) {
  using namespace ptx;
  using SH = WinShape<D>;
  constexpr int TC_TILE_BYTES = SH::TILE_BYTES, TC_SUB_BYTES = SH::SUB_BYTES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sQ = smem_base;                                   // TC_QT tiles
  const uint32_t sK = sQ + TC_QT * TC_TILE_BYTES;                  // TC_STAGES tiles
  const uint32_t sV = sK + TC_STAGES * TC_TILE_BYTES;              // TC_STAGES tiles
  WinBars* bars = reinterpret_cast<WinBars*>(smem + (TC_QT + 2 * TC_STAGES) * TC_TILE_BYTES);
  // one tile = SH::SUBS boxes of 64 columns
  auto load_tile = [&](uint32_t dst, const CUtensorMap* tm, uint32_t bar, int row, int h, int b) {
#pragma unroll
    for (int sb = 0; sb < SH::SUBS; ++sb) tma_load_4d(dst + sb * TC_SUB_BYTES, tm, bar, sb * 64, row, h, b);
  };
  const uint32_t wc = smem_u32(&bars->wctx);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars->q_full), 1); mbar_init(smem_u32(&bars->q_empty), 1);
    for (int s = 0; s < TC_STAGES; ++s) {
      mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 1);
      mbar_init(smem_u32(&bars->v_full[s]), 1); mbar_init(smem_u32(&bars->v_empty[s]), 1);
    }
    for (int i = 0; i < TC_QT; ++i) {
      mbar_init(smem_u32(&bars->s_ready[i]), 1);
      mbar_init(smem_u32(&bars->p_half[i][0]), TC_BM / 32);
      mbar_init(smem_u32(&bars->p_half[i][1]), TC_BM / 32);
      mbar_init(smem_u32(&bars->pv_done[i]), 1);
      mbar_init(smem_u32(&bars->o_free[i]), TC_BM / 32);
    }
    mbar_init(smem_u32(&bars->drained), 1);
    wait_ctx_init(&bars->wctx, wa);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp < 4) setmaxnreg_dec<TC_REGS_OTHER>();
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one() && !wa.withhold_loads) {
      prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
      uint32_t n_k = 0, n_v = 0, n_q = 0;                          // K tiles, V tiles and Q loads issued so far
      bool alive = true;
      for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
        WinItem w;
        if (!win_item(g, item, pairs, w)) continue;
        // Q of the previous item has been read by its last Q K^T
        if (n_q > 0) alive = mbar_wait(smem_u32(&bars->q_empty), (n_q - 1) & 1, wc, TC_ERR_LOAD, TC_HINT_P);
        if (!alive) break;
        const uint32_t qf = smem_u32(&bars->q_full);
        mbar_expect_tx(qf, w.ntiles * TC_TILE_BYTES);
        for (int i = 0; i < w.ntiles; ++i) load_tile(sQ + i * TC_TILE_BYTES, &tm_q, qf, w.row_base - g.q_off + i * TC_BM, w.h_idx, w.b_idx);
        ++n_q;
        for (int j = 0; j < w.n_kv && alive; ++j) {
          const int s = n_k % TC_STAGES;
          const uint32_t ph = (n_k / TC_STAGES) & 1;
          const int key0 = w.lo + j * TC_BN;
          alive = mbar_wait(smem_u32(&bars->k_empty[s]), ph ^ 1, wc, TC_ERR_LOAD, TC_HINT_P);
          if (!alive) break;
          const uint32_t kf = smem_u32(&bars->k_full[s]);
          mbar_expect_tx(kf, TC_TILE_BYTES);
          load_tile(sK + s * TC_TILE_BYTES, &tm_k, kf, key0, w.h_idx, w.b_idx);
          ++n_k;
          alive = mbar_wait(smem_u32(&bars->v_empty[s]), ph ^ 1, wc, TC_ERR_LOAD, TC_HINT_P);
          if (!alive) break;
          const uint32_t vf = smem_u32(&bars->v_full[s]);
          mbar_expect_tx(vf, TC_TILE_BYTES);
          load_tile(sV + s * TC_TILE_BYTES, &tm_v, vf, key0, w.h_idx, w.b_idx);
          ++n_v;
        }
      }
      if (!alive) {
        // Given up: the loads already issued still write shared memory.  Wait for the last one into every
        // buffer (the full barriers complete by byte count, whatever the consumers do) before the CTA exits.
        if (n_q > 0) mbar_wait_drain(smem_u32(&bars->q_full), (n_q - 1) & 1, wc);
        for (uint32_t back = 0; back < (uint32_t)TC_STAGES; ++back) {
          if (n_k > back) mbar_wait_drain(smem_u32(&bars->k_full[(n_k - 1 - back) % TC_STAGES]), ((n_k - 1 - back) / TC_STAGES) & 1, wc);
          if (n_v > back) mbar_wait_drain(smem_u32(&bars->v_full[(n_v - 1 - back) % TC_STAGES]), ((n_v - 1 - back) / TC_STAGES) & 1, wc);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (elect_one()) {
      const WinMma<D> mma(tmem, sQ, sK, sV);
      auto issue_qk = [&](int i, int s) { mma.qk(i, i, s); };         // query tile i into its own slot
      auto issue_pv = [&](int i, int s, int half, bool acc) { mma.pv(i, s, half, acc); };
      uint32_t kv_it = 0, n_done = 0;                                // K/V tiles consumed, items done
      uint32_t n_p[TC_QT] = {0, 0}, n_o[TC_QT] = {0, 0};             // P hand-overs and items per query tile
      bool alive = true;                                             // false once a wait has been given up: issue nothing more
      auto wait = [&](uint64_t* bar, uint32_t parity) {
        alive = alive && mbar_wait(smem_u32(bar), parity, wc, TC_ERR_MMA, TC_HINT_I);
        return alive;
      };
      for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
        WinItem w;
        if (!win_item(g, item, pairs, w)) continue;
        if (!wait(&bars->q_full, n_done & 1)) break;
        if (!wait(&bars->k_full[kv_it % TC_STAGES], (kv_it / TC_STAGES) & 1)) break;
        tc_fence_after();
        for (int i = 0; i < w.ntiles; ++i) {
          issue_qk(i, kv_it % TC_STAGES);
          umma_commit(smem_u32(&bars->s_ready[i]));
        }
        umma_commit(smem_u32(&bars->k_empty[kv_it % TC_STAGES]));
        if (w.n_kv == 1) umma_commit(smem_u32(&bars->q_empty));
        for (int j = 0; j < w.n_kv && alive; ++j, ++kv_it) {
          const int s = kv_it % TC_STAGES;
          if (!wait(&bars->v_full[s], (kv_it / TC_STAGES) & 1)) break;
          for (int i = 0; i < w.ntiles; ++i) {
            // the first P V of an item overwrites O: the epilogue of the tile's previous item must have read it
            if (j == 0 && n_o[i] > 0 && !wait(&bars->o_free[i], (n_o[i] - 1) & 1)) break;
            if (!wait(&bars->p_half[i][0], n_p[i] & 1)) break;
            tc_fence_after();
            issue_pv(i, s, 0, j > 0);
            if (!wait(&bars->p_half[i][1], n_p[i] & 1)) break;
            tc_fence_after();
            issue_pv(i, s, 1, true);
            ++n_p[i];
            umma_commit(smem_u32(&bars->pv_done[i]));
            if (i == w.ntiles - 1) umma_commit(smem_u32(&bars->v_empty[s]));
            if (j + 1 < w.n_kv) {
              const int s1 = (kv_it + 1) % TC_STAGES;
              if (i == 0) {
                if (!wait(&bars->k_full[s1], ((kv_it + 1) / TC_STAGES) & 1)) break;
                tc_fence_after();
              }
              issue_qk(i, s1);
              umma_commit(smem_u32(&bars->s_ready[i]));
              if (i == w.ntiles - 1) {
                umma_commit(smem_u32(&bars->k_empty[s1]));
                if (j + 2 == w.n_kv) umma_commit(smem_u32(&bars->q_empty));   // the item's last Q K^T
              }
            }
          }
        }
        ++n_done;
        for (int i = 0; i < w.ntiles; ++i) ++n_o[i];
      }
      // Everything this thread has issued is complete once `drained` flips.  This wait is not cut short by the
      // abort flag: TMEM must not be freed, nor the CTA exit, with a tcgen05.mma still running.
      umma_commit(smem_u32(&bars->drained));
      mbar_wait_drain(smem_u32(&bars->drained), 0, wc);
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax + epilogue
    setmaxnreg_inc<TC_REGS_SOFTMAX>();
    const int i = (warp - 4) >> 2;                                   // query tile of this warpgroup
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_off + i * TC_BN, tO = tmem + lane_off + 256 + i * 128;
    const float c = scale * 1.4426950408889634f;                     // logits -> log2 domain
    const bool out_32B = ((reinterpret_cast<uintptr_t>(out) | (uintptr_t)(g.ostride_b * 2) | (uintptr_t)(g.ostride_h * 2) |
                           (uintptr_t)(g.ostride_n * 2)) & 31u) == 0;   // every row of out starts on a 32-byte boundary
    uint32_t n_s = 0;                                                // key tiles this query tile has been through
    // A wait that was given up ends the role.  The warp decides together (tcgen05.ld / st and the votes below
    // need all 32 lanes), so every wait is followed by a vote.
    bool alive = true;
    auto wait = [&](uint64_t* bar, uint32_t parity) {
      alive = __all_sync(0xffffffffu, mbar_wait(smem_u32(bar), parity, wc, TC_ERR_SOFTMAX, TC_HINT_S));
      return alive;
    };
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      WinItem w;
      if (!win_item(g, item, pairs, w) || i >= w.ntiles) continue;
      const int n_kv = w.n_kv, lo = w.lo, hi = w.hi;
      SoftmaxRow st;
      for (int j = 0; j < n_kv; ++j) {
        if (!wait(&bars->s_ready[i], (n_s + j) & 1)) break;
        tc_fence_after();
        if (!softmax_key_tile<EMU, D>(tS, tO, hi - (lo + j * TC_BN), c, j > 0, st, smem_u32(&bars->p_half[i][0]),
                                   smem_u32(&bars->p_half[i][1]), lane,
                                   [&]() { return wait(&bars->pv_done[i], (n_s + j - 1) & 1); }))
          break;
      }
      if (!alive) break;
      const float m_true = st.m_true, m_used = st.m_used, l = st.sum();

      // Eq. 5: bring O and l to the final row maximum, add the linear read-out, divide, store.
      const int row = w.row_base + i * TC_BM + (warp & 3) * 32 + lane;
      const bool valid = row < w.q1;
      // the whole read-out row is requested before the wait for the last P V, which hides its latency
      uint4 rdv[D / 8];                                              // fp16 pairs of aL / nL
      float nL = 0.f;
      if (w.linear) {
        const int ric = (valid ? row : w.q0) - w.q0, ci = w.ci;      // row inside the chunk: consecutive threads, consecutive pieces
        const uint4* rdh = reinterpret_cast<const uint4*>(rd);
#pragma unroll
        for (int u = 0; u < D / 8; ++u) rdv[u] = __ldg(rdh + rdh_index(g, rd_rows, D, w.bh, ci, ric, u));
        nL = __ldg(reinterpret_cast<const float*>(rdh + rdh_index(g, rd_rows, D, w.bh, ci, ric, rdh_pieces(D) - 1)));
      } else {
#pragma unroll
        for (int u = 0; u < D / 8; ++u) rdv[u] = make_uint4(0u, 0u, 0u, 0u);
      }
      const float fin = ex2((m_used - m_true) * c);
      float ws = fin, lam = 0.f;
      if (w.linear) {
        lam = 1.f;
        if (c_mode == C_ZERO) {
          const float mm = m_true * scale, r = fmaxf(mm, 0.f);
          ws = fin * __expf(mm - r);
          lam = __expf(-r);
        }
      }
      __nv_bfloat16* orow = out + out_row_offset(g, w.bh, row);
      if (!wait(&bars->pv_done[i], (n_s + n_kv - 1) & 1)) break;
      tc_fence_after();
      n_s += n_kv;
      const float inv = 1.f / (l * ws + lam * nL);
      const float wsi = ws * inv, lami = lam * inv * nL;               // the read-out comes as the ratio aL / nL
      if (share != nullptr && valid) share[(size_t)w.bh * g.N + row] = lami;       // part of the normaliser that is linear
#pragma unroll
      for (int hh = 0; hh < D / 32; ++hh) {                          // 32 columns of O at a time
        uint32_t o[32];
        tmem_ld32(tO + hh * 32, o);
        tmem_wait_ld();
        if (hh == D / 32 - 1) {                                      // O has been read: TMEM is free for the next item
          tc_fence_before();
          mbar_arrive_warp(smem_u32(&bars->o_free[i]), lane);
        }
        if (valid) {
          uint4 v4[4];
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            const uint4 x = rdv[hh * 4 + (e >> 3)];                  // eight columns of aL / nL as fp16 pairs
            auto fin = [&](int q, uint32_t pair) {
              const float2 rr = unpack_f16(pair);
              return pack_bf16(__uint_as_float(o[q]) * wsi + lami * rr.x, __uint_as_float(o[q + 1]) * wsi + lami * rr.y);
            };
            v4[e >> 3].x = fin(e + 0, x.x);
            v4[e >> 3].y = fin(e + 2, x.y);
            v4[e >> 3].z = fin(e + 4, x.z);
            v4[e >> 3].w = fin(e + 6, x.w);
          }
          // a thread writes its own row: whole 32-byte sectors where the output allows it (every lane of a store
          // touches another row, so nothing merges on the way)
          if (out_32B) {
            st_global_32B(orow + hh * 32, v4[0], v4[1]);
            st_global_32B(orow + hh * 32 + 16, v4[2], v4[3]);
          } else {
#pragma unroll
            for (int u = 0; u < 4; ++u) *reinterpret_cast<uint4*>(orow + hh * 32 + u * 8) = v4[u];
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------

struct TcWorkspace {
  void* encode_fn = nullptr;            // cuTensorMapEncodeTiled, resolved through the runtime
  __nv_bfloat16* state_bf16 = nullptr;  // [Gmax][BHmax][256][128]: bf16 copy of s_t for the read-out GEMM
  bool phi_ok = false;                  // the linear branch runs on the tensor-core kernels too
  int n_sm = 148;                       // SMs of the device
  int exp_poly = 1;                     // of every 4 pairs of exponentials, how many the FMA pipe evaluates
  int head_dim = 128;                   // 128 or 64
  int item_tiles = 0;                   // query tiles per window item: 1, 2, or 0 = chosen per launch
  int last_item_tiles = 0;              // what the last window launch used
};

inline bool tc_shape_supported(bool bf16, int d, int, int, int, int, int) { return bf16 && (d == 128 || d == 64); }
// The phi kernels: head_dim 64 or 128, widths that are multiples of 32 between 64 (32 for D') and 256.
// Up to PH_MAX_MID hidden layers between the first and the last.
inline bool tc_phi_supported(int d, int Dh, int Dp, int P, int n_mid) {
  return (d == 64 || d == 128) && Dh >= 64 && Dh <= PH_DH && Dh % 32 == 0 && Dp >= 32 && Dp <= PH_DP && Dp % 32 == 0 &&
         P >= 1 && Dp % P == 0 && n_mid >= 0 && n_mid <= PH_MAX_MID;
}
// Which instantiation serves a map: the fixed-shape kernels for the two-layer map of 128 / 256 / 256, the ones
// that read their extents otherwise; the ReLU fast path needs polynomial parts that end on 32-column blocks.
struct PhiKernelChoice { bool gen, relu; int pc; };
inline PhiKernelChoice tc_phi_choice(int d, int Dh, int Dp, int P, int n_mid, int act_hidden, int act_out) {
  PhiKernelChoice c;
  c.gen = !(d == PH_D && Dh == PH_DH && Dp == PH_DP && n_mid == 0);
  c.relu = act_hidden == ACT_RELU && act_out == ACT_RELU && (Dp / P) % 32 == 0;
  c.pc = (!c.gen && c.relu && P == 2) ? 2 : 0;
  return c;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline bool tc_workspace_create(TcWorkspace* w, int bh_max, int Gmax, int d, int Dp, size_t* extra) {
  *extra = 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn)
    return false;
  w->encode_fn = fn;
  if (w->phi_ok) {
    const size_t bytes = (size_t)Gmax * bh_max * Dp * d * sizeof(__nv_bfloat16);
    if (cudaMalloc(&w->state_bf16, bytes) != cudaSuccess) return false;
    *extra = bytes;
  }
  return true;
}
inline void tc_workspace_destroy(TcWorkspace* w) { cudaFree(w->state_bf16); w->state_bf16 = nullptr; }

// window_tc1 (one query tile per item) and its launcher live in rehyat_tc_single.cuh
inline int tc_launch_window1(int head_dim, int exp_poly, int n_sm, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                             __nv_bfloat16* o, const Geo& g, const float* rd, int rd_rows, float scale, int c_mode,
                             const ptx::WaitArgs& wa, float* share, cudaStream_t st);
inline bool tc_set_attributes1();

inline int tc_set_attributes() {
  bool ok = tc_set_attributes1() &&
            cudaFuncSetAttribute(window_tc<0, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<128>::SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(window_tc<1, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<128>::SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(window_tc<2, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<128>::SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(window_tc<3, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<128>::SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(window_tc<0, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<64>::SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(window_tc<1, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<64>::SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(window_tc<2, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<64>::SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(window_tc<3, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<64>::SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(phi_tc<true, 2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PH_SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(phi_tc<true, 0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PH_SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(phi_tc<false, 0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PH_SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(phi_tc<true, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PH_SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(phi_tc<false, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PH_SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(readout_tc<true, 2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, RD_SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(readout_tc<true, 0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, RD_SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(readout_tc<false, 0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, RD_SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(readout_tc<true, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, RD_SMEM) == cudaSuccess &&
            cudaFuncSetAttribute(readout_tc<false, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, RD_SMEM) == cudaSuccess;
  return ok ? REHYAT_OK : REHYAT_ERR_CUDA;
}

inline bool tc_encode(const TcWorkspace* w, CUtensorMap* tm, const void* base, int rank, const cuuint64_t* dims,
                      const cuuint64_t* strides, const cuuint32_t* box) {
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return ((EncodeTiledFn)w->encode_fn)(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), dims,
                                       strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
         CUDA_SUCCESS;
}

// Tensor map over one of q, k, v: dims (d, N, heads, batch), box [64 x 128 rows], 128-byte swizzle,
// out-of-range rows read as zero.
inline bool tc_make_tmap(const TcWorkspace* w, CUtensorMap* tm, const void* base, const Geo& g, int batch) {
  const cuuint64_t dims[4] = {(cuuint64_t)w->head_dim, (cuuint64_t)g.N, (cuuint64_t)g.n_heads, (cuuint64_t)batch};
  const cuuint64_t strides[3] = {(cuuint64_t)g.stride_n * 2, (cuuint64_t)g.stride_h * 2, (cuuint64_t)g.stride_b * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)TC_BN, 1, 1};
  return tc_encode(w, tm, base, 4, dims, strides, box);
}
// The same over q: its own row count and strides (see Geo).
inline bool tc_make_tmap_q(const TcWorkspace* w, CUtensorMap* tm, const void* base, const Geo& g, int batch) {
  const cuuint64_t dims[4] = {(cuuint64_t)w->head_dim, (cuuint64_t)g.Nq, (cuuint64_t)g.n_heads, (cuuint64_t)batch};
  const cuuint64_t strides[3] = {(cuuint64_t)g.qstride_n * 2, (cuuint64_t)g.qstride_h * 2, (cuuint64_t)g.qstride_b * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)TC_BN, 1, 1};
  return tc_encode(w, tm, base, 4, dims, strides, box);
}
// Row-major [planes][rows][cols] bf16 matrix stack, box [64 cols x box_rows].
inline bool tc_make_tmap_3d(const TcWorkspace* w, CUtensorMap* tm, const void* base, int cols, int rows, int planes,
                            int box_rows) {
  const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)planes};
  const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)cols * rows * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  return tc_encode(w, tm, base, 3, dims, strides, box);
}

// Launches window_tc for the chunks of one group.  `rd` is the linear read-out of the group's queries.
inline int tc_launch_window(TcWorkspace* w, const void* q, const void* k, const void* v, void* out, const Geo& g,
                            int batch, const float* rd, int rd_rows, int c_mode, const ptx::WaitArgs& wa, float* share,
                            cudaStream_t st) {
  CUtensorMap tq, tk, tv;
  if (!tc_make_tmap_q(w, &tq, q, g, batch) || !tc_make_tmap(w, &tk, k, g, batch) || !tc_make_tmap(w, &tv, v, g, batch))
    return REHYAT_ERR_CUDA;
  const int pairs = (g.Np + TC_QT * TC_BM - 1) / (TC_QT * TC_BM);
  const int n_items = pairs * g.G * g.BH;
  const dim3 grid(n_items < w->n_sm ? n_items : w->n_sm);
  const float scale = 1.0f / sqrtf((float)w->head_dim);
  __nv_bfloat16* o = (__nv_bfloat16*)out;
  // Items of two query tiles share their K/V tiles in shared memory; items of one tile (window_tc1) take half
  // as long each and fill the SMs better when there are few of them, as in a chunk-by-chunk step.  Whole waves
  // of items over the SMs decide; per tile a one-tile item costs about 8 % more.
  const long long n1 = (long long)((g.Np + TC_BM - 1) / TC_BM) * g.G * g.BH;
  const double cost2 = 2.0 * (double)((n_items + w->n_sm - 1) / w->n_sm), cost1 = 1.08 * (double)((n1 + w->n_sm - 1) / w->n_sm);
  if (w->item_tiles == 1 || (w->item_tiles == 0 && cost1 < 0.93 * cost2)) {
    w->last_item_tiles = 1;
    return tc_launch_window1(w->head_dim, w->exp_poly, w->n_sm, tq, tk, tv, o, g, rd, rd_rows, scale, c_mode, wa, share, st);
  }
  w->last_item_tiles = 2;
#define REHYAT_LAUNCH_WINDOW(E, D) \
  window_tc<E, D><<<grid, TC_THREADS, WinShape<D>::SMEM, st>>>(tq, tk, tv, o, g, rd, rd_rows, scale, c_mode, wa, n_items, pairs, share)
#define REHYAT_LAUNCH_WINDOW_D(D)                \
  switch (w->exp_poly) {                         \
    case 0: REHYAT_LAUNCH_WINDOW(0, D); break;   \
    case 2: REHYAT_LAUNCH_WINDOW(2, D); break;   \
    case 3: REHYAT_LAUNCH_WINDOW(3, D); break;   \
    default: REHYAT_LAUNCH_WINDOW(1, D); break;  \
  }
  if (w->head_dim == 64) { REHYAT_LAUNCH_WINDOW_D(64) } else { REHYAT_LAUNCH_WINDOW_D(128) }
#undef REHYAT_LAUNCH_WINDOW_D
#undef REHYAT_LAUNCH_WINDOW
  return cudaGetLastError() == cudaSuccess ? REHYAT_OK : REHYAT_ERR_CUDA;
}

// phi_k + chunk-state partial sums of one group (Eq. 17-18).
inline int tc_launch_state(const TcWorkspace* w, const void* k, const void* v, const rehyat_phi_params* phi,
                           const Geo& g, int batch, int Dh, int Dp, int P, int n_mid, int act_hidden, int act_out,
                           int n_split, float* partial, const ptx::WaitArgs& wa, cudaStream_t st) {
  const int d = w->head_dim;
  CUtensorMap tk, tv, tw1, tw2, twm;
  if (!tc_make_tmap(w, &tk, k, g, batch) || !tc_make_tmap(w, &tv, v, g, batch) ||
      !tc_make_tmap_3d(w, &tw1, phi->k_W1, d, Dh, g.n_heads, 128) ||
      !tc_make_tmap_3d(w, &tw2, phi->k_W2, Dh, Dp, g.n_heads, 128))
    return REHYAT_ERR_CUDA;
  twm = tw2;                                                        // not read without hidden layers in between
  if (n_mid > 0 && !tc_make_tmap_3d(w, &twm, phi->k_Wmid, Dh, Dh, g.n_heads * n_mid, 128)) return REHYAT_ERR_CUDA;
  PhiTcArgs a = {};
  a.b1 = (const __nv_bfloat16*)phi->k_b1; a.b2 = (const __nv_bfloat16*)phi->k_b2; a.bm = (const __nv_bfloat16*)phi->k_bmid;
  a.P = P; a.act_hidden = act_hidden; a.act_out = act_out;
  a.d = d; a.Dh = Dh; a.Dp = Dp; a.n_mid = n_mid;
  a.n_split = n_split; a.partial = partial; a.wa = wa;
  const PhiKernelChoice ch = tc_phi_choice(d, Dh, Dp, P, n_mid, act_hidden, act_out);
  const dim3 grid(n_split, g.G, g.BH);
#define REHYAT_LAUNCH_PHI(R, PC, GEN) phi_tc<R, PC, GEN><<<grid, PH_THREADS, PH_SMEM, st>>>(tk, tv, tw1, tw2, twm, g, a)
  if (ch.gen) { if (ch.relu) REHYAT_LAUNCH_PHI(true, 0, true); else REHYAT_LAUNCH_PHI(false, 0, true); }
  else if (ch.pc == 2) REHYAT_LAUNCH_PHI(true, 2, false);
  else if (ch.relu) REHYAT_LAUNCH_PHI(true, 0, false);
  else REHYAT_LAUNCH_PHI(false, 0, false);
#undef REHYAT_LAUNCH_PHI
  return cudaGetLastError() == cudaSuccess ? REHYAT_OK : REHYAT_ERR_CUDA;
}

// phi_q + linear read-out of one group's queries (Eq. 7, 9, 16).
inline int tc_launch_readout(const TcWorkspace* w, const void* q, const rehyat_phi_params* phi, const Geo& g, int batch,
                             int Dh, int Dp, int P, int n_mid, int act_hidden, int act_out, const float* state, float* rd,
                             int rd_rows, const ptx::WaitArgs& wa, cudaStream_t st) {
  const int d = w->head_dim;
  CUtensorMap tq, tw1, tw2, twm, ts;
  if (!tc_make_tmap_q(w, &tq, q, g, batch) || !tc_make_tmap_3d(w, &tw1, phi->q_W1, d, Dh, g.n_heads, 128) ||
      !tc_make_tmap_3d(w, &tw2, phi->q_W2, Dh, Dp, g.n_heads, 128) ||
      !tc_make_tmap_3d(w, &ts, w->state_bf16, d, Dp, g.G * g.BH, 64))
    return REHYAT_ERR_CUDA;
  PhiTcArgs a = {};
  twm = tw2;                                                        // not read without hidden layers in between
  if (n_mid > 0 && !tc_make_tmap_3d(w, &twm, phi->q_Wmid, Dh, Dh, g.n_heads * n_mid, 128)) return REHYAT_ERR_CUDA;
  a.b1 = (const __nv_bfloat16*)phi->q_b1; a.b2 = (const __nv_bfloat16*)phi->q_b2; a.bm = (const __nv_bfloat16*)phi->q_bmid;
  a.P = P; a.act_hidden = act_hidden; a.act_out = act_out;
  a.d = d; a.Dh = Dh; a.Dp = Dp; a.n_mid = n_mid;
  a.state = state; a.rd = rd; a.rd_rows = rd_rows; a.wa = wa;
  // One CTA per SM: split a chunk's query tiles over as many CTAs as costs the fewest tile-times over all waves.
  const int tiles = (g.Np + 127) / 128;
  int busy = 0;
  for (int t = g.t0; t < g.t0 + g.G; ++t) busy += geo_linear(g, t);
  const long long units = (long long)(busy > 0 ? busy : 1) * g.BH;
  long long best = -1;
  int best_s = 1;
  for (int s = 1; s <= 16; ++s) {
    const long long cost = ((units * s + w->n_sm - 1) / w->n_sm) * ((tiles + s - 1) / s);
    if (best < 0 || cost < best) { best = cost; best_s = s; }
  }
  a.tiles_per_cta = (tiles + best_s - 1) / best_s;
  const int ctas = (tiles + a.tiles_per_cta - 1) / a.tiles_per_cta;
  const PhiKernelChoice ch = tc_phi_choice(d, Dh, Dp, P, n_mid, act_hidden, act_out);
  const dim3 grid(ctas, g.G, g.BH);
#define REHYAT_LAUNCH_RD(R, PC, GEN) readout_tc<R, PC, GEN><<<grid, PH_THREADS, RD_SMEM, st>>>(tq, tw1, tw2, twm, ts, g, a)
  if (ch.gen) { if (ch.relu) REHYAT_LAUNCH_RD(true, 0, true); else REHYAT_LAUNCH_RD(false, 0, true); }
  else if (ch.pc == 2) REHYAT_LAUNCH_RD(true, 2, false);
  else if (ch.relu) REHYAT_LAUNCH_RD(true, 0, false);
  else REHYAT_LAUNCH_RD(false, 0, false);
#undef REHYAT_LAUNCH_RD
  return cudaGetLastError() == cudaSuccess ? REHYAT_OK : REHYAT_ERR_CUDA;
}

}  // namespace rehyat
