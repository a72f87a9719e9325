// window_tc1: the softmax-window kernel of rehyat_tc.cuh with ONE 128-row query tile per work item.
//
// It computes what window_tc computes (Eq. 5, 6, 8) and exists for launches with few items -- a chunk-by-chunk
// step has 12 heads x 37 tiles at the Wan2.1-1.3B shape -- where items of two tiles leave SMs idle in the last
// wave.  The roles, the TMEM map (S_0 S_1 O_0 O_1), the K/V rings and the softmax arithmetic are those of
// window_tc; the difference is what the two TMEM slots hold: the key tiles of the item's window alternate between
// them (even tiles in slot 0, odd tiles in slot 1), each slot with its own running maximum, row sum and O, so
// that the tensor core and the two softmax warpgroups overlap exactly as they do for a tile pair.  The epilogue
// merges the two partial softmax results: with m = max(m_0, m_1),
//   O = O_0 2^(m_0 - m) + O_1 2^(m_1 - m),   l = l_0 2^(m_0 - m) + l_1 2^(m_1 - m)
// (Eq. 6 and 8 with the window split in two), then adds the linear read-out and divides (Eq. 5).  Both
// warpgroups own the same 128 TMEM lanes, so each finishes 64 of the 128 output columns.
#pragma once

#include "rehyat_tc.cuh"

namespace rehyat {

struct WinBars1 {
  uint64_t q_full, q_empty;
  uint64_t k_full[TC_STAGES], k_empty[TC_STAGES], v_full[TC_STAGES], v_empty[TC_STAGES];
  uint64_t s_ready[2], p_half[2][2], pv_done[2], o_free[2];
  uint64_t drained;
  uint64_t mrg_ready;       // all 256 softmax threads have written their part of mrg for the current item
  uint32_t tmem_base;
  ptx::WaitCtx wctx;
  float mrg[2][2][3][TC_BM];   // [item parity][slot]: reference maximum, true maximum and row sum of every row
};
static_assert(sizeof(WinBars1) <= 8192, "barrier block");

// Items are numbered (batch*head, chunk, query tile), query tile fastest; `tiles` = tiles of a full chunk.
// Returns false for tiles beyond the end of a short last chunk.
__device__ __forceinline__ bool win_item1(const Geo& g, int item, int tiles, WinItem& w) {
  const int tile = item % tiles, rest = item / tiles, ci = rest % g.G;
  w.bh = rest / g.G;
  w.ci = ci;
  const int t = g.t0 + ci;
  w.q0 = geo_q0(g, t); w.q1 = geo_q1(g, t); w.lo = geo_lo(g, t); w.hi = w.q1;
  w.linear = geo_linear(g, t);
  w.row_base = w.q0 + tile * TC_BM;
  if (w.row_base >= w.q1) return false;
  w.ntiles = 1;
  w.n_kv = (w.hi - w.lo + TC_BN - 1) / TC_BN;
  w.b_idx = w.bh / g.n_heads; w.h_idx = w.bh % g.n_heads;
  return true;
}

// Persistent like window_tc: gridDim.x CTAs walk the items blockIdx.x, blockIdx.x + gridDim.x, ...
// EMU: of every four pairs of exponentials, how many are evaluated on the FMA pipe.  D: head_dim.
template <int EMU, int D>
__global__ void __launch_bounds__(TC_THREADS, 1)
window_tc1(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ out, Geo g,
           const float* __restrict__ rd, int rd_rows, float scale, int c_mode, ptx::WaitArgs wa,
           int n_items, int tiles, float* __restrict__ share) {
  using namespace ptx;
  using SH = WinShape<D>;
  constexpr int TC_TILE_BYTES = SH::TILE_BYTES, TC_SUB_BYTES = SH::SUB_BYTES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sQ = smem_base;                                   // one tile
  const uint32_t sK = sQ + TC_TILE_BYTES;                          // TC_STAGES tiles
  const uint32_t sV = sK + TC_STAGES * TC_TILE_BYTES;              // TC_STAGES tiles
  WinBars1* bars = reinterpret_cast<WinBars1*>(smem + (1 + 2 * TC_STAGES) * TC_TILE_BYTES);
  const uint32_t wc = smem_u32(&bars->wctx);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars->q_full), 1); mbar_init(smem_u32(&bars->q_empty), 1);
    for (int s = 0; s < TC_STAGES; ++s) {
      mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 1);
      mbar_init(smem_u32(&bars->v_full[s]), 1); mbar_init(smem_u32(&bars->v_empty[s]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bars->s_ready[i]), 1);
      mbar_init(smem_u32(&bars->p_half[i][0]), TC_BM / 32);
      mbar_init(smem_u32(&bars->p_half[i][1]), TC_BM / 32);
      mbar_init(smem_u32(&bars->pv_done[i]), 1);
      mbar_init(smem_u32(&bars->o_free[i]), TC_BM / 32);
    }
    mbar_init(smem_u32(&bars->drained), 1);
    mbar_init(smem_u32(&bars->mrg_ready), 2 * TC_BM / 32);
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
      uint32_t kv_it = 0, n_q = 0;                                 // K/V tiles of finished items, Q loads issued
      uint32_t n_k = 0, n_v = 0;                                   // K tiles and V tiles issued so far
      bool alive = true;
      for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
        WinItem w;
        if (!win_item1(g, item, tiles, w)) continue;
        // Q of the previous item has been read by its last Q K^T
        if (n_q > 0) alive = mbar_wait(smem_u32(&bars->q_empty), (n_q - 1) & 1, wc, TC_ERR_LOAD, TC_HINT_P);
        if (!alive) break;
        const uint32_t qf = smem_u32(&bars->q_full);
        mbar_expect_tx(qf, TC_TILE_BYTES);
#pragma unroll
        for (int sb = 0; sb < SH::SUBS; ++sb) tma_load_4d(sQ + sb * TC_SUB_BYTES, &tm_q, qf, sb * 64, w.row_base - g.q_off, w.h_idx, w.b_idx);
        ++n_q;
        auto load_tile = [&](bool is_v, int j) {                     // key tile j of the item into its ring stage
          const uint32_t it = kv_it + j;
          const int s = it % TC_STAGES;
          const uint32_t ph = (it / TC_STAGES) & 1;
          const int key0 = w.lo + j * TC_BN;
          if (!mbar_wait(smem_u32(is_v ? &bars->v_empty[s] : &bars->k_empty[s]), ph ^ 1, wc, TC_ERR_LOAD, TC_HINT_P))
            return false;
          const uint32_t full = smem_u32(is_v ? &bars->v_full[s] : &bars->k_full[s]);
          const uint32_t dst = (is_v ? sV : sK) + s * TC_TILE_BYTES;
          const CUtensorMap* tm = is_v ? &tm_v : &tm_k;
          mbar_expect_tx(full, TC_TILE_BYTES);
#pragma unroll
          for (int sb = 0; sb < SH::SUBS; ++sb) tma_load_4d(dst + sb * TC_SUB_BYTES, tm, full, sb * 64, key0, w.h_idx, w.b_idx);
          if (is_v) ++n_v; else ++n_k;
          return true;
        };
        // Q K^T runs two key tiles ahead of P V, so K stays one tile ahead of V
        alive = load_tile(false, 0);
        for (int j = 0; j < w.n_kv && alive; ++j) {
          if (j + 1 < w.n_kv) alive = load_tile(false, j + 1);
          alive = alive && load_tile(true, j);
        }
        kv_it += w.n_kv;
      }
      if (!alive) {
        // Given up: wait for the last load issued into every buffer before the CTA exits (the full barriers
        // complete by byte count, whatever the consumers do).
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
      auto issue_qk = [&](int i, int s) { mma.qk(i, 0, s); };         // the one query tile into slot i
      auto issue_pv = [&](int i, int s, int half, bool acc) { mma.pv(i, s, half, acc); };
      uint32_t kv_it = 0, n_done = 0;                                // K/V tiles consumed, items done
      uint32_t n_p[2] = {0, 0};                                      // P hand-overs per slot
      bool alive = true;                                             // false once a wait has been given up: issue nothing more
      auto wait = [&](uint64_t* bar, uint32_t parity) {
        alive = alive && mbar_wait(smem_u32(bar), parity, wc, TC_ERR_MMA, TC_HINT_I);
        return alive;
      };
      for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
        WinItem w;
        if (!win_item1(g, item, tiles, w)) continue;
        if (!wait(&bars->q_full, n_done & 1)) break;
        const uint32_t base = kv_it;
        auto qk_of = [&](int jj) {                                   // S of key tile jj into slot jj & 1
          const uint32_t it = base + jj;
          const int s = it % TC_STAGES;
          if (!wait(&bars->k_full[s], (it / TC_STAGES) & 1)) return;
          tc_fence_after();
          issue_qk(jj & 1, s);
          umma_commit(smem_u32(&bars->s_ready[jj & 1]));
          umma_commit(smem_u32(&bars->k_empty[s]));
          if (jj == w.n_kv - 1) umma_commit(smem_u32(&bars->q_empty));   // the item's last Q K^T
        };
        qk_of(0);
        if (w.n_kv > 1) qk_of(1);
        for (int j = 0; j < w.n_kv && alive; ++j, ++kv_it) {
          const int i = j & 1, s = kv_it % TC_STAGES;
          if (!wait(&bars->v_full[s], (kv_it / TC_STAGES) & 1)) break;
          // the first P V of an item overwrites O: both warpgroups read both O slots in the previous epilogue
          if (j == 0 && n_done > 0) {
            if (!wait(&bars->o_free[0], (n_done - 1) & 1)) break;
            if (!wait(&bars->o_free[1], (n_done - 1) & 1)) break;
          }
          if (!wait(&bars->p_half[i][0], n_p[i] & 1)) break;
          tc_fence_after();
          issue_pv(i, s, 0, j >= 2);
          if (!wait(&bars->p_half[i][1], n_p[i] & 1)) break;
          tc_fence_after();
          issue_pv(i, s, 1, true);
          ++n_p[i];
          umma_commit(smem_u32(&bars->pv_done[i]));
          umma_commit(smem_u32(&bars->v_empty[s]));
          if (j + 2 < w.n_kv) qk_of(j + 2);                          // into the slot this P V has just read
        }
        ++n_done;
      }
      // Everything this thread has issued is complete once `drained` flips.  This wait is not cut short by the
      // abort flag: TMEM must not be freed, nor the CTA exit, with a tcgen05.mma still running.
      umma_commit(smem_u32(&bars->drained));
      mbar_wait_drain(smem_u32(&bars->drained), 0, wc);
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax + epilogue
    setmaxnreg_inc<TC_REGS_SOFTMAX>();
    const int i = (warp - 4) >> 2;                                   // TMEM slot of this warpgroup
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_off + i * TC_BN, tO = tmem + lane_off + 256 + i * 128;
    const float c = scale * 1.4426950408889634f;                     // logits -> log2 domain
    const bool out_32B = ((reinterpret_cast<uintptr_t>(out) | (uintptr_t)(g.ostride_b * 2) | (uintptr_t)(g.ostride_h * 2) |
                           (uintptr_t)(g.ostride_n * 2)) & 31u) == 0;   // every row of out starts on a 32-byte boundary
    const int r = (warp & 3) * 32 + lane;                            // row of the query tile
    uint32_t n_s[2] = {0, 0};                                        // key tiles each slot has been through
    uint32_t n_items_done = 0;
    // A wait that was given up ends the role; the warp decides together (tcgen05.ld / st need all 32 lanes).
    bool alive = true;
    auto wait = [&](uint64_t* bar, uint32_t parity) {
      alive = __all_sync(0xffffffffu, mbar_wait(smem_u32(bar), parity, wc, TC_ERR_SOFTMAX, TC_HINT_S));
      return alive;
    };
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      WinItem w;
      if (!win_item1(g, item, tiles, w)) continue;
      const int n_kv = w.n_kv, lo = w.lo, hi = w.hi;
      const int cnt0 = (n_kv + 1) >> 1, cnt1 = n_kv >> 1, cnt = i == 0 ? cnt0 : cnt1;   // this slot: tiles i, i+2, ...
      SoftmaxRow st;
      for (int t = 0; t < cnt; ++t) {
        const int j = i + 2 * t;
        if (!wait(&bars->s_ready[i], (n_s[i] + t) & 1)) break;
        tc_fence_after();
        if (!softmax_key_tile<EMU, D>(tS, tO, hi - (lo + j * TC_BN), c, t > 0, st, smem_u32(&bars->p_half[i][0]),
                                   smem_u32(&bars->p_half[i][1]), lane,
                                   [&]() { return wait(&bars->pv_done[i], (n_s[i] + t - 1) & 1); }))
          break;
      }
      if (!alive) break;
      const float m_true = st.m_true, m_used = st.m_used, l = st.sum();

      // Exchange the slots' maxima and row sums (a slot without key tiles contributes m = -inf, l = 0).  The
      // buffer alternates with the item: a warpgroup can be at most one item ahead of the other, because the
      // barrier of an item completes only with the arrivals of both.
      float (*mrg)[3][TC_BM] = bars->mrg[n_items_done & 1];
      mrg[i][0][r] = m_used; mrg[i][1][r] = m_true; mrg[i][2][r] = l;
      mbar_arrive_warp(smem_u32(&bars->mrg_ready), lane);
      if (!wait(&bars->mrg_ready, n_items_done & 1)) break;
      ++n_items_done;
      const float mu_x = mrg[i ^ 1][0][r], mt_x = mrg[i ^ 1][1][r], l_x = mrg[i ^ 1][2][r];
      const float m_fin = fmaxf(m_true, mt_x);
      const float mu0 = i == 0 ? m_used : mu_x, mu1 = i == 0 ? mu_x : m_used;
      const float l0 = i == 0 ? l : l_x, l1 = i == 0 ? l_x : l;
      const int row = w.row_base + r;
      const bool valid = row < w.q1;
      // this warpgroup's half of the read-out row is requested before the wait for the last P V
      uint4 rdv[D / 16];                                             // fp16 pairs of aL / nL
      float nL = 0.f;
      if (w.linear) {
        const int ric = (valid ? row : w.q0) - w.q0, ci = w.ci;
        const uint4* rdh = reinterpret_cast<const uint4*>(rd);
#pragma unroll
        for (int u = 0; u < D / 16; ++u) rdv[u] = __ldg(rdh + rdh_index(g, rd_rows, D, w.bh, ci, ric, i * (D / 16) + u));
        nL = __ldg(reinterpret_cast<const float*>(rdh + rdh_index(g, rd_rows, D, w.bh, ci, ric, rdh_pieces(D) - 1)));
      } else {
#pragma unroll
        for (int u = 0; u < D / 16; ++u) rdv[u] = make_uint4(0u, 0u, 0u, 0u);
      }
      float f0 = ex2((mu0 - m_fin) * c), f1 = cnt1 > 0 ? ex2((mu1 - m_fin) * c) : 0.f, lam = 0.f;
      if (w.linear) {
        lam = 1.f;
        if (c_mode == C_ZERO) {
          const float mm = m_fin * scale, rr = fmaxf(mm, 0.f), e = __expf(mm - rr);
          f0 *= e; f1 *= e;
          lam = __expf(-rr);
        }
      }
      __nv_bfloat16* orow = out + out_row_offset(g, w.bh, row) + i * (D / 2);
      if (!wait(&bars->pv_done[0], (n_s[0] + cnt0 - 1) & 1)) break;
      if (cnt1 > 0 && !wait(&bars->pv_done[1], (n_s[1] + cnt1 - 1) & 1)) break;
      tc_fence_after();
      n_s[0] += cnt0; n_s[1] += cnt1;
      const float inv = 1.f / (l0 * f0 + l1 * f1 + lam * nL);
      const float w0 = f0 * inv, w1 = f1 * inv, lami = lam * inv * nL;   // the read-out comes as the ratio aL / nL
      if (share != nullptr && valid && i == 0) share[(size_t)w.bh * g.N + row] = lami;   // part of the normaliser that is linear
      const uint32_t tO0 = tmem + lane_off + 256 + i * (D / 2);
#pragma unroll
      for (int hh = 0; hh < D / 64; ++hh) {                          // 32 of this warpgroup's D/2 columns at a time
        uint32_t o0[32], o1[32];
        tmem_ld32(tO0 + hh * 32, o0);
        if (cnt1 > 0) {
          tmem_ld32(tO0 + 128 + hh * 32, o1);
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) o1[e] = 0u;                   // slot 1 was not used
        }
        tmem_wait_ld();
        if (hh == D / 64 - 1) {                                      // this warpgroup has read both slots
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
              return pack_bf16(__uint_as_float(o0[q]) * w0 + __uint_as_float(o1[q]) * w1 + lami * rr.x,
                               __uint_as_float(o0[q + 1]) * w0 + __uint_as_float(o1[q + 1]) * w1 + lami * rr.y);
            };
            v4[e >> 3].x = fin(e + 0, x.x);
            v4[e >> 3].y = fin(e + 2, x.y);
            v4[e >> 3].z = fin(e + 4, x.z);
            v4[e >> 3].w = fin(e + 6, x.w);
          }
          if (out_32B) {                                             // whole 32-byte sectors, as in window_tc
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

// Launches window_tc1 with the tensor maps and arguments tc_launch_window has prepared.
inline int tc_launch_window1(int head_dim, int exp_poly, int n_sm, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                             __nv_bfloat16* o, const Geo& g, const float* rd, int rd_rows, float scale, int c_mode,
                             const ptx::WaitArgs& wa, float* share, cudaStream_t st) {
  const int tiles = (g.Np + TC_BM - 1) / TC_BM;
  const int n_items = tiles * g.G * g.BH;
  const dim3 grid(n_items < n_sm ? n_items : n_sm);
#define REHYAT_LAUNCH_WINDOW1(E, D) \
  window_tc1<E, D><<<grid, TC_THREADS, WinShape<D>::SMEM1, st>>>(tq, tk, tv, o, g, rd, rd_rows, scale, c_mode, wa, n_items, tiles, share)
#define REHYAT_LAUNCH_WINDOW1_D(D)               \
  switch (exp_poly) {                            \
    case 0: REHYAT_LAUNCH_WINDOW1(0, D); break;  \
    case 2: REHYAT_LAUNCH_WINDOW1(2, D); break;  \
    case 3: REHYAT_LAUNCH_WINDOW1(3, D); break;  \
    default: REHYAT_LAUNCH_WINDOW1(1, D); break; \
  }
  if (head_dim == 64) { REHYAT_LAUNCH_WINDOW1_D(64) } else { REHYAT_LAUNCH_WINDOW1_D(128) }
#undef REHYAT_LAUNCH_WINDOW1_D
#undef REHYAT_LAUNCH_WINDOW1
  return cudaGetLastError() == cudaSuccess ? REHYAT_OK : REHYAT_ERR_CUDA;
}

inline bool tc_set_attributes1() {
  return cudaFuncSetAttribute(window_tc1<0, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<128>::SMEM1) == cudaSuccess &&
         cudaFuncSetAttribute(window_tc1<1, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<128>::SMEM1) == cudaSuccess &&
         cudaFuncSetAttribute(window_tc1<2, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<128>::SMEM1) == cudaSuccess &&
         cudaFuncSetAttribute(window_tc1<3, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<128>::SMEM1) == cudaSuccess &&
         cudaFuncSetAttribute(window_tc1<0, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<64>::SMEM1) == cudaSuccess &&
         cudaFuncSetAttribute(window_tc1<1, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<64>::SMEM1) == cudaSuccess &&
         cudaFuncSetAttribute(window_tc1<2, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<64>::SMEM1) == cudaSuccess &&
         cudaFuncSetAttribute(window_tc1<3, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WinShape<64>::SMEM1) == cudaSuccess;
}

}  // namespace rehyat
