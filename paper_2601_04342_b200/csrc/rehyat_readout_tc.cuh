// Tensor-core kernel of the linear read-out for bf16, head_dim 64 or 128, phi widths up to 256 (the schedule is
// laid out for 128 / 256 / 256; GEN = true reads the extents from the arguments as phi_tc does):
//   phi_q on tiles of 128 queries (Section 3.2 "Characterization of phi"), then phi_q(Q tile) s_t on the
//   tensor core and phi_q(Q tile) z_t on the ALUs (Eq. 7, 9, 16), written as the fp32 read-out of the tile.
//
// Per tile  H = act(X W1^T + b1) -> U = act(H W2^T + b2) -> phi = U^(1..P) -> R = phi [s_t]  as 128x128 halves.
// Unlike the state kernel this one has TMEM to spare, which it uses twice:
//   * two scratch accumulators, so that the epilogue of one half runs while the tensor core works on the next;
//   * H (bf16) goes back to TMEM and is the A operand of the second GEMM from there, which frees 64 KB of shared
//     memory for a seven-stage ring of weight / state tiles - a TMA round trip from L2 costs about 1800 cycles
//     under load, so the bytes in flight are what bounds the weight stream.
// Roles (320 threads): warps 0-7 epilogues (two threads per token), warp 8 TMA producer, warp 9 UMMA issuer.
// TMEM columns: scratch A [0,128), scratch B [128,256), H [256,384) (256 hidden units as bf16 pairs), R [384,512).
#pragma once

#include <cuda.h>

#include "rehyat_common.cuh"
#include "rehyat_ptx.cuh"
#include "rehyat_phi_tc.cuh"

namespace rehyat {

constexpr int RD_RING = 7;
constexpr int RD_WT_BYTES = 128 * 64 * 2;                        // one weight / state tile: 16 KB
constexpr int RD_OFF_X = 0;
constexpr int RD_OFF_PHI0 = RD_OFF_X + PH_TILE_BYTES;
constexpr int RD_OFF_PHI1 = RD_OFF_PHI0 + PH_TILE_BYTES;
constexpr int RD_OFF_RING = RD_OFF_PHI1 + PH_TILE_BYTES;
constexpr int RD_OFF_BIAS = RD_OFF_RING + RD_RING * RD_WT_BYTES;  // b1[256], b2[256], z[256], two partial phi.z sums per token (x2: by tile parity), bmid[2][256]
constexpr int RD_OFF_BARS = RD_OFF_BIAS + (5 + PH_MAX_MID) * 256 * 4;
constexpr int RD_SMEM = RD_OFF_BARS + 512 + 1024;

struct RdBars {
  uint64_t x_full, x_empty;
  uint64_t ring_full[RD_RING], ring_empty[RD_RING];
  uint64_t acc_ready[2], epi_done[2], out_ready, out_read;
  uint64_t nl_ready;           // both halves of a tile's phi.z sums are in shared memory
  uint64_t drained;            // every tcgen05.mma of the issuer has completed
  uint32_t tmem_base;
  ptx::WaitCtx wctx;
};

// tm_x: Q, 4-D like the window kernel's maps.  tm_w1: (d, D_h, heads), tm_w2: (D_h, D', heads), tm_wm: (D_h, D_h,
// heads * n_mid) (any valid map when n_mid = 0), boxes [64 x 128].  tm_s: bf16 states (d, D', G*BH), box [64 x 64].
// PC: polynomial degree known at compile time (0: read it from the arguments; 2 needs D' = 256).
// A hidden layer of a deeper map (GEN only) reads H from TMEM and writes it back there: both halves of its GEMM
// have completed before the first column of H is overwritten.
template <bool RELU, int PC, bool GEN>
__global__ void __launch_bounds__(PH_THREADS, 1)
readout_tc(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w1,
           const __grid_constant__ CUtensorMap tm_w2, const __grid_constant__ CUtensorMap tm_wm,
           const __grid_constant__ CUtensorMap tm_s, Geo g, PhiTcArgs a) {
  using namespace ptx;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sb = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (sb - smem_u32(smem_raw));
  RdBars* bars = reinterpret_cast<RdBars*>(smem + RD_OFF_BARS);
  float* s_b1 = reinterpret_cast<float*>(smem + RD_OFF_BIAS);
  float* s_b2 = s_b1 + 256;
  float* s_z = s_b2 + 256;
  float* s_nl = s_z + 256;
  float* s_bm = s_nl + 512;
  const uint32_t wc = smem_u32(&bars->wctx);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ci = blockIdx.y, bh = blockIdx.z, t = g.t0 + ci;
  const int b_idx = bh / g.n_heads, h_idx = bh % g.n_heads;
  if (!geo_linear(g, t)) return;                                    // empty linear set
  const PhiExtents<GEN> ex(a);
  const int d = ex.d, Dp = ex.Dp, SD = ex.sd(), ks1 = ex.ks1(), ks2 = ex.ks2(), nh = ex.nh(), nu = ex.nu();
  const int nf = (Dp + 63) / 64;                                    // 64-feature blocks of the state
  const int n_mid = ex.n_mid;
  const int q0 = geo_q0(g, t), q1 = geo_q1(g, t);
  const int tok_a = min(q0 + (int)blockIdx.x * a.tiles_per_cta * 128, q1);
  const int tok_b = min(tok_a + a.tiles_per_cta * 128, q1);
  if (tok_a >= tok_b) return;
  const int n_tiles = (tok_b - tok_a + 127) / 128;

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars->x_full), 1); mbar_init(smem_u32(&bars->x_empty), 1);
    for (int s = 0; s < RD_RING; ++s) {
      mbar_init(smem_u32(&bars->ring_full[s]), 1); mbar_init(smem_u32(&bars->ring_empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&bars->acc_ready[b]), 1); mbar_init(smem_u32(&bars->epi_done[b]), 8); }
    mbar_init(smem_u32(&bars->out_ready), 1); mbar_init(smem_u32(&bars->out_read), 8);
    mbar_init(smem_u32(&bars->nl_ready), 8); mbar_init(smem_u32(&bars->drained), 1);
    wait_ctx_init(&bars->wctx, a.wa);
    fence_mbar_init();
  }
  for (int i = threadIdx.x; i < 256; i += PH_THREADS) {             // biases and z_t as fp32, zero beyond the widths
    s_b1[i] = i < ex.Dh ? __bfloat162float(a.b1[(size_t)h_idx * ex.Dh + i]) : 0.f;
    s_b2[i] = i < Dp ? __bfloat162float(a.b2[(size_t)h_idx * Dp + i]) : 0.f;
    s_z[i] = i < Dp ? a.state[(((size_t)ci * g.BH + bh) * Dp + i) * SD + d] : 0.f;
    for (int m = 0; m < n_mid; ++m)
      s_bm[m * 256 + i] = i < ex.Dh ? __bfloat162float(a.bm[((size_t)h_idx * n_mid + m) * ex.Dh + i]) : 0.f;
  }
  if (warp == 9) {
    tmem_alloc(smem_u32(&bars->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  constexpr uint32_t T_SCR = 0, T_H = 256, T_R = 384;
  const uint32_t sX = sb + RD_OFF_X, sPhi0 = sb + RD_OFF_PHI0, sPhi1 = sb + RD_OFF_PHI1, sRing = sb + RD_OFF_RING;

  if (warp == 8) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one() && !a.wa.withhold_loads) {
      prefetch_tensormap(&tm_x); prefetch_tensormap(&tm_w1); prefetch_tensormap(&tm_w2); prefetch_tensormap(&tm_s);
      if (n_mid > 0) prefetch_tensormap(&tm_wm);
      uint32_t ring_i = 0, n_x = 0;                                 // ring tiles and X tiles issued so far
      bool alive = true;
      auto ring_slot = [&](uint32_t& full, uint32_t bytes) -> uint32_t {   // waits for the next stage to be free; 0 on abort
        const int s = ring_i % RD_RING;
        alive = alive && mbar_wait(smem_u32(&bars->ring_empty[s]), ((ring_i / RD_RING) & 1) ^ 1, wc, PH_ERR_LOAD);
        if (!alive) return 0u;
        full = smem_u32(&bars->ring_full[s]);
        mbar_expect_tx(full, bytes);
        ++ring_i;
        return sRing + s * RD_WT_BYTES;
      };
      auto weight_load = [&](const CUtensorMap* tm, int x, int y, int plane) {
        uint32_t full = 0;
        const uint32_t dst = ring_slot(full, RD_WT_BYTES);
        if (dst) tma_load_3d(dst, tm, full, x, y, plane);
      };
      auto state_load = [&](int f) {                                // [64 features x d] as 64-column boxes
        uint32_t full = 0;
        const uint32_t dst = ring_slot(full, 8192u * ks1);
        if (dst)
          for (int ks = 0; ks < ks1; ++ks) tma_load_3d(dst + ks * 8192, &tm_s, full, ks * 64, f * 64, ci * g.BH + bh);
      };
      auto state_half = [&](int c) {                                // the blocks of features [128 c, 128 c + 128)
        for (int f = 2 * c; f < 2 * c + 2 && f < nf; ++f) state_load(f);
      };
      for (int j = 0; j < n_tiles && alive; ++j) {
        alive = mbar_wait(smem_u32(&bars->x_empty), (j & 1) ^ 1, wc, PH_ERR_LOAD);
        if (!alive) break;
        const uint32_t xf = smem_u32(&bars->x_full);
        mbar_expect_tx(xf, PH_SUB * ks1);
        for (int ks = 0; ks < ks1; ++ks)
          tma_load_4d(sX + ks * PH_SUB, &tm_x, xf, ks * 64, tok_a - g.q_off + j * 128, h_idx, b_idx);
        ++n_x;
        // the ring follows the issue order of the MMAs: read-out of the previous tile between this tile's H halves
        for (int ks = 0; ks < ks1; ++ks) weight_load(&tm_w1, ks * 64, 0, h_idx);
        if (j > 0) state_half(0);
        if (nh == 2)
          for (int ks = 0; ks < ks1; ++ks) weight_load(&tm_w1, ks * 64, 128, h_idx);
        if (j > 0 && nu == 2) state_half(1);
        for (int m = 0; m < n_mid; ++m)
          for (int half = 0; half < nh; ++half)
            for (int ks = 0; ks < ks2; ++ks) weight_load(&tm_wm, ks * 64, half * 128, h_idx * n_mid + m);
        for (int half = 0; half < nu; ++half)
          for (int ks = 0; ks < ks2; ++ks) weight_load(&tm_w2, ks * 64, half * 128, h_idx);
      }
      for (int c = 0; c < nu && alive; ++c) state_half(c);
      if (!alive) {
        // Given up: wait for the last load issued into every buffer before the CTA exits (the full barriers
        // complete by byte count, whatever the consumers do).
        if (n_x > 0) mbar_wait_drain(smem_u32(&bars->x_full), (n_x - 1) & 1, wc);
        for (uint32_t back = 0; back < (uint32_t)RD_RING; ++back)
          if (ring_i > back)
            mbar_wait_drain(smem_u32(&bars->ring_full[(ring_i - 1 - back) % RD_RING]), ((ring_i - 1 - back) / RD_RING) & 1, wc);
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ UMMA issuer
    if (elect_one()) {
      constexpr uint32_t id_kk = idesc_bf16(128, 128, 0, 0);       // A K-major (smem or TMEM), B K-major: the MLP GEMMs
      const uint32_t id_rd = idesc_bf16(128, d, 0, 1);             // A = phi (K-major), B = state (MN-major)
      uint32_t ring_i = 0, n_epi[2] = {0, 0};
      const uint64_t d_x = smem_desc_sw128(sX, 16, 1024);
      // A wait that is given up ends the role at once: the helpers return false and run() returns, so nothing
      // further is issued.  No flag is carried along; the hot path pays one predicated branch per wait.
      auto wait = [&](uint64_t* bar, uint32_t parity) -> bool {
        if (!mbar_wait(smem_u32(bar), parity, wc, PH_ERR_MMA)) return false;
        tc_fence_after();
        return true;
      };
      auto ring_wait = [&]() -> uint32_t {                          // 0 on abort
        const int s = ring_i % RD_RING;
        return wait(&bars->ring_full[s], (ring_i / RD_RING) & 1) ? sRing + s * RD_WT_BYTES : 0u;
      };
      auto ring_release = [&]() {
        umma_commit(smem_u32(&bars->ring_empty[ring_i % RD_RING]));
        ++ring_i;
      };
      auto wait_epi = [&](int b) -> bool {                          // the next epilogue that used scratch b is done
        if (!wait(&bars->epi_done[b], n_epi[b] & 1)) return false;
        ++n_epi[b];
        return true;
      };
      auto h_half = [&](int b) -> bool {                            // H[:, 128 b : 128 b + 128] = X W1[...]^T into scratch b
        for (int ks = 0; ks < ks1; ++ks) {
          const uint32_t bt = ring_wait();
          if (!bt) return false;
          const uint64_t da = smem_desc_advance(d_x, ks * PH_SUB), db = smem_desc_sw128(bt, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            umma_ss(tmem + T_SCR + b * 128, smem_desc_advance(da, kk * 32), smem_desc_advance(db, kk * 32), id_kk, (ks | kk) != 0);
          ring_release();
        }
        umma_commit(smem_u32(&bars->acc_ready[b]));
        return true;
      };
      auto u_half = [&](int b) -> bool {                            // U[:, 128 b : ...] = H W2[...]^T with H read from TMEM
        for (int ks = 0; ks < ks2; ++ks) {
          const uint32_t bt = ring_wait();
          if (!bt) return false;
          const uint64_t db = smem_desc_sw128(bt, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            umma_ts(tmem + T_SCR + b * 128, tmem + T_H + (ks * 4 + kk) * 8, smem_desc_advance(db, kk * 32), id_kk, (ks | kk) != 0);
          ring_release();
        }
        umma_commit(smem_u32(&bars->acc_ready[b]));
        return true;
      };
      auto readout_half = [&](int c, uint32_t phi_base) -> bool {   // R (+)= phi[:, 128 c : ...] s_t[128 c : ..., :]
        for (int f = 0; f < 2 && 2 * c + f < nf; ++f) {
          const uint32_t bt = ring_wait();
          if (!bt) return false;
          const uint64_t da = smem_desc_sw128(phi_base + f * PH_SUB, 16, 1024), db = smem_desc_sw128(bt, 8192, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            umma_ss(tmem + T_R, smem_desc_advance(da, kk * 32), smem_desc_advance(db, kk * 2048), id_rd, (c | f | kk) != 0);
          ring_release();
        }
        return true;
      };
      auto run = [&]() {
        for (int j = 0; j < n_tiles; ++j) {
          if (!wait(&bars->x_full, j & 1)) return;
          if (j > 0 && !wait_epi(0)) return;                          // U half 0 of tile j-1: scratch A free, phi half 0 written
          if (!h_half(0)) return;
          if (j > 0) {
            if (j > 1 && !wait(&bars->out_read, (j - 2) & 1)) return; // the read-out of tile j-2 has left TMEM
            if (!readout_half(0, sPhi0)) return;
            if (nu == 2 && !wait_epi(1)) return;                      // U half 1 of tile j-1
          }
          if (nh == 2 && !h_half(1)) return;
          umma_commit(smem_u32(&bars->x_empty));
          if (j > 0) {
            if (nu == 2 && !readout_half(1, sPhi1)) return;
            umma_commit(smem_u32(&bars->out_ready));
          }
          if (!wait_epi(0) || (nh == 2 && !wait_epi(1))) return;      // all of H is in TMEM
          for (int m = 0; m < n_mid; ++m) {                           // hidden layers: H -> scratch -> H
            if (!u_half(0) || (nh == 2 && !u_half(1))) return;
            if (!wait_epi(0) || (nh == 2 && !wait_epi(1))) return;
          }
          if (!u_half(0) || (nu == 2 && !u_half(1))) return;
        }
        if (!wait_epi(0)) return;
        if (n_tiles > 1 && !wait(&bars->out_read, (n_tiles - 2) & 1)) return;
        if (!readout_half(0, sPhi0)) return;
        if (nu == 2) {
          if (!wait_epi(1)) return;
          if (!readout_half(1, sPhi1)) return;
        }
        umma_commit(smem_u32(&bars->out_ready));
      };
      run();
      // Everything this thread has issued is complete once `drained` flips; the abort flag does not cut this
      // wait short, so that TMEM is never freed with a tcgen05.mma still running.
      umma_commit(smem_u32(&bars->drained));
      mbar_wait_drain(smem_u32(&bars->drained), 0, wc);
    }
  } else {
    // ------------------------------------------------------------------ epilogues
    // Eight warps: warp w serves TMEM lanes 32*(w%4).. (one token per thread) and the column half w/4 of every
    // 128-column accumulator, so two threads share a token.
    const int qd = warp & 3, ch = warp >> 2;
    const int r = qd * 32 + lane;
    const uint32_t lane_off = (uint32_t)(qd * 32) << 16;
    const int part_w = Dp / (PC ? PC : a.P);                        // RELU: a multiple of 32
    // After a wait has been given up anywhere in the CTA every later wait returns at once.  These warps then run
    // through the rest of the current tile on whatever the accumulators hold (tcgen05.ld / st need all 32 lanes,
    // so nothing is skipped lane by lane; every address stays inside the CTA's TMEM and shared memory) and leave
    // at the head of the next tile, where the whole warp looks at the flag together.
    auto aborted = [&]() -> bool { return __any_sync(0xffffffffu, wait_ctx_aborted(wc) != 0); };
    auto wait = [&](uint64_t* bar, uint32_t parity) { mbar_wait(smem_u32(bar), parity, wc, PH_ERR_EPI); };
    // bias + activation (+ power) of 32 accumulator columns -> 16 bf16 pairs
    auto activate = [&](const auto& x, const float* bias, bool is_u, int col0, auto& w) {
      constexpr int NC = sizeof(x) / sizeof(x[0]);                 // columns of this block
      if (RELU) {
        const int part = !is_u ? 0 : PC == 1 ? 0 : PC == 2 ? (col0 >> 7) : col0 / part_w;   // uniform over the block's columns
#pragma unroll
        for (int e = 0; e < NC; e += 4) {
          const float4 b4 = *reinterpret_cast<const float4*>(bias + e);
          float y0, y1, y2, y3;
          upk2(add2(pk2u(x[e], x[e + 1]), pk2(b4.x, b4.y)), y0, y1);
          upk2(add2(pk2u(x[e + 2], x[e + 3]), pk2(b4.z, b4.w)), y2, y3);
          if (part == 0) {
            w[e >> 1] = pack_bf16_relu(y0, y1);
            w[(e >> 1) + 1] = pack_bf16_relu(y2, y3);
          } else {
            y0 = fmaxf(y0, 0.f); y1 = fmaxf(y1, 0.f); y2 = fmaxf(y2, 0.f); y3 = fmaxf(y3, 0.f);
            float p0 = y0 * y0, p1 = y1 * y1, p2 = y2 * y2, p3 = y3 * y3;
            if (part == 2) { p0 *= y0; p1 *= y1; p2 *= y2; p3 *= y3; }
            if (part == 3) { p0 *= p0; p1 *= p1; p2 *= p2; p3 *= p3; }
            w[e >> 1] = pack_bf16(p0, p1);
            w[(e >> 1) + 1] = pack_bf16(p2, p3);
          }
        }
      } else {
        const int act = is_u ? a.act_out : a.act_hidden;
        if (GEN && is_u) {                                          // parts end anywhere; features beyond D' are zero
#pragma unroll
          for (int e = 0; e < NC; e += 2) {
            const int f0 = col0 + e;
            const float y0 = apply_act(__uint_as_float(x[e]) + bias[e], act);
            const float y1 = apply_act(__uint_as_float(x[e + 1]) + bias[e + 1], act);
            w[e >> 1] = pack_bf16(f0 < Dp ? poly_power(y0, f0 / part_w) : 0.f,
                                  f0 + 1 < Dp ? poly_power(y1, (f0 + 1) / part_w) : 0.f);
          }
        } else {
          const int part = is_u ? col0 / part_w : 0;
#pragma unroll
          for (int e = 0; e < NC; e += 2) {
            const float y0 = apply_act(__uint_as_float(x[e]) + bias[e], act);
            const float y1 = apply_act(__uint_as_float(x[e + 1]) + bias[e + 1], act);
            w[e >> 1] = pack_bf16(poly_power(y0, part), poly_power(y1, part));
          }
        }
      }
    };
    auto readout_store = [&](int jt) {                              // fp32 read-out of tile jt leaves TMEM
      wait(&bars->out_ready, jt & 1);
      tc_fence_after();
      wait(&bars->nl_ready, jt & 1);                                 // both halves of the tile's phi.z sums are written
      if (aborted()) return;                                         // nothing of an abandoned launch is stored
      const float* nlp = s_nl + (jt & 1) * 256;
      const bool tok_valid = tok_a + jt * 128 + r < tok_b;
      const int ric = tok_a + jt * 128 + r - q0;                    // row inside the chunk; its tile is 128-aligned
      uint4* rdh = reinterpret_cast<uint4*>(a.rd);
      const float nl_row = nlp[r] + nlp[128 + r];
      const float inv_nl = nl_row != 0.f ? 1.f / nl_row : 0.f;       // the read-out is stored as the ratio aL / nL
#pragma unroll 1
      for (int cb = 0; cb < 2; ++cb) {
        if (ch * 64 + cb * 32 >= d) continue;                        // the same for the whole warp
        uint32_t x[32];
        tmem_ld32(tmem + lane_off + T_R + ch * 64 + cb * 32, x);
        tmem_wait_ld();
        if (tok_valid) {
#pragma unroll
          for (int e = 0; e < 32; e += 8)
            rdh[rdh_index(g, a.rd_rows, d, bh, ci, ric, (ch * 64 + cb * 32 + e) >> 3)] =
                make_uint4(pack_ratio_f16(__uint_as_float(x[e]) * inv_nl, __uint_as_float(x[e + 1]) * inv_nl),
                           pack_ratio_f16(__uint_as_float(x[e + 2]) * inv_nl, __uint_as_float(x[e + 3]) * inv_nl),
                           pack_ratio_f16(__uint_as_float(x[e + 4]) * inv_nl, __uint_as_float(x[e + 5]) * inv_nl),
                           pack_ratio_f16(__uint_as_float(x[e + 6]) * inv_nl, __uint_as_float(x[e + 7]) * inv_nl));
        }
      }
      if (tok_valid && ch == 1)
        rdh[rdh_index(g, a.rd_rows, d, bh, ci, ric, rdh_pieces(d) - 1)] = make_uint4(__float_as_uint(nl_row), 0u, 0u, 0u);
      tc_fence_before();
      mbar_arrive_warp(smem_u32(&bars->out_read), lane);
    };
    // The loops over halves and 16-column blocks below are kept rolled (and the read-out store has one call
    // site): the straight-line form of this role was larger than the instruction cache next to the warp schedulers
    // and spent most of its time waiting for instructions (3.6 stall cycles per issue); rolled, the kernel is 15 %
    // faster.  Blocks of 32 columns measured 12 %, blocks of 8 columns 13 %.
    uint32_t acc_phase = 0;                                         // bit `half`: parity of acc_ready[half] to wait for
    auto wait_acc = [&](int half) {
      wait(&bars->acc_ready[half], (acc_phase >> half) & 1u);
      acc_phase ^= 1u << half;
      tc_fence_after();
    };
    for (int j = 0; j <= n_tiles; ++j) {
      if (j < n_tiles) {
        if (aborted()) break;
        // H halves: bias, activation, bf16, back to TMEM as the A operand of the second GEMM
#pragma unroll 1
        for (int half = 0; half < nh; ++half) {                     // a width of at most 128 has no second half
          wait_acc(half);
#pragma unroll 1
          for (int cb = 0; cb < 4; ++cb) {
            const int col0 = half * 128 + ch * 64 + cb * 16;        // hidden unit of the first column
            uint32_t x[16], w[8];
            tmem_ld16(tmem + lane_off + T_SCR + col0, x);
            tmem_wait_ld();
            activate(x, s_b1 + col0, false, col0, w);
            tmem_st8(tmem + lane_off + T_H + (col0 >> 1), w);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive_warp(smem_u32(&bars->epi_done[half]), lane);
        }
      }
      if (j > 0) readout_store(j - 1);
      if (j == n_tiles) break;
      // hidden layers of a deeper map: both halves of the GEMM are complete before H is overwritten
      for (int m = 0; m < n_mid; ++m) {
        wait_acc(0);
        if (nh == 2) wait_acc(1);
#pragma unroll 1
        for (int half = 0; half < nh; ++half) {
#pragma unroll 1
          for (int cb = 0; cb < 4; ++cb) {
            const int col0 = half * 128 + ch * 64 + cb * 16;
            uint32_t x[16], w[8];
            tmem_ld16(tmem + lane_off + T_SCR + col0, x);
            tmem_wait_ld();
            activate(x, s_bm + m * 256 + col0, false, col0, w);
            tmem_st8(tmem + lane_off + T_H + (col0 >> 1), w);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive_warp(smem_u32(&bars->epi_done[half]), lane);
        }
      }
      // U halves: bias, activation, power, bf16, to the swizzled phi tiles; phi . z_t on the way
      const bool tok_valid = tok_a + j * 128 + r < tok_b;
      float nl4[4] = {0.f, 0.f, 0.f, 0.f};                          // four chains: the sum is not one dependent sequence
#pragma unroll 1
      for (int half = 0; half < nu; ++half) {
        wait_acc(half);
        const uint32_t dst = half == 0 ? sPhi0 : sPhi1;
#pragma unroll 1
        for (int cb = 0; cb < 4; ++cb) {
          const int col0 = half * 128 + ch * 64 + cb * 16;          // feature of the first column
          uint32_t x[16], w[8];
          tmem_ld16(tmem + lane_off + T_SCR + col0, x);
          tmem_wait_ld();
          activate(x, s_b2 + col0, true, col0, w);
          if (!tok_valid) {
#pragma unroll
            for (int e = 0; e < 8; ++e) w[e] = 0u;
          }
#pragma unroll
          for (int e = 0; e < 16; e += 8) {
            const uint4 w4 = make_uint4(w[e >> 1], w[(e >> 1) + 1], w[(e >> 1) + 2], w[(e >> 1) + 3]);
            // phi_q(q_r) . z_t with the same bf16-rounded features the tensor core sees
            const float* zz = s_z + col0 + e;
            const uint32_t ww[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              nl4[u] = fmaf(__uint_as_float(ww[u] << 16), zz[2 * u], nl4[u]);
              nl4[u] = fmaf(__uint_as_float(ww[u] & 0xffff0000u), zz[2 * u + 1], nl4[u]);
            }
            st_tile_chunk_sw128(dst, PH_SUB, r, ch * 64 + cb * 16 + e, w4);
          }
        }
        if (half == nu - 1) {
          // The buffer alternates with the tile.  It is free: its last reader (read-out store of tile j-2)
          // precedes, for every thread, that thread's arrival for U half 0 of tile j-1, which the issuer
          // waited for before the MMAs of this tile could start.
          s_nl[(j & 1) * 256 + ch * 128 + r] = (nl4[0] + nl4[1]) + (nl4[2] + nl4[3]);
          mbar_arrive_warp(smem_u32(&bars->nl_ready), lane);
        }
        fence_proxy_async_smem();
        tc_fence_before();
        mbar_arrive_warp(smem_u32(&bars->epi_done[half]), lane);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace rehyat
