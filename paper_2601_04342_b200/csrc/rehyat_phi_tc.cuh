// Tensor-core kernel of the chunk-state increments for bf16, head_dim 64 or 128, phi widths up to 256.
//
// phi_tc evaluates the feature map phi_k of Section 3.2 ("Characterization of phi") on tiles of 128 keys with
// tcgen05.mma and feeds it straight into the contraction that consumes it: phi_k(K tile)^T [V | 1] accumulated
// in TMEM over the CTA's share of the keys a chunk newly admits (Eq. 17-18), flushed once as an fp32 partial
// state.  (The read-out kernel, readout_tc, has a file of its own; it shares the constants and PhiTcArgs.)
//
// Per tile the chain is  H = act(X W1^T + b1) -> U = act(H W2^T + b2) -> phi = U^(1..P)  with the
// two GEMMs done as 128x128 halves through one 128-column TMEM scratch accumulator (the state accumulators
// take 288 of the 512 columns):
//   warps 0-7  epilogues, two threads per token (= TMEM lane): bias, activation, power, bf16, swizzled smem tile
//   warp 8     TMA producer: X and V, weight tiles [128 x 64] through a 3-stage ring
//   warp 9     UMMA issuer
// The phi tile is written once in the 128-byte-swizzled [token][feature] image; the state GEMM reads
// it as an MN-major A operand (features are M).
//
// The schedule is laid out for head_dim 128 and D_h = D' = 256 (GEN = false: every extent a constant).  With
// GEN = true the extents come from the arguments: head_dim 64 halves the K extent of the first GEMM and the N
// extent of the state GEMM, a width of at most 128 drops the second half of its GEMM, and a width that is not
// a multiple of 128 (or 64) relies on the tensor maps, which read rows and columns beyond the matrix as zero:
// hidden units beyond D_h meet zero columns of W2, features beyond D' are zero (or masked) and never stored.
// A map of more than two layers (GEN only) runs its hidden layers h <- act(Wmid h + bmid) between the two: the
// hidden activations alternate between the H buffer and a second one made of the X tile and the phi half 0
// tile, both idle at that point (the next X tile is then requested later, after the last reader of that buffer).
#pragma once

#include <cuda.h>

#include "rehyat_common.cuh"
#include "rehyat_ptx.cuh"

namespace rehyat {

constexpr int PH_D = 128, PH_DH = 256, PH_DP = 256, PH_SD = PH_D + 4;
constexpr int PH_THREADS = 320;            // 8 epilogue warps, TMA producer, UMMA issuer
constexpr int PH_RING = 3;                // weight tiles in flight
constexpr int PH_WT_BYTES = 128 * 64 * 2;          // one weight / state tile: 16 KB
constexpr int PH_TILE_BYTES = 128 * 128 * 2;       // X, V, phi half: 32 KB (two swizzled sub-tiles)
constexpr int PH_SUB = PH_TILE_BYTES / 2;
// shared memory map (bytes from the 1024-aligned base)
constexpr int PH_OFF_X = 0;
constexpr int PH_OFF_V = PH_OFF_X + PH_TILE_BYTES;
constexpr int PH_OFF_HB = PH_OFF_V + PH_TILE_BYTES;            // 64 KB; one of its halves doubles as phi half 1
constexpr int PH_OFF_PHI0 = PH_OFF_HB + 2 * PH_TILE_BYTES;
constexpr int PH_OFF_RING = PH_OFF_PHI0 + PH_TILE_BYTES;
constexpr int PH_OFF_ONES = PH_OFF_RING + PH_RING * PH_WT_BYTES; // [16 x 128] K-major, row 0 = 1
constexpr int PH_OFF_BIAS = PH_OFF_ONES + 4096;                 // b1[256], b2[256], bmid[2][256] fp32
constexpr int PH_MAX_MID = 2;                                   // hidden layers between the first and the last
constexpr int PH_OFF_BARS = PH_OFF_BIAS + (2 + PH_MAX_MID) * 256 * 4;
constexpr int PH_SMEM = PH_OFF_BARS + 512 + 1024;

enum PhErr : int { PH_ERR_LOAD = 16, PH_ERR_MMA = 32, PH_ERR_EPI = 64 };

struct PhBars {
  uint64_t x_full, x_empty, v_full, v_empty;
  uint64_t ring_full[PH_RING], ring_empty[PH_RING];
  uint64_t acc_ready, epi_done, out_ready;
  uint64_t drained;            // every tcgen05.mma of the issuer has completed
  uint32_t tmem_base;
  ptx::WaitCtx wctx;
};

struct PhiTcArgs {
  const __nv_bfloat16* b1;     // [heads][D_h]
  const __nv_bfloat16* b2;     // [heads][D']
  int P, act_hidden, act_out;
  int d, Dh, Dp;               // head_dim (64 or 128), phi widths (read by the GEN = true kernels)
  int n_mid;                   // hidden layers between the first and the last (GEN = true kernels), at most PH_MAX_MID
  const __nv_bfloat16* bm;     // [heads][n_mid][D_h]
  int n_split;                 // state kernel: splits of a chunk's increment
  float* partial;              // state kernel: [G][n_split][BH][D'][d + 4]
  const float* state;          // read-out kernel: fp32 states (z column is read)
  float* rd;                   // read-out kernel: the read-out workspace (see rdh_index)
  int rd_rows;
  int tiles_per_cta;           // read-out kernel
  ptx::WaitArgs wa;            // status word, launch epoch, wait limit
};

// Extents of one launch: constants for the default shape, read from the arguments otherwise.
template <bool GEN>
struct PhiExtents {
  int d, Dh, Dp, n_mid;
  __device__ explicit PhiExtents(const PhiTcArgs& a)
      : d(GEN ? a.d : PH_D), Dh(GEN ? a.Dh : PH_DH), Dp(GEN ? a.Dp : PH_DP), n_mid(GEN ? a.n_mid : 0) {}
  __device__ int sd() const { return d + 4; }              // row of a state: d columns of s, then z, padded
  __device__ int ks1() const { return d / 64; }            // 64-column K blocks of the first GEMM
  __device__ int ks2() const { return (Dh + 63) / 64; }    // ... of the second
  __device__ int nh() const { return (Dh + 127) / 128; }   // 128-column halves of H
  __device__ int nu() const { return (Dp + 127) / 128; }   // ... of U
};

// tm_x: K, tm_v: V, 4-D like the window kernel's maps.  tm_w1: (d, D_h, heads), tm_w2: (D_h, D', heads),
// tm_wm: (D_h, D_h, heads * n_mid) (any valid map when n_mid = 0), boxes [64 x 128].  PC: polynomial degree known
// at compile time (0: read it from the arguments; 2 needs D' = 256).
template <bool RELU, int PC, bool GEN>
__global__ void __launch_bounds__(PH_THREADS, 1)
phi_tc(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_v,
       const __grid_constant__ CUtensorMap tm_w1, const __grid_constant__ CUtensorMap tm_w2,
       const __grid_constant__ CUtensorMap tm_wm, Geo g, PhiTcArgs a) {
  using namespace ptx;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sb = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (sb - smem_u32(smem_raw));
  PhBars* bars = reinterpret_cast<PhBars*>(smem + PH_OFF_BARS);
  float* s_b1 = reinterpret_cast<float*>(smem + PH_OFF_BIAS);
  float* s_b2 = s_b1 + 256;
  const uint32_t wc = smem_u32(&bars->wctx);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ci = blockIdx.y, bh = blockIdx.z, t = g.t0 + ci;
  const int b_idx = bh / g.n_heads, h_idx = bh % g.n_heads;
  const PhiExtents<GEN> ex(a);
  const int Dp = ex.Dp, SD = ex.sd(), ks1 = ex.ks1(), ks2 = ex.ks2(), nh = ex.nh(), nu = ex.nu(), n_mid = ex.n_mid;

  // token range [tok_a, tok_b) of this CTA
  const int lo_prev = t > 0 ? geo_lo(g, t - 1) : 0, lo = geo_lo(g, t);
  int per = (lo - lo_prev + a.n_split - 1) / a.n_split;
  per = (per + 127) / 128 * 128;
  const int tok_a = min(lo_prev + (int)blockIdx.x * per, lo);
  const int tok_b = min(tok_a + per, lo);
  const int n_tiles = (tok_b - tok_a + 127) / 128;

  if (n_tiles == 0) {                          // nothing admitted: the partial is zero
    float* dst = a.partial + (((size_t)ci * a.n_split + blockIdx.x) * g.BH + bh) * Dp * SD;
    for (int i = threadIdx.x; i < Dp * SD / 4; i += PH_THREADS)
      reinterpret_cast<float4*>(dst)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    return;
  }

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars->x_full), 1); mbar_init(smem_u32(&bars->x_empty), 1);
    mbar_init(smem_u32(&bars->v_full), 1); mbar_init(smem_u32(&bars->v_empty), 1);
    for (int s = 0; s < PH_RING; ++s) {
      mbar_init(smem_u32(&bars->ring_full[s]), 1); mbar_init(smem_u32(&bars->ring_empty[s]), 1);
    }
    mbar_init(smem_u32(&bars->acc_ready), 1); mbar_init(smem_u32(&bars->epi_done), 8);
    mbar_init(smem_u32(&bars->out_ready), 1);
    mbar_init(smem_u32(&bars->drained), 1);
    wait_ctx_init(&bars->wctx, a.wa);
    fence_mbar_init();
  }
  // biases as fp32; the ones tile: row 0 of both 64-column sub-tiles is 1, the rest 0
  for (int i = threadIdx.x; i < 256; i += PH_THREADS) {          // zero beyond the widths
    s_b1[i] = i < ex.Dh ? __bfloat162float(a.b1[(size_t)h_idx * ex.Dh + i]) : 0.f;
    s_b2[i] = i < Dp ? __bfloat162float(a.b2[(size_t)h_idx * Dp + i]) : 0.f;
    for (int m = 0; m < n_mid; ++m)
      s_b2[(1 + m) * 256 + i] = i < ex.Dh ? __bfloat162float(a.bm[((size_t)h_idx * n_mid + m) * ex.Dh + i]) : 0.f;
  }
  {
    uint32_t* ones = reinterpret_cast<uint32_t*>(smem + PH_OFF_ONES);
    for (int i = threadIdx.x; i < 1024; i += PH_THREADS) {
      const int byte = i * 4, sub = byte / 2048, within = byte % 2048;
      ones[i] = (within < 128 && sub < 2) ? 0x3F803F80u : 0u;       // two bf16 ones
    }
    fence_proxy_async_smem();
  }
  if (warp == 9) {
    tmem_alloc(smem_u32(&bars->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  // TMEM columns: scratch [0,128), S half 0 [128,256), S half 1 [256,384), z half 0 [384,400), z half 1 [400,416)
  constexpr uint32_t T_SCR = 0, T_ACC = 128, T_Z = 384;
  constexpr int RING = PH_RING;

  const uint32_t sX = sb + PH_OFF_X, sV = sb + PH_OFF_V, sHb = sb + PH_OFF_HB, sPhi0 = sb + PH_OFF_PHI0,
                 sRing = sb + PH_OFF_RING, sOnes = sb + PH_OFF_ONES;
  auto ring_addr = [&](int s) -> uint32_t { return sRing + s * PH_WT_BYTES; };
  // The two buffers of hidden activations, each four [128 x 64] sub-tiles: 0 = the H buffer, 1 = the X tile
  // followed by the phi half 0 tile.  The first layer writes buffer 0, hidden layer m reads m % 2 and writes the other.
  auto hid_sub = [&](int buf, int sub) -> uint32_t {
    return buf == 0 ? sHb + sub * PH_SUB : (sub < 2 ? sX + sub * PH_SUB : sPhi0 + (sub - 2) * PH_SUB);
  };
  const int last_hid = n_mid & 1;                                   // where the last hidden activations are
  const uint32_t sPhiHalf0 = last_hid ? sHb + 2 * PH_SUB : sPhi0;   // phi half 0: away from the buffer the last GEMMs read
  // phi half 1 takes a half of the H buffer once the last GEMM has read it.  Where the first layer writes that
  // buffer again (last_hid == 0) it is the second half: the first half-GEMM of the next tile and its epilogue (which
  // writes the first half) then need not wait for the state GEMM that reads phi half 1.
  const uint32_t sPhiHalf1 = last_hid ? sHb : sHb + 2 * PH_SUB;

  if (warp == 8) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one() && !a.wa.withhold_loads) {
      prefetch_tensormap(&tm_x); prefetch_tensormap(&tm_w1); prefetch_tensormap(&tm_w2);
      if (n_mid > 0) prefetch_tensormap(&tm_wm);
      uint32_t ring_i = 0, n_x = 0, n_v = 0;                       // ring tiles, X tiles and V tiles issued so far
      bool alive = true;
      auto ring_load = [&](const CUtensorMap* tm, int x, int y, int z) {
        const int s = ring_i % RING;
        const uint32_t ph = (ring_i / RING) & 1;
        alive = alive && mbar_wait(smem_u32(&bars->ring_empty[s]), ph ^ 1, wc, PH_ERR_LOAD);
        if (!alive) return;
        const uint32_t full = smem_u32(&bars->ring_full[s]);
        mbar_expect_tx(full, PH_WT_BYTES);
        tma_load_3d(ring_addr(s), tm, full, x, y, z);
        ++ring_i;
      };
      for (int j = 0; j < n_tiles && alive; ++j) {
        const int tok0 = tok_a + j * 128;
        alive = mbar_wait(smem_u32(&bars->x_empty), (j & 1) ^ 1, wc, PH_ERR_LOAD);
        if (!alive) break;
        const uint32_t xf = smem_u32(&bars->x_full);
        mbar_expect_tx(xf, PH_SUB * ks1);
        for (int ks = 0; ks < ks1; ++ks) tma_load_4d(sX + ks * PH_SUB, &tm_x, xf, ks * 64, tok0, h_idx, b_idx);
        ++n_x;
        for (int half = 0; half < nh; ++half)
          for (int ks = 0; ks < ks1; ++ks) ring_load(&tm_w1, ks * 64, half * 128, h_idx);
        for (int m = 0; m < n_mid; ++m)
          for (int half = 0; half < nh; ++half)
            for (int ks = 0; ks < ks2; ++ks) ring_load(&tm_wm, ks * 64, half * 128, h_idx * n_mid + m);
        {
          alive = alive && mbar_wait(smem_u32(&bars->v_empty), (j & 1) ^ 1, wc, PH_ERR_LOAD);
          if (!alive) break;
          const uint32_t vf = smem_u32(&bars->v_full);
          mbar_expect_tx(vf, PH_SUB * ks1);
          for (int ks = 0; ks < ks1; ++ks) tma_load_4d(sV + ks * PH_SUB, &tm_v, vf, ks * 64, tok0, h_idx, b_idx);
          ++n_v;
        }
        for (int half = 0; half < nu; ++half)
          for (int ks = 0; ks < ks2; ++ks) ring_load(&tm_w2, ks * 64, half * 128, h_idx);
      }
      if (!alive) {
        // Given up: wait for the last load issued into every buffer before the CTA exits (the full barriers
        // complete by byte count, whatever the consumers do).
        if (n_x > 0) mbar_wait_drain(smem_u32(&bars->x_full), (n_x - 1) & 1, wc);
        if (n_v > 0) mbar_wait_drain(smem_u32(&bars->v_full), (n_v - 1) & 1, wc);
        for (uint32_t back = 0; back < (uint32_t)RING; ++back)
          if (ring_i > back)
            mbar_wait_drain(smem_u32(&bars->ring_full[(ring_i - 1 - back) % RING]), ((ring_i - 1 - back) / RING) & 1, wc);
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ UMMA issuer
    if (elect_one()) {
      constexpr uint32_t id_kk = idesc_bf16(128, 128, 0, 0);       // A K-major, B K-major   (the two MLP GEMMs)
      const uint32_t id_st = idesc_bf16(128, ex.d, 1, 1);          // A = phi^T (MN-major), B = V (MN-major)
      constexpr uint32_t id_z = idesc_bf16(128, 16, 1, 0);         // A = phi^T (MN-major), B = ones (K-major)
      uint32_t ring_i = 0, n_epi = 0;
      // A wait that is given up ends the role at once: the helpers return false and run() returns, so nothing
      // further is issued.  No flag is carried along; the hot path pays one predicated branch per wait.
      auto wait = [&](uint64_t* bar, uint32_t parity) -> bool {
        if (!mbar_wait(smem_u32(bar), parity, wc, PH_ERR_MMA)) return false;
        tc_fence_after();
        return true;
      };
      auto ring_release = [&]() {
        umma_commit(smem_u32(&bars->ring_empty[ring_i % RING]));
        ++ring_i;
      };
      auto wait_epi = [&]() -> bool {
        if (!wait(&bars->epi_done, n_epi & 1)) return false;
        ++n_epi;
        return true;
      };
      // one 128x128 half of an MLP GEMM: A = the X tile (buf < 0) or a buffer of hidden activations, [128 x 64*nks]
      // K-major in 64-column sub-tiles, B tiles from the ring
      auto mlp_half = [&](int buf, int nks) -> bool {
        for (int ks = 0; ks < nks; ++ks) {
          const uint64_t da = smem_desc_sw128(buf < 0 ? sX + ks * PH_SUB : hid_sub(buf, ks), 16, 1024);
          if (!wait(&bars->ring_full[ring_i % RING], (ring_i / RING) & 1)) return false;
          const uint64_t db = smem_desc_sw128(ring_addr(ring_i % RING), 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            umma_ss(tmem + T_SCR, smem_desc_advance(da, kk * 32), smem_desc_advance(db, kk * 32), id_kk, (ks | kk) != 0);
          ring_release();
        }
        umma_commit(smem_u32(&bars->acc_ready));
        return true;
      };
      // contraction that consumes phi half `c` (its tile is at phi_base)
      const uint64_t d_v = smem_desc_sw128(sV, PH_SUB, 1024), d_ones = smem_desc_sw128(sOnes, 16, 1024);
      auto consume_half = [&](int c, uint32_t phi_base, bool first_tile) {
        const uint64_t d_phi = smem_desc_sw128(phi_base, PH_SUB, 1024);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {                            // 16 tokens per step
          const uint64_t ad = smem_desc_advance(d_phi, kk * 2048);
          umma_ss(tmem + T_ACC + c * 128, ad, smem_desc_advance(d_v, kk * 2048), id_st, (!first_tile || kk > 0) ? 1u : 0u);
          umma_ss(tmem + T_Z + c * 16, ad, smem_desc_advance(d_ones, (kk >> 2) * 2048 + (kk & 3) * 32), id_z,
                  (!first_tile || kk > 0) ? 1u : 0u);
        }
      };
      auto run = [&]() {
        for (int j = 0; j < n_tiles; ++j) {
          if (!wait(&bars->x_full, j & 1)) return;
          const bool owe_half1 = j > 0 && nu == 2;                    // phi half 1 of tile j-1 is not yet in the state
          if (owe_half1 && !wait_epi()) return;                       // scratch free: phi half 1 of tile j-1 written
          if (owe_half1 && last_hid == 1) {
            if (!wait(&bars->v_full, (j - 1) & 1)) return;
            consume_half(1, sPhiHalf1, j == 1);
            umma_commit(smem_u32(&bars->v_empty));
          }
          if (!mlp_half(-1, ks1)) return;                             // H[:, 0:128]
          if (owe_half1 && last_hid == 0) {                           // behind the half-GEMM: it runs during that half's epilogue
            if (!wait(&bars->v_full, (j - 1) & 1)) return;
            consume_half(1, sPhiHalf1, j == 1);
            umma_commit(smem_u32(&bars->v_empty));
          }
          if (!wait_epi()) return;
          if (nh == 2 && !mlp_half(-1, ks1)) return;                  // H[:, 128:256]
          // The X tile is free after its last reader: the first layer, or the last GEMMs that read hidden buffer 1.
          if (n_mid == 0) umma_commit(smem_u32(&bars->x_empty));
          if (nh == 2 && !wait_epi()) return;
          for (int m = 0; m < n_mid; ++m) {                           // hidden layer m: buffer m % 2 -> the other
            if (!mlp_half(m & 1, ks2)) return;
            if (!wait_epi()) return;
            if (nh == 2 && !mlp_half(m & 1, ks2)) return;
            if (m == n_mid - 1 && last_hid == 0) umma_commit(smem_u32(&bars->x_empty));
            if (nh == 2 && !wait_epi()) return;
          }
          if (!mlp_half(last_hid, ks2)) return;                       // U[:, 0:128]
          if (!wait_epi()) return;
          if (nu == 2 && !mlp_half(last_hid, ks2)) return;            // U[:, 128:256]
          if (last_hid == 1) umma_commit(smem_u32(&bars->x_empty));
          if (!wait(&bars->v_full, j & 1)) return;
          consume_half(0, sPhiHalf0, j == 0);
          if (nu == 1) umma_commit(smem_u32(&bars->v_empty));         // no second half: V is free once these have run
        }
        if (nu == 2) {
          if (!wait_epi()) return;
          consume_half(1, sPhiHalf1, n_tiles == 1);
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
    // Eight warps: warp w serves TMEM lanes 32*(w%4).. (one token per thread) and the column half
    // w/4 of every 128-column accumulator, so two threads share a token.
    const int qd = warp & 3, ch = warp >> 2;
    const int r = qd * 32 + lane;
    const uint32_t lane_off = (uint32_t)(qd * 32) << 16;
    uint32_t n_acc = 0;
    const int part_w = Dp / (PC ? PC : a.P);                        // RELU: a multiple of 32
    // After a wait has been given up anywhere in the CTA every later wait returns at once.  These warps then run
    // through the rest of the current tile on whatever the accumulators hold (tcgen05.ld needs all 32 lanes, so
    // nothing is skipped lane by lane; every address stays inside the CTA's TMEM and shared memory) and leave
    // at the head of the next tile, where the whole warp looks at the flag together.
    auto aborted = [&]() -> bool { return __any_sync(0xffffffffu, wait_ctx_aborted(wc) != 0); };
    auto wait = [&](uint64_t* bar, uint32_t parity) { mbar_wait(smem_u32(bar), parity, wc, PH_ERR_EPI); };
    bool tok_valid = false;
    // One 128-column half of a layer leaves the scratch accumulator: bias (`bias` points at this half's first
    // column), activation, for the last layer (is_u) the power of its polynomial part, bf16, into columns
    // [64 ch, 64 ch + 64) of the half's destination, the swizzled [128 x 64] sub-tile at dst_sub.
    auto epi_step = [&](const bool is_u, const int half, const float* bias, const uint32_t dst_sub) {
        wait(&bars->acc_ready, n_acc & 1);
        ++n_acc;
        tc_fence_after();
        uint32_t x[2][32];
        tmem_ld32(tmem + lane_off + T_SCR + ch * 64, x[0]);
        tmem_ld32(tmem + lane_off + T_SCR + ch * 64 + 32, x[1]);
        tmem_wait_ld();
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
          const int col0 = ch * 64 + cb * 32;
          uint32_t w[16];                                           // 32 features as bf16 pairs
          if (RELU) {
            const int part = !is_u ? 0 : PC == 1 ? 0 : PC == 2 ? half : (half * 128 + col0) / part_w;   // uniform over the 32 columns
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
              const float4 b4 = *reinterpret_cast<const float4*>(bias + col0 + e);
              float y0, y1, y2, y3;
              upk2(add2(pk2u(x[cb][e], x[cb][e + 1]), pk2(b4.x, b4.y)), y0, y1);
              upk2(add2(pk2u(x[cb][e + 2], x[cb][e + 3]), pk2(b4.z, b4.w)), y2, y3);
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
            if (GEN && is_u) {                                      // parts end anywhere; features beyond D' are zero
#pragma unroll
              for (int e = 0; e < 32; e += 2) {
                const int f0 = half * 128 + col0 + e;
                const float y0 = apply_act(__uint_as_float(x[cb][e]) + bias[col0 + e], act);
                const float y1 = apply_act(__uint_as_float(x[cb][e + 1]) + bias[col0 + e + 1], act);
                w[e >> 1] = pack_bf16(f0 < Dp ? poly_power(y0, f0 / part_w) : 0.f,
                                      f0 + 1 < Dp ? poly_power(y1, (f0 + 1) / part_w) : 0.f);
              }
            } else {
              const int part = is_u ? (half * 128 + col0) / part_w : 0;
#pragma unroll
              for (int e = 0; e < 32; e += 2) {
                float y0 = apply_act(__uint_as_float(x[cb][e]) + bias[col0 + e], act);
                float y1 = apply_act(__uint_as_float(x[cb][e + 1]) + bias[col0 + e + 1], act);
                w[e >> 1] = pack_bf16(poly_power(y0, part), poly_power(y1, part));
              }
            }
          }
          if (is_u && !tok_valid) {
#pragma unroll
            for (int e = 0; e < 16; ++e) w[e] = 0u;
          }
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            const uint4 w4 = make_uint4(w[e >> 1], w[(e >> 1) + 1], w[(e >> 1) + 2], w[(e >> 1) + 3]);
            st_tile_chunk_sw128(dst_sub, PH_SUB, r, cb * 32 + e, w4);
          }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        mbar_arrive_warp(smem_u32(&bars->epi_done), lane);
    };
    for (int j = 0; j < n_tiles; ++j) {
      if (aborted()) break;
      tok_valid = tok_a + j * 128 + r < tok_b;
      // a width of at most 128 has no second half
#pragma unroll
      for (int half = 0; half < 2; ++half)                          // first layer -> hidden buffer 0
        if (half < nh) epi_step(false, half, s_b1 + half * 128, hid_sub(0, half * 2 + ch));
      for (int m = 0; m < n_mid; ++m)                               // hidden layer m -> the buffer it does not read
#pragma unroll
        for (int half = 0; half < 2; ++half)
          if (half < nh) epi_step(false, half, s_b2 + (1 + m) * 256 + half * 128, hid_sub((m & 1) ^ 1, half * 2 + ch));
#pragma unroll
      for (int half = 0; half < 2; ++half)                          // last layer -> the phi tiles
        if (half < nu) epi_step(true, half, s_b2 + half * 128, (half == 0 ? sPhiHalf0 : sPhiHalf1) + ch * PH_SUB);
    }
    wait(&bars->out_ready, 0);
    if (!aborted()) {
      // flush: lane r holds feature c*128 + r of half c; this thread writes its share of the d columns
      tc_fence_after();
      float* base = a.partial + (((size_t)ci * a.n_split + blockIdx.x) * g.BH + bh) * Dp * SD;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        if (c >= nu) continue;
        const bool feat_valid = c * 128 + r < Dp;
        float* dst = base + (size_t)(c * 128 + r) * SD;
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
          const int col = ch * 64 + cb * 32;
          if (col >= ex.d) continue;                                // the same for the whole warp
          uint32_t x[32];
          tmem_ld32(tmem + lane_off + T_ACC + c * 128 + col, x);
          tmem_wait_ld();
          if (feat_valid) {
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              *reinterpret_cast<float4*>(dst + col + e) =
                  make_float4(__uint_as_float(x[e]), __uint_as_float(x[e + 1]), __uint_as_float(x[e + 2]),
                              __uint_as_float(x[e + 3]));
          }
        }
        if (ch == 1) {
          uint32_t zc[16];
          tmem_ld16(tmem + lane_off + T_Z + c * 16, zc);
          tmem_wait_ld();
          if (feat_valid) *reinterpret_cast<float4*>(dst + ex.d) = make_float4(__uint_as_float(zc[0]), 0.f, 0.f, 0.f);
        }
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
