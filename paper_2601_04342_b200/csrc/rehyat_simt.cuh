// SIMT fp32 kernels of the operator: the fp32 mode and the path for shapes the tensor-core
// kernels do not cover.  Inputs are fp32 or bf16 (template T); all arithmetic is fp32.
//
//   state_partial_simt  phi_k on a range of keys and its outer-product sums (Eq. 17-18)
//   scan_states         exclusive running sum of the chunk increments along the chunk axis
//   readout_simt        phi_q on a query tile and phi_q(Q) s_t, phi_q(Q) z_t (Eq. 7, 9, 16)
//   window_simt         softmax window with an online maximum (Eq. 6, 8) + joint normaliser (Eq. 5)
#pragma once

#include "rehyat_common.cuh"

namespace rehyat {

constexpr int SIMT_TM = 32;         // tokens per phi tile
constexpr int SIMT_PHI_THREADS = 512;

struct PhiDims {
  int d, Dh, Dp, P, act_hidden, act_out;
  int n_mid;     // hidden layers between the first and the last (0 for the two-layer map)
};

template <typename T>
struct PhiPtrs {
  const T* W1; const T* b1; const T* W2; const T* b2;   // already offset to the head
  const T* Wm; const T* bm;                             // [n_mid][Dh][Dh], [n_mid][Dh] of the head (n_mid > 0)
};

// Shared memory (floats) of the hidden activations: one [TM][Dh] buffer, two when there are hidden layers in
// between (they alternate as input and output).
__host__ __device__ inline int phi_hidden_floats(int Dh, int n_mid) { return SIMT_TM * Dh * (n_mid > 0 ? 2 : 1); }

// phi of SIMT_TM tokens held in Xs [TM][d] -> Fs [TM][Dp].  Hs (phi_hidden_floats) is scratch.
// `valid` rows carry tokens; the rest of Fs is forced to zero.
template <typename T>
__device__ void phi_tile_simt(const float* Xs, float* Hs, float* Fs, const PhiPtrs<T>& w,
                              const PhiDims& pd, int valid) {
  const int tid = threadIdx.x, NT = blockDim.x;
  constexpr int RG = 4, RPG = SIMT_TM / RG;   // row groups of 8 rows
  // layer 1
  for (int idx = tid; idx < pd.Dh * RG; idx += NT) {
    const int j = idx % pd.Dh, r0 = (idx / pd.Dh) * RPG;
    float acc[RPG];
#pragma unroll
    for (int r = 0; r < RPG; ++r) acc[r] = 0.f;
    const T* wrow = w.W1 + (size_t)j * pd.d;
    for (int k = 0; k < pd.d; k += 4) {
      float4 wv = ld4(wrow + k);
#pragma unroll
      for (int r = 0; r < RPG; ++r) {
        float4 x = *reinterpret_cast<const float4*>(Xs + (r0 + r) * pd.d + k);
        acc[r] = fmaf(x.x, wv.x, acc[r]); acc[r] = fmaf(x.y, wv.y, acc[r]);
        acc[r] = fmaf(x.z, wv.z, acc[r]); acc[r] = fmaf(x.w, wv.w, acc[r]);
      }
    }
    const float b = ldf(w.b1 + j);
#pragma unroll
    for (int r = 0; r < RPG; ++r) Hs[(r0 + r) * pd.Dh + j] = apply_act(acc[r] + b, pd.act_hidden);
  }
  __syncthreads();
  // hidden layers in between: h <- act_hidden(Wm h + bm), the two buffers alternating
  for (int m = 0; m < pd.n_mid; ++m) {
    float* Hn = Hs + ((m & 1) ? 0 : SIMT_TM * pd.Dh);
    const float* Hp = Hs + ((m & 1) ? SIMT_TM * pd.Dh : 0);
    for (int idx = tid; idx < pd.Dh * RG; idx += NT) {
      const int j = idx % pd.Dh, r0 = (idx / pd.Dh) * RPG;
      float acc[RPG];
#pragma unroll
      for (int r = 0; r < RPG; ++r) acc[r] = 0.f;
      const T* wrow = w.Wm + ((size_t)m * pd.Dh + j) * pd.Dh;
      for (int k = 0; k < pd.Dh; k += 4) {
        float4 wv = ld4(wrow + k);
#pragma unroll
        for (int r = 0; r < RPG; ++r) {
          float4 x = *reinterpret_cast<const float4*>(Hp + (r0 + r) * pd.Dh + k);
          acc[r] = fmaf(x.x, wv.x, acc[r]); acc[r] = fmaf(x.y, wv.y, acc[r]);
          acc[r] = fmaf(x.z, wv.z, acc[r]); acc[r] = fmaf(x.w, wv.w, acc[r]);
        }
      }
      const float b = ldf(w.bm + (size_t)m * pd.Dh + j);
#pragma unroll
      for (int r = 0; r < RPG; ++r) Hn[(r0 + r) * pd.Dh + j] = apply_act(acc[r] + b, pd.act_hidden);
    }
    __syncthreads();
  }
  Hs += (pd.n_mid & 1) ? SIMT_TM * pd.Dh : 0;          // where the last hidden activations are
  // last layer + polynomial expansion
  const int part_w = pd.Dp / pd.P;
  for (int idx = tid; idx < pd.Dp * RG; idx += NT) {
    const int j = idx % pd.Dp, r0 = (idx / pd.Dp) * RPG;
    float acc[RPG];
#pragma unroll
    for (int r = 0; r < RPG; ++r) acc[r] = 0.f;
    const T* wrow = w.W2 + (size_t)j * pd.Dh;
    for (int k = 0; k < pd.Dh; k += 4) {
      float4 wv = ld4(wrow + k);
#pragma unroll
      for (int r = 0; r < RPG; ++r) {
        float4 x = *reinterpret_cast<const float4*>(Hs + (r0 + r) * pd.Dh + k);
        acc[r] = fmaf(x.x, wv.x, acc[r]); acc[r] = fmaf(x.y, wv.y, acc[r]);
        acc[r] = fmaf(x.z, wv.z, acc[r]); acc[r] = fmaf(x.w, wv.w, acc[r]);
      }
    }
    const float b = ldf(w.b2 + j);
    const int part = j / part_w;
#pragma unroll
    for (int r = 0; r < RPG; ++r) {
      float u = apply_act(acc[r] + b, pd.act_out);
      Fs[(r0 + r) * pd.Dp + j] = (r0 + r) < valid ? poly_power(u, part) : 0.f;
    }
  }
  __syncthreads();
}

// Loads rows [tok0, tok0+TM) x [0, ncol) of one head into smem as floats (zero beyond tok_end).
template <typename T>
__device__ void load_rows_simt(float* dst, const T* base, long long stride_n, int tok0, int tok_end,
                               int ncol) {
  const int per_row = ncol / 4;
  for (int idx = threadIdx.x; idx < SIMT_TM * per_row; idx += blockDim.x) {
    const int r = idx / per_row, c = (idx % per_row) * 4;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (tok0 + r < tok_end) x = ld4(base + (long long)(tok0 + r) * stride_n + c);
    *reinterpret_cast<float4*>(dst + r * ncol + c) = x;
  }
}

// grid (n_split, G, BH), SIMT_PHI_THREADS threads, dynamic smem TM*(2d + Dp) + phi_hidden_floats floats.
// Chunk t = t0 + blockIdx.y admits the keys [lo_{t-1}, lo_t) into the state (Eq. 17-18: only the
// newly admitted tokens).  Split s takes a contiguous share of them and writes
// partial[blockIdx.y][s][bh] = sum_j phi_k(k_j) [v_j | 1]  as [Dp][SD] floats, SD = d + 4,
// column d holding the z part.
template <typename T, int D>
__global__ void __launch_bounds__(SIMT_PHI_THREADS)
state_partial_simt(const T* __restrict__ k, const T* __restrict__ v, PhiPtrs<T> wk, PhiDims pd, Geo g,
                   int n_split, float* __restrict__ partial) {
  extern __shared__ __align__(16) float smem[];
  constexpr int SD = D + 4;
  float* Xs = smem;
  float* Vs = Xs + SIMT_TM * D;
  float* Hs = Vs + SIMT_TM * D;
  float* Fs = Hs + phi_hidden_floats(pd.Dh, pd.n_mid);

  const int s = blockIdx.x, ci = blockIdx.y, bh = blockIdx.z, t = g.t0 + ci;
  const int head = bh % g.n_heads;
  const int lo_prev = t > 0 ? geo_lo(g, t - 1) : 0, lo = geo_lo(g, t);
  const int len = lo - lo_prev;
  int per = (len + n_split - 1) / n_split;
  per = (per + SIMT_TM - 1) / SIMT_TM * SIMT_TM;
  const int a = min(lo_prev + s * per, lo), b = min(a + per, lo);

  PhiPtrs<T> w = {wk.W1 + (size_t)head * pd.Dh * D, wk.b1 + (size_t)head * pd.Dh,
                  wk.W2 + (size_t)head * pd.Dp * pd.Dh, wk.b2 + (size_t)head * pd.Dp,
                  pd.n_mid ? wk.Wm + (size_t)head * pd.n_mid * pd.Dh * pd.Dh : nullptr,
                  pd.n_mid ? wk.bm + (size_t)head * pd.n_mid * pd.Dh : nullptr};
  const long long hoff = head_offset(g, bh);

  // thread -> (feature f, half of the value columns)
  const int f = threadIdx.x % 256, half = threadIdx.x / 256;
  constexpr int HC = D / 2;
  float acc[HC];
  float zacc = 0.f;
#pragma unroll
  for (int c = 0; c < HC; ++c) acc[c] = 0.f;

  for (int tok0 = a; tok0 < b; tok0 += SIMT_TM) {
    load_rows_simt(Xs, k + hoff, g.stride_n, tok0, b, D);
    load_rows_simt(Vs, v + hoff, g.stride_n, tok0, b, D);
    __syncthreads();
    phi_tile_simt(Xs, Hs, Fs, w, pd, b - tok0);
    if (f < pd.Dp) {
      for (int r = 0; r < SIMT_TM; ++r) {
        const float fv = Fs[r * pd.Dp + f];
        zacc += fv;
        const float* vr = Vs + r * D + half * HC;
#pragma unroll
        for (int c = 0; c < HC; c += 4) {
          float4 x = *reinterpret_cast<const float4*>(vr + c);
          acc[c] = fmaf(fv, x.x, acc[c]); acc[c + 1] = fmaf(fv, x.y, acc[c + 1]);
          acc[c + 2] = fmaf(fv, x.z, acc[c + 2]); acc[c + 3] = fmaf(fv, x.w, acc[c + 3]);
        }
      }
    }
    __syncthreads();
  }
  if (f < pd.Dp) {
    float* dst = partial + (((size_t)ci * n_split + s) * g.BH + bh) * pd.Dp * SD + (size_t)f * SD;
#pragma unroll
    for (int c = 0; c < HC; c += 4)
      *reinterpret_cast<float4*>(dst + half * HC + c) = make_float4(acc[c], acc[c + 1], acc[c + 2], acc[c + 3]);
    if (half == 1) *reinterpret_cast<float4*>(dst + D) = make_float4(zacc, 0.f, 0.f, 0.f);
  }
}

// state[i] = carry + sum_{u<=i} sum_s partial[u][s]   for the G chunks of the group, where carry
// is the state of the chunk before the group (slot `carry_slot`, or zero: s_0 = z_0 = 0, Eq. 14-15).
// One thread per state element; the chunk axis is walked in order, splits in fixed order, so the
// result does not depend on scheduling.
__global__ void scan_states(const float* __restrict__ partial, float* __restrict__ state,
                            size_t per_slot, int G, int n_split, int carry_slot,
                            __nv_bfloat16* __restrict__ state_bf16 = nullptr, int D = 0) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= per_slot) return;
  float run = carry_slot >= 0 ? state[(size_t)carry_slot * per_slot + e] : 0.f;
  // optional bf16 copy of the s part, [slot][bh][feature][D], the B operand of the tensor-core read-out
  const size_t row = e / (D + 4), col = e % (D + 4);
  const size_t per_slot_b = per_slot / (D + 4) * D;
  for (int i = 0; i < G; ++i) {
    float inc = 0.f;
    for (int s = 0; s < n_split; ++s) inc += partial[((size_t)i * n_split + s) * per_slot + e];
    run += inc;
    state[(size_t)i * per_slot + e] = run;
    if (state_bf16 != nullptr && col < (size_t)D) state_bf16[(size_t)i * per_slot_b + row * D + col] = __float2bfloat16_rn(run);
  }
}

// Bidirectional linear sets (Eq. 10-12): TL_t = [0, lo_t) + [hi_t, N).  `cum[f]` is the state summed over the
// frames before frame f (cum[0] = 0, cum[T] = all tokens), so the state of chunk t is
// cum[lo_t / HW] + (cum[T] - cum[hi_t / HW]).  One thread per state element, written into the slots the
// read-out uses (plus the bf16 copy of the s part for the tensor-core read-out).
__global__ void combine_bidirectional(const float* __restrict__ cum, float* __restrict__ state, size_t per_slot, Geo g,
                                      int HW, int T, __nv_bfloat16* __restrict__ state_bf16 = nullptr, int D = 0) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= per_slot) return;
  const size_t row = e / (D + 4), col = e % (D + 4);
  const size_t per_slot_b = per_slot / (D + 4) * D;
  const float total = cum[(size_t)T * per_slot + e];
  for (int i = 0; i < g.G; ++i) {
    const int t = g.t0 + i, lo_f = geo_lo(g, t) / HW, hi_f = geo_q1(g, t) / HW;
    const float sv = cum[(size_t)lo_f * per_slot + e] + (total - cum[(size_t)hi_f * per_slot + e]);
    state[(size_t)i * per_slot + e] = sv;
    if (state_bf16 != nullptr && col < (size_t)D) state_bf16[(size_t)i * per_slot_b + row * D + col] = __float2bfloat16_rn(sv);
  }
}

// grid (tiles per chunk, G, BH), SIMT_PHI_THREADS threads.  Linear read-out of one tile of
// SIMT_TM queries of chunk t: rd[bh][row in group][0..d) = phi_q(q_i) s_t, [d] = phi_q(q_i) z_t, in the fp32
// layout of rd_index or (rd_half, for the tensor-core window kernels) as fp16 ratios in the layout of rdh_index.
template <typename T, int D>
__global__ void __launch_bounds__(SIMT_PHI_THREADS)
readout_simt(const T* __restrict__ q, PhiPtrs<T> wq, PhiDims pd, Geo g, const float* __restrict__ state,
             float* __restrict__ rd, int rd_rows, int rd_half) {
  extern __shared__ __align__(16) float smem[];
  constexpr int SD = D + 4;
  float* Xs = smem;
  float* Hs = Xs + SIMT_TM * D;
  float* Fs = Hs + phi_hidden_floats(pd.Dh, pd.n_mid);

  const int ci = blockIdx.y, bh = blockIdx.z, t = g.t0 + ci;
  if (!geo_linear(g, t)) return;                       // empty linear set: nothing to read out
  const int q0 = geo_q0(g, t), q1 = geo_q1(g, t);
  const int tok0 = q0 + blockIdx.x * SIMT_TM;
  if (tok0 >= q1) return;
  const int head = bh % g.n_heads;
  PhiPtrs<T> w = {wq.W1 + (size_t)head * pd.Dh * D, wq.b1 + (size_t)head * pd.Dh,
                  wq.W2 + (size_t)head * pd.Dp * pd.Dh, wq.b2 + (size_t)head * pd.Dp,
                  pd.n_mid ? wq.Wm + (size_t)head * pd.n_mid * pd.Dh * pd.Dh : nullptr,
                  pd.n_mid ? wq.bm + (size_t)head * pd.n_mid * pd.Dh : nullptr};
  load_rows_simt(Xs, q + q_row_offset(g, bh, 0), g.qstride_n, tok0, q1, D);
  __syncthreads();
  phi_tile_simt(Xs, Hs, Fs, w, pd, q1 - tok0);

  const float* S = state + ((size_t)ci * g.BH + bh) * pd.Dp * SD;
  constexpr int RG = 4, RPG = SIMT_TM / RG;
  float* nl_s = Xs;                                    // phi_q(q_i) z_t of the tile's rows (Xs is no longer needed)
  if (rd_half) {
    // the tensor-core window kernels read the ratio aL / nL (see rdh_index): the denominators come first
    for (int r = threadIdx.x; r < SIMT_TM; r += blockDim.x) {
      float acc = 0.f;
      for (int ff = 0; ff < pd.Dp; ++ff) acc = fmaf(Fs[r * pd.Dp + ff], S[(size_t)ff * SD + D], acc);
      nl_s[r] = acc;
      if (tok0 + r < q1) rd[rdh_index(g, rd_rows, D, bh, ci, tok0 + r - q0, rdh_pieces(D) - 1) * 4] = acc;
    }
    __syncthreads();
  }
  const int ncol = rd_half ? D : D + 1;
  for (int idx = threadIdx.x; idx < ncol * RG; idx += blockDim.x) {
    const int c = idx % ncol, r0 = (idx / ncol) * RPG;
    float acc[RPG];
#pragma unroll
    for (int r = 0; r < RPG; ++r) acc[r] = 0.f;
    for (int ff = 0; ff < pd.Dp; ++ff) {
      const float sv = S[(size_t)ff * SD + c];
#pragma unroll
      for (int r = 0; r < RPG; ++r) acc[r] = fmaf(Fs[(r0 + r) * pd.Dp + ff], sv, acc[r]);
    }
#pragma unroll
    for (int r = 0; r < RPG; ++r) {
      const int tok = tok0 + r0 + r;
      if (tok >= q1) continue;
      if (!rd_half) {
        rd[rd_index(g, rd_rows, D, bh, ci, tok - q0, c >> 2) + (c & 3)] = acc[r];
      } else {
        const float nl = nl_s[r0 + r], ratio = nl != 0.f ? acc[r] / nl : 0.f;
        reinterpret_cast<__half*>(rd)[rdh_index(g, rd_rows, D, bh, ci, tok - q0, c >> 3) * 8 + (c & 7)] =
            __float2half_rn(fminf(fmaxf(ratio, -65504.f), 65504.f));
      }
    }
  }
}

// What a DiT block does to q and k before the attention operator (the block of Eq. 1 around A_l): per-head RMS
// normalisation x / sqrt(mean(x^2) + eps) * weight, then the rotary embedding with caller-supplied tables (the
// pair (x[2i], x[2i+1]) of token n turned by the angle of cos[n][i], sin[n][i]).  One pass over q and k, bound by
// HBM: every element is read once and written once, in the layout it came in.
// grid (row blocks, BH, 2: q / k), 256 threads; a row of d elements is shared by d/8 lanes, eight elements each.
struct QkPrepArgs {
  const void* wq; const void* wk;       // [n_heads][d] in the operator dtype, or null
  const float* cos; const float* sin;   // [positions][d/2], or null
  float eps;
  int rms_norm;
  int rows, n_heads;                    // token rows per (batch, head), heads
  int pos0;                             // position of row 0 in the rotation tables (tokens of earlier chunks)
  long long sb, sh, sn;                 // element strides of the sources (q and k share them)
  long long qb, qh, qn;                 // ... of the transformed q
  long long kb, kh, kn;                 // ... of the transformed k
};
template <typename T, int D>
__global__ void __launch_bounds__(256)
qk_prepare(const T* __restrict__ q, const T* __restrict__ k, T* __restrict__ qo, T* __restrict__ ko, QkPrepArgs a) {
  constexpr int LPR = D / 8;                                        // lanes per row
  const T* __restrict__ src = blockIdx.z ? k : q;
  T* __restrict__ dst = blockIdx.z ? ko : qo;
  const T* __restrict__ wgt = static_cast<const T*>(blockIdx.z ? a.wk : a.wq);
  const int bh = blockIdx.y, head = bh % a.n_heads, bat = bh / a.n_heads;
  const long long hoff = (long long)bat * a.sb + (long long)head * a.sh;
  const long long doff = blockIdx.z ? (long long)bat * a.kb + (long long)head * a.kh : (long long)bat * a.qb + (long long)head * a.qh;
  const long long dn = blockIdx.z ? a.kn : a.qn;
  const int lane_in_row = threadIdx.x % LPR, col = lane_in_row * 8;
  const int rows_per_block = 256 / LPR;
  // a thread keeps its eight columns for all its rows: their norm weights are loaded once
  float wv[8] = {1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f};
  if (a.rms_norm && wgt != nullptr) {
    const float4 w0 = ld4(wgt + (size_t)head * D + col), w1 = ld4(wgt + (size_t)head * D + col + 4);
    wv[0] = w0.x; wv[1] = w0.y; wv[2] = w0.z; wv[3] = w0.w; wv[4] = w1.x; wv[5] = w1.y; wv[6] = w1.z; wv[7] = w1.w;
  }
  // the lanes that share a row reduce among themselves: row groups of one warp may leave the loop at different times
  const unsigned row_lanes = (LPR >= 32 ? 0xffffffffu : ((1u << LPR) - 1u) << ((threadIdx.x & 31) / LPR * LPR));
  // two rows per step, both loaded before either is worked on: twice the bytes in flight per thread
  const int stride = gridDim.x * rows_per_block;
  const int first = blockIdx.x * rows_per_block + threadIdx.x / LPR;
  // the addresses of a thread's rows advance by constants: pointers of the first of the two rows, stepped per turn
  const T* sp = src + hoff + (long long)first * a.sn + col;
  T* dp = dst + doff + (long long)first * dn + col;
  const float* cp = a.cos != nullptr ? a.cos + (size_t)(a.pos0 + first) * (D / 2) + col / 2 : nullptr;
  const float* np_ = a.cos != nullptr ? a.sin + (size_t)(a.pos0 + first) * (D / 2) + col / 2 : nullptr;
  const long long s_row = (long long)stride * a.sn, d_row = (long long)stride * dn;       // one row group further
  const size_t t_row = (size_t)stride * (D / 2);
  for (int row0 = first; row0 < a.rows; row0 += 2 * stride, sp += 2 * s_row, dp += 2 * d_row, cp += 2 * t_row, np_ += 2 * t_row) {
    float x[2][8];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int row = row0 + u * stride;
      if (row < a.rows) {
        const T* p = sp + u * s_row;
        const float4 x0 = ld4(p), x1 = ld4(p + 4);
        x[u][0] = x0.x; x[u][1] = x0.y; x[u][2] = x0.z; x[u][3] = x0.w;
        x[u][4] = x1.x; x[u][5] = x1.y; x[u][6] = x1.z; x[u][7] = x1.w;
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) x[u][e] = 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int row = row0 + u * stride;                 // rows beyond the end take part in the shuffles, nothing else
      if (a.rms_norm) {
        float ss = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) ss = fmaf(x[u][e], x[u][e], ss);
#pragma unroll
        for (int o = 1; o < LPR; o <<= 1) ss += __shfl_xor_sync(row_lanes, ss, o);
        const float inv = rsqrtf(ss * (1.f / D) + a.eps);
#pragma unroll
        for (int e = 0; e < 8; ++e) x[u][e] *= inv * wv[e];
      }
      if (row >= a.rows) continue;
      if (a.cos != nullptr) {
        const float4 c = *reinterpret_cast<const float4*>(cp + u * t_row);
        const float4 s = *reinterpret_cast<const float4*>(np_ + u * t_row);
        const float cs[4] = {c.x, c.y, c.z, c.w}, sn[4] = {s.x, s.y, s.z, s.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float p0 = x[u][2 * e], p1 = x[u][2 * e + 1];
          x[u][2 * e] = p0 * cs[e] - p1 * sn[e];
          x[u][2 * e + 1] = p0 * sn[e] + p1 * cs[e];
        }
      }
      st8(dp + u * d_row, x[u]);
    }
  }
}

// grid (tiles per chunk of WIN_BM rows, G, BH), 128 threads.  Softmax window of Eq. 6 and 8 with a
// running row maximum, then the joint normalisation of Eq. 5 with the linear read-out `rd`.
constexpr int WIN_BM = 32, WIN_BN = 64, WIN_THREADS = 128;

template <typename T, int D>
__global__ void __launch_bounds__(WIN_THREADS)
window_simt(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, T* __restrict__ out,
            Geo g, const float* __restrict__ rd, int rd_rows, float scale, int c_mode, float* __restrict__ share) {
  extern __shared__ __align__(16) float smem[];
  constexpr int LDK = D + 4, LDP = WIN_BN + 4;
  constexpr int DC = D / 16;                 // output columns per thread
  float* Qs = smem;                          // [BM][LDK]
  float* Ks = Qs + WIN_BM * LDK;             // [BN][LDK]
  float* Vs = Ks + WIN_BN * LDK;             // [BN][D]
  float* Ps = Vs + WIN_BN * D;               // [BM][LDP]

  const int ci = blockIdx.y, bh = blockIdx.z, t = g.t0 + ci;
  const int q0 = geo_q0(g, t), q1 = geo_q1(g, t), lo = geo_lo(g, t), hi = q1;
  const bool linear = geo_linear(g, t);
  const int row0 = q0 + blockIdx.x * WIN_BM;
  if (row0 >= q1) return;
  const long long hoff = head_offset(g, bh);
  const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;

  for (int idx = tid; idx < WIN_BM * (D / 4); idx += WIN_THREADS) {
    const int r = idx / (D / 4), c = (idx % (D / 4)) * 4;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row0 + r < q1) x = ld4(q + q_row_offset(g, bh, row0 + r) + c);
    *reinterpret_cast<float4*>(Qs + r * LDK + c) = x;
  }

  float m[4], l[4], acc[4][DC];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m[i] = -INFINITY; l[i] = 0.f;
#pragma unroll
    for (int c = 0; c < DC; ++c) acc[i][c] = 0.f;
  }

  for (int j0 = lo; j0 < hi; j0 += WIN_BN) {
    __syncthreads();
    for (int idx = tid; idx < WIN_BN * (D / 4); idx += WIN_THREADS) {
      const int r = idx / (D / 4), c = (idx % (D / 4)) * 4;
      float4 kk = make_float4(0.f, 0.f, 0.f, 0.f), vv = kk;
      if (j0 + r < hi) {
        kk = ld4(k + hoff + (long long)(j0 + r) * g.stride_n + c);
        vv = ld4(v + hoff + (long long)(j0 + r) * g.stride_n + c);
      }
      *reinterpret_cast<float4*>(Ks + r * LDK + c) = kk;
      *reinterpret_cast<float4*>(Vs + r * D + c) = vv;
    }
    __syncthreads();
    // scaled logits of rows ty*4+i, columns tx + 16*jj
    float sv[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) sv[i][jj] = 0.f;
    for (int kk = 0; kk < D; kk += 4) {
      float4 qa[4], kb[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) qa[i] = *reinterpret_cast<const float4*>(Qs + (ty * 4 + i) * LDK + kk);
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) kb[jj] = *reinterpret_cast<const float4*>(Ks + (tx + 16 * jj) * LDK + kk);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          sv[i][jj] = fmaf(qa[i].x, kb[jj].x, sv[i][jj]); sv[i][jj] = fmaf(qa[i].y, kb[jj].y, sv[i][jj]);
          sv[i][jj] = fmaf(qa[i].z, kb[jj].z, sv[i][jj]); sv[i][jj] = fmaf(qa[i].w, kb[jj].w, sv[i][jj]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float tmax = -INFINITY;
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        sv[i][jj] = (j0 + tx + 16 * jj < hi) ? sv[i][jj] * scale : -INFINITY;
        tmax = fmaxf(tmax, sv[i][jj]);
      }
#pragma unroll
      for (int o = 1; o < 16; o <<= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
      const float m_new = fmaxf(m[i], tmax);          // finite: every tile has a valid column
      const float alpha = expf(m[i] - m_new);         // exp(-inf) = 0 on the first tile
      float psum = 0.f;
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const float p = expf(sv[i][jj] - m_new);
        psum += p;
        Ps[(ty * 4 + i) * LDP + tx + 16 * jj] = p;
      }
#pragma unroll
      for (int o = 1; o < 16; o <<= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
      l[i] = l[i] * alpha + psum;
      m[i] = m_new;
#pragma unroll
      for (int c = 0; c < DC; ++c) acc[i][c] *= alpha;
    }
    __syncthreads();
    for (int j = 0; j < WIN_BN; ++j) {
      float vv[DC];
#pragma unroll
      for (int c = 0; c < DC; c += 4) {
        float4 x = *reinterpret_cast<const float4*>(Vs + j * D + tx * DC + c);
        vv[c] = x.x; vv[c + 1] = x.y; vv[c + 2] = x.z; vv[c + 3] = x.w;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float p = Ps[(ty * 4 + i) * LDP + j];
#pragma unroll
        for (int c = 0; c < DC; ++c) acc[i][c] = fmaf(p, vv[c], acc[i][c]);
      }
    }
  }

  // Eq. 5: the window sums are relative to c_i = final row maximum m_i.  ROWMAX: the linear terms
  // enter unscaled.  ZERO (c = 0): window terms carry exp(m_i), evaluated stably by measuring both
  // branches against r = max(m_i, 0): window * exp(m_i - r), linear * exp(-r).
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = row0 + ty * 4 + i;
    if (row >= q1) continue;
    float ws = 1.f, lam = 0.f, nL = 0.f;
    if (linear) {
      lam = 1.f;
      if (c_mode == C_ZERO) {
        const float r = fmaxf(m[i], 0.f);
        ws = expf(m[i] - r);
        lam = expf(-r);
      }
      nL = rd[rd_index(g, rd_rows, D, bh, ci, row - q0, D / 4)];
    }
    const float inv = 1.f / (l[i] * ws + lam * nL);
    if (share != nullptr && tx == 0) share[(size_t)bh * g.N + row] = lam * nL * inv;   // part of the normaliser that is linear
    T* orow = out + out_row_offset(g, bh, row) + tx * DC;
#pragma unroll
    for (int c = 0; c < DC; ++c) {
      const float aL = linear ? rd[rd_index(g, rd_rows, D, bh, ci, row - q0, (tx * DC + c) >> 2) + ((tx * DC + c) & 3)] : 0.f;
      stf(orow + c, (acc[i][c] * ws + lam * aL) * inv);
    }
  }
}

}  // namespace rehyat
