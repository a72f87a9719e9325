// Shared device-side definitions of the ReHyAt kernels: geometry of one chunk group, element
// load/store helpers, the phi activations.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rehyat {

// Activations of the phi MLP (same numbering as rehyat_act in the public header).
enum Act : int { ACT_RELU = 0, ACT_IDENTITY = 1, ACT_SOFTPLUS = 2, ACT_ELU1 = 3, ACT_GELU = 4 };
enum CMode : int { C_ROWMAX = 0, C_ZERO = 1 };

// Everything a kernel needs to find chunk t = t0 + (chunk index inside the group).
// Chunk t (Section 3.3, Eq. 13): queries [q0_t, q1_t) = [t*Np + q_shift, min((t+1)*Np + q_shift, N)), softmax
// window [lo_t, q1_t), lo_t = max(q0_t - ToHW, 0); linear prefix [0, lo_t) plus, when `prefix` is set, tokens
// that are no longer in the buffers and live only in the carried state (the chunk-by-chunk entry points).
struct Geo {
  int N;        // tokens per (batch, head) in the buffers
  int Np;       // tokens per chunk, chunk*H*W
  int ToHW;     // overlap*H*W (clamped to N by the host so that it cannot overflow)
  int t0;       // first chunk of the group
  int G;        // chunks in the group
  int n_heads;
  int BH;       // batch * n_heads
  long long stride_b, stride_h, stride_n;   // element strides of k and v
  int q_shift;  // buffer index of the first query of chunk 0 (0 for a whole sequence)
  int prefix;   // 1: the carried state of chunk t0 covers tokens before buffer index 0
  // q and out may live in tensors of their own (a chunk-by-chunk step reads the caller's chunk in place while k
  // and v sit behind the kept overlap frames): row r of the k / v buffers is row r - q_off of q and out, which
  // have Nq rows and their own strides.  A whole-sequence call has q_off = 0, Nq = N and the strides of k, v.
  long long qstride_b, qstride_h, qstride_n;
  int q_off, Nq;
  long long ostride_b, ostride_h, ostride_n;   // out: the rows of q, strides of its own (a step may read a transformed copy of q)
};

__host__ __device__ inline int geo_q0(const Geo& g, int t) { return t * g.Np + g.q_shift; }
__host__ __device__ inline int geo_q1(const Geo& g, int t) {
  long long e = (long long)(t + 1) * g.Np + g.q_shift;
  return e < g.N ? (int)e : g.N;
}
__host__ __device__ inline int geo_lo(const Geo& g, int t) {
  long long a = (long long)t * g.Np + g.q_shift - g.ToHW;
  return a > 0 ? (int)a : 0;
}
// Does chunk t have a non-empty linear set TL_t?
__host__ __device__ inline bool geo_linear(const Geo& g, int t) { return geo_lo(g, t) > 0 || g.prefix != 0; }

// Linear read-out workspace (phi_q(q_i) s_t in columns [0, d), phi_q(q_i) z_t in column d).  Per (batch*head)
// it is cut into tiles of 128 query rows - tile k of chunk ci of the group has index ci*ceil(Np/128) + k - and a
// tile into d/4 + 1 pieces of four columns, each piece holding the tile's 128 rows contiguously (16 bytes per row).
// Threads that own consecutive rows therefore read and write consecutive 16-byte pieces.  `rd_rows` is the row
// capacity per (batch*head), a multiple of 128.  Returns the float index of piece `c4` of the row.
__host__ __device__ inline size_t rd_index(const Geo& g, int rd_rows, int d, int bh, int ci, int row_in_chunk, int c4) {
  const int tiles = (g.Np + 127) >> 7;
  const size_t tile = (size_t)bh * (size_t)(rd_rows >> 7) + (size_t)ci * tiles + (size_t)(row_in_chunk >> 7);
  return ((tile * (size_t)(d / 4 + 1) + (size_t)c4) * 128 + (size_t)(row_in_chunk & 127)) * 4;
}

// The same workspace as the tensor-core kernels keep it (bf16 operator, head_dim 128): nL_i = phi_q(q_i) z_t in
// fp32 and the d columns of the RATIO aL_i / nL_i = phi_q(q_i) s_t / nL_i in fp16, eight to a 16-byte piece:
// rdh_pieces(d) = d/8 + 1 pieces per 128-row tile (the last one holds nL in its first word), each with the tile's rows
// contiguous.  For non-negative features the ratio is a weighted mean of the v_j, so it fits fp16 whatever the
// size of the sums, and its rounding (2^-11 relative) is below the bf16 rounding of the output; a ratio beyond the
// fp16 range (features of both signs, nL near zero: Eq. 5 is then indefinite anyway) is clamped.  The workspace
// and the traffic between the read-out and the window kernel are half of the fp32 form.  Returns the index of
// the 16-byte piece `piece` of the row.
__host__ __device__ constexpr int rdh_pieces(int d) { return d / 8 + 1; }
__host__ __device__ inline size_t rdh_index(const Geo& g, int rd_rows, int d, int bh, int ci, int row_in_chunk, int piece) {
  const int tiles = (g.Np + 127) >> 7;
  const size_t tile = (size_t)bh * (size_t)(rd_rows >> 7) + (size_t)ci * tiles + (size_t)(row_in_chunk >> 7);
  return (tile * (size_t)rdh_pieces(d) + (size_t)piece) * 128 + (size_t)(row_in_chunk & 127);
}

// Packs two ratios (see rdh_index) into one fp16 pair, clamped to the finite fp16 range.
__device__ __forceinline__ uint32_t pack_ratio_f16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float2 unpack_f16(uint32_t pair) {
  return __half22float2(*reinterpret_cast<const __half2*>(&pair));
}

__device__ __forceinline__ long long head_offset(const Geo& g, int bh) {
  return (long long)(bh / g.n_heads) * g.stride_b + (long long)(bh % g.n_heads) * g.stride_h;
}
// Element offset of buffer row `row` (a query row) of (batch*head) bh inside q, and inside out.
__device__ __forceinline__ long long q_row_offset(const Geo& g, int bh, int row) {
  return (long long)(bh / g.n_heads) * g.qstride_b + (long long)(bh % g.n_heads) * g.qstride_h +
         (long long)(row - g.q_off) * g.qstride_n;
}
__device__ __forceinline__ long long out_row_offset(const Geo& g, int bh, int row) {
  return (long long)(bh / g.n_heads) * g.ostride_b + (long long)(bh % g.n_heads) * g.ostride_h +
         (long long)(row - g.q_off) * g.ostride_n;
}

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float x) { *p = x; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// Four consecutive elements as floats (pointer must be aligned to four elements).
__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 ld4(const __nv_bfloat16* p) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
  float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}

// Eight consecutive elements from floats (pointer aligned to eight elements).
__device__ __forceinline__ void st8(float* p, const float (&x)[8]) {
  *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(x[4], x[5], x[6], x[7]);
}
__device__ __forceinline__ void st8(__nv_bfloat16* p, const float (&x)[8]) {
  __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]), b = __floats2bfloat162_rn(x[2], x[3]);
  __nv_bfloat162 c = __floats2bfloat162_rn(x[4], x[5]), d = __floats2bfloat162_rn(x[6], x[7]);
  *reinterpret_cast<uint4*>(p) = make_uint4(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b),
                                            *reinterpret_cast<uint32_t*>(&c), *reinterpret_cast<uint32_t*>(&d));
}

__device__ __forceinline__ float apply_act(float x, int act) {
  switch (act) {
    case ACT_RELU: return fmaxf(x, 0.f);
    case ACT_IDENTITY: return x;
    case ACT_SOFTPLUS: return x > 20.f ? x : log1pf(expf(x));
    case ACT_ELU1: return x > 0.f ? x + 1.f : expf(x);
    default: return 0.5f * x * (1.f + erff(x * 0.70710678118654752f));
  }
}

// Element-wise power of the polynomial expansion: output feature j of D' belongs to part
// j / (D'/P) (0-based) and is raised to that index plus one.
__device__ __forceinline__ float poly_power(float u, int part) {
  float r = u;
  for (int i = 0; i < part; ++i) r *= u;
  return r;
}

}  // namespace rehyat
