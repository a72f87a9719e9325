// Host side of the C ABI declared in include/rehyat.h: argument validation, the fixed
// workspace, the chunk-group schedule and the kernel launches.
//
// Schedule of one forward call.  The T' chunks are walked in groups of G consecutive chunks
// (G*N' <= the read-out rows the workspace holds), so the workspace does not grow with the
// number of frames (Section 3.3, note 3).  Per group:
//   1. state increments: sum of phi_k(k_j)[v_j|1] over the keys each chunk newly admits (Eq. 17-18)
//   2. scan along the chunk axis, carrying the last state of the previous group (Eq. 14-15)
//   3. linear read-out phi_q(Q_t) s_t, phi_q(Q_t) z_t of the group's queries (Eq. 7, 9, 16)
//   4. softmax window (Eq. 6, 8) and the joint normalisation (Eq. 5), writing y.
#include <cuda_runtime.h>

#include <climits>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/rehyat.h"
#include "rehyat_common.cuh"
#include "rehyat_simt.cuh"
#include "rehyat_tc.cuh"
#include "rehyat_tc_single.cuh"

using namespace rehyat;

// Optional per-kernel timing: CUDA events recorded on the launching stream around every launch
// of each kernel kind, summed when read.
struct Profiler {
  bool on = false;
  std::vector<cudaEvent_t> ev[REHYAT_PROF_KINDS];   // begin/end pairs
  void begin(int kind, cudaStream_t st) {
    if (!on) return;
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    cudaEventRecord(e, st);
    ev[kind].push_back(e);
  }
  void end(int kind, cudaStream_t st) { begin(kind, st); }
  void clear() {
    for (auto& v : ev) { for (cudaEvent_t e : v) cudaEventDestroy(e); v.clear(); }
  }
};

struct rehyat_ctx {
  rehyat_config cfg;
  Profiler prof;
  float* state = nullptr;      // [Gmax][BHmax][Dp][d+4]
  float* partial = nullptr;    // [partial_units][BHmax][Dp][d+4]
  float* readout = nullptr;    // linear read-out of one chunk group, rd_cap rows per (batch, head), laid out by rd_index
  int* status_dev = nullptr;
  float* cum = nullptr;        // bidirectional mode: [frames + 1][BHmax][Dp][d+4] states summed over whole frames
  int cum_frames = 0;
  TcWorkspace tc;              // extra buffers of the tensor-core path
  size_t ws_bytes = 0;
  int Gmax = 0, partial_units = 0, rd_rows = 0, rd_cap = 0, bh_max = 0;
  void* stage[4] = {nullptr, nullptr, nullptr, nullptr};
  size_t stage_bytes = 0;
  cudaStream_t copy_in = nullptr, copy_out = nullptr;   // rehyat_forward_host: copies overlap the kernels
  std::vector<cudaEvent_t> host_events;
  int head_count = 0;          // > 0: rehyat_forward works on this many heads (pointers already offset to the first)
  int last_launches = 0, last_impl = 0;
  bool tensor_ok = false;
  int epoch = 0;               // number of the last tensor-core launch, 1, 2, ... (see ptx::WaitCtx)
  unsigned wait_limit_us = 1000000u;   // bound of every device-side wait
  int withhold_loads = 0;      // test hook of rehyat_set_wait_limit
  void* qprep = nullptr;       // q and k after rehyat_set_qk_transform (cfg.qk_transform), same layout as the inputs
  void* kprep = nullptr;
  size_t prep_elems = 0;       // elements each of the two holds
  bool qk_on = false;
  rehyat_qk_transform qk = {};
  float* share_out = nullptr;  // rehyat_set_linear_share_output
  float* share_now = nullptr;  // what the window launches of the call in progress write (null in chunk-by-chunk steps)
  // chunk-by-chunk processing (rehyat_stream_*): the running state lives in slot 0 of `state`; k and v of the
  // softmax window (the kept overlap frames, then the chunk being processed) sit in two buffers
  // [BH][cap_tokens][d] at token index `start`.  Every step appends its chunk behind the window and moves
  // `start` past the tokens that leave it; only when the end of the buffers is reached are the kept frames
  // copied back to the front.  q and out are used in place.
  struct Stream {
    bool active = false;
    int batch = 0, H = 0, W = 0, chunk = 0, overlap = 0;
    int halo = 0;                 // tokens of earlier chunks still inside the softmax window
    int has_state = 0;            // the running state covers at least one token
    long long chunks_done = 0;
    int cap_tokens = 0;           // tokens per (batch, head) each buffer holds
    int start = 0;                // token index of the window's first token
    long long tokens_done = 0;    // tokens per (batch, head) of the chunks processed so far (position of the next chunk)
    void* kbuf = nullptr;
    void* vbuf = nullptr;
    void* qbuf = nullptr;         // the chunk's q after the q/k transform (contexts made with qk_transform only)
    int chunk_cap = 0;            // tokens per (batch, head) qbuf holds
    size_t bytes = 0;
  } stream;
};

namespace {

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

inline size_t elem_size(int dtype) { return dtype == REHYAT_DTYPE_FP32 ? 4 : 2; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_config(const rehyat_config* c) {
  if (c->dtype != REHYAT_DTYPE_BF16 && c->dtype != REHYAT_DTYPE_FP32) return REHYAT_ERR_INVALID_ARG;
  if (c->n_heads < 1 || c->n_heads > 1024) return REHYAT_ERR_INVALID_ARG;
  if (c->max_batch < 1 || (long long)c->max_batch * c->n_heads > 65535) return REHYAT_ERR_INVALID_ARG;
  if (c->poly_degree < 1 || c->poly_degree > 4) return REHYAT_ERR_INVALID_ARG;
  if (c->phi_hidden < 8 || c->phi_hidden > 256 || c->phi_hidden % 8) return REHYAT_ERR_INVALID_ARG;
  if (c->phi_dim < 8 || c->phi_dim > 256 || c->phi_dim % 8 || c->phi_dim % c->poly_degree)
    return REHYAT_ERR_INVALID_ARG;
  if (c->act_hidden < 0 || c->act_hidden > 4 || c->act_out < 0 || c->act_out > 4) return REHYAT_ERR_INVALID_ARG;
  if (c->c_mode != REHYAT_C_ROWMAX && c->c_mode != REHYAT_C_ZERO) return REHYAT_ERR_INVALID_ARG;
  if (c->impl < REHYAT_IMPL_AUTO || c->impl > REHYAT_IMPL_TENSOR_WINDOW) return REHYAT_ERR_INVALID_ARG;
  if (c->max_tokens_per_frame < 1 || c->max_chunk_frames < 1 || c->group_tokens < 0) return REHYAT_ERR_INVALID_ARG;
  if ((long long)c->max_tokens_per_frame * c->max_chunk_frames > (1 << 24)) return REHYAT_ERR_INVALID_ARG;
  if (c->head_dim < 1) return REHYAT_ERR_INVALID_ARG;
  if (c->bidirectional != 0 && c->bidirectional != 1) return REHYAT_ERR_INVALID_ARG;
  if (c->max_frames < 0 || c->max_frames > (1 << 20) || (c->bidirectional && c->max_frames < 1)) return REHYAT_ERR_INVALID_ARG;
  if (c->exp_poly < -1 || c->exp_poly > 3) return REHYAT_ERR_INVALID_ARG;
  if (c->phi_layers != 0 && (c->phi_layers < 2 || c->phi_layers > 4)) return REHYAT_ERR_INVALID_ARG;
  if (c->qk_transform != 0 && (c->qk_transform != 1 || c->max_frames < 1)) return REHYAT_ERR_INVALID_ARG;
  if (c->window_tiles < 0 || c->window_tiles > 2) return REHYAT_ERR_INVALID_ARG;
  if (c->head_dim != 64 && c->head_dim != 128) return REHYAT_ERR_UNSUPPORTED;
  return REHYAT_OK;
}

// The shared-memory limit of a kernel is a property of the function, not of a context, so it is always set to
// what the widest phi check_config admits (D_h = D' = 256) needs: a later context with narrower widths then
// cannot lower it under a live one.
template <typename T, int D>
int set_simt_attributes() {
  const int smem_state = (SIMT_TM * (2 * D + 256) + phi_hidden_floats(256, 1)) * (int)sizeof(float);
  const int smem_rd = (SIMT_TM * (D + 256) + phi_hidden_floats(256, 1)) * (int)sizeof(float);
  const int smem_win = (WIN_BM * (D + 4) + WIN_BN * (D + 4) + WIN_BN * D + WIN_BM * (WIN_BN + 4)) * (int)sizeof(float);
  if (cudaFuncSetAttribute(state_partial_simt<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_state) != cudaSuccess ||
      cudaFuncSetAttribute(readout_simt<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_rd) != cudaSuccess ||
      cudaFuncSetAttribute(window_simt<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_win) != cudaSuccess)
    return REHYAT_ERR_CUDA;
  return REHYAT_OK;
}

int set_simt_attributes_for(int dtype, int head_dim) {
  if (dtype == REHYAT_DTYPE_FP32) return head_dim == 64 ? set_simt_attributes<float, 64>() : set_simt_attributes<float, 128>();
  return head_dim == 64 ? set_simt_attributes<__nv_bfloat16, 64>() : set_simt_attributes<__nv_bfloat16, 128>();
}

// What every tensor-core launch is told about waiting: a fresh epoch per launch, the limit of one wait.
ptx::WaitArgs next_wait(rehyat_ctx* ctx) {
  ctx->epoch = ctx->epoch == INT_MAX ? 1 : ctx->epoch + 1;
  ptx::WaitArgs wa;
  wa.status = ctx->status_dev;
  wa.epoch = ctx->epoch;
  wa.limit_us = ctx->wait_limit_us;
  wa.withhold_loads = ctx->withhold_loads;
  return wa;
}

// Which steps of a chunk group to enqueue.
enum Parts : int { PART_STATE = 1 /* increments + scan */, PART_READOUT = 2, PART_WINDOW = 4 };

template <typename T, int D>
int launch_group_simt(rehyat_ctx* ctx, const T* q, const T* k, const T* v, T* out, const rehyat_phi_params* phi,
                      const Geo& g, int n_split, int carry_slot, int parts, cudaStream_t st) {
  const rehyat_config& c = ctx->cfg;
  const int rd_half = ctx->tensor_ok ? 1 : 0;     // the tensor-core window kernels read the bf16 form of the read-out
  PhiDims pd = {D, c.phi_hidden, c.phi_dim, c.poly_degree, c.act_hidden, c.act_out, c.phi_layers > 2 ? c.phi_layers - 2 : 0};
  constexpr int SD = D + 4;
  const int tiles = (g.Np + SIMT_TM - 1) / SIMT_TM;
  if (parts & PART_STATE) {
    PhiPtrs<T> wk = {(const T*)phi->k_W1, (const T*)phi->k_b1, (const T*)phi->k_W2, (const T*)phi->k_b2,
                     (const T*)phi->k_Wmid, (const T*)phi->k_bmid};
    const size_t smem_state = ((size_t)SIMT_TM * (2 * D + pd.Dp) + phi_hidden_floats(pd.Dh, pd.n_mid)) * sizeof(float);
    ctx->prof.begin(REHYAT_PROF_STATE, st);
    state_partial_simt<T, D><<<dim3(n_split, g.G, g.BH), SIMT_PHI_THREADS, smem_state, st>>>(
        k, v, wk, pd, g, n_split, ctx->partial);
    ctx->prof.end(REHYAT_PROF_STATE, st);
    const size_t per_slot = (size_t)g.BH * pd.Dp * SD;
    ctx->prof.begin(REHYAT_PROF_SCAN, st);
    scan_states<<<(unsigned)((per_slot + 255) / 256), 256, 0, st>>>(ctx->partial, ctx->state, per_slot, g.G,
                                                                     n_split, carry_slot);
    ctx->prof.end(REHYAT_PROF_SCAN, st);
    ctx->last_launches += 2;
  }
  if (parts & PART_READOUT) {
    PhiPtrs<T> wq = {(const T*)phi->q_W1, (const T*)phi->q_b1, (const T*)phi->q_W2, (const T*)phi->q_b2,
                     (const T*)phi->q_Wmid, (const T*)phi->q_bmid};
    const size_t smem_rd = ((size_t)SIMT_TM * (D + pd.Dp) + phi_hidden_floats(pd.Dh, pd.n_mid)) * sizeof(float);
    ctx->prof.begin(REHYAT_PROF_READOUT, st);
    readout_simt<T, D><<<dim3(tiles, g.G, g.BH), SIMT_PHI_THREADS, smem_rd, st>>>(q, wq, pd, g, ctx->state,
                                                                                 ctx->readout, ctx->rd_cap, rd_half);
    ctx->prof.end(REHYAT_PROF_READOUT, st);
    ctx->last_launches += 1;
  }
  if (parts & PART_WINDOW) {
    const size_t smem_win = (size_t)(WIN_BM * (D + 4) + WIN_BN * (D + 4) + WIN_BN * D + WIN_BM * (WIN_BN + 4)) * sizeof(float);
    const int wtiles = (g.Np + WIN_BM - 1) / WIN_BM;
    ctx->prof.begin(REHYAT_PROF_WINDOW, st);
    window_simt<T, D><<<dim3(wtiles, g.G, g.BH), WIN_THREADS, smem_win, st>>>(
        q, k, v, out, g, ctx->readout, ctx->rd_cap, 1.0f / sqrtf((float)D), c.c_mode, ctx->share_now);
    ctx->prof.end(REHYAT_PROF_WINDOW, st);
    ctx->last_launches += 1;
  }
  return cudaGetLastError() == cudaSuccess ? REHYAT_OK : REHYAT_ERR_CUDA;
}

// Split of a chunk's state increment over CTAs.  Tensor-core kernels: one CTA per (split, chunk, head)
// and one CTA per SM, so pick the split that needs the fewest token tiles per SM over all waves.
int pick_state_split(const rehyat_ctx* ctx, const Geo& g, int n_chunks_in_group, int tokens_per_increment) {
  int n_split = ctx->partial_units / (n_chunks_in_group > 0 ? n_chunks_in_group : 1);
  const int most = ctx->tensor_ok && ctx->tc.phi_ok ? 16 : 8;   // a lone chunk (a chunk-by-chunk step) over all SMs
  if (n_split > most) n_split = most;
  if (n_split < 1) n_split = 1;
  if (ctx->tensor_ok && ctx->tc.phi_ok) {
    const int n_sm = ctx->tc.n_sm;
    int busy = 0;                                   // chunks of the group that admit keys into the state
    for (int t = g.t0 > 1 ? g.t0 : 1; t < g.t0 + n_chunks_in_group; ++t) busy += geo_lo(g, t) > geo_lo(g, t - 1);
    const long long units = (long long)(busy > 0 ? busy : 1) * g.BH, tiles = (tokens_per_increment + 127) / 128;
    long long best = -1;
    int best_s = 1;
    for (int s = 1; s <= n_split; ++s) {
      const long long cost = ((units * s + n_sm - 1) / n_sm) * ((tiles + s - 1) / s);
      if (best < 0 || cost < best) { best = cost; best_s = s; }
    }
    n_split = best_s;
  }
  return n_split;
}

// Enqueues the requested steps for the chunks [g.t0, g.t0 + g.G) with whichever kernel family the context uses.
int run_parts(rehyat_ctx* ctx, const void* q, const void* k, const void* v, void* out, const rehyat_phi_params* phi,
              const Geo& g, int batch, int n_split, int carry_slot, int parts, cudaStream_t st) {
  const rehyat_config& c = ctx->cfg;
  int rc = REHYAT_OK;
  if (ctx->tensor_ok) {
    using B = __nv_bfloat16;
    if (!ctx->tc.phi_ok) {
      rc = c.head_dim == 64
               ? launch_group_simt<B, 64>(ctx, (const B*)q, (const B*)k, (const B*)v, (B*)out, phi, g, n_split, carry_slot,
                                          parts & (PART_STATE | PART_READOUT), st)
               : launch_group_simt<B, 128>(ctx, (const B*)q, (const B*)k, (const B*)v, (B*)out, phi, g, n_split, carry_slot,
                                           parts & (PART_STATE | PART_READOUT), st);
    } else {
      if (parts & PART_STATE) {
        ctx->prof.begin(REHYAT_PROF_STATE, st);
        rc = tc_launch_state(&ctx->tc, k, v, phi, g, batch, c.phi_hidden, c.phi_dim, c.poly_degree,
                             c.phi_layers > 2 ? c.phi_layers - 2 : 0, c.act_hidden, c.act_out, n_split,
                             ctx->partial, next_wait(ctx), st);
        ctx->prof.end(REHYAT_PROF_STATE, st);
        const size_t per_slot = (size_t)g.BH * c.phi_dim * (c.head_dim + 4);
        ctx->prof.begin(REHYAT_PROF_SCAN, st);
        scan_states<<<(unsigned)((per_slot + 255) / 256), 256, 0, st>>>(ctx->partial, ctx->state, per_slot, g.G, n_split,
                                                                         carry_slot, ctx->tc.state_bf16, c.head_dim);
        ctx->prof.end(REHYAT_PROF_SCAN, st);
        ctx->last_launches += 2;
      }
      if (rc == REHYAT_OK && (parts & PART_READOUT)) {
        ctx->prof.begin(REHYAT_PROF_READOUT, st);
        rc = tc_launch_readout(&ctx->tc, q, phi, g, batch, c.phi_hidden, c.phi_dim, c.poly_degree,
                               c.phi_layers > 2 ? c.phi_layers - 2 : 0, c.act_hidden, c.act_out, ctx->state,
                               ctx->readout, ctx->rd_cap, next_wait(ctx), st);
        ctx->prof.end(REHYAT_PROF_READOUT, st);
        ctx->last_launches += 1;
      }
    }
    if (rc == REHYAT_OK && (parts & PART_WINDOW)) {
      ctx->prof.begin(REHYAT_PROF_WINDOW, st);
      rc = tc_launch_window(&ctx->tc, q, k, v, out, g, batch, ctx->readout, ctx->rd_cap, c.c_mode, next_wait(ctx), ctx->share_now, st);
      ctx->prof.end(REHYAT_PROF_WINDOW, st);
      ctx->last_launches += 1;
    }
  } else if (c.dtype == REHYAT_DTYPE_FP32) {
    rc = c.head_dim == 64
             ? launch_group_simt<float, 64>(ctx, (const float*)q, (const float*)k, (const float*)v, (float*)out, phi, g, n_split, carry_slot, parts, st)
             : launch_group_simt<float, 128>(ctx, (const float*)q, (const float*)k, (const float*)v, (float*)out, phi, g, n_split, carry_slot, parts, st);
  } else {
    using B = __nv_bfloat16;
    rc = c.head_dim == 64
             ? launch_group_simt<B, 64>(ctx, (const B*)q, (const B*)k, (const B*)v, (B*)out, phi, g, n_split, carry_slot, parts, st)
             : launch_group_simt<B, 128>(ctx, (const B*)q, (const B*)k, (const B*)v, (B*)out, phi, g, n_split, carry_slot, parts, st);
  }
  return rc;
}

// The phi parameter pointers: all there and 16-byte aligned (the hidden layers in between only for deeper maps).
bool phi_pointers_ok(const rehyat_config& c, const rehyat_phi_params* phi) {
  const void* two[] = {phi->q_W1, phi->q_b1, phi->q_W2, phi->q_b2, phi->k_W1, phi->k_b1, phi->k_W2, phi->k_b2};
  for (const void* p : two)
    if (!p || !aligned16(p)) return false;
  if (c.phi_layers > 2) {
    const void* mid[] = {phi->q_Wmid, phi->q_bmid, phi->k_Wmid, phi->k_bmid};
    for (const void* p : mid)
      if (!p || !aligned16(p)) return false;
  }
  return true;
}

// The size arguments of a forward call against the limits of the context (nothing is enqueued before this passes).
int check_sizes(const rehyat_ctx* ctx, int batch, int frames, int H, int W, int chunk, int overlap) {
  const rehyat_config& c = ctx->cfg;
  if (batch < 1 || batch > c.max_batch || frames < 1 || H < 1 || W < 1 || chunk < 1 || overlap < 0)
    return REHYAT_ERR_INVALID_ARG;
  const long long HW = (long long)H * W;
  if (HW > c.max_tokens_per_frame) return REHYAT_ERR_INVALID_ARG;
  if (HW * frames > INT_MAX / 2) return REHYAT_ERR_INVALID_ARG;
  if ((chunk < frames ? chunk : frames) > c.max_chunk_frames) return REHYAT_ERR_INVALID_ARG;   // one chunk covers everything beyond `frames`
  if (c.bidirectional && frames + 1 > ctx->cum_frames) return REHYAT_ERR_INVALID_ARG;
  if (ctx->qk_on && frames > c.max_frames) return REHYAT_ERR_INVALID_ARG;
  return REHYAT_OK;
}

// Enqueues the q/k transform set with rehyat_set_qk_transform: `rows` token rows per (batch, head) of q and k (source
// strides in `pa.s*`) into qo and ko (strides in `pa.q*`, `pa.k*`), rotation tables read from position pa.pos0 on.
void launch_qk_prepare(rehyat_ctx* ctx, const void* q, const void* k, void* qo, void* ko, QkPrepArgs pa, int BH, cudaStream_t st) {
  const rehyat_config& c = ctx->cfg;
  pa.wq = ctx->qk.q_norm_weight; pa.wk = ctx->qk.k_norm_weight;
  pa.cos = ctx->qk.rope_cos; pa.sin = ctx->qk.rope_sin;
  pa.eps = ctx->qk.norm_eps; pa.rms_norm = ctx->qk.rms_norm;
  const int rows_per_block = 256 / (c.head_dim / 8);
  // about thirty-two CTAs per SM over the whole grid, every thread walking several pairs of rows of its columns
  const long long want = (32LL * ctx->tc.n_sm + 2 * BH - 1) / (2 * BH), need = (pa.rows + 2 * rows_per_block - 1) / (2 * rows_per_block);
  const unsigned blocks = (unsigned)(need < want ? need : (want > 0 ? want : 1));
  const dim3 grid(blocks, BH, 2);
  ctx->prof.begin(REHYAT_PROF_QKPREP, st);
  if (c.dtype == REHYAT_DTYPE_FP32) {
    if (c.head_dim == 64) qk_prepare<float, 64><<<grid, 256, 0, st>>>((const float*)q, (const float*)k, (float*)qo, (float*)ko, pa);
    else qk_prepare<float, 128><<<grid, 256, 0, st>>>((const float*)q, (const float*)k, (float*)qo, (float*)ko, pa);
  } else {
    using B = __nv_bfloat16;
    if (c.head_dim == 64) qk_prepare<B, 64><<<grid, 256, 0, st>>>((const B*)q, (const B*)k, (B*)qo, (B*)ko, pa);
    else qk_prepare<B, 128><<<grid, 256, 0, st>>>((const B*)q, (const B*)k, (B*)qo, (B*)ko, pa);
  }
  ctx->prof.end(REHYAT_PROF_QKPREP, st);
  ctx->last_launches += 1;
}

// Copies `rows` token rows of `row_bytes` bytes for each of BH (batch, head) problems between two strided
// layouts (byte strides; rows are contiguous and 16-byte aligned).  grid (row tiles, BH), 256 threads.
__global__ void copy_rows(uint8_t* __restrict__ dst0, uint8_t* __restrict__ dst1, long long dst_b, long long dst_h, long long dst_n,
                          const uint8_t* __restrict__ src0, const uint8_t* __restrict__ src1, long long src_b, long long src_h,
                          long long src_n, int rows, int row_bytes, int n_heads) {
  // blockIdx.z picks one of two tensor pairs that share their layouts (k and v)
  uint8_t* __restrict__ dst = blockIdx.z ? dst1 : dst0;
  const uint8_t* __restrict__ src = blockIdx.z ? src1 : src0;
  const int bh = blockIdx.y, b = bh / n_heads, h = bh % n_heads;
  const int per_row = row_bytes / 16;
  const long long total = (long long)rows * per_row;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / per_row, c = (i % per_row) * 16;
    *reinterpret_cast<uint4*>(dst + b * dst_b + h * dst_h + r * dst_n + c) =
        *reinterpret_cast<const uint4*>(src + b * src_b + h * src_h + r * src_n + c);
  }
}

}  // namespace

extern "C" {

int rehyat_version(void) { return 100; }

const char* rehyat_strerror(int code) {
  switch (code) {
    case REHYAT_OK: return "ok";
    case REHYAT_ERR_INVALID_ARG: return "invalid argument";
    case REHYAT_ERR_UNSUPPORTED: return "unsupported shape or mode";
    case REHYAT_ERR_CUDA: return "CUDA call failed";
    case REHYAT_ERR_ARCH: return "device is not compute capability 10.x (sm_100)";
    case REHYAT_ERR_ALLOC: return "device allocation failed";
    case REHYAT_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case REHYAT_ERR_TOO_LARGE: return "problem does not fit the fixed scratch of rehyat_forward_static";
    default: return "unknown error code";
  }
}

int rehyat_create(rehyat_ctx** out, const rehyat_config* cfg) {
  if (!out || !cfg) return REHYAT_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = check_config(cfg);
  if (rc != REHYAT_OK) return rc;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess) { cudaGetLastError(); return REHYAT_ERR_CUDA; }
  if (cfg->device < 0 || cfg->device >= ndev) return REHYAT_ERR_INVALID_ARG;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return REHYAT_ERR_CUDA;
  if (prop.major != 10) return REHYAT_ERR_ARCH;
  DeviceGuard guard(cfg->device);
  if (!guard.ok) return REHYAT_ERR_CUDA;

  rehyat_ctx* ctx = new (std::nothrow) rehyat_ctx();
  if (!ctx) return REHYAT_ERR_ALLOC;
  ctx->cfg = *cfg;
  const rehyat_config& c = ctx->cfg;
  ctx->tensor_ok = tc_shape_supported(c.dtype == REHYAT_DTYPE_BF16, c.head_dim, c.phi_hidden, c.phi_dim,
                                      c.poly_degree, c.act_hidden, c.act_out);
  if ((c.impl == REHYAT_IMPL_TENSOR || c.impl == REHYAT_IMPL_TENSOR_WINDOW) && !ctx->tensor_ok) { delete ctx; return REHYAT_ERR_UNSUPPORTED; }
  if (c.impl == REHYAT_IMPL_SIMT) ctx->tensor_ok = false;
  ctx->tc.phi_ok = ctx->tensor_ok && c.impl != REHYAT_IMPL_TENSOR_WINDOW &&
                   tc_phi_supported(c.head_dim, c.phi_hidden, c.phi_dim, c.poly_degree, c.phi_layers > 2 ? c.phi_layers - 2 : 0);
  ctx->tc.head_dim = c.head_dim;

  const int np_max = c.max_tokens_per_frame * c.max_chunk_frames;
  const int want = c.group_tokens > 0 ? c.group_tokens : 32768;
  ctx->rd_rows = ((want > np_max ? want : np_max) + 127) / 128 * 128 + 128;
  ctx->Gmax = 16;
  ctx->rd_cap = ctx->rd_rows + ctx->Gmax * 128;          // every chunk's last 128-row tile may be partly empty
  ctx->partial_units = 32;
  ctx->bh_max = c.max_batch * c.n_heads;
  const size_t SD = c.head_dim + 4;
  const size_t slot = (size_t)ctx->bh_max * c.phi_dim * SD * sizeof(float);
  const size_t b_state = slot * ctx->Gmax, b_partial = slot * ctx->partial_units;
  // read-out of one chunk group: fp32 rows of d + 4 for the SIMT window kernel, d/8 + 1 16-byte pieces per row
  // (fp16 ratios) for the tensor-core ones
  const size_t b_rd = ctx->tensor_ok ? (size_t)ctx->bh_max * ctx->rd_cap * rdh_pieces(c.head_dim) * 16
                                     : (size_t)ctx->bh_max * ctx->rd_cap * SD * sizeof(float);
  bool ok = cudaMalloc(&ctx->state, b_state) == cudaSuccess && cudaMalloc(&ctx->partial, b_partial) == cudaSuccess &&
            cudaMalloc(&ctx->readout, b_rd) == cudaSuccess && cudaMalloc(&ctx->status_dev, 256) == cudaSuccess;
  ctx->ws_bytes = b_state + b_partial + b_rd + 256;
  if (ok && c.qk_transform) {
    ctx->prep_elems = (size_t)ctx->bh_max * c.max_frames * c.max_tokens_per_frame * c.head_dim;
    const size_t b_prep = ctx->prep_elems * elem_size(c.dtype);
    ok = cudaMalloc(&ctx->qprep, b_prep) == cudaSuccess && cudaMalloc(&ctx->kprep, b_prep) == cudaSuccess;
    ctx->ws_bytes += 2 * b_prep;
  }
  if (ok && c.bidirectional) {
    // Eq. 10-12 is not a recurrence: one running state per latent frame, sized here so that forward never allocates
    const size_t b_cum = slot * ((size_t)c.max_frames + 1);
    ok = cudaMalloc(&ctx->cum, b_cum) == cudaSuccess;
    ctx->cum_frames = c.max_frames + 1;
    ctx->ws_bytes += b_cum;
  }
  cudaDeviceGetAttribute(&ctx->tc.n_sm, cudaDevAttrMultiProcessorCount, c.device);
  ctx->tc.exp_poly = c.exp_poly == 0 ? 1 : (c.exp_poly < 0 ? 0 : c.exp_poly);
  ctx->tc.item_tiles = c.window_tiles;
  if (ok && ctx->tensor_ok) {
    size_t extra = 0;
    ok = tc_workspace_create(&ctx->tc, ctx->bh_max, ctx->Gmax, c.head_dim, c.phi_dim, &extra);
    ctx->ws_bytes += extra;
  }
  if (!ok) { cudaGetLastError(); rehyat_destroy(ctx); return REHYAT_ERR_ALLOC; }
  if (cudaMemset(ctx->status_dev, 0, 256) != cudaSuccess) { rehyat_destroy(ctx); return REHYAT_ERR_CUDA; }

  rc = set_simt_attributes_for(c.dtype, c.head_dim);
  if (rc == REHYAT_OK && ctx->tensor_ok) rc = tc_set_attributes();
  if (rc != REHYAT_OK) { rehyat_destroy(ctx); return rc; }
  *out = ctx;
  return REHYAT_OK;
}

int rehyat_destroy(rehyat_ctx* ctx) {
  if (!ctx) return REHYAT_OK;
  DeviceGuard guard(ctx->cfg.device);
  cudaFree(ctx->state); cudaFree(ctx->partial); cudaFree(ctx->readout); cudaFree(ctx->status_dev); cudaFree(ctx->cum);
  cudaFree(ctx->qprep); cudaFree(ctx->kprep);
  tc_workspace_destroy(&ctx->tc);
  ctx->prof.clear();
  for (void* p : ctx->stage) cudaFree(p);
  if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
  if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
  for (cudaEvent_t e : ctx->host_events) cudaEventDestroy(e);
  cudaFree(ctx->stream.kbuf); cudaFree(ctx->stream.vbuf); cudaFree(ctx->stream.qbuf);
  delete ctx;
  return REHYAT_OK;
}

size_t rehyat_workspace_bytes(const rehyat_ctx* ctx) { return ctx ? ctx->ws_bytes : 0; }
int rehyat_last_launches(const rehyat_ctx* ctx) { return ctx ? ctx->last_launches : 0; }
int rehyat_last_impl(const rehyat_ctx* ctx) { return ctx ? ctx->last_impl : 0; }
int rehyat_last_window_tiles(const rehyat_ctx* ctx) { return ctx && ctx->last_impl ? ctx->tc.last_item_tiles : 0; }

int rehyat_set_linear_share_output(rehyat_ctx* ctx, float* share) {
  if (!ctx || (share && !aligned16(share))) return REHYAT_ERR_INVALID_ARG;
  ctx->share_out = share;
  return REHYAT_OK;
}

int rehyat_profile_enable(rehyat_ctx* ctx, int on) {
  if (!ctx) return REHYAT_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->cfg.device);
  ctx->prof.clear();
  ctx->prof.on = on != 0;
  return REHYAT_OK;
}

int rehyat_profile_read(rehyat_ctx* ctx, double* ms, int32_t* launches) {
  if (!ctx || !ms || !launches) return REHYAT_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->cfg.device);
  for (int kind = 0; kind < REHYAT_PROF_KINDS; ++kind) {
    auto& v = ctx->prof.ev[kind];
    ms[kind] = 0.0;
    launches[kind] = (int32_t)(v.size() / 2);
    for (size_t i = 0; i + 1 < v.size(); i += 2) {
      float t = 0.f;
      if (cudaEventSynchronize(v[i + 1]) != cudaSuccess || cudaEventElapsedTime(&t, v[i], v[i + 1]) != cudaSuccess)
        return REHYAT_ERR_CUDA;
      ms[kind] += t;
    }
  }
  ctx->prof.clear();
  return REHYAT_OK;
}

int rehyat_status(rehyat_ctx* ctx, void* cuda_stream) {
  if (!ctx) return REHYAT_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->cfg.device);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int word = 0;
  if (cudaStreamSynchronize(st) != cudaSuccess) return REHYAT_ERR_CUDA;
  if (cudaMemcpy(&word, ctx->status_dev, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return REHYAT_ERR_CUDA;
  if (word != 0) {
    // the sticky bits are cleared; launches after the one that timed out carry another epoch and are not affected
    if (cudaMemset(ctx->status_dev, 0, 256) != cudaSuccess) return REHYAT_ERR_CUDA;
    return REHYAT_ERR_DEVICE_TIMEOUT;
  }
  return REHYAT_OK;
}

int rehyat_set_qk_transform(rehyat_ctx* ctx, const rehyat_qk_transform* t) {
  if (!ctx) return REHYAT_ERR_INVALID_ARG;
  if (!t) { ctx->qk_on = false; return REHYAT_OK; }
  if (!ctx->cfg.qk_transform) return REHYAT_ERR_UNSUPPORTED;     // the context was made without room for it
  const void* ptrs[] = {t->q_norm_weight, t->k_norm_weight, t->rope_cos, t->rope_sin};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return REHYAT_ERR_INVALID_ARG;
  if ((t->rope_cos == nullptr) != (t->rope_sin == nullptr) || !(t->norm_eps >= 0.f)) return REHYAT_ERR_INVALID_ARG;
  ctx->qk = *t;
  ctx->qk_on = true;
  return REHYAT_OK;
}

int rehyat_set_wait_limit(rehyat_ctx* ctx, int32_t wait_limit_us, int32_t withhold_loads) {
  if (!ctx || wait_limit_us < 0) return REHYAT_ERR_INVALID_ARG;
  ctx->wait_limit_us = wait_limit_us > 0 ? (unsigned)wait_limit_us : 1000000u;
  ctx->withhold_loads = withhold_loads != 0;
  return REHYAT_OK;
}

int rehyat_forward(rehyat_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                   const rehyat_layout* lay, const rehyat_phi_params* phi, int32_t batch, int32_t frames,
                   int32_t H, int32_t W, int32_t chunk, int32_t overlap, void* cuda_stream) {
  if (!ctx || !q || !k || !v || !out || !lay || !phi) return REHYAT_ERR_INVALID_ARG;
  const rehyat_config& c = ctx->cfg;
  if (const int bad = check_sizes(ctx, batch, frames, H, W, chunk, overlap)) return bad;
  const long long HW = (long long)H * W;
  const long long N = HW * frames;
  const int chunk_eff = chunk < frames ? chunk : frames;      // one chunk covers everything beyond that
  const int overlap_eff = overlap < frames ? overlap : frames; // the window is clamped at token 0 anyway
  if (out == q || out == k || out == v) return REHYAT_ERR_INVALID_ARG;
  const void* ptrs[] = {q, k, v, out};
  for (const void* p : ptrs)
    if (!aligned16(p)) return REHYAT_ERR_INVALID_ARG;
  if (!phi_pointers_ok(c, phi)) return REHYAT_ERR_INVALID_ARG;
  const size_t es = elem_size(c.dtype);
  const long long strides[] = {lay->stride_batch, lay->stride_head, lay->stride_token};
  for (long long s : strides)
    if (s < 0 || (s * (long long)es) % 16 != 0) return REHYAT_ERR_INVALID_ARG;
  if (lay->stride_token < c.head_dim) return REHYAT_ERR_INVALID_ARG;
  const int heads_here = ctx->head_count > 0 ? ctx->head_count : c.n_heads;
  // an axis of more than one element needs a stride that keeps its elements apart
  if ((heads_here > 1 && lay->stride_head < c.head_dim) || (batch > 1 && lay->stride_batch < c.head_dim))
    return REHYAT_ERR_INVALID_ARG;

  DeviceGuard guard(c.device);
  if (!guard.ok) return REHYAT_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;

  Geo g;
  g.N = (int)N;
  g.Np = (int)(chunk_eff * HW);
  g.ToHW = (int)(overlap_eff * HW);
  g.n_heads = ctx->head_count > 0 ? ctx->head_count : c.n_heads;
  g.BH = batch * g.n_heads;
  g.stride_b = lay->stride_batch; g.stride_h = lay->stride_head; g.stride_n = lay->stride_token;
  // the stride of a one-element axis is never used for addressing; tensor maps still want it non-zero
  if (g.stride_h == 0) g.stride_h = g.stride_n * N;
  if (g.stride_b == 0) g.stride_b = g.stride_h * g.n_heads;
  g.qstride_b = g.stride_b; g.qstride_h = g.stride_h; g.qstride_n = g.stride_n;   // q and out: laid out like k and v
  g.ostride_b = g.stride_b; g.ostride_h = g.stride_h; g.ostride_n = g.stride_n;
  g.q_off = 0; g.Nq = g.N;
  const int n_chunks = (frames + chunk_eff - 1) / chunk_eff;
  g.q_shift = 0;
  g.prefix = 0;
  int G = ctx->rd_rows / g.Np;
  if (G < 1) return REHYAT_ERR_INVALID_ARG;   // cannot happen: rd_rows >= max chunk size
  if (G > ctx->Gmax) G = ctx->Gmax;
  g.t0 = 0;
  const int n_split = pick_state_split(ctx, g, G < n_chunks ? G : n_chunks, g.Np);

  ctx->last_launches = 0;
  ctx->last_impl = ctx->tensor_ok ? (ctx->tc.phi_ok ? 2 : 1) : 0;
  ctx->stream.active = false;                 // the workspace is about to be overwritten
  if (ctx->qk_on) {
    // q and k are normalised and rotated into the context's buffers, in the layout they came in
    const long long last = (batch - 1) * g.stride_b + (g.n_heads - 1) * g.stride_h + (N - 1) * g.stride_n + c.head_dim;
    if (ctx->head_count > 0 || (size_t)last > ctx->prep_elems) return REHYAT_ERR_INVALID_ARG;
    QkPrepArgs pa = {};
    pa.rows = (int)N; pa.n_heads = g.n_heads; pa.pos0 = 0;
    pa.sb = pa.qb = pa.kb = g.stride_b; pa.sh = pa.qh = pa.kh = g.stride_h; pa.sn = pa.qn = pa.kn = g.stride_n;
    launch_qk_prepare(ctx, q, k, ctx->qprep, ctx->kprep, pa, g.BH, st);
    q = ctx->qprep;
    k = ctx->kprep;
  }
  ctx->share_now = ctx->head_count > 0 ? nullptr : ctx->share_out;   // not through rehyat_forward_host
  if (c.bidirectional && n_chunks > 1) {
    // Eq. 10-12: the linear set of a chunk is everything outside its window.  Pass 1 sums the state frame by
    // frame (running sums cum[0..frames]); pass 2 forms each chunk's state from three of those sums.
    const size_t per_slot = (size_t)g.BH * c.phi_dim * (c.head_dim + 4), slot_bytes = per_slot * sizeof(float);
    if (cudaMemsetAsync(ctx->cum, 0, slot_bytes, st) != cudaSuccess) return REHYAT_ERR_CUDA;
    Geo gs = g;
    gs.Np = (int)HW; gs.ToHW = 0;
    int carry = -1;
    for (int f0 = 1; f0 <= frames; f0 += ctx->Gmax) {
      gs.t0 = f0;                                // "chunk" f admits frame f-1: [lo_{f-1}, lo_f) = [(f-1) HW, f HW)
      gs.G = frames + 1 - f0 < ctx->Gmax ? frames + 1 - f0 : ctx->Gmax;
      const int ns = pick_state_split(ctx, gs, gs.G, (int)HW);
      const int rc = run_parts(ctx, nullptr, k, v, nullptr, phi, gs, batch, ns, carry, PART_STATE, st);
      if (rc != REHYAT_OK) return rc;
      if (cudaMemcpyAsync((uint8_t*)ctx->cum + (size_t)f0 * slot_bytes, ctx->state, (size_t)gs.G * slot_bytes,
                          cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return REHYAT_ERR_CUDA;
      carry = gs.G - 1;
    }
    g.prefix = 1;                                // every chunk reads its state, whatever lo_t is
    for (int t0 = 0; t0 < n_chunks; t0 += G) {
      g.t0 = t0;
      g.G = (n_chunks - t0) < G ? (n_chunks - t0) : G;
      combine_bidirectional<<<(unsigned)((per_slot + 255) / 256), 256, 0, st>>>(
          ctx->cum, ctx->state, per_slot, g, (int)HW, frames,
          (ctx->tensor_ok && ctx->tc.phi_ok) ? ctx->tc.state_bf16 : nullptr, c.head_dim);
      ctx->last_launches += 1;
      const int rc = run_parts(ctx, q, k, v, out, phi, g, batch, 1, -1, PART_READOUT | PART_WINDOW, st);
      if (rc != REHYAT_OK) return rc;
    }
    return REHYAT_OK;
  }
  int carry_slot = -1;
  for (int t0 = 0; t0 < n_chunks; t0 += G) {
    g.t0 = t0;
    g.G = (n_chunks - t0) < G ? (n_chunks - t0) : G;
    const bool any_linear = geo_lo(g, t0 + g.G - 1) > 0;
    const int rc = run_parts(ctx, q, k, v, out, phi, g, batch, n_split, carry_slot,
                             (any_linear ? PART_STATE | PART_READOUT : 0) | PART_WINDOW, st);
    if (rc != REHYAT_OK) return rc;
    if (any_linear) carry_slot = g.G - 1;
  }
  return REHYAT_OK;
}

int rehyat_forward_host(rehyat_ctx* ctx, const void* q_host, const void* k_host, const void* v_host,
                        void* out_host, const rehyat_phi_params* phi, int32_t batch, int32_t frames, int32_t H,
                        int32_t W, int32_t chunk, int32_t overlap, void* cuda_stream) {
  if (!ctx || !q_host || !k_host || !v_host || !out_host || !phi) return REHYAT_ERR_INVALID_ARG;
  if (ctx->qk_on) return REHYAT_ERR_UNSUPPORTED;
  // every argument is checked before the first copy is enqueued
  if (const int bad = check_sizes(ctx, batch, frames, H, W, chunk, overlap)) return bad;
  const rehyat_config& c = ctx->cfg;
  if (!phi_pointers_ok(c, phi)) return REHYAT_ERR_INVALID_ARG;
  const long long N = (long long)H * W * frames;
  const size_t bytes = (size_t)batch * c.n_heads * N * c.head_dim * elem_size(c.dtype);
  DeviceGuard guard(c.device);
  if (!guard.ok) return REHYAT_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (bytes > ctx->stage_bytes) {
    if (cudaStreamSynchronize(st) != cudaSuccess) return REHYAT_ERR_CUDA;
    for (void*& p : ctx->stage) { cudaFree(p); p = nullptr; }
    ctx->stage_bytes = 0;
    for (void*& p : ctx->stage)
      if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return REHYAT_ERR_ALLOC; }
    ctx->stage_bytes = bytes;
  }
  // The (batch, head) problems are independent, so the call is pipelined over groups of heads: while group g
  // is computed on `cuda_stream`, group g+1 is copied in and group g-1 copied out on two streams of the context.
  if (!ctx->copy_in && cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking) != cudaSuccess) return REHYAT_ERR_CUDA;
  if (!ctx->copy_out && cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking) != cudaSuccess) return REHYAT_ERR_CUDA;
  const int per_group = (c.n_heads + 15) / 16, n_groups = (c.n_heads + per_group - 1) / per_group;
  while ((int)ctx->host_events.size() < 2 * n_groups + 1) {
    cudaEvent_t e;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return REHYAT_ERR_CUDA;
    ctx->host_events.push_back(e);
  }
  const size_t es = elem_size(c.dtype), head_bytes = (size_t)N * c.head_dim * es;
  rehyat_layout lay = {(int64_t)c.n_heads * N * c.head_dim, (int64_t)N * c.head_dim, (int64_t)c.head_dim};
  // earlier work on the caller's stream may still read the staging buffers
  cudaEvent_t e_start = ctx->host_events[2 * n_groups];
  if (cudaEventRecord(e_start, st) != cudaSuccess || cudaStreamWaitEvent(ctx->copy_in, e_start, 0) != cudaSuccess) return REHYAT_ERR_CUDA;
  const void* src[3] = {q_host, k_host, v_host};
  int rc = REHYAT_OK;
  for (int gi = 0; gi < n_groups && rc == REHYAT_OK; ++gi) {
    const int h0 = gi * per_group, cnt = (c.n_heads - h0) < per_group ? (c.n_heads - h0) : per_group;
    const size_t off0 = (size_t)h0 * head_bytes, gbytes = (size_t)cnt * head_bytes;
    for (int b = 0; b < batch; ++b) {
      const size_t off = (size_t)b * c.n_heads * head_bytes + off0;
      for (int i = 0; i < 3; ++i)
        if (cudaMemcpyAsync((uint8_t*)ctx->stage[i] + off, (const uint8_t*)src[i] + off, gbytes, cudaMemcpyHostToDevice,
                            ctx->copy_in) != cudaSuccess)
          return REHYAT_ERR_CUDA;
    }
    cudaEvent_t e_in = ctx->host_events[2 * gi], e_done = ctx->host_events[2 * gi + 1];
    if (cudaEventRecord(e_in, ctx->copy_in) != cudaSuccess || cudaStreamWaitEvent(st, e_in, 0) != cudaSuccess) return REHYAT_ERR_CUDA;
    rehyat_phi_params ph = *phi;                           // parameters of the group's first head
    const size_t w1 = (size_t)h0 * c.phi_hidden * c.head_dim * es, b1 = (size_t)h0 * c.phi_hidden * es;
    const size_t w2 = (size_t)h0 * c.phi_dim * c.phi_hidden * es, b2 = (size_t)h0 * c.phi_dim * es;
    ph.q_W1 = (const uint8_t*)phi->q_W1 + w1; ph.q_b1 = (const uint8_t*)phi->q_b1 + b1;
    ph.q_W2 = (const uint8_t*)phi->q_W2 + w2; ph.q_b2 = (const uint8_t*)phi->q_b2 + b2;
    ph.k_W1 = (const uint8_t*)phi->k_W1 + w1; ph.k_b1 = (const uint8_t*)phi->k_b1 + b1;
    ph.k_W2 = (const uint8_t*)phi->k_W2 + w2; ph.k_b2 = (const uint8_t*)phi->k_b2 + b2;
    if (c.phi_layers > 2) {
      const size_t wm = (size_t)h0 * (c.phi_layers - 2) * c.phi_hidden * c.phi_hidden * es, bm = (size_t)h0 * (c.phi_layers - 2) * c.phi_hidden * es;
      ph.q_Wmid = (const uint8_t*)phi->q_Wmid + wm; ph.q_bmid = (const uint8_t*)phi->q_bmid + bm;
      ph.k_Wmid = (const uint8_t*)phi->k_Wmid + wm; ph.k_bmid = (const uint8_t*)phi->k_bmid + bm;
    }
    ctx->head_count = cnt;
    const int launches_before = gi == 0 ? 0 : ctx->last_launches;
    rc = rehyat_forward(ctx, (uint8_t*)ctx->stage[0] + off0, (uint8_t*)ctx->stage[1] + off0, (uint8_t*)ctx->stage[2] + off0,
                        (uint8_t*)ctx->stage[3] + off0, &lay, &ph, batch, frames, H, W, chunk, overlap, cuda_stream);
    ctx->head_count = 0;
    ctx->last_launches += launches_before;
    if (rc != REHYAT_OK) break;
    if (cudaEventRecord(e_done, st) != cudaSuccess || cudaStreamWaitEvent(ctx->copy_out, e_done, 0) != cudaSuccess) return REHYAT_ERR_CUDA;
    for (int b = 0; b < batch; ++b) {
      const size_t off = (size_t)b * c.n_heads * head_bytes + off0;
      if (cudaMemcpyAsync((uint8_t*)out_host + off, (uint8_t*)ctx->stage[3] + off, gbytes, cudaMemcpyDeviceToHost,
                          ctx->copy_out) != cudaSuccess)
        return REHYAT_ERR_CUDA;
    }
  }
  // the call returns with `out_host` filled, also after an error in the middle
  const bool ok = cudaStreamSynchronize(ctx->copy_in) == cudaSuccess && cudaStreamSynchronize(st) == cudaSuccess &&
                  cudaStreamSynchronize(ctx->copy_out) == cudaSuccess;
  if (rc != REHYAT_OK) return rc;
  return ok ? REHYAT_OK : REHYAT_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Chunk-by-chunk processing: the recurrence of Eq. 14-18 with the state held by the context.
// ---------------------------------------------------------------------------------------------
namespace {

struct StreamHeader {          // first bytes of an exported state
  uint32_t magic, version;
  int32_t dtype, n_heads, head_dim, phi_dim, batch, H, W, chunk, overlap, halo, has_state, reserved;
  int64_t chunks_done;
  int64_t tokens_done;         // position of the next chunk's first token (rotation tables of a q/k transform)
};
constexpr uint32_t kStreamMagic = 0x52485953u;   // "RHYS"

size_t stream_state_floats(const rehyat_ctx* ctx) {
  return (size_t)ctx->stream.batch * ctx->cfg.n_heads * ctx->cfg.phi_dim * (ctx->cfg.head_dim + 4);
}
size_t stream_halo_bytes(const rehyat_ctx* ctx) {      // of k (and as much again of v)
  return (size_t)ctx->stream.batch * ctx->cfg.n_heads * ctx->stream.halo * ctx->cfg.head_dim * elem_size(ctx->cfg.dtype);
}

// Copies dst0 <- src0 and dst1 <- src1 (two tensors with the same layouts) in one launch.
void launch_copy_rows2(void* dst0, void* dst1, long long dst_b, long long dst_h, long long dst_n, const void* src0,
                       const void* src1, long long src_b, long long src_h, long long src_n, int rows, int row_bytes, int BH,
                       int n_heads, cudaStream_t st) {
  if (rows <= 0) return;
  const long long total = (long long)rows * (row_bytes / 16);
  const unsigned blocks = (unsigned)((total + 255) / 256 < 256 ? (total + 255) / 256 : 256);
  copy_rows<<<dim3(blocks, BH, dst1 ? 2 : 1), 256, 0, st>>>((uint8_t*)dst0, (uint8_t*)dst1, dst_b, dst_h, dst_n, (const uint8_t*)src0,
                                                 (const uint8_t*)src1, src_b, src_h, src_n, rows, row_bytes, n_heads);
}

}  // namespace

int rehyat_stream_begin(rehyat_ctx* ctx, int32_t batch, int32_t H, int32_t W, int32_t chunk, int32_t overlap,
                        void* cuda_stream) {
  if (!ctx) return REHYAT_ERR_INVALID_ARG;
  const rehyat_config& c = ctx->cfg;
  if (c.bidirectional) return REHYAT_ERR_UNSUPPORTED;     // later tokens are not known chunk by chunk
  if (batch < 1 || batch > c.max_batch || H < 1 || W < 1 || chunk < 1 || overlap < 0) return REHYAT_ERR_INVALID_ARG;
  const long long HW = (long long)H * W;
  if (HW > c.max_tokens_per_frame || chunk > c.max_chunk_frames) return REHYAT_ERR_INVALID_ARG;
  // room for the kept frames and several chunks behind them, so that the kept frames go back to the front only
  // every few steps; (rounds - 1) chunks >= overlap keeps that copy from overlapping itself
  const long long rounds = 4 > (overlap + chunk - 1) / chunk + 1 ? 4 : (overlap + chunk - 1) / chunk + 1;
  const long long cap = ((long long)overlap + rounds * chunk) * HW;
  if (cap > (1 << 24)) return REHYAT_ERR_INVALID_ARG;
  DeviceGuard guard(c.device);
  if (!guard.ok) return REHYAT_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  rehyat_ctx::Stream& s = ctx->stream;
  const size_t one = (size_t)batch * c.n_heads * cap * c.head_dim * elem_size(c.dtype);
  const size_t qone = c.qk_transform ? (size_t)batch * c.n_heads * chunk * HW * c.head_dim * elem_size(c.dtype) : 0;
  if (one * 2 + qone > s.bytes) {                   // grow the buffers (the only allocation of this API)
    if (cudaStreamSynchronize(st) != cudaSuccess) return REHYAT_ERR_CUDA;
    void** all[3] = {&s.kbuf, &s.vbuf, &s.qbuf};
    for (void** p : all) { cudaFree(*p); *p = nullptr; }
    s.bytes = 0;
    if (cudaMalloc(&s.kbuf, one) != cudaSuccess || cudaMalloc(&s.vbuf, one) != cudaSuccess ||
        (qone && cudaMalloc(&s.qbuf, qone) != cudaSuccess)) { cudaGetLastError(); return REHYAT_ERR_ALLOC; }
    s.bytes = one * 2 + qone;
  }
  s.chunk_cap = (int)(chunk * HW);
  s.active = true;
  s.batch = batch; s.H = H; s.W = W; s.chunk = chunk; s.overlap = overlap;
  s.cap_tokens = (int)cap;
  s.halo = 0; s.has_state = 0; s.chunks_done = 0; s.start = 0; s.tokens_done = 0;
  return REHYAT_OK;
}

int rehyat_stream_step(rehyat_ctx* ctx, const void* q_chunk, const void* k_chunk, const void* v_chunk, void* out_chunk,
                       const rehyat_layout* lay, const rehyat_phi_params* phi, int32_t frames_in_chunk,
                       void* cuda_stream) {
  if (!ctx || !q_chunk || !k_chunk || !v_chunk || !out_chunk || !lay || !phi) return REHYAT_ERR_INVALID_ARG;
  rehyat_ctx::Stream& s = ctx->stream;
  if (!s.active || frames_in_chunk < 1 || frames_in_chunk > s.chunk) return REHYAT_ERR_INVALID_ARG;
  const rehyat_config& c = ctx->cfg;
  if (out_chunk == q_chunk || out_chunk == k_chunk || out_chunk == v_chunk) return REHYAT_ERR_INVALID_ARG;
  const void* ptrs[] = {q_chunk, k_chunk, v_chunk, out_chunk};
  for (const void* p : ptrs)
    if (!aligned16(p)) return REHYAT_ERR_INVALID_ARG;
  if (!phi_pointers_ok(c, phi)) return REHYAT_ERR_INVALID_ARG;
  const long long es = (long long)elem_size(c.dtype);
  const long long strides[] = {lay->stride_batch, lay->stride_head, lay->stride_token};
  for (long long x : strides)
    if (x < 0 || (x * es) % 16 != 0) return REHYAT_ERR_INVALID_ARG;
  if (lay->stride_token < c.head_dim) return REHYAT_ERR_INVALID_ARG;
  if ((c.n_heads > 1 && lay->stride_head < c.head_dim) || (s.batch > 1 && lay->stride_batch < c.head_dim))
    return REHYAT_ERR_INVALID_ARG;
  DeviceGuard guard(c.device);
  if (!guard.ok) return REHYAT_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;

  const int HW = s.H * s.W, Np = frames_in_chunk * HW, h = s.halo, BH = s.batch * c.n_heads;
  const int row_bytes = c.head_dim * (int)es;
  // buffer layout [batch][head][cap_tokens][d]
  const long long sn = c.head_dim, sh = (long long)s.cap_tokens * c.head_dim, sb = sh * c.n_heads;
  // 0. at the end of the buffers the kept frames go back to the front (every few steps)
  if (s.start + h + Np > s.cap_tokens) {
    const long long off = (long long)s.start * sn * es;
    launch_copy_rows2(s.kbuf, s.vbuf, sb * es, sh * es, sn * es, (uint8_t*)s.kbuf + off, (uint8_t*)s.vbuf + off, sb * es, sh * es,
                      sn * es, h, row_bytes, BH, c.n_heads, st);
    s.start = 0;
  }
  uint8_t* kwin = (uint8_t*)s.kbuf + (long long)s.start * sn * es;     // first token of the softmax window
  uint8_t* vwin = (uint8_t*)s.vbuf + (long long)s.start * sn * es;
  // 1. k and v of the chunk go behind the kept frames (they have to outlive the call); q and out stay where they are.
  //    With a q/k transform set, k is normalised and rotated on its way into the window (instead of being copied)
  //    and q into a buffer of its own, both at the positions that follow the chunks processed so far.
  ctx->last_launches = 0;
  const void* q_used = q_chunk;
  if (ctx->qk_on) {
    QkPrepArgs pa = {};
    pa.rows = Np; pa.n_heads = c.n_heads; pa.pos0 = (int)s.tokens_done;
    pa.sb = lay->stride_batch; pa.sh = lay->stride_head; pa.sn = lay->stride_token;
    pa.qn = c.head_dim; pa.qh = (long long)s.chunk_cap * c.head_dim; pa.qb = pa.qh * c.n_heads;
    pa.kb = sb; pa.kh = sh; pa.kn = sn;
    launch_qk_prepare(ctx, q_chunk, k_chunk, s.qbuf, kwin + (long long)h * sn * es, pa, BH, st);
    launch_copy_rows2(vwin + (long long)h * sn * es, nullptr, sb * es, sh * es, sn * es, v_chunk, nullptr,
                      lay->stride_batch * es, lay->stride_head * es, lay->stride_token * es, Np, row_bytes, BH, c.n_heads, st);
    q_used = s.qbuf;
  } else {
    launch_copy_rows2(kwin + (long long)h * sn * es, vwin + (long long)h * sn * es, sb * es, sh * es, sn * es, k_chunk, v_chunk,
                      lay->stride_batch * es, lay->stride_head * es, lay->stride_token * es, Np, row_bytes, BH, c.n_heads, st);
  }
  // 2. Eq. 16 for this chunk: one chunk whose queries are rows [h, h + Np) of the window and whose softmax set
  //    is the whole window
  Geo g;
  g.N = h + Np; g.Np = Np; g.ToHW = h; g.t0 = 0; g.G = 1; g.n_heads = c.n_heads; g.BH = BH;
  g.stride_b = sb; g.stride_h = sh; g.stride_n = sn;
  g.q_shift = h; g.prefix = s.has_state;
  g.ostride_b = lay->stride_batch; g.ostride_h = lay->stride_head; g.ostride_n = lay->stride_token;
  if (g.ostride_h == 0) g.ostride_h = g.ostride_n * Np;
  if (g.ostride_b == 0) g.ostride_b = g.ostride_h * c.n_heads;
  g.qstride_b = g.ostride_b; g.qstride_h = g.ostride_h; g.qstride_n = g.ostride_n;
  if (ctx->qk_on) { g.qstride_n = c.head_dim; g.qstride_h = (long long)s.chunk_cap * c.head_dim; g.qstride_b = g.qstride_h * c.n_heads; }
  g.q_off = h; g.Nq = Np;
  ctx->share_now = nullptr;
  ctx->last_impl = ctx->tensor_ok ? (ctx->tc.phi_ok ? 2 : 1) : 0;
  int rc = run_parts(ctx, q_used, kwin, vwin, out_chunk, phi, g, s.batch, 1, -1, (s.has_state ? PART_READOUT : 0) | PART_WINDOW, st);
  if (rc != REHYAT_OK) return rc;
  // 3. Eq. 17-18: the tokens that leave the window before the next chunk enter the running state
  const int keep = (long long)s.overlap * HW < (long long)h + Np ? s.overlap * HW : h + Np;
  const int leave = h + Np - keep;
  if (leave > 0) {
    Geo gs = g;
    gs.Np = leave; gs.ToHW = 0; gs.q_shift = 0; gs.prefix = 0; gs.t0 = 1; gs.G = 1;   // increment of "chunk 1" = [0, leave)
    const int n_split = pick_state_split(ctx, gs, 1, leave);
    rc = run_parts(ctx, nullptr, kwin, vwin, nullptr, phi, gs, s.batch, n_split, s.has_state ? 0 : -1, PART_STATE, st);
    if (rc != REHYAT_OK) return rc;
    s.has_state = 1;
  }
  // 4. the window moves on: the frames that stay are addressed, not copied
  s.start += leave;
  s.halo = keep;
  s.tokens_done += Np;
  ++s.chunks_done;
  return cudaGetLastError() == cudaSuccess ? REHYAT_OK : REHYAT_ERR_CUDA;
}

size_t rehyat_stream_state_bytes(const rehyat_ctx* ctx) {
  if (!ctx || !ctx->stream.active) return 0;
  return sizeof(StreamHeader) + stream_state_floats(ctx) * sizeof(float) + 2 * stream_halo_bytes(ctx);
}

int rehyat_stream_export(rehyat_ctx* ctx, void* host_buf, size_t capacity, void* cuda_stream) {
  if (!ctx || !host_buf || !ctx->stream.active) return REHYAT_ERR_INVALID_ARG;
  if (capacity < rehyat_stream_state_bytes(ctx)) return REHYAT_ERR_INVALID_ARG;
  const rehyat_config& c = ctx->cfg;
  const rehyat_ctx::Stream& s = ctx->stream;
  DeviceGuard guard(c.device);
  if (!guard.ok) return REHYAT_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaStreamSynchronize(st) != cudaSuccess) return REHYAT_ERR_CUDA;
  StreamHeader hd = {kStreamMagic, 2, c.dtype, c.n_heads, c.head_dim, c.phi_dim, s.batch, s.H, s.W, s.chunk, s.overlap,
                     s.halo, s.has_state, 0, s.chunks_done, s.tokens_done};
  uint8_t* p = (uint8_t*)host_buf;
  memcpy(p, &hd, sizeof(hd));
  p += sizeof(hd);
  const size_t sbytes = stream_state_floats(ctx) * sizeof(float);
  if (s.has_state) {
    if (cudaMemcpy(p, ctx->state, sbytes, cudaMemcpyDeviceToHost) != cudaSuccess) return REHYAT_ERR_CUDA;
  } else {
    memset(p, 0, sbytes);
  }
  p += sbytes;
  const size_t es = elem_size(c.dtype), width = (size_t)s.halo * c.head_dim * es, pitch = (size_t)s.cap_tokens * c.head_dim * es;
  const int BH = s.batch * c.n_heads;
  if (width > 0) {
    const size_t first = (size_t)s.start * c.head_dim * es;          // the kept frames begin at token `start`
    if (cudaMemcpy2D(p, width, (const uint8_t*)s.kbuf + first, pitch, width, BH, cudaMemcpyDeviceToHost) != cudaSuccess) return REHYAT_ERR_CUDA;
    p += width * BH;
    if (cudaMemcpy2D(p, width, (const uint8_t*)s.vbuf + first, pitch, width, BH, cudaMemcpyDeviceToHost) != cudaSuccess) return REHYAT_ERR_CUDA;
  }
  return REHYAT_OK;
}

int rehyat_stream_import(rehyat_ctx* ctx, const void* host_buf, size_t bytes, void* cuda_stream) {
  if (!ctx || !host_buf || bytes < sizeof(StreamHeader)) return REHYAT_ERR_INVALID_ARG;
  const rehyat_config& c = ctx->cfg;
  StreamHeader hd;
  memcpy(&hd, host_buf, sizeof(hd));
  if (hd.magic != kStreamMagic || hd.version != 2 || hd.dtype != c.dtype || hd.n_heads != c.n_heads ||
      hd.head_dim != c.head_dim || hd.phi_dim != c.phi_dim)
    return REHYAT_ERR_INVALID_ARG;
  if (hd.halo < 0 || (long long)hd.halo > (long long)hd.overlap * hd.H * hd.W) return REHYAT_ERR_INVALID_ARG;
  int rc = rehyat_stream_begin(ctx, hd.batch, hd.H, hd.W, hd.chunk, hd.overlap, cuda_stream);
  if (rc != REHYAT_OK) return rc;
  rehyat_ctx::Stream& s = ctx->stream;
  s.halo = hd.halo; s.has_state = hd.has_state ? 1 : 0; s.chunks_done = hd.chunks_done; s.tokens_done = hd.tokens_done;
  if (bytes < rehyat_stream_state_bytes(ctx)) { s.active = false; return REHYAT_ERR_INVALID_ARG; }
  DeviceGuard guard(c.device);
  if (!guard.ok) return REHYAT_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaStreamSynchronize(st) != cudaSuccess) return REHYAT_ERR_CUDA;
  const uint8_t* p = (const uint8_t*)host_buf + sizeof(hd);
  const size_t sbytes = stream_state_floats(ctx) * sizeof(float);
  if (cudaMemcpy(ctx->state, p, sbytes, cudaMemcpyHostToDevice) != cudaSuccess) return REHYAT_ERR_CUDA;
  p += sbytes;
  if (s.has_state && ctx->tensor_ok && ctx->tc.phi_ok) {
    // the bf16 copy of the state that the tensor-core read-out multiplies with: a scan over zero increments
    const size_t per_slot = stream_state_floats(ctx);
    scan_states<<<(unsigned)((per_slot + 255) / 256), 256, 0, st>>>(ctx->partial, ctx->state, per_slot, 1, 0, 0,
                                                                     ctx->tc.state_bf16, c.head_dim);
  }
  const size_t es = elem_size(c.dtype), width = (size_t)s.halo * c.head_dim * es, pitch = (size_t)s.cap_tokens * c.head_dim * es;
  const int BH = s.batch * c.n_heads;
  if (width > 0) {
    if (cudaMemcpy2D(s.kbuf, pitch, p, width, width, BH, cudaMemcpyHostToDevice) != cudaSuccess) return REHYAT_ERR_CUDA;
    p += width * BH;
    if (cudaMemcpy2D(s.vbuf, pitch, p, width, width, BH, cudaMemcpyHostToDevice) != cudaSuccess) return REHYAT_ERR_CUDA;
  }
  return cudaStreamSynchronize(st) == cudaSuccess ? REHYAT_OK : REHYAT_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Forward pass for callers that may not allocate device memory.
// ---------------------------------------------------------------------------------------------
// The workspace of the SIMT kernels (chunk states, partial state sums, linear read-out) lives in
// this fixed array instead of cudaMalloc'ed buffers.  Every GPU that loads the library holds the
// 8 MiB until the process exits.  All calls share it and it keeps the previous call's contents;
// nothing relies on it starting at zero, because every word a call reads it has written earlier
// in the same call.
constexpr size_t kStaticScratchFloats = (size_t)2 << 20;
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

// In host code `g_static_scratch` is only a handle of the symbol, not a device address, so the
// address is looked up once per device (with that device current) and cached.
constexpr int kMaxDevices = 64;
static float* g_static_scratch_addr[kMaxDevices] = {};
static unsigned g_static_attr_done[kMaxDevices] = {};     // bit (2*dtype + (head_dim == 128)): kernel attributes set
static std::mutex g_static_scratch_mutex;

// First call on a device (with that device current): checks that it exists and is an sm_100 part, looks up the
// array's address and sets the attributes of the kernels this dtype / head_dim uses.  Later calls only read.
static int static_device_setup(int device, int dtype, int head_dim, float** out) {
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (!g_static_scratch_addr[device]) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { cudaGetLastError(); return REHYAT_ERR_CUDA; }
    if (prop.major != 10) return REHYAT_ERR_ARCH;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return REHYAT_ERR_CUDA; }
    g_static_scratch_addr[device] = static_cast<float*>(p);
  }
  const unsigned bit = 1u << (2 * (dtype == REHYAT_DTYPE_FP32 ? 1 : 0) + (head_dim == 128 ? 1 : 0));
  if (!(g_static_attr_done[device] & bit)) {
    const int rc = set_simt_attributes_for(dtype, head_dim);
    if (rc != REHYAT_OK) { cudaGetLastError(); return rc; }
    g_static_attr_done[device] |= bit;
  }
  *out = g_static_scratch_addr[device];
  return REHYAT_OK;
}

size_t rehyat_static_scratch_bytes(void) { return kStaticScratchFloats * sizeof(float); }

int rehyat_forward_static(const rehyat_config* cfg, const void* q, const void* k, const void* v, void* out,
                          const rehyat_layout* lay, const rehyat_phi_params* phi, int32_t batch, int32_t frames,
                          int32_t H, int32_t W, int32_t chunk, int32_t overlap, void* cuda_stream) {
  if (!cfg) return REHYAT_ERR_INVALID_ARG;
  int rc = check_config(cfg);
  if (rc != REHYAT_OK) return rc;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess) { cudaGetLastError(); return REHYAT_ERR_CUDA; }
  if (cfg->device < 0 || cfg->device >= ndev || cfg->device >= kMaxDevices) return REHYAT_ERR_INVALID_ARG;
  if (cfg->bidirectional) return REHYAT_ERR_UNSUPPORTED;
  if (batch < 1 || frames < 1 || H < 1 || W < 1 || chunk < 1 || overlap < 0) return REHYAT_ERR_INVALID_ARG;
  const long long HW = (long long)H * W, N = HW * frames;
  if (N > (1 << 24)) return REHYAT_ERR_TOO_LARGE;
  const int chunk_eff = chunk < frames ? chunk : frames;
  const long long n_chunks = (frames + chunk_eff - 1) / chunk_eff;
  const long long Np = chunk_eff * HW;
  const long long BH = (long long)batch * cfg->n_heads, SD = cfg->head_dim + 4;
  if (n_chunks > 16 || BH > 65535) return REHYAT_ERR_TOO_LARGE;
  const long long slot = BH * cfg->phi_dim * SD;                 // one chunk state, floats
  const long long rd_rows = n_chunks * Np;                       // all chunks form one group
  const long long rd_cap = n_chunks * ((Np + 127) / 128 * 128);  // whole 128-row tiles per chunk
  const long long need = 2 * n_chunks * slot + BH * rd_cap * SD;
  if (need > (long long)kStaticScratchFloats) return REHYAT_ERR_TOO_LARGE;

  DeviceGuard guard(cfg->device);
  if (!guard.ok) return REHYAT_ERR_CUDA;
  float* base = nullptr;
  rc = static_device_setup(cfg->device, cfg->dtype, cfg->head_dim, &base);
  if (rc != REHYAT_OK) return rc;

  // A context on the stack that points into the static array; the SIMT kernels do the work.
  rehyat_ctx tmp;
  tmp.cfg = *cfg;
  tmp.cfg.impl = REHYAT_IMPL_SIMT;
  tmp.cfg.max_batch = batch;
  tmp.cfg.max_tokens_per_frame = (int32_t)HW;
  tmp.cfg.max_chunk_frames = chunk_eff;
  tmp.state = base;
  tmp.partial = base + n_chunks * slot;
  tmp.readout = base + 2 * n_chunks * slot;
  tmp.Gmax = (int)n_chunks;
  tmp.partial_units = (int)n_chunks;
  tmp.rd_rows = (int)rd_rows;
  tmp.rd_cap = (int)rd_cap;
  tmp.bh_max = (int)BH;
  tmp.tensor_ok = false;
  return rehyat_forward(&tmp, q, k, v, out, lay, phi, batch, frames, H, W, chunk, overlap, cuda_stream);
}

}  // extern "C"
