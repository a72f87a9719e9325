/*
 * rehyat.h - C ABI of the ReHyAt recurrent hybrid attention operator for NVIDIA B200 (sm_100a).
 *
 * The operator (paper Section 3.2 "Hybrid Attention Formulation" and Section 3.3 "Recurrent
 * HyAt"): N = frames*H*W tokens of a video latent are cut into temporal chunks of `chunk`
 * frames.  A query i of chunk t attends
 *   - with exact softmax weights exp(q_i.k_j/sqrt(head_dim) - c_i) to the keys of its window
 *     TS_t = [max(t*N' - overlap*H*W, 0), min((t+1)*N', N)),  N' = chunk*H*W       (Eq. 12/13)
 *   - with linear-attention weights phi_q(q_i).phi_k(k_j) to every earlier key
 *     TL_t = [0, max(t*N' - overlap*H*W, 0))                                          (Eq. 13)
 * and the output is  y_i = (aS_i + aL_i) / (nS_i + nL_i)                          (Eq. 5-9),
 * the linear sums being carried from chunk to chunk as the state
 *   s_t = sum_{j in TL_t} phi_k(k_j) v_j^T,   z_t = sum_{j in TL_t} phi_k(k_j)    (Eq. 14-18).
 * phi_q, phi_k (Section 3.2 "Characterization of phi", Appendix "Training Details"): per-head
 * two-layer MLP u = act_out(W2 act_hidden(W1 x + b1) + b2), u split into poly_degree equal
 * contiguous parts, part p (1-based) raised element-wise to the power p, parts concatenated.
 *
 * Conventions
 *   - All functions return REHYAT_OK (0) or a negative REHYAT_ERR_* code; nothing throws.
 *   - Unless a parameter says "host", tensor pointers are DEVICE pointers owned by the caller,
 *     16-byte aligned, and `out` must not alias an input.
 *   - rehyat_forward only enqueues work on the given stream: no host synchronisation and no
 *     allocation, in the causal and in the bidirectional form.  A context serves one stream at a
 *     time (it owns the workspace).  The library keeps no process-wide state and reads no
 *     environment variable.
 *   - There is no CPU fallback: on a machine without an sm_100 device rehyat_create fails.
 */
#ifndef REHYAT_H
#define REHYAT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define REHYAT_OK                   0
#define REHYAT_ERR_INVALID_ARG     -1   /* null / misaligned pointer, size out of range        */
#define REHYAT_ERR_UNSUPPORTED     -2   /* legal request this build has no kernel for          */
#define REHYAT_ERR_CUDA            -3   /* a CUDA runtime or driver call failed                */
#define REHYAT_ERR_ARCH            -4   /* the device is not compute capability 10.x           */
#define REHYAT_ERR_ALLOC           -5   /* workspace allocation failed                         */
#define REHYAT_ERR_DEVICE_TIMEOUT  -6   /* a bounded wait inside a kernel ran out (see status) */
#define REHYAT_ERR_TOO_LARGE       -7   /* rehyat_forward_static: problem exceeds its fixed scratch */

typedef enum { REHYAT_DTYPE_BF16 = 0, REHYAT_DTYPE_FP32 = 1 } rehyat_dtype;

/* Activations of the phi MLP.  The paper names none; ReLU/ReLU is the default reading. */
typedef enum {
  REHYAT_ACT_RELU = 0, REHYAT_ACT_IDENTITY = 1, REHYAT_ACT_SOFTPLUS = 2,
  REHYAT_ACT_ELU1 = 3 /* 1 + elu(x) */, REHYAT_ACT_GELU = 4 /* erf form */
} rehyat_act;

/* The stabilising constant c of Eq. 6 and 8.  It is NOT applied to the linear terms (Eq. 7, 9),
 * so the result depends on it.  ROWMAX: c_i = max over the window of the scaled logits of row i
 * ("typically the maximum exponent").  ZERO: c = 0 (evaluated stably). */
typedef enum { REHYAT_C_ROWMAX = 0, REHYAT_C_ZERO = 1 } rehyat_c_mode;

/* Kernel family.  AUTO: tensor-core (tcgen05) kernels when dtype is bf16 (head_dim 64 or 128 for
 * the softmax window; for phi, state and read-out also D_h and D' multiples of 32 with
 * 64 <= D_h <= 256, 32 <= D' <= 256; other widths keep the window on the tensor cores and run
 * the linear branch on the fp32 kernels), SIMT fp32 kernels otherwise.  SIMT / TENSOR force one (TENSOR fails with REHYAT_ERR_UNSUPPORTED
 * where it does not apply).  TENSOR_WINDOW: tensor-core window, SIMT linear branch (a cross-check). */
typedef enum {
  REHYAT_IMPL_AUTO = 0, REHYAT_IMPL_SIMT = 1, REHYAT_IMPL_TENSOR = 2, REHYAT_IMPL_TENSOR_WINDOW = 3
} rehyat_impl;

typedef struct rehyat_config {
  int32_t device;               /* CUDA device ordinal                                        */
  int32_t dtype;                /* rehyat_dtype of q, k, v, out and the phi parameters        */
  int32_t n_heads;
  int32_t head_dim;             /* d: 64 or 128                                               */
  int32_t phi_hidden;           /* D_h, hidden width of the phi MLP (<= 256, multiple of 8)   */
  int32_t phi_dim;              /* D', output width of phi (<= 256, divisible by poly_degree) */
  int32_t poly_degree;          /* P in 1..4                                                  */
  int32_t act_hidden;           /* rehyat_act                                                 */
  int32_t act_out;              /* rehyat_act                                                 */
  int32_t c_mode;               /* rehyat_c_mode                                              */
  int32_t impl;                 /* rehyat_impl                                                */
  int32_t max_batch;            /* largest `batch` a forward call may pass                    */
  int32_t max_tokens_per_frame; /* largest H*W                                                */
  int32_t max_chunk_frames;     /* largest `chunk`                                            */
  int32_t group_tokens;         /* 0 = default.  Queries per (batch, head) that one pass over
                                   a group of chunks handles; the workspace grows with it and
                                   with max_chunk_frames*max_tokens_per_frame, never with
                                   `frames`.                                                  */
  int32_t bidirectional;        /* 0 (default): causal linear branch, TL_t = tokens before the
                                   window (Eq. 13), the recurrent form.  1: TL_t = every token
                                   outside the window, earlier AND later (Eq. 10-12), the form
                                   the paper distils first.  Not a recurrence: rehyat_forward
                                   then keeps one state per latent frame ((max_frames+1) x 132 KB
                                   per (batch, head) at d=128, D'=256), allocated by
                                   rehyat_create; rehyat_stream_* and rehyat_forward_static
                                   refuse it (REHYAT_ERR_UNSUPPORTED).                         */
  int32_t max_frames;           /* bidirectional = 1 only: largest `frames` a forward call may
                                   pass (>= 1).  Ignored, and may be 0, in the causal form,
                                   whose memory does not depend on the video length.          */
  int32_t exp_poly;             /* tensor-core window kernel: of every four pairs of softmax
                                   exponentials, how many are evaluated as a cubic on the FMA
                                   pipe instead of the special-function unit.  0 = the
                                   library's choice (1, the fastest measured on B200), 1..3 =
                                   that many, -1 = none.  Results agree within bf16 rounding. */
  int32_t phi_layers;           /* layers of the phi MLP: 0 or 2 = the two-layer map of the paper's
                                   experiments; 3 or 4 = one or two further hidden layers
                                   h <- act_hidden(Wmid h + bmid) of width D_h between the two
                                   (Section 4.3 varies the "transformation complexity" of phi).
                                   The tensor-core kernels cover them too.                     */
  int32_t qk_transform;         /* 1: the context can normalise and rotate q and k ahead of the
                                   operator (rehyat_set_qk_transform); rehyat_create then also
                                   allocates room for the transformed q and k of max_frames
                                   frames (max_frames >= 1 required).  0: q and k are used as
                                   given.                                                      */
  int32_t window_tiles;         /* tensor-core window kernel: 128-row query tiles per work
                                   item.  0 = chosen per launch from how many items there are
                                   for the SMs; 1 or 2 fixes it (same results up to the order
                                   of fp32 sums).                                              */
} rehyat_config;

/* Element strides of q, k, v and out (all four share them); the head_dim axis is contiguous.
 * [B, n_heads, N, d] contiguous: {n_heads*N*d, N*d, d};  [B, N, n_heads, d]: {N*n_heads*d, d,
 * n_heads*d}.  Each stride times the element size must be a multiple of 16 bytes. */
typedef struct rehyat_layout {
  int64_t stride_batch;
  int64_t stride_head;
  int64_t stride_token;
} rehyat_layout;

/* Device pointers to the parameters of phi_q and phi_k in the operator dtype, row-major:
 * W1 [n_heads, D_h, d], b1 [n_heads, D_h], W2 [n_heads, D', D_h], b2 [n_heads, D'] (W2, b2: the LAST layer),
 * and with phi_layers = L > 2 the hidden layers in between, in the order they are applied:
 * Wmid [n_heads, L-2, D_h, D_h], bmid [n_heads, L-2, D_h] (ignored, and may be NULL, for two layers). */
typedef struct rehyat_phi_params {
  const void* q_W1; const void* q_b1; const void* q_W2; const void* q_b2;
  const void* k_W1; const void* k_b1; const void* k_W2; const void* k_b2;
  const void* q_Wmid; const void* q_bmid; const void* k_Wmid; const void* k_bmid;
} rehyat_phi_params;

typedef struct rehyat_ctx rehyat_ctx;

/* Creates a context on cfg->device and allocates its fixed workspace (chunk states, partial
 * state sums, the linear read-out of one chunk group, a status word).  The workspace size is a
 * function of the config only (Section 3.3, note 3: memory constant in the video length).
 * In the bidirectional form it also allocates the per-frame states for max_frames frames.
 * Nothing is read from the environment: every tuning knob is a field of the config.
 * Errors: INVALID_ARG (null, sizes out of range), UNSUPPORTED, ARCH, CUDA, ALLOC. */
int rehyat_create(rehyat_ctx** out, const rehyat_config* cfg);

/* Enqueues the operator of Eq. 5-9 with the causal sets of Eq. 13 on `cuda_stream`
 * (a cudaStream_t passed as void*; NULL is the default stream).
 *   q, k, v  device, [batch, n_heads, frames*H*W, head_dim] through `lay`, read only
 *   out      device, same shape and strides, written
 *   H, W     the latent patch grid (tokens per frame = H*W), not attention heads
 *   chunk    T_c >= 1 frames per chunk; frames need not be a multiple (the last chunk is short)
 *   overlap  T_o >= 0 frames of overlap; any value is legal, the window is clamped at token 0
 * Validation failures return INVALID_ARG before anything is enqueued.  Asynchronous errors
 * (a bounded device wait that ran out) are reported by rehyat_status. */
int rehyat_forward(rehyat_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                   const rehyat_layout* lay, const rehyat_phi_params* phi,
                   int32_t batch, int32_t frames, int32_t H, int32_t W,
                   int32_t chunk, int32_t overlap, void* cuda_stream);

/* Same operator with q, k, v, out in HOST memory as contiguous [batch, n_heads, N, head_dim]
 * (pinned memory makes the copies asynchronous).  Copies the inputs to device staging buffers
 * owned by the context (grown on demand: the one allocation whose size follows N, because it
 * holds the tensors themselves), runs the operator, copies `out` back and synchronises the
 * stream.  The (batch, head) problems are independent, so the call is pipelined over groups of heads
 * on two extra streams of the context: one group is copied in and another copied out while a third
 * is computed.  `phi` stays device-resident. */
int rehyat_forward_host(rehyat_ctx* ctx, const void* q_host, const void* k_host,
                        const void* v_host, void* out_host, const rehyat_phi_params* phi,
                        int32_t batch, int32_t frames, int32_t H, int32_t W,
                        int32_t chunk, int32_t overlap, void* cuda_stream);

/* Chunk-by-chunk processing: the recurrent form of Section 3.3 (Eq. 14-18) with the state kept by the
 * context, for callers that produce or hold one chunk of the video at a time.  Device memory then scales
 * with one chunk plus the overlap, not with the video (Section 3.3, note 3).
 *
 * rehyat_stream_begin starts a sequence (s_0 = 0, z_0 = 0, Eq. 14-15) for chunks of at most `chunk` frames
 * with `overlap` frames of overlap, and sizes two buffers (k and v) of (overlap + 4*chunk)*H*W tokens per
 * (batch, head) - more chunks where overlap > 3*chunk: the only allocation of this API, repeated only when a
 * later sequence needs more.  The softmax window slides through these buffers: a step appends its chunk's k and
 * v behind the kept overlap frames, the frames that stay are addressed rather than moved, and only at the end
 * of the buffers (every few steps) are they copied back to the front.  q and out are read and written in place.
 * rehyat_stream_step takes the next chunk,
 *   q_chunk, k_chunk, v_chunk, out_chunk   device, [batch, n_heads, frames_in_chunk*H*W, head_dim] through `lay`
 *   frames_in_chunk                        1..chunk; only the last chunk of a video may be shorter than `chunk`
 * computes its output from the softmax window (the overlap frames kept from earlier chunks plus the chunk,
 * Eq. 12-13) and the running state (Eq. 16), then folds the tokens that leave the window into the state
 * (Eq. 17-18, new tokens only).  Asynchronous on `cuda_stream`; the same stream must be used for all steps
 * of a sequence.  rehyat_forward on the same context ends the sequence (both use the context's workspace).
 *
 * rehyat_stream_export writes the sequence's state (a small header, s and z in fp32, the overlap frames of
 * k and v) to HOST memory after synchronising the stream; rehyat_stream_state_bytes is its size right now.
 * rehyat_stream_import starts a sequence from such a blob on any context with the same dtype, head count,
 * head_dim and phi_dim: a checkpoint.  A resumed sequence continues bit-for-bit.
 * Errors: INVALID_ARG (no active sequence, sizes beyond the context's max_* fields, a blob that does not
 * match), ALLOC, CUDA. */
int rehyat_stream_begin(rehyat_ctx* ctx, int32_t batch, int32_t H, int32_t W, int32_t chunk, int32_t overlap,
                        void* cuda_stream);
int rehyat_stream_step(rehyat_ctx* ctx, const void* q_chunk, const void* k_chunk, const void* v_chunk,
                       void* out_chunk, const rehyat_layout* lay, const rehyat_phi_params* phi,
                       int32_t frames_in_chunk, void* cuda_stream);
size_t rehyat_stream_state_bytes(const rehyat_ctx* ctx);
int rehyat_stream_export(rehyat_ctx* ctx, void* host_buf, size_t capacity, void* cuda_stream);
int rehyat_stream_import(rehyat_ctx* ctx, const void* host_buf, size_t bytes, void* cuda_stream);

/* The same operator for callers that must not allocate device memory: code that runs inside a
 * memory plan fixed up front (all device memory already handed to another allocator or pool), a
 * latency-critical loop that cannot afford the device-wide synchronisation cudaMalloc / cudaFree
 * imply, or a plug-in whose host forbids allocation calls.  (The paper has no counterpart: this is
 * a convenience of the library, not a step of the method.)
 *
 * No context is needed.  The workspace that rehyat_create would allocate (chunk states, partial
 * state sums, linear read-out) is a fixed 8 MiB array inside the library
 * (rehyat_static_scratch_bytes), which every GPU that loads the library keeps until the process
 * ends.  The SIMT fp32-arithmetic kernels do the work for both dtypes.  The call uses no
 * cudaMalloc, cudaFree or any allocating routine.
 *   cfg      device, dtype, n_heads, head_dim, phi_*, poly_degree, act_*, c_mode are used; impl,
 *            max_* and group_tokens are ignored
 *   others   as rehyat_forward (device pointers, caller-owned; asynchronous on `cuda_stream`)
 * Limits: at most 16 chunks, and  2*chunks*B*n_heads*D'*(d+4) + B*n_heads*chunks*ceil(N'/128)*128*(d+4)
 * floats must fit the array; larger problems return REHYAT_ERR_TOO_LARGE and launch nothing.
 * The first call on each device looks up the array's device address and sets kernel attributes;
 * make that first call before any stream capture begins.  All calls share the one array, which
 * keeps the last call's contents (nothing needs it zeroed: a call writes every word before it
 * reads it), so two calls that overlap on the GPU - different streams, or different threads -
 * race; serialise them. */
int rehyat_forward_static(const rehyat_config* cfg, const void* q, const void* k, const void* v, void* out,
                          const rehyat_layout* lay, const rehyat_phi_params* phi,
                          int32_t batch, int32_t frames, int32_t H, int32_t W,
                          int32_t chunk, int32_t overlap, void* cuda_stream);
size_t rehyat_static_scratch_bytes(void);

/* What a DiT block does to q and k between its projections and the attention operator (the block of Eq. 1
 * around A_l, which the paper takes over from the pretrained model): per-head RMS normalisation
 *   x <- x / sqrt(mean_d(x^2) + norm_eps) * weight        (weight [n_heads, head_dim], or NULL for none)
 * followed by the rotary embedding from caller-supplied tables: the pair (x[2i], x[2i+1]) of token n is turned by
 * the angle with cosine rope_cos[n*head_dim/2 + i] and sine rope_sin[n*head_dim/2 + i] (how the angles follow from
 * the frame / row / column of a token is the caller's business).  Either step can be left out (rms_norm = 0;
 * rope_cos = NULL).  All pointers are device pointers that must stay valid while the transform is set; the
 * tables are fp32 and cover the frames*H*W tokens of every forward call that follows.
 *
 * rehyat_set_qk_transform(ctx, t) switches it on for the rehyat_forward calls that follow (a context made with
 * qk_transform = 1, frames <= max_frames; q, k must be laid out so that the last element of the batch lies
 * within max_batch*n_heads*max_frames*max_tokens_per_frame*head_dim elements of the first), t = NULL switches
 * it off.  Each call then runs one more kernel, bound by HBM, that writes the transformed q and k into the
 * context's buffers; both branches (softmax window and phi) see the transformed tensors; v is untouched.
 * rehyat_stream_step applies it chunk by chunk: k is normalised and rotated on its way into the window buffer
 * (in place of the copy it needs anyway), q into a buffer of one chunk; the tables are read at the positions
 * that follow the tokens of the chunks processed so far, so they must cover the whole sequence, and the kept
 * frames inside an exported state are the transformed ones (resume with the same transform set).
 * rehyat_forward_host returns REHYAT_ERR_UNSUPPORTED while a transform is set. */
typedef struct rehyat_qk_transform {
  const void* q_norm_weight;    /* [n_heads, head_dim], operator dtype, or NULL */
  const void* k_norm_weight;
  int32_t rms_norm;             /* 1: normalise, 0: skip the normalisation (the weights are then ignored) */
  float norm_eps;
  const float* rope_cos;        /* [frames*H*W, head_dim/2] fp32, or NULL: no rotation */
  const float* rope_sin;
} rehyat_qk_transform;
int rehyat_set_qk_transform(rehyat_ctx* ctx, const rehyat_qk_transform* t);

/* Frees the workspace.  NULL is a no-op returning REHYAT_OK. */
int rehyat_destroy(rehyat_ctx* ctx);

/* Bytes of device workspace the context holds (staging of rehyat_forward_host excluded). */
size_t rehyat_workspace_bytes(const rehyat_ctx* ctx);

/* Synchronises `cuda_stream`, reads the device status word and clears it.  Returns REHYAT_OK,
 * REHYAT_ERR_DEVICE_TIMEOUT or REHYAT_ERR_CUDA.
 * Every wait inside the tensor-core kernels (on an mbarrier: for a TMA load, a tcgen05.mma, another
 * role of the CTA) is bounded in wall time.  A wait that runs out makes its CTA stop issuing work,
 * wait for what it has already put in flight, free its TMEM and return; the other CTAs of the same
 * launch follow at their next wait.  The output of that launch is then undefined, the status word
 * records the time-out until it is read here, and later launches are not affected. */
int rehyat_status(rehyat_ctx* ctx, void* cuda_stream);

/* Sets the bound of those waits for the launches that follow: wait_limit_us microseconds
 * (0 = the default of one second).  withhold_loads is a test hook, 0 in production: non-zero makes
 * the producers of the tensor-core kernels issue no loads at all, so that every launch runs into
 * the bound with nothing in flight - the way to exercise the time-out path without a fault. */
int rehyat_set_wait_limit(rehyat_ctx* ctx, int32_t wait_limit_us, int32_t withhold_loads);

/* Number of kernel launches the last rehyat_forward on this context enqueued. */
int rehyat_last_launches(const rehyat_ctx* ctx);

/* Kernels of the last forward: 2 = every step on the tensor cores, 1 = the softmax window on the tensor cores
 * and phi, state and read-out on the fp32 SIMT kernels (phi widths the tensor-core kernels do not cover, or
 * REHYAT_IMPL_TENSOR_WINDOW), 0 = SIMT kernels throughout. */
int rehyat_last_impl(const rehyat_ctx* ctx);

/* Query tiles per work item of the last tensor-core window launch: 2 (window_tc) or 1 (window_tc1);
 * 0 after a forward on the SIMT kernels. */
int rehyat_last_window_tiles(const rehyat_ctx* ctx);

/* Diagnostic output for measurement.  `share` is a device buffer of batch*n_heads*frames*H*W floats
 * (caller-owned, 16-byte aligned), or NULL to switch it off.  While set, every rehyat_forward also
 * writes, for query i of (batch b, head h) at share[(b*n_heads + h)*N + i], the part of the joint
 * normaliser of Eq. 5 that comes from the linear branch, nL_i / (nS_i + nL_i) with both terms as the
 * kernel weighs them (Eq. 8, 9; 0 for chunks with an empty linear set).  Not written by
 * rehyat_forward_host or rehyat_stream_step. */
int rehyat_set_linear_share_output(rehyat_ctx* ctx, float* share);

/* Per-kernel timing for measurement.  While enabled, every kernel launch of rehyat_forward is
 * bracketed by CUDA events recorded on the launching stream (a few microseconds of overhead per
 * launch).  rehyat_profile_read waits for the recorded events, writes the summed milliseconds and
 * the launch counts of each kernel kind into ms[REHYAT_PROF_KINDS] / launches[REHYAT_PROF_KINDS]
 * (host arrays) and clears the record.  Read at least once per few hundred forwards. */
#define REHYAT_PROF_STATE   0   /* phi_k + chunk-state increments (Eq. 17-18)    */
#define REHYAT_PROF_SCAN    1   /* running sum along the chunk axis (Eq. 14-15) */
#define REHYAT_PROF_READOUT 2   /* phi_q + linear read-out (Eq. 7, 9)            */
#define REHYAT_PROF_WINDOW  3   /* softmax window + joint normaliser (Eq. 5-8)   */
#define REHYAT_PROF_QKPREP  4   /* q/k normalisation + rotation, when set         */
#define REHYAT_PROF_KINDS   5
int rehyat_profile_enable(rehyat_ctx* ctx, int on);
int rehyat_profile_read(rehyat_ctx* ctx, double* ms, int32_t* launches);

const char* rehyat_strerror(int code);
int rehyat_version(void);

#ifdef __cplusplus
}
#endif
#endif /* REHYAT_H */
