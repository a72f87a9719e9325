"""Thin ctypes binding of librehyat.so (include/rehyat.h).  Argument marshalling only: every step
of the operator runs inside the library's CUDA kernels.  PyTorch supplies device memory and
streams, nothing else.  There is no fallback: a missing library raises."""
from __future__ import annotations

import ctypes as C
import os

import torch

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "librehyat.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_ARCH, ERR_ALLOC, ERR_DEVICE_TIMEOUT = 0, -1, -2, -3, -4, -5, -6
ERR_TOO_LARGE = -7
DTYPE = {"bf16": 0, "fp32": 1}
ACT = {"relu": 0, "identity": 1, "softplus": 2, "elu1": 3, "gelu": 4}
C_MODE = {"rowmax": 0, "zero": 1}
IMPL = {"auto": 0, "simt": 1, "tensor": 2, "tensor_window": 3}

EXPORTS = ["rehyat_create", "rehyat_forward", "rehyat_forward_host", "rehyat_forward_static",
           "rehyat_static_scratch_bytes", "rehyat_destroy",
           "rehyat_stream_begin", "rehyat_stream_step", "rehyat_stream_state_bytes", "rehyat_stream_export",
           "rehyat_stream_import",
           "rehyat_workspace_bytes", "rehyat_status", "rehyat_set_wait_limit", "rehyat_last_launches", "rehyat_last_impl",
           "rehyat_last_window_tiles", "rehyat_set_linear_share_output", "rehyat_set_qk_transform",
           "rehyat_profile_enable", "rehyat_profile_read", "rehyat_strerror", "rehyat_version"]
PROF_KINDS = ("state", "scan", "readout", "window", "qk_prep")


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "device", "dtype", "n_heads", "head_dim", "phi_hidden", "phi_dim", "poly_degree", "act_hidden",
        "act_out", "c_mode", "impl", "max_batch", "max_tokens_per_frame", "max_chunk_frames", "group_tokens",
        "bidirectional", "max_frames", "exp_poly", "phi_layers", "qk_transform", "window_tiles")]


# Values of the tuning fields of rehyat_config that a Rehyat(...) call does not name (0 = the library's choice).
TUNING_DEFAULTS = {"exp_poly": 0, "window_tiles": 0}


class Layout(C.Structure):
    _fields_ = [("stride_batch", C.c_int64), ("stride_head", C.c_int64), ("stride_token", C.c_int64)]


class QkTransform(C.Structure):
    _fields_ = [("q_norm_weight", C.c_void_p), ("k_norm_weight", C.c_void_p), ("rms_norm", C.c_int32),
                ("norm_eps", C.c_float), ("rope_cos", C.c_void_p), ("rope_sin", C.c_void_p)]


class PhiParams(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("q_W1", "q_b1", "q_W2", "q_b2", "k_W1", "k_b1", "k_W2", "k_b2",
                                          "q_Wmid", "q_bmid", "k_Wmid", "k_bmid")]


_lib = None


def lib():
    """Loads librehyat.so on first use.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2601_04342_b200.build`; "
                               "there is no fallback path")
        L = C.CDLL(LIB_PATH)
        L.rehyat_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(Config)]
        L.rehyat_forward.argtypes = [C.c_void_p] + [C.c_void_p] * 4 + [C.POINTER(Layout), C.POINTER(PhiParams)] + \
            [C.c_int32] * 6 + [C.c_void_p]
        L.rehyat_forward_host.argtypes = [C.c_void_p] + [C.c_void_p] * 4 + [C.POINTER(PhiParams)] + \
            [C.c_int32] * 6 + [C.c_void_p]
        L.rehyat_forward_static.argtypes = [C.POINTER(Config)] + [C.c_void_p] * 4 + \
            [C.POINTER(Layout), C.POINTER(PhiParams)] + [C.c_int32] * 6 + [C.c_void_p]
        L.rehyat_static_scratch_bytes.argtypes = []
        L.rehyat_static_scratch_bytes.restype = C.c_size_t
        L.rehyat_destroy.argtypes = [C.c_void_p]
        L.rehyat_stream_begin.argtypes = [C.c_void_p] + [C.c_int32] * 5 + [C.c_void_p]
        L.rehyat_stream_step.argtypes = [C.c_void_p] + [C.c_void_p] * 4 + [C.POINTER(Layout), C.POINTER(PhiParams),
                                                                          C.c_int32, C.c_void_p]
        L.rehyat_stream_state_bytes.argtypes = [C.c_void_p]
        L.rehyat_stream_state_bytes.restype = C.c_size_t
        L.rehyat_stream_export.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.rehyat_stream_import.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.rehyat_workspace_bytes.argtypes = [C.c_void_p]
        L.rehyat_workspace_bytes.restype = C.c_size_t
        L.rehyat_status.argtypes = [C.c_void_p, C.c_void_p]
        L.rehyat_set_wait_limit.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        L.rehyat_last_launches.argtypes = [C.c_void_p]
        L.rehyat_last_impl.argtypes = [C.c_void_p]
        L.rehyat_last_window_tiles.argtypes = [C.c_void_p]
        L.rehyat_set_linear_share_output.argtypes = [C.c_void_p, C.c_void_p]
        L.rehyat_set_qk_transform.argtypes = [C.c_void_p, C.POINTER(QkTransform)]
        L.rehyat_profile_enable.argtypes = [C.c_void_p, C.c_int]
        L.rehyat_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int32)]
        L.rehyat_strerror.argtypes = [C.c_int]
        L.rehyat_strerror.restype = C.c_char_p
        for name in EXPORTS:
            if getattr(L, name).restype is None:
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


class RehyatError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {lib().rehyat_strerror(code).decode()} ({code})")


def _check(code, where):
    if code != OK:
        raise RehyatError(code, where)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(None)


class Rehyat:
    """One operator context (rehyat_create ... rehyat_destroy)."""

    def __init__(self, *, n_heads, head_dim, dtype="bf16", phi_hidden=None, phi_dim=None, poly_degree=2,
                 act_hidden="relu", act_out="relu", c_mode="rowmax", impl="auto", max_batch=1,
                 max_tokens_per_frame=1560, max_chunk_frames=3, group_tokens=0, device=0, bidirectional=False,
                 max_frames=0, phi_layers=2, qk_transform=False, **tuning):
        unknown = set(tuning) - set(TUNING_DEFAULTS)
        if unknown:
            raise TypeError(f"unknown arguments {sorted(unknown)}")
        tune = {**TUNING_DEFAULTS, **tuning}
        self.cfg = Config(device, DTYPE[dtype], n_heads, head_dim, phi_hidden or 2 * head_dim,
                          phi_dim or 2 * head_dim, poly_degree, ACT[act_hidden], ACT[act_out], C_MODE[c_mode],
                          IMPL[impl], max_batch, max_tokens_per_frame, max_chunk_frames, group_tokens,
                          int(bool(bidirectional)), max_frames, int(tune["exp_poly"]), phi_layers, int(bool(qk_transform)),
                          int(tune["window_tiles"]))
        self.dtype = dtype
        self._h = C.c_void_p(None)
        _check(lib().rehyat_create(C.byref(self._h), C.byref(self.cfg)), "rehyat_create")

    def close(self):
        if self._h:
            lib().rehyat_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def workspace_bytes(self):
        return lib().rehyat_workspace_bytes(self._h)

    @property
    def last_launches(self):
        return lib().rehyat_last_launches(self._h)

    @property
    def last_impl(self):
        return "tensor" if lib().rehyat_last_impl(self._h) else "simt"

    @property
    def last_phi_impl(self):
        """Kernels of phi, state and read-out in the last forward."""
        return "tensor" if lib().rehyat_last_impl(self._h) == 2 else "simt"

    @property
    def last_window_tiles(self):
        return lib().rehyat_last_window_tiles(self._h)

    def set_linear_share_output(self, share):
        """share: float32 CUDA tensor [B, n_heads, N] the window kernels fill with nL / (nS + nL), or None."""
        _check(lib().rehyat_set_linear_share_output(self._h, _ptr(share)), "rehyat_set_linear_share_output")

    def set_qk_transform(self, *, q_weight=None, k_weight=None, rms_norm=True, eps=1e-6, cos=None, sin=None, off=False):
        """rehyat_set_qk_transform: per-head RMS normalisation (weights [n_heads, d] CUDA tensors in the operator
        dtype, or None) and / or the rotary embedding from fp32 CUDA tables cos, sin [N, d/2].  off=True: as given."""
        if off:
            _check(lib().rehyat_set_qk_transform(self._h, None), "rehyat_set_qk_transform")
            self._qk_keep = None
            return
        t = QkTransform(_ptr(q_weight), _ptr(k_weight), int(bool(rms_norm)), float(eps), _ptr(cos), _ptr(sin))
        _check(lib().rehyat_set_qk_transform(self._h, C.byref(t)), "rehyat_set_qk_transform")
        self._qk_keep = (q_weight, k_weight, cos, sin)         # the library keeps the pointers, not the tensors

    @staticmethod
    def phi_struct(phi_q, phi_k):
        return PhiParams(*[_ptr(phi_q[n]) for n in ("W1", "b1", "W2", "b2")],
                         *[_ptr(phi_k[n]) for n in ("W1", "b1", "W2", "b2")],
                         _ptr(phi_q.get("Wmid")), _ptr(phi_q.get("bmid")), _ptr(phi_k.get("Wmid")), _ptr(phi_k.get("bmid")))

    def forward(self, q, k, v, phi_q, phi_k, frames, H, W, chunk, overlap, out=None, layout="bhnd", stream=None):
        """q, k, v: CUDA tensors [B, n_heads, N, d] ("bhnd") or [B, N, n_heads, d] ("bnhd"), contiguous.
        Returns `out` (same shape).  Asynchronous on `stream` (default: torch's current stream)."""
        if out is None:
            out = torch.empty_like(q)
        if layout == "bhnd":
            B, nh, N, d = q.shape
            lay = Layout(nh * N * d, N * d, d)
        elif layout == "bnhd":
            B, N, nh, d = q.shape
            lay = Layout(N * nh * d, d, nh * d)
        else:
            raise ValueError(layout)
        for t in (q, k, v, out):
            if not (t.is_cuda and t.is_contiguous() and t.shape == q.shape):
                raise ValueError("q, k, v, out must be contiguous CUDA tensors of one shape")
        st = stream if stream is not None else torch.cuda.current_stream(q.device)
        phi = self.phi_struct(phi_q, phi_k)
        _check(lib().rehyat_forward(self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(out), C.byref(lay), C.byref(phi),
                                    B, frames, H, W, chunk, overlap, C.c_void_p(st.cuda_stream)), "rehyat_forward")
        return out

    def forward_host(self, q, k, v, out, phi_q, phi_k, frames, H, W, chunk, overlap, stream=None):
        """q, k, v, out: CPU tensors [B, n_heads, N, d] (pinned for asynchronous copies); phi on the device.
        Returns after `out` has been filled."""
        B = q.shape[0]
        st = stream if stream is not None else torch.cuda.current_stream(self.cfg.device)
        phi = self.phi_struct(phi_q, phi_k)
        _check(lib().rehyat_forward_host(self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(out), C.byref(phi), B, frames, H,
                                         W, chunk, overlap, C.c_void_p(st.cuda_stream)), "rehyat_forward_host")
        return out

    # ---- chunk-by-chunk processing (rehyat_stream_*)
    def stream_begin(self, batch, H, W, chunk, overlap, stream=None):
        st = stream if stream is not None else torch.cuda.current_stream(self.cfg.device)
        _check(lib().rehyat_stream_begin(self._h, batch, H, W, chunk, overlap, C.c_void_p(st.cuda_stream)),
               "rehyat_stream_begin")

    def stream_step(self, q, k, v, phi_q, phi_k, frames_in_chunk, out=None, stream=None):
        """q, k, v: CUDA tensors [B, n_heads, frames_in_chunk*H*W, d] of the next chunk, contiguous or views that
        share their strides (head_dim contiguous), e.g. slices of the whole sequence; `out` likewise."""
        if out is None:
            out = torch.empty_like(q)
        sb, sh, sn, sd = q.stride()
        if sd != 1 or any(t.stride() != q.stride() or t.shape != q.shape for t in (k, v, out)):
            raise ValueError("q, k, v, out must share shape and strides, with head_dim contiguous")
        lay = Layout(sb, sh, sn)
        st = stream if stream is not None else torch.cuda.current_stream(q.device)
        phi = self.phi_struct(phi_q, phi_k)
        _check(lib().rehyat_stream_step(self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(out), C.byref(lay), C.byref(phi),
                                        frames_in_chunk, C.c_void_p(st.cuda_stream)), "rehyat_stream_step")
        return out

    def stream_export(self, stream=None):
        """The sequence's state as bytes (header, s and z, the overlap frames of k and v)."""
        st = stream if stream is not None else torch.cuda.current_stream(self.cfg.device)
        n = lib().rehyat_stream_state_bytes(self._h)
        buf = (C.c_uint8 * n)()
        _check(lib().rehyat_stream_export(self._h, buf, n, C.c_void_p(st.cuda_stream)), "rehyat_stream_export")
        return bytes(buf)

    def stream_import(self, blob, stream=None):
        st = stream if stream is not None else torch.cuda.current_stream(self.cfg.device)
        buf = (C.c_uint8 * len(blob)).from_buffer_copy(blob)
        _check(lib().rehyat_stream_import(self._h, buf, len(blob), C.c_void_p(st.cuda_stream)), "rehyat_stream_import")

    def profile_enable(self, on=True):
        _check(lib().rehyat_profile_enable(self._h, int(on)), "rehyat_profile_enable")

    def profile_read(self):
        """{kind: (summed ms, launches)} since the last read; waits for the recorded events."""
        ms = (C.c_double * len(PROF_KINDS))()
        n = (C.c_int32 * len(PROF_KINDS))()
        _check(lib().rehyat_profile_read(self._h, ms, n), "rehyat_profile_read")
        return {k: (ms[i], n[i]) for i, k in enumerate(PROF_KINDS)}

    def set_wait_limit(self, wait_limit_us=0, withhold_loads=False):
        _check(lib().rehyat_set_wait_limit(self._h, int(wait_limit_us), int(bool(withhold_loads))), "rehyat_set_wait_limit")

    def status(self, stream=None):
        st = stream if stream is not None else torch.cuda.current_stream(self.cfg.device)
        return lib().rehyat_status(self._h, C.c_void_p(st.cuda_stream))


def forward_static(q, k, v, phi_q, phi_k, frames, H, W, chunk, overlap, *, dtype, poly_degree=2, phi_hidden=None,
                   phi_dim=None, act_hidden="relu", act_out="relu", c_mode="rowmax", phi_layers=2, out=None, stream=None):
    """rehyat_forward_static: the operator without a context and without any device allocation by the
    library; its workspace is a fixed array inside librehyat.so.  For callers that cannot allocate
    (fixed memory plans, loops that cannot take cudaMalloc's synchronisation).  q, k, v: contiguous CUDA
    tensors [B, n_heads, N, d]; `out` must be passed by such callers (it is allocated here with torch
    only when omitted).  Raises RehyatError(ERR_TOO_LARGE) beyond the fixed capacity."""
    B, nh, N, d = q.shape
    if out is None:
        out = torch.empty_like(q)
    cfg = Config(q.device.index or 0, DTYPE[dtype], nh, d, phi_hidden or 2 * d, phi_dim or 2 * d, poly_degree,
                 ACT[act_hidden], ACT[act_out], C_MODE[c_mode], 0, 1, 1, 1, 0, 0, 0, 0, phi_layers, 0, 0)
    lay = Layout(nh * N * d, N * d, d)
    st = stream if stream is not None else torch.cuda.current_stream(q.device)
    phi = Rehyat.phi_struct(phi_q, phi_k)
    _check(lib().rehyat_forward_static(C.byref(cfg), _ptr(q), _ptr(k), _ptr(v), _ptr(out), C.byref(lay), C.byref(phi),
                                       B, frames, H, W, chunk, overlap, C.c_void_p(st.cuda_stream)),
           "rehyat_forward_static")
    return out


def shard_call_args(q, k, v, out, phi_q, phi_k, rect):
    """Arguments of the operator call for one rectangle (b0, nb, h0, nh) of geometry.shard_rects: views of the
    [B, n_heads, N, d] tensors that start at (b0, h0) and keep the parent's strides, the phi parameters of heads
    [h0, h0 + nh), and the layout of those strides.  Marshalling only: nothing is copied."""
    b0, nb, h0, nh = rect
    views = tuple(t.narrow(0, b0, nb).narrow(1, h0, nh) for t in (q, k, v, out))
    sb, sh, sn, sd = q.stride()
    if sd != 1 or any(t.stride() != q.stride() for t in (k, v, out)):
        raise ValueError("q, k, v, out must share their strides, with head_dim contiguous")
    pq = {n: t.narrow(0, h0, nh) for n, t in phi_q.items()}
    pk = {n: t.narrow(0, h0, nh) for n, t in phi_k.items()}
    return views, pq, pk, Layout(sb, sh, sn)


class ShardedRehyat:
    """The (batch, head) problems of one operator call split over `world_size` ranks (geometry.shard_rects):
    this rank's rectangles, one context per distinct head count.  No exchange between ranks is needed."""

    def __init__(self, world_size, rank, *, batch, n_heads, **ctx_args):
        from . import geometry
        self.rects = geometry.shard_rects(batch, n_heads, world_size, rank)
        self._ops = {}
        for (_, nb, _, nh) in self.rects:
            if nh not in self._ops:
                self._ops[nh] = Rehyat(n_heads=nh, max_batch=max(r[1] for r in self.rects if r[3] == nh), **ctx_args)

    def forward(self, q, k, v, out, phi_q, phi_k, frames, H, W, chunk, overlap, stream=None):
        """q, k, v, out: the FULL [B, n_heads, N, d] CUDA tensors; only this rank's rectangles of `out` are written."""
        st = stream if stream is not None else torch.cuda.current_stream(q.device)
        self.last_launches = 0
        for rect in self.rects:
            (vq, vk, vv, vo), pq, pk, lay = shard_call_args(q, k, v, out, phi_q, phi_k, rect)
            op = self._ops[rect[3]]
            phi = Rehyat.phi_struct(pq, pk)
            _check(lib().rehyat_forward(op._h, _ptr(vq), _ptr(vk), _ptr(vv), _ptr(vo), C.byref(lay), C.byref(phi),
                                        rect[1], frames, H, W, chunk, overlap, C.c_void_p(st.cuda_stream)),
                   "rehyat_forward")
            self.last_launches += op.last_launches
        return out

    def status(self, stream=None):
        return min((op.status(stream) for op in self._ops.values()), default=OK)

    def close(self):
        for op in self._ops.values():
            op.close()


def for_workload(wl, **kw):
    """A context sized for a synth.Workload."""
    args = dict(n_heads=wl.n_heads, head_dim=wl.head_dim, dtype=wl.dtype, phi_hidden=wl.D_h, phi_dim=wl.D_out,
                poly_degree=wl.P, max_batch=wl.B, max_tokens_per_frame=wl.HW, max_chunk_frames=min(wl.Tc, wl.T),
                max_frames=wl.T, phi_layers=wl.phi_layers)
    args.update(kw)
    return Rehyat(**args)
