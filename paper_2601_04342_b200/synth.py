"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds NO arithmetic of the method: it only draws numbers.  Both the oracle-side
tests and the CUDA-side callers take their inputs from here, so that the two are compared on
the same bits.  The tensors stand in for Wan2.1-1.3B self-attention activations at latent
grid 21 x 30 x 52 (Section 4.1: 81 x 480 x 832 videos) and for trained phi parameters,
neither of which is available offline.

Recipe: a counter-based generator (numpy Philox, key = (seed, stream)) with one stream per
tensor; q, k, v ~ N(0, 1); optionally q and k are divided by their per-token per-head RMS
(the q/k-norm of the Wan blocks); phi parameters ~ N(0, 0.02^2) for all of W1, b1, W2, b2
of both maps.  In bf16 workloads every tensor is rounded to bf16 once, here, so the oracle
and the kernels see identical values.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

BASE_SEED = 260104342

_STREAMS = {"q": 1, "k": 2, "v": 3, "phi_q": 4, "phi_k": 5, "v_frame": 6}


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    n_heads: int
    head_dim: int
    T: int            # latent frames
    H: int            # latent patch rows
    W: int            # latent patch columns
    Tc: int           # chunk frames
    To: int           # overlap frames
    dtype: str        # "fp32" | "bf16"
    rms_norm_qk: bool = False
    P: int = 2
    seed: int = BASE_SEED
    phi_hidden: int = 0   # 0: the default width 2 * head_dim
    phi_dim: int = 0      # 0: the default width 2 * head_dim
    phi_layers: int = 2   # layers of the phi MLP; beyond two, hidden layers [D_h, D_h] sit between the first and the last

    @property
    def HW(self):
        return self.H * self.W

    @property
    def N(self):
        return self.T * self.H * self.W

    @property
    def D_h(self):     # phi hidden width: 2 * head_dim (gives the paper's ~2.4 M parameters)
        return self.phi_hidden or 2 * self.head_dim

    @property
    def D_out(self):   # phi output width D'
        return self.phi_dim or 2 * self.head_dim

    def with_(self, **kw):
        return replace(self, **kw)


CONFIGS = {
    "tiny_fp32": Workload("tiny_fp32", 1, 2, 64, 4, 8, 8, 1, 1, "fp32", False, seed=BASE_SEED + 1),
    "wan13b_layer": Workload("wan13b_layer", 1, 12, 128, 21, 30, 52, 3, 1, "bf16", True,
                             seed=BASE_SEED + 2),
    "cfg_long": Workload("cfg_long", 2, 12, 128, 41, 30, 52, 3, 1, "bf16", True,
                         seed=BASE_SEED + 3),
    "long_constant_memory": Workload("long_constant_memory", 1, 12, 128, 81, 30, 52, 3, 1, "bf16",
                                     True, seed=BASE_SEED + 4),
    # the 320x480 resolution of the paper's on-device tables: latent 21 x 20 x 30 (12,600 tokens)
    "wan13b_320x480": Workload("wan13b_320x480", 1, 12, 128, 21, 20, 30, 3, 1, "bf16", True,
                               seed=BASE_SEED + 6),
}


def sweep_configs():
    """The chunk/overlap sweep: 21 frames of 30x52 and 20x32, chunk {1,3,7} x overlap {0,1,2}."""
    out = []
    for (H, W) in ((30, 52), (20, 32)):
        for Tc in (1, 3, 7):
            for To in (0, 1, 2):
                out.append(Workload(f"sweep_{H}x{W}_c{Tc}_o{To}", 1, 12, 128, 21, H, W, Tc, To,
                                    "bf16", False, seed=BASE_SEED + 5))
    return out


def _normal(seed, stream, shape):
    gen = np.random.Generator(np.random.Philox(key=[seed, stream]))
    return gen.standard_normal(size=shape, dtype=np.float32)


def _torch_dtype(name):
    return {"fp32": torch.float32, "bf16": torch.bfloat16}[name]


def make_phi_params(wl: Workload, which: str, scale: float = 1.0, std: float = 0.02):
    """Parameters of phi_q ("phi_q") or phi_k ("phi_k"): W1 [n_h, D_h, d], b1 [n_h, D_h],
    W2 [n_h, D', D_h], b2 [n_h, D'] (and Wmid, bmid of a deeper map), in the workload's dtype."""
    nh, d, Dh, Do = wl.n_heads, wl.head_dim, wl.D_h, wl.D_out
    sizes = {"W1": (nh, Dh, d), "b1": (nh, Dh), "W2": (nh, Do, Dh), "b2": (nh, Do)}
    if wl.phi_layers > 2:       # drawn after the others, so that the two-layer tensors do not depend on the depth
        sizes["Wmid"] = (nh, wl.phi_layers - 2, Dh, Dh)
        sizes["bmid"] = (nh, wl.phi_layers - 2, Dh)
    flat = _normal(wl.seed, _STREAMS[which], (sum(int(np.prod(s)) for s in sizes.values()),))
    out, off = {}, 0
    for name, shp in sizes.items():
        n = int(np.prod(shp))
        out[name] = torch.from_numpy(flat[off:off + n].reshape(shp) * np.float32(std * scale)) \
            .to(_torch_dtype(wl.dtype)).contiguous()
        off += n
    return out


def make_inputs(wl: Workload, *, q_scale: float = 1.0, phi_scale: float = 1.0,
                v_frame_offsets: bool = False, v_ones: bool = False):
    """Returns {"q","k","v": [B, n_h, N, d] CPU tensors in the workload's dtype,
    "phi_q","phi_k": parameter dictionaries}.

    q_scale          multiplies q (a "peaky" run uses 4: window logits of std 4)
    phi_scale        multiplies every phi parameter (a stress run so the squared features carry mass)
    v_frame_offsets  adds one N(0,1) vector per latent frame to v, so that y is O(1) and
                     depends on which frames receive weight
    v_ones           v = 1 everywhere (row-sum invariant: y must be 1)
    """
    B, nh, N, d = wl.B, wl.n_heads, wl.N, wl.head_dim
    dt = _torch_dtype(wl.dtype)
    out = {}
    for name in ("q", "k", "v"):
        if name == "v" and v_ones:
            out[name] = torch.ones((B, nh, N, d), dtype=dt)
            continue
        x = _normal(wl.seed, _STREAMS[name], (B, nh, N, d))
        if wl.rms_norm_qk and name in ("q", "k"):
            x /= np.sqrt(np.mean(np.square(x), axis=-1, keepdims=True, dtype=np.float32))
        if name == "q" and q_scale != 1.0:
            x *= np.float32(q_scale)
        if name == "v" and v_frame_offsets:
            m = _normal(wl.seed, _STREAMS["v_frame"], (wl.T, d))
            x = x.reshape(B, nh, wl.T, wl.HW, d)
            x += m[None, None, :, None, :]
            x = x.reshape(B, nh, N, d)
        out[name] = torch.from_numpy(x).to(dt).contiguous()
    out["phi_q"] = make_phi_params(wl, "phi_q", phi_scale)
    out["phi_k"] = make_phi_params(wl, "phi_k", phi_scale)
    return out


def to_f64(inputs):
    """The same values widened to float64 numpy arrays (what the oracle consumes)."""
    conv = lambda t: t.to(torch.float64).numpy()
    return {
        "q": conv(inputs["q"]), "k": conv(inputs["k"]), "v": conv(inputs["v"]),
        "phi_q": {n: conv(t) for n, t in inputs["phi_q"].items()},
        "phi_k": {n: conv(t) for n, t in inputs["phi_k"].items()},
    }
