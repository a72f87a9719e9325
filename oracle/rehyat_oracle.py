"""Plain fp64 oracle of the ReHyAt recurrent hybrid attention operator.

TEST INFRASTRUCTURE ONLY: slow, obviously-correct numpy, written from the paper's
equations.  It shares no code with the CUDA path and is never on the product path.

What the operator computes (paper Section 3.2-3.3).  N = T*HW tokens flattened from a
(T, H, W) latent grid, chunks of T_c latent frames (N' = T_c*HW tokens), overlap of
T_o frames.  For a query i in chunk t the keys are split into a softmax set TS_t and a
linear set TL_t, and

    y_i = (aS_i + aL_i) / (nS_i + nL_i)                                   (Eq. 5)
    aS_i = sum_{j in TS_t} exp(q_i.k_j/sqrt(d) - c_i) v_j                  (Eq. 6)
    aL_i = phi_q(q_i) . sum_{j in TL_t} phi_k(k_j) v_j^T                   (Eq. 7)
    nS_i = sum_{j in TS_t} exp(q_i.k_j/sqrt(d) - c_i)                      (Eq. 8)
    nL_i = phi_q(q_i) . sum_{j in TL_t} phi_k(k_j)                         (Eq. 9)

Token sets:
    non-overlapping, bidirectional  TS_t = [tN', (t+1)N'),  TL_t = all - TS_t   (Eq. 10-11)
    overlapping, bidirectional      TS_t = [max(tN'-T_o HW,0), (t+1)N')         (Eq. 12)
    causal (the recurrent form)     TL_t = [0, max(tN'-T_o HW,0))               (Eq. 13)

Three independent evaluations live here:
    hybrid_brute   explicit N x N weight matrix, Python loops (tiny inputs only)
    hybrid_direct  Eq. 5-9 chunk by chunk with explicit sums over the two sets
    hybrid_rnn     the chunk-wise RNN of Eq. 14-18

Readings taken where the paper is silent or garbled (each is restated in the design notes):
  * c is per query row and equals the row maximum of the scaled window logits
    ("typically the maximum exponent", text after Eq. 9): mode "rowmax".  The linear terms
    are NOT rescaled by it (Eq. 7 and 9 carry no c), so the result depends on c;
    mode "zero" is the other literal choice c = 0.
  * Eq. 17-18 as printed add the whole cumulative set TL_t again at every step; since the
    state is defined as s_t = sum_{j in TL_t} phi_k(k_j) v_j^T (Eq. 7 with Eq. 13), the
    update adds only the newly admitted tokens TL_{t+1} - TL_t.
  * T not divisible by T_c: T' = ceil(T/T_c) and the LAST chunk is short.
  * multi-head: the softmax scale is 1/sqrt(head_dim); the linear similarity has no scale
    and no epsilon.
  * phi (text "Characterization of phi" and appendix "Training Details"): a per-head
    two-layer MLP  u = act_out(W2 act_hidden(W1 x + b1) + b2), u split into P equal
    contiguous parts, part p (1-based) raised element-wise to the power p, concatenated.
    The text also speaks of varying the "transformation complexity" of phi; the deeper maps
    taken here put further hidden layers h <- act_hidden(Wm h + bm) of width D_h between the
    two (the widths and activation of the two-layer map, nothing new to choose).

Parity unpinned (the paper prints no numbers that would decide them): rowmax vs zero,
the activation functions, which chunk is the short one, which deeper phi maps the authors
tried, and the convention of the block's q/k normalisation and rotation (rms_norm,
rope_rotate: the block is taken over from the pretrained model and not restated).
"""
from __future__ import annotations

import math

import numpy as np

# ----------------------------------------------------------------------------------------
# feature map phi
# ----------------------------------------------------------------------------------------

ACTIVATIONS = ("relu", "identity", "softplus", "elu1", "gelu")


def _act(x: np.ndarray, name: str) -> np.ndarray:
    if name == "relu":
        return np.maximum(x, 0.0)
    if name == "identity":
        return x
    if name == "softplus":
        return np.logaddexp(0.0, x)
    if name == "elu1":  # 1 + elu(x), the map of Katharopoulos et al. quoted below Eq. 4
        return np.where(x > 0, x + 1.0, np.exp(np.minimum(x, 0.0)))
    if name == "gelu":  # exact (erf) form
        erf = np.vectorize(math.erf, otypes=[np.float64])
        return 0.5 * x * (1.0 + erf(x / math.sqrt(2.0)))
    raise ValueError(f"unknown activation {name!r}")


def phi_map(x, W1, b1, W2, b2, P=2, act_hidden="relu", act_out="relu", Wmid=None, bmid=None):
    """phi(x) = [psi_1(x)^1, psi_2(x)^2, ..., psi_P(x)^P]  (text "Characterization of phi").

    x [n, d]; W1 [D_h, d]; b1 [D_h]; W2 [D', D_h]; b2 [D'] of ONE head.  Returns [n, D'].
    Wmid [L-2, D_h, D_h], bmid [L-2, D_h]: further hidden layers of an L-layer map, applied in order between
    the first and the last layer (None or empty: the two-layer map).
    """
    x = np.asarray(x, dtype=np.float64)
    h = _act(x @ np.asarray(W1, np.float64).T + np.asarray(b1, np.float64), act_hidden)
    if Wmid is not None:
        for Wm, bm in zip(np.asarray(Wmid, np.float64), np.asarray(bmid, np.float64)):
            h = _act(h @ Wm.T + bm, act_hidden)
    u = _act(h @ np.asarray(W2, np.float64).T + np.asarray(b2, np.float64), act_out)
    Dp = u.shape[-1]
    if Dp % P != 0:
        raise ValueError("D' must be divisible by the polynomial degree P")
    w = Dp // P
    parts = [u[..., p * w:(p + 1) * w] ** (p + 1) for p in range(P)]
    return np.concatenate(parts, axis=-1)


def phi_param_count(n_heads, d, D_h, D_out, with_bias=False):
    """Parameters of phi_q plus phi_k for one block (Section 4.3: about 2.4 M per block)."""
    per_map = n_heads * (d * D_h + D_h * D_out)
    if with_bias:
        per_map += n_heads * (D_h + D_out)
    return 2 * per_map


# ----------------------------------------------------------------------------------------
# what a DiT block does to q and k before the attention operator (the block of Eq. 1 around
# A_l; the paper takes it over from the pretrained model and does not restate it)
# ----------------------------------------------------------------------------------------

def rms_norm(x, weight=None, eps=1e-6):
    """x / sqrt(mean(x^2 over the last axis) + eps) * weight, the RMS normalisation applied to the
    queries and keys of each head (weight [d] or broadcastable; None: ones)."""
    x = np.asarray(x, np.float64)
    y = x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    return y if weight is None else y * np.asarray(weight, np.float64)


def rope_rotate(x, cos, sin):
    """Rotary position embedding with caller-supplied tables: the pair (x[..., n, 2i], x[..., n, 2i+1]) of token n
    is rotated by the angle whose cosine and sine are cos[n, i], sin[n, i] (x [..., N, d]; cos, sin [N, d/2])."""
    x = np.asarray(x, np.float64)
    cos = np.asarray(cos, np.float64); sin = np.asarray(sin, np.float64)
    a, b = x[..., 0::2], x[..., 1::2]
    out = np.empty_like(x)
    out[..., 0::2] = a * cos - b * sin
    out[..., 1::2] = a * sin + b * cos
    return out


def qk_transform(q, k, q_weight=None, k_weight=None, eps=1e-6, cos=None, sin=None, norm=True):
    """q, k [B, n_h, N, d] as the block hands them over -> what the attention operator sees: per-head RMS norm
    (weights [n_h, d] or None) followed by the rotation.  Either step can be left out (norm=False; cos=None)."""
    q = np.asarray(q, np.float64); k = np.asarray(k, np.float64)
    if norm:
        q = rms_norm(q, None if q_weight is None else np.asarray(q_weight, np.float64)[None, :, None, :], eps)
        k = rms_norm(k, None if k_weight is None else np.asarray(k_weight, np.float64)[None, :, None, :], eps)
    if cos is not None:
        q, k = rope_rotate(q, cos, sin), rope_rotate(k, cos, sin)
    return q, k


# ----------------------------------------------------------------------------------------
# token sets
# ----------------------------------------------------------------------------------------

def num_chunks(T, Tc):
    return -(-T // Tc)


def chunk_queries(t, T, HW, Tc):
    """Query range [q0, q1) of chunk t; the last chunk is short when Tc does not divide T."""
    N = T * HW
    return t * Tc * HW, min((t + 1) * Tc * HW, N)


def softmax_set(t, T, HW, Tc, To):
    """TS_t of Eq. 12 / Eq. 13 as a half-open range [lo, hi)."""
    N = T * HW
    lo = max(t * Tc * HW - To * HW, 0)
    hi = min((t + 1) * Tc * HW, N)
    return lo, hi


def linear_set(t, T, HW, Tc, To, causal=True):
    """TL_t as a sorted index array: Eq. 13 when causal, else Eq. 11/12 (complement)."""
    N = T * HW
    lo, hi = softmax_set(t, T, HW, Tc, To)
    if causal:
        return np.arange(0, lo)
    return np.concatenate([np.arange(0, lo), np.arange(hi, N)])


# ----------------------------------------------------------------------------------------
# helpers
# ----------------------------------------------------------------------------------------

def _phi_pair(phi_q, phi_k, h):
    """Slice head h out of the per-head parameter dictionaries."""
    pq = {n: np.asarray(phi_q[n][h], np.float64) for n in ("W1", "b1", "W2", "b2", "Wmid", "bmid") if n in phi_q}
    pk = {n: np.asarray(phi_k[n][h], np.float64) for n in ("W1", "b1", "W2", "b2", "Wmid", "bmid") if n in phi_k}
    return pq, pk


def _phi(x, p, P, act_hidden, act_out):
    return phi_map(x, p["W1"], p["b1"], p["W2"], p["b2"], P, act_hidden, act_out, p.get("Wmid"), p.get("bmid"))


def _stabiliser(S, c_mode):
    if c_mode == "rowmax":
        return S.max(axis=1, keepdims=True) if S.shape[1] else np.zeros((S.shape[0], 1))
    if c_mode == "zero":
        return np.zeros((S.shape[0], 1))
    raise ValueError(f"unknown c_mode {c_mode!r}")


# ----------------------------------------------------------------------------------------
# (1) brute force: explicit N x N weight matrix
# ----------------------------------------------------------------------------------------

def hybrid_weights_brute(q, k, phi_q, phi_k, T, HW, Tc, To, *, P=2, act_hidden="relu",
                         act_out="relu", c_mode="rowmax", causal=True, partition=None,
                         logit_bias=None):
    """Un-normalised weight matrix W[i, j] of ONE head, by explicit loops (Eq. 5-9).

    q, k [N, d]; phi_q/phi_k dictionaries of ONE head.  `partition(t) -> (TS, TL)` (index
    lists) overrides the paper's sets: a test hook used for the pure-linear limit.
    `logit_bias[i]` is added to every window logit of query i: a test hook.
    """
    N, d = q.shape
    fq = _phi(q, phi_q, P, act_hidden, act_out)
    fk = _phi(k, phi_k, P, act_hidden, act_out)
    W = np.zeros((N, N))
    Np = Tc * HW
    for i in range(N):
        t = i // Np
        if partition is None:
            lo, hi = softmax_set(t, T, HW, Tc, To)
            TS = list(range(lo, hi))
            TL = [int(j) for j in linear_set(t, T, HW, Tc, To, causal)]
        else:
            TS, TL = partition(t)
        logits = {}
        for j in TS:
            s = 0.0
            for a in range(d):
                s += q[i, a] * k[j, a]
            s /= math.sqrt(d)
            if logit_bias is not None:
                s += logit_bias[i]
            logits[j] = s
        if c_mode == "rowmax":
            c = max(logits.values()) if logits else 0.0
        elif c_mode == "zero":
            c = 0.0
        else:
            raise ValueError(c_mode)
        for j in TS:
            W[i, j] += math.exp(logits[j] - c)
        for j in TL:
            w = 0.0
            for a in range(fq.shape[1]):
                w += fq[i, a] * fk[j, a]
            W[i, j] += w
    return W


def hybrid_brute(q, k, v, phi_q, phi_k, T, HW, Tc, To, **kw):
    """y [B, n_h, N, d] from the explicit weight matrix: y_i = sum_j W_ij v_j / sum_j W_ij."""
    q = np.asarray(q, np.float64); k = np.asarray(k, np.float64); v = np.asarray(v, np.float64)
    B, nh, N, d = q.shape
    y = np.zeros_like(v)
    for b in range(B):
        for h in range(nh):
            pq, pk = _phi_pair(phi_q, phi_k, h)
            W = hybrid_weights_brute(q[b, h], k[b, h], pq, pk, T, HW, Tc, To, **kw)
            y[b, h] = (W @ v[b, h]) / W.sum(axis=1, keepdims=True)
    return y


# ----------------------------------------------------------------------------------------
# (2) direct form: Eq. 5-9 per chunk with explicit sums over TS_t and TL_t
# ----------------------------------------------------------------------------------------

def hybrid_direct(q, k, v, phi_q, phi_k, T, HW, Tc, To, *, P=2, act_hidden="relu",
                  act_out="relu", c_mode="rowmax", causal=True, return_parts=False):
    q = np.asarray(q, np.float64); k = np.asarray(k, np.float64); v = np.asarray(v, np.float64)
    B, nh, N, d = q.shape
    assert N == T * HW
    y = np.zeros_like(v)
    lin_frac = np.zeros((B, nh, N))
    for b in range(B):
        for h in range(nh):
            pq, pk = _phi_pair(phi_q, phi_k, h)
            for t in range(num_chunks(T, Tc)):
                q0, q1 = chunk_queries(t, T, HW, Tc)
                lo, hi = softmax_set(t, T, HW, Tc, To)
                TL = linear_set(t, T, HW, Tc, To, causal)
                Qt = q[b, h, q0:q1]
                S = Qt @ k[b, h, lo:hi].T / math.sqrt(d)
                c = _stabiliser(S, c_mode)
                E = np.exp(S - c)
                aS = E @ v[b, h, lo:hi]                                   # Eq. 6
                nS = E.sum(axis=1, keepdims=True)                         # Eq. 8
                fq = _phi(Qt, pq, P, act_hidden, act_out)
                fk = _phi(k[b, h, TL], pk, P, act_hidden, act_out)
                aL = fq @ (fk.T @ v[b, h, TL])                            # Eq. 7
                nL = fq @ fk.sum(axis=0)[:, None]                         # Eq. 9
                y[b, h, q0:q1] = (aS + aL) / (nS + nL)                    # Eq. 5
                lin_frac[b, h, q0:q1] = (nL / (nS + nL))[:, 0]
    if return_parts:
        return y, lin_frac
    return y


# ----------------------------------------------------------------------------------------
# (3) recurrent form: Eq. 14-18
# ----------------------------------------------------------------------------------------

def hybrid_rnn(q, k, v, phi_q, phi_k, T, HW, Tc, To, *, P=2, act_hidden="relu",
               act_out="relu", c_mode="rowmax", heads=None):
    """Chunk-wise RNN.  `heads` restricts the evaluation to some heads (timing samples)."""
    q = np.asarray(q, np.float64); k = np.asarray(k, np.float64); v = np.asarray(v, np.float64)
    B, nh, N, d = q.shape
    assert N == T * HW
    y = np.zeros_like(v)
    Tp = num_chunks(T, Tc)
    for b in range(B):
        for h in (range(nh) if heads is None else heads):
            pq, pk = _phi_pair(phi_q, phi_k, h)
            Dp = pq["W2"].shape[0]
            s = np.zeros((Dp, d))                                         # Eq. 14
            z = np.zeros((Dp, 1))                                         # Eq. 15
            for t in range(Tp):
                q0, q1 = chunk_queries(t, T, HW, Tc)
                lo, hi = softmax_set(t, T, HW, Tc, To)
                Qt = q[b, h, q0:q1]
                S = Qt @ k[b, h, lo:hi].T / math.sqrt(d)
                c = _stabiliser(S, c_mode)
                E = np.exp(S - c)
                aS = E @ v[b, h, lo:hi]
                nS = E.sum(axis=1, keepdims=True)
                fq = _phi(Qt, pq, P, act_hidden, act_out)
                y[b, h, q0:q1] = (aS + fq @ s) / (nS + fq @ z)            # Eq. 16
                if t + 1 < Tp:
                    lo_next, _ = softmax_set(t + 1, T, HW, Tc, To)
                    fk = _phi(k[b, h, lo:lo_next], pk, P, act_hidden, act_out)
                    s = s + fk.T @ v[b, h, lo:lo_next]                    # Eq. 17 (new tokens)
                    z = z + fk.sum(axis=0)[:, None]                       # Eq. 18 (new tokens)
    return y


# ----------------------------------------------------------------------------------------
# sampled rows at sizes where the full evaluation is too slow
# ----------------------------------------------------------------------------------------

def hybrid_rows(q, k, v, phi_q, phi_k, T, HW, Tc, To, b, h, rows, *, P=2,
                act_hidden="relu", act_out="relu", c_mode="rowmax"):
    """Rows `rows` of head (b, h) of the causal operator, each from Eq. 5-9 directly.

    The linear sums of Eq. 7 and 9 over TL_t = [0, lo_t) are formed once per chunk that is
    asked for.  Returns (y [len(rows), d], nL/(nS+nL) per row).
    """
    q = np.asarray(q[b, h], np.float64); k = np.asarray(k[b, h], np.float64)
    v = np.asarray(v[b, h], np.float64)
    N, d = q.shape
    pq, pk = _phi_pair(phi_q, phi_k, h)
    rows = np.asarray(rows, dtype=np.int64)
    Np = Tc * HW
    out = np.zeros((len(rows), d))
    frac = np.zeros(len(rows))
    for t in np.unique(rows // Np):
        sel = np.nonzero(rows // Np == t)[0]
        lo, hi = softmax_set(int(t), T, HW, Tc, To)
        fk = _phi(k[:lo], pk, P, act_hidden, act_out)
        s = fk.T @ v[:lo]
        z = fk.sum(axis=0)[:, None]
        Qs = q[rows[sel]]
        S = Qs @ k[lo:hi].T / math.sqrt(d)
        c = _stabiliser(S, c_mode)
        E = np.exp(S - c)
        nS = E.sum(axis=1, keepdims=True)
        fq = _phi(Qs, pq, P, act_hidden, act_out)
        nL = fq @ z
        out[sel] = (E @ v[lo:hi] + fq @ s) / (nS + nL)
        frac[sel] = (nL / (nS + nL))[:, 0]
    return out, frac


# ----------------------------------------------------------------------------------------
# the two limiting operators, written from their own definitions
# ----------------------------------------------------------------------------------------

def softmax_attention(q, k, v):
    """Eq. 2 per head: softmax(q k^T / sqrt(d)) v."""
    q = np.asarray(q, np.float64); k = np.asarray(k, np.float64); v = np.asarray(v, np.float64)
    d = q.shape[-1]
    S = q @ np.swapaxes(k, -1, -2) / math.sqrt(d)
    S = S - S.max(axis=-1, keepdims=True)
    E = np.exp(S)
    return (E / E.sum(axis=-1, keepdims=True)) @ v


def linear_attention(fq, fk, v):
    """Eq. 4 for one head: phi(q_i) sum_j phi(k_j) v_j^T / phi(q_i) sum_j phi(k_j)."""
    kv = fk.T @ v
    ksum = fk.sum(axis=0)
    return (fq @ kv) / (fq @ ksum)[:, None]
