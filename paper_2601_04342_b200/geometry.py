"""Host-side geometry of the chunked operator: chunk bounds, the algorithmic FLOP model and
the way independent (batch, head) problems are split over ranks.  No tensor arithmetic.

Chunk t (Section 3.3, causal overlapping sets): queries [t N', min((t+1) N', N)), softmax
window [lo_t, hi_t) with lo_t = max(t N' - T_o HW, 0), linear prefix [0, lo_t).
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass(frozen=True)
class Chunk:
    t: int
    q0: int      # first query token
    q1: int      # one past the last query token
    lo: int      # first key of the softmax window (= length of the linear prefix)
    hi: int      # one past the last key of the softmax window


def chunk_plan(T: int, HW: int, Tc: int, To: int):
    if T < 1 or HW < 1 or Tc < 1 or To < 0:
        raise ValueError("need T>=1, HW>=1, Tc>=1, To>=0")
    N = T * HW
    Np = Tc * HW
    n_chunks = -(-T // Tc)
    plan = []
    for t in range(n_chunks):
        q0 = t * Np
        q1 = min(q0 + Np, N)
        plan.append(Chunk(t, q0, q1, max(q0 - To * HW, 0), q1))
    return plan


def flop_model(B, n_heads, d, T, HW, Tc, To, D_h, D_out):
    """Algorithmic FLOPs of one operator call.

    window  4 d per (query, key) pair inside a softmax window (q.k and p.v)
    phi     2 (d D_h + D_h D') per token per map, for keys that ever enter a state
            (j < lo of the last chunk) and for queries of chunks with a non-empty prefix
    state   2 D' (d+1) per such key;  readout 2 D' (d+1) per such query
    Masked padding, recomputation and the avoided N^2 work are not counted.
    """
    plan = chunk_plan(T, HW, Tc, To)
    pairs = sum((c.q1 - c.q0) * (c.hi - c.lo) for c in plan)
    keys_in_state = plan[-1].lo
    queries_with_prefix = sum(c.q1 - c.q0 for c in plan if c.lo > 0)
    per_tok_phi = 2 * (d * D_h + D_h * D_out)
    mult = B * n_heads
    out = {
        "pairs": pairs * mult,
        "window": 4 * d * pairs * mult,
        "phi": per_tok_phi * (keys_in_state + queries_with_prefix) * mult,
        "state": 2 * D_out * (d + 1) * keys_in_state * mult,
        "readout": 2 * D_out * (d + 1) * queries_with_prefix * mult,
        "full_softmax": 4 * d * (T * HW) ** 2 * mult,
    }
    out["total"] = out["window"] + out["phi"] + out["state"] + out["readout"]
    return out


def io_bytes(B, n_heads, d, N, elem_bytes):
    """Algorithmic HBM traffic of one call: q, k, v read once, y written once."""
    return 4 * B * n_heads * N * d * elem_bytes


def shard_heads(B: int, n_heads: int, world_size: int, rank: int):
    """Contiguous slice [u0, u1) of the B*n_heads independent (batch, head) problems that
    `rank` owns.  Units are spread as evenly as possible; no exchange is needed between ranks."""
    units = B * n_heads
    base, rem = divmod(units, world_size)
    u0 = rank * base + min(rank, rem)
    return u0, u0 + base + (1 if rank < rem else 0)


def shard_rects(B: int, n_heads: int, world_size: int, rank: int):
    """The slice of shard_heads as rectangles (b0, nb, h0, nh) of whole (batch, head) blocks, in unit order:
    a slice that starts or ends inside a batch item is cut at the batch boundaries.  Each rectangle is one
    operator call on `nh` heads (a context with that head count, tensor and phi pointers offset to head h0)."""
    u0, u1 = shard_heads(B, n_heads, world_size, rank)
    rects = []
    u = u0
    while u < u1:
        b, h = divmod(u, n_heads)
        if h == 0 and u1 - u >= n_heads:                 # whole batch items
            nb = (u1 - u) // n_heads
            rects.append((b, nb, 0, n_heads))
            u += nb * n_heads
        else:                                            # the rest of batch item b, or up to the slice's end
            nh = min(n_heads - h, u1 - u)
            rects.append((b, 1, h, nh))
            u += nh
    return rects


def shard_efficiency(B: int, n_heads: int, world_size: int):
    """Units the busiest rank owns against a perfectly even split: the efficiency a head-sharded layer can
    reach at most (12 heads over 8 ranks: 12 / (8 * 2) = 0.75)."""
    most = max(u1 - u0 for u0, u1 in (shard_heads(B, n_heads, world_size, r) for r in range(world_size)))
    return B * n_heads / (world_size * most) if most else 0.0
