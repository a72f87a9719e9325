"""q and k normalised and rotated ahead of the operator (rehyat_set_qk_transform): the fused pre-pass against the
oracle's rms_norm / rope_rotate in fp64, then the whole operator on the transformed tensors.

Inputs: q and k are NOT pre-normalised here (scaled rows of N(0,1), so the normalisation has something to do),
the norm weights are 1 + 0.1 N(0,1), the rotation tables are those of one-dimensional positions n with
frequencies 10000^(-2i/d), as fp32 - the oracle reads the same fp32 bits."""
import numpy as np
import pytest
import torch

from oracle import rehyat_oracle as orc
from paper_2601_04342_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2601_04342_b200 import build
    build.build()


def _case(wl, seed):
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    rng = np.random.default_rng(seed)
    dt = x["q"].dtype
    # rows of different lengths: the normalisation must undo this
    scale = torch.from_numpy(rng.uniform(0.5, 1.5, size=(wl.B, wl.n_heads, wl.N, 1)).astype(np.float32))
    x["q"] = (x["q"].float() * scale).to(dt)
    x["k"] = (x["k"].float() * scale.flip(2)).to(dt)
    wq = torch.from_numpy((1.0 + 0.1 * rng.standard_normal((wl.n_heads, wl.head_dim))).astype(np.float32)).to(dt)
    wk = torch.from_numpy((1.0 + 0.1 * rng.standard_normal((wl.n_heads, wl.head_dim))).astype(np.float32)).to(dt)
    half = wl.head_dim // 2
    ang = np.arange(wl.N)[:, None] * (10000.0 ** (-np.arange(half) / half))[None, :]
    cos = torch.from_numpy(np.cos(ang).astype(np.float32)).contiguous()
    sin = torch.from_numpy(np.sin(ang).astype(np.float32)).contiguous()
    return x, wq, wk, cos, sin


def _run(wl, x, wq, wk, cos, sin, *, rms_norm=True, rope=True, weights=True, **kw):
    from paper_2601_04342_b200 import binding
    op = binding.for_workload(wl, qk_transform=True, **kw)
    d = {n: x[n].cuda() for n in ("q", "k", "v")}
    pq = {n: t.cuda() for n, t in x["phi_q"].items()}
    pk = {n: t.cuda() for n, t in x["phi_k"].items()}
    keep = [wq.cuda(), wk.cuda(), cos.cuda(), sin.cuda()]
    op.set_qk_transform(q_weight=keep[0] if weights else None, k_weight=keep[1] if weights else None, rms_norm=rms_norm,
                        eps=1e-6, cos=keep[2] if rope else None, sin=keep[3] if rope else None)
    q_before = d["q"].clone()
    y = op.forward(d["q"], d["k"], d["v"], pq, pk, wl.T, wl.H, wl.W, wl.Tc, wl.To)
    assert op.status() == 0
    assert torch.equal(d["q"], q_before)                       # the caller's q is not touched
    launches_on = op.last_launches
    prof_names = binding.PROF_KINDS
    op.set_qk_transform(off=True)
    y_off = op.forward(d["q"], d["k"], d["v"], pq, pk, wl.T, wl.H, wl.W, wl.Tc, wl.To)
    assert op.status() == 0 and op.last_launches == launches_on - 1 and "qk_prep" in prof_names
    used = op.last_impl
    op.close()
    return y.double().cpu().numpy(), y_off.double().cpu().numpy(), used


def _oracle(wl, x, wq, wk, cos, sin, *, rms_norm=True, rope=True, weights=True):
    f = synth.to_f64(x)
    q, k = orc.qk_transform(f["q"], f["k"], wq.double().numpy() if weights else None, wk.double().numpy() if weights else None,
                            1e-6, cos.double().numpy() if rope else None, sin.double().numpy() if rope else None, norm=rms_norm)
    plain = orc.hybrid_rnn(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To, P=wl.P)
    # the block hands q and k to the attention operator in the operator's dtype: the transformed tensors are rounded to it
    dt = x["q"].dtype
    q, k = (torch.from_numpy(t).to(dt).double().numpy() for t in (q, k))
    return orc.hybrid_rnn(q, k, f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To, P=wl.P), plain


def _check(y, ref, dtype):
    err = np.abs(y - ref)
    if dtype == "fp32":
        assert err.max() <= 1e-4, f"max-abs {err.max():.3e}"
        return
    assert err.max() <= 2e-2, f"max-abs {err.max():.3e}"
    assert (err / (3e-3 + 2.0 ** -7 * np.abs(ref))).max() <= 1.0
    assert np.sqrt((err ** 2).mean() / (ref ** 2).mean()) <= 1e-2


CASES = [
    synth.Workload("qk_bf16", 2, 2, 128, 5, 10, 20, 2, 1, "bf16", False, seed=synth.BASE_SEED + 95),
    synth.Workload("qk_fp32", 1, 2, 64, 4, 8, 8, 1, 1, "fp32", False, seed=synth.BASE_SEED + 96),
    # an odd number of tokens (1071): the last row of the pass has no neighbour in its warp
    synth.Workload("qk_bf16_odd", 1, 2, 128, 7, 9, 17, 3, 1, "bf16", False, seed=synth.BASE_SEED + 98),
    synth.Workload("qk_bf16_d64", 1, 3, 64, 5, 10, 20, 2, 1, "bf16", False, seed=synth.BASE_SEED + 94),
]


@pytest.mark.parametrize("wl", CASES, ids=[w.name for w in CASES])
@pytest.mark.parametrize("steps", ["norm+rope", "norm_only_unweighted", "rope_only"])
def test_norm_and_rotation_ahead_of_the_operator(wl, steps):
    x, wq, wk, cos, sin = _case(wl, 17)
    flags = {"norm+rope": {}, "norm_only_unweighted": dict(rope=False, weights=False), "rope_only": dict(rms_norm=False)}[steps]
    ref, plain = _oracle(wl, x, wq, wk, cos, sin, **flags)
    y, y_off, used = _run(wl, x, wq, wk, cos, sin, **flags)
    assert used == ("tensor" if wl.dtype == "bf16" else "simt")
    assert np.abs(ref - plain).max() > 0.05                    # the transform matters on these inputs
    _check(y, ref, wl.dtype)
    _check(y_off, plain, wl.dtype)                             # and switching it off gives the plain operator back


def test_transform_needs_a_context_made_for_it_and_respects_max_frames():
    from paper_2601_04342_b200 import binding
    wl = CASES[0]
    x, wq, wk, cos, sin = _case(wl, 18)
    op = binding.for_workload(wl)                              # qk_transform = 0
    with pytest.raises(binding.RehyatError) as e:
        op.set_qk_transform(q_weight=wq.cuda(), k_weight=wk.cuda(), cos=cos.cuda(), sin=sin.cuda())
    assert e.value.code == binding.ERR_UNSUPPORTED
    op.close()
    op = binding.for_workload(wl, qk_transform=True, max_frames=wl.T - 1)
    op.set_qk_transform(rms_norm=True)
    d = {n: x[n].cuda() for n in ("q", "k", "v")}
    pq = {n: t.cuda() for n, t in x["phi_q"].items()}
    pk = {n: t.cuda() for n, t in x["phi_k"].items()}
    with pytest.raises(binding.RehyatError) as e:
        op.forward(d["q"], d["k"], d["v"], pq, pk, wl.T, wl.H, wl.W, wl.Tc, wl.To)
    assert e.value.code == binding.ERR_INVALID_ARG
    op.close()


@pytest.mark.parametrize("resume_after", [None, 2])
def test_transform_chunk_by_chunk(resume_after):
    """rehyat_stream_step with a transform set: k is transformed on its way into the window buffer, q into a buffer
    of one chunk, rotation tables read at the running position.  All steps together equal the oracle on the whole
    transformed sequence; a sequence resumed from an exported state continues bit for bit."""
    from paper_2601_04342_b200 import binding
    wl = synth.Workload("qk_stream", 2, 2, 128, 7, 9, 17, 2, 1, "bf16", False, seed=synth.BASE_SEED + 99)
    x, wq, wk, cos, sin = _case(wl, 19)
    ref, _ = _oracle(wl, x, wq, wk, cos, sin)
    d = {n: x[n].cuda() for n in ("q", "k", "v")}
    pq = {n: t.cuda() for n, t in x["phi_q"].items()}
    pk = {n: t.cuda() for n, t in x["phi_k"].items()}
    keep = [wq.cuda(), wk.cuda(), cos.cuda(), sin.cuda()]

    def make():
        op = binding.for_workload(wl, qk_transform=True)
        op.set_qk_transform(q_weight=keep[0], k_weight=keep[1], eps=1e-6, cos=keep[2], sin=keep[3])
        return op

    def run(resume):
        op = make()
        out = torch.full_like(d["q"], float("nan"))
        op.stream_begin(wl.B, wl.H, wl.W, wl.Tc, wl.To)
        for t in range(-(-wl.T // wl.Tc)):
            f0, f1 = t * wl.Tc, min((t + 1) * wl.Tc, wl.T)
            sl = slice(f0 * wl.HW, f1 * wl.HW)
            op.stream_step(d["q"][:, :, sl], d["k"][:, :, sl], d["v"][:, :, sl], pq, pk, f1 - f0, out=out[:, :, sl])
            assert op.status() == 0
            if resume is not None and t + 1 == resume:
                blob = op.stream_export()
                op.close()
                op = make()
                op.stream_import(blob)
        op.close()
        return out

    y = run(None)
    _check(y.double().cpu().numpy(), ref, "bf16")
    if resume_after is not None:
        assert torch.equal(run(resume_after), y)
