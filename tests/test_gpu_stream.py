"""Chunk-by-chunk processing (rehyat_stream_*): the recurrence of Eq. 14-18 with the state held by the
context.  The outputs of all steps together must match the fp64 oracle of the whole sequence within the
tolerances of test_gpu_parity.py, whatever the chunk / overlap geometry; a sequence resumed from an
exported state must continue bit-for-bit."""
import numpy as np
import pytest
import torch

from oracle import rehyat_oracle as orc
from paper_2601_04342_b200 import synth

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("both_window_kernels")]


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2601_04342_b200 import build
    build.build()


def _dev(x):
    d = {n: x[n].cuda() for n in ("q", "k", "v")}
    d["phi_q"] = {n: t.cuda() for n, t in x["phi_q"].items()}
    d["phi_k"] = {n: t.cuda() for n, t in x["phi_k"].items()}
    return d


def stream_all(op, wl, d, resume_after=None, make_op=None):
    """Feeds the sequence chunk by chunk; optionally exports the state after `resume_after` chunks and
    continues on a fresh context made by `make_op`."""
    HW = wl.HW
    out = torch.empty_like(d["q"])
    op.stream_begin(wl.B, wl.H, wl.W, wl.Tc, wl.To)
    n_chunks = -(-wl.T // wl.Tc)
    for t in range(n_chunks):
        f0, f1 = t * wl.Tc, min((t + 1) * wl.Tc, wl.T)
        sl = slice(f0 * HW, f1 * HW)
        q, k, v = (d[n][:, :, sl].contiguous() for n in ("q", "k", "v"))
        out[:, :, sl] = op.stream_step(q, k, v, d["phi_q"], d["phi_k"], f1 - f0)
        assert op.status() == 0
        if resume_after is not None and t + 1 == resume_after:
            blob = op.stream_export()
            op.close()
            op = make_op()
            op.stream_import(blob)
    op.close()
    return out


def gate(y, ref, dtype):
    err = np.abs(y - ref)
    if dtype == "fp32":
        assert err.max() <= 1e-4, f"max-abs {err.max():.3e}"
        return
    assert err.max() <= 2e-2, f"max-abs {err.max():.3e}"
    worst = (err / (3e-3 + 2.0 ** -7 * np.abs(ref))).max()
    assert worst <= 1.0, f"internal gate exceeded x{worst:.2f}, max-abs {err.max():.3e}"
    assert np.sqrt((err ** 2).mean() / (ref ** 2).mean()) <= 1e-2


CASES = [
    # name, B, heads, d, T, H, W, Tc, To, dtype
    ("fp32_tiny", 1, 2, 64, 4, 8, 8, 1, 1, "fp32"),
    ("fp32_short_last_chunk", 2, 2, 128, 5, 9, 11, 2, 1, "fp32"),
    ("bf16_multi_tile", 1, 2, 128, 7, 10, 20, 2, 1, "bf16"),            # last chunk 1 frame
    ("bf16_no_overlap", 1, 3, 128, 6, 13, 11, 2, 0, "bf16"),
    ("bf16_overlap_ge_chunk", 1, 2, 128, 6, 12, 12, 1, 3, "bf16"),
    ("bf16_d64", 1, 2, 64, 5, 10, 13, 2, 1, "bf16"),
    ("bf16_d64_multi_tile", 2, 3, 64, 7, 10, 20, 2, 1, "bf16"),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_stream_matches_the_oracle_of_the_whole_sequence(case):
    from paper_2601_04342_b200 import binding
    name, B, nh, d, T, H, W, Tc, To, dtype = case
    wl = synth.Workload(name, B, nh, d, T, H, W, Tc, To, dtype, dtype == "bf16", seed=synth.BASE_SEED + 91)
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    f = synth.to_f64(x)
    ref, frac = orc.hybrid_direct(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To,
                                  return_parts=True)
    dev = _dev(x)
    y = stream_all(binding.for_workload(wl), wl, dev)
    gate(y.double().cpu().numpy(), ref, dtype)
    assert frac.max() > 0.05                         # the carried state matters in this case
    # and the one-call entry point agrees up to the rounding of a different summation order
    op = binding.for_workload(wl)
    y_full = op.forward(dev["q"], dev["k"], dev["v"], dev["phi_q"], dev["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To)
    op.close()
    tol = 1e-5 if dtype == "fp32" else 2.0 ** -6
    assert float(((y.float() - y_full.float()).abs() / (1e-3 + y_full.float().abs())).max()) <= tol


def test_resumed_sequence_continues_bit_for_bit():
    from paper_2601_04342_b200 import binding
    wl = synth.Workload("resume", 1, 2, 128, 9, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 92)
    dev = _dev(synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True))
    make = lambda: binding.for_workload(wl)
    straight = stream_all(make(), wl, dev)
    for after in (1, 3):
        resumed = stream_all(make(), wl, dev, resume_after=after, make_op=make)
        assert torch.equal(straight, resumed)


def test_stream_at_the_wan_layer_shape_sampled_rows():
    """21 frames of 30x52 fed as seven chunks of three frames: device memory of the sequence is one chunk
    plus the overlap, the result that of the whole-sequence operator."""
    from paper_2601_04342_b200 import binding
    wl = synth.CONFIGS["wan13b_layer"]
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    f = synth.to_f64(x)
    y = stream_all(binding.for_workload(wl), wl, _dev(x)).cpu()
    rng = np.random.default_rng(5)
    for h in (0, 11):
        rows = np.unique(np.concatenate([np.arange(0, 128), np.arange(4680 - 72, 4680 + 128), np.arange(wl.N - 200, wl.N),
                                         rng.integers(0, wl.N, 256)]))
        ref, _ = orc.hybrid_rows(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To, 0, h, rows)
        gate(y[0, h, rows].double().numpy(), ref, "bf16")


def test_stream_argument_checks():
    from paper_2601_04342_b200 import binding
    wl = synth.CONFIGS["tiny_fp32"]
    d = _dev(synth.make_inputs(wl))
    op = binding.for_workload(wl)
    q = d["q"][:, :, :wl.HW].contiguous()
    with pytest.raises(binding.RehyatError):            # no sequence started
        op.stream_step(q, q, q, d["phi_q"], d["phi_k"], 1)
    with pytest.raises(binding.RehyatError):            # chunk beyond the context's maximum
        op.stream_begin(1, wl.H, wl.W, 2, 1)
    op.stream_begin(1, wl.H, wl.W, 1, 1)
    with pytest.raises(binding.RehyatError):            # more frames than the chunk size
        op.stream_step(q, q, q, d["phi_q"], d["phi_k"], 2)
    blob = op.stream_export()
    with pytest.raises(binding.RehyatError):            # a damaged blob
        op.stream_import(b"\x00" * len(blob))
    op.close()


@pytest.mark.parametrize("layout", ["bhnd", "bnhd"])
def test_chunks_as_views_of_the_whole_sequence(layout):
    """q is read and out is written in place, with the caller's strides: the chunks are passed as views of the
    whole [B, heads, N, d] (or token-major [B, N, heads, d]) tensors, nothing is made contiguous."""
    from paper_2601_04342_b200 import binding
    wl = synth.Workload("views", 2, 3, 128, 7, 9, 17, 2, 1, "bf16", True, seed=synth.BASE_SEED + 97)
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    f = synth.to_f64(x)
    ref = orc.hybrid_rnn(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To, P=wl.P)
    d = _dev(x)
    if layout == "bnhd":                                     # token-major storage, seen as [B, heads, N, d]
        full = {n: d[n].transpose(1, 2).contiguous().transpose(1, 2) for n in ("q", "k", "v")}
    else:
        full = {n: d[n] for n in ("q", "k", "v")}
    out = torch.full_like(full["q"], float("nan"))
    assert out.stride() == full["q"].stride()
    op = binding.for_workload(wl)
    op.stream_begin(wl.B, wl.H, wl.W, wl.Tc, wl.To)
    for t in range(-(-wl.T // wl.Tc)):
        f0, f1 = t * wl.Tc, min((t + 1) * wl.Tc, wl.T)
        sl = slice(f0 * wl.HW, f1 * wl.HW)
        q, k, v = (full[n][:, :, sl] for n in ("q", "k", "v"))
        o = out[:, :, sl]
        assert not q.is_contiguous()
        op.stream_step(q, k, v, d["phi_q"], d["phi_k"], f1 - f0, out=o)
        assert op.status() == 0
    op.close()
    gate(out.double().cpu().numpy(), ref, "bf16")
