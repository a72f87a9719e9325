"""The bidirectional variant (Eq. 10-12: the linear branch covers every token outside the softmax window,
earlier and later) against the fp64 oracle evaluated with the same sets, element by element."""
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


def run(wl, x, **kw):
    from paper_2601_04342_b200 import binding
    op = binding.for_workload(wl, bidirectional=True, **kw)
    q, k, v = (x[n].cuda() for n in ("q", "k", "v"))
    pq = {n: t.cuda() for n, t in x["phi_q"].items()}
    pk = {n: t.cuda() for n, t in x["phi_k"].items()}
    y = op.forward(q, k, v, pq, pk, wl.T, wl.H, wl.W, wl.Tc, wl.To)
    assert op.status() == 0
    y2 = op.forward(q, k, v, pq, pk, wl.T, wl.H, wl.W, wl.Tc, wl.To)      # the per-frame sums are reused buffers
    assert torch.equal(y, y2)
    used = op.last_impl
    op.close()
    return y.double().cpu().numpy(), used


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
    ("fp32_non_overlapping", 1, 2, 64, 4, 8, 8, 1, 0, "fp32"),             # Eq. 10-11
    ("fp32_overlapping_ragged", 2, 2, 128, 5, 9, 11, 2, 1, "fp32"),        # Eq. 12, last chunk short
    ("bf16_non_overlapping", 1, 2, 128, 6, 10, 20, 2, 0, "bf16"),
    ("bf16_overlapping", 1, 3, 128, 7, 10, 20, 3, 1, "bf16"),
    ("bf16_overlap_ge_chunk", 1, 2, 128, 6, 12, 12, 1, 3, "bf16"),
    ("bf16_many_frames", 1, 2, 128, 19, 6, 8, 2, 1, "bf16"),                # more frames than one scan group
    ("bf16_d64", 1, 2, 64, 5, 10, 13, 2, 1, "bf16"),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_bidirectional_matches_the_oracle(case):
    name, B, nh, d, T, H, W, Tc, To, dtype = case
    wl = synth.Workload(name, B, nh, d, T, H, W, Tc, To, dtype, dtype == "bf16", seed=synth.BASE_SEED + 95)
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    f = synth.to_f64(x)
    ref = orc.hybrid_direct(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To, causal=False)
    causal = orc.hybrid_direct(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To, causal=True)
    assert np.abs(ref - causal).max() > 0.05          # the two variants differ visibly on these inputs
    y, used = run(wl, x)
    assert used == ("tensor" if dtype == "bf16" else "simt")
    gate(y, ref, dtype)


def test_one_chunk_is_full_softmax_in_both_variants():
    wl = synth.Workload("full", 1, 2, 128, 3, 10, 20, 3, 0, "bf16", True, seed=synth.BASE_SEED + 96)
    x = synth.make_inputs(wl)
    f = synth.to_f64(x)
    y, _ = run(wl, x)
    gate(y, orc.softmax_attention(f["q"], f["k"], f["v"]), "bf16")


def test_chunk_by_chunk_and_static_entry_points_refuse_it():
    from paper_2601_04342_b200 import binding
    wl = synth.CONFIGS["tiny_fp32"]
    op = binding.for_workload(wl, bidirectional=True)
    with pytest.raises(binding.RehyatError) as e:
        op.stream_begin(1, wl.H, wl.W, 1, 1)
    assert e.value.code == binding.ERR_UNSUPPORTED
    op.close()
