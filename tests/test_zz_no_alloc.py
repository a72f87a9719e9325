"""rehyat_forward_static: the entry point for callers that cannot allocate device memory (a fixed
memory plan, a loop that cannot take cudaMalloc's synchronisation).  Its workspace is a fixed array
inside the library, shared by all calls and never cleared, so every case is run on two calls in a
row with different inputs: the second call must not be disturbed by what the first one left behind.

Each output is checked against the fp64 oracle (the gates of the other parity tests) and against the
context entry point running the same SIMT kernels.  The two entry points differ in one thing only, the
number of pieces a chunk's state sum is split into (the context has room for more partial sums), so
they agree to the rounding of an fp32 sum taken in another order, not bit for bit.

Collected last on purpose: a run that stops at the first failure has then run every other test."""
import numpy as np
import pytest
import torch

from oracle import rehyat_oracle as orc
from paper_2601_04342_b200 import synth

pytestmark = pytest.mark.gpu


def _dev(x):
    d = {n: x[n].cuda() for n in ("q", "k", "v")}
    d["phi_q"] = {n: t.cuda() for n, t in x["phi_q"].items()}
    d["phi_k"] = {n: t.cuda() for n, t in x["phi_k"].items()}
    return d


def _scratch_floats(wl):
    """The capacity formula of include/rehyat.h."""
    chunks = -(-wl.T // min(wl.Tc, wl.T))
    BH, SD, Np = wl.B * wl.n_heads, wl.head_dim + 4, min(wl.Tc, wl.T) * wl.HW
    return 2 * chunks * BH * wl.D_out * SD + BH * chunks * (-(-Np // 128) * 128) * SD


CASES = [
    (synth.CONFIGS["tiny_fp32"], dict(phi_scale=1.0)),
    (synth.Workload("static_bf16", 1, 2, 128, 5, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 90),
     dict(phi_scale=1.5, v_frame_offsets=True)),
    # the largest number of chunks the entry point takes
    (synth.Workload("static_16_chunks", 1, 2, 64, 16, 8, 8, 1, 1, "fp32", False, seed=synth.BASE_SEED + 92),
     dict(phi_scale=3.0, v_frame_offsets=True)),
    # 2,095,104 of the 2,097,152 floats of the array: two chunks of 27 tiles of 128 rows
    (synth.Workload("static_near_capacity", 1, 2, 128, 2, 48, 72, 1, 0, "bf16", True, seed=synth.BASE_SEED + 93),
     dict(phi_scale=1.5, v_frame_offsets=True)),
]


@pytest.mark.parametrize("wl,kw", CASES, ids=[c[0].name for c in CASES])
def test_static_entry_point_twice_in_a_row_against_the_oracle_and_the_context_entry_point(wl, kw):
    from paper_2601_04342_b200 import binding, build
    build.build()
    cap = binding.lib().rehyat_static_scratch_bytes()
    assert cap == 8 << 20 and _scratch_floats(wl) * 4 <= cap
    if wl.name == "static_near_capacity":
        assert _scratch_floats(wl) * 4 > 0.99 * cap
    for call in range(2):
        w = wl.with_(seed=wl.seed + call)
        x = synth.make_inputs(w, **kw)
        f = synth.to_f64(x)
        ref = orc.hybrid_rnn(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], w.T, w.HW, w.Tc, w.To, P=w.P)
        d = _dev(x)
        op = binding.for_workload(w, impl="simt")
        want = op.forward(d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"], w.T, w.H, w.W, w.Tc, w.To)
        assert op.status() == 0
        op.close()
        out = torch.full_like(d["q"], float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]      # driver-level: a cudaMalloc in the library would lower it
        got = binding.forward_static(d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"], w.T, w.H, w.W, w.Tc, w.To,
                                     dtype=w.dtype, poly_degree=w.P, phi_hidden=w.D_h, phi_dim=w.D_out, out=out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        y = got.double().cpu().numpy()
        err = np.abs(y - ref)
        assert np.isfinite(y).all()
        if w.dtype == "fp32":
            assert err.max() <= 1e-4, f"{w.name} call {call}: max-abs {err.max():.3e}"
            same = 1e-5 + 1e-5 * np.abs(ref)
        else:
            assert err.max() <= 2e-2, f"{w.name} call {call}: max-abs {err.max():.3e}"
            assert (err / (3e-3 + 2.0 ** -7 * np.abs(ref))).max() <= 1.0
            assert np.sqrt((err ** 2).mean() / (ref ** 2).mean()) <= 1e-2
            same = 1e-5 + 2.0 ** -7 * np.abs(ref)      # one bf16 step of the output
        assert (np.abs(y - want.double().cpu().numpy()) <= same).all(), f"{w.name} call {call}: differs from the context call"


def test_static_entry_point_rejects_what_does_not_fit():
    from paper_2601_04342_b200 import binding, build
    build.build()
    big = synth.Workload("too_big", 1, 12, 128, 6, 30, 52, 3, 1, "bf16", True)
    one_tile_too_many = synth.Workload("over_capacity", 1, 2, 128, 2, 49, 71, 1, 0, "bf16", True)   # 28 tiles per chunk
    seventeen_chunks = synth.Workload("17_chunks", 1, 2, 64, 17, 8, 8, 1, 1, "fp32", False)
    assert _scratch_floats(one_tile_too_many) * 4 > binding.lib().rehyat_static_scratch_bytes()
    for wl in (big, one_tile_too_many, seventeen_chunks):
        dt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
        q = torch.zeros((1, wl.n_heads, wl.N, wl.head_dim), dtype=dt, device="cuda")
        out = torch.full_like(q, 5.0)
        p = {n: t.cuda() for n, t in synth.make_phi_params(wl, "phi_q").items()}
        with pytest.raises(binding.RehyatError) as e:
            binding.forward_static(q, q.clone(), q.clone(), p, p, wl.T, wl.H, wl.W, wl.Tc, wl.To, dtype=wl.dtype, out=out)
        assert e.value.code == binding.ERR_TOO_LARGE, wl.name
        torch.cuda.synchronize()
        assert bool((out == 5.0).all())                 # nothing was launched
    assert b"fixed scratch" in binding.lib().rehyat_strerror(binding.ERR_TOO_LARGE)
