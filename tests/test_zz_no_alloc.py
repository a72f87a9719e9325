"""rehyat_forward_static: the entry point for callers that cannot allocate device memory (a fixed
memory plan, a loop that cannot take cudaMalloc's synchronisation).  Its workspace is a fixed array
inside the library, shared by all calls and never cleared, so the check is made on two calls in a
row with different inputs: the second call must not be disturbed by what the first one left behind.
Collected last on purpose: a run that stops at the first failure has then run every other test."""
import numpy as np
import pytest
import torch

from paper_2601_04342_b200 import synth

pytestmark = pytest.mark.gpu


def _dev(x):
    d = {n: x[n].cuda() for n in ("q", "k", "v")}
    d["phi_q"] = {n: t.cuda() for n, t in x["phi_q"].items()}
    d["phi_k"] = {n: t.cuda() for n, t in x["phi_k"].items()}
    return d


CASES = [
    (synth.CONFIGS["tiny_fp32"], dict(phi_scale=1.0), 1e-4),
    (synth.Workload("static_bf16", 1, 2, 128, 5, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 90),
     dict(phi_scale=1.5, v_frame_offsets=True), 2e-2),
]


def test_static_entry_point_matches_the_context_entry_point_twice_in_a_row():
    from paper_2601_04342_b200 import binding, build
    build.build()
    assert binding.lib().rehyat_static_scratch_bytes() == 8 << 20
    for wl, kw, tol in CASES:
        for call in range(2):
            x = synth.make_inputs(wl.with_(seed=wl.seed + call), **kw)
            d = _dev(x)
            op = binding.for_workload(wl, impl="simt")
            want = op.forward(d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To)
            assert op.status() == 0
            op.close()
            out = torch.full_like(d["q"], float("nan"))
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]      # driver-level: a cudaMalloc in the library would lower it
            got = binding.forward_static(d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To,
                                         dtype=wl.dtype, poly_degree=wl.P, phi_hidden=wl.D_h, phi_dim=wl.D_out, out=out)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before
            err = (got.double() - want.double()).abs().max().item()
            assert np.isfinite(err) and err <= tol, f"{wl.name} call {call}: max-abs {err:.3e}"


def test_static_entry_point_rejects_what_does_not_fit():
    from paper_2601_04342_b200 import binding, build
    build.build()
    wl = synth.Workload("too_big", 1, 12, 128, 6, 30, 52, 3, 1, "bf16", True)
    q = torch.zeros((1, 12, wl.N, 128), dtype=torch.bfloat16, device="cuda")
    p = {n: t.cuda() for n, t in synth.make_phi_params(wl, "phi_q").items()}
    with pytest.raises(binding.RehyatError) as e:
        binding.forward_static(q, q.clone(), q.clone(), p, p, wl.T, wl.H, wl.W, wl.Tc, wl.To, dtype="bf16")
    assert e.value.code == binding.ERR_TOO_LARGE
    assert b"fixed scratch" in binding.lib().rehyat_strerror(binding.ERR_TOO_LARGE)
