"""Behaviour of the C ABI beyond the arithmetic: the bounded device-side waits and what the host sees when one
runs out, contexts that live side by side, and validation before anything is enqueued or copied.

No test here faults, traps or hangs the GPU: the time-out test makes the producers of the tensor-core kernels
issue no loads at all (rehyat_set_wait_limit's test hook), so that the waits run out with nothing in flight,
every CTA frees its TMEM and returns, and the context stays usable."""
import ctypes as C

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


def _dev(x):
    d = {n: x[n].cuda() for n in ("q", "k", "v")}
    d["phi_q"] = {n: t.cuda() for n, t in x["phi_q"].items()}
    d["phi_k"] = {n: t.cuda() for n, t in x["phi_k"].items()}
    return d


def _oracle(wl, x, **kw):
    f = synth.to_f64(x)
    return orc.hybrid_rnn(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To, P=wl.P, **kw)


@pytest.mark.parametrize("shape", ["default", "heads_of_64", "three_layers"])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(both_window_kernels, shape):
    """All four tensor-core kernels (state, read-out and either window kernel) run into their wait limit, the
    host reads REHYAT_ERR_DEVICE_TIMEOUT exactly once, and the next forward on the same context gives the bits
    it gave before.  The default shape runs the fixed-extent phi kernels, the other two the ones that read their
    extents (64-column tiles; hidden layers in between)."""
    from paper_2601_04342_b200 import binding
    d, layers = {"default": (128, 2), "heads_of_64": (64, 2), "three_layers": (128, 3)}[shape]
    wl = synth.Workload("timeout", 1, 2, d, 6, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 70, phi_layers=layers)
    x = synth.make_inputs(wl, phi_scale=1.5 if layers == 2 else 2.0, v_frame_offsets=True)
    d = _dev(x)
    op = binding.for_workload(wl)
    args = (d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To)
    before = op.forward(*args).clone()
    assert op.status() == binding.OK and op.last_impl == op.last_phi_impl == "tensor"
    assert np.abs(before.double().cpu().numpy() - _oracle(wl, x)).max() <= 2e-2

    op.set_wait_limit(2000, withhold_loads=True)              # 2 ms per wait, no loads: every launch gives up
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    op.forward(*args)                                          # enqueues; the output of this call is undefined
    t1.record()
    assert op.status() == binding.ERR_DEVICE_TIMEOUT
    assert t0.elapsed_time(t1) < 500.0                         # the launches ended by themselves, quickly
    assert op.status() == binding.OK                           # reading clears the record

    op.set_wait_limit(0, withhold_loads=False)
    after = op.forward(*args)
    assert op.status() == binding.OK
    assert torch.equal(after, before)
    op.close()


def test_contexts_with_different_phi_widths_live_side_by_side():
    """The shared-memory limit of a kernel belongs to the function, not to a context: a context with narrow phi
    widths created (or a static call made) while a wider one is alive must not break the wider one."""
    from paper_2601_04342_b200 import binding
    wide = synth.Workload("wide", 1, 2, 128, 5, 9, 11, 2, 1, "bf16", True, seed=synth.BASE_SEED + 71)
    narrow = wide.with_(name="narrow", phi_hidden=64, phi_dim=64, seed=synth.BASE_SEED + 72)
    xs = {w.name: synth.make_inputs(w, phi_scale=1.5, v_frame_offsets=True) for w in (wide, narrow)}
    refs = {w.name: _oracle(w, xs[w.name]) for w in (wide, narrow)}
    devs = {n: _dev(x) for n, x in xs.items()}
    ops = {"wide": binding.for_workload(wide, impl="simt")}

    def run(w):
        d = devs[w.name]
        y = ops[w.name].forward(d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"], w.T, w.H, w.W, w.Tc, w.To)
        assert ops[w.name].status() == binding.OK
        assert np.abs(y.double().cpu().numpy() - refs[w.name]).max() <= 2e-2

    run(wide)
    ops["narrow"] = binding.for_workload(narrow, impl="simt")   # created under the live wide context
    run(narrow)
    run(wide)
    d = devs["narrow"]
    y = binding.forward_static(d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"], narrow.T, narrow.H, narrow.W, narrow.Tc,
                               narrow.To, dtype="bf16", phi_hidden=64, phi_dim=64)
    assert np.abs(y.double().cpu().numpy() - refs["narrow"]).max() <= 2e-2
    run(wide)
    run(narrow)
    for op in ops.values():
        op.close()


def test_forward_host_validates_before_the_first_copy():
    """A chunk beyond max_chunk_frames is refused with INVALID_ARG before staging memory is allocated or a byte is
    copied: device memory in use does not move and the host output keeps its sentinel."""
    from paper_2601_04342_b200 import binding
    wl = synth.Workload("hostval", 1, 2, 128, 6, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 73)
    x = synth.make_inputs(wl)
    op = binding.for_workload(wl)
    pq = {n: t.cuda() for n, t in x["phi_q"].items()}
    pk = {n: t.cuda() for n, t in x["phi_k"].items()}
    out = torch.full_like(x["q"], 7.0)
    torch.cuda.synchronize()
    free = torch.cuda.mem_get_info()[0]
    for bad in (dict(chunk=wl.Tc + 1), dict(chunk=0), dict(overlap=-1), dict(frames=0), dict(H=wl.H * 2)):
        a = dict(frames=wl.T, H=wl.H, W=wl.W, chunk=wl.Tc, overlap=wl.To)
        a.update(bad)
        with pytest.raises(binding.RehyatError) as e:
            op.forward_host(x["q"], x["k"], x["v"], out, pq, pk, a["frames"], a["H"], a["W"], a["chunk"], a["overlap"])
        assert e.value.code == binding.ERR_INVALID_ARG, bad
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free
    assert bool((out == 7.0).all())
    # and the same call with legal arguments works
    op.forward_host(x["q"], x["k"], x["v"], out, pq, pk, wl.T, wl.H, wl.W, wl.Tc, wl.To)
    assert np.abs(out.double().numpy() - _oracle(wl, x)).max() <= 2e-2
    op.close()


def test_zero_strides_of_one_element_axes_and_bad_strides():
    """batch = 1 with stride_batch = 0 is accepted (the stride is never used); a head stride that would put two
    heads on top of each other is refused before launch."""
    from paper_2601_04342_b200 import binding
    wl = synth.Workload("strides", 1, 2, 128, 4, 8, 10, 2, 1, "bf16", True, seed=synth.BASE_SEED + 74)
    x = synth.make_inputs(wl)
    d = _dev(x)
    op = binding.for_workload(wl)
    out = torch.empty_like(d["q"])
    phi = op.phi_struct(d["phi_q"], d["phi_k"])
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    L = binding.lib()

    def call(lay):
        return L.rehyat_forward(op._h, binding._ptr(d["q"]), binding._ptr(d["k"]), binding._ptr(d["v"]), binding._ptr(out),
                                C.byref(lay), C.byref(phi), 1, wl.T, wl.H, wl.W, wl.Tc, wl.To, st)

    N, dd = wl.N, wl.head_dim
    assert call(binding.Layout(0, N * dd, dd)) == binding.OK
    assert op.status() == binding.OK
    assert np.abs(out.double().cpu().numpy() - _oracle(wl, x)).max() <= 2e-2
    assert call(binding.Layout(2 * N * dd, 0, dd)) == binding.ERR_INVALID_ARG
    assert call(binding.Layout(2 * N * dd, N * dd, dd - 8)) == binding.ERR_INVALID_ARG
    op.close()


def test_a_layer_split_over_three_ranks_equals_the_layer_in_one_call():
    """binding.ShardedRehyat with the ranks run one after the other on this GPU (independent launches, nothing
    waits on another rank): every rank writes only its own (batch, head) blocks, and together they give, bit for
    bit, what one call on all heads gives."""
    from paper_2601_04342_b200 import binding, geometry
    wl = synth.Workload("shard", 2, 4, 128, 5, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 75)
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    d = _dev(x)
    op = binding.for_workload(wl, window_tiles=2)
    whole = op.forward(d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To)
    assert op.status() == binding.OK
    op.close()
    assert np.abs(whole.double().cpu().numpy() - _oracle(wl, x)).max() <= 2e-2
    out = torch.full_like(d["q"], float("nan"))
    world = 3                                                 # 8 problems over 3 ranks: 3, 3, 2, with cuts inside batch items
    for rank in range(world):
        sh = binding.ShardedRehyat(world, rank, batch=wl.B, n_heads=wl.n_heads, head_dim=wl.head_dim, dtype=wl.dtype,
                                   phi_hidden=wl.D_h, phi_dim=wl.D_out, poly_degree=wl.P, max_tokens_per_frame=wl.HW,
                                   max_chunk_frames=wl.Tc, window_tiles=2)
        before = out.clone()
        sh.forward(d["q"], d["k"], d["v"], out, d["phi_q"], d["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To)
        assert sh.status() == binding.OK and sh.last_launches > 0
        mine = torch.zeros((wl.B, wl.n_heads), dtype=torch.bool)
        for (b0, nb, h0, nh) in geometry.shard_rects(wl.B, wl.n_heads, world, rank):
            mine[b0:b0 + nb, h0:h0 + nh] = True
        changed = ~(torch.isnan(out) == torch.isnan(before)).flatten(2).all(dim=2).cpu()
        assert torch.equal(changed, mine)                     # exactly this rank's blocks were written
        sh.close()
    assert torch.equal(out, whole)


def test_output_that_starts_off_a_32_byte_boundary(both_window_kernels):
    """The window kernel writes whole 32-byte sectors where every output row starts on a 32-byte boundary and
    16-byte pieces otherwise (the ABI asks for 16-byte alignment only): both forms give the same bits."""
    from paper_2601_04342_b200 import binding
    wl = synth.Workload("align", 1, 2, 128, 5, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 76)
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    d = _dev(x)
    op = binding.for_workload(wl)
    args = (d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To)
    aligned = op.forward(*args).clone()
    assert aligned.data_ptr() % 32 == 0
    flat = torch.full((d["q"].numel() + 16,), float("nan"), device="cuda", dtype=d["q"].dtype)
    shifted = flat[8:8 + d["q"].numel()].view_as(d["q"])          # 16 bytes further: rows no longer start on 32 bytes
    assert shifted.data_ptr() % 32 == 16
    op.forward(*args, out=shifted)
    assert op.status() == binding.OK
    assert torch.equal(shifted, aligned)
    assert bool(torch.isnan(flat[:8]).all()) and bool(torch.isnan(flat[8 + d["q"].numel():]).all())
    assert np.abs(aligned.double().cpu().numpy() - _oracle(wl, x)).max() <= 2e-2
    op.close()
