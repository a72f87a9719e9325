"""Parity of the CUDA path (through the C ABI) with the fp64 oracle, element by element, on the
same seeded inputs.

Tolerances.  fp32 mode: max-abs <= 1e-4.  bf16 mode: the contract is max-abs <= 2e-2; because
y is an average over thousands of keys and small on N(0,1) values, every bf16 case must also
meet an internal gate: |err| <= 3e-3 + 2^-7 |y| element-wise (bf16 rounding of the output is
2^-9 |y|, of the softmax weights and phi features 2^-9 relative each) and rel-RMS <= 1e-2.
"""
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


def _to_dev(x):
    dev = {n: x[n].cuda() for n in ("q", "k", "v")}
    dev["phi_q"] = {n: t.cuda() for n, t in x["phi_q"].items()}
    dev["phi_k"] = {n: t.cuda() for n, t in x["phi_k"].items()}
    return dev


def run_gpu(wl, x, *, impl="auto", c_mode="rowmax", layout="bhnd", **kw):
    from paper_2601_04342_b200 import binding
    op = binding.for_workload(wl, impl=impl, c_mode=c_mode, **kw)
    d = _to_dev(x)
    q, k, v = d["q"], d["k"], d["v"]
    if layout == "bnhd":
        q, k, v = (t.transpose(1, 2).contiguous() for t in (q, k, v))
    y = op.forward(q, k, v, d["phi_q"], d["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To, layout=layout)
    assert op.status() == 0
    assert op.last_launches > 0
    if layout == "bnhd":
        y = y.transpose(1, 2)
    used = op.last_impl
    run_gpu.phi_kernels = op.last_phi_impl          # kernels of phi, state and read-out in this call
    op.close()
    return y.double().cpu().numpy(), used


def check(y, ref, dtype):
    err = np.abs(y - ref)
    if dtype == "fp32":
        assert err.max() <= 1e-4, f"max-abs {err.max():.3e}"
    else:
        assert err.max() <= 2e-2, f"max-abs {err.max():.3e}"
        bound = 3e-3 + 2.0 ** -7 * np.abs(ref)
        worst = (err / bound).max()
        assert worst <= 1.0, f"internal gate exceeded x{worst:.2f}, max-abs {err.max():.3e}"
        rel_rms = np.sqrt((err ** 2).mean() / (ref ** 2).mean())
        assert rel_rms <= 1e-2, f"rel-RMS {rel_rms:.3e}"


def oracle_full(wl, x, c_mode="rowmax"):
    f = synth.to_f64(x)
    return orc.hybrid_direct(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To,
                             c_mode=c_mode, return_parts=True)


# ------------------------------------------------------------------ config 1: tiny fp32
@pytest.mark.parametrize("c_mode", ["rowmax", "zero"])
def test_tiny_fp32_every_element(c_mode):
    wl = synth.CONFIGS["tiny_fp32"]
    x = synth.make_inputs(wl)
    ref, frac = oracle_full(wl, x, c_mode)
    y, used = run_gpu(wl, x, c_mode=c_mode)
    assert used == "simt"
    check(y, ref, "fp32")
    if c_mode == "rowmax":
        assert frac[:, :, 128:].mean() > 0.05  # the linear branch carries visible mass: not vacuous


def test_tiny_fp32_stored_rows():
    import os
    wl = synth.CONFIGS["tiny_fp32"]
    y, _ = run_gpu(wl, synth.make_inputs(wl))
    path = os.path.join(os.path.dirname(__file__), "golden", "tiny_fp32_rows.txt")
    for line in open(path):
        if line.startswith("#"):
            continue
        tok = line.split()
        h, r = int(tok[0]), int(tok[1])
        assert np.max(np.abs(y[0, h, r] - np.array([float(t) for t in tok[2:]]))) <= 1e-4


def test_fp32_stress_variants():
    wl = synth.CONFIGS["tiny_fp32"]
    for kw in (dict(phi_scale=3.0), dict(q_scale=4.0), dict(v_frame_offsets=True, phi_scale=1.5)):
        x = synth.make_inputs(wl, **kw)
        ref, _ = oracle_full(wl, x)
        y, _ = run_gpu(wl, x)
        err = np.abs(y - ref)
        assert (err / (1e-4 + 1e-5 * np.abs(ref))).max() <= 1.0


# ------------------------------------------------------------------ small cases, several tiles + ragged tails
SMALL = [
    # name, B, heads, d, T, H, W, Tc, To, dtype
    ("fp32_d128_ragged", 1, 2, 128, 5, 9, 11, 2, 1, "fp32"),
    ("fp32_d64_overlap_ge_chunk", 2, 2, 64, 6, 5, 7, 1, 2, "fp32"),
    ("bf16_d128_multi_tile", 1, 2, 128, 5, 10, 20, 2, 1, "bf16"),       # HW=200: tiles of 128 end mid-frame
    ("bf16_d128_T_not_divisible", 2, 2, 128, 7, 9, 17, 3, 1, "bf16"),   # HW=153, last chunk 1 frame
    ("bf16_d128_no_overlap", 1, 3, 128, 6, 13, 11, 2, 0, "bf16"),
    ("bf16_d128_overlap_ge_chunk", 1, 2, 128, 6, 12, 12, 1, 3, "bf16"),
    ("bf16_d128_tiny_frames", 1, 2, 128, 9, 3, 5, 2, 1, "bf16"),        # HW=15 < one tile
    ("bf16_d64", 1, 2, 64, 5, 10, 13, 2, 1, "bf16"),
    ("bf16_d64_ragged_batch", 2, 3, 64, 7, 9, 17, 3, 1, "bf16"),        # HW=153, last chunk 1 frame, several key tiles
    ("bf16_d64_no_overlap", 1, 2, 64, 6, 13, 11, 2, 0, "bf16"),
]


@pytest.mark.parametrize("case", SMALL, ids=[c[0] for c in SMALL])
@pytest.mark.parametrize("c_mode", ["rowmax", "zero"])
def test_small_cases_every_element(case, c_mode):
    name, B, nh, d, T, H, W, Tc, To, dtype = case
    wl = synth.Workload(name, B, nh, d, T, H, W, Tc, To, dtype, dtype == "bf16", seed=synth.BASE_SEED + 77)
    # phi parameters x1.5: about 0.8 of the normaliser is linear, 13-20 % of phi in the squared part
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    ref, frac = oracle_full(wl, x, c_mode)
    y, used = run_gpu(wl, x, c_mode=c_mode)
    assert used == run_gpu.phi_kernels == ("tensor" if dtype == "bf16" else "simt")   # bf16: every step on the tensor cores, d = 64 and 128
    check(y, ref, dtype)
    if To < T - Tc and c_mode == "rowmax":
        assert frac.max() > 0.05


@pytest.mark.parametrize("impl", ["simt", "auto"])
def test_bf16_variants_peaky_and_phi_stress(impl):
    wl = synth.Workload("v", 1, 2, 128, 6, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 78)
    for kw in (dict(q_scale=4.0, phi_scale=1.5), dict(phi_scale=3.0), dict(phi_scale=1.0)):
        x = synth.make_inputs(wl, **kw)
        ref, _ = oracle_full(wl, x)
        y, _ = run_gpu(wl, x, impl=impl)
        check(y, ref, "bf16")


def test_groups_smaller_than_the_sequence_carry_the_state():
    """group_tokens below N forces several chunk groups: the state must be carried across them."""
    wl = synth.Workload("g", 1, 2, 128, 9, 10, 20, 1, 1, "bf16", True, seed=synth.BASE_SEED + 79)
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    ref, _ = oracle_full(wl, x)
    y_one, _ = run_gpu(wl, x)
    y_many, _ = run_gpu(wl, x, group_tokens=400)          # 2 chunks per group
    check(y_many, ref, "bf16")
    # the split of the partial state sums differs with the group size, so only rounding may differ
    assert np.max(np.abs(y_one - y_many) / (1e-3 + np.abs(y_one))) <= 2.0 ** -6


@pytest.mark.parametrize("impl,c_mode", [("auto", "rowmax"), ("auto", "zero"), ("simt", "rowmax")])
def test_linear_share_of_the_normaliser(impl, c_mode):
    """rehyat_set_linear_share_output: nL / (nS + nL) per query row (Eq. 8, 9) as the window kernels weigh it,
    against the same ratio from the oracle's explicit sums."""
    from paper_2601_04342_b200 import binding
    wl = synth.Workload("share", 2, 2, 128, 5, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 88)
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    ref, frac = oracle_full(wl, x, c_mode)
    d = _to_dev(x)
    op = binding.for_workload(wl, impl=impl, c_mode=c_mode)
    share = torch.full((wl.B, wl.n_heads, wl.N), -1.0, device="cuda")
    op.set_linear_share_output(share)
    y = op.forward(d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To)
    assert op.status() == 0
    check(y.double().cpu().numpy(), ref, "bf16")
    got = share.double().cpu().numpy()
    assert frac.max() > 0.3 and np.abs(got - frac).max() <= 5e-3
    assert (got[:, :, :wl.Tc * wl.HW] == 0).all()            # chunk 0 has no linear set
    op.set_linear_share_output(None)
    op.close()


def test_token_major_layout():
    wl = synth.Workload("l", 2, 2, 128, 4, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 80)
    x = synth.make_inputs(wl, phi_scale=1.5)
    ref, _ = oracle_full(wl, x)
    y, _ = run_gpu(wl, x, layout="bnhd")
    check(y, ref, "bf16")


# ------------------------------------------------------------------ limiting cases on the GPU
def test_chunk_covering_everything_is_full_softmax():
    wl = synth.Workload("full", 1, 2, 128, 3, 10, 20, 3, 1, "bf16", True, seed=synth.BASE_SEED + 81)
    x = synth.make_inputs(wl)
    f = synth.to_f64(x)
    ref = orc.softmax_attention(f["q"], f["k"], f["v"])
    for Tc in (3, 50):
        y, _ = run_gpu(wl.with_(Tc=Tc), x)
        check(y, ref, "bf16")


def test_rows_sum_to_one():
    wl = synth.Workload("ones", 1, 2, 128, 6, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 82)
    x = synth.make_inputs(wl, v_ones=True, phi_scale=1.5)
    y, _ = run_gpu(wl, x)
    assert np.max(np.abs(y - 1.0)) <= 2.0 ** -8


def test_same_input_twice_is_bitwise_equal():
    wl = synth.Workload("det", 1, 2, 128, 6, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 83)
    x = synth.make_inputs(wl, phi_scale=1.5)
    a, _ = run_gpu(wl, x)
    b, _ = run_gpu(wl, x)
    assert np.array_equal(a, b)


# ------------------------------------------------------------------ argument validation (host side only)
def test_invalid_arguments_are_rejected_before_launch():
    from paper_2601_04342_b200 import binding
    wl = synth.CONFIGS["tiny_fp32"]
    d = _to_dev(synth.make_inputs(wl))
    op = binding.for_workload(wl)
    args = (d["q"], d["k"], d["v"], d["phi_q"], d["phi_k"])
    for bad in (dict(chunk=0), dict(overlap=-1), dict(frames=0), dict(H=9)):      # H*W over max
        kw = dict(frames=wl.T, H=wl.H, W=wl.W, chunk=wl.Tc, overlap=wl.To)
        kw.update(bad)
        with pytest.raises(binding.RehyatError) as e:
            op.forward(*args, kw["frames"], kw["H"], kw["W"], kw["chunk"], kw["overlap"])
        assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.RehyatError):                                       # out aliases q
        op.forward(*args, wl.T, wl.H, wl.W, wl.Tc, wl.To, out=d["q"])
    with pytest.raises(binding.RehyatError):                                       # misaligned pointer
        qq = torch.empty(d["q"].numel() + 1, device="cuda")[1:].view_as(d["q"])
        op.forward(qq, d["k"], d["v"], d["phi_q"], d["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To)
    # after all the refusals the context still works
    y = op.forward(*args, wl.T, wl.H, wl.W, wl.Tc, wl.To)
    assert op.status() == 0 and torch.isfinite(y).all()
    op.close()
    with pytest.raises(binding.RehyatError) as e:
        binding.Rehyat(n_heads=2, head_dim=64, dtype="fp32", impl="tensor")
    assert e.value.code == binding.ERR_UNSUPPORTED


@pytest.mark.parametrize("d", [128, 64])
def test_host_buffer_entry_point_matches_device_entry_point(d):
    from paper_2601_04342_b200 import binding
    wl = synth.Workload("host", 1, 2, d, 4, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 84)
    x = synth.make_inputs(wl, phi_scale=1.5)
    y_dev, _ = run_gpu(wl, x)
    op = binding.for_workload(wl)
    d = _to_dev(x)
    pinned = {n: x[n].pin_memory() for n in ("q", "k", "v")}
    out = torch.empty_like(x["q"]).pin_memory()
    op.forward_host(pinned["q"], pinned["k"], pinned["v"], out, d["phi_q"], d["phi_k"], wl.T, wl.H, wl.W, wl.Tc, wl.To)
    assert np.array_equal(out.double().numpy(), y_dev)
    op.close()


# ------------------------------------------------------------------ other feature maps (activations, degree, widths)
PHI_VARIANTS = [
    # id, P, act_hidden, act_out, phi_hidden, phi_dim, kernels of phi, state and read-out expected for bf16
    ("degree1_relu", 1, "relu", "relu", 0, 0, "tensor"),
    ("degree4_relu", 4, "relu", "relu", 0, 0, "tensor"),
    ("degree2_gelu_softplus", 2, "gelu", "softplus", 0, 0, "tensor"),
    ("degree2_identity_elu1", 2, "identity", "elu1", 0, 0, "tensor"),
    ("degree3_width192", 3, "relu", "relu", 128, 192, "tensor"),      # one half of H, one and a half of U; parts of 64
    ("degree2_narrow", 2, "relu", "softplus", 64, 96, "tensor"),      # parts of 48 features: they end inside a 32-column block
    ("degree3_relu_parts_of_32", 3, "relu", "relu", 192, 96, "tensor"),
    ("degree4_hidden96_width128", 4, "gelu", "relu", 96, 128, "tensor"),   # K extent of the second GEMM ends inside a 64-column block
    ("degree2_hidden256_width64", 2, "relu", "elu1", 0, 64, "tensor"),
    ("degree2_widths_not_multiples_of_32", 2, "relu", "relu", 72, 104, "simt"),
]


@pytest.mark.parametrize("variant", PHI_VARIANTS, ids=[v[0] for v in PHI_VARIANTS])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_other_feature_maps(variant, dtype):
    _, P, ah, ao, Dh, Dp, expect = variant
    wl = synth.Workload("phi", 1, 2, 128, 5, 10, 20, 2, 1, dtype, dtype == "bf16", P=P, seed=synth.BASE_SEED + 85,
                        phi_hidden=Dh, phi_dim=Dp)
    # softplus / elu1 outputs are O(1) per feature, so the linear branch dominates without scaling phi
    x = synth.make_inputs(wl, phi_scale=1.5 if ao == "relu" else 1.0, v_frame_offsets=True)
    f = synth.to_f64(x)
    ref = orc.hybrid_direct(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To, P=P,
                            act_hidden=ah, act_out=ao)
    y, used = run_gpu(wl, x, act_hidden=ah, act_out=ao)
    assert used == ("tensor" if dtype == "bf16" else "simt")
    assert run_gpu.phi_kernels == (expect if dtype == "bf16" else "simt")
    check(y, ref, dtype)


@pytest.mark.parametrize("variant", [v for v in PHI_VARIANTS if v[6] == "tensor"], ids=[v[0] for v in PHI_VARIANTS if v[6] == "tensor"])
def test_other_feature_maps_with_heads_of_64(variant):
    """The same maps on heads of 64 channels (bf16): half the K extent of the first GEMM, 64-column state and
    read-out accumulators.  Default widths are 2 d = 128 here."""
    _, P, ah, ao, Dh, Dp, _ = variant
    wl = synth.Workload("phi64", 1, 3, 64, 5, 10, 20, 2, 1, "bf16", True, P=P, seed=synth.BASE_SEED + 87,
                        phi_hidden=Dh, phi_dim=Dp)
    x = synth.make_inputs(wl, phi_scale=1.5 if ao == "relu" else 1.0, v_frame_offsets=True)
    f = synth.to_f64(x)
    ref = orc.hybrid_direct(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To, P=P,
                            act_hidden=ah, act_out=ao)
    y, used = run_gpu(wl, x, act_hidden=ah, act_out=ao)
    assert used == run_gpu.phi_kernels == "tensor"
    check(y, ref, "bf16")


@pytest.mark.parametrize("layers", [3, 4])
@pytest.mark.parametrize("dtype,d,Dh", [("bf16", 128, 0), ("fp32", 128, 0), ("bf16", 64, 0), ("bf16", 128, 160)],
                         ids=["bf16", "fp32", "bf16_d64", "bf16_hidden160"])
def test_deeper_feature_maps(layers, dtype, d, Dh):
    """phi with one or two further hidden layers (rehyat_config.phi_layers); bf16 runs them on the tensor cores,
    the hidden activations going from one buffer to the other."""
    wl = synth.Workload("deep", 1, 2, d, 5, 10, 20, 2, 1, dtype, dtype == "bf16", seed=synth.BASE_SEED + 89,
                        phi_layers=layers, phi_hidden=Dh)
    # every further layer of std-0.02 parameters shrinks the features: scaled so that about half of the normaliser is linear
    scale = {3: 2.0, 4: 2.5}[layers] * ({3: 1.25, 4: 1.5}[layers] if wl.D_h == 128 else 1.0)
    x = synth.make_inputs(wl, phi_scale=scale, v_frame_offsets=True)
    assert x["phi_q"]["Wmid"].shape == (2, layers - 2, wl.D_h, wl.D_h)
    f = synth.to_f64(x)
    ref, frac = orc.hybrid_direct(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To,
                                  return_parts=True)
    assert 0.3 < frac[:, :, 2 * wl.HW * wl.Tc:].mean() < 0.9   # neither branch drowns the other
    two = {n: t for n, t in f["phi_q"].items() if n not in ("Wmid", "bmid")}
    assert np.abs(orc.hybrid_direct(f["q"], f["k"], f["v"], two, f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To) - ref).max() > 1e-2
    y, used = run_gpu(wl, x)
    assert used == run_gpu.phi_kernels == ("tensor" if dtype == "bf16" else "simt")
    check(y, ref, dtype)


def test_tensor_window_with_simt_linear_branch_matches_the_all_tensor_path():
    wl = synth.Workload("tw", 1, 2, 128, 6, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 86)
    x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
    ref, _ = oracle_full(wl, x)
    y, used = run_gpu(wl, x, impl="tensor_window")
    assert used == "tensor"
    check(y, ref, "bf16")


@pytest.mark.parametrize("n_poly", [-1, 1, 2, 3])
def test_every_share_of_polynomial_exponentials(n_poly):
    """rehyat_config.exp_poly picks how many of every four pairs of exponentials run as a cubic on the FMA pipe
    (-1: none, 0 would be the library's own choice, which is 1)."""
    wl = synth.Workload("poly", 1, 2, 128, 6, 10, 20, 2, 1, "bf16", True, seed=synth.BASE_SEED + 87)
    for kw in (dict(phi_scale=1.5, v_frame_offsets=True), dict(q_scale=4.0, phi_scale=1.5)):
        x = synth.make_inputs(wl, **kw)
        ref, _ = oracle_full(wl, x)
        y, used = run_gpu(wl, x, exp_poly=n_poly)
        assert used == "tensor"
        check(y, ref, "bf16")


def test_window_items_of_one_tile_edge_shapes():
    """Shapes that matter to window_tc1, where the key tiles of one query tile alternate between the two TMEM
    slots and the epilogue merges the two partial softmax results (Eq. 5 with the window split in two): windows
    of one key tile (the second slot stays empty), of an odd and of an even number of tiles, both c modes."""
    for name, args in (("a", (1, 2, 128, 6, 10, 20, 2, 1)), ("b", (2, 3, 128, 5, 9, 13, 1, 0)), ("c", (1, 2, 128, 3, 5, 7, 3, 2))):
        wl = synth.Workload("tiles_" + name, *args, "bf16", True, seed=synth.BASE_SEED + 91)
        for c_mode in ("rowmax", "zero"):
            x = synth.make_inputs(wl, phi_scale=1.5, v_frame_offsets=True)
            ref, _ = oracle_full(wl, x, c_mode=c_mode)
            y, used = run_gpu(wl, x, c_mode=c_mode)
            assert used == "tensor"
            check(y, ref, "bf16")


# ------------------------------------------------------------------ seeded random geometries
def _random_case(seed):
    """A small random problem: geometry (chunk and overlap against the frame count, ragged tiles), head size, phi
    widths and degree, c mode, layout.  Widths are multiples of 32 so that bf16 runs every step on the tensor cores."""
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128]))
    T = int(rng.integers(2, 9))
    Tc = int(rng.integers(1, min(T, 4) + 1))
    To = int(rng.integers(0, 4))
    H, W = int(rng.integers(3, 13)), int(rng.integers(5, 21))
    P = int(rng.choice([1, 2, 3, 4]))
    Dp = int(rng.choice([w for w in (96, 128, 192, 256) if w % P == 0 and (w // P) % 8 == 0]))
    Dh = int(rng.choice([64, 96, 128, 192, 256]))
    layers = int(rng.choice([2, 2, 3, 4]))
    wl = synth.Workload(f"rand{seed}", int(rng.integers(1, 3)), int(rng.integers(1, 4)), d, T, H, W, Tc, To, "bf16", True,
                        P=P, seed=synth.BASE_SEED + 300 + seed, phi_hidden=Dh, phi_dim=Dp, phi_layers=layers)
    return wl, str(rng.choice(["rowmax", "zero"])), str(rng.choice(["bhnd", "bnhd"])), {2: 1.5, 3: 2.0, 4: 2.5}[layers]


@pytest.mark.parametrize("seed", range(16))
def test_random_geometries(seed):
    wl, c_mode, layout, scale = _random_case(seed)
    x = synth.make_inputs(wl, phi_scale=scale, v_frame_offsets=True)
    f = synth.to_f64(x)
    ref = orc.hybrid_direct(f["q"], f["k"], f["v"], f["phi_q"], f["phi_k"], wl.T, wl.HW, wl.Tc, wl.To, P=wl.P, c_mode=c_mode)
    y, used = run_gpu(wl, x, c_mode=c_mode, layout=layout)
    assert used == run_gpu.phi_kernels == "tensor", (wl, c_mode, layout)
    check(y, ref, "bf16")
