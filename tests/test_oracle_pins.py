"""Pins of the fp64 oracle against what the paper's equations and plain mathematics fix.

No value here comes from the CUDA path.  Each pin is chosen so that a plausible mistake in
the oracle (a dropped term, a wrong set bound, a transposed operand, a missing power) fails
at least one of them.
"""
import math

import numpy as np
import pytest
import torch

from oracle import rehyat_oracle as orc


def _rand_problem(seed, B, nh, d, T, HW, Dh=None, Do=None, std=0.3):
    rng = np.random.default_rng(seed)
    N = T * HW
    Dh = Dh or 2 * d
    Do = Do or 2 * d
    q = rng.standard_normal((B, nh, N, d))
    k = rng.standard_normal((B, nh, N, d))
    v = rng.standard_normal((B, nh, N, d))

    def params():
        return {"W1": rng.standard_normal((nh, Dh, d)) * std, "b1": rng.standard_normal((nh, Dh)) * std,
                "W2": rng.standard_normal((nh, Do, Dh)) * std, "b2": rng.standard_normal((nh, Do)) * std}
    return q, k, v, params(), params()


GEOMS = [  # (T, HW, Tc, To)
    (4, 4, 1, 1), (4, 3, 1, 0), (5, 3, 2, 1), (6, 2, 3, 1), (6, 2, 2, 0),
    (5, 3, 1, 2), (6, 2, 1, 3), (4, 3, 1, 2),      # overlap >= chunk
    (5, 2, 3, 1), (7, 2, 3, 2), (5, 2, 2, 2),      # T not divisible by Tc
    (3, 4, 3, 0), (3, 4, 5, 1),                    # one chunk covers everything
]


# ------------------------------------------------------------------ I1: brute force
@pytest.mark.parametrize("geom", GEOMS)
@pytest.mark.parametrize("c_mode", ["rowmax", "zero"])
def test_direct_and_rnn_equal_brute_force(geom, c_mode):
    T, HW, Tc, To = geom
    q, k, v, pq, pk = _rand_problem(11 + T * 7 + HW, 1, 2, 4, T, HW)
    yb = orc.hybrid_brute(q, k, v, pq, pk, T, HW, Tc, To, c_mode=c_mode)
    yd = orc.hybrid_direct(q, k, v, pq, pk, T, HW, Tc, To, c_mode=c_mode)
    yr = orc.hybrid_rnn(q, k, v, pq, pk, T, HW, Tc, To, c_mode=c_mode)
    assert np.max(np.abs(yd - yb)) < 1e-12
    assert np.max(np.abs(yr - yb)) < 1e-12


@pytest.mark.parametrize("geom", [(4, 3, 1, 1), (5, 2, 2, 1), (6, 2, 3, 0)])
def test_bidirectional_direct_equals_brute_force(geom):
    T, HW, Tc, To = geom
    q, k, v, pq, pk = _rand_problem(5, 1, 1, 4, T, HW)
    yb = orc.hybrid_brute(q, k, v, pq, pk, T, HW, Tc, To, causal=False)
    yd = orc.hybrid_direct(q, k, v, pq, pk, T, HW, Tc, To, causal=False)
    assert np.max(np.abs(yd - yb)) < 1e-12
    # the causal operator differs from it as soon as a later chunk exists
    yc = orc.hybrid_direct(q, k, v, pq, pk, T, HW, Tc, To, causal=True)
    assert np.max(np.abs(yc - yd)) > 1e-3


def test_sampled_rows_equal_full_evaluation():
    T, HW, Tc, To = 7, 5, 2, 1
    q, k, v, pq, pk = _rand_problem(3, 2, 2, 8, T, HW)
    full = orc.hybrid_direct(q, k, v, pq, pk, T, HW, Tc, To)
    rows = np.array([0, 3, 9, 10, 17, 29, 34])
    got, frac = orc.hybrid_rows(q, k, v, pq, pk, T, HW, Tc, To, 1, 0, rows)
    assert np.max(np.abs(got - full[1, 0, rows])) < 1e-12
    assert frac[0] == 0.0 and frac[-1] > 0.0


# ------------------------------------------------------------------ I2: full softmax limit
@pytest.mark.parametrize("c_mode", ["rowmax", "zero"])
def test_chunk_covering_everything_is_full_softmax(c_mode):
    T, HW = 4, 6
    q, k, v, pq, pk = _rand_problem(21, 2, 2, 8, T, HW)
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v)).numpy()
    for f in (orc.hybrid_direct, orc.hybrid_rnn):
        got = f(q, k, v, pq, pk, T, HW, T, 1, c_mode=c_mode)
        assert np.max(np.abs(got - want)) < 1e-12
    assert np.max(np.abs(orc.softmax_attention(q, k, v) - want)) < 1e-12


# ------------------------------------------------------------------ I3: rows sum to one
@pytest.mark.parametrize("c_mode", ["rowmax", "zero"])
def test_rows_sum_to_one_and_are_nonnegative(c_mode):
    T, HW, Tc, To = 5, 3, 2, 1
    N = T * HW
    q, k, v, pq, pk = _rand_problem(2, 1, 1, 4, T, HW)
    ones = np.ones_like(v)
    for f in (orc.hybrid_direct, orc.hybrid_rnn):
        assert np.max(np.abs(f(q, k, ones, pq, pk, T, HW, Tc, To, c_mode=c_mode) - 1.0)) < 1e-13
    # identity values recover the normalised weight matrix
    d = 4
    Wn = np.zeros((N, N))
    for c0 in range(0, N, d):
        w = min(d, N - c0)
        vv = np.zeros((1, 1, N, d))
        for a in range(w):
            vv[0, 0, c0 + a, a] = 1.0
        y = orc.hybrid_direct(q, k, vv, pq, pk, T, HW, Tc, To, c_mode=c_mode)
        Wn[:, c0:c0 + w] = y[0, 0][:, :w]
    assert np.all(Wn >= 0.0)
    assert np.max(np.abs(Wn.sum(axis=1) - 1.0)) < 1e-13
    # causality of the linear branch and locality of the window: no weight on later chunks
    Np = Tc * HW
    for i in range(N):
        t = i // Np
        assert np.all(Wn[i, (t + 1) * Np:] == 0.0)
    # and the brute-force matrix, normalised, is the same matrix
    Wb = orc.hybrid_weights_brute(q[0, 0], k[0, 0], {n: pq[n][0] for n in pq}, {n: pk[n][0] for n in pk},
                                  T, HW, Tc, To, c_mode=c_mode)
    assert np.max(np.abs(Wb / Wb.sum(axis=1, keepdims=True) - Wn)) < 1e-13


# ------------------------------------------------------------------ I4: pure linear limit
def test_empty_softmax_set_is_textbook_linear_attention():
    T, HW = 3, 4
    N = T * HW
    d = 6
    rng = np.random.default_rng(8)
    q = rng.standard_normal((N, d)); k = rng.standard_normal((N, d)); v = rng.standard_normal((N, d))
    # phi(x) = 1 + elu(x) (Katharopoulos et al.) expressed through the MLP: identity weights
    eye = {"W1": np.eye(d), "b1": np.zeros(d), "W2": np.eye(d), "b2": np.zeros(d)}
    kw = dict(P=1, act_hidden="identity", act_out="elu1")
    W = orc.hybrid_weights_brute(q, k, eye, eye, T, HW, 1, 0,
                                 partition=lambda t: ([], list(range(N))), **kw)
    got = (W @ v) / W.sum(axis=1, keepdims=True)
    elu1 = lambda x: np.where(x > 0, x + 1.0, np.exp(x))
    want = orc.linear_attention(elu1(q), elu1(k), v)
    assert np.max(np.abs(got - want)) < 1e-12
    # Eq. 4 spelled out once more for one row, by hand
    i = 5
    num = sum((elu1(q[i]) @ elu1(k[j])) * v[j] for j in range(N))
    den = sum((elu1(q[i]) @ elu1(k[j])) for j in range(N))
    assert np.max(np.abs(got[i] - num / den)) < 1e-12


# ------------------------------------------------------------------ I5: chunk 0
def test_first_chunk_is_softmax_over_first_chunk():
    T, HW, Tc, To = 6, 3, 2, 1
    q, k, v, pq, pk = _rand_problem(4, 1, 2, 8, T, HW)
    y = orc.hybrid_rnn(q, k, v, pq, pk, T, HW, Tc, To)
    n0 = Tc * HW
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q[:, :, :n0]), torch.from_numpy(k[:, :, :n0]), torch.from_numpy(v[:, :, :n0])).numpy()
    assert np.max(np.abs(y[:, :, :n0] - want)) < 1e-12


# ------------------------------------------------------------------ I6 / I7: masked SDPA
def _window_mask(T, HW, Tc, To):
    N = T * HW
    m = np.zeros((N, N), dtype=bool)
    for i in range(N):
        t = i // (Tc * HW)
        lo = max(t * Tc * HW - To * HW, 0)
        hi = min((t + 1) * Tc * HW, N)
        m[i, lo:hi] = True
    return m


@pytest.mark.parametrize("geom", [(6, 3, 2, 1), (5, 4, 1, 2), (7, 2, 3, 0)])
def test_zero_phi_is_sliding_window_softmax(geom):
    T, HW, Tc, To = geom
    q, k, v, pq, pk = _rand_problem(9, 1, 2, 8, T, HW)
    for p in (pq, pk):
        p["W2"] = np.zeros_like(p["W2"]); p["b2"] = np.zeros_like(p["b2"])
    mask = torch.from_numpy(_window_mask(T, HW, Tc, To))
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), attn_mask=mask).numpy()
    for f in (orc.hybrid_direct, orc.hybrid_rnn):
        assert np.max(np.abs(f(q, k, v, pq, pk, T, HW, Tc, To) - want)) < 1e-12


def test_huge_overlap_is_frame_block_causal_softmax():
    T, HW, Tc = 5, 3, 2
    q, k, v, pq, pk = _rand_problem(10, 1, 1, 8, T, HW)
    N = T * HW
    mask = np.zeros((N, N), dtype=bool)
    for i in range(N):
        mask[i, :min((i // (Tc * HW) + 1) * Tc * HW, N)] = True
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v),
        attn_mask=torch.from_numpy(mask)).numpy()
    got = orc.hybrid_rnn(q, k, v, pq, pk, T, HW, Tc, T + 3)
    assert np.max(np.abs(got - want)) < 1e-12


# ------------------------------------------------------------------ I8: structure
def test_linear_in_v_and_permutation_structure():
    T, HW, Tc, To = 6, 4, 2, 1
    q, k, v, pq, pk = _rand_problem(12, 1, 1, 8, T, HW)
    f = lambda q_, k_, v_: orc.hybrid_rnn(q_, k_, v_, pq, pk, T, HW, Tc, To)
    y = f(q, k, v)
    v2 = np.random.default_rng(0).standard_normal(v.shape)
    assert np.max(np.abs(f(q, k, 2.0 * v - 3.0 * v2) - (2.0 * y - 3.0 * f(q, k, v2)))) < 1e-12
    # permuting the tokens inside each frame permutes the output the same way
    rng = np.random.default_rng(1)
    perm = np.concatenate([fr * HW + rng.permutation(HW) for fr in range(T)])
    assert np.max(np.abs(f(q[:, :, perm], k[:, :, perm], v[:, :, perm]) - y[:, :, perm])) < 1e-12
    # permuting keys inside the linear prefix of the last chunk leaves that chunk unchanged
    lo, _ = orc.softmax_set(2, T, HW, Tc, To)
    pk_perm = np.arange(T * HW)
    pk_perm[:lo] = rng.permutation(lo)
    y2 = f(q, k[:, :, pk_perm], v[:, :, pk_perm])
    q0, q1 = orc.chunk_queries(2, T, HW, Tc)
    assert np.max(np.abs(y2[:, :, q0:q1] - y[:, :, q0:q1])) < 1e-12


def test_logit_bias_discriminates_the_two_stabiliser_readings():
    T, HW, Tc, To = 4, 3, 1, 0
    q, k, v, pq, pk = _rand_problem(13, 1, 1, 4, T, HW)
    N = T * HW
    h = lambda p: {n: p[n][0] for n in p}
    bias = np.linspace(-1.0, 2.0, N)

    def run(c_mode, b):
        W = orc.hybrid_weights_brute(q[0, 0], k[0, 0], h(pq), h(pk), T, HW, Tc, To,
                                     c_mode=c_mode, logit_bias=b)
        return (W @ v[0, 0]) / W.sum(axis=1, keepdims=True)
    # rowmax: c moves with the bias, nothing changes
    assert np.max(np.abs(run("rowmax", bias) - run("rowmax", None))) < 1e-12
    # zero: unchanged only where the linear set is empty (chunk 0)
    dz = np.abs(run("zero", bias) - run("zero", None)).max(axis=1)
    assert np.all(dz[:Tc * HW] < 1e-12) and np.all(dz[Tc * HW:] > 1e-6)


# ------------------------------------------------------------------ I9: two-token hand formula
def test_two_token_closed_form():
    # T=2, HW=1, Tc=1, To=0: y_0 = v_0;  rowmax: y_1 = (v_1 + w v_0)/(1 + w);
    # zero: y_1 = (e^{s11} v_1 + w v_0)/(e^{s11} + w), w = phi_q(q_1).phi_k(k_0), s11 = q_1.k_1/sqrt(d)
    d = 2
    q = np.array([[[[0.3, -0.2], [1.0, 2.0]]]])
    k = np.array([[[[0.5, 0.1], [0.5, -1.0]]]])
    v = np.array([[[[1.0, 2.0], [-3.0, 0.5]]]])
    # phi = [relu(x)_0, relu(x)_1^2] through identity weights (D_h = D' = 2, P = 2)
    eye = {"W1": np.eye(2)[None], "b1": np.zeros((1, 2)), "W2": np.eye(2)[None], "b2": np.zeros((1, 2))}
    fq1 = np.array([1.0, 2.0 ** 2])
    fk0 = np.array([0.5, 0.1 ** 2])
    w = float(fq1 @ fk0)                      # 0.5 + 0.04
    assert abs(w - 0.54) < 1e-15
    s11 = (1.0 * 0.5 + 2.0 * -1.0) / math.sqrt(2.0)
    for f in (orc.hybrid_brute, orc.hybrid_direct, orc.hybrid_rnn):
        y = f(q, k, v, eye, eye, 2, 1, 1, 0, c_mode="rowmax")
        assert np.max(np.abs(y[0, 0, 0] - v[0, 0, 0])) < 1e-15
        assert np.max(np.abs(y[0, 0, 1] - (v[0, 0, 1] + w * v[0, 0, 0]) / (1.0 + w))) < 1e-15
        y = f(q, k, v, eye, eye, 2, 1, 1, 0, c_mode="zero")
        e = math.exp(s11)
        assert np.max(np.abs(y[0, 0, 1] - (e * v[0, 0, 1] + w * v[0, 0, 0]) / (e + w))) < 1e-15


# ------------------------------------------------------------------ phi
def test_phi_by_hand_and_polynomial_order():
    W1 = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])          # D_h = 3
    b1 = np.array([0.0, -1.0, 0.5])
    W2 = np.array([[1.0, 0.0, 0.0], [0.0, 2.0, 0.0], [0.0, 0.0, 1.0], [1.0, 1.0, 1.0],
                   [0.5, 0.0, 0.0], [-1.0, 0.0, 0.0]])            # D' = 6
    b2 = np.array([0.0, 0.0, 0.0, 0.0, 1.0, 0.0])
    x = np.array([[2.0, 3.0]])
    h = np.array([2.0, 2.0, 5.5])
    u = np.array([2.0, 4.0, 5.5, 9.5, 2.0, 0.0])
    got = orc.phi_map(x, W1, b1, W2, b2, P=2)
    assert np.allclose(got, [[u[0], u[1], u[2], u[3] ** 2, u[4] ** 2, u[5] ** 2]], atol=1e-15)
    got = orc.phi_map(x, W1, b1, W2, b2, P=3)
    assert np.allclose(got, [[u[0], u[1], u[2] ** 2, u[3] ** 2, u[4] ** 3, u[5] ** 3]], atol=1e-15)
    got = orc.phi_map(x, W1, b1, W2, b2, P=1)
    assert np.allclose(got, [u], atol=1e-15)
    # relu on the hidden layer matters: a negative pre-activation is cut
    got = orc.phi_map(np.array([[2.0, 0.0]]), W1, b1, W2, b2, P=1)
    assert np.allclose(got, [[2.0, 0.0, 2.5, 4.5, 2.0, 0.0]], atol=1e-15)
    with pytest.raises(ValueError):
        orc.phi_map(x, W1, b1, W2, b2, P=4)


def test_deeper_phi_by_hand():
    """Three and four layers, every value worked out by hand: x = (1, -2);
    layer 1: (1, -1, 1) -> relu (1, 0, 1); hidden layer A: (1, 1.5, 0); hidden layer B after A: (1.5 - 1, 1, 2.5);
    last layer after A: (1, 1.5, 0.5, -1) -> relu, degree 2: (1, 1.5, 0.25, 0);
    last layer after A, B: (0.5, 3.5, 0.5, 4) -> degree 2: (0.5, 3.5, 0.25, 16).  The order of A and B matters."""
    x = np.array([[1.0, -2.0]])
    W1 = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]]); b1 = np.array([0.0, 1.0, 2.0])
    A = np.array([[1.0, 1.0, 0.0], [0.0, -1.0, 1.0], [2.0, 0.0, -1.0]]); a = np.array([0.0, 0.5, -1.0])
    B = np.array([[0.0, 1.0, 0.0], [1.0, 0.0, 0.0], [1.0, 1.0, 1.0]]); b = np.array([-1.0, 0.0, 0.0])
    W2 = np.array([[1.0, 0.0, 0.0], [0.0, 1.0, 1.0], [1.0, -1.0, 0.0], [0.0, 0.0, 2.0]]); b2 = np.array([0.0, 0.0, 1.0, -1.0])
    three = orc.phi_map(x, W1, b1, W2, b2, P=2, Wmid=A[None], bmid=a[None])
    assert np.allclose(three, [[1.0, 1.5, 0.25, 0.0]], atol=1e-15)
    four = orc.phi_map(x, W1, b1, W2, b2, P=2, Wmid=np.stack([A, B]), bmid=np.stack([a, b]))
    assert np.allclose(four, [[0.5, 3.5, 0.25, 16.0]], atol=1e-15)
    swapped = orc.phi_map(x, W1, b1, W2, b2, P=2, Wmid=np.stack([B, A]), bmid=np.stack([b, a]))
    assert np.allclose(swapped, [[1.0, 1.5, 0.25, 0.0]], atol=1e-15) and not np.allclose(swapped, four)
    # no hidden layers in between: the two-layer map
    assert np.allclose(orc.phi_map(x, W1, b1, W2, b2, P=2, Wmid=np.zeros((0, 3, 3)), bmid=np.zeros((0, 3))),
                       orc.phi_map(x, W1, b1, W2, b2, P=2))
    # an identity hidden layer changes nothing after a relu
    assert np.allclose(orc.phi_map(x, W1, b1, W2, b2, P=2, Wmid=np.eye(3)[None], bmid=np.zeros((1, 3))),
                       orc.phi_map(x, W1, b1, W2, b2, P=2))


def test_deeper_phi_through_the_operator():
    """The three evaluations of the operator agree with a three-layer phi as they do with two layers."""
    rng = np.random.default_rng(5)
    nh, d, Dh, Dp, T, HW = 2, 4, 6, 4, 4, 3
    mk = lambda: {"W1": rng.standard_normal((nh, Dh, d)), "b1": rng.standard_normal((nh, Dh)),
                  "W2": rng.standard_normal((nh, Dp, Dh)), "b2": rng.standard_normal((nh, Dp)),
                  "Wmid": rng.standard_normal((nh, 1, Dh, Dh)), "bmid": rng.standard_normal((nh, 1, Dh))}
    pq, pk = mk(), mk()
    q, k, v = (rng.standard_normal((1, nh, T * HW, d)) for _ in range(3))
    brute = orc.hybrid_brute(q, k, v, pq, pk, T, HW, 1, 1)
    assert np.abs(orc.hybrid_direct(q, k, v, pq, pk, T, HW, 1, 1) - brute).max() < 1e-12
    assert np.abs(orc.hybrid_rnn(q, k, v, pq, pk, T, HW, 1, 1) - brute).max() < 1e-12
    two = {n: t for n, t in pq.items() if n not in ("Wmid", "bmid")}
    assert np.abs(orc.hybrid_direct(q, k, v, two, pk, T, HW, 1, 1) - brute).max() > 1e-3   # the hidden layer is not ignored


def test_phi_is_nonnegative_with_relu_output():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((50, 8))
    f = orc.phi_map(x, rng.standard_normal((16, 8)), rng.standard_normal(16),
                    rng.standard_normal((16, 16)), rng.standard_normal(16), P=2)
    assert np.all(f >= 0.0)


def test_activation_values():
    x = np.array([-2.0, 0.0, 1.5])
    assert np.allclose(orc._act(x, "softplus"), np.log1p(np.exp(x)))
    assert np.allclose(orc._act(x, "elu1"), [math.exp(-2.0), 1.0, 2.5])
    assert np.allclose(orc._act(x, "gelu"), torch.nn.functional.gelu(torch.from_numpy(x)).numpy())


def test_phi_parameter_count_matches_the_paper():
    # Wan2.1-1.3B: 12 heads of 128; widths 2d give 2,359,296 weights: "about 2.4 M" per block
    n = orc.phi_param_count(12, 128, 256, 256)
    assert n == 2359296
    assert abs(n / 2.4e6 - 1.0) < 0.02
    assert orc.phi_param_count(12, 128, 256, 256, with_bias=True) == 2359296 + 12288


# ------------------------------------------------------------------ sets
def test_token_sets():
    # Eq. 13 with T=7 frames of 10 tokens, Tc=3, To=1
    assert orc.num_chunks(7, 3) == 3
    assert orc.softmax_set(0, 7, 10, 3, 1) == (0, 30)
    assert orc.softmax_set(1, 7, 10, 3, 1) == (20, 60)
    assert orc.softmax_set(2, 7, 10, 3, 1) == (50, 70)          # short last chunk
    assert orc.chunk_queries(2, 7, 10, 3) == (60, 70)
    assert list(orc.linear_set(1, 7, 10, 3, 1)) == list(range(20))
    assert list(orc.linear_set(1, 7, 10, 3, 1, causal=False)) == list(range(20)) + list(range(60, 70))
    # Eq. 10-11: no overlap, bidirectional
    assert orc.softmax_set(1, 6, 5, 2, 0) == (10, 20)
    assert len(orc.linear_set(1, 6, 5, 2, 0, causal=False)) == 20


def test_a_planted_mistake_would_be_caught():
    """The pins are sensitive: variants of the oracle with one deliberate mistake each
    (built here, on the CPU) disagree with the brute-force matrix."""
    T, HW, Tc, To = 5, 3, 2, 1
    q, k, v, pq, pk = _rand_problem(30, 1, 1, 4, T, HW)
    ref = orc.hybrid_brute(q, k, v, pq, pk, T, HW, Tc, To)
    # (a) state update that re-adds the cumulative set (Eq. 17-18 read literally)
    d = 4
    h = lambda p: {n: p[n][0] for n in p}
    y = np.zeros_like(v)
    s = np.zeros((8, d)); z = np.zeros((8, 1))
    for t in range(orc.num_chunks(T, Tc)):
        q0, q1 = orc.chunk_queries(t, T, HW, Tc)
        lo, hi = orc.softmax_set(t, T, HW, Tc, To)
        S = q[0, 0, q0:q1] @ k[0, 0, lo:hi].T / math.sqrt(d)
        E = np.exp(S - S.max(axis=1, keepdims=True))
        fq = orc.phi_map(q[0, 0, q0:q1], **h(pq))
        y[0, 0, q0:q1] = (E @ v[0, 0, lo:hi] + fq @ s) / (E.sum(1, keepdims=True) + fq @ z)
        fk = orc.phi_map(k[0, 0, :lo], **h(pk))                 # whole TL_t again: wrong
        s = s + fk.T @ v[0, 0, :lo]; z = z + fk.sum(0)[:, None]
    assert np.max(np.abs(y - ref)) > 1e-3
    # (b) overlap ignored
    assert np.max(np.abs(orc.hybrid_direct(q, k, v, pq, pk, T, HW, Tc, 0) - ref)) > 1e-3
    # (c) phi_q and phi_k swapped
    assert np.max(np.abs(orc.hybrid_direct(q, k, v, pk, pq, T, HW, Tc, To) - ref)) > 1e-3


# ------------------------------------------------------------------ stored rows
def test_stored_rows_are_reproduced_by_the_recurrent_form():
    """tests/golden/tiny_fp32_rows.txt was written by the direct form; the RNN form, a
    different evaluation order, must land on the same numbers."""
    import os
    from paper_2601_04342_b200 import synth
    wl = synth.CONFIGS["tiny_fp32"]
    x = synth.to_f64(synth.make_inputs(wl))
    y = orc.hybrid_rnn(x["q"], x["k"], x["v"], x["phi_q"], x["phi_k"], wl.T, wl.HW, wl.Tc, wl.To)
    path = os.path.join(os.path.dirname(__file__), "golden", "tiny_fp32_rows.txt")
    n = 0
    for line in open(path):
        if line.startswith("#"):
            continue
        tok = line.split()
        h, r = int(tok[0]), int(tok[1])
        want = np.array([float(t) for t in tok[2:]])
        assert np.max(np.abs(y[0, h, r] - want)) < 1e-13
        n += 1
    assert n == 22


# ------------------------------------------------------------------ q/k normalisation and rotation
def test_rms_norm_by_hand():
    y = orc.rms_norm(np.array([3.0, 4.0]), eps=0.0)
    assert np.allclose(y, np.array([3.0, 4.0]) / math.sqrt(12.5), atol=1e-15)          # mean square (9 + 16) / 2
    assert np.allclose(orc.rms_norm(np.array([3.0, 4.0]), weight=np.array([2.0, -1.0]), eps=0.0),
                       [6.0 / math.sqrt(12.5), -4.0 / math.sqrt(12.5)], atol=1e-15)
    assert np.allclose(orc.rms_norm(np.array([1.0, 1.0, 1.0, 1.0]), eps=3.0), 0.5)     # 1 / sqrt(1 + 3)
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 7, 16))
    y = orc.rms_norm(x, eps=0.0)
    assert np.allclose(np.sqrt((y * y).mean(-1)), 1.0)                                 # unit RMS, any scale of the input
    assert np.allclose(orc.rms_norm(10.0 * x, eps=0.0), y)
    assert np.allclose(orc.rms_norm(x, eps=0.0), torch.nn.functional.rms_norm(torch.from_numpy(x), (16,), eps=0.0).numpy())


def test_rope_by_hand_and_its_invariants():
    # a quarter turn maps (1, 0) to (0, 1) and (0, 1) to (-1, 0); angle 0 is the identity
    x = np.array([[1.0, 0.0, 0.0, 1.0]])
    cos = np.array([[0.0, 0.0]]); sin = np.array([[1.0, 1.0]])
    assert np.allclose(orc.rope_rotate(x, cos, sin), [[0.0, 1.0, -1.0, 0.0]], atol=1e-15)
    assert np.allclose(orc.rope_rotate(x, np.ones((1, 2)), np.zeros((1, 2))), x)
    # 30 degrees on (2, 0): (sqrt 3, 1)
    assert np.allclose(orc.rope_rotate(np.array([[2.0, 0.0]]), [[math.sqrt(3) / 2]], [[0.5]]), [[math.sqrt(3.0), 1.0]], atol=1e-15)
    rng = np.random.default_rng(4)
    N, d = 9, 8
    theta = 1.0 / 100.0 ** (np.arange(d // 2) / (d // 2))
    ang = np.arange(N)[:, None] * theta[None, :]
    q, k = rng.standard_normal((N, d)), rng.standard_normal((N, d))
    rq, rk = orc.rope_rotate(q, np.cos(ang), np.sin(ang)), orc.rope_rotate(k, np.cos(ang), np.sin(ang))
    # the same thing as a complex multiplication of the pairs
    zq = (q[:, 0::2] + 1j * q[:, 1::2]) * np.exp(1j * ang)
    assert np.allclose(rq[:, 0::2], zq.real) and np.allclose(rq[:, 1::2], zq.imag)
    # a rotation: pair norms are kept
    assert np.allclose(rq[:, 0::2] ** 2 + rq[:, 1::2] ** 2, q[:, 0::2] ** 2 + q[:, 1::2] ** 2)
    # relative positions: <R_m q, R_n k> depends on n - m only
    q0, k0 = q[0], k[0]
    dots = np.array([[orc.rope_rotate(q0[None], np.cos(ang[m:m + 1]), np.sin(ang[m:m + 1]))[0] @
                      orc.rope_rotate(k0[None], np.cos(ang[n:n + 1]), np.sin(ang[n:n + 1]))[0] for n in range(N)] for m in range(N)])
    for s_ in range(1, N - 1):
        assert np.allclose(np.diag(dots, s_), np.diag(dots, s_)[0])
    assert not np.allclose(np.diag(dots, 1), np.diag(dots, 2)[:1])


def test_qk_transform_composes_norm_then_rotation():
    rng = np.random.default_rng(6)
    B, nh, N, d = 2, 3, 5, 4
    q, k = rng.standard_normal((B, nh, N, d)), rng.standard_normal((B, nh, N, d))
    wq, wk = rng.standard_normal((nh, d)), rng.standard_normal((nh, d))
    ang = rng.standard_normal((N, d // 2))
    tq, tk = orc.qk_transform(q, k, wq, wk, 1e-6, np.cos(ang), np.sin(ang))
    for b in range(B):
        for h in range(nh):
            assert np.allclose(tq[b, h], orc.rope_rotate(orc.rms_norm(q[b, h], wq[h], 1e-6), np.cos(ang), np.sin(ang)))
            assert np.allclose(tk[b, h], orc.rope_rotate(orc.rms_norm(k[b, h], wk[h], 1e-6), np.cos(ang), np.sin(ang)))
    # the order matters when the weight is not constant inside a pair (norm first, as the block does)
    other = orc.rms_norm(orc.rope_rotate(q[0, 0], np.cos(ang), np.sin(ang)), wq[0], 1e-6)
    assert not np.allclose(tq[0, 0], other)
    nq, _ = orc.qk_transform(q, k, None, None, 0.0, None, None)
    assert np.allclose(np.sqrt((nq * nq).mean(-1)), 1.0)
    rq, _ = orc.qk_transform(q, k, cos=np.cos(ang), sin=np.sin(ang), norm=False)
    assert np.allclose(rq, orc.rope_rotate(q, np.cos(ang), np.sin(ang)))
