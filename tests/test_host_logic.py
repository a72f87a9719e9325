"""Host-side geometry: chunk plan, FLOP model, head sharding."""
import pytest

from paper_2601_04342_b200 import geometry as geo
from paper_2601_04342_b200 import synth


def test_chunk_plan_config2():
    plan = geo.chunk_plan(21, 1560, 3, 1)
    assert len(plan) == 7
    assert (plan[0].lo, plan[0].hi) == (0, 4680)
    assert (plan[1].q0, plan[1].lo, plan[1].hi) == (4680, 3120, 9360)
    assert plan[-1].hi == 32760 and plan[-1].lo == 26520
    assert all(c.hi - c.lo == 6240 for c in plan[1:])


def test_chunk_plan_ragged_and_large_overlap():
    plan = geo.chunk_plan(41, 1560, 3, 1)
    assert len(plan) == 14 and plan[-1].q1 - plan[-1].q0 == 2 * 1560
    plan = geo.chunk_plan(5, 10, 1, 2)
    assert [c.lo for c in plan] == [0, 0, 0, 10, 20]
    plan = geo.chunk_plan(4, 10, 9, 0)
    assert len(plan) == 1 and (plan[0].lo, plan[0].hi) == (0, 40)
    with pytest.raises(ValueError):
        geo.chunk_plan(4, 10, 0, 0)


def test_flop_model_matches_closed_forms():
    f = geo.flop_model(1, 12, 128, 21, 1560, 3, 1, 256, 256)
    assert f["pairs"] == 12 * 81 * 1560 * 1560            # 81 frame pairs per head
    assert abs(f["total"] / 1e12 - 1.383) < 1e-3
    assert abs(f["full_softmax"] / 1e12 - 6.594) < 1e-3
    assert abs(geo.flop_model(2, 12, 128, 41, 1560, 3, 1, 256, 256)["total"] / 1e12 - 5.50) < 1e-2
    assert abs(geo.flop_model(1, 12, 128, 81, 1560, 3, 1, 256, 256)["total"] / 1e12 - 5.56) < 1e-2
    # one chunk covering everything: only the window term remains and equals full softmax
    f = geo.flop_model(1, 2, 64, 4, 64, 4, 0, 128, 128)
    assert f["total"] == f["window"] == f["full_softmax"]


def test_shard_heads_partitions_all_units():
    for B, nh, ws in [(1, 12, 8), (2, 12, 8), (1, 12, 5), (1, 2, 4), (1, 12, 1)]:
        got = [geo.shard_heads(B, nh, ws, r) for r in range(ws)]
        assert got[0][0] == 0 and got[-1][1] == B * nh
        assert all(a[1] == b[0] for a, b in zip(got, got[1:]))
        sizes = [b - a for a, b in got]
        assert max(sizes) - min(sizes) <= 1


def test_synth_is_seeded_and_shaped():
    wl = synth.CONFIGS["tiny_fp32"]
    a, b = synth.make_inputs(wl), synth.make_inputs(wl)
    assert a["q"].shape == (1, 2, 256, 64)
    assert all((a[n] == b[n]).all() for n in ("q", "k", "v"))
    assert (a["phi_q"]["W2"] == b["phi_q"]["W2"]).all() and not (a["phi_q"]["W1"] == a["phi_k"]["W1"]).all()
    assert abs(float(a["phi_q"]["W1"].std()) - 0.02) < 2e-3
    wl2 = synth.Workload("t", 1, 2, 128, 2, 4, 4, 1, 0, "bf16", True)
    x = synth.make_inputs(wl2)
    rms = x["q"].float().pow(2).mean(-1).sqrt()
    assert (rms - 1).abs().max() < 2e-2
    assert len(synth.sweep_configs()) == 18


def test_shard_rects_cover_every_unit_once_and_in_order():
    for B, nh, world in ((1, 12, 8), (2, 12, 8), (2, 12, 5), (3, 5, 4), (1, 3, 8), (4, 2, 3)):
        seen = []
        for r in range(world):
            u0, u1 = geo.shard_heads(B, nh, world, r)
            mine = []
            for (b0, nb, h0, n) in geo.shard_rects(B, nh, world, r):
                assert nb >= 1 and n >= 1 and h0 + n <= nh and b0 + nb <= B
                assert nb == 1 or (h0 == 0 and n == nh)            # several batch items only as whole items
                mine += [b * nh + h for b in range(b0, b0 + nb) for h in range(h0, h0 + n)]
            assert mine == list(range(u0, u1))
            seen += mine
        assert seen == list(range(B * nh))


def test_shard_efficiency():
    assert geo.shard_efficiency(1, 12, 8) == 0.75                  # 12 heads over 8 ranks: 2/1 imbalance
    assert geo.shard_efficiency(1, 12, 4) == 1.0
    assert geo.shard_efficiency(2, 12, 8) == 1.0
    assert geo.shard_efficiency(1, 12, 1) == 1.0
