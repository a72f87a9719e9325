"""Multi-rank host logic on CPU (gloo, world size 2): the (batch, head) problems are split over
ranks with no exchange on the data path; timing is reduced with MAX over ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2601_04342_b200 import geometry, synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import rehyat_oracle as orc
        wl = synth.Workload("dist", 1, 3, 8, 4, 2, 3, 1, 1, "fp32", seed=synth.BASE_SEED + 500)
        x = synth.to_f64(synth.make_inputs(wl, phi_scale=5.0))
        u0, u1 = geometry.shard_heads(wl.B, wl.n_heads, world, rank)
        # every rank evaluates only its own heads; nothing is exchanged until the results are gathered
        y = orc.hybrid_rnn(x["q"], x["k"], x["v"], x["phi_q"], x["phi_k"], wl.T, wl.HW, wl.Tc, wl.To,
                           heads=range(u0, u1))
        mine = torch.from_numpy(y)
        dist.all_reduce(mine, op=dist.ReduceOp.SUM)            # heads a rank does not own are zero
        bounds = [None] * world
        dist.all_gather_object(bounds, (u0, u1))
        t = torch.tensor([1.0 + rank], dtype=torch.float64)    # the slowest rank decides the time
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        if rank == 0:
            full = orc.hybrid_rnn(x["q"], x["k"], x["v"], x["phi_q"], x["phi_k"], wl.T, wl.HW, wl.Tc, wl.To)
            np.save(os.path.join(out_dir, "err.npy"), np.array([np.abs(mine.numpy() - full).max(), t.item()]))
            np.save(os.path.join(out_dir, "bounds.npy"), np.array(bounds))
    finally:
        dist.destroy_process_group()


def _call_worker(rank, world, port, out_dir):
    """Every rank builds the arguments of its own operator calls from the full tensors (the marshalling helper
    of the binding) and reports which (batch, head) blocks they address and where the pointers land."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2601_04342_b200 import binding
        wl = synth.Workload("calls", 2, 3, 64, 2, 2, 3, 1, 1, "bf16", seed=synth.BASE_SEED + 501)
        x = synth.make_inputs(wl)
        out = torch.zeros_like(x["q"])
        es = x["q"].element_size()
        covered = torch.zeros((wl.B, wl.n_heads), dtype=torch.int32)
        ok = True
        for rect in geometry.shard_rects(wl.B, wl.n_heads, world, rank):
            b0, nb, h0, nh = rect
            (vq, vk, vv, vo), pq, pk, lay = binding.shard_call_args(x["q"], x["k"], x["v"], out, x["phi_q"], x["phi_k"], rect)
            first = (b0 * wl.n_heads + h0) * wl.N * wl.head_dim * es
            ok &= all(v.data_ptr() - t.data_ptr() == first for v, t in ((vq, x["q"]), (vk, x["k"]), (vv, x["v"]), (vo, out)))
            ok &= (lay.stride_batch, lay.stride_head, lay.stride_token) == (wl.n_heads * wl.N * wl.head_dim, wl.N * wl.head_dim, wl.head_dim)
            ok &= pq["W1"].data_ptr() - x["phi_q"]["W1"].data_ptr() == h0 * wl.D_h * wl.head_dim * es
            ok &= pk["W2"].data_ptr() - x["phi_k"]["W2"].data_ptr() == h0 * wl.D_out * wl.D_h * es
            ok &= pk["b2"].data_ptr() - x["phi_k"]["b2"].data_ptr() == h0 * wl.D_out * es
            ok &= tuple(vq.shape) == (nb, nh, wl.N, wl.head_dim) and pq["b1"].shape[0] == nh
            vo.fill_(1.0)                                          # what the call of this rectangle would write
            covered[b0:b0 + nb, h0:h0 + nh] += 1
        written = (out.float().abs().amax(dim=(2, 3)) > 0).to(torch.int32)
        ok &= bool((written == covered).all())
        flag = torch.tensor([int(ok)], dtype=torch.int32)
        dist.all_reduce(flag, op=dist.ReduceOp.MIN)
        dist.all_reduce(covered, op=dist.ReduceOp.SUM)
        if rank == 0:
            np.save(os.path.join(out_dir, "covered.npy"), covered.numpy())
            np.save(os.path.join(out_dir, "ok.npy"), flag.numpy())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 4])
def test_sharded_call_arguments_cover_every_problem_once(tmp_path, world):
    mp.spawn(_call_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert np.load(tmp_path / "ok.npy")[0] == 1
    assert (np.load(tmp_path / "covered.npy") == 1).all()


def test_head_sharding_over_two_ranks(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    err, tmax = np.load(tmp_path / "err.npy")
    bounds = np.load(tmp_path / "bounds.npy")
    assert err == 0.0
    assert tmax == 2.0
    assert bounds[0][0] == 0 and bounds[-1][1] == 3 and bounds[0][1] == bounds[1][0]
