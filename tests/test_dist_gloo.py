"""Multi-rank host logic on CPU (gloo, world size 2): the (batch, head) problems are split over
ranks with no exchange on the data path; timing is reduced with MAX over ranks."""
import os
import socket

import numpy as np
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


def test_head_sharding_over_two_ranks(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    err, tmax = np.load(tmp_path / "err.npy")
    bounds = np.load(tmp_path / "bounds.npy")
    assert err == 0.0
    assert tmax == 2.0
    assert bounds[0][0] == 0 and bounds[-1][1] == 3 and bounds[0][1] == bounds[1][0]
