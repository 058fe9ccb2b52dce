"""world_size-2 gloo test of the N>1 path on the CPU: ranks take disjoint batch shards, need no
exchange to produce their outputs, and the reported time is the MAX over ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import synth_inputs as si
from paper_2410_18517_b200 import dist_util


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert dist_util.env_rank() == (rank, rank, world)
        w = si.Workload("mr", L=3, Hq=4, Hkv=2, D=16, B=5, context=20, dtype="f32", n_shared=1, map_seed=0, steps=1,
                        fixed_map=(0, 1, 0))
        lo, hi = si.shard_batch(w.B, world, rank)
        # every rank decodes only its own sequences; nothing is exchanged to compute them
        orc = oracle.Oracle(w.L, w.Hq, w.Hkv, w.D, hi - lo, w.share_map())
        outs = []
        for l in range(w.L):
            k, v = si.context_kv(w, l)
            orc.layer_forward(l, None, k[lo:hi].double().numpy(), v[lo:hi].double().numpy())
        for l in range(w.L):
            q, k, v = si.step_qkv(w, 0, l)
            outs.append(orc.layer_forward(l, q[lo:hi].double().numpy(), k[lo:hi].double().numpy(),
                                          v[lo:hi].double().numpy()))
        mine = torch.from_numpy(np.stack(outs))                       # [L][b_local][Hq][D]
        gathered = [None] * world
        dist.all_gather_object(gathered, (lo, hi, mine))
        t = dist_util.max_over_ranks(10.0 + rank)                     # slowest rank decides
        if rank == 0:
            ret["spans"] = [(a, b) for a, b, _ in gathered]
            ret["out"] = torch.cat([x for _, _, x in sorted(gathered, key=lambda g: g[0])], dim=1).numpy()
            ret["tmax"] = t
            ret["rate"] = dist_util.whole_job_rate(8, world, t)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_the_batch_without_exchange():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_worker, args=(world, port, ret), nprocs=world, join=True)
        spans, out, tmax, rate = ret["spans"], ret["out"], ret["tmax"], ret["rate"]
    assert sorted(spans) == [(0, 3), (3, 5)]
    assert tmax == 11.0 and rate == 8 * 2 / 11e-3
    # the unsharded oracle gives the same numbers: the shards were independent
    w = si.Workload("mr", L=3, Hq=4, Hkv=2, D=16, B=5, context=20, dtype="f32", n_shared=1, map_seed=0, steps=1,
                    fixed_map=(0, 1, 0))
    orc = oracle.Oracle(w.L, w.Hq, w.Hkv, w.D, w.B, w.share_map())
    for l in range(w.L):
        k, v = si.context_kv(w, l)
        orc.layer_forward(l, None, k.double().numpy(), v.double().numpy())
    ref = np.stack([orc.layer_forward(l, *[t.double().numpy() for t in si.step_qkv(w, 0, l)]) for l in range(w.L)])
    np.testing.assert_array_equal(out, ref)


def test_max_over_ranks_without_a_process_group_is_identity():
    assert dist_util.max_over_ranks(3.5) == 3.5
    assert dist_util.env_rank()[2] >= 1
