"""World-size-2 gloo test (CPU) of the multi-GPU plumbing: a batch cut into contiguous token ranges,
each rank gating its own range, gives after concatenation exactly the unsharded mask / ids / count;
head outputs of the shards equal the unsharded ones row for row (tokens are independent).
The per-rank compute here is the oracle (this is a CPU test of the host logic, not a parity test)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import synth
from paper_2512_08537_b200 import shard


def test_token_ranges_partition_any_n():
    for n in (0, 1, 7, 64, 1000, 4099):
        for world in (1, 2, 3, 8):
            ranges = [shard.token_range(n, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            for (a, b), (c, d) in zip(ranges, ranges[1:]):
                assert b == c and a <= b
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 1


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, n, tau, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = synth.workload("cfg1", n=n)
        lo, hi = shard.token_range(n, world, rank)
        feat = synth.features(wl, lo, hi - lo)
        _, mask, idx, count = oracle.gate(feat, tau)
        ids, counts = shard.gather_survivor_ids(torch.from_numpy(idx.astype(np.int32)), count, lo)
        w, t = synth.head_weights(wl), synth.t_sched(wl.K)
        out = oracle.head_sample(w, synth.cond(wl, lo, hi - lo), synth.noise(wl, lo, hi - lo), t, idx)
        slowest = shard.max_over_ranks(10.0 + rank)
        np.savez(os.path.join(out_dir, f"r{rank}.npz"), mask=mask, ids=ids.numpy(), counts=np.array(counts),
                 out=out, lo=lo, hi=hi, slowest=slowest)
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_result(tmp_path):
    n, world = 203, 2
    wl = synth.workload("cfg1", n=n)
    feat = synth.features(wl)
    H = oracle.entropy(feat)
    tau = float(np.median(H))
    _, mask_ref, idx_ref, count_ref = oracle.gate(feat, tau)
    out_ref = oracle.head_sample(synth.head_weights(wl), synth.cond(wl), synth.noise(wl), synth.t_sched(wl.K), idx_ref)
    mp.spawn(_worker, args=(world, _free_port(), n, tau, str(tmp_path)), nprocs=world, join=True)
    parts = [np.load(tmp_path / f"r{r}.npz") for r in range(world)]
    assert np.array_equal(np.concatenate([p["mask"] for p in parts]), mask_ref)
    for p in parts:                                  # every rank sees the same global list
        assert np.array_equal(p["ids"], idx_ref.astype(np.int64))
        assert int(p["counts"].sum()) == count_ref
        assert float(p["slowest"]) == 11.0
    assert np.array_equal(np.concatenate([p["out"] for p in parts]), out_ref)
