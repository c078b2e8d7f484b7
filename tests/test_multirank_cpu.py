"""The N > 1 path of the benchmark on CPU: two gloo ranks run the replica sharding and the
max / sum over ranks that bench.py uses (the data path itself has no collective)."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import synth
    spec = bench.rank_spec(synth.SPECS["cfg2_b16_u1k_8k_p16"], rank, world)
    lens = synth.make_lengths(spec)
    ms = 1.0 + rank                                   # rank 1 is the slow one
    mx = bench.over_ranks([ms, 10.0 - rank], "max", "cpu")
    sm = bench.over_ranks([float(lens.sum()), 1.0], "sum", "cpu")
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([spec.seed, lens.sum(), *mx, *sm], dtype=np.float64))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_reduce(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0 = np.load(tmp_path / "r0.npy")
    r1 = np.load(tmp_path / "r1.npy")
    assert r0[0] != r1[0] and r0[1] != r1[1]           # replicas draw different batches
    for r in (r0, r1):
        assert r[2] == 2.0 and r[3] == 10.0            # max over ranks (time of the slowest rank)
        assert r[4] == r0[1] + r1[1] and r[5] == 2.0   # units all ranks processed


def test_single_process_reductions_are_identity():
    sys.path.insert(0, ROOT)
    import bench
    import synth
    assert bench.over_ranks([3.0, 4.0], "max", "cpu") == [3.0, 4.0]
    spec = synth.SPECS["cfg3_b64_ctx16384_p64"]
    assert bench.rank_spec(spec, 0, 1) is spec
    assert bench.rank_spec(spec, 3, 8).seed == spec.seed + 300
