"""One rank of a CPU stand-in for `bench.py --gpus N`, started by bench.spawn_ranks from the
multi-rank test: it joins the job through bench.init_ranks (gloo), takes its share of a small
workload through bench.rank_workload, computes that share's result with the CPU oracle (there is no
GPU here), reduces a made-up timing with bench.over_ranks and leaves everything in a file."""
import argparse
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, required=True)
    ap.add_argument("--shard", default="replicas")
    ap.add_argument("--out", required=True)
    ap.add_argument("--fail-rank", type=int, default=-1)
    a = ap.parse_args()
    import bench
    import oracle
    import synth
    import torch.distributed as dist

    rank, local, world, dev = bench.init_ranks(a.gpus, backend="gloo")
    if rank == a.fail_rank:
        raise SystemExit(3)                      # a rank that dies before doing any work
    spec = synth.tiny_spec("ranks", (300, 1, 0, 64, 777, 1300), 16, 9100)
    w = bench.rank_workload(spec, rank, world, a.shard, "cpu")
    out, lse = oracle.decode_attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    if a.shard == "context":
        # the path's one exchange step: every rank's (out, lse) over its token range is gathered on all ranks
        # and merged by log-sum-exp (here by the oracle's merge; on a GPU by concur_lse_merge)
        import torch
        parts_o = [torch.empty(out.shape, dtype=torch.float64) for _ in range(world)]
        parts_l = [torch.empty(lse.shape, dtype=torch.float64) for _ in range(world)]
        if world > 1:
            dist.all_gather(parts_o, torch.from_numpy(out))
            dist.all_gather(parts_l, torch.from_numpy(lse))
        else:
            parts_o, parts_l = [torch.from_numpy(out)], [torch.from_numpy(lse)]
        po = np.stack([t.numpy() for t in parts_o]); pl = np.stack([t.numpy() for t in parts_l])
        out = np.empty_like(out); lse = np.empty_like(lse)
        for b in range(out.shape[0]):
            for h in range(out.shape[1]):
                out[b, h], lse[b, h] = oracle.lse_merge(po[:, b, h], pl[:, b, h])
    ms = 1.0 + rank                              # the last rank is the slow one
    mx = bench.over_ranks([ms], "max", dev)
    sm = bench.over_ranks([float(w.algorithmic_bytes()), float(w.kv_tokens)], "sum", dev)
    np.savez(os.path.join(a.out, f"rank{rank}.npz"), out=out, lse=lse, seed=w.spec.seed, hq=w.spec.num_q_heads,
             hkv=w.spec.num_kv_heads, max_ms=mx[0], sum_bytes=sm[0], sum_tokens=sm[1], bytes=w.algorithmic_bytes(),
             world=world)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
