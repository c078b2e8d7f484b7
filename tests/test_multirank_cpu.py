"""The N > 1 path of the benchmark on CPU: bench.py's own launcher starts two gloo ranks, which take
their shares through bench.rank_workload and reduce through bench.over_ranks (the data path itself has
no collective; with no GPU here each rank's share is computed by the CPU oracle)."""
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
WORKER = os.path.join(ROOT, "tests", "bench_rank_worker.py")
sys.path.insert(0, ROOT)


def _load(tmp_path, world):
    return [np.load(tmp_path / f"rank{r}.npz") for r in range(world)]


def test_kv_head_shards_of_two_ranks_put_together_equal_the_unsharded_oracle(tmp_path):
    import bench
    import oracle
    import synth
    world = 2
    rc = bench.spawn_ranks(WORKER, ["--gpus", str(world), "--shard", "kv-heads", "--out", str(tmp_path)], world,
                           timeout_s=300)
    assert rc == 0
    r = _load(tmp_path, world)
    full = synth.make_workload(synth.tiny_spec("ranks", (300, 1, 0, 64, 777, 1300), 16, 9100), "cpu")
    ref_out, ref_lse = oracle.decode_attn(full.q, full.k_pages, full.v_pages, full.block_table, full.seq_lens,
                                          full.scale)
    assert [int(x["hkv"]) for x in r] == [4, 4] and [int(x["hq"]) for x in r] == [32, 32]
    # query heads 0..31 belong to rank 0 (KV heads 0..3), 32..63 to rank 1: side by side they are the
    # whole result, bit for bit (a head's result depends on nothing outside its own KV head)
    assert np.array_equal(np.concatenate([x["out"] for x in r], axis=1), ref_out, equal_nan=True)
    assert np.array_equal(np.concatenate([x["lse"] for x in r], axis=1), ref_lse)
    for x in r:
        assert x["max_ms"] == 2.0 and int(x["world"]) == 2              # time of the slowest rank
        assert x["sum_bytes"] == float(r[0]["bytes"]) + float(r[1]["bytes"])
    # K and V bytes are split, tables and lengths are read by both
    assert r[0]["sum_bytes"] > full.algorithmic_bytes() - 1 and r[0]["sum_bytes"] < full.algorithmic_bytes() + 4096


def test_context_shards_of_two_ranks_gathered_and_merged_equal_the_unsharded_oracle(tmp_path):
    import bench
    import oracle
    import synth
    world = 2
    rc = bench.spawn_ranks(WORKER, ["--gpus", str(world), "--shard", "context", "--out", str(tmp_path)], world,
                           timeout_s=300)
    assert rc == 0
    r = _load(tmp_path, world)
    full = synth.make_workload(synth.tiny_spec("ranks", (300, 1, 0, 64, 777, 1300), 16, 9100), "cpu")
    ref_out, ref_lse = oracle.decode_attn(full.q, full.k_pages, full.v_pages, full.block_table, full.seq_lens,
                                          full.scale)
    for x in r:                                   # every rank ends up with the whole result
        assert int(x["hq"]) == 64 and int(x["hkv"]) == 8
        assert np.allclose(x["out"], ref_out, rtol=0, atol=1e-12, equal_nan=True)
        assert np.array_equal(np.isneginf(x["lse"]), np.isneginf(ref_lse))
        fin = np.isfinite(ref_lse)
        assert np.allclose(x["lse"][fin], ref_lse[fin], rtol=0, atol=1e-12)
    # the ranks' token ranges are disjoint and together the whole cache
    assert r[0]["sum_tokens"] == float(300 + 1 + 64 + 777 + 1300)


def test_context_shards_partition_every_sequence():
    import synth
    full = synth.make_workload(synth.tiny_spec("ctxp", (300, 1, 0, 64, 777, 1300, 16, 17), 16, 9101), "cpu")
    for world in (1, 2, 3, 8):
        shards = [synth.shard_context(full, r, world) for r in range(world)]
        assert sum(int(s.lens_host.sum()) for s in shards) == int(full.lens_host.sum())
        for b in range(full.spec.batch):
            pages = []
            for s in shards:
                n = -(-int(s.lens_host[b]) // 16)
                pages += s.table_host[b, :n].tolist()
            assert pages == full.table_host[b, :-(-int(full.lens_host[b]) // 16)].tolist()
            # only a sequence's last non-empty shard may end inside a page
            ragged = [int(s.lens_host[b]) % 16 != 0 for s in shards if s.lens_host[b] > 0]
            assert not any(ragged[:-1])


def test_replica_ranks_draw_their_own_batches(tmp_path):
    import bench
    world = 2
    rc = bench.spawn_ranks(WORKER, ["--gpus", str(world), "--shard", "replicas", "--out", str(tmp_path)], world,
                           timeout_s=300)
    assert rc == 0
    r = _load(tmp_path, world)
    assert int(r[0]["seed"]) != int(r[1]["seed"]) and int(r[0]["hkv"]) == 8
    assert not np.array_equal(r[0]["out"], r[1]["out"], equal_nan=True)
    assert r[0]["sum_tokens"] == r[1]["sum_tokens"] == 2 * (300 + 1 + 64 + 777 + 1300)


def test_a_failing_rank_fails_the_job(tmp_path):
    import bench
    rc = bench.spawn_ranks(WORKER, ["--gpus", "2", "--out", str(tmp_path), "--fail-rank", "1"], 2, timeout_s=300)
    assert rc != 0


def test_world_size_must_match_gpus(tmp_path):
    import bench
    # two ranks started, three asked for: every rank refuses
    rc = bench.spawn_ranks(WORKER, ["--gpus", "3", "--out", str(tmp_path)], 2, timeout_s=300)
    assert rc != 0
    assert not list(tmp_path.glob("rank*.npz"))


def test_bench_cli_launches_its_own_ranks_and_fails_without_gpus():
    import torch
    if torch.cuda.is_available() and torch.cuda.device_count() >= 2:
        return                                   # on a multi-GPU machine this would be a real run
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    pr = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1", "--warmup", "0",
                         "--workload", "cfg1_b1_ctx512_p16", "--no-cpu", "--no-e2e"],
                        env=env, capture_output=True, text=True, timeout=600)
    assert pr.returncode != 0                    # fewer GPUs than ranks: no result line, non-zero exit
    assert '"metric"' not in pr.stdout


def test_single_process_reductions_are_identity():
    import bench
    import synth
    assert bench.over_ranks([3.0, 4.0], "max", "cpu") == [3.0, 4.0]
    spec = synth.SPECS["cfg3_b64_ctx16384_p64"]
    assert bench.rank_spec(spec, 0, 1) is spec
    assert bench.rank_spec(spec, 3, 8).seed == spec.seed + 300
