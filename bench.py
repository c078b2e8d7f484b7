"""Benchmark of one decode-attention step (plan + split-KV partial + LSE combine) through the
C ABI on seeded synthetic long-trace workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
                    [--shard replicas|kv-heads]

With --gpus N > 1 and no WORLD_SIZE in the environment the script starts its N ranks itself (one
process per GPU, rendezvous on 127.0.0.1); under an outside launcher that sets RANK / LOCAL_RANK /
WORLD_SIZE it is one of the ranks.  Either way the world size must equal N or the run fails.
--shard replicas (default): every rank decodes its own batch of the workload's shape (weak scaling);
--shard kv-heads: the ranks split ONE batch the way tensor parallelism does, each holding Hkv / N KV
heads of every page and the query heads that attend to them (strong scaling, no collective inside
attention); --shard context: every sequence's tokens are split by range, each rank attends to its range
and the ranks' (out, lse) pairs are all-gathered (NCCL, 260 bytes per query row and rank) and merged by
concur_lse_merge inside the timed step (strong scaling; the one exchange step this path can have).
Otherwise NCCL carries only the barrier and the max / sum of the timings.

NAME is one of synth.SPECS (plain decode step; the default is the 64 x 16,384 configuration) or of
synth.CASCADE_SPECS (shared-prefix step: `value` counts the shared pages once, `logical_gbs` as if
every sequence had read its whole context, `roofline` is the prefix-pass kernel) or of
synth.PREFILL_SPECS (causal prefill: `value` is useful TFLOP/s against the measured bf16 tensor peak).

One JSON line on stdout (rank 0).  `value` is the algorithmic bytes of the step (K and V of
every cached token, q/out/lse, used table entries) divided by the device time of the whole
step with all inputs resident in HBM; `e2e` is the same through the host-buffer entry point
with every host<->device copy inside the timed region; `roofline` times the partial kernel
alone with events the library records around it; `cpu_baseline` is the fp64 CPU oracle on a
bounded sample of the same workload, and `parity` compares the library's rows of those sampled
sequences with the oracle's (one-GPU runs only); `sustained` repeats the step (and the read-only
stream yardstick) back to back for two seconds with the clocks sampled, because a burst of 30 steps and
a long run can differ under the power cap.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attention_kv_bandwidth"
UNIT = "GB/s"
DEFAULT_WORKLOAD = "cfg3_b64_ctx16384_p64"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one partial_mma_kernel launch divided by its KV tokens, from
# an ncu capture of a quarter of the 64 x 16,384 configuration (page size 64, fused combine, one range per
# CTA).  Set to None whenever that kernel changes until the counters are taken again.
MMA_P64_TRAFFIC_BYTES_PER_KV_TOKEN = (1.074894e9 + 5.013248e6) / 262144
# The same two counters of one attn_tc_kernel / prefill_pair_kernel launch on exactly these workloads; None for any other
# workload, and to be removed whenever that kernel changes until the counters are taken again.
ATTN_TC_TRAFFIC_BYTES = {
    ("casc_16x10_pre16384_p64", "tcgen05"): 1.078966e9 + 10.120704e6,
    ("prefill_16x2048_p64", "single"): 671.184640e6 + 506.286592e6,
    ("prefill_16x2048_p64", "pair"): 671.258368e6 + 501.190400e6,
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--shard", default="replicas", choices=["replicas", "kv-heads", "context"],
                    help="N > 1: independent batches per rank, one batch split over the KV heads, or one batch "
                         "split over every sequence's token range (partials gathered and merged)")
    ap.add_argument("--kernel", type=int, default=0, help="0 tensor-core partial kernel, 1 scalar-FMA")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU time of the oracle sample")
    ap.add_argument("--no-cpu", action="store_true", help="skip the cpu_baseline leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--ranges-per-cta", type=int, default=0)
    ap.add_argument("--min-range-tiles", type=int, default=0)
    ap.add_argument("--num-ranges", type=int, default=0)
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="large workloads: also run the step back to back for this long (0 = skip)")
    ap.add_argument("--loop-steps", type=int, default=16, help="append+attention steps replayed from a CUDA graph")
    ap.add_argument("--fuse-combine", type=int, default=-1)
    ap.add_argument("--claim-ahead", type=int, default=-1)
    ap.add_argument("--small-page-copy", type=int, default=-1,
                    help="16/32-token pages: 1 per-lane copies (library default), 0 TMA boxes")
    ap.add_argument("--kv-layout", type=int, default=0, help="decode workloads: 0 head-major pools, 1 token-major")
    ap.add_argument("--prefix-kernel", type=int, default=0, help="cascade workloads: 0 tcgen05 prefix pass, 1 mma.sync")
    ap.add_argument("--prefill-kernel", type=int, default=0,
                    help="prefill workloads: 0 two query tiles per CTA over 128-token steps, 1 one tile over 64-token tiles")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap,power.draw")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50", "-i", str(self.index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def mark(self):
        return time.time()

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if (t0 is None or t >= t0 - 0.05) and (t1 is None or t <= t1 + 0.1)]
        if not rows:
            rows = [l for _, l in self.lines]
        sm, mx, reasons, watts = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            parts = [x.strip() for x in r.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
            try:
                watts.append(float(parts[6]))
            except (IndexError, ValueError):
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons), "samples": len(sm),
                "power_w": statistics.median(watts) if watts else None}


class L2Flush:
    """Takes a step's inputs out of the 126 MB L2 between timed steps: a 256 MB buffer is written, then
    another 256 MB buffer is read.  The read pushes the first buffer's dirty lines out to DRAM here, so
    that their write-back does not compete with the timed step's reads (on a 300 MB step that write-back
    is 40 % extra DRAM traffic and says nothing about the kernel)."""

    def __init__(self, dev):
        import torch
        self.written = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
        self.read = torch.zeros(32 * 1024 * 1024, dtype=torch.int64, device=dev)
        self.sink = None

    def __call__(self):
        self.written.zero_()
        self.sink = self.read.sum()


def oracle_sample_throughput(w_host, seqs, threads, keep=None):
    """Times the CPU oracle (as it stands) on whole sequences handed to a thread pool.  `keep`, a dict,
    receives the oracle's rows: keep[(b, h0)] = (out [8][D], lse [8]) in fp64."""
    from concurrent.futures import ThreadPoolExecutor
    import oracle
    qb = oracle._u16(w_host.q); kb = oracle._u16(w_host.k_pages); vb = oracle._u16(w_host.v_pages)
    tb = oracle._i32(w_host.block_table); lb = oracle._i32(w_host.seq_lens)
    Hq = w_host.spec.num_q_heads
    units = [(b, h0) for b in seqs for h0 in range(0, Hq, 8)]      # one KV-head group per unit

    def one(u):
        b, h0 = u
        o, l = oracle.decode_attn(qb, kb, vb, tb, lb, w_host.scale, seqs=(b, b + 1), heads=(h0, h0 + 8))
        if keep is not None:
            keep[(b, h0)] = (o[b, h0:h0 + 8].copy(), l[b, h0:h0 + 8].copy())

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(one, units))
    return time.perf_counter() - t0


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


OUT_ATOL, OUT_RTOL, LSE_ATOL = 4e-3, 1.6e-2, 1e-3        # the parity bar of the tests


def parity_of(rows, seqs, out, lse):
    """Compares the library's rows of the sampled sequences with the oracle's (the same figures the
    parity tests gate on; here they are reported, on the bench's own workload and launch shape)."""
    import numpy as np
    Hq = out.shape[1]
    ref_o = np.stack([np.concatenate([rows[(i, h0)][0] for h0 in range(0, Hq, 8)]) for i in range(len(seqs))])
    ref_l = np.stack([np.concatenate([rows[(i, h0)][1] for h0 in range(0, Hq, 8)]) for i in range(len(seqs))])
    got_o = out[seqs].float().cpu().numpy().astype(np.float64)
    got_l = lse[seqs].cpu().numpy().astype(np.float64)
    err = np.abs(got_o - ref_o)
    fin = np.isfinite(ref_l)
    den = float(np.sqrt(np.mean(ref_o ** 2)))
    return {"sequences": len(seqs), "elements": int(err.size),
            "max_abs_err": float(err.max()), "rel_rms_err": float(np.sqrt(np.mean(err ** 2)) / den) if den > 0 else 0.0,
            "worst_err_over_tolerance": float((err / (OUT_ATOL + OUT_RTOL * np.abs(ref_o))).max()),
            "lse_max_abs_err": float(np.abs(got_l - ref_l)[fin].max()) if fin.any() else 0.0,
            "within_tolerance": bool((err <= OUT_ATOL + OUT_RTOL * np.abs(ref_o)).all()
                                     and (np.abs(got_l - ref_l)[fin] <= LSE_ATOL).all()
                                     and np.array_equal(np.isneginf(got_l), np.isneginf(ref_l))),
            "tolerance": f"|out - ref| <= {OUT_ATOL} + {OUT_RTOL} |ref|, |lse - ref| <= {LSE_ATOL}"}


def cpu_baseline(w, target_seconds, results=None):
    """Oracle throughput on a bounded sample of the workload's sequences (all query heads each).  With
    `results` = (out, lse) of the library for the whole batch, also returns the parity figures of the
    sampled sequences: (baseline, parity)."""
    import numpy as np
    import synth
    cores = host_cores()
    order = np.random.default_rng(7).permutation(w.spec.batch).tolist()
    # calibrate on one KV-head group of the first sampled sequence
    first = synth.gather_sequences(w, order[:1])
    import oracle
    oracle.build()
    t0 = time.perf_counter()
    oracle.decode_attn(first.q, first.k_pages, first.v_pages, first.block_table, first.seq_lens,
                       first.scale, seqs=(0, 1), heads=(0, 8))
    cal = time.perf_counter() - t0
    per_token_core = cal * 8 / max(1, int(first.lens_host[0]))        # seconds per KV token on one core
    budget_tokens = target_seconds * cores / max(per_token_core, 1e-12)
    seqs, tok = [], 0
    for b in order:
        seqs.append(b)
        tok += int(w.lens_host[b])
        if tok >= budget_tokens:
            break
    sub = synth.gather_sequences(w, seqs)
    rows = {} if results is not None else None
    dt = oracle_sample_throughput(sub, list(range(len(seqs))), cores, rows)
    nbytes = sub.algorithmic_bytes()
    base = {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(seqs)} of {w.spec.batch} sequences ({tok} of {w.kv_tokens} KV tokens), all {w.spec.num_q_heads} query heads, "
                      f"{dt:.1f} s wall", "kv_tokens_per_s": tok / dt,
            "one_core_kv_tokens_per_s": 1.0 / max(per_token_core, 1e-12)}      # from the calibration call
    if results is None:
        return base
    return base, parity_of(rows, seqs, results[0], results[1])


def rank_spec(spec, rank: int, world: int):
    """Replicas: every rank decodes its own batch of the same shape, drawn from its own seed."""
    if world <= 1:
        return spec
    from dataclasses import replace
    return replace(spec, seed=spec.seed + 100 * rank)


def rank_workload(spec, rank: int, world: int, shard: str, device, **kw):
    """What rank `rank` of `world` works on.  replicas: its own batch of the workload's shape (own
    seed).  kv-heads: the one batch every rank draws identically, cut to this rank's KV heads of
    every page and the query heads that attend to them."""
    import synth
    if shard == "kv-heads" and world > 1:
        if spec.num_kv_heads % world:
            raise SystemExit(f"--shard kv-heads: {spec.num_kv_heads} KV heads do not split over {world} ranks")
        return synth.shard_kv_heads(synth.make_workload(spec, device, **kw), rank, world)
    if shard == "context":
        return synth.shard_context(synth.make_workload(spec, device, **kw), rank, world)
    return synth.make_workload(rank_spec(spec, rank, world), device, **kw)


def free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(script: str, argv, world: int, timeout_s: float = 3600.0) -> int:
    """Starts `world` processes of `python script argv...`, one per rank, with RANK / LOCAL_RANK /
    WORLD_SIZE / MASTER_ADDR / MASTER_PORT set, and waits for them.  Returns 0 only if every rank
    exited 0; as soon as one fails (or the time runs out) the others are terminated, so that a job with
    fewer ranks than asked for never reports a result."""
    port = free_port()
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.setdefault("NCCL_DEBUG", "INFO")               # the communicator's own log shows the rank count
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        procs.append(subprocess.Popen([sys.executable, script, *argv], env=env))
    deadline = time.time() + timeout_s
    rc = 0
    while procs and rc == 0:
        for pr in list(procs):
            code = pr.poll()
            if code is not None:
                procs.remove(pr)
                if code != 0:
                    rc = code if code > 0 else 1
        if time.time() > deadline:
            rc = 124
        time.sleep(0.05)
    for pr in procs:                                       # only after a failure: stop exactly what we started
        pr.terminate()
    for pr in procs:
        try:
            pr.wait(timeout=10)
        except subprocess.TimeoutExpired:
            pr.kill()
    return rc


def init_ranks(gpus: int, backend: str | None = None):
    """Reads this process's place in the job from the environment, joins the process group when there
    is more than one rank and returns (rank, local_rank, world, device).  The world size must be the
    --gpus the run was asked for.  backend None: nccl on cuda:LOCAL_RANK; "gloo": CPU (host-side tests)."""
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != gpus:
        raise SystemExit(f"bench.py: --gpus {gpus} but the job has {world} rank(s)")
    if backend == "gloo":
        dev = torch.device("cpu")
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
        if local >= torch.cuda.device_count():
            raise SystemExit(f"bench.py: rank {rank} has no GPU (LOCAL_RANK {local}, {torch.cuda.device_count()} visible)")
        torch.cuda.set_device(local)
        dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend == "gloo":
            dist.init_process_group("gloo", rank=rank, world_size=world)
        else:
            dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
        if dist.get_world_size() != gpus:
            raise SystemExit(f"bench.py: process group has {dist.get_world_size()} ranks, {gpus} asked for")
    return rank, local, world, dev


def over_ranks(values, op, device):
    """Element-wise MAX or SUM of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return t.tolist()


def run_reference(args):
    """The oracle timed on the host cores; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np
    import synth
    # the sample is built from the workload's lengths without building its full pools
    if args.workload in synth.CASCADE_SPECS:     # the oracle reads every sequence's whole context itself
        lens_list = [sh + o for sh, owns in synth.cascade_groups(args.workload) for o in owns]
        spec = synth.tiny_spec(args.workload, lens_list, synth.CASCADE_SPECS[args.workload][4],
                               synth.CASCADE_SPECS[args.workload][5])
    else:
        spec = synth.SPECS[args.workload]
    lens = synth.make_lengths(spec)
    cores = host_cores()
    # bounded sample: sequences in a seeded order, sized by a one-group calibration
    order = np.random.default_rng(7).permutation(spec.batch).tolist()
    probe = synth.make_workload(synth.tiny_spec("probe", (int(lens[order[0]]),), spec.page_size, spec.seed,
                                                q_std=spec.q_std, num_q_heads=spec.num_q_heads), "cpu")
    import oracle
    oracle.build()
    t0 = time.perf_counter()
    oracle.decode_attn(probe.q, probe.k_pages, probe.v_pages, probe.block_table, probe.seq_lens, probe.scale,
                       seqs=(0, 1), heads=(0, 8))
    per_token_core = (time.perf_counter() - t0) * 8 / max(1, int(lens[order[0]]))
    total_steps = args.steps + args.warmup
    budget_tokens = (120.0 / total_steps) * cores / max(per_token_core, 1e-12)
    seqs, tok = [], 0
    for b in order:
        seqs.append(b); tok += int(lens[b])
        if tok >= budget_tokens:
            break
    sample = synth.make_workload(
        synth.tiny_spec("sample", [int(lens[b]) for b in seqs], spec.page_size, spec.seed, q_std=spec.q_std,
                        k_outlier_prob=spec.k_outlier_prob, num_q_heads=spec.num_q_heads), "cpu")
    for _ in range(args.warmup):
        oracle_sample_throughput(sample, list(range(len(seqs))), cores)
    t = [oracle_sample_throughput(sample, list(range(len(seqs))), cores) for _ in range(args.steps)]
    dt = sum(t) / len(t)
    nbytes = sample.algorithmic_bytes()
    value = nbytes / dt / 1e9
    desc = (f"{len(seqs)} of {spec.batch} sequences ({tok} of {int(lens.sum())} KV tokens), all {spec.num_q_heads} query heads, per step")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "kv_tokens_per_s": tok / dt, "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_cascade(args):
    """Shared-prefix (cascade) decode step on a named cascade workload, 1 GPU or replicas."""
    import torch
    import torch.distributed as dist
    import synth
    import paper_2510_07356_b200 as P

    rank, local, world, dev = init_ranks(args.gpus)
    cw = synth.make_named_cascade(args.workload, dev)
    w, spec = cw.w, cw.w.spec
    attn = P.DecodeAttention(spec.page_size, spec.batch, w.block_table.shape[1], local)
    attn.set_option(P.CONCUR_OPT_PREFIX_KERNEL, args.prefix_kernel)
    out = torch.empty_like(w.q)
    lse = torch.empty((spec.batch, spec.num_q_heads), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)
    G = len(cw.prefix_lens_host)

    def step():
        P.concur_decode_attn_cascade(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens,
                                     cw.group_start, cw.prefix_lens, w.scale, out, lse, spec.batch, G,
                                     w.num_pages, w.block_table.shape[1], stream.cuda_stream)

    def plain_step():
        attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale, out=out, lse=lse)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    K = args.steps
    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    assert attn.status() == 0, "device-side flags set during warm-up"
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(K + 2)]
    for row in ev:
        for e in row:
            e.record(stream)
    barrier()
    t_mark0 = time.time()
    ev[K][0].record(stream)
    for _ in range(K):
        step()
    ev[K][1].record(stream)
    barrier()
    ms_per_step = ev[K][0].elapsed_time(ev[K][1]) / K
    for i in range(K):                       # the same steps with events around the prefix-pass kernel
        attn.set_option(P.CONCUR_OPT_EVENT_BEFORE_PARTIAL, ev[i][0].cuda_event)
        attn.set_option(P.CONCUR_OPT_EVENT_AFTER_PARTIAL, ev[i][1].cuda_event)
        step()
    barrier()
    t_mark1 = time.time()
    clocks = sampler.stop(t_mark0, t_mark1) if rank == 0 else None
    attn.set_option(P.CONCUR_OPT_EVENT_BEFORE_PARTIAL, 0)
    attn.set_option(P.CONCUR_OPT_EVENT_AFTER_PARTIAL, 0)
    pre_ms = [ev[i][0].elapsed_time(ev[i][1]) for i in range(K)]
    ev[K + 1][0].record(stream)              # the plain step on the same tables, for comparison
    for _ in range(K):
        plain_step()
    ev[K + 1][1].record(stream)
    barrier()
    plain_ms = ev[K + 1][0].elapsed_time(ev[K + 1][1]) / K
    ms_per_step, pre_ms_avg, plain_ms = over_ranks([ms_per_step, sum(pre_ms) / K, plain_ms], "max", dev)
    shared_b, logical_b, pre_b = cw.shared_bytes(), cw.logical_bytes(), synth.cascade_prefix_bytes(cw)
    job_shared, job_logical, job_tokens = over_ranks([shared_b, logical_b, w.kv_tokens], "sum", dev)
    flags = attn.status()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_peak()
    value = job_shared / (ms_per_step * 1e-3) / 1e9
    achieved = pre_b / (pre_ms_avg * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(3, args.warmup),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": spec.name, "batch": spec.batch, "groups": G, "kv_tokens_logical": w.kv_tokens,
                   "page_size": spec.page_size, "heads": "64q/8kv", "head_dim": 128,
                   "algorithmic_bytes": shared_b, "logical_bytes": logical_b, "prefix_pass_bytes": pre_b,
                   "l2": "inputs larger than L2", "entry": "concur_decode_attn_cascade",
                   "prefix_kernel": "tcgen05" if args.prefix_kernel == 0 else "mma.sync",
                   "parallelism": f"replicas x{world}" if world > 1 else "1 gpu"},
        "kv_tokens_per_s": job_tokens / (ms_per_step * 1e-3),
        "logical_gbs": job_logical / (ms_per_step * 1e-3) / 1e9,
        "plain_step_ms": plain_ms, "speedup_over_plain_step": plain_ms / ms_per_step,
        "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
        "frac_of_measured_copy": value / world / peak,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}",
                     "traffic": ATTN_TC_TRAFFIC_BYTES.get((args.workload, "tcgen05" if args.prefix_kernel == 0 else "mma.sync")),
                     "kernel": "prefix pass", "ms": pre_ms_avg,
                     "ms_min": min(pre_ms)},
        "e2e": None, "gpu_launches": 4 * K, "clocks": clocks, "device_flags": flags,
    }
    if not args.no_cpu and world == 1:       # the oracle leg belongs to the one-GPU run
        line["cpu_baseline"] = cpu_baseline(w, args.cpu_seconds)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_loop(args):
    """A token step of a model with L layers, replayed from one CUDA graph: per layer the new token's
    K/V rows are appended to that layer's pools and the layer's decode attention runs on them; the
    lengths (one set for all layers) grow by one per replay.  `loop<L>_<decode workload>`."""
    import torch
    import synth
    import paper_2510_07356_b200 as P

    rank, local, world, dev = init_ranks(args.gpus)
    head, base_name = args.workload.split("_", 1)
    L = int(head[len("loop"):])
    base = rank_spec(synth.SPECS[base_name], rank, world)
    K, W_ = args.steps, max(3, args.warmup)
    replays = 3 * (W_ + K) + 8                           # two full-step variants, attention-only, eager passes
    ws = [synth.make_workload(base, dev, spare_tokens=replays, value_seed=base.seed + 7919 * i) for i in range(L)]
    w0 = ws[0]
    spec = w0.spec
    B, stride = spec.batch, w0.block_table.shape[1]
    attn = P.DecodeAttention(spec.page_size, B, stride, local, num_q_heads=spec.num_q_heads,
                             num_kv_heads=spec.num_kv_heads)
    g = torch.Generator(device=dev); g.manual_seed(base.seed + 17)
    kn = torch.randn((L, B, spec.num_kv_heads, spec.head_dim), generator=g, device=dev).to(torch.bfloat16)
    vn = torch.randn((L, B, spec.num_kv_heads, spec.head_dim), generator=g, device=dev).to(torch.bfloat16)
    lens = w0.seq_lens.clone()
    outs = [torch.empty_like(w0.q) for _ in range(L)]
    lses = [torch.empty((B, spec.num_q_heads), dtype=torch.float32, device=dev) for _ in range(L)]
    stream = torch.cuda.current_stream(dev)
    flush = L2Flush(dev)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(dev)

    def append(i, s_):
        P.concur_kv_append_layer(attn.handle, kn[i], vn[i], ws[i].k_pages, ws[i].v_pages, w0.block_table, lens, B,
                                 w0.num_pages, stride, 1 if i == 0 else 0, s_)

    def attend(i, s_):
        P.concur_decode_attn(attn.handle, ws[i].q, ws[i].k_pages, ws[i].v_pages, w0.block_table, lens, w0.scale,
                             outs[i], lses[i], B, w0.num_pages, stride, s_)

    def token_step():                                    # what a model does: layer by layer
        s_ = torch.cuda.current_stream(dev).cuda_stream
        for i in range(L):
            append(i, s_)
            attend(i, s_)

    def fused_step():                                    # the same work with the append inside the attention kernel
        s_ = torch.cuda.current_stream(dev).cuda_stream
        append(0, s_)                                    # the step's first append advances the lengths ...
        attend(0, s_)
        for i in range(1, L):                            # ... the other layers' rows go in with their attention call
            P.concur_decode_attn_append(attn.handle, ws[i].q, kn[i], vn[i], ws[i].k_pages, ws[i].v_pages, w0.block_table,
                                        lens, w0.scale, outs[i], lses[i], B, w0.num_pages, stride, s_)

    def attention_chain():                               # the L attention calls alone, back to back
        s_ = torch.cuda.current_stream(dev).cuda_stream
        for i in range(L):
            attend(i, s_)

    def capture(fn):
        side = torch.cuda.Stream(dev)
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            fn()                                         # first-call set-up stays outside the capture
        stream.wait_stream(side)
        torch.cuda.synchronize(dev)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            fn()
        return graph

    def timed(graph, n):
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n)]
        for row in ev:
            for e in row:
                e.record(stream)
        barrier()
        for i in range(n):
            flush()                                      # every replay starts with none of the pools in L2
            ev[i][0].record(stream)
            graph.replay()
            ev[i][1].record(stream)
        barrier()
        return [ev[i][0].elapsed_time(ev[i][1]) for i in range(n)]

    results = {}
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)
    clocks = None
    for name, fn, overlap in (("fused", fused_step, 1), ("interleaved", token_step, 0),
                              ("attention_only", attention_chain, 0), ("attention_only_overlapped", attention_chain, 1)):
        attn.set_option(P.CONCUR_OPT_OVERLAP_CALLS, overlap)
        graph = capture(fn)
        timed(graph, W_)
        if name == "fused" and rank == 0:
            sampler.start(); time.sleep(0.2)
        t0m = time.time()
        ms = timed(graph, K)
        if name == "fused" and rank == 0:
            clocks = sampler.stop(t0m, time.time())
        results[name] = over_ranks([sum(ms) / K, min(ms)], "max", dev)
        del graph
    attn.set_option(P.CONCUR_OPT_OVERLAP_CALLS, 0)
    assert attn.status() == 0, "device-side flags set"
    # the partial kernel alone, eagerly, with the library's events around it (one pass over the layers)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(L)]
    for row in ev:
        for e in row:
            e.record(stream)
    part = []
    for _ in range(2):
        flush()
        for i in range(L):
            attn.set_option(P.CONCUR_OPT_EVENT_BEFORE_PARTIAL, ev[i][0].cuda_event)
            attn.set_option(P.CONCUR_OPT_EVENT_AFTER_PARTIAL, ev[i][1].cuda_event)
            attend(i, stream.cuda_stream)
        barrier()
        part = [ev[i][0].elapsed_time(ev[i][1]) for i in range(L)]
    attn.set_option(P.CONCUR_OPT_EVENT_BEFORE_PARTIAL, 0)
    attn.set_option(P.CONCUR_OPT_EVENT_AFTER_PARTIAL, 0)
    part_ms = over_ranks([sum(part) / L], "max", dev)[0]
    # parity of the last layer, as the loop left it, against the oracle (one-GPU runs)
    lens_now = lens.cpu().numpy().astype("int32")
    w_last = ws[L - 1]
    w_last.seq_lens = lens.clone(); w_last.lens_host = lens_now
    token_bytes = 2 * spec.num_kv_heads * spec.head_dim * 2
    layer_bytes = w_last.algorithmic_bytes() + B * token_bytes       # the layer's attention plus its appended rows
    job_bytes = over_ranks([float(layer_bytes) * L], "sum", dev)[0]
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    if rank != 0:
        return
    peak, peak_kind = measured_peak()
    ms_step, ms_min = results["fused"]
    achieved = w_last.algorithmic_bytes() / (part_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": job_bytes / (ms_step * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W_, "warmup_requested": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "layers": L, "batch": B, "kv_tokens_per_layer": int(lens_now.sum()),
                   "page_size": spec.page_size, "heads": f"{spec.num_q_heads}q/{spec.num_kv_heads}kv", "head_dim": 128,
                   "algorithmic_bytes_per_layer": layer_bytes,
                   "l2": "flushed before every replay (256 MB written, then 256 MB read)",
                   "step": "one CUDA graph: the first layer concur_kv_append_layer + concur_decode_attn, every other "
                           "layer one concur_decode_attn_append launch; calls may overlap (CONCUR_OPT_OVERLAP_CALLS)",
                   "parallelism": f"replicas x{world}" if world > 1 else "1 gpu"},
        "us_per_layer": ms_step * 1e3 / L, "us_per_layer_min": ms_min * 1e3 / L,
        "append_then_attend_us_per_layer": results["interleaved"][0] * 1e3 / L,
        "attention_only_us_per_layer": results["attention_only"][0] * 1e3 / L,
        "attention_only_overlapped_us_per_layer": results["attention_only_overlapped"][0] * 1e3 / L,
        "frac_of_measured_copy": job_bytes / world / (ms_step * 1e-3) / 1e9 / peak,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "traffic": None, "kernel": "partial (mean over the layers, eager pass)",
                     "ms": part_ms},
        "e2e": None, "gpu_launches": (L + 1) * K, "clocks": clocks,
    }
    if not args.no_cpu and world == 1:
        line["cpu_baseline"], line["parity"] = cpu_baseline(w_last, args.cpu_seconds, (outs[L - 1], lses[L - 1]))
    print(json.dumps(line), flush=True)


def measured_tensor_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        return 1590.0, "fallback"


def run_prefill(args):
    """Causal prefill attention on a named prefill workload (1 GPU or replicas): useful TFLOP/s."""
    import torch
    import torch.distributed as dist
    import synth
    import paper_2510_07356_b200 as P

    rank, local, world, dev = init_ranks(args.gpus)
    pw = synth.make_named_prefill(args.workload, dev)
    w, spec = pw.w, pw.w.spec
    attn = P.DecodeAttention(spec.page_size, spec.batch, w.block_table.shape[1], local)
    attn.set_option(P.CONCUR_OPT_PREFILL_KERNEL, args.prefill_kernel)
    pf_kernel = "pair" if args.prefill_kernel == 0 else "single"
    tq = pw.total_q
    out = torch.empty((tq, spec.num_q_heads, spec.head_dim), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((tq, spec.num_q_heads), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)

    def step():
        P.concur_prefill_attn(attn.handle, w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, pw.q_start,
                              w.scale, out, lse, spec.batch, tq, w.num_pages, w.block_table.shape[1],
                              stream.cuda_stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    K = args.steps
    flush_buf = L2Flush(dev)                                                      # the caches fit in L2
    for _ in range(max(3, args.warmup)):
        flush_buf()
        step()
    barrier()
    assert attn.status() == 0, "device-side flags set during warm-up"
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(K)]
    for row in ev:                       # materialise the cudaEvent_t handles outside the timed region
        for e in row:
            e.record(stream)
    barrier()
    t_mark0 = time.time()
    for i in range(K):
        flush_buf()
        ev[i][0].record(stream)
        step()
        ev[i][1].record(stream)
    barrier()
    t_mark1 = time.time()
    clocks = sampler.stop(t_mark0, t_mark1) if rank == 0 else None
    step_ms = [ev[i][0].elapsed_time(ev[i][1]) for i in range(K)]
    ms_per_step = over_ranks([sum(step_ms) / K], "max", dev)[0]
    flops = pw.flops()
    job_flops, job_q = over_ranks([flops, tq], "sum", dev)
    flags = attn.status()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_tensor_peak()
    value = job_flops / (ms_per_step * 1e-3) / 1e12
    line = {
        "metric": "prefill_attention_useful_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": K,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": spec.name, "prompts": spec.batch, "query_tokens": tq, "kv_tokens": w.kv_tokens,
                   "page_size": spec.page_size, "heads": f"{spec.num_q_heads}q/{spec.num_kv_heads}kv", "head_dim": 128,
                   "causal_flops": flops, "l2": "flushed between steps (256 MB written, then 256 MB read)", "entry": "concur_prefill_attn",
                   "parallelism": f"replicas x{world}" if world > 1 else "1 gpu"},
        "query_tokens_per_s": job_q / (ms_per_step * 1e-3),
        "roofline": {"bound": "tensor", "achieved": value / world, "peak": peak, "unit": "TFLOP/s",
                     "frac": value / world / peak, "peak_kind": f"of {peak_kind}",
                     "traffic": ATTN_TC_TRAFFIC_BYTES.get((spec.name, pf_kernel)),
                     "kernel": "plan + " + ("prefill_pair_kernel" if pf_kernel == "pair" else "attn_tc_kernel<prefill>"), "ms": ms_per_step, "ms_min": min(step_ms)},
        "e2e": None, "gpu_launches": 2 * K, "clocks": clocks, "device_flags": flags,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_curate(args):
    """The curation arithmetic on the synthesis-run-shaped record table (rank 0 only; the job is
    tiny and does not shard)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np
    import torch
    import paper_2510_07356_b200 as P
    from synth import records as R
    B = P.binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    rec = R.make_records()
    N, M = rec.correct.shape
    host = [rec.correct, rec.t_torch, rec.t_kernel, rec.length, rec.sample_key, rec.task_key]
    pinned = [torch.from_numpy(np.ascontiguousarray(a)).pin_memory() for a in host]
    ins = [t.to(dev) for t in pinned]
    outs = [torch.empty((N, M), device=dev), torch.empty((N,), dtype=torch.int32, device=dev),
            torch.empty((N, M), dtype=torch.uint8, device=dev), torch.empty((4, N), dtype=torch.int32, device=dev),
            torch.empty((4, N), dtype=torch.uint8, device=dev), torch.empty((N,), dtype=torch.uint8, device=dev),
            torch.empty((B.CONCUR_CURATE_NUM_STATS,), dtype=torch.float64, device=dev)]
    prm = B.concur_curate_params_t(N, M, 5.0, 1.0, 4892, 4000, 8500, 0)
    stream = torch.cuda.current_stream(dev)

    def step():
        B.concur_curate(prm, *ins, *outs, stream.cuda_stream)

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize(dev)
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = "0"
    sampler = ClockSampler(gpu_id)
    sampler.start(); time.sleep(0.2)
    K = args.steps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream); e1.record(stream); torch.cuda.synchronize(dev)
    t0m = time.time()
    e0.record(stream)
    for _ in range(K):
        step()
    e1.record(stream)
    torch.cuda.synchronize(dev)
    ms = e0.elapsed_time(e1) / K
    # end to end: records from pinned host memory, the statistics and the rule (a) picks read back
    stats_h = torch.empty(B.CONCUR_CURATE_NUM_STATS, dtype=torch.float64).pin_memory()
    rule_a_h = torch.empty(N, dtype=torch.int32).pin_memory()
    e0.record(stream)
    for _ in range(K):
        for d, h in zip(ins, pinned):
            d.copy_(h, non_blocking=True)
        step()
        stats_h.copy_(outs[6], non_blocking=True); rule_a_h.copy_(outs[1], non_blocking=True)
    e1.record(stream)
    torch.cuda.synchronize(dev)
    e2e_ms = e0.elapsed_time(e1) / K
    clocks = sampler.stop(t0m, time.time())
    # CPU baseline: the oracle, as it stands, on the whole table
    from oracle import curation as C
    t0 = time.perf_counter()
    sp = C.speedup(rec.correct, rec.t_torch, rec.t_kernel)
    C.rule_a(rec.correct, sp, rec.length); C.rule_b(sp); C.difficulty(rec.length); C.pearson(rec.length, sp, rec.correct)
    C.select_random(rec.correct, rec.sample_key, rec.task_key, 4892); C.select_max_length(rec.correct, rec.length, 4892)
    C.select_min_length(rec.correct, rec.length, 4892); C.select_speedup(rec.correct, sp, 4892)
    cpu_s = time.perf_counter() - t0
    records = N * M
    # the counting rank dominates: 4 selections x N^2 (key, index) comparisons of about 4 lane
    # operations each, against 148 SMs x 128 lanes at the sampled SM clock
    comparisons = 4.0 * N * N
    mhz = (clocks or {}).get("sm_mhz") or 1965.0
    alu_peak = 148 * 128 * mhz * 1e6 / 4.0
    line = {"metric": "curation_records_per_s", "value": records / (ms * 1e-3), "unit": "records/s", "n_gpus": 1,
            "steps": K, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "replicas only", "vs_baseline": None, "dtype": "f32/f64/int32", "data": "synthetic",
            "config": {"workload": "curate_18162x5", "tasks": N, "generations": M, "top_k": 4892},
            "roofline": {"bound": "alu", "achieved": comparisons / (ms * 1e-3), "peak": alu_peak,
                         "unit": "rank comparisons/s", "frac": comparisons / (ms * 1e-3) / alu_peak, "traffic": None,
                         "kernel": "curate_rank_kernel (whole call timed; it is > 90 % of it)"},
            "e2e": {"value": records / (e2e_ms * 1e-3), "unit": "records/s", "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": int(sum(t.numel() * t.element_size() for t in pinned)),
                    "d2h_bytes_per_step": int(stats_h.numel() * 8 + rule_a_h.numel() * 4), "entry": "concur_curate"},
            "cpu_baseline": {"value": records / cpu_s, "unit": "records/s", "cores": 1, "kind": "oracle",
                             "sample": f"the whole table once, {cpu_s:.1f} s"},
            "gpu_launches": 3 * K, "clocks": clocks}
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    if args.impl == "reference":
        run_reference(args)
        return
    if args.shard == "kv-heads" and args.workload.startswith(("casc", "prefill", "curate", "loop")):
        raise SystemExit("bench.py: --shard kv-heads is implemented for the plain decode workloads")
    if args.shard == "context" and args.workload.startswith(("casc", "prefill", "curate", "loop")):
        raise SystemExit("bench.py: --shard context is implemented for the plain decode workloads")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no outside launcher: this process becomes the launcher of its own N ranks
        raise SystemExit(spawn_ranks(os.path.abspath(__file__), sys.argv[1:], args.gpus))
    if args.workload.startswith("loop"):
        run_loop(args)
        return
    if args.workload.startswith("casc"):
        run_cascade(args)
        return
    if args.workload.startswith("prefill"):
        run_prefill(args)
        return
    if args.workload.startswith("curate"):
        run_curate(args)
        return

    import torch
    import torch.distributed as dist
    import synth
    import paper_2510_07356_b200 as P
    from paper_2510_07356_b200 import bench_probe

    rank, local, world, dev = init_ranks(args.gpus)

    # replicas: every rank decodes its own batch of the same shape; kv-heads: the ranks split one batch
    # over its KV heads.  Neither has a data-path collective.
    w = rank_workload(synth.SPECS[args.workload], rank, world, args.shard, dev, spare_tokens=args.loop_steps)
    spec = w.spec
    attn = P.DecodeAttention(spec.page_size, spec.batch, w.block_table.shape[1], local,
                             num_q_heads=spec.num_q_heads, num_kv_heads=spec.num_kv_heads,
                             kv_layout=args.kv_layout)
    if args.kv_layout == 1:              # the same cache as [page][slot][KV head][D]
        w.k_pages = w.k_pages.permute(0, 2, 1, 3).contiguous()
        w.v_pages = w.v_pages.permute(0, 2, 1, 3).contiguous()
        args.no_cpu = True               # the oracle reads head-major pools; parity is the tests' business
    attn.set_option(P.CONCUR_OPT_KERNEL, args.kernel)
    attn.set_option(P.CONCUR_OPT_RANGES_PER_CTA, args.ranges_per_cta)
    attn.set_option(P.CONCUR_OPT_MIN_RANGE_TILES, args.min_range_tiles)
    attn.set_option(P.CONCUR_OPT_NUM_RANGES, args.num_ranges)
    if args.fuse_combine >= 0:
        attn.set_option(P.CONCUR_OPT_FUSE_COMBINE, args.fuse_combine)
    if args.small_page_copy >= 0:
        attn.set_option(P.CONCUR_OPT_SMALL_PAGE_COPY, args.small_page_copy)
    if args.claim_ahead >= 0:
        attn.set_option(P.CONCUR_OPT_CLAIM_AHEAD, args.claim_ahead)
    out = torch.empty_like(w.q)
    lse = torch.empty((spec.batch, spec.num_q_heads), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)
    nbytes = w.algorithmic_bytes()
    kv_bytes = w.kv_tokens * 2 * spec.num_kv_heads * spec.head_dim * 2
    flush_needed = kv_bytes < 512 * 1024 * 1024          # inputs not well above the 126 MB L2
    flush_buf = L2Flush(dev) if flush_needed else None

    ctx = args.shard == "context"
    if ctx:
        # every rank's (out, lse) over its token range, gathered from all ranks, then merged on every rank
        args.loop_steps = 0
        args.no_e2e = True
        rows = spec.batch * spec.num_q_heads
        out_part = torch.empty_like(w.q)
        lse_part = torch.empty((spec.batch, spec.num_q_heads), dtype=torch.float32, device=dev)
        gath_out = torch.empty((world,) + tuple(w.q.shape), dtype=torch.bfloat16, device=dev)
        gath_lse = torch.empty((world, spec.batch, spec.num_q_heads), dtype=torch.float32, device=dev)

    def step():
        if not ctx:
            attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale, out=out, lse=lse)
            return
        attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale, out=out_part, lse=lse_part)
        if world > 1:
            dist.all_gather_into_tensor(gath_out, out_part)
            dist.all_gather_into_tensor(gath_lse, lse_part)
        else:
            gath_out[0].copy_(out_part); gath_lse[0].copy_(lse_part)
        P.concur_lse_merge(gath_out, gath_lse, world, rows, out, lse, torch.cuda.current_stream(dev).cuda_stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(max(3, args.warmup)):
        if flush_buf is not None:
            flush_buf()
        step()
    barrier()
    assert attn.status() == 0, "device-side flags set during warm-up"

    # ---- timed region: K whole steps, one event pair around the region
    K = args.steps
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(K + 1)]
    for row in ev:                       # materialise the cudaEvent_t handles
        for e in row:
            e.record(stream)
    barrier()
    t_mark0 = time.time()
    if flush_buf is None:
        ev[K][0].record(stream)
        for i in range(K):
            step()
        ev[K][1].record(stream)
        barrier()
        ms_per_step = ev[K][0].elapsed_time(ev[K][1]) / K
        step_ms = [ms_per_step]
    else:                                # small inputs: L2 is flushed before every step, steps timed one by one
        for i in range(K):
            flush_buf()
            ev[i][0].record(stream)
            step()
            ev[i][1].record(stream)
        barrier()
        step_ms = [ev[i][0].elapsed_time(ev[i][1]) for i in range(K)]
        ms_per_step = sum(step_ms) / K
    # ---- the same K steps again with events recorded by the library around its partial kernel
    for i in range(K):
        if flush_buf is not None:
            flush_buf()
        attn.set_option(P.CONCUR_OPT_EVENT_BEFORE_PARTIAL, ev[i][0].cuda_event)
        attn.set_option(P.CONCUR_OPT_EVENT_AFTER_PARTIAL, ev[i][1].cuda_event)
        step()
    barrier()
    t_mark1 = time.time()
    clocks = sampler.stop(t_mark0, t_mark1) if rank == 0 else None
    attn.set_option(P.CONCUR_OPT_EVENT_BEFORE_PARTIAL, 0)
    attn.set_option(P.CONCUR_OPT_EVENT_AFTER_PARTIAL, 0)
    part_ms = [ev[i][0].elapsed_time(ev[i][1]) for i in range(K)]
    part_ms_avg = sum(part_ms) / K
    ms_per_step, part_ms_avg = over_ranks([ms_per_step, part_ms_avg], "max", dev)
    job_bytes, job_tokens = over_ranks([nbytes, w.kv_tokens], "sum", dev)     # units all ranks processed
    flags = attn.status()
    R, W, _ = attn.last_plan()

    # ---- end to end: host buffers, every copy inside the timed region
    e2e = None
    if not args.no_e2e:
        pin = lambda t: t.cpu().contiguous().pin_memory()
        hq, hk, hv, hbt, hsl = pin(w.q), pin(w.k_pages), pin(w.v_pages), pin(w.block_table), pin(w.seq_lens)
        hout = torch.empty(w.q.shape, dtype=torch.bfloat16).pin_memory()
        hlse = torch.empty((spec.batch, spec.num_q_heads), dtype=torch.float32).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hbt, hsl))
        d2h = hout.numel() * 2 + hlse.numel() * 4

        def host_step():
            P.concur_decode_attn_host(attn.handle, hq, hk, hv, hbt, hsl, w.scale, hout, hlse, spec.batch,
                                      hk.shape[0], hbt.shape[1], stream.cuda_stream)
        host_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.e2e_steps):
            host_step()
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1) / args.e2e_steps
        e2e_ms = over_ranks([e2e_ms], "max", dev)[0]
        e2e = {"value": job_bytes / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": args.e2e_steps,
               "entry": "concur_decode_attn_host"}
        assert torch.equal(hout.view(torch.int16), out.cpu().view(torch.int16)), "host path differs from device path"
        del hq, hk, hv

    # ---- the same step back to back for about two seconds: what the power cap leaves of the burst figure
    sustained = None
    if flush_buf is None and args.sustained_seconds > 0:
        def back_to_back(fn, one_ms, seconds, stamps=None):
            chunk = max(10, int(0.1 / max(one_ms * 1e-3, 1e-6)))           # about 0.1 s of calls per event pair
            marks, t_end = [], time.time() + seconds
            while time.time() < t_end:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                t_a = time.time()
                e0.record(stream)
                for _ in range(chunk):
                    fn()
                e1.record(stream)
                e1.synchronize()
                marks.append(e0.elapsed_time(e1) / chunk)
                if stamps is not None:
                    stamps.append((0.5 * (t_a + time.time()), marks[-1]))
            tail = marks[len(marks) // 2:]                                 # the second half: clocks have settled
            return sum(tail) / len(tail), marks[0], chunk * len(marks)

        def by_clock(stamps, sampler_lines):
            """Chunks of the sustained run grouped by the SM clock sampled nearest to them: how the step
            time moves with the clock the power cap leaves (no clock is ever set from here)."""
            pts = []
            for t, l in sampler_lines:
                try:
                    pts.append((t, float(l.split(",")[0])))
                except ValueError:
                    pass
            if not pts:
                return None
            bins = {}
            for t, ms in stamps:
                mhz = min(pts, key=lambda q: abs(q[0] - t))[1]
                bins.setdefault(mhz, []).append(ms)
            return [{"sm_mhz": k, "chunks": len(v), "ms_per_step": sum(v) / len(v), "ms_x_ghz": sum(v) / len(v) * k / 1e3}
                    for k, v in sorted(bins.items())]

        sampler2 = ClockSampler(gpu_id)
        if rank == 0:
            sampler2.start()
            time.sleep(0.2)
        t_s0 = time.time()
        stamps = []
        sus_ms, first_ms, n_steps = back_to_back(step, ms_per_step, args.sustained_seconds, stamps)
        t_s1 = time.time()
        sus_clocks = sampler2.stop(t_s0, t_s1) if rank == 0 else None
        sus_ms = over_ranks([sus_ms], "max", dev)[0]
        sustained = {"ms_per_step": sus_ms, "value": job_bytes / (sus_ms * 1e-3) / 1e9, "unit": UNIT,
                     "seconds": args.sustained_seconds, "steps": n_steps, "first_chunk_ms_per_step": first_ms,
                     "clocks": sus_clocks, "by_clock": by_clock(stamps, sampler2.lines) if rank == 0 else None,
                     "what": "steps back to back; mean of the second half of the interval"}
        # the read-only stream under the same regime, so that the two can be compared like for like
        pool_b = w.k_pages.numel() * 2 + w.v_pages.numel() * 2
        chk_s = torch.zeros(2, dtype=torch.int32, device=dev)

        def probe_s():
            bench_probe.read_probe(w.k_pages, w.k_pages.numel() * 2, chk_s[0:1], 0, stream.cuda_stream)
            bench_probe.read_probe(w.v_pages, w.v_pages.numel() * 2, chk_s[1:2], 0, stream.cuda_stream)

        sampler3 = ClockSampler(gpu_id)
        if rank == 0:
            sampler3.start()
            time.sleep(0.2)
        stamps_p = []
        t_p0 = time.time()
        probe_ms, _, _ = back_to_back(probe_s, ms_per_step, args.sustained_seconds / 2, stamps_p)
        probe_clocks = sampler3.stop(t_p0, time.time()) if rank == 0 else None
        sustained["read_stream_gbs"] = pool_b / (probe_ms * 1e-3) / 1e9
        sustained["read_stream_clocks"] = probe_clocks
        sustained["read_stream_by_clock"] = by_clock(stamps_p, sampler3.lines) if rank == 0 else None

    # ---- yardstick: a plain read-only stream over the same two pools (only where they are well above L2)
    read_stream = None
    pool_bytes = w.k_pages.numel() * 2 + w.v_pages.numel() * 2
    if pool_bytes >= 512 * 1024 * 1024:
        chk = torch.zeros(2, dtype=torch.int32, device=dev)

        def probe():
            bench_probe.read_probe(w.k_pages, w.k_pages.numel() * 2, chk[0:1], 0, stream.cuda_stream)
            bench_probe.read_probe(w.v_pages, w.v_pages.numel() * 2, chk[1:2], 0, stream.cuda_stream)

        for _ in range(3):
            probe()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(10):
            probe()
        e1.record(stream)
        barrier()
        probe_ms = over_ranks([e0.elapsed_time(e1) / 10], "max", dev)[0]
        read_stream = {"gbs": pool_bytes / (probe_ms * 1e-3) / 1e9, "bytes": pool_bytes, "ms": probe_ms,
                       "what": "read-only stream kernel of the bench's helper library over k_pages then v_pages (16-byte loads, xor checksum), 10 passes"}

    # ---- decode loop: KV append + attention per step, replayed from one CUDA graph
    loop = None
    if args.loop_steps > 0:
        g = torch.Generator(device=dev); g.manual_seed(spec.seed + 17)
        kn = torch.randn((spec.batch, spec.num_kv_heads, spec.head_dim), generator=g, device=dev).to(torch.bfloat16)
        vn = torch.randn((spec.batch, spec.num_kv_heads, spec.head_dim), generator=g, device=dev).to(torch.bfloat16)
        lens_loop = w.seq_lens.clone()

        def loop_step():
            s_ = torch.cuda.current_stream(dev).cuda_stream
            P.concur_kv_append(attn.handle, kn, vn, w.k_pages, w.v_pages, w.block_table, lens_loop, spec.batch,
                               w.num_pages, w.block_table.shape[1], s_)
            attn(w.q, w.k_pages, w.v_pages, w.block_table, lens_loop, w.scale, out=out, lse=lse)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            loop_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.loop_steps):
            graph.replay()
        e1.record(stream)
        barrier()
        loop_ms = over_ranks([e0.elapsed_time(e1) / args.loop_steps], "max", dev)[0]
        assert int(lens_loop[0]) == int(w.lens_host[0]) + args.loop_steps
        loop = {"steps": args.loop_steps, "ms_per_step": loop_ms,
                "launches_per_step": 2 if (args.kernel == 0 and args.fuse_combine != 0 and spec.batch <= 511) else 3,
                "what": "concur_kv_append + concur_decode_attn replayed from a CUDA graph, lengths +1 per step"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    value = job_bytes / (ms_per_step * 1e-3) / 1e9
    achieved = nbytes / (part_ms_avg * 1e-3) / 1e9
    # the tensor-core kernel with the merge fused is the whole step for up to 511 sequences; beyond that a
    # plan kernel runs ahead of it; the scalar kernel, or an unfused merge, adds the combine kernel
    fused = args.kernel == 0 and args.fuse_combine != 0
    launches_per_step = ((1 if spec.batch <= 511 else 2) if fused else 3) + (1 if ctx else 0)
    traffic = None
    if args.kernel == 0 and spec.page_size == 64 and MMA_P64_TRAFFIC_BYTES_PER_KV_TOKEN:
        traffic = MMA_P64_TRAFFIC_BYTES_PER_KV_TOKEN * w.kv_tokens     # scaled from the quarter-size capture
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(3, args.warmup),
        "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "strong" if (args.shard in ("kv-heads", "context") and world > 1) else "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "warmup_requested": args.warmup,
        "config": {"workload": args.workload, "rank0_shard": spec.name, "seed": spec.seed, "batch": spec.batch, "kv_tokens": w.kv_tokens, "page_size": spec.page_size,
                   "heads": f"{spec.num_q_heads}q/{spec.num_kv_heads}kv", "head_dim": 128, "algorithmic_bytes": nbytes,
                   "l2": "flushed between steps (256 MB written, then 256 MB read)" if flush_needed else "inputs larger than L2",
                   "kernel": "mma" if args.kernel == 0 else "scalar", "ranges": R, "tiles": W,
                   "kv_layout": "token-major" if args.kv_layout == 1 else "head-major",
                   "parallelism": "1 gpu" if world == 1 else
                                  (f"kv-heads x{world} ({spec.num_kv_heads} KV heads per rank)" if args.shard == "kv-heads"
                                   else (f"context x{world} (token ranges; all-gather of (out, lse) + concur_lse_merge in the step)"
                                         if ctx else f"replicas x{world}"))},
        "kv_tokens_per_s": (w.kv_tokens if args.shard == "kv-heads" else job_tokens) / (ms_per_step * 1e-3),
        "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
        "frac_of_measured_copy": value / world / peak,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "traffic": traffic, "kernel": "partial", "ms": part_ms_avg,
                     "ms_min": min(part_ms)},
        "step_ms_min": min(step_ms), "step_ms_median": statistics.median(step_ms),
        "sustained": sustained,
        "read_stream": read_stream,
        "frac_of_measured_read_stream": (achieved / read_stream["gbs"]) if read_stream else None,
        "decode_loop": loop, "e2e": e2e, "gpu_launches": launches_per_step * K, "clocks": clocks, "device_flags": flags,
    }
    if not args.no_cpu and world == 1:       # the oracle leg belongs to the one-GPU run
        step()                                   # the inputs as they are now, once more, for the comparison
        torch.cuda.synchronize(dev)
        line["cpu_baseline"], line["parity"] = cpu_baseline(w, args.cpu_seconds, (out, lse))
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
