"""Seeded synthetic inputs for paged-KV decode attention.

Shared by the tests, the benchmark and the smoke check; holds none of the
method's arithmetic (no dot products, no softmax) -- only random tensors, context
lengths and block tables shaped like the decoding of long reasoning traces by a
32B-class GQA model (64 query heads, 8 KV heads, head_dim 128, bf16; traces of a
few thousand to 32,768 tokens, several samples per prompt).

Conventions
-----------
* pools are ``[num_pages][Hkv][P][D]`` bf16; K and V share page ids;
* the pool holds exactly ``sum_b ceil(len_b / P)`` pages; the i-th logical page
  in sequence-major order lives in physical page ``perm[i]`` (identity when the
  table is "contiguous", one seeded permutation otherwise);
* unused block-table entries are -1; slots at or beyond a sequence's length in its
  last page are filled with bf16 NaN in K and V (a correct kernel never lets them
  reach its output);
* "uniform in [a, b]" is integer, both ends inclusive; "log-uniform" is
  ``round(a * (b/a)**u)``, u ~ U[0,1), clamped to [a, b];
* every random draw comes from a counter-based generator (numpy Philox for
  lengths and permutations, torch's Philox-backed generator for tensors) seeded
  from the workload's seed and a per-tensor stream id, so a workload is a pure
  function of (name, seed, device type).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

NUM_Q_HEADS = 64
NUM_KV_HEADS = 8
HEAD_DIM = 128


@dataclass
class Spec:
    name: str
    batch: int
    page_size: int
    lengths: tuple            # ("const", n) | ("uniform", a, b) | ("loguniform", a, b) | ("skew", long, a, b) | ("list", [...])
    permute_pages: bool = True
    q_std: float = 1.0
    k_outlier_prob: float = 0.0   # probability that a token position's K rows (all KV heads) are scaled
    k_outlier_scale: float = 20.0
    seed: int = 0
    num_q_heads: int = NUM_Q_HEADS
    num_kv_heads: int = NUM_KV_HEADS
    head_dim: int = HEAD_DIM


# The five decode configurations (batch / context mix / page size), seeds 73561..73565.
SPECS = {
    "cfg1_b1_ctx512_p16": Spec("cfg1_b1_ctx512_p16", 1, 16, ("const", 512), permute_pages=False, seed=73561),
    "cfg2_b16_u1k_8k_p16": Spec("cfg2_b16_u1k_8k_p16", 16, 16, ("uniform", 1024, 8192), seed=73562),
    "cfg3_b64_ctx16384_p64": Spec("cfg3_b64_ctx16384_p64", 64, 64, ("const", 16384), q_std=0.5, seed=73563),
    # a quarter of cfg3 (same lengths, page size and values): small enough for profiler captures
    "cfg3q_b16_ctx16384_p64": Spec("cfg3q_b16_ctx16384_p64", 16, 64, ("const", 16384), q_std=0.5, seed=73563),
    # config 3 with every sequence's pages in logical order, one sequence after the other (no shuffle): the
    # same bytes as one linear stream per (sequence, head), to tell page placement from everything else
    "cfg3c_b64_ctx16384_p64": Spec("cfg3c_b64_ctx16384_p64", 64, 64, ("const", 16384), permute_pages=False,
                                   q_std=0.5, seed=73563),
    # config 3 with 40 query heads (group size 5): the geometry variant of the same workload
    "cfg3h40_b64_ctx16384_p64": Spec("cfg3h40_b64_ctx16384_p64", 64, 64, ("const", 16384), q_std=0.5, seed=73563,
                                     num_q_heads=40),
    # what one rank of config 3 holds when the model is tensor-parallel over its KV heads on 8 / 4 / 2 GPUs
    "cfg3kv1_b64_ctx16384_p64": Spec("cfg3kv1_b64_ctx16384_p64", 64, 64, ("const", 16384), q_std=0.5, seed=73563,
                                     num_q_heads=8, num_kv_heads=1),
    "cfg3kv2_b64_ctx16384_p64": Spec("cfg3kv2_b64_ctx16384_p64", 64, 64, ("const", 16384), q_std=0.5, seed=73563,
                                     num_q_heads=16, num_kv_heads=2),
    "cfg3kv4_b64_ctx16384_p64": Spec("cfg3kv4_b64_ctx16384_p64", 64, 64, ("const", 16384), q_std=0.5, seed=73563,
                                     num_q_heads=32, num_kv_heads=4),
    "cfg4_b256_logu2k_32k_p64": Spec("cfg4_b256_logu2k_32k_p64", 256, 64, ("loguniform", 2048, 32768), seed=73564),
    "cfg5_b32_skew128k_p64": Spec("cfg5_b32_skew128k_p64", 32, 64, ("skew", 131072, 256, 4096),
                                  k_outlier_prob=0.01, seed=73565),
}


@dataclass
class Workload:
    spec: Spec
    q: torch.Tensor            # [B][Hq][D] bf16
    k_pages: torch.Tensor      # [pages][Hkv][P][D] bf16
    v_pages: torch.Tensor
    block_table: torch.Tensor  # [B][stride] int32
    seq_lens: torch.Tensor     # [B] int32
    scale: float
    lens_host: np.ndarray = field(default=None)
    table_host: np.ndarray = field(default=None)

    @property
    def num_pages(self) -> int:
        return self.k_pages.shape[0]

    @property
    def kv_tokens(self) -> int:
        return int(self.lens_host.sum())

    def algorithmic_bytes(self) -> int:
        """K+V bytes of every cached token, q/out/lse of every sequence, and the block-table
        entries and lengths the operation must read."""
        s = self.spec
        per_token = 2 * s.num_kv_heads * s.head_dim * 2
        per_seq = 2 * s.num_q_heads * s.head_dim * 2 + s.num_q_heads * 4
        pages = int(np.sum((self.lens_host.astype(np.int64) + s.page_size - 1) // s.page_size))
        return self.kv_tokens * per_token + s.batch * (per_seq + 4) + pages * 4


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def make_lengths(spec: Spec) -> np.ndarray:
    r = _rng(spec.seed, 1)
    kind = spec.lengths[0]
    B = spec.batch
    if kind == "const":
        lens = np.full(B, spec.lengths[1], dtype=np.int64)
    elif kind == "list":
        lens = np.asarray(spec.lengths[1], dtype=np.int64)
        assert lens.shape == (B,)
    elif kind == "uniform":
        _, a, b = spec.lengths
        lens = r.integers(a, b + 1, size=B)
    elif kind == "loguniform":
        _, a, b = spec.lengths
        u = r.random(B)
        lens = np.clip(np.rint(a * (b / a) ** u), a, b).astype(np.int64)
    elif kind == "skew":
        _, long_len, a, b = spec.lengths
        lens = r.integers(a, b + 1, size=B)
        lens[0] = long_len
    else:
        raise ValueError(kind)
    return lens.astype(np.int32)


def make_block_table(spec: Spec, lens: np.ndarray, stride: int | None = None, spare_tokens: int = 0):
    """Returns (table [B][stride] int32 with -1 tails, num_pages).  `spare_tokens` allocates room
    for that many more tokens per sequence (pages a decode loop will append into)."""
    P = spec.page_size
    pages_per_seq = (lens.astype(np.int64) + spare_tokens + P - 1) // P
    total = int(pages_per_seq.sum())
    perm = np.arange(total, dtype=np.int64)
    if spec.permute_pages:
        perm = _rng(spec.seed, 2).permutation(total)
    width = max(1, int(pages_per_seq.max())) if stride is None else stride
    table = np.full((len(lens), width), -1, dtype=np.int32)
    at = 0
    for b, n in enumerate(pages_per_seq):
        table[b, :n] = perm[at:at + n]
        at += n
    return table, max(total, 1)


def _normal_bf16(shape, std, gen, device, chunk_elems=1 << 28):
    """bf16 tensor of N(0, std^2) values rounded to nearest-even, drawn chunk by chunk."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    n = flat.numel()
    for at in range(0, n, chunk_elems):
        m = min(chunk_elems, n - at)
        x = torch.randn(m, generator=gen, device=device, dtype=torch.float32)
        if std != 1.0:
            x *= std
        flat[at:at + m] = x.to(torch.bfloat16)
    return out


def make_workload(spec: Spec | str, device="cpu", table_stride: int | None = None,
                  spare_tokens: int = 0, value_seed: int | None = None) -> Workload:
    """`value_seed` (default: the spec's seed) seeds q, K and V only: workloads that differ in it alone
    share lengths and block table and hold different values -- the layers of one model."""
    if isinstance(spec, str):
        spec = SPECS[spec]
    device = torch.device(device)
    lens = make_lengths(spec)
    table, num_pages = make_block_table(spec, lens, table_stride, spare_tokens)
    Hq, Hkv, D, P = spec.num_q_heads, spec.num_kv_heads, spec.head_dim, spec.page_size

    def gen(stream):
        g = torch.Generator(device=device)
        g.manual_seed((spec.seed if value_seed is None else value_seed) * 1000 + stream)
        return g

    q = _normal_bf16((spec.batch, Hq, D), spec.q_std, gen(3), device)
    v = _normal_bf16((num_pages, Hkv, P, D), 1.0, gen(5), device)
    if spec.k_outlier_prob > 0.0:
        # outliers are per token position: the K rows of all KV heads of that slot are
        # scaled in fp32 before the rounding to bf16
        k = torch.empty((num_pages, Hkv, P, D), dtype=torch.bfloat16, device=device)
        gk, gm = gen(4), gen(6)
        step = max(1, (1 << 26) // (Hkv * P * D))
        for at in range(0, num_pages, step):
            m = min(step, num_pages - at)
            x = torch.randn((m, Hkv, P, D), generator=gk, device=device, dtype=torch.float32)
            hit = torch.rand((m, 1, P, 1), generator=gm, device=device) < spec.k_outlier_prob
            x = torch.where(hit, x * spec.k_outlier_scale, x)
            k[at:at + m] = x.to(torch.bfloat16)
    else:
        k = _normal_bf16((num_pages, Hkv, P, D), 1.0, gen(4), device)

    # poison the slots past each sequence's end: the rest of its last page and any spare pages
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16, device=device)
    for b, n in enumerate(lens):
        n = int(n)
        if n % P:
            page = int(table[b, (n - 1) // P])
            k[page, :, n % P:, :] = nan
            v[page, :, n % P:, :] = nan
        if spare_tokens:
            spare = torch.from_numpy(table[b, (n + P - 1) // P:(n + spare_tokens + P - 1) // P].astype(np.int64)).to(device)
            k[spare] = nan
            v[spare] = nan

    return Workload(
        spec=spec, q=q, k_pages=k, v_pages=v,
        block_table=torch.from_numpy(table).to(device),
        seq_lens=torch.from_numpy(lens).to(device),
        scale=float(np.float32(1.0) / np.sqrt(np.float32(D))),
        lens_host=lens, table_host=table)


def shard_kv_heads(w: Workload, rank: int, world: int) -> Workload:
    """Rank `rank`'s slice of a workload under tensor parallelism over the KV heads: KV heads
    [rank * Hkv / world, (rank + 1) * Hkv / world) of every page, and the query heads that attend to
    them.  Tables and lengths are shared by all ranks.  Slicing only (contiguous copies)."""
    s = w.spec
    assert s.num_kv_heads % world == 0 and 0 <= rank < world
    hkv = s.num_kv_heads // world
    hq = s.num_q_heads // world
    from dataclasses import replace
    spec = replace(s, name=f"{s.name}_kvshard{rank}of{world}", num_q_heads=hq, num_kv_heads=hkv)
    return Workload(spec=spec, q=w.q[:, rank * hq:(rank + 1) * hq].contiguous(),
                    k_pages=w.k_pages[:, rank * hkv:(rank + 1) * hkv].contiguous(),
                    v_pages=w.v_pages[:, rank * hkv:(rank + 1) * hkv].contiguous(),
                    block_table=w.block_table, seq_lens=w.seq_lens, scale=w.scale,
                    lens_host=w.lens_host, table_host=w.table_host)


def shard_context(w: Workload, rank: int, world: int) -> Workload:
    """Rank `rank`'s share of a workload when every sequence's tokens are spread over `world` ranks by
    range: sequence b's pages are cut into `world` runs of (nearly) equal page counts, the rank keeps run
    `rank` -- its table row holds those page ids, its length the tokens in them.  Pools and queries are the
    whole workload's (a real deployment holds only its own pages; the ids stay valid here).  Slicing only."""
    s = w.spec
    P = s.page_size
    assert 0 <= rank < world
    pages = (w.lens_host.astype(np.int64) + P - 1) // P
    lo = pages * rank // world
    hi = pages * (rank + 1) // world
    width = max(1, int((hi - lo).max()))
    table = np.full((s.batch, width), -1, dtype=np.int32)
    lens = np.zeros(s.batch, dtype=np.int32)
    for b in range(s.batch):
        n = int(hi[b] - lo[b])
        table[b, :n] = w.table_host[b, lo[b]:hi[b]]
        lens[b] = max(0, min(int(w.lens_host[b]), int(hi[b]) * P) - int(lo[b]) * P)
    from dataclasses import replace
    spec = replace(s, name=f"{s.name}_ctxshard{rank}of{world}", lengths=("list", [int(x) for x in lens]))
    dev = w.q.device
    return Workload(spec=spec, q=w.q, k_pages=w.k_pages, v_pages=w.v_pages,
                    block_table=torch.from_numpy(table).to(dev), seq_lens=torch.from_numpy(lens).to(dev),
                    scale=w.scale, lens_host=lens, table_host=table)


def tiny_spec(name, lens, page_size, seed, permute=True, **kw) -> Spec:
    """A small hand-sized workload with the given context lengths."""
    return Spec(name, len(lens), page_size, ("list", list(lens)), permute_pages=permute, seed=seed, **kw)


def gather_sequences(w: Workload, seqs) -> Workload:
    """A host-side copy of the given sequences only: their pages are renumbered
    0..n-1 in logical order.  Lets a CPU checker look at a few sequences of a
    workload whose pools are too large to copy whole."""
    seqs = list(seqs)
    P = w.spec.page_size
    lens = w.lens_host[seqs]
    pages_per_seq = (lens.astype(np.int64) + P - 1) // P
    phys = np.concatenate([w.table_host[b, :n] for b, n in zip(seqs, pages_per_seq)]).astype(np.int64) \
        if len(seqs) else np.zeros(0, np.int64)
    idx = torch.from_numpy(phys).to(w.k_pages.device)
    k = w.k_pages.index_select(0, idx).cpu()
    v = w.v_pages.index_select(0, idx).cpu()
    width = max(1, int(pages_per_seq.max())) if len(seqs) else 1
    table = np.full((len(seqs), width), -1, dtype=np.int32)
    at = 0
    for i, n in enumerate(pages_per_seq):
        table[i, :n] = np.arange(at, at + n)
        at += n
    sub = Spec(w.spec.name + "_subset", len(seqs), P, ("list", [int(x) for x in lens]),
               seed=w.spec.seed, num_q_heads=w.spec.num_q_heads, num_kv_heads=w.spec.num_kv_heads,
               head_dim=w.spec.head_dim)
    return Workload(spec=sub, q=w.q[seqs].cpu(), k_pages=k, v_pages=v,
                    block_table=torch.from_numpy(table), seq_lens=torch.from_numpy(lens.astype(np.int32)),
                    scale=w.scale, lens_host=lens.astype(np.int32), table_host=table)


@dataclass
class CascadeWorkload:
    """A workload whose sequences come in groups of siblings that share their first tokens'
    pages (the samples drawn for one prompt)."""
    w: Workload
    group_start: torch.Tensor      # [G + 1] int32
    prefix_lens: torch.Tensor      # [G] int32: tokens whose pages the group's sequences share
    group_start_host: np.ndarray = field(default=None)
    prefix_lens_host: np.ndarray = field(default=None)

    def logical_bytes(self) -> int:
        """Algorithmic bytes if every sequence read its whole context itself."""
        return self.w.algorithmic_bytes()

    def shared_bytes(self) -> int:
        """Algorithmic bytes when the shared pages of a group are counted once."""
        s = self.w.spec
        per_token = 2 * s.num_kv_heads * s.head_dim * 2
        saved = 0
        for i, pre in enumerate(self.prefix_lens_host):
            n = int(self.group_start_host[i + 1] - self.group_start_host[i])
            saved += (n - 1) * int(pre) * per_token
        return self.w.algorithmic_bytes() - saved


def make_cascade_workload(name, groups, page_size, seed, device="cpu", q_std=1.0,
                          num_q_heads=NUM_Q_HEADS, num_kv_heads=NUM_KV_HEADS) -> CascadeWorkload:
    """groups: list of (shared_tokens, [own_tokens of each sibling]).  `shared_tokens` must be a
    multiple of the page size (only whole pages can be shared physically).  Sequence lengths are
    shared + own; siblings point at the same physical pages for the shared part; all pages are
    shuffled in one seeded permutation; values are i.i.d. N(0,1) (q: N(0, q_std^2))."""
    P = page_size
    lens, gstart, pre = [], [0], []
    for shared, owns in groups:
        assert shared % P == 0 and len(owns) >= 1
        lens += [shared + int(o) for o in owns]
        gstart.append(len(lens))
        pre.append(shared)
    lens = np.asarray(lens, dtype=np.int32)
    spec = Spec(name, len(lens), P, ("list", [int(x) for x in lens]), seed=seed, q_std=q_std,
                num_q_heads=num_q_heads, num_kv_heads=num_kv_heads)
    # page allocation: shared pages once per group, then each sibling's own pages
    rows, total = [], 0
    for (shared, owns), b0 in zip(groups, gstart[:-1]):
        shared_pages = list(range(total, total + shared // P))
        total += shared // P
        for j, o in enumerate(owns):
            n_own = (shared + int(o) + P - 1) // P - shared // P
            rows.append(shared_pages + list(range(total, total + n_own)))
            total += n_own
    num_pages = max(total, 1)
    perm = _rng(seed, 2).permutation(num_pages)
    width = max(1, max(len(r) for r in rows))
    table = np.full((len(lens), width), -1, dtype=np.int32)
    for b, r in enumerate(rows):
        table[b, :len(r)] = perm[np.asarray(r, dtype=np.int64)] if r else []
    device = torch.device(device)

    def gen(stream):
        g = torch.Generator(device=device)
        g.manual_seed(seed * 1000 + stream)
        return g

    Hq, Hkv, D = spec.num_q_heads, spec.num_kv_heads, spec.head_dim
    q = _normal_bf16((spec.batch, Hq, D), q_std, gen(3), device)
    k = _normal_bf16((num_pages, Hkv, P, D), 1.0, gen(4), device)
    v = _normal_bf16((num_pages, Hkv, P, D), 1.0, gen(5), device)
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16, device=device)
    for b, n in enumerate(lens):
        n = int(n)
        if n % P:
            page = int(table[b, (n - 1) // P])
            k[page, :, n % P:, :] = nan
            v[page, :, n % P:, :] = nan
    w = Workload(spec=spec, q=q, k_pages=k, v_pages=v, block_table=torch.from_numpy(table).to(device),
                 seq_lens=torch.from_numpy(lens).to(device),
                 scale=float(np.float32(1.0) / np.sqrt(np.float32(D))), lens_host=lens, table_host=table)
    gs = np.asarray(gstart, dtype=np.int32)
    pl = np.asarray(pre, dtype=np.int32)
    return CascadeWorkload(w=w, group_start=torch.from_numpy(gs).to(device), prefix_lens=torch.from_numpy(pl).to(device),
                           group_start_host=gs, prefix_lens_host=pl)


# Shared-prefix decode workloads: (tasks, samples per task, shared prompt tokens, range of each
# sample's own tokens, page size, seed).  Shaped like the sampling of the paper's pipeline: one
# fixed prompt per task, 5 samples per task in synthesis and 10 in evaluation, traces of a few
# thousand tokens; the third is a long-prompt stress case for the prefix pass.
CASCADE_SPECS = {
    "casc_24x10_pre2048_p64": (24, 10, 2048, (256, 8192), 64, 73571),
    "casc_32x5_pre2048_p64": (32, 5, 2048, (256, 8192), 64, 73572),
    "casc_16x10_pre16384_p64": (16, 10, 16384, (1, 256), 64, 73573),
}


def cascade_groups(name: str):
    """[(shared tokens, [own tokens per sample])] of a named cascade workload."""
    tasks, samples, shared, (a, b), page_size, seed = CASCADE_SPECS[name]
    r = _rng(seed, 7)
    return [(shared, r.integers(a, b + 1, size=samples).tolist()) for _ in range(tasks)]


def make_named_cascade(name: str, device="cpu") -> CascadeWorkload:
    page_size, seed = CASCADE_SPECS[name][4], CASCADE_SPECS[name][5]
    return make_cascade_workload(name, cascade_groups(name), page_size, seed, device)


def cascade_prefix_bytes(cw: CascadeWorkload) -> int:
    """Bytes the prefix pass must read: K and V of every group's shared whole 64-token tiles
    (counted once per group) plus the sharing siblings' query rows per KV head."""
    s = cw.w.spec
    per_token = 2 * s.num_kv_heads * s.head_dim * 2
    total = 0
    for i, pre in enumerate(cw.prefix_lens_host):
        n = int(cw.group_start_host[i + 1] - cw.group_start_host[i])
        if n >= 2:
            total += (int(pre) // 64) * 64 * per_token + n * s.num_q_heads * s.head_dim * 2
    return total


@dataclass
class PrefillWorkload:
    """A paged cache plus, per sequence, the query rows of its last `q_lens[b]` cached tokens."""
    w: Workload                    # w.q is [total_q][Hq][D] here
    q_start: torch.Tensor          # [B + 1] int32
    q_start_host: np.ndarray = field(default=None)

    @property
    def total_q(self) -> int:
        return int(self.q_start_host[-1])

    def flops(self) -> int:
        """Multiply-adds x 2 of the causal products: every query row against the tokens it sees,
        for Q.K^T and for P.V."""
        s = self.w.spec
        total = 0
        for b in range(s.batch):
            n, ql = int(self.w.lens_host[b]), int(self.q_start_host[b + 1] - self.q_start_host[b])
            seen = ql * (n - ql) + ql * (ql + 1) // 2       # tokens visible to the ql query tokens together
            total += seen * s.num_q_heads * s.head_dim * 2 * 2
        return total


def make_prefill_workload(name, lens, q_lens, page_size, seed, device="cpu", num_q_heads=NUM_Q_HEADS,
                          q_std=1.0, num_kv_heads=NUM_KV_HEADS) -> PrefillWorkload:
    """Sequences of `lens` cached tokens whose last `q_lens` tokens are the query tokens
    (q_lens[b] <= lens[b]; q_lens == lens is the prefill of a whole prompt, smaller values a
    chunk of it).  Pools, tables and poisoning as in make_workload; q ~ N(0, q_std^2)."""
    spec = tiny_spec(name, [int(x) for x in lens], page_size, seed, num_q_heads=num_q_heads, q_std=q_std,
                     num_kv_heads=num_kv_heads)
    w = make_workload(spec, device)
    qs = np.zeros(len(lens) + 1, dtype=np.int32)
    qs[1:] = np.cumsum(np.asarray(q_lens, dtype=np.int64))
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(seed * 1000 + 9)
    w.q = _normal_bf16((max(int(qs[-1]), 1), num_q_heads, spec.head_dim), q_std, g, dev)[:int(qs[-1])]
    return PrefillWorkload(w=w, q_start=torch.from_numpy(qs).to(dev), q_start_host=qs)


def prefill_as_decode(pw: PrefillWorkload, tokens) -> Workload:
    """Host-side restatement of some query tokens of a prefill workload as a decode batch: query
    token t of sequence b becomes a 'sequence' with b's block-table row and length position + 1.
    (Index bookkeeping only: what is computed per row is then the plain decode definition.)"""
    w = pw.w
    tokens = [int(t) for t in tokens]
    rows, lens = [], []
    for t in tokens:
        b = int(np.searchsorted(pw.q_start_host, t, side="right") - 1)
        ql = int(pw.q_start_host[b + 1] - pw.q_start_host[b])
        pos = int(w.lens_host[b]) - ql + (t - int(pw.q_start_host[b]))
        rows.append(w.table_host[b]); lens.append(pos + 1)
    lens = np.asarray(lens, dtype=np.int32)
    table = np.stack(rows).astype(np.int32) if rows else np.zeros((0, w.table_host.shape[1]), np.int32)
    spec = Spec(w.spec.name + "_as_decode", len(lens), w.spec.page_size, ("list", [int(x) for x in lens]),
                seed=w.spec.seed, num_q_heads=w.spec.num_q_heads, num_kv_heads=w.spec.num_kv_heads)
    idx = torch.as_tensor(tokens, dtype=torch.long)
    return Workload(spec=spec, q=w.q.cpu()[idx], k_pages=w.k_pages.cpu(), v_pages=w.v_pages.cpu(),
                    block_table=torch.from_numpy(table), seq_lens=torch.from_numpy(lens), scale=w.scale,
                    lens_host=lens, table_host=table)


# Prefill workloads: (prompts, prompt tokens, query tokens per prompt, page size, seed).  The first is
# shaped like the paper's prompts (one fixed template around a task's program, one or two thousand
# tokens, prefilled whole); the others are longer prompts and a chunk at the end of a long context.
PREFILL_SPECS = {
    "prefill_16x2048_p64": (16, 2048, 2048, 64, 73581),
    "prefill_4x8192_p64": (4, 8192, 8192, 64, 73582),
    "prefill_2x32768_p64": (2, 32768, 32768, 64, 73583),
    "prefill_chunk_8x2048_of_16384_p64": (8, 16384, 2048, 64, 73584),
}


def make_named_prefill(name: str, device="cpu") -> PrefillWorkload:
    prompts, n, ql, page_size, seed = PREFILL_SPECS[name]
    return make_prefill_workload(name, [n] * prompts, [ql] * prompts, page_size, seed, device)
