"""Do the pins pin?  The closed forms and invariants that tests/test_oracle_pins.py holds the CPU oracle
to are run here, as one battery, against a small numpy restatement of the operation into which
plausible mistakes are planted one at a time (on the CPU, in this file only): a dropped scale, the
wrong q-head -> KV-head map, a sign, an index, a missing normalisation, slots past the sequence end.
Every planted mistake must fail at least one pin; the unplanted restatement and the real oracle must
pass all of them.  (Nothing here touches the CUDA path.)"""
import math

import numpy as np
import pytest
import torch

import oracle


def bf16(x):
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def val(bits):
    return torch.from_numpy(np.asarray(bits).view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()


MISTAKES = ("scale_dropped", "head_map_modulo", "lse_without_max", "table_ignored", "page_slot_swapped",
            "not_normalised", "v_for_k", "one_token_short", "reads_past_the_end", "sign_of_exponent",
            "scale_squared", "k_of_other_head")


def attn_np(qb, kb, vb, table, lens, scale, mistake=None):
    """softmax(scale q K^T) V over a paged cache, restated in numpy (fp64), with one optional mistake."""
    q, K, V = val(qb), val(kb), val(vb)
    B, Hq, D = q.shape
    _, Hkv, P, _ = K.shape
    G = Hq // Hkv
    sc = float(np.float32(scale))
    out = np.zeros((B, Hq, D)); lse = np.full((B, Hq), -np.inf)
    for b in range(B):
        n = int(lens[b])
        if mistake == "one_token_short":
            n = max(n - 1, 0)
        if mistake == "reads_past_the_end" and n > 0:
            n = -(-n // P) * P
        if n == 0:
            continue
        for h in range(Hq):
            g = h % Hkv if mistake == "head_map_modulo" else h // G
            gk = (g + 1) % Hkv if mistake == "k_of_other_head" else g
            ks, vs = [], []
            for j in range(n):
                page, slot = j // P, j % P
                if mistake == "page_slot_swapped":
                    page, slot = j % max(1, -(-n // P)), (j // max(1, -(-n // P))) % P
                phys = page if mistake == "table_ignored" else int(table[b][page])
                ks.append((V if mistake == "v_for_k" else K)[phys, gk, slot])
                vs.append(V[phys, g, slot])
            ks, vs = np.array(ks), np.array(vs)
            s = (ks @ q[b, h]) * (1.0 if mistake == "scale_dropped" else sc * sc if mistake == "scale_squared" else sc)
            m = s.max()
            w = np.exp(m - s) if mistake == "sign_of_exponent" else np.exp(s - m)
            l = w.sum()
            out[b, h] = (w @ vs) if mistake == "not_normalised" else (w @ vs) / l
            lse[b, h] = math.log(l) if mistake == "lse_without_max" else m + math.log(l)
    return out, lse


def paged(q, k, v, P, Hkv, perm=None, poison=False):
    """One sequence.  q [Hq][D]; k, v [n][Hkv][D].  Pages in the order `perm` (physical id of logical page)."""
    q, k, v = (np.asarray(a, dtype=np.float32) for a in (q, k, v))
    n, _, D = k.shape
    pages = max(1, -(-n // P))
    perm = np.arange(pages) if perm is None else np.asarray(perm)
    fill = np.nan if poison else 0.0
    kp = np.full((pages, Hkv, P, D), fill, dtype=np.float32); vp = np.full_like(kp, fill)
    for j in range(n):
        kp[perm[j // P], :, j % P] = k[j]; vp[perm[j // P], :, j % P] = v[j]
    return bf16(q[None]), bf16(kp), bf16(vp), perm.astype(np.int32)[None, :], np.array([n], dtype=np.int32)


def close(a, b, tol=1e-9):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return a.shape == b.shape and bool(np.all(np.isfinite(a) == np.isfinite(b))) and \
        bool(np.all(np.abs(a - b)[np.isfinite(b)] <= tol * (1.0 + np.abs(b[np.isfinite(b)]))))


def battery(impl):
    """Runs the pins against impl(qb, kb, vb, table, lens, scale) -> (out, lse); returns the names of those that fail."""
    failed = []
    rng = np.random.default_rng(7)

    def check(name, ok):
        if not ok:
            failed.append(name)

    # 1. one cached token: out is that V row, lse = scale q.k
    D = 16
    q = rng.standard_normal((4, D)); k = rng.standard_normal((1, 2, D)); v = rng.standard_normal((1, 2, D))
    a = paged(q, k, v, 4, 2)
    out, lse = impl(*a, 0.3)
    dots = [float(np.float32(0.3)) * float(val(a[0][0, h]) @ val(a[1][0, h // 2, 0])) for h in range(4)]
    check("single token", close(out[0], [val(a[2][0, h // 2, 0]) for h in range(4)]) and close(lse[0], dots))
    # 2. two tokens with scores (0, ln 3): weights 1/4, 3/4
    q = np.zeros((1, 4)); q[0, 1] = 1.0
    k = np.zeros((2, 1, 4)); k[1, 0, 1] = 1.0
    v = np.zeros((2, 1, 4)); v[0, 0] = [1, 0, 2, -4]; v[1, 0] = [0, 1, 2, 4]
    out, lse = impl(*paged(q, k, v, 2, 1), math.log(3.0))
    check("quarter / three quarters", close(out[0, 0], [0.25, 0.75, 2.0, 2.0], 1e-6) and close(lse[0, 0], math.log(4.0), 1e-6))
    # 3. geometric series: s_j = scale j, v_j = j
    n, scale = 100, 0.0625
    k = np.zeros((n, 1, 8)); k[:, 0, 0] = np.arange(n)
    v = np.tile(np.arange(n, dtype=np.float64)[:, None, None], (1, 1, 8))
    q = np.zeros((1, 8)); q[0, 0] = 1.0
    out, lse = impl(*paged(q, k, v, 16, 1), scale)
    r = math.exp(scale); z = (r ** n - 1) / (r - 1)
    num = r * (1 - n * r ** (n - 1) + (n - 1) * r ** n) / (1 - r) ** 2
    check("geometric series", close(out[0, 0], np.full(8, num / z), 1e-9) and close(lse[0, 0], math.log(z), 1e-9))
    # 4. equal K rows: out = mean of V, lse = s + ln n (n not a multiple of the page size; unused slots hold NaN)
    n = 37
    krow = rng.standard_normal(8); v = rng.standard_normal((n, 1, 8)); q = rng.standard_normal((1, 8))
    a = paged(q, np.tile(krow, (n, 1, 1)), v, 8, 1, poison=True)
    out, lse = impl(*a, 0.25)
    vv = np.array([val(a[2][j // 8, 0, j % 8]) for j in range(n)])
    s = float(np.float32(0.25)) * float(val(a[0][0, 0]) @ val(a[1][0, 0, 0]))
    check("equal scores", close(out[0, 0], vv.mean(axis=0)) and close(lse[0, 0], s + math.log(n)))
    # 5. which KV head a query head reads: V of head g is the constant g, K differs per head
    Hq, Hkv, n = 8, 4, 9
    k = rng.standard_normal((n, Hkv, 8)); v = np.tile(np.arange(Hkv, dtype=np.float64)[None, :, None], (n, 1, 8))
    out, lse = impl(*paged(rng.standard_normal((Hq, 8)), k, v, 4, Hkv), 0.5)
    check("head map (V)", close(out[0], np.repeat(np.arange(Hkv), Hq // Hkv)[:, None] * np.ones((1, 8))))
    # 6. the same, seen through K: q = e0, head g's keys are (j == g) e0 * 4, values one-hot of the token
    n = Hkv
    k = np.zeros((n, Hkv, 8)); v = np.zeros((n, Hkv, 8))
    for g in range(Hkv):
        k[g, g, 0] = 4.0
    for j in range(n):
        v[j, :, j] = 1.0
    q = np.zeros((Hq, 8)); q[:, 0] = 1.0
    out, _ = impl(*paged(q, k, v, 2, Hkv), 1.0)
    check("head map (K)", all(int(np.argmax(out[0, h])) == h // (Hq // Hkv) for h in range(Hq)))
    # 7. shuffled pages with the table updated: nothing changes
    n, P = 45, 4
    q = rng.standard_normal((2, 8)); k = rng.standard_normal((n, 1, 8)); v = rng.standard_normal((n, 1, 8))
    o0, l0 = impl(*paged(q, k, v, P, 1), 0.35)
    perm = rng.permutation(-(-n // P))
    o1, l1 = impl(*paged(q, k, v, P, 1, perm=perm), 0.35)
    check("page permutation", close(o0, o1, 1e-12) and close(l0, l1, 1e-12))
    # 8. token order does not matter (pages of 1 token, tokens permuted)
    tp = rng.permutation(n)
    o2, l2 = impl(*paged(q, k[tp], v[tp], 1, 1), 0.35)
    check("token permutation", close(o0, o2, 1e-9) and close(l0, l2, 1e-9))
    # 9. adding c to every score (k += c e, q.e = 1) shifts lse by scale c and leaves out alone
    q = np.zeros((1, 8)); q[0, 0] = 1.0; q[0, 1:] = rng.standard_normal(7)
    k = rng.standard_normal((20, 1, 8)); k[:, 0, 0] = np.round(k[:, 0, 0] * 8) / 8
    v = rng.standard_normal((20, 1, 8))
    k2 = k.copy(); k2[:, 0, 0] += 2.0
    oa, la = impl(*paged(q, k, v, 4, 1), 0.5)
    ob, lb = impl(*paged(q, k2, v, 4, 1), 0.5)
    check("score shift", close(oa, ob, 1e-9) and close(lb[0, 0] - la[0, 0], 1.0, 1e-9))
    # 10. out lies between the smallest and the largest value, and an empty sequence gives (0, -inf)
    lo, hi = val(bf16(v)).min(axis=(0, 1)), val(bf16(v)).max(axis=(0, 1))
    check("convexity", bool(np.all(oa[0, 0] >= lo - 1e-12) and np.all(oa[0, 0] <= hi + 1e-12)))
    a = paged(q, k[:0], v[:0], 4, 1)
    oe, le = impl(a[0], a[1], a[2], a[3], np.array([0], dtype=np.int32), 0.5)
    check("empty sequence", bool(np.all(oe == 0.0)) and bool(np.isneginf(le).all()))
    return failed


def test_the_restatement_without_a_mistake_passes_every_pin():
    assert battery(attn_np) == []


def test_the_oracle_passes_every_pin():
    assert battery(lambda *a: oracle.decode_attn(*a)) == []


@pytest.mark.parametrize("mistake", MISTAKES)
def test_every_planted_mistake_fails_some_pin(mistake):
    failed = battery(lambda *a: attn_np(*a, mistake=mistake))
    assert failed, f"no pin notices '{mistake}'"
