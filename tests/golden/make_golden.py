"""Writes tests/golden/tiny_decode_oracle.json from the CPU oracle alone (never from the CUDA
path).  The paper (arXiv 2510.07356) prints no worked attention example, so this fixture is
not a pin of the oracle against the paper: it freezes the oracle's output on one seeded tiny
workload so that any later change to the oracle's arithmetic or to the input generator shows
up as a diff.  Run from the repository root:  python tests/golden/make_golden.py
"""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import synth  # noqa: E402

LENS = (5, 70, 0, 16)
PAGE = 16
SEED = 2510


def compute():
    w = synth.make_workload(synth.tiny_spec("golden", LENS, PAGE, SEED), "cpu")
    out, lse = oracle.decode_attn(w.q, w.k_pages, w.v_pages, w.block_table, w.seq_lens, w.scale)
    return w, out, lse


if __name__ == "__main__":
    w, out, lse = compute()
    doc = {
        "source": "oracle/attn_oracle.c on synth.tiny_spec('golden', (5, 70, 0, 16), 16, 2510), cpu generator",
        "scale": w.scale,
        "q_first_bits": w.q.view(-1)[:8].view(dtype=__import__("torch").int16).tolist(),
        "lse": [[repr(float(x)) for x in row] for row in lse],
        "out_first4": [[[repr(float(x)) for x in out[b, h, :4]] for h in range(0, 64, 8)] for b in range(len(LENS))],
    }
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_decode_oracle.json")
    with open(path, "w") as f:
        json.dump(doc, f, indent=0)
    print("wrote", path)
