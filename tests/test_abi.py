"""The C-ABI shared library: it loads without a GPU, exports every function that
include/*.h declares, and its host-only logic behaves."""
import ctypes
import re
from pathlib import Path

import pytest
import torch

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module")
def P():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_07356_b200 as pkg
    return pkg


def declared_functions():
    names = set()
    for header in sorted((ROOT / "include").glob("*.h")):
        text = re.sub(r"/\*.*?\*/", "", header.read_text(), flags=re.S)
        names |= set(re.findall(r"\b(concur_\w+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(P):
    names = declared_functions()
    assert "concur_attn_create" in names and "concur_decode_attn" in names and "concur_attn_destroy" in names
    raw = ctypes.CDLL(str(ROOT / "paper_2510_07356_b200" / "libconcur_attn.so"))
    for n in names:
        assert hasattr(raw, n), n
    assert sorted(P.binding.EXPORTS) == names


def test_workspace_bytes_and_config_checks(P):
    good = P.make_config(64, 256, 512)
    n = P.concur_attn_workspace_bytes(good)
    assert n > 2 * 4096 * 8 * 128 * 4 and n % 256 == 0
    bigger = P.concur_attn_workspace_bytes(P.make_config(64, 4096, 512))
    assert bigger > n
    assert P.concur_attn_workspace_bytes(P.make_config(64, 256, 512, num_q_heads=40)) == n      # group size 5
    assert P.concur_attn_workspace_bytes(P.make_config(64, 256, 512, num_q_heads=44)) == 0      # not a multiple of 8
    assert P.concur_attn_workspace_bytes(P.make_config(64, 256, 512, num_q_heads=72)) == 0
    assert P.concur_attn_workspace_bytes(P.make_config(48, 256, 512)) == 0
    assert P.concur_attn_workspace_bytes(P.make_config(64, 0, 512)) == 0


def test_strerror(P):
    assert P.concur_attn_strerror(0) == "ok"
    seen = {P.concur_attn_strerror(c) for c in range(-5, 1)}
    assert len(seen) == 6
    assert P.concur_attn_strerror(-99) == "unknown status"


def test_invalid_configs_are_rejected_before_any_cuda_call(P):
    B = P.binding
    for cfg, code in [
        (P.make_config(64, 256, 512, head_dim=64), B.CONCUR_ERR_UNSUPPORTED),
        (P.make_config(8, 256, 512), B.CONCUR_ERR_UNSUPPORTED),
        (P.make_config(64, 70000, 512), B.CONCUR_ERR_INVALID_ARG),
        (P.make_config(64, 65536, 1 << 20), B.CONCUR_ERR_TOO_LARGE),
    ]:
        with pytest.raises(B.ConcurError) as e:
            P.concur_attn_create(cfg)
        assert e.value.code == code
    assert P.concur_attn_destroy(None) == 0


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device error path")
def test_no_device_fails_loudly(P):
    with pytest.raises(P.binding.ConcurError) as e:
        P.concur_attn_create(P.make_config(64, 16, 64))
    assert e.value.code == P.binding.CONCUR_ERR_CUDA
    with pytest.raises(RuntimeError):
        P.DecodeAttention(64, 16, 64)
