"""The benchmark's read-only stream probe (concur_bench_read_probe): its checksum proves that every 16-byte piece of the
buffer was read exactly once, whatever the grid size and the ragged tail."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2510_07356_b200 import bench_probe
    return bench_probe


@pytest.mark.parametrize("n16,ctas", [(0, 0), (1, 0), (7, 1), (512 * 8 - 1, 1), (512 * 8 * 3 + 5, 3), (1_000_003, 0),
                                      (4_194_304, 148), (3_000_017, 592)])
def test_checksum_is_the_xor_of_all_words(P, n16, ctas):
    g = torch.Generator(device="cuda:0").manual_seed(77 + n16 % 1000)
    buf = torch.randint(-2**31, 2**31 - 1, (max(1, n16) * 4,), dtype=torch.int32, device="cuda:0", generator=g)
    chk = torch.full((1,), 12345, dtype=torch.int32, device="cuda:0")
    P.read_probe(buf, n16 * 16, chk, ctas, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    words = buf[: n16 * 4].cpu().numpy().view(np.uint32)
    want = int(np.bitwise_xor.reduce(words)) if n16 else 0
    assert int(chk.cpu().numpy().view(np.uint32)[0]) == want


def test_argument_errors(P):
    buf = torch.zeros(64, dtype=torch.int32, device="cuda:0")
    chk = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    bad = P.ERR_INVALID_ARG
    assert P.read_probe(None, 16, chk, check=False) == bad
    assert P.read_probe(buf, 16, None, check=False) == bad
    assert P.read_probe(buf, 24, chk, check=False) == bad                       # not a multiple of 16
    assert P.read_probe(buf.data_ptr() + 4, 16, chk, check=False) == bad         # misaligned buffer
    assert P.read_probe(buf, 16, chk, ctas=-1, check=False) == bad
    assert P.read_probe(buf, 16, chk, ctas=70000, check=False) == bad
    torch.cuda.synchronize()
