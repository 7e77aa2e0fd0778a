"""The read-only streaming probe (the benchmark's second bandwidth denominator): its checksum is the XOR of the
buffer's 64-bit words, so the kernel provably reads every byte once."""
import numpy as np
import pytest
import torch

from paper_2010_04902_b200 import binding as bz

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("staged", [False, True])
@pytest.mark.parametrize("n_words", [0, 1, 2, 3, 1000, 1001, 4096, 4097, 148 * 8 * 256 * 8 * 2 + 5, 5_000_001])
def test_checksum_is_the_xor_of_all_words(n_words, staged):
    rng = np.random.default_rng(n_words)
    host = rng.integers(-2**63, 2**63 - 1, size=n_words, dtype=np.int64)
    buf = torch.from_numpy(host).cuda()
    want = int(np.bitwise_xor.reduce(host)) if n_words else 0
    got = int(bz.stream_probe(buf, staged=staged).cpu()[0])
    assert got == want
    # a second call into the same checksum word starts from zero again
    sink = torch.full((1,), 123, dtype=torch.int64, device="cuda")
    assert int(bz.stream_probe(buf, sink, staged=staged).cpu()[0]) == want


def test_argument_errors():
    buf = torch.zeros(16, dtype=torch.int64, device="cuda")
    sink = torch.zeros(1, dtype=torch.int64, device="cuda")
    st = bz.lib().bz_stream_probe(buf.data_ptr() + 8, 64, 0, sink.data_ptr(), None)
    assert st == bz.ERR_INVALID_ARG          # not 16-byte aligned
    st = bz.lib().bz_stream_probe(buf.data_ptr(), 60, 1, sink.data_ptr(), None)
    assert st == bz.ERR_INVALID_ARG          # not a multiple of 8 bytes
    assert bz.lib().bz_stream_probe(buf.data_ptr(), 64, 0, None, None) == bz.ERR_INVALID_ARG
