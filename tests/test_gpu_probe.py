"""The read-only stream probe reads what it claims to read: its checksums equal sums computed by torch
over the same bytes (so the timed kernels cannot have skipped any part of the buffer)."""
import pytest
import torch

from paper_2405_10637_b200 import binding as lk

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("nbytes", [8192 * 5, 8192 * 3000 + 4096 + 48])
def test_probe_checksums(nbytes):
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev).manual_seed(7)
    words = torch.randint(-2 ** 31, 2 ** 31 - 1, ((nbytes + 3) // 4,), generator=g, device=dev, dtype=torch.int64)
    buf = words.to(torch.int32)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    for kind in (0, 2):                       # all 32-bit words of the whole 16- (32-) byte units
        unit = 16 if kind == 0 else 32
        n_words = nbytes // unit * unit // 4
        acc = torch.zeros(1, dtype=torch.int32, device=dev)
        lk.lckv_read_stream_probe(buf, nbytes, kind, acc, status, repeats=3)
        torch.cuda.synchronize()
        want = 3 * int(words[:n_words].sum().item()) & 0xFFFFFFFF
        assert int(acc.item()) & 0xFFFFFFFF == want, kind
    acc = torch.zeros(1, dtype=torch.int32, device=dev)
    lk.lckv_read_stream_probe(buf, nbytes, 1, acc, status, repeats=2, l2_keep=0.5)   # first word of every whole 8 KB piece
    torch.cuda.synchronize()
    want = 2 * int(words[:nbytes // 8192 * 2048:2048].sum().item()) & 0xFFFFFFFF
    assert int(acc.item()) & 0xFFFFFFFF == want
    assert int(status.item()) == 0


def test_probe_rejects_bad_arguments():
    dev = torch.device("cuda:0")
    t = torch.zeros(64, dtype=torch.int32, device=dev)
    f = lk.lib().lckv_read_stream_probe
    p = t.data_ptr()
    assert f(None, 256, 0, 1, 0.0, p, p, None) == lk.EINVAL
    assert f(p + 4, 128, 0, 1, 0.0, p, p, None) == lk.EINVAL
    assert f(p + 16, 128, 2, 1, 0.0, p, p, None) == lk.EINVAL
    assert f(p, 256, 3, 1, 0.0, p, p, None) == lk.EINVAL
    assert f(p, 8, 0, 1, 0.0, p, p, None) == lk.EINVAL
    assert f(p, 256, 0, 0, 0.0, p, p, None) == lk.EINVAL
    assert f(p, 256, 1, 1, 1.5, p, p, None) == lk.EINVAL
