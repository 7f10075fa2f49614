"""The allocation-free entry point against the regular one.

lckv_decode_attention_static serves callers that are not allowed to allocate device memory (an
engine that owns the whole GPU heap, a plugin that may not allocate after start-up, a latency path
that cannot afford cudaMalloc's synchronisation): its work plan, merge tickets and split-K partials
live in a fixed array inside the library instead of a caller-provided workspace.  It must give what
lckv_decode_attention gives on the same cache, and must keep doing so when called again, since every
call reuses the same scratch and finds the previous call's leftovers in it.

Collected last on purpose (file name), so a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

from paper_2405_10637_b200 import binding as lk
from paper_2405_10637_b200 import inputs as syn
from helpers import MAX_ABS, REL_L2

pytestmark = pytest.mark.gpu


def close_enough(got, ref, what):
    g, r = got.float().cpu().numpy().astype(np.float64), ref.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(g).all(), what
    assert np.abs(g - r).max() <= MAX_ABS, f"{what}: max-abs {np.abs(g - r).max():.3e}"
    assert np.linalg.norm(g - r) <= REL_L2 * np.linalg.norm(r), what


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 8, 8), (64, 8, 2)])
def test_static_entry_matches_cache_entry_twice_in_a_row(d, Hq, Hkv):
    B, T_cap = 6, 700
    lens = [0, 1, 16, 333, 699, 64]
    # kernel_kind = 1: the reference call runs the FP32-ALU kernel, the kernel the static entry point
    # wraps, so the two agree to rounding of the last bit (grouped heads would otherwise take the
    # tensor-core kernel, which rounds the probabilities to bf16)
    cfg = lk.make_config(2, 0, Hq, Hkv, d, B, T_cap, kernel_kind=1)
    cache = lk.Cache(cfg)
    dev = cache.device
    kt, vt = cache.slot_tensors(0)
    kt.copy_(syn.randn_bf16((B, Hkv, T_cap, d), 71)); vt.copy_(syn.randn_bf16((B, Hkv, T_cap, d), 72))
    cache.lckv_cache_reset(lens)
    lens_dev = torch.tensor(lens, dtype=torch.int32, device=dev)
    status = torch.full((1,), -1, dtype=torch.int32, device=dev)
    for call, (mode, seed) in enumerate([(lk.MODE_CONDENSED, 81), (lk.MODE_CONDENSED, 82)]):
        q = syn.randn_bf16((B, Hq, d), seed).to(dev)
        lse_ref = torch.empty((B, Hq), dtype=torch.float32, device=dev)
        ref = cache.lckv_decode_attention(0, mode, q, lse=lse_ref)
        out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=dev)
        lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=dev)
        lk.lckv_decode_attention_static(kt, vt, lens_dev, q, out, mode, lse=lse, dev_status=status)
        torch.cuda.synchronize()
        assert status.item() == 0
        close_enough(out, ref, f"call {call}")
        np.testing.assert_allclose(lse.cpu().numpy(), lse_ref.cpu().numpy(), atol=1e-5)
    # the cache-based path is unaffected by the static calls
    assert cache.lckv_cache_status() == 0
    cache.close()


def test_static_entry_rejects_sizes_beyond_its_scratch_and_bad_arguments():
    dev = torch.device("cuda:0")
    t = torch.zeros(16, dtype=torch.int32, device=dev)
    p = t.data_ptr()
    f = lk.lib().lckv_decode_attention_static
    assert f(p, p, p, p, p, None, None, 4097, 8, 8, 128, 64, 0, 0.0, 0, None) == lk.ESTATICLIMIT
    assert f(p, p, p, p, p, None, None, 4, 8, 8, 96, 64, 0, 0.0, 0, None) == lk.EINVAL
    assert f(p, p, p, p, p, None, None, 4, 8, 3, 128, 64, 0, 0.0, 0, None) == lk.EINVAL
    assert f(None, p, p, p, p, None, None, 4, 8, 8, 128, 64, 0, 0.0, 0, None) == lk.EINVAL
    assert f(p, p, p, p, p, None, None, 4, 8, 8, 128, 64, 2, 0.0, 0, None) == lk.EINVAL
    assert b"static scratch" in lk.lib().lckv_status_string(lk.ESTATICLIMIT)
