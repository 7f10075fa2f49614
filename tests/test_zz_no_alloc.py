"""The allocation-free entry point against the regular one and against the oracle.

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

from oracle import lckv_oracle as orc
from paper_2405_10637_b200 import binding as lk
from paper_2405_10637_b200 import inputs as syn
from helpers import MAX_ABS, REL_L2, compare

pytestmark = pytest.mark.gpu


def close_enough(got, ref, what):
    g, r = got.float().cpu().numpy().astype(np.float64), ref.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(g).all(), what
    assert np.abs(g - r).max() <= MAX_ABS, f"{what}: max-abs {np.abs(g - r).max():.3e}"
    assert np.linalg.norm(g - r) <= REL_L2 * np.linalg.norm(r), what


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 8, 8), (64, 8, 2)])
def test_static_entry_matches_cache_entry_and_oracle_on_calls_in_a_row(d, Hq, Hkv):
    """Four calls one after another on the same scratch: condensed mask, standard mask (row len[b] is
    this token's own), fp32 outputs, and a call that leaves the status word to the library."""
    B, T_cap = 6, 700
    lens = [0, 1, 16, 333, 699, 64]
    # kernel_kind = 1: the cache-based call runs the FP32-ALU kernel, the kernel the static entry point
    # wraps, so the two agree to rounding of the last bit (grouped heads would otherwise take the
    # tensor-core kernel, which rounds the probabilities to bf16)
    caches = {odt: lk.Cache(lk.make_config(2, 0, Hq, Hkv, d, B, T_cap, kernel_kind=1, out_dtype=odt))
              for odt in (0, 1)}
    dev = caches[0].device
    kt, vt = caches[0].slot_tensors(0)
    kt.copy_(syn.randn_bf16((B, Hkv, T_cap, d), 71)); vt.copy_(syn.randn_bf16((B, Hkv, T_cap, d), 72))
    for c in caches.values():
        c.slot_tensors(0)[0].copy_(kt); c.slot_tensors(0)[1].copy_(vt)
        c.lckv_cache_reset(lens)
    kb, vb = syn.bits(kt), syn.bits(vt)
    lens_dev = torch.tensor(lens, dtype=torch.int32, device=dev)
    status = torch.full((1,), -1, dtype=torch.int32, device=dev)
    calls = [(lk.MODE_CONDENSED, 81, 0, True), (lk.MODE_STANDARD, 82, 0, True),
             (lk.MODE_CONDENSED, 83, 1, True), (lk.MODE_STANDARD, 84, 0, False)]
    for call, (mode, seed, odt, with_status) in enumerate(calls):
        q = syn.randn_bf16((B, Hq, d), seed).to(dev)
        tdt = torch.float32 if odt else torch.bfloat16
        lse_ref = torch.empty((B, Hq), dtype=torch.float32, device=dev)
        ref = caches[odt].lckv_decode_attention(0, mode, q, lse=lse_ref)
        out = torch.full((B, Hq, d), float("nan"), dtype=tdt, device=dev)
        lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=dev)
        status.fill_(-1)
        lk.lckv_decode_attention_static(kt, vt, lens_dev, q, out, mode, lse=lse,
                                        dev_status=status if with_status else None)
        torch.cuda.synchronize()
        if with_status:
            assert status.item() == 0
        close_enough(out, ref, f"call {call}")
        np.testing.assert_allclose(lse.cpu().numpy(), lse_ref.cpu().numpy(), atol=1e-5)
        want, want_lse = orc.decode_attention(syn.bits(q.cpu()), kb, vb, np.asarray(lens, np.int32), mode, d ** -0.5)
        compare(out, want, f"call {call} against the oracle")
        np.testing.assert_allclose(lse.cpu().numpy(), want_lse, atol=2e-3)
    # the cache-based path is unaffected by the static calls
    for c in caches.values():
        assert c.lckv_cache_status() == 0
        c.close()


def test_static_entry_one_long_sequence_split_over_every_worker():
    """One 16 384-token sequence with 4 heads: each (sequence, head) pair is cut into hundreds of parts (far
    more than the 24 above which the cache-based path merges in two levels); the static entry point has no
    room for the second level's tickets and merges them in one pass.  Twice in a row."""
    B, Hq, Hkv, d, T = 1, 4, 4, 128, 16384
    cache = lk.Cache(lk.make_config(2, 0, Hq, Hkv, d, B, T, kernel_kind=1))
    dev = cache.device
    kt, vt = cache.slot_tensors(0)
    kt.copy_(syn.randn_bf16((B, Hkv, T, d), 91)); vt.copy_(syn.randn_bf16((B, Hkv, T, d), 92))
    cache.lckv_cache_reset([T - 1])
    assert min(T // cache.info.rows_per_tile, cache.info.n_workers // Hq) > 24   # parts per pair
    lens_dev = torch.tensor([T - 1], dtype=torch.int32, device=dev)
    kb, vb = syn.bits(kt), syn.bits(vt)
    for call, mode in enumerate([lk.MODE_CONDENSED, lk.MODE_STANDARD]):
        q = syn.randn_bf16((B, Hq, d), 93 + call).to(dev)
        ref = cache.lckv_decode_attention(0, mode, q)
        out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=dev)
        lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=dev)
        lk.lckv_decode_attention_static(kt, vt, lens_dev, q, out, mode, lse=lse)
        torch.cuda.synchronize()
        close_enough(out, ref, f"call {call}")
        want, want_lse = orc.decode_attention(syn.bits(q.cpu()), kb, vb, np.asarray([T - 1], np.int32), mode, d ** -0.5)
        compare(out, want, f"call {call} against the oracle")
        np.testing.assert_allclose(lse.cpu().numpy(), want_lse, atol=2e-3)
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
    assert f(p + 4, p, p, p, p, None, None, 4, 8, 8, 128, 64, 0, 0.0, 0, None) == lk.EINVAL
    assert b"static scratch" in lk.lib().lckv_status_string(lk.ESTATICLIMIT)
