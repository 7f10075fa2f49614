"""GPU parity of the prompt-encoding calls (token-parallel causal attention over a cache slot,
cache writes, one whole iteration of the stack) against the float64 oracle."""
import numpy as np
import pytest
import torch

from oracle import lckv_oracle as orc
from paper_2405_10637_b200 import binding as lk
from paper_2405_10637_b200 import inputs as syn
from helpers import compare, NAN_BITS

pytestmark = pytest.mark.gpu


@pytest.fixture(params=["tc5", "mma"], autouse=True)
def prefill_kernel(request, monkeypatch):
    """Every test runs on both kernels of the operation: tcgen05 (the default) and mma.sync (the choice
    is read when a cache is created)."""
    if request.param == "tc5":
        monkeypatch.delenv("LCKV_PREFILL_KERNEL", raising=False)
    else:
        monkeypatch.setenv("LCKV_PREFILL_KERNEL", request.param)
    return request.param


def make_cache(L, w, Hq, Hkv, d, lens, T_cap, out_dtype=0, variant=0, seed=0, std=1.0, poison=True):
    B = len(lens)
    cfg = lk.make_config(L, w, Hq, Hkv, d, B, T_cap, out_dtype=out_dtype, top_variant=variant)
    cache = lk.Cache(cfg)
    hK, hV = [], []
    for s in range(cache.info.n_slots):
        kb = syn.bits(syn.randn_bf16((B, Hkv, T_cap, d), seed + 2 * s, std=std))
        vb = syn.bits(syn.randn_bf16((B, Hkv, T_cap, d), seed + 2 * s + 1, std=std))
        if poison:
            for b in range(B):
                kb[b, :, lens[b]:] = NAN_BITS
                vb[b, :, lens[b]:] = NAN_BITS
        kt, vt = cache.slot_tensors(s)
        kt.copy_(syn.from_bits(kb)); vt.copy_(syn.from_bits(vb))
        hK.append(kb); hV.append(vb)
    cache.lckv_cache_reset(list(lens))
    return cache, hK, hV


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 4, 4), (64, 8, 2)])
@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("out_dtype", [0, 1])
def test_prefill_attention_ragged(d, Hq, Hkv, mode, out_dtype):
    lens = [0, 1, 2, 63, 64, 65, 130, 200]
    n_max, T_cap = 203, 210
    cache, hK, hV = make_cache(2, 0, Hq, Hkv, d, lens, T_cap, out_dtype=out_dtype, seed=7 + d)
    q = syn.randn_bf16((len(lens), n_max, Hq, d), 99)
    sentinel = 12288.0   # exactly representable in bf16
    out = torch.full(q.shape, sentinel, dtype=cache.out_torch_dtype, device=cache.device)
    cache.lckv_prefill_attention(0, mode, q.to(cache.device), out=out)
    torch.cuda.synchronize()
    assert cache.lckv_cache_status() == 0
    want = orc.prefill_attention(syn.bits(q), hK[0], hV[0], np.array(lens, np.int32), mode, d ** -0.5)
    for b, nb in enumerate(lens):
        if nb:
            compare(out[b, :nb], want[b, :nb], f"seq {b}")
        assert (out[b, nb:].float() == sentinel).all(), "rows past the prompt must not be written"
    if out_dtype == 1:
        g = out.cpu().numpy().astype(np.float64)
        for b, nb in enumerate(lens):   # P is rounded to bf16 for the second product: ~1e-3 relative
            if nb > 1:
                err = np.linalg.norm(g[b, :nb] - want[b, :nb]) / np.linalg.norm(want[b, :nb])
                assert err < 3e-3, err
    cache.close()


def test_prefill_write_kv_bit_exact():
    lens = [5, 0, 64, 33]
    B, Hkv, d, n_max, T_cap = 4, 2, 64, 70, 80
    cache, hK, hV = make_cache(2, 0, 4, Hkv, d, lens, T_cap, seed=3, poison=False)
    k = syn.randn_bf16((B, n_max, Hkv, d), 1); v = syn.randn_bf16((B, n_max, Hkv, d), 2)
    cache.lckv_prefill_write_kv(0, k.to(cache.device), v.to(cache.device))
    orc.prefill_write_kv(hK[0], hV[0], syn.bits(k), syn.bits(v), np.array(lens, np.int32))
    kt, vt = cache.slot_tensors(0)
    assert np.array_equal(syn.bits(kt), hK[0]) and np.array_equal(syn.bits(vt), hV[0])
    assert cache.lckv_cache_lengths(B) == lens
    cache.close()


@pytest.mark.parametrize("w,variant", [(0, 0), (2, 0), (2, 1), (4, 0)])
def test_prefill_iterations_then_decode(w, variant):
    """Three iterations of the whole stack from zeroed caches, then one decode step: outputs within
    tolerance each time, caches and lengths bit-exact throughout."""
    L, Hq, Hkv, d = 4, 8, 2, 64
    lens = [100, 37, 64, 1]
    B, n_max, T_cap = 4, 100, 128
    cfg = lk.make_config(L, w, Hq, Hkv, d, B, T_cap, top_variant=variant)
    cache = lk.Cache(cfg)
    dev = cache.device
    plan = orc.plan(L, w, variant)
    ns = plan["n_slots"]
    hK = [np.zeros((B, Hkv, T_cap, d), np.uint16) for _ in range(ns)]
    hV = [np.zeros_like(hK[0]) for _ in range(ns)]
    for s in range(ns):
        kt, vt = cache.slot_tensors(s); kt.zero_(); vt.zero_()
    cache.lckv_cache_reset(lens)
    hl = np.array(lens, np.int32)
    for it in range(3):
        q = [syn.randn_bf16((B, n_max, Hq, d), 100 * it + l, std=0.5) for l in range(L)]
        k = [syn.randn_bf16((B, n_max, Hkv, d), 100 * it + 20 + l, std=0.5)
             if plan["write_slot"][l] >= 0 else None for l in range(L)]
        v = [syn.randn_bf16((B, n_max, Hkv, d), 100 * it + 40 + l, std=0.5)
             if plan["write_slot"][l] >= 0 else None for l in range(L)]
        outs = [torch.zeros((B, n_max, Hq, d), dtype=torch.bfloat16, device=dev) for _ in range(L)]
        cache.lckv_prefill_iteration([t.to(dev) for t in q], outs,
                                     [None if t is None else t.to(dev) for t in k],
                                     [None if t is None else t.to(dev) for t in v])
        torch.cuda.synchronize()
        want = orc.prefill_iteration(L, w, [syn.bits(t) for t in q],
                                     [None if t is None else syn.bits(t) for t in k],
                                     [None if t is None else syn.bits(t) for t in v],
                                     hK, hV, hl, d ** -0.5, top_variant=variant)
        for l in range(L):
            for b, nb in enumerate(lens):
                compare(outs[l][b, :nb], want[l][b, :nb], f"iteration {it} layer {l} seq {b}")
        for s in range(ns):
            kt, vt = cache.slot_tensors(s)
            assert np.array_equal(syn.bits(kt), hK[s]) and np.array_equal(syn.bits(vt), hV[s])
    # decoding continues from the encoded prompt
    q = [syn.randn_bf16((B, Hq, d), 900 + l, std=0.5) for l in range(L)]
    kv = [syn.randn_bf16((B, Hkv, d), 950 + l, std=0.5) if plan["write_slot"][l] >= 0 else None
          for l in range(L)]
    outs = [torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=dev) for _ in range(L)]
    dkv = [None if t is None else t.to(dev) for t in kv]
    cache.lckv_layer_stack_step([t.to(dev) for t in q], outs, dkv, dkv)
    torch.cuda.synchronize()
    bkv = [None if t is None else syn.bits(t) for t in kv]
    want, _ = orc.stack_step(L, w, [syn.bits(t) for t in q], bkv, bkv, hK, hV, hl, d ** -0.5,
                             top_variant=variant)
    for l in range(L):
        compare(outs[l], want[l], f"decode layer {l}")
    assert cache.lckv_cache_lengths(B) == hl.tolist() == [x + 1 for x in lens]
    cache.close()


def test_prefill_long_prompt_mha_d128():
    """A 7B-shaped head layout at a prompt of 1000 tokens (16 query blocks, 15 full KV tiles)."""
    lens = [1000, 777]
    cache, hK, hV = make_cache(2, 0, 8, 8, 128, lens, 1024, seed=11)
    q = syn.randn_bf16((2, 1000, 8, 128), 5)
    out = cache.lckv_prefill_attention(0, lk.MODE_CONDENSED, q.to(cache.device))
    torch.cuda.synchronize()
    want = orc.prefill_attention(syn.bits(q), hK[0], hV[0], np.array(lens, np.int32), 0, 128 ** -0.5)
    for b, nb in enumerate(lens):
        compare(out[b, :nb], want[b, :nb])
    cache.close()


def test_prefill_errors():
    cache, _, _ = make_cache(2, 0, 4, 4, 64, [10, 3], 16, poison=False)
    dev = cache.device
    q = torch.zeros((2, 8, 4, 64), dtype=torch.bfloat16, device=dev)   # n_max 8 < len 10
    with pytest.raises(lk.LckvError) as e:
        cache.lckv_prefill_attention(0, 0, q)
    assert e.value.status == lk.EINVAL
    q = torch.zeros((2, 10, 4, 64), dtype=torch.bfloat16, device=dev)
    with pytest.raises(lk.LckvError) as e:
        cache.lckv_prefill_attention(0, 3, q)
    assert e.value.status == lk.EINVAL
    with pytest.raises(lk.LckvError) as e:
        cache.lckv_prefill_attention(1, 0, q)
    assert e.value.status == lk.EINVAL
    cache.close()
    cfg = lk.make_config(2, 0, 4, 4, 64, 2, 16, stream_sink=4)
    c2 = lk.Cache(cfg)
    with pytest.raises(lk.LckvError) as e:
        c2.lckv_prefill_attention(0, 0, q)
    assert e.value.status == lk.EINVAL
    c2.close()


def test_prefill_on_paged_cache():
    """Prompt encoding over slots made of 64-row pages (scrambled page order)."""
    from helpers import Case
    lens = [130, 64, 1, 200, 65]
    c = Case(L=4, w=2, Hq=8, Hkv=2, d=64, lens=lens, T_cap=256, seed=17, std=0.5, page_rows=64, n_pages=14)
    dev, B, n_max = c.cache.device, len(lens), 200
    plan = c.plan
    for it in range(2):
        q = [syn.randn_bf16((B, n_max, c.Hq, c.d), 300 + 10 * it + l, std=0.5) for l in range(c.L)]
        k = [syn.randn_bf16((B, n_max, c.Hkv, c.d), 400 + 10 * it + l, std=0.5)
             if plan["write_slot"][l] >= 0 else None for l in range(c.L)]
        v = [syn.randn_bf16((B, n_max, c.Hkv, c.d), 500 + 10 * it + l, std=0.5)
             if plan["write_slot"][l] >= 0 else None for l in range(c.L)]
        outs = [torch.zeros((B, n_max, c.Hq, c.d), dtype=torch.bfloat16, device=dev) for _ in range(c.L)]
        c.cache.lckv_prefill_iteration([t.to(dev) for t in q], outs,
                                       [None if t is None else t.to(dev) for t in k],
                                       [None if t is None else t.to(dev) for t in v])
        torch.cuda.synchronize()
        assert c.cache.lckv_cache_status() == 0
        want = orc.prefill_iteration(c.L, c.w, [syn.bits(t) for t in q],
                                     [None if t is None else syn.bits(t) for t in k],
                                     [None if t is None else syn.bits(t) for t in v],
                                     c.hK, c.hV, c.lens, c.scale)
        for l in range(c.L):
            for b, nb in enumerate(lens):
                compare(outs[l][b, :nb], want[l][b, :nb], f"iteration {it} layer {l} seq {b}")
        c.check_state()
    c.step()   # and decoding continues on the same pages
    c.close()


@pytest.mark.parametrize("n", [4096, 8192])
def test_prefill_attention_at_the_timed_sizes(n):
    """The shape bench.py times (7B head layout, 8 prompts of n tokens, j < i mask), checked on whole
    query rows (all 32 heads) the oracle computes one by one: the first rows, rows around the 64- and
    128-row tile edges, the last rows of the last query blocks, and seeded random rows."""
    B, H, d = 8, 32, 128
    dev = torch.device("cuda:0")
    cfg = lk.make_config(2, 0, H, H, d, B, n)
    cache = lk.Cache(cfg, device=dev)
    kt, vt = cache.slot_tensors(0)
    syn.fill_randn_bf16_(kt, 1); syn.fill_randn_bf16_(vt, 2)
    cache.lckv_cache_reset([n] * B)
    q = syn.randn_bf16((B, n, H, d), 3, device=dev)
    out = cache.lckv_prefill_attention(0, lk.MODE_CONDENSED, q)
    torch.cuda.synchronize()
    assert cache.lckv_cache_status() == 0
    rng = np.random.default_rng(11)
    rows = [0, 1, 2, 63, 64, 65, 127, 128, 129, n // 2 - 1, n // 2, n - 130, n - 129, n - 128, n - 127,
            n - 65, n - 64, n - 63, n - 2, n - 1] + [int(x) for x in rng.integers(0, n, 12)]
    for b in (0, B - 1):
        hk, hv = syn.bits(kt[b:b + 1]), syn.bits(vt[b:b + 1])
        hq = syn.bits(q[b])
        for i in rows:
            want, _ = orc.decode_attention(hq[i:i + 1], hk, hv, np.array([i], np.int32), 0, d ** -0.5)
            compare(out[b, i], want[0], f"seq {b} row {i}")
    cache.close()
