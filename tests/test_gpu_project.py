"""GPU parity of the fused key/value producer (lckv_project_append_kv) against the oracle: produced
rows within one bf16 rounding of the float64 values, every other cache byte untouched, indices
(ring rows, pages, lengths) exact, and the rows usable by the decode attention that follows."""
import numpy as np
import pytest
import torch

from oracle import lckv_oracle as orc
from paper_2405_10637_b200 import binding as lk
from paper_2405_10637_b200 import inputs as syn

from helpers import Case, compare

pytestmark = pytest.mark.gpu


def f64(bits_arr):
    return (np.asarray(bits_arr).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rope_tables(n_pos, d, base=10000.0):
    i = np.arange(d // 2, dtype=np.float64)
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * base ** (-2.0 * i / d)[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def check_rows(got_bits, want_f64, want_bits, what):
    """A produced row: fp32 tensor-core accumulation, then one rounding to bf16.  It must lie within
    half a bf16 unit (2^-9 relative, written 2^-8 to cover a binade edge) of the float64 value plus the
    accumulation error, and agree bit for bit with the oracle's own rounding almost everywhere."""
    g = f64(got_bits)
    assert np.isfinite(g).all(), what
    err = np.abs(g - want_f64)
    tol = np.abs(want_f64) * 2.0 ** -8 + 1e-5 * (1.0 + np.abs(want_f64))
    assert (err <= tol).all(), f"{what}: worst excess {(err - tol).max():.3e}"
    same = (np.asarray(got_bits) == np.asarray(want_bits)).mean()
    assert same >= 0.98, f"{what}: only {same:.4f} of the elements round like the oracle"


def set_row(c, pool, b, row, bits_hd):
    """Overwrite logical row `row` of sequence b ([H_kv, d] bits) in a contiguous or paged slot tensor."""
    src = syn.from_bits(bits_hd).to(pool.device)
    if c.page_rows:
        pt = c.cache.lckv_cache_page_table()
        pool[int(pt[b, row // c.page_rows]), :, row % c.page_rows] = src
    else:
        pool[b, :, row] = src


def produce(c, slot, d_model, rope, seed, advance=1):
    """One produce-and-append call on Case c, checked against the oracle; c.lens advances with it."""
    B, Hkv, d = c.B, c.Hkv, c.d
    F = Hkv * d
    x = syn.randn_bf16((B, d_model), seed)
    wk = syn.randn_bf16((F, d_model), seed + 1, std=d_model ** -0.5)
    wv = syn.randn_bf16((F, d_model), seed + 2, std=d_model ** -0.5)
    cos = sin = cos_d = sin_d = None
    dev = c.cache.device
    if rope:
        cos, sin = rope_tables(int(c.lens.max()) + 2, d)
        cos_d, sin_d = torch.from_numpy(cos).to(dev), torch.from_numpy(sin).to(dev)
    c.cache.lckv_project_append_kv(slot, x.to(dev), wk.to(dev), wv.to(dev), cos_d, sin_d,
                                   advance_len=advance)
    torch.cuda.synchronize()
    assert c.cache.lckv_cache_status() == 0
    kb, vb, kf, vf = orc.project_kv(syn.bits(x), syn.bits(wk), syn.bits(wv), c.lens, Hkv, d, cos, sin)
    # rows the call must have written, from the oracle's append rule
    before_k, before_v = c.hK[slot].copy(), c.hV[slot].copy()
    orc.append(c.hK[slot], c.hV[slot], kb, vb, c.lens, n_sink=c.stream_sink)
    kt, vt = c.cache.slot_tensors(slot)
    for b in range(B):
        t = int(c.lens[b])
        row = t if (c.stream_sink == 0 or t < c.T_cap) else \
            c.stream_sink + (t - c.stream_sink) % (c.T_cap - c.stream_sink)
        if c.page_rows:
            gk, gv = c._gather(kt, b), c._gather(vt, b)
        else:
            gk, gv = syn.bits(kt[b]), syn.bits(vt[b])
        check_rows(gk[:, row], kf[b], kb[b], f"K seq {b}")
        check_rows(gv[:, row], vf[b], vb[b], f"V seq {b}")
        # everything else the sequence holds is untouched, bit for bit (rows of owned pages past the
        # new row were never defined)
        n = min(gk.shape[1], c.T_cap)
        keep = np.ones(n, bool)
        keep[row] = False
        if c.page_rows:
            keep[row + 1:] = False
        assert np.array_equal(gk[:, :n][:, keep], before_k[b][:, :n][:, keep]), f"K seq {b}: other rows changed"
        assert np.array_equal(gv[:, :n][:, keep], before_v[b][:, :n][:, keep]), f"V seq {b}: other rows changed"
        # The two sides may round an element of the new row differently (checked above to be within
        # one unit); give the GPU cache the oracle's bits so that later calls start from equal caches.
        set_row(c, kt, b, row, kb[b])
        set_row(c, vt, b, row, vb[b])
    if advance:
        c.lens += 1
    assert c.cache.lckv_cache_lengths(B) == c.lens.tolist()


def attend_and_compare(c, slot, seed):
    """Condensed attention over the slot (it now includes the produced row) on both sides."""
    q = syn.randn_bf16((c.B, c.Hq, c.d), seed)
    out = c.cache.lckv_decode_attention(slot, lk.MODE_CONDENSED, q.to(c.cache.device))
    torch.cuda.synchronize()
    want, _ = orc.decode_attention(syn.bits(q), c.hK[slot], c.hV[slot], c.lens, 0, c.scale,
                                   n_sink=c.stream_sink)
    compare(out, want, "attention over produced rows")


@pytest.mark.parametrize("rope", [False, True])
@pytest.mark.parametrize("B", [1, 5, 16, 17, 40, 130, 300])
@pytest.mark.parametrize("shape", ["d64", "d128"])
def test_produced_rows_match_oracle(shape, B, rope):
    kw = {"d64": dict(Hq=4, Hkv=4, d=64), "d128": dict(Hq=2, Hkv=2, d=128)}[shape]
    d_model = {"d64": 256, "d128": 192}[shape]
    T_cap = 24
    lens = syn.ragged_lengths(B, 0, T_cap - 3, 77 + B).numpy()
    lens[0] = 0
    c = Case(L=2, w=0, lens=lens, T_cap=T_cap, seed=5, poison=False, **kw)
    produce(c, 0, d_model, rope, seed=900 + B)
    attend_and_compare(c, 0, seed=31)
    produce(c, 0, d_model, rope, seed=1900 + B)      # a second token: positions moved on
    attend_and_compare(c, 0, seed=32)
    c.close()


@pytest.mark.parametrize("rope", [False, True])
@pytest.mark.parametrize("B", [3, 40, 300])
@pytest.mark.parametrize("shape", ["d64_split4", "d128_split2", "d128_split8"])
def test_hidden_width_split_over_a_cluster(shape, B, rope):
    """Hidden widths with enough k-steps that the launch shares a tile among 2, 4 or 8 CTAs (their
    partial tiles are added through distributed shared memory before the rows are stored)."""
    kw = {"d64_split4": dict(Hq=4, Hkv=4, d=64), "d128_split2": dict(Hq=2, Hkv=2, d=128),
          "d128_split8": dict(Hq=1, Hkv=1, d=128)}[shape]
    d_model = {"d64_split4": 1024, "d128_split2": 512, "d128_split8": 2048}[shape]
    T_cap = 12
    lens = syn.ragged_lengths(B, 0, T_cap - 2, 177 + B).numpy()
    c = Case(L=2, w=0, lens=lens, T_cap=T_cap, seed=9, poison=False, **kw)
    produce(c, 0, d_model, rope, seed=2900 + B)
    attend_and_compare(c, 0, seed=33)
    c.close()


def test_produce_into_warmup_slot_without_advancing():
    """A warmup layer's own cache (slot 1), lengths left alone (the step's other layers follow)."""
    lens = [3, 0, 9, 1]
    c = Case(L=4, w=2, Hq=4, Hkv=2, d=64, lens=lens, T_cap=16, seed=6, poison=False)
    produce(c, 1, 128, True, seed=50, advance=0)
    assert c.cache.lckv_cache_lengths(4) == lens
    c.close()


def test_ring_rows_of_a_streaming_cache():
    """Sink + window cache: tokens past the capacity land on ring rows; rotation uses the token's
    true position, not the row."""
    lens = [2, 15, 16, 17, 40, 29]
    c = Case(L=2, w=0, Hq=2, Hkv=2, d=64, lens=lens, T_cap=16, seed=7, poison=False, stream_sink=4)
    for i in range(3):
        produce(c, 0, 128, True, seed=60 + 10 * i)
        attend_and_compare(c, 0, seed=70 + i)
    c.close()


def test_paged_slot_takes_new_pages():
    lens = [0, 63, 64, 65, 127, 128, 5]
    c = Case(L=2, w=0, Hq=2, Hkv=2, d=64, lens=lens, T_cap=200, seed=8, page_rows=64, n_pages=24)
    for i in range(2):
        produce(c, 0, 128, i == 1, seed=80 + 10 * i)
        attend_and_compare(c, 0, seed=90 + i)
    pt = c.cache.lckv_cache_page_table()
    assert [int((pt[b] >= 0).sum()) for b in range(len(lens))] == [(n + 2 + 63) // 64 for n in lens]
    c.close()


def test_argument_errors_change_nothing():
    B, Hkv, d, dm = 4, 2, 64, 128
    cfg = lk.make_config(2, 0, 2, Hkv, d, B, 8)
    cache = lk.Cache(cfg)
    dev = cache.device
    cache.lckv_cache_reset([1, 2, 3, 7])
    x = torch.zeros((B, dm), dtype=torch.bfloat16, device=dev)
    w = torch.zeros((Hkv * d, dm), dtype=torch.bfloat16, device=dev)
    cos = torch.ones((8, d // 2), dtype=torch.float32, device=dev)
    kt, _ = cache.slot_tensors(0)
    before = syn.bits(kt).copy()

    def expect(status, *args, **kwargs):
        with pytest.raises(lk.LckvError) as e:
            cache.lckv_project_append_kv(*args, **kwargs)
        assert e.value.status == status

    expect(lk.EINVAL, 0, x[:, :100].contiguous(), w[:, :100].contiguous(), w[:, :100].contiguous())  # d_model % 64
    expect(lk.EINVAL, 1, x, w, w)                                   # no such slot
    expect(lk.EINVAL, 0, x, w, w, cos, None)                        # one table without the other
    expect(lk.EINVAL, 0, x, w, w, cos[:7], cos[:7])                 # position 7 needs 8 table rows
    expect(lk.EINVAL, 0, x.view(-1)[4:4 + 2 * dm].view(2, dm), w, w)  # 8-byte aligned only
    cache.lckv_cache_reset([1, 2, 3, 8])
    expect(lk.ECAPACITY, 0, x, w, w)                                # sequence 3 is full
    torch.cuda.synchronize()
    assert np.array_equal(syn.bits(kt), before)
    assert cache.lckv_cache_lengths(B) == [1, 2, 3, 8]
    cache.close()
    # feature count not a multiple of 128: refused
    cache = lk.Cache(lk.make_config(2, 0, 1, 1, 64, 2, 8))
    cache.lckv_cache_reset([0, 0])
    with pytest.raises(lk.LckvError) as e:
        cache.lckv_project_append_kv(0, x[:2], w[:64], w[:64])
    assert e.value.status == lk.EINVAL
    cache.close()


def test_llama7b_width_sampled_sequences():
    """The 7B layer width (32 heads x 128, d_model 4096) at B = 512 (two batch tiles of 256); the
    oracle recomputes a sample of the sequences one by one."""
    B, Hkv, d, dm, T_cap = 512, 32, 128, 4096, 8
    cfg = lk.make_config(2, 0, Hkv, Hkv, d, B, T_cap)
    cache = lk.Cache(cfg)
    dev = cache.device
    lens = syn.ragged_lengths(B, 0, T_cap - 1, 4242).numpy()
    cache.lckv_cache_reset(lens.tolist())
    kt, vt = cache.slot_tensors(0)
    kt.zero_(); vt.zero_()
    x = syn.randn_bf16((B, dm), 1)
    wk = syn.randn_bf16((Hkv * d, dm), 2, std=dm ** -0.5)
    wv = syn.randn_bf16((Hkv * d, dm), 3, std=dm ** -0.5)
    cos, sin = rope_tables(T_cap, d)
    cache.lckv_project_append_kv(0, x.to(dev), wk.to(dev), wv.to(dev), torch.from_numpy(cos).to(dev),
                                 torch.from_numpy(sin).to(dev), advance_len=1)
    torch.cuda.synchronize()
    assert cache.lckv_cache_status() == 0
    assert cache.lckv_cache_lengths(B) == (lens + 1).tolist()
    sample = np.array([0, 1, 255, 256, 257, 300, 510, 511])
    kb, vb, kf, vf = orc.project_kv(syn.bits(x)[sample], syn.bits(wk), syn.bits(wv), lens[sample], Hkv, d,
                                    cos, sin)
    for i, b in enumerate(sample):
        check_rows(syn.bits(kt[b, :, lens[b]]), kf[i], kb[i], f"K seq {b}")
        check_rows(syn.bits(vt[b, :, lens[b]]), vf[i], vb[i], f"V seq {b}")
    # exactly one row per (sequence, head) was written
    nz = (kt != 0).any(dim=-1).sum().item()
    assert nz == B * Hkv
    cache.close()
