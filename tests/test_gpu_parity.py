"""GPU parity: the CUDA library (through its C ABI) against the float64 oracle, element by element
on the same seeded bf16 inputs.  Tolerances: max-abs 1e-2, relative L2 5e-3 (bf16 inputs and
outputs, fp32 arithmetic); lengths, append positions and every cache byte bit-exact."""
import numpy as np
import pytest
import torch

from oracle import lckv_oracle as orc
from paper_2405_10637_b200 import binding as lk
from paper_2405_10637_b200 import inputs as syn
from helpers import Case, compare, NAN_BITS

pytestmark = pytest.mark.gpu


def test_toy_config_w0_all_layers_read_shared_cache():
    """4 layers, MHA 4 heads, d_h 64, w = 0, batch 2, 128 cached tokens, everything from seed 0 in
    the order K, V, q, k_new, v_new."""
    L, H, d, B, T = 4, 4, 64, 2, 128
    K, V, *rest = syn.draw_sequence([(B, H, T + 1, d)] * 2 + [(B, H, d)] * L + [(B, H, d)] * 2, 0)
    q, (kn, vn) = rest[:L], rest[L:]
    cfg = lk.make_config(L, 0, H, H, d, B, T + 1)
    cache = lk.Cache(cfg)
    kt, vt = cache.slot_tensors(0)
    kt.copy_(K); vt.copy_(V)
    cache.lckv_cache_reset([T] * B)
    dev = cache.device
    outs = [torch.empty((B, H, d), dtype=torch.bfloat16, device=dev) for _ in range(L)]
    cache.lckv_layer_stack_step([t.to(dev) for t in q], outs, [None] * (L - 1) + [kn.to(dev)],
                                [None] * (L - 1) + [vn.to(dev)])
    torch.cuda.synchronize()
    hK, hV = syn.bits(K), syn.bits(V)
    lens = np.full(B, T, np.int32)
    want, _ = orc.stack_step(L, 0, [syn.bits(t) for t in q], [None] * (L - 1) + [syn.bits(kn)],
                             [None] * (L - 1) + [syn.bits(vn)], [hK], [hV], lens, d ** -0.5)
    for l in range(L):
        compare(outs[l], want[l], f"layer {l}")
    assert cache.lckv_cache_lengths(B) == [T + 1] * B
    kt, vt = cache.slot_tensors(0)
    assert np.array_equal(syn.bits(kt), hK) and np.array_equal(syn.bits(vt), hV)
    cache.close()


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("variant", [0, 1])
def test_small_ragged_stack_with_edge_lengths(d, variant):
    """Lengths around the tile edges (0, 1, R-1, R, R+1, ...), T_cap not a multiple of the tile,
    NaN poison beyond every length, w = 2 sandwich, three consecutive steps."""
    lens = [0, 1, 15, 16, 17, 31, 32, 33, 63, 64, 65, 100, 257, 300]
    c = Case(L=5, w=2, Hq=4, Hkv=4, d=d, lens=lens, T_cap=303, variant=variant, seed=77 + d)
    for _ in range(3):
        c.step()
    c.close()


@pytest.mark.parametrize("w", [0, 2, 4])
def test_many_pairs_per_worker(w):
    """More tiles than workers: whole (sequence, head) pairs inside one worker's range are written
    directly, pairs cut by a range boundary go through the partial merge."""
    lens = syn.ragged_lengths(96, 40, 400, 5).tolist()
    c = Case(L=4, w=w, Hq=16, Hkv=16, d=128, lens=lens, T_cap=402, seed=900 + w)
    c.step(); c.step()
    c.close()


def test_w_equals_L_standard_transformer():
    c = Case(L=3, w=3, Hq=8, Hkv=8, d=128, lens=[5, 0, 77, 130], T_cap=140, seed=31)
    c.step(); c.step()
    c.close()


def test_gqa_group_of_8_and_of_2():
    """Grouped heads: q head h reads kv head h // g."""
    c = Case(L=4, w=2, Hq=32, Hkv=4, d=64, lens=[3, 64, 200, 511], T_cap=520, seed=8, std=0.125)
    c.step(); c.step()
    c.close()
    c = Case(L=3, w=0, Hq=8, Hkv=4, d=128, lens=[1, 90, 33], T_cap=100, seed=9)
    c.step()
    c.close()


def test_fp32_outputs_are_tight():
    """With fp32 outputs only the arithmetic differs: errors two orders below the bf16 bound."""
    c = Case(L=3, w=2, Hq=8, Hkv=8, d=128, lens=[9, 500, 1000, 17], T_cap=1024, out_dtype=1, seed=5)
    _, _, stats = c.step()
    assert max(s[0] for s in stats) < 2e-5 and max(s[1] for s in stats) < 2e-5
    c.close()


def test_single_long_sequence_split_over_many_workers():
    """One sequence, one head: every worker holds a slice of the same pair (deepest merge)."""
    c = Case(L=2, w=0, Hq=1, Hkv=1, d=128, lens=[40000], T_cap=40010, seed=3, out_dtype=1)
    c.step()
    c.close()


@pytest.mark.parametrize("d,H", [(128, 2), (64, 3)])
def test_few_pairs_split_over_many_workers_two_level_merge(d, H):
    """Multi-head attention with very few (sequence, head) pairs and long sequences: a pair is split
    over hundreds of workers and its parts are merged in two levels; results repeat bit for bit."""
    lens = [30000, 4100]
    c = Case(L=2, w=0, Hq=H, Hkv=H, d=d, lens=lens, T_cap=30010, seed=177 + d, std=0.25, poison=False)
    assert c.cache.info.kernel_kind == 1
    c.step(); c.step()
    q = syn.randn_bf16((2, H, d), 9, std=0.25).to(c.cache.device)
    a = c.cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q).clone()
    b = c.cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    c.close()


def test_decode_attention_entry_lse_and_single_key_exactness():
    """Per-layer entry point: log-sum-exp output; one visible key gives o = v_0 bit-exactly."""
    B, H, d, T = 3, 4, 128, 50
    cfg = lk.make_config(2, 0, H, H, d, B, T)
    cache = lk.Cache(cfg)
    K = syn.randn_bf16((B, H, T, d), 1); V = syn.randn_bf16((B, H, T, d), 2)
    kt, vt = cache.slot_tensors(0); kt.copy_(K); vt.copy_(V)
    lens = [1, 0, 37]
    cache.lckv_cache_reset(lens)
    q = syn.randn_bf16((B, H, d), 3)
    lse = torch.full((B, H), float("nan"), device=cache.device)
    out = cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q.to(cache.device), lse=lse)
    torch.cuda.synchronize()
    want, want_lse = orc.decode_attention(syn.bits(q), syn.bits(K), syn.bits(V),
                                          np.array(lens, np.int32), 0, d ** -0.5)
    compare(out, want)
    np.testing.assert_allclose(lse.cpu().numpy(), want_lse, atol=2e-3)
    assert np.array_equal(syn.bits(out[0]), syn.bits(V[0, :, 0]))      # len 1: o = v_0 exactly
    assert not out[1].float().abs().sum().item() and not lse[1].abs().sum().item()  # len 0
    # standard mode needs row len appended first (without advancing)
    kn = syn.randn_bf16((B, H, d), 4); vn = syn.randn_bf16((B, H, d), 5)
    cache.lckv_append_kv(0, kn.to(cache.device), vn.to(cache.device), advance_len=0)
    out1 = cache.lckv_decode_attention(0, lk.MODE_STANDARD, q.to(cache.device))
    hK, hV = syn.bits(K), syn.bits(V)
    orc.append(hK, hV, syn.bits(kn), syn.bits(vn), np.array(lens, np.int32))
    want1, _ = orc.decode_attention(syn.bits(q), hK, hV, np.array(lens, np.int32), 1, d ** -0.5)
    compare(out1, want1)
    assert cache.lckv_cache_lengths(B) == lens
    cache.close()


def test_errors_capacity_and_arguments():
    B, H, d, T = 2, 2, 64, 8
    cfg = lk.make_config(2, 0, H, H, d, B, T)
    cache = lk.Cache(cfg)
    cache.lckv_cache_reset([8, 3])          # sequence 0 is full
    dev = cache.device
    q = torch.zeros((B, H, d), dtype=torch.bfloat16, device=dev)
    kt0 = syn.bits(cache.slot_tensors(0)[0]).copy()
    with pytest.raises(lk.LckvError) as e:
        cache.lckv_layer_stack_step([q, q], [q.clone(), q.clone()], [None, q], [None, q])
    assert e.value.status == lk.ECAPACITY
    with pytest.raises(lk.LckvError) as e:
        cache.lckv_append_kv(0, q, q)
    assert e.value.status == lk.ECAPACITY
    assert cache.lckv_cache_lengths(B) == [8, 3]
    assert np.array_equal(syn.bits(cache.slot_tensors(0)[0]), kt0)
    cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q)   # reading a full cache is fine
    for bad in [dict(slot=1, mode=0), dict(slot=0, mode=2), dict(slot=-1, mode=0)]:
        with pytest.raises(lk.LckvError) as e:
            cache.lckv_decode_attention(bad["slot"], bad["mode"], q)
        assert e.value.status == lk.EINVAL
    with pytest.raises(lk.LckvError) as e:
        cache.lckv_cache_reset([9, 0])
    assert e.value.status == lk.ECAPACITY
    with pytest.raises(lk.LckvError) as e:
        cache.lckv_layer_stack_step([q, q], [q, q], [None, None], [None, None])  # top k,v missing
    assert e.value.status == lk.EINVAL
    with pytest.raises(lk.LckvError) as e:
        cache.lckv_decode_attention(0, 0, q, batch=3)
    assert e.value.status == lk.EINVAL
    cache.close()


def test_host_buffer_entry_point_matches():
    c = Case(L=4, w=2, Hq=8, Hkv=8, d=128, lens=[5, 100, 33], T_cap=120, seed=61, host_staging=1)
    c.step(host=True); c.step(host=True)
    c.step(host=True, contiguous=True); c.step(host=True, contiguous=True)   # single pitched copies
    c.close()
    # q bytes per layer not a multiple of the staging pitch (256): pitched copy with padding
    c = Case(L=3, w=2, Hq=3, Hkv=3, d=64, lens=[5, 9, 33], T_cap=40, seed=62, host_staging=1)
    c.step(host=True, contiguous=True); c.step(host=True)
    c.close()


def test_host_buffer_steps_queued_back_to_back():
    """More layers than copy chunks, mixed with device-buffer steps, and two host-buffer steps queued
    without a synchronisation in between (the second step's input copies must not overtake the first
    step's kernels, which still read the staging area)."""
    c = Case(L=12, w=2, Hq=4, Hkv=2, d=64, lens=[7, 0, 130, 64], T_cap=160, seed=63, host_staging=1)
    c.step(host=True)
    c.step()
    c.step(host=True, contiguous=True)
    odt = torch.float32 if c.cfg.out_dtype else torch.bfloat16
    queued = []
    for _ in range(2):
        q, kn, vn = c.step_inputs()
        c.step_no += 1
        qd = [t.pin_memory() for t in q]
        knd = [None if t is None else t.pin_memory() for t in kn]
        vnd = [None if t is None else t.pin_memory() for t in vn]
        outs = [torch.empty((c.B, c.Hq, c.d), dtype=odt).pin_memory() for _ in range(c.L)]
        c.cache.lckv_layer_stack_step_host(qd, outs, knd, vnd)
        queued.append((q, kn, vn, outs, (qd, knd, vnd)))
    torch.cuda.synchronize()
    assert c.cache.lckv_cache_status() == 0
    for q, kn, vn, outs, _ in queued:
        want, _ = orc.stack_step(c.L, c.w, [syn.bits(t) for t in q],
                                 [None if t is None else syn.bits(t) for t in kn],
                                 [None if t is None else syn.bits(t) for t in vn],
                                 c.hK, c.hV, c.lens, c.scale, top_variant=c.variant)
        for l in range(c.L):
            compare(outs[l], want[l], f"queued host step, layer {l}")
    c.check_state()
    c.close()


def test_repeatable_bitwise():
    """Same inputs twice: identical bits (the merge order is fixed, not arrival order)."""
    outs = []
    for _ in range(2):
        c = Case(L=2, w=0, Hq=4, Hkv=4, d=128, lens=[3000, 700, 1234], T_cap=3001, seed=12)
        o, _, _ = c.step()
        outs.append([syn.bits(t) for t in o])
        c.close()
    for a, b in zip(*outs):
        assert np.array_equal(a, b)


# ---- tensor-core kernel (grouped query heads) ------------------------------------------------------

@pytest.mark.parametrize("d,Hq,Hkv", [(64, 32, 4), (128, 16, 2), (64, 32, 2), (128, 8, 1)])
def test_mma_kernel_edge_lengths(d, Hq, Hkv):
    lens = [0, 1, 15, 16, 17, 31, 32, 33, 47, 48, 49, 64, 100, 257, 300]
    c = Case(L=4, w=2, Hq=Hq, Hkv=Hkv, d=d, lens=lens, T_cap=303, seed=500 + d + Hq, std=0.5)
    assert c.cache.info.kernel_kind == 2
    for _ in range(3):
        c.step()
    c.close()


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 8, 4), (128, 12, 4), (64, 16, 4), (128, 6, 1), (64, 14, 2)])
@pytest.mark.parametrize("out_dtype", [0, 1])
def test_mma_kernel_groups_smaller_than_8(d, Hq, Hkv, out_dtype):
    """Query groups of 2, 3, 4, 6 and 7 use the tensor-core kernel with the unused columns of the
    N = 8 tile zero: K and V are read once per group; only the real heads are written."""
    lens = [0, 1, 15, 16, 17, 33, 64, 100, 257, 300]
    c = Case(L=4, w=2, Hq=Hq, Hkv=Hkv, d=d, lens=lens, T_cap=303, seed=700 + d + Hq, std=0.5,
             out_dtype=out_dtype)
    assert c.cache.info.kernel_kind == 2
    for _ in range(2):
        c.step()
    # lse of the real heads through the single-call entry
    q = syn.randn_bf16((c.B, Hq, d), 5, std=0.5)
    lse = torch.full((c.B, Hq), float("nan"), dtype=torch.float32, device=c.cache.device)
    out = c.cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q.to(c.cache.device), lse=lse)
    torch.cuda.synchronize()
    want, want_lse = orc.decode_attention(syn.bits(q), c.hK[0], c.hV[0], c.lens, 0, c.scale)
    compare(out, want, "small group, single call")
    assert np.abs(lse.cpu().numpy() - want_lse).max() < 2e-3
    c.close()


def test_mma_kernel_many_pairs_per_worker_and_fp32_out():
    lens = syn.ragged_lengths(200, 100, 900, 6).tolist()
    c = Case(L=3, w=2, Hq=32, Hkv=4, d=64, lens=lens, T_cap=910, seed=41, std=0.125, out_dtype=1)
    _, _, stats = c.step()
    # P is rounded to bf16 for the second MMA: errors stay far below the bf16-output bound
    assert max(s[1] for s in stats) < 2e-3
    c.step()
    c.close()


def test_mma_kernel_single_long_pair():
    c = Case(L=2, w=0, Hq=8, Hkv=1, d=64, lens=[50000], T_cap=50010, seed=4, std=0.125)
    c.step()
    c.close()


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 16, 2), (64, 8, 2), (128, 8, 1)])
def test_mma_kernel_few_pairs_split_over_many_workers(d, Hq, Hkv):
    """Few (sequence, kv head) pairs and long sequences: a pair is split over tens to hundreds of
    workers and its parts are merged in two levels (chunks of contributors, then chunk results)."""
    lens = [30000, 4100, 123]
    c = Case(L=2, w=0, Hq=Hq, Hkv=Hkv, d=d, lens=lens, T_cap=30010, seed=77 + d, std=0.25, poison=False)
    assert c.cache.info.kernel_kind == 2
    c.step(); c.step()
    # twice the same call: the merge order is fixed, so the results repeat bit for bit
    q = syn.randn_bf16((3, Hq, d), 9, std=0.25).to(c.cache.device)
    a = c.cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q).clone()
    b = c.cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    c.close()


def test_tinyllama_shape_stack():
    """22 layers, 32 q heads, 4 kv heads, d_h 64, w = 2, values scaled by 1/sqrt(d_h) (rel-L2 binds)."""
    lens = [512, 513, 1024, 1535, 700, 511, 33, 1200]
    c = Case(L=22, w=2, Hq=32, Hkv=4, d=64, lens=lens, T_cap=1540, seed=2, std=0.125)
    c.step(); c.step()
    c.close()


def test_alu_kernel_forced_for_grouped_heads():
    c = Case(L=3, w=2, Hq=16, Hkv=2, d=64, lens=[3, 64, 200, 511], T_cap=520, seed=8, std=0.125,
             kernel_kind=1)
    assert c.cache.info.kernel_kind == 1
    c.step()
    c.close()


@pytest.mark.parametrize("shape", ["mha", "gqa"])
def test_graph_replay_steps_match(shape):
    """use_graph = 1: the step is captured once and replayed while the argument pointers repeat;
    lengths live on the device, so every replay sees the grown caches."""
    kw = dict(Hq=8, Hkv=8, d=128, std=1.0) if shape == "mha" else dict(Hq=16, Hkv=2, d=64, std=0.25)
    torch.cuda.set_stream(torch.cuda.Stream())   # the legacy default stream cannot be captured
    c = Case(L=5, w=2, lens=[0, 3, 16, 200, 333], T_cap=400, seed=77, use_graph=1, **kw)
    dev = c.cache.device
    odt = torch.bfloat16
    # fixed device buffers, new contents each step -> same pointers -> replay
    q = [torch.empty((c.B, c.Hq, c.d), dtype=torch.bfloat16, device=dev) for _ in range(c.L)]
    kn = [torch.empty((c.B, c.Hkv, c.d), dtype=torch.bfloat16, device=dev)
          if c.plan["write_slot"][l] >= 0 else None for l in range(c.L)]
    vn = [None if t is None else torch.empty_like(t) for t in kn]
    outs = [torch.empty((c.B, c.Hq, c.d), dtype=odt, device=dev) for _ in range(c.L)]
    for step in range(4):
        hq, hk, hv = c.step_inputs()
        for l in range(c.L):
            q[l].copy_(hq[l])
            if kn[l] is not None:
                kn[l].copy_(hk[l]); vn[l].copy_(hv[l])
        c.cache.lckv_layer_stack_step(q, outs, kn, vn)
        torch.cuda.synchronize()
        want, _ = orc.stack_step(c.L, c.w, [syn.bits(t) for t in hq],
                                 [None if t is None else syn.bits(t) for t in hk],
                                 [None if t is None else syn.bits(t) for t in hv],
                                 c.hK, c.hV, c.lens, c.scale)
        c.step_no += 1
        for l in range(c.L):
            compare(outs[l], want[l], f"graph step {step} layer {l}")
        c.check_state()
    c.close()
    torch.cuda.synchronize()
    torch.cuda.set_stream(torch.cuda.default_stream())


@pytest.mark.parametrize("shape", ["mha", "gqa"])
def test_same_case_at_several_split_counts(shape):
    """The worker limit moves the cut points of a launch's tile sequence: with all workers most pairs
    are whole or cut in two, with 37 or 5 workers the long sequences are cut differently and the short
    ones share a worker, with 1 nothing is split at all.  Every setting must meet the oracle (the
    split-K merge is exact up to rounding whatever the partition), also through a captured step."""
    kw = dict(Hq=8, Hkv=8, d=128, std=1.0) if shape == "mha" else dict(Hq=16, Hkv=2, d=64, std=0.25)
    torch.cuda.set_stream(torch.cuda.Stream())
    c = Case(L=4, w=2, lens=[0, 1, 70, 700, 3000, 129, 64, 2047], T_cap=3100, seed=123, use_graph=1, **kw)
    n_all = c.cache.info.n_workers
    with pytest.raises(lk.LckvError):
        c.cache.lckv_cache_set_worker_limit(n_all + 1)
    for limit in (0, 37, 5, 1, n_all // 2 + 1, 0):
        c.cache.lckv_cache_set_worker_limit(limit)
        c.step()
    c.close()
    torch.cuda.synchronize()
    torch.cuda.set_stream(torch.cuda.default_stream())


def test_graph_replay_with_alternating_buffer_sets():
    """use_graph = 1 with a caller that rotates through several sets of buffers (more sets than the
    library remembers captured steps for): every step, whether replayed or captured anew, matches."""
    torch.cuda.set_stream(torch.cuda.Stream())
    c = Case(L=4, w=2, Hq=8, Hkv=8, d=128, lens=[1, 40, 257], T_cap=300, seed=79, use_graph=1)
    dev = c.cache.device
    n_sets = 6
    sets = []
    for _ in range(n_sets):
        q = [torch.empty((c.B, c.Hq, c.d), dtype=torch.bfloat16, device=dev) for _ in range(c.L)]
        kn = [torch.empty((c.B, c.Hkv, c.d), dtype=torch.bfloat16, device=dev)
              if c.plan["write_slot"][l] >= 0 else None for l in range(c.L)]
        vn = [None if t is None else torch.empty_like(t) for t in kn]
        outs = [torch.empty((c.B, c.Hq, c.d), dtype=torch.bfloat16, device=dev) for _ in range(c.L)]
        sets.append((q, kn, vn, outs))
    order = [0, 1, 0, 1, 2, 3, 4, 5, 0, 5, 1, 1]
    for step, i in enumerate(order):
        q, kn, vn, outs = sets[i]
        hq, hk, hv = c.step_inputs()
        for l in range(c.L):
            q[l].copy_(hq[l])
            if kn[l] is not None:
                kn[l].copy_(hk[l]); vn[l].copy_(hv[l])
        c.cache.lckv_layer_stack_step(q, outs, kn, vn)
        torch.cuda.synchronize()
        want, _ = orc.stack_step(c.L, c.w, [syn.bits(t) for t in hq],
                                 [None if t is None else syn.bits(t) for t in hk],
                                 [None if t is None else syn.bits(t) for t in hv],
                                 c.hK, c.hV, c.lens, c.scale)
        c.step_no += 1
        for l in range(c.L):
            compare(outs[l], want[l], f"step {step} set {i} layer {l}")
        c.check_state()
    c.close()
    torch.cuda.synchronize()
    torch.cuda.set_stream(torch.cuda.default_stream())


@pytest.mark.parametrize("shape", ["mha", "gqa"])
def test_streaming_sink_and_window_cache(shape):
    """StreamingLLM-style caches (4 sinks + recent window): decode across the point where the ring
    wraps, some sequences already far past the capacity; outputs, ring rows and lengths exact."""
    kw = dict(Hq=4, Hkv=4, d=128, std=1.0) if shape == "mha" else dict(Hq=16, Hkv=2, d=64, std=0.25)
    T_cap = 37
    c = Case(L=4, w=2, lens=[0, 30, 35, 36, 37, 38, 100, 5000], T_cap=T_cap, seed=91, stream_sink=4, **kw)
    for _ in range(8):
        c.step()
    assert c.lens.tolist() == [8, 38, 43, 44, 45, 46, 108, 5008]
    c.close()


# ---- properties that hold at any size ---------------------------------------------------------------

def _attn_case(Hq, Hkv, d, lens, T_cap, out_dtype=1, seed=0, std=1.0):
    B = len(lens)
    cfg = lk.make_config(2, 0, Hq, Hkv, d, B, T_cap, out_dtype=out_dtype)
    cache = lk.Cache(cfg)
    K = syn.randn_bf16((B, Hkv, T_cap, d), seed + 1, std=std)
    V = syn.randn_bf16((B, Hkv, T_cap, d), seed + 2, std=std)
    kt, vt = cache.slot_tensors(0); kt.copy_(K); vt.copy_(V)
    cache.lckv_cache_reset(lens)
    q = syn.randn_bf16((B, Hq, d), seed + 3, std=std).to(cache.device)
    return cache, K, V, q


@pytest.mark.parametrize("Hq,Hkv,d", [(8, 8, 128), (16, 2, 64)])
def test_rows_at_and_beyond_the_new_token_are_never_read(Hq, Hkv, d):
    """Diagonal mask: poisoning row t (the position of the new token) and everything after it
    leaves every condensed output bit-identical."""
    lens = [0, 7, 16, 100, 255]
    cache, K, V, q = _attn_case(Hq, Hkv, d, lens, 256, out_dtype=0, seed=10)
    a = cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q).clone()
    kt, vt = cache.slot_tensors(0)
    for b, n in enumerate(lens):
        kt[b, :, n:] = float("nan"); vt[b, :, n:] = float("nan")
    bb = cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q)
    torch.cuda.synchronize()
    assert np.array_equal(syn.bits(a), syn.bits(bb))
    cache.close()


@pytest.mark.parametrize("Hq,Hkv,d", [(8, 8, 128), (16, 2, 64)])
def test_joint_permutation_of_cached_rows(Hq, Hkv, d):
    """Attention does not depend on the order of the visible rows (only on the set)."""
    lens = [33, 200, 999]
    cache, K, V, q = _attn_case(Hq, Hkv, d, lens, 1000, seed=20, std=0.5)
    a = cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q).clone()
    kt, vt = cache.slot_tensors(0)
    g = torch.Generator().manual_seed(1)
    for b, n in enumerate(lens):
        perm = torch.randperm(n, generator=g).to(cache.device)
        kt[b, :, :n] = kt[b, :, :n][:, perm]
        vt[b, :, :n] = vt[b, :, :n][:, perm]
    p2 = cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q)
    torch.cuda.synchronize()
    tol = 1e-5 if Hq == Hkv else 2e-3   # the tensor-core kernel rounds P to bf16 per tile
    assert (a - p2).abs().max().item() < tol
    cache.close()


def test_a_sequence_does_not_depend_on_its_batch_mates():
    """Sequences are independent: the first two rows of a batch of five equal a batch of two (up to
    the summation order, which follows the work split)."""
    lens = [500, 77, 1000, 3, 640]
    cache, K, V, q = _attn_case(8, 8, 128, lens, 1024, seed=30)
    a5 = cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q).clone()
    a2 = cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q[:2].contiguous(), batch=2)
    torch.cuda.synchronize()
    assert (a5[:2] - a2).abs().max().item() < 1e-5
    cache.close()


# ---- paged caches ---------------------------------------------------------------------------------

@pytest.mark.parametrize("shape", ["mha128", "mha64", "gqa64", "gqa128"])
def test_paged_cache_matches_oracle(shape):
    """Slots as pools of 64-row pages: a sequence owns ceil(len / 64) pages, assigned in a scrambled
    order; decode steps that cross page boundaries (new pages taken from the pool) stay exact."""
    kw = {"mha128": dict(Hq=4, Hkv=4, d=128, std=1.0), "mha64": dict(Hq=4, Hkv=4, d=64, std=1.0),
          "gqa64": dict(Hq=16, Hkv=2, d=64, std=0.25), "gqa128": dict(Hq=8, Hkv=1, d=128, std=0.25)}[shape]
    lens = [0, 1, 63, 64, 65, 127, 128, 300, 500, 62]
    c = Case(L=4, w=2, lens=lens, T_cap=520, seed=123, page_rows=64, n_pages=40, **kw)
    pt0 = c.cache.lckv_cache_page_table()
    assert [(int((pt0[b] >= 0).sum())) for b in range(len(lens))] == [(n + 63) // 64 for n in lens]
    for _ in range(4):
        c.step()
    pt = c.cache.lckv_cache_page_table()
    assert [(int((pt[b] >= 0).sum())) for b in range(len(lens))] == [(n + 4 + 63) // 64 for n in lens]
    used = pt[pt >= 0].tolist()
    assert len(used) == len(set(used)), "a page is owned twice"
    c.close()


def test_paged_cache_pool_exhaustion_and_reuse():
    B, H, d = 3, 2, 64
    cfg = lk.make_config(2, 0, H, H, d, B, 256, page_rows=64, n_pages=4)
    cache = lk.Cache(cfg)
    with pytest.raises(lk.LckvError) as e:
        cache.lckv_cache_reset([100, 100, 100])            # needs 6 pages
    assert e.value.status == lk.ECAPACITY
    cache.lckv_cache_reset([64, 64, 100])                  # 1 + 1 + 2 pages: pool full
    dev = cache.device
    x = torch.zeros((B, H, d), dtype=torch.bfloat16, device=dev)
    with pytest.raises(lk.LckvError) as e:                  # rows 64 need a new page each: none left
        cache.lckv_layer_stack_step([x, x], [x.clone(), x.clone()], [None, x], [None, x])
    assert e.value.status == lk.ECAPACITY
    assert cache.lckv_cache_lengths(B) == [64, 64, 100]
    pt = cache.lckv_cache_page_table()
    assert int((pt >= 0).sum()) == 4
    cache.lckv_cache_reset([10, 0, 0])                     # pages go back to the pool
    assert int((cache.lckv_cache_page_table() >= 0).sum()) == 1
    cache.lckv_layer_stack_step([x, x], [x.clone(), x.clone()], [None, x], [None, x])
    torch.cuda.synchronize()
    assert cache.lckv_cache_lengths(B) == [11, 1, 1]
    cache.close()
    bad = lk.make_config(2, 0, H, H, d, B, 256, page_rows=48, n_pages=4)   # not a power of two
    assert lk.lckv_cache_bytes(bad) == 0


@pytest.mark.parametrize("Hq,Hkv,d", [(4, 4, 128), (16, 2, 64)])
def test_wait_that_runs_out_is_reported_and_recoverable(Hq, Hkv, d):
    """The bounded device-side wait, made to run out without anything hanging: with a limit of 0 polls
    every worker's first wait on a copy gives up at once (the copies themselves are healthy and land
    during the kernel's bounded drain).  The status word must read LCKV_ETIMEOUT, lckv_cache_reset must
    clear it, and the next step on the same cache must be correct again.  Both decode kernels."""
    c = Case(L=3, w=2, Hq=Hq, Hkv=Hkv, d=d, lens=[40, 200, 7], T_cap=260, seed=4242)
    c.step()                                         # a healthy step first
    c.cache.lckv_cache_set_wait_limit(0)
    q, kn, vn = c.step_inputs()
    dev = c.cache.device
    out = torch.zeros((c.B, Hq, d), dtype=torch.bfloat16, device=dev)
    c.cache.lckv_decode_attention(0, lk.MODE_CONDENSED, q[0].to(dev), out=out)
    torch.cuda.synchronize()
    assert c.cache.lckv_cache_status() == lk.ETIMEOUT
    # recovery: default limit back, reset clears the status word and the merge tickets
    c.cache.lckv_cache_set_wait_limit(1 << 18)
    c.cache.lckv_cache_reset(c.lens.tolist())
    assert c.cache.lckv_cache_status() == 0
    c.step()
    c.step()
    c.close()
