"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The oracle cannot run a whole 0.5 TB step, so it checks sampled output rows one by one: for a
sampled (layer, sequence, head) the visible K/V rows and the query are copied from the device and
attended on the CPU in float64.  On top of that: every output finite, lengths advanced by exactly
one, appended rows bit-identical to the step's k/v.  Inputs are the bench's (seeded, device-drawn).
"""
import numpy as np
import pytest
import torch

from oracle import lckv_oracle as orc
from paper_2405_10637_b200 import binding as lk
from paper_2405_10637_b200 import inputs as syn
from helpers import REL_L2, bf16_tolerance, compare

pytestmark = pytest.mark.gpu


def run_full(wl, B, lens, T_cap, n_samples, seed, top_variant=0, steps=1, check_at=None, fixed_inputs=False):
    L, Hq, Hkv, d = wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
    g = Hq // Hkv
    cfg = lk.make_config(L, wl.n_warmup, Hq, Hkv, d, B, T_cap, top_variant=top_variant)
    cache = lk.Cache(cfg)
    dev = cache.device
    plan = lk.lckv_plan(L, wl.n_warmup, top_variant)
    for s in range(cache.info.n_slots):
        kt, vt = cache.slot_tensors(s)
        syn.fill_randn_bf16_(kt, syn.seed_for(wl, syn.T_K, s), std=wl.std)
        syn.fill_randn_bf16_(vt, syn.seed_for(wl, syn.T_V, s), std=wl.std)
    cache.lckv_cache_reset(lens.tolist())
    rng = np.random.default_rng(seed)
    scale = d ** -0.5
    cur = lens.astype(np.int64).copy()
    q = kv = outs = None
    for step in range(steps):
        if q is None or not fixed_inputs:
            q = [syn.randn_bf16((B, Hq, d), 900 + l + 100 * step, device=dev, std=wl.std) for l in range(L)]
            kv = [syn.randn_bf16((B, Hkv, d), 950 + l + 100 * step, device=dev, std=wl.std)
                  if plan["write_slot"][l] >= 0 else None for l in range(L)]
            outs = [torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=dev) for _ in range(L)]
        cache.lckv_layer_stack_step(q, outs, kv, kv)
        if check_at is not None and step not in check_at:
            cur += 1
            continue
        torch.cuda.synchronize()
        assert cache.lckv_cache_status() == 0
        for l in range(L):
            assert torch.isfinite(outs[l].float()).all(), f"layer {l}: non-finite output"
        errs, refs = [], []
        for _ in range(n_samples):
            l, b, h = int(rng.integers(L)), int(rng.integers(B)), int(rng.integers(Hq))
            slot, mode = plan["read_slot"][l], plan["mode"][l]
            n_vis = int(cur[b]) + mode
            kt, vt = cache.slot_tensors(slot)
            o, _ = orc.attend_row(syn.bits(q[l][b, h]), syn.bits(kt[b, h // g, :n_vis]),
                                  syn.bits(vt[b, h // g, :n_vis]), scale)
            got = outs[l][b, h].float().cpu().numpy().astype(np.float64)
            assert (np.abs(got - o) <= bf16_tolerance(o)).all(), (l, b, h, np.abs(got - o).max())
            errs.append(got - o); refs.append(o)
        rel = np.linalg.norm(np.stack(errs)) / np.linalg.norm(np.stack(refs))
        assert rel <= REL_L2, rel
        # appended rows and lengths (bit-exact), on a few sequences
        for l in range(L):
            if plan["write_slot"][l] < 0:
                continue
            kt, vt = cache.slot_tensors(plan["write_slot"][l])
            for b in rng.integers(B, size=3):
                row = int(cur[b])
                assert torch.equal(kt[b, :, row], kv[l][b]) and torch.equal(vt[b, :, row], kv[l][b])
        cur += 1
        assert cache.lckv_cache_lengths(B) == cur.tolist()
    if fixed_inputs:
        # every step appended the same k/v: the rows [len0, len0 + steps) of each fed slot must all
        # hold them, bit for bit, and nothing beyond
        torch.cuda.synchronize()
        assert cache.lckv_cache_status() == 0
        for l in range(L):
            if plan["write_slot"][l] < 0:
                continue
            kt, vt = cache.slot_tensors(plan["write_slot"][l])
            for b in rng.integers(B, size=min(B, 4)):
                lo = int(lens[b])
                want = kv[l][b][:, None, :].expand(-1, steps, -1)
                assert torch.equal(kt[b, :, lo:lo + steps], want) and torch.equal(vt[b, :, lo:lo + steps], want)
    cache.close()


def test_llama7b_ragged_batch_512():
    """Llama-7B shape, w = 2, ragged lengths uniform in [256, 4096], B = 512 (the headline case)."""
    wl = syn.WORKLOADS["llama7b"]
    B = 512
    lens = syn.ragged_lengths(B, 256, 4096, syn.seed_for(wl, syn.T_LENS)).numpy()
    run_full(wl, B, lens, 4096 + 64, n_samples=48, seed=1)


def test_llama7b_small_batch_8_variant1():
    """The small end of the batch sweep (every pair split over several workers), reading 2 of 'top layer'."""
    wl = syn.WORKLOADS["llama7b"]
    lens = syn.ragged_lengths(8, 256, 4096, syn.seed_for(wl, syn.T_LENS)).numpy()
    run_full(wl, 8, lens, 4096 + 64, n_samples=48, seed=2, top_variant=1, steps=2)


def test_tinyllama_batch_128_decode_steps():
    """TinyLlama shape (GQA 8:1), B = 128, prompt 512, three decode steps."""
    wl = syn.WORKLOADS["tinyllama"]
    lens = np.full(128, 512, np.int32)
    run_full(wl, 128, lens, 1536, n_samples=48, seed=3, steps=3)


def test_tinyllama_1024_decode_steps_fill_the_cache():
    """TinyLlama shape, B = 128, prompt 512 + 1024 generated tokens (the paper's 512+1024 setting): the
    caches end exactly full; sampled rows are checked at the first steps, in the middle and at the end."""
    wl = syn.WORKLOADS["tinyllama"]
    lens = np.full(128, 512, np.int32)
    run_full(wl, 128, lens, 1536, n_samples=24, seed=13, steps=1024, check_at={0, 1, 511, 1023},
             fixed_inputs=True)


def test_llama30b_2048_appends_small_batch():
    """Llama-30B shape (60 layers, 52 heads), prompt 2048 + 2048 generated tokens at B = 2: every one
    of the 2048 appended rows lands where it should."""
    wl = syn.WORKLOADS["llama30b"]
    lens = np.full(2, 2048, np.int32)
    run_full(wl, 2, lens, 4096, n_samples=16, seed=14, steps=2048, check_at={0, 1024, 2047},
             fixed_inputs=True)


def test_llama30b_batch_256():
    """Llama-30B shape: 60 layers, 52 heads (not a power of two), context 2048, B = 256."""
    wl = syn.WORKLOADS["llama30b"]
    lens = np.full(256, 2048, np.int32)
    run_full(wl, 256, lens, 2048 + 64, n_samples=32, seed=4)


@pytest.mark.parametrize("w,B,T", [(0, 64, 8192), (2, 64, 8192), (4, 64, 8192), (8, 64, 8192), (32, 40, 8192),
                                   (0, 8, 32768), (2, 8, 32768), (4, 8, 32768), (8, 8, 32768), (32, 8, 32768)])
def test_long_context_warmup_sweep(w, B, T):
    """7B shape at long context for every warmup count of the sweep, w = 0, 2, 4, 8 and 32 (footprint
    max(w,1) caches).  w = 32 is the standard transformer: 32 caches, which at 8192 tokens hold 4.3 GB per
    sequence, so 64 sequences (275 GB) do not fit one GPU and the batch is 40 (173 GB) - the growth of
    the footprint with w is the paper's point (Section 3.1, Table 1)."""
    wl = syn.WORKLOADS["sweep7b"].with_(n_warmup=w)
    lens = np.full(B, T, np.int32)
    run_full(wl, B, lens, T + 64, n_samples=24, seed=5 + w)


def per_sequence_cache_bytes(wl, T_cap, n_slots):
    return n_slots * 4 * wl.n_kv_heads * wl.head_dim * T_cap


@pytest.mark.parametrize("top_variant", [0, 1])
def test_llama30b_largest_batch_that_fits(top_variant):
    """Llama-30B shape, prompt 2048 + 2048 generated tokens, at the largest batch whose caches fit 180 GB
    (Section 3.1, Table 1 sizes batches by what fits): a sequence takes 109.05 MB per cache at 4096 rows, so
    825 sequences with the two caches of the literal reading of "top layer" (179.9 GB) and 550 with the
    three caches of the other reading (also 179.9 GB).  The batch is lowered only as far as the free memory of
    this GPU requires (never below 800 / 512).  Checked at the first decode step (2048 cached tokens) and
    at the last one (4095: the step fills the caches)."""
    wl = syn.WORKLOADS["llama30b"]
    n_slots = 2 if top_variant == 0 else 3
    per_seq = per_sequence_cache_bytes(wl, 4096, n_slots)
    target, floor = (825, 800) if top_variant == 0 else (550, 512)
    assert target == int(180e9 // per_seq)
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    act = 2 * wl.n_layers * wl.n_q_heads * wl.head_dim * 2 + 4 * 3 * wl.n_kv_heads * wl.head_dim * 2
    B = min(target, int((free - 4e9) // (per_seq + 2 * act)))
    assert B >= floor, (B, free)
    for first_len in (2048, 4095):
        run_full(wl, B, np.full(B, first_len, np.int32), 4096, n_samples=24, seed=40 + top_variant,
                 top_variant=top_variant)


def check_sequences_against_oracle(wl, cache, plan, lens_before, seqs, q, kv, outs, pre_K, pre_V, what):
    """Whole sequences: every layer, head and element of the outputs of the sequences `seqs`, and their
    caches after the step bit for bit.  pre_K / pre_V: host copies (bits) of those sequences' rows of
    every slot taken BEFORE the step; the oracle steps them on the CPU."""
    L, d = wl.n_layers, wl.head_dim
    idx = torch.as_tensor(seqs, device=outs[0].device)
    ln = np.ascontiguousarray(np.asarray(lens_before)[seqs], np.int32)
    want, _ = orc.stack_step(L, wl.n_warmup, [syn.bits(t[idx]) for t in q],
                             [None if t is None else syn.bits(t[idx]) for t in kv],
                             [None if t is None else syn.bits(t[idx]) for t in kv],
                             pre_K, pre_V, ln, d ** -0.5, top_variant=0)
    worst = (0.0, 0.0)
    for l in range(L):
        m = compare(outs[l][idx], want[l], f"{what} layer {l}")
        worst = (max(worst[0], m[0]), max(worst[1], m[1]))
    assert ln.tolist() == (np.asarray(lens_before)[seqs] + 1).tolist()
    for s in range(cache.info.n_slots):
        kt, vt = cache.slot_tensors(s)
        assert np.array_equal(syn.bits(kt[idx]), pre_K[s]), f"{what}: slot {s} K differs after the step"
        assert np.array_equal(syn.bits(vt[idx]), pre_V[s]), f"{what}: slot {s} V differs after the step"
    return worst


def test_tinyllama_every_row_at_first_middle_and_last_steps():
    """TinyLlama shape, B = 128, prompt 512 + 1024 decode steps: at steps 0, 1, 511 and 1023 EVERY output
    element of every layer, sequence and head is compared with the oracle, and after each of those steps
    every byte of both caches (the oracle steps host copies of the caches taken just before)."""
    wl = syn.WORKLOADS["tinyllama"]
    L, Hq, Hkv, d, B, T_cap = wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, 128, 1536
    cache = lk.Cache(lk.make_config(L, wl.n_warmup, Hq, Hkv, d, B, T_cap))
    dev = cache.device
    plan = lk.lckv_plan(L, wl.n_warmup, 0)
    for s in range(cache.info.n_slots):
        kt, vt = cache.slot_tensors(s)
        syn.fill_randn_bf16_(kt, syn.seed_for(wl, syn.T_K, s), std=wl.std)
        syn.fill_randn_bf16_(vt, syn.seed_for(wl, syn.T_V, s), std=wl.std)
    lens = np.full(B, 512, np.int32)
    cache.lckv_cache_reset(lens.tolist())
    seqs = list(range(B))
    for step in range(1024):
        checked = step in (0, 1, 511, 1023)
        if checked or step == 2:   # fresh inputs at the checked steps, then reused in between
            q = [syn.randn_bf16((B, Hq, d), 900 + l + 100 * step, device=dev, std=wl.std) for l in range(L)]
            kv = [syn.randn_bf16((B, Hkv, d), 950 + l + 100 * step, device=dev, std=wl.std)
                  if plan["write_slot"][l] >= 0 else None for l in range(L)]
            outs = [torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=dev) for _ in range(L)]
        if checked:
            torch.cuda.synchronize()
            pre_K = [syn.bits(cache.slot_tensors(s)[0]) for s in range(cache.info.n_slots)]
            pre_V = [syn.bits(cache.slot_tensors(s)[1]) for s in range(cache.info.n_slots)]
        cache.lckv_layer_stack_step(q, outs, kv, kv)
        if checked:
            torch.cuda.synchronize()
            assert cache.lckv_cache_status() == 0
            check_sequences_against_oracle(wl, cache, plan, lens, seqs, q, kv, outs, pre_K, pre_V, f"step {step}")
        lens += 1
    assert cache.lckv_cache_lengths(B) == [1536] * B
    cache.close()


def test_llama7b_batch_512_whole_sequences():
    """The headline case (7B shape, w = 2, ragged U[256, 4096], B = 512): whole sequences instead of sampled
    rows - the shortest, the longest, the first and the last of the batch, a run of 12 neighbours and 16
    drawn at random: all 32 layers x 32 heads x 128 elements of each, and their cache rows after the step."""
    wl = syn.WORKLOADS["llama7b"]
    L, Hq, Hkv, d, B = wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, 512
    lens = syn.ragged_lengths(B, 256, 4096, syn.seed_for(wl, syn.T_LENS)).numpy()
    T_cap = 4096 + 64
    cache = lk.Cache(lk.make_config(L, wl.n_warmup, Hq, Hkv, d, B, T_cap))
    dev = cache.device
    plan = lk.lckv_plan(L, wl.n_warmup, 0)
    for s in range(cache.info.n_slots):
        kt, vt = cache.slot_tensors(s)
        syn.fill_randn_bf16_(kt, syn.seed_for(wl, syn.T_K, s), std=wl.std)
        syn.fill_randn_bf16_(vt, syn.seed_for(wl, syn.T_V, s), std=wl.std)
    cache.lckv_cache_reset(lens.tolist())
    rng = np.random.default_rng(33)
    chosen = {int(np.argmin(lens)), int(np.argmax(lens)), 0, B - 1} | set(range(200, 212))
    while len(chosen) < 32:
        chosen.add(int(rng.integers(B)))
    seqs = sorted(chosen)
    idx = torch.as_tensor(seqs, device=dev)
    pre_K = [syn.bits(cache.slot_tensors(s)[0][idx]) for s in range(cache.info.n_slots)]
    pre_V = [syn.bits(cache.slot_tensors(s)[1][idx]) for s in range(cache.info.n_slots)]
    q = [syn.randn_bf16((B, Hq, d), 900 + l, device=dev, std=wl.std) for l in range(L)]
    kv = [syn.randn_bf16((B, Hkv, d), 950 + l, device=dev, std=wl.std)
          if plan["write_slot"][l] >= 0 else None for l in range(L)]
    outs = [torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=dev) for _ in range(L)]
    cache.lckv_layer_stack_step(q, outs, kv, kv)
    torch.cuda.synchronize()
    assert cache.lckv_cache_status() == 0
    for l in range(L):
        assert torch.isfinite(outs[l].float()).all(), f"layer {l}: non-finite output"
    check_sequences_against_oracle(wl, cache, plan, lens, seqs, q, kv, outs, pre_K, pre_V, "B=512")
    assert cache.lckv_cache_lengths(B) == (lens + 1).tolist()
    cache.close()
