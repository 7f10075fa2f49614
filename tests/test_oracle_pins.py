"""Pins of the float64 CPU oracle against things it did not compute itself.

Each test names the statement of the paper (arXiv 2405.10637) or the piece of
mathematics that fixes the expected value.  Nothing here needs a GPU.
"""
import numpy as np
import pytest
import torch

from oracle import lckv_oracle as orc
from paper_2405_10637_b200 import inputs as syn


def f64(bits_arr):
    """bf16 bits -> float64, written independently of the oracle (numpy view, not a C cast)."""
    return (bits_arr.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rand_bits(shape, seed, std=1.0):
    return syn.bits(syn.randn_bf16(shape, seed, std=std))


def brute_force_rows(qs, K, V, scale, strict):
    """Second, independent formulation: the whole n x n score matrix of an n-token sequence,
    an explicit boolean mask (strictly lower triangular when the diagonal is dropped,
    Section 2.1), dense row softmax.  qs, K, V: float64 [n, d].  Rows with an empty mask are 0."""
    n = qs.shape[0]
    S = scale * (qs @ K.T)
    i, j = np.meshgrid(np.arange(n), np.arange(n), indexing="ij")
    mask = (j < i) if strict else (j <= i)
    out = np.zeros_like(V)
    for r in range(n):
        cols = np.nonzero(mask[r])[0]
        if cols.size == 0:
            continue
        e = np.exp(S[r, cols] - S[r, cols].max())
        p = e / e.sum()
        out[r] = p @ V[cols]
    return out


@pytest.mark.parametrize("strict", [True, False])
@pytest.mark.parametrize("n,d", [(1, 8), (7, 16), (33, 64)])
def test_brute_force_masked_matrix(n, d, strict):
    """Token t of a sequence sees j < t (condensed layers, diagonal masked) or j <= t (warmup
    layers).  Decoding token by token with the oracle must equal the rows of the dense
    masked-matrix attention."""
    qb, Kb, Vb = rand_bits((n, d), 11), rand_bits((n, d), 12), rand_bits((n, d), 13)
    scale = d ** -0.5
    want = brute_force_rows(f64(qb), f64(Kb), f64(Vb), scale, strict)
    for t in range(n):
        n_vis = t if strict else t + 1
        o, _ = orc.attend_row(qb[t], Kb[:n_vis], Vb[:n_vis], scale)
        np.testing.assert_allclose(o, want[t], rtol=0, atol=1e-12)


def test_batched_equals_brute_force_with_gqa_and_ragged_lengths():
    """Batched entry: ragged lengths, grouped heads h -> h // g (Llama's repeat-interleave
    convention), both masks; checked against dense numpy per row."""
    B, Hq, Hkv, T, d = 3, 6, 2, 20, 16
    g = Hq // Hkv
    qb, Kb, Vb = rand_bits((B, Hq, d), 1), rand_bits((B, Hkv, T, d), 2), rand_bits((B, Hkv, T, d), 3)
    lens = np.array([0, 5, 19], np.int32)
    scale = 0.37
    for mode in (0, 1):
        out, lse = orc.decode_attention(qb, Kb, Vb, lens, mode, scale)
        Krep = np.repeat(f64(Kb), g, axis=1)   # repeat_interleave over heads
        Vrep = np.repeat(f64(Vb), g, axis=1)
        for b in range(B):
            nv = lens[b] + mode
            for h in range(Hq):
                if nv == 0:
                    assert np.all(out[b, h] == 0) and lse[b, h] == 0
                    continue
                s = scale * (Krep[b, h, :nv] @ f64(qb)[b, h])
                p = np.exp(s - s.max()); p /= p.sum()
                np.testing.assert_allclose(out[b, h], p @ Vrep[b, h, :nv], atol=1e-12)
                np.testing.assert_allclose(lse[b, h], np.log(np.exp(s - s.max()).sum()) + s.max(),
                                           atol=1e-12)


def test_w_equals_L_is_textbook_causal_attention_sdpa():
    """Section 4.2: with w = L the model is exactly the standard transformer.  The last row of
    torch's float64 causal scaled_dot_product_attention is the library routine it reduces to."""
    L, B, Hq, Hkv, T, d = 3, 2, 4, 2, 9, 32
    g = Hq // Hkv
    scale = d ** -0.5
    lens = np.full(B, T - 1, np.int32)          # T-1 cached, the new token is position T-1
    Ks = [rand_bits((B, Hkv, T, d), 100 + l) for l in range(L)]
    Vs = [rand_bits((B, Hkv, T, d), 200 + l) for l in range(L)]
    qs = [rand_bits((B, Hq, d), 300 + l) for l in range(L)]
    kn = [rand_bits((B, Hkv, d), 400 + l) for l in range(L)]
    vn = [rand_bits((B, Hkv, d), 500 + l) for l in range(L)]
    plan = orc.plan(L, L)
    Kslots = [None] * L
    Vslots = [None] * L
    for l in range(L):
        Kslots[plan["read_slot"][l]] = Ks[l].copy()
        Vslots[plan["read_slot"][l]] = Vs[l].copy()
    ln = lens.copy()
    outs, _ = orc.stack_step(L, L, qs, kn, vn, Kslots, Vslots, ln, scale)
    for l in range(L):
        Kfull = f64(Ks[l]); Vfull = f64(Vs[l])
        Kfull[:, :, T - 1] = f64(kn[l]); Vfull[:, :, T - 1] = f64(vn[l])
        # queries of earlier positions are irrelevant for the last row: fill with zeros
        Q = np.zeros((B, Hq, T, d)); Q[:, :, T - 1] = f64(qs[l])
        Kt = torch.from_numpy(Kfull).repeat_interleave(g, dim=1)
        Vt = torch.from_numpy(Vfull).repeat_interleave(g, dim=1)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q), Kt, Vt, is_causal=True, scale=scale)[:, :, T - 1].numpy()
        np.testing.assert_allclose(outs[l], ref, atol=1e-12)


def test_closed_forms():
    d, n = 16, 12
    Kb, Vb = rand_bits((n, d), 5), rand_bits((n, d), 6)
    V = f64(Vb)
    # q = 0: every score is 0, softmax is uniform, o = arithmetic mean of the visible values
    q0 = np.zeros(d, np.uint16)
    o, lse = orc.attend_row(q0, Kb, Vb, 0.25)
    np.testing.assert_allclose(o, V.mean(0), atol=1e-14)
    np.testing.assert_allclose(lse, np.log(n), atol=1e-14)
    # all keys equal: uniform again, whatever q is
    qb = rand_bits((d,), 7)
    Keq = np.repeat(Kb[:1], n, axis=0)
    o, _ = orc.attend_row(qb, Keq, Vb, 0.25)
    np.testing.assert_allclose(o, V.mean(0), atol=1e-13)
    # one visible key: weight exactly 1, o = v_0 exactly
    o, _ = orc.attend_row(qb, Kb[:1], Vb[:1], 0.25)
    assert np.array_equal(o, V[0])
    # nothing visible (first token under the diagonal mask): zero dummy KV, o = 0, lse = 0
    o, lse = orc.attend_row(qb, Kb[:0], Vb[:0], 0.25)
    assert np.all(o == 0) and lse == 0
    # a key that is a large multiple of q dominates: o -> its value row
    q = f64(qb)
    big = syn.bits(torch.tensor(64.0 * q, dtype=torch.float32).to(torch.bfloat16))
    Kd = Kb.copy(); Kd[4] = big
    o, _ = orc.attend_row(qb, Kd, Vb, 1.0)
    np.testing.assert_allclose(o, V[4], atol=1e-9)


def test_probabilities_sum_to_one_and_reproduce_output():
    d, n = 32, 50
    qb, Kb, Vb = rand_bits((d,), 21), rand_bits((n, d), 22), rand_bits((n, d), 23)
    for sink in (False, True):
        o, lse, p = orc.attend_row(qb, Kb, Vb, d ** -0.5, always_sink=sink, want_probs=True)
        assert np.all(p >= 0)
        np.testing.assert_allclose(p.sum(), 1.0, atol=1e-14)
        np.testing.assert_allclose(o, p[:n] @ f64(Vb), atol=1e-14)
        assert (p[n] > 0) == sink
    # empty visible set: the dummy column carries all the weight
    _, _, p = orc.attend_row(qb, Kb[:0], Vb[:0], 1.0, want_probs=True)
    assert p.tolist() == [1.0]


def test_always_sink_reading_differs_and_matches_extra_zero_column():
    """The alternative reading of the dummy KV (a permanent zero key/value column) equals plain
    attention over the cache with one all-zero row added; it is NOT the default."""
    d, n = 16, 9
    qb, Kb, Vb = rand_bits((d,), 31), rand_bits((n, d), 32), rand_bits((n, d), 33)
    o_def, _ = orc.attend_row(qb, Kb, Vb, 0.3)
    o_sink, _ = orc.attend_row(qb, Kb, Vb, 0.3, always_sink=True)
    Kz = np.concatenate([Kb, np.zeros((1, d), np.uint16)])
    Vz = np.concatenate([Vb, np.zeros((1, d), np.uint16)])
    o_z, _ = orc.attend_row(qb, Kz, Vz, 0.3)
    np.testing.assert_allclose(o_sink, o_z, atol=1e-14)
    assert np.abs(o_sink - o_def).max() > 1e-3


def test_permutation_invariance():
    d, n = 16, 40
    qb, Kb, Vb = rand_bits((d,), 41), rand_bits((n, d), 42), rand_bits((n, d), 43)
    o, lse = orc.attend_row(qb, Kb, Vb, 0.2)
    perm = np.random.default_rng(0).permutation(n)
    o2, lse2 = orc.attend_row(qb, Kb[perm], Vb[perm], 0.2)
    np.testing.assert_allclose(o2, o, atol=1e-13)
    np.testing.assert_allclose(lse2, lse, atol=1e-13)


@pytest.mark.parametrize("cuts", [[13], [1, 2, 30], [5, 10, 15, 20, 25, 37]])
def test_lse_merge_of_any_partition_equals_unsplit(cuts):
    """Split-K identity: attention over disjoint chunks, merged with
    m = max m_c, l = sum l_c e^{m_c - m}, o = sum o_c l_c e^{m_c - m} / l, is the unsplit result.
    This pins the oracle's lse output, which the merge consumes."""
    d, n = 16, 38
    qb, Kb, Vb = rand_bits((d,), 51), rand_bits((n, d), 52), rand_bits((n, d), 53)
    o, lse = orc.attend_row(qb, Kb, Vb, 0.5)
    edges = [0] + cuts + [n]
    parts = [orc.attend_row(qb, Kb[a:b], Vb[a:b], 0.5) for a, b in zip(edges[:-1], edges[1:])]
    lses = np.array([p[1] for p in parts])
    wts = np.exp(lses - lses.max())
    merged = sum(wt * p[0] for wt, p in zip(wts, parts)) / wts.sum()
    np.testing.assert_allclose(merged, o, atol=1e-13)
    np.testing.assert_allclose(lses.max() + np.log(wts.sum()), lse, atol=1e-13)


def test_plan_enumerated_by_hand():
    """Section 2.1: top w/2 and bottom w/2 layers are warmup layers.  Sets written out by hand."""
    cases = {
        (4, 0): [], (4, 2): [0, 3], (4, 4): [0, 1, 2, 3], (22, 2): [0, 21],
        (22, 10): [0, 1, 2, 3, 4, 17, 18, 19, 20, 21], (32, 8): [0, 1, 2, 3, 28, 29, 30, 31],
        (60, 2): [0, 59], (8, 8): list(range(8)),
    }
    for (L, w), W in cases.items():
        for variant in (0, 1):
            p = orc.plan(L, w, variant)
            assert np.nonzero(p["is_warmup"])[0].tolist() == W
            # footprint in cached layers: max(w, 1) when the shared cache is layer L-1's own,
            # min(w + 1, L) when a separate layer feeds it
            want_slots = max(w, 1) if (variant == 0 or w in (0, L)) else min(w + 1, L)
            assert p["n_slots"] == want_slots
            for l in range(L):
                if l in W:
                    assert p["mode"][l] == 1 and p["write_slot"][l] == p["read_slot"][l]
                    assert p["write_before"][l] == 1
                else:
                    assert p["mode"][l] == 0 and p["read_slot"][l] == 0
            # warmup layers never share a cache with each other
            ws = [p["read_slot"][l] for l in W]
            assert len(set(ws)) == len(ws)
            # exactly one layer feeds slot 0
            feeders = [l for l in range(L) if p["write_slot"][l] == 0]
            if variant == 0 or w in (0, L):
                assert feeders == [L - 1]
            else:
                assert feeders == [L - 1 - w // 2] and p["mode"][feeders[0]] == 0


def test_plan_rejects_odd_or_out_of_range_w():
    for L, w in [(4, 1), (4, 3), (4, 5), (4, -2), (0, 0)]:
        with pytest.raises(orc.OracleError):
            orc.plan(L, w)


def _stack_inputs(L, B, Hq, Hkv, T, d, n_slots, seed):
    Ks = [rand_bits((B, Hkv, T, d), seed + 10 + s) for s in range(n_slots)]
    Vs = [rand_bits((B, Hkv, T, d), seed + 30 + s) for s in range(n_slots)]
    qs = [rand_bits((B, Hq, d), seed + 50 + l) for l in range(L)]
    kn = [rand_bits((B, Hkv, d), seed + 100 + l) for l in range(L)]
    vn = [rand_bits((B, Hkv, d), seed + 150 + l) for l in range(L)]
    return Ks, Vs, qs, kn, vn


def test_w0_every_layer_reads_the_same_top_layer_cache():
    """w = 0: all layers pair with the one shared cache; the same q gives the same output in
    every layer, and the step's new k,v (row t) are invisible to all of them."""
    L, B, Hq, Hkv, T, d = 4, 2, 4, 4, 12, 16
    Ks, Vs, qs, kn, vn = _stack_inputs(L, B, Hq, Hkv, T, d, 1, 700)
    qs = [qs[0]] * L
    lens = np.array([3, 11], np.int32)
    K0, V0 = Ks[0].copy(), Vs[0].copy()
    outs, _ = orc.stack_step(L, 0, qs, [None] * (L - 1) + [kn[-1]], [None] * (L - 1) + [vn[-1]],
                             Ks, Vs, lens, 0.25)
    for l in range(1, L):
        assert np.array_equal(outs[l], outs[0])
    # poisoning row t and everything after it before the step changes nothing
    Kp, Vp = K0.copy(), V0.copy()
    for b, t in enumerate([3, 11]):
        Kp[b, :, t:] = 0x7FC0  # NaN
        Vp[b, :, t:] = 0x7FC0
    outs2, _ = orc.stack_step(L, 0, qs, [None] * (L - 1) + [kn[-1]], [None] * (L - 1) + [vn[-1]],
                              [Kp], [Vp], np.array([3, 11], np.int32), 0.25)
    for l in range(L):
        assert np.array_equal(outs2[l], outs[l])
    assert lens.tolist() == [4, 12]


def test_warmup_layer_sees_its_own_new_kv_and_only_it_does():
    L, w, B, Hq, Hkv, T, d = 6, 2, 2, 4, 2, 10, 16
    p = orc.plan(L, w)
    Ks, Vs, qs, kn, vn = _stack_inputs(L, B, Hq, Hkv, T, d, p["n_slots"], 900)
    has_kv = [p["write_slot"][l] >= 0 for l in range(L)]
    knl = [kn[l] if has_kv[l] else None for l in range(L)]
    vnl = [vn[l] if has_kv[l] else None for l in range(L)]
    lens0 = np.array([4, 9], np.int32)

    def run(knl_):
        return orc.stack_step(L, w, qs, knl_, vnl, [k.copy() for k in Ks], [v.copy() for v in Vs],
                              lens0.copy(), 0.3)[0]
    base = run(knl)
    for l in [0, L - 1]:
        alt = list(knl); alt[l] = rand_bits((B, Hkv, d), 4242 + l)
        got = run(alt)
        for m in range(L):
            same = np.array_equal(got[m], base[m])
            assert same == (m != l), (l, m)


def test_append_positions_lengths_and_untouched_bytes():
    """After a step: lens + 1; row lens of every written cache holds the new bits exactly; every
    other element of every cache is unchanged."""
    for variant in (0, 1):
        L, w, B, Hq, Hkv, T, d = 6, 2, 3, 4, 2, 8, 8
        p = orc.plan(L, w, variant)
        Ks, Vs, qs, kn, vn = _stack_inputs(L, B, Hq, Hkv, T, d, p["n_slots"], 1200)
        has_kv = [p["write_slot"][l] >= 0 for l in range(L)]
        knl = [kn[l] if has_kv[l] else None for l in range(L)]
        vnl = [vn[l] if has_kv[l] else None for l in range(L)]
        lens = np.array([0, 3, 7], np.int32)
        K0 = [k.copy() for k in Ks]; V0 = [v.copy() for v in Vs]
        orc.stack_step(L, w, qs, knl, vnl, Ks, Vs, lens, 0.3, top_variant=variant)
        assert lens.tolist() == [1, 4, 8]
        written = {p["write_slot"][l]: l for l in range(L) if has_kv[l]}
        assert sorted(written) == list(range(p["n_slots"]))
        for s in range(p["n_slots"]):
            l = written[s]
            expK, expV = K0[s].copy(), V0[s].copy()
            for b, t in enumerate([0, 3, 7]):
                expK[b, :, t] = kn[l][b]; expV[b, :, t] = vn[l][b]
            assert np.array_equal(Ks[s], expK) and np.array_equal(Vs[s], expV)
    # capacity: a full sequence cannot take another token, nothing is written
    lens = np.array([0, 3, 8], np.int32)
    Kc = [k.copy() for k in Ks]
    with pytest.raises(orc.OracleError):
        orc.stack_step(L, w, qs, knl, vnl, Ks, Vs, lens, 0.3, top_variant=1)
    assert lens.tolist() == [0, 3, 8] and all(np.array_equal(a, b) for a, b in zip(Ks, Kc))


def test_variant1_condensed_layers_never_see_top_warmup_cache():
    """Reading 2 of 'the top layer': slot 0 is fed by the topmost non-warmup layer and the top
    warmup layers keep their own caches; changing those caches changes only their own outputs."""
    L, w, B, Hq, Hkv, T, d = 6, 2, 1, 2, 2, 6, 8
    p = orc.plan(L, w, 1)
    assert p["n_slots"] == 3
    Ks, Vs, qs, kn, vn = _stack_inputs(L, B, Hq, Hkv, T, d, 3, 1500)
    has_kv = [p["write_slot"][l] >= 0 for l in range(L)]
    knl = [kn[l] if has_kv[l] else None for l in range(L)]
    vnl = [vn[l] if has_kv[l] else None for l in range(L)]
    lens0 = np.array([5], np.int32)
    base = orc.stack_step(L, w, qs, knl, vnl, [k.copy() for k in Ks], [v.copy() for v in Vs],
                          lens0.copy(), 0.3, top_variant=1)[0]
    top_slot = p["read_slot"][L - 1]
    K2 = [k.copy() for k in Ks]; K2[top_slot] = rand_bits((B, Hkv, T, d), 99)
    got = orc.stack_step(L, w, qs, knl, vnl, K2, [v.copy() for v in Vs], lens0.copy(), 0.3,
                         top_variant=1)[0]
    for l in range(L):
        assert np.array_equal(got[l], base[l]) == (l != L - 1)


def test_multi_step_decode_equals_dense_sequence_attention():
    """Several consecutive steps from an empty cache (w = 0, one layer): the outputs are the rows of
    strictly-lower-triangular attention over the keys/values appended so far."""
    n, d = 6, 8
    qb, kb, vb = rand_bits((n, 1, 1, d), 61), rand_bits((n, 1, 1, d), 62), rand_bits((n, 1, 1, d), 63)
    K = np.zeros((1, 1, n, d), np.uint16); V = np.zeros_like(K)
    lens = np.zeros(1, np.int32)
    rows = []
    for t in range(n):
        outs, _ = orc.stack_step(1, 0, [qb[t]], [kb[t]], [vb[t]], [K], [V], lens, 0.4)
        rows.append(outs[0][0, 0])
    want = brute_force_rows(f64(qb[:, 0, 0]), f64(kb[:, 0, 0]), f64(vb[:, 0, 0]), 0.4, True)
    np.testing.assert_allclose(np.stack(rows), want, atol=1e-12)
    assert lens[0] == n and np.array_equal(K[0, 0], kb[:, 0, 0])


def test_golden_two_key_example():
    """Hand-derived fixture (tests/golden/two_key_softmax.txt): q=[1], K=[[0],[1]], V=[[0],[1]]."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "two_key_softmax.txt")
    rows = [l.split() for l in open(path) if not l.startswith("#")]
    one, zero = 0x3F80, 0x0000
    q = np.array([one], np.uint16)
    K = np.array([[zero], [one]], np.uint16)
    V = np.array([[zero], [one]], np.uint16)
    for name, n_vis, want_o, want_lse in rows:
        o, lse = orc.attend_row(q, K[:int(n_vis)], V[:int(n_vis)], 1.0)
        np.testing.assert_allclose(o[0], float(want_o), atol=1e-15)
        np.testing.assert_allclose(lse, float(want_lse), atol=1e-15)


# ---- sink + recent-window caches (Section 3.3: integration with StreamingLLM) ---------------------

def test_streaming_ring_rows_enumerated_by_hand():
    """Cache of 6 rows with 2 sinks: tokens 0..5 fill rows 0..5, then the 4 non-sink rows are reused
    in turn.  Written out by hand."""
    C_, s = 6, 2
    want_rows = [0, 1, 2, 3, 4, 5, 2, 3, 4, 5, 2, 3]
    K = np.zeros((1, 1, C_, 4), np.uint16); V = np.zeros_like(K)
    for t, row in enumerate(want_rows):
        k = np.full((1, 1, 4), 100 + t, np.uint16)
        before = K.copy()
        orc.append(K, V, k, k, np.array([t], np.int32), n_sink=s)
        changed = np.nonzero((K != before).any(axis=-1)[0, 0])[0].tolist()
        assert changed == [row], (t, changed)
        assert (K[0, 0, row] == 100 + t).all()


@pytest.mark.parametrize("w", [0, 1])
def test_streaming_equals_attention_over_sinks_plus_recent_tokens(w):
    """Decode n tokens through a small ring cache; each output must equal plain attention, computed
    here from the full history, over the first s tokens plus the most recent C - s tokens that the
    query may see (before t for the diagonal-masked layers, up to and including t for standard
    layers).  Row order inside the ring is irrelevant (permutation invariance)."""
    n, d, C_, s = 25, 8, 9, 3
    qb, kb, vb = rand_bits((n, 1, 1, d), 71), rand_bits((n, 1, 1, d), 72), rand_bits((n, 1, 1, d), 73)
    K = np.zeros((1, 1, C_, d), np.uint16); V = np.zeros_like(K)
    lens = np.zeros(1, np.int32)
    Kh, Vh, Q = f64(kb[:, 0, 0]), f64(vb[:, 0, 0]), f64(qb[:, 0, 0])
    for t in range(n):
        outs, _ = orc.stack_step(1, w, [qb[t]], [kb[t]], [vb[t]], [K], [V], lens, 0.4, n_sink=s)
        last = t + 1 if w else t                      # exclusive end of what the query may see
        vis = list(range(min(s, last))) + list(range(max(s, last - (C_ - s)), last))
        if not vis:
            assert not outs[0].any()
            continue
        sc = 0.4 * (Kh[vis] @ Q[t]); p = np.exp(sc - sc.max()); p /= p.sum()
        np.testing.assert_allclose(outs[0][0, 0], p @ Vh[vis], atol=1e-12)
    assert lens[0] == n
    # until the cache is full the policy changes nothing
    K2 = np.zeros((1, 1, C_, d), np.uint16); V2 = np.zeros_like(K2); l2 = np.zeros(1, np.int32)
    K3 = K2.copy(); V3 = V2.copy(); l3 = np.zeros(1, np.int32)
    for t in range(C_):
        a, _ = orc.stack_step(1, w, [qb[t]], [kb[t]], [vb[t]], [K2], [V2], l2, 0.4, n_sink=s)
        b, _ = orc.stack_step(1, w, [qb[t]], [kb[t]], [vb[t]], [K3], [V3], l3, 0.4)
        assert np.array_equal(a[0], b[0])
    assert np.array_equal(K2, K3)
    with pytest.raises(orc.OracleError):   # without the policy the 10th token does not fit
        orc.stack_step(1, w, [qb[C_]], [kb[C_]], [vb[C_]], [K3], [V3], l3, 0.4)
