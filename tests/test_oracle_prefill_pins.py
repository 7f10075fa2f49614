"""Pins of the oracle's prompt-encoding functions (paper Section 2.3; one parallel iteration as in
Section 2.2.1) against dense masked attention, a library routine, and - through the paper's own
equivalence lemma (Appendix A) - against the already pinned token-by-token decode path."""
import numpy as np
import pytest
import torch

from oracle import lckv_oracle as orc
from paper_2405_10637_b200 import inputs as syn


def f64(bits_arr):
    return (bits_arr.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def to_bits(x):
    """float64 array -> bf16 bits (round to nearest even), via torch."""
    return syn.bits(torch.from_numpy(np.ascontiguousarray(x, np.float32)).to(torch.bfloat16))


def rand_bits(shape, seed, std=1.0):
    return syn.bits(syn.randn_bf16(shape, seed, std=std))


@pytest.mark.parametrize("mode", [0, 1])
def test_prefill_equals_dense_masked_attention_ragged_gqa(mode):
    """All prompt tokens at once = rows of the dense attention matrix with the strictly lower
    triangular (mode 0) or lower triangular (mode 1) mask; ragged prompts, grouped heads."""
    B, n, Hq, Hkv, T, d = 3, 13, 4, 2, 16, 8
    g = Hq // Hkv
    qb, Kb, Vb = rand_bits((B, n, Hq, d), 1), rand_bits((B, Hkv, T, d), 2), rand_bits((B, Hkv, T, d), 3)
    lens = np.array([13, 1, 7], np.int32)
    out = orc.prefill_attention(qb, Kb, Vb, lens, mode, 0.3)
    Q, K, V = f64(qb), np.repeat(f64(Kb), g, axis=1), np.repeat(f64(Vb), g, axis=1)
    for b in range(B):
        nb = lens[b]
        for h in range(Hq):
            S = 0.3 * (Q[b, :nb, h] @ K[b, h, :nb].T)
            i, j = np.meshgrid(np.arange(nb), np.arange(nb), indexing="ij")
            mask = (j < i) if mode == 0 else (j <= i)
            for r in range(nb):
                cols = np.nonzero(mask[r])[0]
                if cols.size == 0:
                    assert not out[b, r, h].any()
                    continue
                e = np.exp(S[r, cols] - S[r, cols].max()); p = e / e.sum()
                np.testing.assert_allclose(out[b, r, h], p @ V[b, h, cols], atol=1e-12)
        assert not out[b, nb:].any()          # rows past the prompt are untouched


def test_prefill_standard_mode_is_sdpa_causal():
    B, n, Hq, Hkv, d = 2, 11, 4, 4, 16
    qb, Kb, Vb = rand_bits((B, n, Hq, d), 4), rand_bits((B, Hkv, n, d), 5), rand_bits((B, Hkv, n, d), 6)
    lens = np.full(B, n, np.int32)
    out = orc.prefill_attention(qb, Kb, Vb, lens, 1, d ** -0.5)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(f64(qb)).transpose(1, 2), torch.from_numpy(f64(Kb)), torch.from_numpy(f64(Vb)),
        is_causal=True).transpose(1, 2).numpy()
    np.testing.assert_allclose(out, ref, atol=1e-12)


def test_first_iteration_pairs_with_zero_kv():
    """Before the first iteration the shared cache holds the dummy zero vectors (Section 2.2.1):
    every condensed layer's output is zero, and the write of the new k,v is bit-exact."""
    L, B, n, Hq, Hkv, d, T = 3, 2, 6, 2, 1, 8, 8
    lens = np.array([6, 4], np.int32)
    qs = [rand_bits((B, n, Hq, d), 10 + l) for l in range(L)]
    k, v = rand_bits((B, n, Hkv, d), 20), rand_bits((B, n, Hkv, d), 21)
    K = np.zeros((B, Hkv, T, d), np.uint16); V = np.zeros_like(K)
    outs = orc.prefill_iteration(L, 0, qs, [None, None, k], [None, None, v], [K], [V], lens, 0.5)
    assert all(not o.any() for o in outs)
    for b in range(B):
        assert np.array_equal(K[b, 0, :lens[b]], k[b, :lens[b], 0])
        assert np.array_equal(V[b, 0, :lens[b]], v[b, :lens[b], 0])
        assert not K[b, 0, lens[b]:].any()


class ToyModel:
    """A tiny random-weight LCKV decoder in float64: residual stream h, per layer
    q = h Wq, (k, v = h Wk, h Wv for layers that have K/V), h += tanh(attn Wo).  q, k, v are rounded
    to bf16 (the oracle's input type).  Projections are done token by token so that the sequential
    and the parallel computation perform bit-identical arithmetic."""

    def __init__(self, L, w, Hq, Hkv, d, hidden, seed, variant=0):
        r = np.random.default_rng(seed)
        self.L, self.w, self.Hq, self.Hkv, self.d, self.variant = L, w, Hq, Hkv, d, variant
        self.plan = orc.plan(L, w, variant)
        self.Wq = r.normal(size=(L, hidden, Hq * d)) / np.sqrt(hidden)
        self.Wk = r.normal(size=(L, hidden, Hkv * d)) / np.sqrt(hidden)
        self.Wv = r.normal(size=(L, hidden, Hkv * d)) / np.sqrt(hidden)
        self.Wo = r.normal(size=(L, Hq * d, hidden)) / np.sqrt(Hq * d)
        self.scale = d ** -0.5

    def proj(self, H, W):
        return np.stack([h @ W for h in H])

    def decode_all(self, X, T_cap):
        """Token by token (Section 2.2: 'decoding one token at a time').  Returns final hidden
        states [n, hidden] and the caches."""
        n = X.shape[0]
        ns = self.plan["n_slots"]
        K = [np.zeros((1, self.Hkv, T_cap, self.d), np.uint16) for _ in range(ns)]
        V = [np.zeros_like(K[0]) for _ in range(ns)]
        lens = np.zeros(1, np.int32)
        out_h = []
        for t in range(n):
            h = X[t:t + 1]
            late = None
            for l in range(self.L):
                q = to_bits(self.proj(h, self.Wq[l]).reshape(1, self.Hq, self.d))
                ws = self.plan["write_slot"][l]
                if ws >= 0:
                    k = to_bits(self.proj(h, self.Wk[l]).reshape(1, self.Hkv, self.d))
                    v = to_bits(self.proj(h, self.Wv[l]).reshape(1, self.Hkv, self.d))
                    if self.plan["write_before"][l]:
                        orc.append(K[ws], V[ws], k, v, lens)
                    else:
                        late = (ws, k, v)
                rs = self.plan["read_slot"][l]
                a, _ = orc.decode_attention(q, K[rs], V[rs], lens, self.plan["mode"][l], self.scale)
                h = h + np.tanh(a.reshape(1, -1) @ self.Wo[l])
            if late:
                orc.append(K[late[0]], V[late[0]], late[1], late[2], lens)
            lens += 1
            out_h.append(h[0])
        return np.stack(out_h), K, V

    def iterate(self, X, K, V, lens):
        """One parallel iteration over all prompt tokens (Section 2.2.1 / 2.3)."""
        n = X.shape[0]
        H = X.copy()
        late = None
        for l in range(self.L):
            q = to_bits(self.proj(H, self.Wq[l]).reshape(1, n, self.Hq, self.d))
            ws = self.plan["write_slot"][l]
            if ws >= 0:
                k = to_bits(self.proj(H, self.Wk[l]).reshape(1, n, self.Hkv, self.d))
                v = to_bits(self.proj(H, self.Wv[l]).reshape(1, n, self.Hkv, self.d))
                if self.plan["write_before"][l]:
                    orc.prefill_write_kv(K[ws], V[ws], k, v, lens)
                else:
                    late = (ws, k, v)
            rs = self.plan["read_slot"][l]
            a = orc.prefill_attention(q, K[rs], V[rs], lens, self.plan["mode"][l], self.scale)
            H = H + np.tanh(np.stack([x.reshape(-1) @ self.Wo[l] for x in a[0]]))
        if late:
            orc.prefill_write_kv(K[late[0]], V[late[0]], late[1], late[2], lens)
        return H


@pytest.mark.parametrize("L,w,variant", [(3, 0, 0), (4, 2, 0), (4, 2, 1), (3, 3, 0)])
def test_lemma_parallel_iterations_reproduce_sequential_decoding(L, w, variant):
    """Appendix A: in the parallel computation token i is correct from iteration i on, whatever the
    initial k,v; after n iterations everything equals token-by-token decoding - hidden states and
    every cache bit.  This ties the prefill functions to the decode functions."""
    n, T_cap = 7, 8
    m = ToyModel(L, w, Hq=2, Hkv=1, d=8, hidden=12, seed=5 + L + w, variant=variant)
    X = np.random.default_rng(99).normal(size=(n, 12))
    H_seq, K_seq, V_seq = m.decode_all(X, T_cap)
    ns = m.plan["n_slots"]
    K = [np.zeros((1, 1, T_cap, 8), np.uint16) for _ in range(ns)]
    V = [np.zeros_like(K[0]) for _ in range(ns)]
    lens = np.array([n], np.int32)
    for it in range(1, n + 1):
        H = m.iterate(X, K, V, lens)
        # tokens 0 .. it-1 are final after iteration `it`
        assert np.array_equal(H[:it], H_seq[:it]), it
    assert np.array_equal(H, H_seq)
    for s in range(ns):
        assert np.array_equal(K[s], K_seq[s]) and np.array_equal(V[s], V_seq[s])
    if w < L:   # ... and one iteration is NOT enough (the test can tell the difference)
        K1 = [np.zeros((1, 1, T_cap, 8), np.uint16) for _ in range(ns)]
        V1 = [np.zeros_like(K1[0]) for _ in range(ns)]
        assert not np.array_equal(m.iterate(X, K1, V1, lens), H_seq)


def test_prefill_iteration_is_the_plan_applied_layer_by_layer():
    """The stack-level function equals the per-layer functions composed by hand along the plan."""
    L, w, B, n, Hq, Hkv, d, T = 4, 2, 2, 5, 2, 2, 8, 6
    p = orc.plan(L, w)
    lens = np.array([5, 3], np.int32)
    qs = [rand_bits((B, n, Hq, d), 40 + l) for l in range(L)]
    ks = [rand_bits((B, n, Hkv, d), 50 + l) if p["write_slot"][l] >= 0 else None for l in range(L)]
    vs = [rand_bits((B, n, Hkv, d), 60 + l) if p["write_slot"][l] >= 0 else None for l in range(L)]
    K0 = [rand_bits((B, Hkv, T, d), 70 + s) for s in range(p["n_slots"])]
    V0 = [rand_bits((B, Hkv, T, d), 80 + s) for s in range(p["n_slots"])]
    Ka, Va = [k.copy() for k in K0], [v.copy() for v in V0]
    outs = orc.prefill_iteration(L, w, qs, ks, vs, Ka, Va, lens, 0.4)
    Kb, Vb = [k.copy() for k in K0], [v.copy() for v in V0]
    for l in range(L):
        if p["write_slot"][l] >= 0 and p["write_before"][l]:
            orc.prefill_write_kv(Kb[p["write_slot"][l]], Vb[p["write_slot"][l]], ks[l], vs[l], lens)
        o = orc.prefill_attention(qs[l], Kb[p["read_slot"][l]], Vb[p["read_slot"][l]], lens,
                                  p["mode"][l], 0.4)
        assert np.array_equal(o, outs[l])
    for l in range(L):
        if p["write_slot"][l] >= 0 and not p["write_before"][l]:
            orc.prefill_write_kv(Kb[p["write_slot"][l]], Vb[p["write_slot"][l]], ks[l], vs[l], lens)
    assert all(np.array_equal(a, b) for a, b in zip(Ka + Va, Kb + Vb))
