"""Shared machinery of the GPU parity tests: build a cache, fill it, step it, compare with the oracle."""
import numpy as np
import torch

from oracle import lckv_oracle as orc
from paper_2405_10637_b200 import binding as lk
from paper_2405_10637_b200 import inputs as syn

MAX_ABS = 1e-2     # tolerance on |gpu - oracle| per element
REL_L2 = 5e-3      # tolerance on ||gpu - oracle||_2 / ||oracle||_2
NAN_BITS = 0x7FC0  # bf16 quiet NaN, used to poison rows that must never be read


def bf16_tolerance(want):
    """Per-element bound on |gpu - oracle| for a bf16 output: MAX_ABS, except where the value is so
    large that one rounding to bf16 alone can exceed it.  In the binade [4, 8) half an ulp is 2^-6 =
    0.0156 > MAX_ABS (below 4 it is at most 0.0078, so the plain bound is attainable there); such
    elements - they occur with N(0,1) values at contexts of a few tokens - get 2^-8 |o|, between half
    an ulp and one ulp of their binade."""
    a = np.abs(want)
    return np.where(a >= 4.0, a * 2.0 ** -8, MAX_ABS)


def compare(got, want, what=""):
    """got: torch tensor (bf16/fp32) from the GPU; want: float64 numpy from the oracle.
    Returns the observed (max-abs, rel-L2), as measured."""
    g = got.detach().float().cpu().numpy().astype(np.float64)
    assert g.shape == want.shape, (g.shape, want.shape)
    assert np.isfinite(g).all(), f"{what}: non-finite GPU output"
    zero_rows = ~want.any(axis=-1)
    assert not g[zero_rows].any(), f"{what}: rows the oracle gives as exactly 0 are not 0"
    err = np.abs(g - want)
    max_abs = float(err.max()) if g.size else 0.0
    tol = bf16_tolerance(want) if got.dtype == torch.bfloat16 else MAX_ABS
    excess = err - tol
    if g.size:
        i = np.unravel_index(np.argmax(excess), excess.shape)
        assert excess[i] <= 0, f"{what}: |gpu - oracle| = {err[i]:.3e} at {i} (oracle {want[i]:.4f})"
    denom = np.linalg.norm(want[~zero_rows])
    rel = float(np.linalg.norm((g - want)[~zero_rows]) / denom) if denom > 0 else 0.0
    assert rel <= REL_L2, f"{what}: rel-L2 {rel:.3e}"
    return max_abs, rel


class Case:
    """One layer stack with GPU cache and host (oracle) caches holding the same bits."""

    def __init__(self, L, w, Hq, Hkv, d, lens, T_cap, variant=0, out_dtype=0, seed=1234, std=1.0,
                 poison=True, B_max=None, scale=0.0, kernel_kind=0, host_staging=0, use_graph=0,
                 stream_sink=0, page_rows=0, n_pages=0):
        self.L, self.w, self.Hq, self.Hkv, self.d = L, w, Hq, Hkv, d
        self.lens = np.asarray(lens, np.int32).copy()
        self.B = len(lens)
        self.T_cap, self.variant, self.seed, self.std = T_cap, variant, seed, std
        B_max = B_max or self.B
        self.cfg = lk.make_config(L, w, Hq, Hkv, d, B_max, T_cap, softmax_scale=scale,
                                  top_variant=variant, out_dtype=out_dtype, kernel_kind=kernel_kind,
                                  host_staging=host_staging, use_graph=use_graph,
                                  stream_sink=stream_sink, page_rows=page_rows, n_pages=n_pages)
        self.stream_sink = stream_sink
        self.page_rows = page_rows
        self.scale = scale if scale > 0 else d ** -0.5
        self.cache = lk.Cache(self.cfg)
        self.plan = orc.plan(L, w, variant)
        self.n_slots = self.plan["n_slots"]
        assert self.cache.info.n_slots == self.n_slots
        self.hK, self.hV = [], []
        if page_rows:
            # pages are assigned on reset; a first reset with the lengths reversed leaves the free
            # list in a different order, so the final assignment is not simply 0, 1, 2, ...
            self.cache.lckv_cache_reset(self.lens[::-1].tolist())
            self.cache.lckv_cache_reset(self.lens.tolist())
        for s in range(self.n_slots):
            kb = syn.bits(syn.randn_bf16((B_max, Hkv, T_cap, d), seed + 2 * s, std=std))
            vb = syn.bits(syn.randn_bf16((B_max, Hkv, T_cap, d), seed + 2 * s + 1, std=std))
            if poison:
                for b in range(B_max):
                    n = min(int(self.lens[b]), T_cap) if b < self.B else 0
                    kb[b, :, n:] = NAN_BITS
                    vb[b, :, n:] = NAN_BITS
            kt, vt = self.cache.slot_tensors(s)
            if page_rows:
                kt.copy_(syn.from_bits(np.full(tuple(kt.shape), NAN_BITS, np.uint16)))
                vt.copy_(kt)
                self._scatter(kt, kb); self._scatter(vt, vb)
            else:
                kt.copy_(syn.from_bits(kb)); vt.copy_(syn.from_bits(vb))
            self.hK.append(kb); self.hV.append(vb)
        if not page_rows:
            self.cache.lckv_cache_reset(self.lens.tolist())
        self.step_no = 0

    def step_inputs(self):
        s0 = self.seed + 1000 * (self.step_no + 1)
        q = [syn.randn_bf16((self.B, self.Hq, self.d), s0 + l, std=self.std) for l in range(self.L)]
        kn = [syn.randn_bf16((self.B, self.Hkv, self.d), s0 + 200 + l, std=self.std)
              if self.plan["write_slot"][l] >= 0 else None for l in range(self.L)]
        vn = [syn.randn_bf16((self.B, self.Hkv, self.d), s0 + 400 + l, std=self.std)
              if self.plan["write_slot"][l] >= 0 else None for l in range(self.L)]
        return q, kn, vn

    def step(self, check=True, host=False, contiguous=False):
        q, kn, vn = self.step_inputs()
        odt = torch.float32 if self.cfg.out_dtype else torch.bfloat16
        if host:
            if contiguous:   # one pinned block per tensor kind, sliced per layer
                qa = torch.stack(q).pin_memory()
                qd = [qa[l] for l in range(self.L)]
                idx = [l for l in range(self.L) if kn[l] is not None]
                ka = torch.stack([kn[l] for l in idx]).pin_memory()
                va = torch.stack([vn[l] for l in idx]).pin_memory()
                knd, vnd = [None] * self.L, [None] * self.L
                for i, l in enumerate(idx):
                    knd[l], vnd[l] = ka[i], va[i]
                oa = torch.empty((self.L, self.B, self.Hq, self.d), dtype=odt).pin_memory()
                outs = [oa[l] for l in range(self.L)]
            else:
                qd = [t.pin_memory() for t in q]
                knd = [None if t is None else t.pin_memory() for t in kn]
                vnd = [None if t is None else t.pin_memory() for t in vn]
                outs = [torch.empty((self.B, self.Hq, self.d), dtype=odt).pin_memory()
                        for _ in range(self.L)]
            self.cache.lckv_layer_stack_step_host(qd, outs, knd, vnd)
        else:
            dev = self.cache.device
            qd = [t.to(dev) for t in q]
            knd = [None if t is None else t.to(dev) for t in kn]
            vnd = [None if t is None else t.to(dev) for t in vn]
            outs = [torch.full((self.B, self.Hq, self.d), float("nan"), dtype=odt, device=dev)
                    for _ in range(self.L)]
            self.cache.lckv_layer_stack_step(qd, outs, knd, vnd)
        torch.cuda.synchronize()
        assert self.cache.lckv_cache_status() == 0
        want, _ = orc.stack_step(self.L, self.w, [syn.bits(t) for t in q],
                                 [None if t is None else syn.bits(t) for t in kn],
                                 [None if t is None else syn.bits(t) for t in vn],
                                 self.hK, self.hV, self.lens, self.scale, top_variant=self.variant,
                                 n_sink=self.stream_sink)
        self.step_no += 1
        stats = []
        if check:
            for l in range(self.L):
                stats.append(compare(outs[l], want[l], f"layer {l} step {self.step_no}"))
            self.check_state()
        return outs, want, stats

    def _scatter(self, pool, logical_bits):
        """Paged cache: copy the logical rows [B, Hkv, T_cap, d] into the pages each sequence owns."""
        P = self.page_rows
        pt = self.cache.lckv_cache_page_table()
        for b in range(pt.shape[0]):
            for i in range(pt.shape[1]):
                pg = int(pt[b, i])
                if pg < 0:
                    break
                rows = logical_bits[b, :, i * P:(i + 1) * P]
                pool[pg, :, :rows.shape[1]].copy_(syn.from_bits(rows))

    def _gather(self, pool, b):
        """Paged cache: the logical rows sequence b owns, [Hkv, n_owned_rows, d] as bits."""
        pt = self.cache.lckv_cache_page_table()
        pages = [int(x) for x in pt[b] if int(x) >= 0]
        if not pages:
            return np.zeros((self.Hkv, 0, self.d), np.uint16)
        return np.concatenate([syn.bits(pool[pg]) for pg in pages], axis=1)

    def check_state(self):
        """Lengths and every byte of every cache, bit for bit."""
        assert self.cache.lckv_cache_lengths(self.B) == self.lens.tolist()
        for s in range(self.n_slots):
            kt, vt = self.cache.slot_tensors(s)
            if self.page_rows:
                for b in range(self.B):
                    gk, gv = self._gather(kt, b), self._gather(vt, b)
                    n = min(gk.shape[1], self.T_cap)
                    assert n >= min(int(self.lens[b]), self.T_cap)
                    assert np.array_equal(gk[:, :n], self.hK[s][b][:, :n]), f"slot {s} seq {b} K differs"
                    assert np.array_equal(gv[:, :n], self.hV[s][b][:, :n]), f"slot {s} seq {b} V differs"
                continue
            assert np.array_equal(syn.bits(kt), self.hK[s]), f"slot {s} K differs"
            assert np.array_equal(syn.bits(vt), self.hV[s]), f"slot {s} V differs"

    def close(self):
        self.cache.close()
