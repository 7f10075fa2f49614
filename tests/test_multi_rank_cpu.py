"""The N > 1 path on CPU (gloo, world size 2): sharding one batch by sequences or by kv heads is exact
(the union of the ranks' results is the one-rank result, bit for bit) and needs no data-path collective; timing aggregation is max over ranks, throughput is the sum of units over that time."""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np

from paper_2405_10637_b200 import inputs as syn

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import sys, numpy as np, torch, torch.distributed as dist
    sys.path.insert(0, %(root)r)
    from paper_2405_10637_b200 import inputs as syn, multi
    from oracle import lckv_oracle as orc
    multi.init("gloo")
    r, w = multi.rank(), multi.world()
    B, Hq, Hkv, T, d = 5, 4, 2, 40, 16
    K = syn.bits(syn.randn_bf16((B, Hkv, T, d), 1)); V = syn.bits(syn.randn_bf16((B, Hkv, T, d), 2))
    q = syn.bits(syn.randn_bf16((B, Hq, d), 3))
    lens = np.array([0, 7, 39, 16, 1], np.int32)
    lo, hi = syn.shard_batch(B, r, w)
    out, _ = orc.decode_attention(q[lo:hi], K[lo:hi], V[lo:hi], lens[lo:hi], 0, 0.25)
    full, _ = orc.decode_attention(q, K, V, lens, 0, 0.25)
    assert np.array_equal(out, full[lo:hi])          # a shard needs nothing from the other rank
    parts = [None] * w
    dist.all_gather_object(parts, (lo, hi))
    if r == 0:
        covered = sorted(parts)
        assert covered[0][0] == 0 and covered[-1][1] == B
        assert all(a[1] == b[0] for a, b in zip(covered, covered[1:]))
    # both shard rules, whole stack step: each rank steps ITS shard of one batch with the oracle; the
    # union of the ranks' outputs, caches and lengths is what one rank computes for the whole batch
    L, wm = 4, 2
    qs = [syn.bits(syn.randn_bf16((B, Hq, d), 10 + l)) for l in range(L)]
    plan = orc.plan(L, wm)
    kn = [syn.bits(syn.randn_bf16((B, Hkv, d), 20 + l)) if plan["write_slot"][l] >= 0 else None for l in range(L)]
    vn = [syn.bits(syn.randn_bf16((B, Hkv, d), 30 + l)) if plan["write_slot"][l] >= 0 else None for l in range(L)]
    Ks = [syn.bits(syn.randn_bf16((B, Hkv, T, d), 40 + s)) for s in range(plan["n_slots"])]
    Vs = [syn.bits(syn.randn_bf16((B, Hkv, T, d), 50 + s)) for s in range(plan["n_slots"])]
    ln = np.array([0, 7, 38, 16, 1], np.int32)
    cp = lambda xs: [None if x is None else np.ascontiguousarray(x) for x in xs]
    fK, fV, fl = cp(Ks), cp(Vs), ln.copy()
    full_out, _ = orc.stack_step(L, wm, qs, kn, vn, fK, fV, fl, 0.25)
    g = Hq // Hkv
    for rule in ("batch", "heads"):
        if rule == "batch":
            (b0, b1), (h0, h1) = syn.shard_batch(B, r, w), (0, Hkv)
        else:
            (b0, b1), (h0, h1) = (0, B), syn.shard_heads(Hkv, r, w)
        cut = lambda x, hs: None if x is None else np.ascontiguousarray(x[b0:b1, hs[0]:hs[1]])
        sK = [cut(x, (h0, h1)) for x in Ks]; sV = [cut(x, (h0, h1)) for x in Vs]
        sl = ln[b0:b1].copy()
        out, _ = orc.stack_step(L, wm, [cut(x, (h0 * g, h1 * g)) for x in qs], [cut(x, (h0, h1)) for x in kn],
                                [cut(x, (h0, h1)) for x in vn], sK, sV, sl, 0.25)
        got = [None] * w
        dist.all_gather_object(got, (b0, b1, h0, h1, out, sK, sV, sl))
        if r == 0:
            uo = [np.full_like(x, np.nan) for x in full_out]
            uK = [np.zeros_like(x) for x in fK]; uV = [np.zeros_like(x) for x in fV]
            ul = np.full(B, -1, np.int32)
            for (a0, a1, c0, c1, o, pk, pv, pl) in got:
                for l in range(L):
                    uo[l][a0:a1, c0 * g:c1 * g] = o[l]
                for s in range(len(fK)):
                    uK[s][a0:a1, c0:c1] = pk[s]; uV[s][a0:a1, c0:c1] = pv[s]
                ul[a0:a1] = pl
            for l in range(L):
                assert np.array_equal(uo[l], full_out[l]), (rule, l)
            for s in range(len(fK)):
                assert np.array_equal(uK[s], fK[s]) and np.array_equal(uV[s], fV[s]), (rule, s)
            assert np.array_equal(ul, fl), rule
    ms = 10.0 + 5.0 * r                               # rank 1 is the slow one
    assert multi.max_over_ranks(ms) == 15.0
    thr = multi.job_throughput(float(hi - lo), ms)
    assert abs(thr - B / 15e-3) < 1e-6
    multi.barrier()
    dist.destroy_process_group()
    print("rank", r, "ok")
""")


def test_shard_batch_partitions_exactly():
    for B in (1, 5, 8, 512, 513):
        for w in (1, 2, 3, 8):
            parts = [syn.shard_batch(B, r, w) for r in range(w)]
            assert parts[0][0] == 0 and parts[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
            sizes = [b - a for a, b in parts]
            assert max(sizes) - min(sizes) <= 1


def test_shard_heads_takes_whole_query_groups():
    for Hkv, w in ((4, 1), (4, 2), (4, 4), (32, 8), (52, 4)):
        parts = [syn.shard_heads(Hkv, r, w) for r in range(w)]
        assert parts[0][0] == 0 and parts[-1][1] == Hkv
        assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
        assert len({b - a for a, b in parts}) == 1
    import pytest
    with pytest.raises(ValueError):
        syn.shard_heads(52, 0, 8)


def test_two_ranks_gloo():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    script = WORKER % {"root": ROOT}
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", LOCAL_RANK=str(r),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, "-c", script], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    for r, p in enumerate(procs):
        out, _ = p.communicate(timeout=240)
        assert p.returncode == 0, out
        assert f"rank {r} ok" in out
