"""The N > 1 path on CPU (gloo, world size 2): batch sharding is exact and needs no data-path
collective; timing aggregation is max over ranks, throughput is the sum of units over that time."""
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
