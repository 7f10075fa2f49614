"""Host-side logic of bench.py that needs no GPU: workload parameters and the scaling of the captured
DRAM counters to a launch's size."""
import argparse
import importlib.util
import os

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def args_for(**kw):
    base = dict(workload="llama7b", batch=0, context=0, warmup_layers=None, stream_sink=0, page_rows=0,
                steps=10, warmup=3, shard="")
    base.update(kw)
    return argparse.Namespace(**base)


def test_workload_parameters(bench):
    wl, p = bench.workload_params(args_for())
    assert (wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.n_warmup) == (32, 32, 32, 128, 2)
    assert p["batch"] == 512 and p["lo"] == 256 and p["hi"] == 4096
    assert p["t_cap"] >= 4096 + 13                      # room for the tokens the run appends
    assert p["sweep"] == [8, 16, 32, 64, 128, 256, 512]
    wl, p = bench.workload_params(args_for(workload="sweep7b", warmup_layers=8, batch=8, context=32768))
    assert wl.n_warmup == 8 and p["batch"] == 8 and p["lo"] == p["hi"] == 32768
    wl, p = bench.workload_params(args_for(workload="tinyllama"))
    assert (wl.n_q_heads, wl.n_kv_heads, wl.head_dim) == (32, 4, 64) and p["batch"] == 128


def test_traffic_is_scaled_from_the_capture_only_where_it_applies(bench):
    alg = 17.9e9
    out = 512 * 32 * 128 * 2
    caps = bench.load_captures()
    t = bench.scaled_traffic("attn_alu_kernel", args_for(), alg, out, caps, check_sources=False)
    assert alg < t < 1.01 * alg                          # every K/V byte once, plus partials and write-backs
    f = lambda k, a, x, o: bench.scaled_traffic(k, a, x, o, caps, check_sources=False)
    assert f("attn_alu_kernel", args_for(page_rows=256), alg, out) is None
    assert f("attn_mma_kernel", args_for(workload="tinyllama"), 135.3e6, 524288) is not None
    assert f("attn_mma_kernel", args_for(workload="tinyllama", context=512), 67e6, 524288) is None


def test_captured_counters_are_the_ones_in_the_summaries(bench):
    """bench.py takes the DRAM counters from profiles/ncu_captures.json; the figures there must be the
    ones the ncu summaries beside it print (to the precision they print)."""
    caps = bench.load_captures()
    for name in ("attn_alu_kernel", "attn_mma_kernel"):
        cap = caps[name]
        text = open(os.path.join(ROOT, cap["source"])).read()
        rows = {ln.split("|")[1].strip(): [c.strip() for c in ln.split("|")[2:-1]]
                for ln in text.splitlines() if ln.startswith("| `dram__bytes")}
        reads = [float(c.split()[0]) * 1e6 for c in rows["`dram__bytes_read.sum`"]]
        writes = [float(c.split()[0]) * 1e6 for c in rows["`dram__bytes_write.sum`"]]
        assert min(reads) - 0.02e6 <= cap["dram_read_bytes"] <= max(reads) + 0.02e6
        assert min(writes) - 0.02e6 <= cap["dram_write_bytes"] <= max(writes) + 0.02e6
        assert cap["output_bytes"] < cap["dram_write_bytes"] < 0.05 * cap["dram_read_bytes"]
        assert 0.9 * cap["dram_read_bytes"] < cap["algorithmic_input_bytes"] <= cap["dram_read_bytes"]
        for src in cap["sources"]:
            assert os.path.exists(os.path.join(bench.CSRC, src))


def test_a_capture_is_void_once_the_kernel_changed(bench):
    caps = bench.load_captures()
    caps = {k: dict(v) if isinstance(v, dict) else v for k, v in caps.items()}
    caps["attn_alu_kernel"]["sources_digest"] = bench.source_digest(caps["attn_alu_kernel"]["sources"])
    assert bench.scaled_traffic("attn_alu_kernel", args_for(), 17.9e9, 4e6, caps) is not None
    caps["attn_alu_kernel"]["sources_digest"] = "0" * 16
    assert bench.scaled_traffic("attn_alu_kernel", args_for(), 17.9e9, 4e6, caps) is None


def test_largest_batch_that_fits(bench):
    from paper_2405_10637_b200 import inputs as syn
    wl = syn.WORKLOADS["llama30b"]
    assert bench.largest_batch(wl, 4096, 2) == 825      # 109.05 MB per sequence and cache
    assert bench.largest_batch(wl, 4096, 3) == 550
    wl = syn.WORKLOADS["sweep7b"]
    assert bench.largest_batch(wl, 8192, 32) == 41      # the standard transformer's 32 caches: 64 do not fit
