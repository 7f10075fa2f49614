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
                steps=10, warmup=3)
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
    t = bench.scaled_traffic("attn_alu_kernel", args_for(), alg, out)
    assert alg < t < 1.01 * alg                          # every K/V byte once, plus partials and write-backs
    assert bench.scaled_traffic("attn_alu_kernel", args_for(page_rows=256), alg, out) is None
    assert bench.scaled_traffic("attn_mma_kernel", args_for(workload="tinyllama"), 135.3e6, 524288) is not None
    assert bench.scaled_traffic("attn_mma_kernel", args_for(workload="tinyllama", context=512), 67e6, 524288) is None
    for cap in bench.NCU_CAPTURES.values():
        assert os.path.exists(os.path.join(ROOT, cap["source"]))
