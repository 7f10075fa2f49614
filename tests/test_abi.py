"""Host-side checks of the C ABI that need no GPU: the library loads, exports what the header
declares, and its layer plan equals the oracle's (and the hand-enumerated sets)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import lckv_oracle as orc
from paper_2405_10637_b200 import binding as lk

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_symbols():
    text = open(os.path.join(ROOT, "include", "lckv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lckv_[a-z_]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    lib = lk.lib()
    names = header_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/lckv.h but not exported"
    assert set(names) == set(lk.SIGNATURES), "binding and header disagree on the entry points"


def test_status_strings():
    lib = lk.lib()
    assert lib.lckv_status_string(0) == b"ok"
    for s in range(1, 6):
        assert len(lib.lckv_status_string(s)) > 3


@pytest.mark.parametrize("variant", [0, 1])
@pytest.mark.parametrize("L,w", [(4, 0), (4, 2), (4, 4), (22, 2), (22, 10), (32, 8), (60, 2), (1, 0)])
def test_plan_matches_oracle(L, w, variant):
    got = lk.lckv_plan(L, w, variant)
    want = orc.plan(L, w, variant)
    for k in ("is_warmup", "read_slot", "mode", "write_slot", "write_before"):
        assert got[k] == want[k].tolist(), k
    assert got["n_slots"] == want["n_slots"]


def test_plan_rejects_bad_arguments():
    for L, w, v in [(4, 1, 0), (4, 3, 0), (4, 6, 0), (0, 0, 0), (4, 2, 2), (4, -2, 0)]:
        with pytest.raises(lk.LckvError) as e:
            lk.lckv_plan(L, w, v)
        assert e.value.status == lk.EINVAL
    arr = (C.c_int32 * 4)()
    n = C.c_int32()
    assert lk.lib().lckv_plan(4, 2, 0, None, arr, arr, arr, arr, C.byref(n)) == lk.EINVAL


def test_null_and_invalid_handles_return_errors_without_a_gpu():
    lib = lk.lib()
    assert lib.lckv_cache_free(None) == lk.EINVAL
    assert lib.lckv_cache_info(None, None) == lk.EINVAL
    assert lib.lckv_decode_attention(None, 0, 0, None, None, None, 1, None) == lk.EINVAL
    assert lib.lckv_append_kv(None, 0, None, None, 1, 0, None) == lk.EINVAL
    assert lib.lckv_layer_stack_step(None, None, None, None, None, 1, None) == lk.EINVAL
    bad = lk.make_config(4, 1, 4, 4, 64, 2, 16)   # odd w
    assert lib.lckv_cache_bytes(C.byref(bad)) == 0
    bad = lk.make_config(4, 2, 4, 3, 64, 2, 16)   # H_q % H_kv != 0
    assert lib.lckv_cache_bytes(C.byref(bad)) == 0
    bad = lk.make_config(4, 2, 4, 4, 96, 2, 16)   # unsupported head_dim
    assert lib.lckv_cache_bytes(C.byref(bad)) == 0


def test_static_entry_refuses_bad_arguments_before_touching_a_gpu():
    """The allocation-free entry point checks its arguments before any CUDA call, so a pointer that
    would fault on the device (off the 16-byte grid of the bulk copies and vector accesses) or a size
    beyond the fixed scratch comes back as an error code.  The pointers here are never dereferenced."""
    f = lk.lib().lckv_decode_attention_static
    a = 0x10000     # a plausible, aligned address

    def call(k=a, v=a, lens=a, q=a, out=a, lse=None, status=None, batch=4, hq=8, hkv=8, d=128, T=64, mode=0,
             scale=0.0, odt=0):
        return f(k, v, lens, q, out, lse, status, batch, hq, hkv, d, T, mode, scale, odt, None)
    for name in ("k", "v", "q", "out"):
        assert call(**{name: a + 8}) == lk.EINVAL, name       # 8-byte aligned is not enough
        assert call(**{name: a + 2}) == lk.EINVAL, name
        assert call(**{name: None}) == lk.EINVAL, name
    assert call(lens=a + 2) == lk.EINVAL
    assert call(lens=None) == lk.EINVAL
    assert call(lse=a + 1) == lk.EINVAL
    assert call(status=a + 2) == lk.EINVAL
    assert call(batch=0) == lk.EINVAL
    assert call(hkv=3) == lk.EINVAL
    assert call(d=96) == lk.EINVAL
    assert call(T=0) == lk.EINVAL
    assert call(T=1 << 31) == lk.EINVAL
    assert call(mode=2) == lk.EINVAL
    assert call(odt=2) == lk.EINVAL
    assert call(scale=-1.0) == lk.EINVAL
    assert call(scale=float("nan")) == lk.EINVAL
    assert call(batch=4097) == lk.ESTATICLIMIT


def test_wait_limit_call_checks_its_handle():
    assert lk.lib().lckv_cache_set_wait_limit(None, 0) == lk.EINVAL
    assert lk.lib().lckv_cache_set_worker_limit(None, 0) == lk.EINVAL
