"""ctypes/numpy front end of the float64 CPU oracle (oracle/lckv_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
CPU-baseline leg of the benchmark.  Nothing here touches CUDA, and the CUDA
package never imports this module.

bf16 tensors travel as numpy uint16 arrays holding the raw bits.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

_LIB = None


def lib():
    global _LIB
    if _LIB is None:
        path = _build.build()
        L = C.CDLL(path)
        u16p, i32p, f64p = C.POINTER(C.c_uint16), C.POINTER(C.c_int32), C.POINTER(C.c_double)
        L.lckv_oracle_plan.argtypes = [C.c_int, C.c_int, C.c_int] + [i32p] * 6
        L.lckv_oracle_plan.restype = C.c_int
        L.lckv_oracle_attend_row.argtypes = [u16p, u16p, u16p, C.c_int64, C.c_int, C.c_double,
                                             C.c_int, f64p, f64p, f64p]
        L.lckv_oracle_attend_row.restype = C.c_int
        L.lckv_oracle_decode_attention.argtypes = [u16p, u16p, u16p, i32p, C.c_int, C.c_int,
                                                   C.c_int, C.c_int64, C.c_int, C.c_int,
                                                   C.c_double, C.c_int, C.c_int, f64p, f64p]
        L.lckv_oracle_decode_attention.restype = C.c_int
        L.lckv_oracle_append.argtypes = [u16p, u16p, u16p, u16p, i32p, C.c_int, C.c_int,
                                         C.c_int64, C.c_int, C.c_int]
        L.lckv_oracle_append.restype = C.c_int
        pp = C.POINTER(C.c_void_p)
        L.lckv_oracle_stack_step.argtypes = [C.c_int, C.c_int, C.c_int, pp, pp, pp, pp, pp, i32p,
                                             C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int,
                                             C.c_double, C.c_int, C.c_int, pp, pp]
        L.lckv_oracle_stack_step.restype = C.c_int
        L.lckv_oracle_prefill_attention.argtypes = [u16p, u16p, u16p, i32p, C.c_int, C.c_int,
                                                    C.c_int, C.c_int, C.c_int64, C.c_int, C.c_int,
                                                    C.c_double, C.c_int, f64p]
        L.lckv_oracle_prefill_attention.restype = C.c_int
        L.lckv_oracle_prefill_write_kv.argtypes = [u16p, u16p, u16p, u16p, i32p, C.c_int, C.c_int,
                                                   C.c_int, C.c_int64, C.c_int]
        L.lckv_oracle_prefill_write_kv.restype = C.c_int
        L.lckv_oracle_prefill_iteration.argtypes = [C.c_int, C.c_int, C.c_int, pp, pp, pp, pp, pp,
                                                    i32p, C.c_int, C.c_int, C.c_int, C.c_int,
                                                    C.c_int64, C.c_int, C.c_double, C.c_int, pp]
        L.lckv_oracle_prefill_iteration.restype = C.c_int
        f32p = C.POINTER(C.c_float)
        f64p = C.POINTER(C.c_double)
        L.lckv_oracle_project_kv.argtypes = [u16p, u16p, u16p, f32p, f32p, C.c_int, i32p, C.c_int,
                                             C.c_int, C.c_int, C.c_int, u16p, u16p, f64p, f64p]
        L.lckv_oracle_project_kv.restype = C.c_int
        L.lckv_oracle_num_threads.restype = C.c_int
        _LIB = L
    return _LIB


class OracleError(RuntimeError):
    pass


def _chk(rc, what):
    if rc != 0:
        raise OracleError(f"{what}: oracle status {rc} ({ {1: 'EINVAL', 2: 'ECAPACITY'}.get(rc, '?') })")


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _p(a, ct):
    return a.ctypes.data_as(C.POINTER(ct))


def num_threads():
    return int(lib().lckv_oracle_num_threads())


def plan(L, w, top_variant=0):
    """Layer plan (Section 2.1 sandwich rule).  Returns a dict of int32 arrays + n_slots."""
    arrs = [np.zeros(L, np.int32) for _ in range(5)]
    n = np.zeros(1, np.int32)
    rc = lib().lckv_oracle_plan(L, w, top_variant, *[_p(a, C.c_int32) for a in arrs],
                                _p(n, C.c_int32))
    _chk(rc, "plan")
    keys = ["is_warmup", "read_slot", "mode", "write_slot", "write_before"]
    out = dict(zip(keys, arrs))
    out["n_slots"] = int(n[0])
    return out


def attend_row(q, K, V, scale, always_sink=False, want_probs=False):
    """One query q[d] against K,V [n, d] (uint16 bf16 bits).  Returns (o, lse[, probs])."""
    q, K, V = _u16(q), _u16(K), _u16(V)
    d = q.shape[-1]
    n = K.shape[0] if K.size else 0
    o = np.zeros(d, np.float64)
    lse = np.zeros(1, np.float64)
    probs = np.zeros(n + 1, np.float64)
    rc = lib().lckv_oracle_attend_row(_p(q, C.c_uint16), _p(K, C.c_uint16), _p(V, C.c_uint16),
                                      n, d, float(scale), int(always_sink), _p(o, C.c_double),
                                      _p(lse, C.c_double), _p(probs, C.c_double))
    _chk(rc, "attend_row")
    return (o, float(lse[0]), probs) if want_probs else (o, float(lse[0]))


def decode_attention(q, K, V, lens, mode, scale, always_sink=False, n_sink=0):
    """q [B,Hq,d], K,V [B,Hkv,Tcap,d] uint16, lens [B] int32 -> (out [B,Hq,d], lse [B,Hq]) float64."""
    q, K, V = _u16(q), _u16(K), _u16(V)
    lens = np.ascontiguousarray(lens, np.int32)
    B, Hq, d = q.shape
    _, Hkv, Tcap, _ = K.shape
    assert K.shape[0] >= B and V.shape == K.shape
    out = np.zeros((B, Hq, d), np.float64)
    lse = np.zeros((B, Hq), np.float64)
    rc = lib().lckv_oracle_decode_attention(_p(q, C.c_uint16), _p(K, C.c_uint16),
                                            _p(V, C.c_uint16), _p(lens, C.c_int32), B, Hq, Hkv,
                                            Tcap, d, int(mode), float(scale), int(always_sink),
                                            int(n_sink), _p(out, C.c_double), _p(lse, C.c_double))
    _chk(rc, "decode_attention")
    return out, lse


def append(K, V, k_new, v_new, lens, n_sink=0):
    """In place: row lens[b] of K,V [B,Hkv,Tcap,d] <- k_new, v_new [B,Hkv,d]."""
    assert K.flags.c_contiguous and V.flags.c_contiguous and K.dtype == np.uint16
    k_new, v_new = _u16(k_new), _u16(v_new)
    lens = np.ascontiguousarray(lens, np.int32)
    B, Hkv, d = k_new.shape
    rc = lib().lckv_oracle_append(_p(K, C.c_uint16), _p(V, C.c_uint16), _p(k_new, C.c_uint16),
                                  _p(v_new, C.c_uint16), _p(lens, C.c_int32), B, Hkv,
                                  K.shape[2], d, int(n_sink))
    _chk(rc, "append")


def _ptr_array(arrs):
    t = (C.c_void_p * len(arrs))()
    for i, a in enumerate(arrs):
        t[i] = None if a is None else a.ctypes.data
    return C.cast(t, C.POINTER(C.c_void_p))


def stack_step(L, w, q_layers, k_new_layers, v_new_layers, K_slots, V_slots, lens, scale,
               top_variant=0, always_sink=False, n_sink=0):
    """One decode step of the whole stack; caches and lens are updated in place.

    q_layers: list of L arrays [B,Hq,d]; k_new_layers/v_new_layers: list of L arrays
    [B,Hkv,d] or None; K_slots/V_slots: list of caches [Bmax,Hkv,Tcap,d]; lens int32 [B].
    Returns (outs, lses): lists of L float64 arrays.
    """
    q_layers = [_u16(q) for q in q_layers]
    k_new_layers = [None if k is None else _u16(k) for k in k_new_layers]
    v_new_layers = [None if v is None else _u16(v) for v in v_new_layers]
    for a in list(K_slots) + list(V_slots):
        assert a.flags.c_contiguous and a.dtype == np.uint16
    assert lens.dtype == np.int32 and lens.flags.c_contiguous
    B, Hq, d = q_layers[0].shape
    _, Hkv, Tcap, _ = K_slots[0].shape
    outs = [np.zeros((B, Hq, d), np.float64) for _ in range(L)]
    lses = [np.zeros((B, Hq), np.float64) for _ in range(L)]
    rc = lib().lckv_oracle_stack_step(L, w, int(top_variant), _ptr_array(q_layers),
                                      _ptr_array(k_new_layers), _ptr_array(v_new_layers),
                                      _ptr_array(K_slots), _ptr_array(V_slots),
                                      _p(lens, C.c_int32), B, Hq, Hkv, Tcap, d, float(scale),
                                      int(always_sink), int(n_sink), _ptr_array(outs),
                                      _ptr_array(lses))
    _chk(rc, "stack_step")
    return outs, lses


def prefill_attention(q, K, V, lens, mode, scale, always_sink=False):
    """Token-parallel attention of one layer (prompt encoding, Section 2.3).
    q [B,n_max,Hq,d], K,V [B,Hkv,Tcap,d] uint16, lens [B] -> out [B,n_max,Hq,d] float64
    (rows i >= lens[b] are zero)."""
    q, K, V = _u16(q), _u16(K), _u16(V)
    lens = np.ascontiguousarray(lens, np.int32)
    B, n_max, Hq, d = q.shape
    _, Hkv, Tcap, _ = K.shape
    out = np.zeros((B, n_max, Hq, d), np.float64)
    rc = lib().lckv_oracle_prefill_attention(_p(q, C.c_uint16), _p(K, C.c_uint16),
                                             _p(V, C.c_uint16), _p(lens, C.c_int32), B, n_max, Hq,
                                             Hkv, Tcap, d, int(mode), float(scale),
                                             int(always_sink), _p(out, C.c_double))
    _chk(rc, "prefill_attention")
    return out


def prefill_write_kv(K, V, k, v, lens):
    """In place: rows [0, lens[b]) of K,V [B,Hkv,Tcap,d] <- k, v [B,n_max,Hkv,d]."""
    assert K.flags.c_contiguous and V.flags.c_contiguous and K.dtype == np.uint16
    k, v = _u16(k), _u16(v)
    lens = np.ascontiguousarray(lens, np.int32)
    B, n_max, Hkv, d = k.shape
    rc = lib().lckv_oracle_prefill_write_kv(_p(K, C.c_uint16), _p(V, C.c_uint16),
                                            _p(k, C.c_uint16), _p(v, C.c_uint16),
                                            _p(lens, C.c_int32), B, n_max, Hkv, K.shape[2], d)
    _chk(rc, "prefill_write_kv")


def prefill_iteration(L, w, q_layers, k_layers, v_layers, K_slots, V_slots, lens, scale,
                      top_variant=0, always_sink=False):
    """One parallel iteration over the stack; caches updated in place.  Returns the list of L
    outputs [B,n_max,Hq,d] float64."""
    q_layers = [_u16(q) for q in q_layers]
    k_layers = [None if k is None else _u16(k) for k in k_layers]
    v_layers = [None if v is None else _u16(v) for v in v_layers]
    for a in list(K_slots) + list(V_slots):
        assert a.flags.c_contiguous and a.dtype == np.uint16
    lens = np.ascontiguousarray(lens, np.int32)
    B, n_max, Hq, d = q_layers[0].shape
    _, Hkv, Tcap, _ = K_slots[0].shape
    outs = [np.zeros((B, n_max, Hq, d), np.float64) for _ in range(L)]
    rc = lib().lckv_oracle_prefill_iteration(L, w, int(top_variant), _ptr_array(q_layers),
                                             _ptr_array(k_layers), _ptr_array(v_layers),
                                             _ptr_array(K_slots), _ptr_array(V_slots),
                                             _p(lens, C.c_int32), B, n_max, Hq, Hkv, Tcap, d,
                                             float(scale), int(always_sink), _ptr_array(outs))
    _chk(rc, "prefill_iteration")
    return outs


def project_kv(x, w_k, w_v, lens, n_kv_heads, head_dim, rope_cos=None, rope_sin=None):
    """Keys and values of the new token from hidden states: x [B, d_model], w_k / w_v
    [H_kv*d, d_model] (bf16 bits); optional rotary tables [n_pos, d/2] float32 applied to the key at
    position lens[b].  Returns (k_bits, v_bits [B, H_kv, d] uint16, k_f64, v_f64 the unrounded values)."""
    x, w_k, w_v = _u16(x), _u16(w_k), _u16(w_v)
    lens = np.ascontiguousarray(lens, np.int32)
    B, d_model = x.shape
    F = n_kv_heads * head_dim
    assert w_k.shape == (F, d_model) and w_v.shape == (F, d_model)
    k_bits = np.empty((B, n_kv_heads, head_dim), np.uint16)
    v_bits = np.empty_like(k_bits)
    k_f = np.empty((B, n_kv_heads, head_dim), np.float64)
    v_f = np.empty_like(k_f)
    cp = sp = None
    n_pos = 0
    if rope_cos is not None:
        rope_cos = np.ascontiguousarray(rope_cos, np.float32)
        rope_sin = np.ascontiguousarray(rope_sin, np.float32)
        assert rope_cos.shape == rope_sin.shape and rope_cos.shape[1] == head_dim // 2
        n_pos = rope_cos.shape[0]
        cp, sp = _p(rope_cos, C.c_float), _p(rope_sin, C.c_float)
    rc = lib().lckv_oracle_project_kv(_p(x, C.c_uint16), _p(w_k, C.c_uint16), _p(w_v, C.c_uint16),
                                      cp, sp, n_pos, _p(lens, C.c_int32), B, n_kv_heads, head_dim,
                                      d_model, _p(k_bits, C.c_uint16), _p(v_bits, C.c_uint16),
                                      _p(k_f, C.c_double), _p(v_f, C.c_double))
    _chk(rc, "project_kv")
    return k_bits, v_bits, k_f, v_f
