"""ctypes binding of liblckv.so: the same entry points as include/lckv.h, argument marshalling only.

Tensors are torch CUDA tensors (torch supplies device memory and streams); every step of the
computation runs in the library's own kernels.  There is no fallback: if the library is missing
or does not load, the first call raises.
"""
import ctypes as C
import os

import torch

from . import build as _build

OK, EINVAL, ECAPACITY, ENOMEM, ECUDA, ETIMEOUT, ESTATICLIMIT = range(7)
MODE_CONDENSED, MODE_STANDARD = 0, 1


class Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_layers", C.c_int32), ("n_warmup", C.c_int32),
                ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("max_batch", C.c_int32), ("max_seq", C.c_int32), ("softmax_scale", C.c_float),
                ("top_variant", C.c_int32), ("out_dtype", C.c_int32), ("host_staging", C.c_int32),
                ("use_graph", C.c_int32), ("stream_sink", C.c_int32), ("page_rows", C.c_int32), ("n_pages", C.c_int32),
                ("kernel_kind", C.c_int32)]


class Info(C.Structure):
    _fields_ = [("n_slots", C.c_int32), ("n_workers", C.c_int32), ("rows_per_tile", C.c_int32),
                ("kernel_kind", C.c_int32), ("launches_per_step", C.c_int32),
                ("sm_count", C.c_int32), ("slot_bytes", C.c_uint64),
                ("workspace_bytes", C.c_uint64)]


# name -> (restype, argtypes); also the list of symbols the header declares
_vp, _i32, _i32p = C.c_void_p, C.c_int32, C.POINTER(C.c_int32)
_vpp = C.POINTER(C.c_void_p)
SIGNATURES = {
    "lckv_plan": (C.c_int, [_i32, _i32, _i32, _i32p, _i32p, _i32p, _i32p, _i32p, _i32p]),
    "lckv_cache_bytes": (C.c_size_t, [C.POINTER(Config)]),
    "lckv_cache_alloc": (C.c_int, [_vpp, C.POINTER(Config), _vp, C.c_size_t]),
    "lckv_cache_free": (C.c_int, [_vp]),
    "lckv_cache_info": (C.c_int, [_vp, C.POINTER(Info)]),
    "lckv_cache_reset": (C.c_int, [_vp, _i32p, _i32, _vp]),
    "lckv_cache_lengths": (C.c_int, [_vp, _i32p, _i32, _vp]),
    "lckv_cache_status": (C.c_int, [_vp, _i32p, _vp]),
    "lckv_cache_set_wait_limit": (C.c_int, [_vp, C.c_uint32]),
    "lckv_cache_set_worker_limit": (C.c_int, [_vp, _i32]),
    "lckv_cache_slot_ptrs": (C.c_int, [_vp, _i32, _vpp, _vpp]),
    "lckv_cache_page_table": (C.c_int, [_vp, _i32p, _i32p]),
    "lckv_append_kv": (C.c_int, [_vp, _i32, _vp, _vp, _i32, _i32, _vp]),
    "lckv_project_append_kv": (C.c_int, [_vp, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _vp]),
    "lckv_decode_attention": (C.c_int, [_vp, _i32, _i32, _vp, _vp, _vp, _i32, _vp]),
    "lckv_layer_stack_step": (C.c_int, [_vp, _vpp, _vpp, _vpp, _vpp, _i32, _vp]),
    "lckv_layer_stack_step_host": (C.c_int, [_vp, _vpp, _vpp, _vpp, _vpp, _i32, _vp]),
    "lckv_prefill_write_kv": (C.c_int, [_vp, _i32, _vp, _vp, _i32, _i32, _vp]),
    "lckv_prefill_attention": (C.c_int, [_vp, _i32, _i32, _vp, _vp, _i32, _i32, _vp]),
    "lckv_prefill_iteration": (C.c_int, [_vp, _vpp, _vpp, _vpp, _vpp, _i32, _i32, _vp]),
    "lckv_decode_attention_static": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32,
                                              _i32, C.c_int64, _i32, C.c_float, _i32, _vp]),
    "lckv_read_stream_probe": (C.c_int, [_vp, C.c_size_t, _i32, _i32, C.c_float, _vp, _vp, _vp]),
    "lckv_status_string": (C.c_char_p, [C.c_int]),
    "lckv_last_cuda_error": (C.c_int, []),
}

_LIB = None


def lib():
    """Load (building first if the sources are newer) the CUDA library.  Raises if impossible."""
    global _LIB
    if _LIB is None:
        path = _build.build()
        L = C.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _LIB = L
    return _LIB


class LckvError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        msg = lib().lckv_status_string(status).decode()
        extra = f", cudaError {lib().lckv_last_cuda_error()}" if status == ECUDA else ""
        super().__init__(f"{what}: {msg} (status {status}{extra})")


def _chk(rc, what):
    if rc != OK:
        raise LckvError(rc, what)


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _ptr_array(ts):
    arr = (C.c_void_p * len(ts))()
    for i, t in enumerate(ts):
        arr[i] = None if t is None else t.data_ptr()
    return C.cast(arr, _vpp)


def lckv_plan(n_layers, n_warmup, top_variant=0):
    """Host-only layer plan; returns a dict of lists + n_slots."""
    arrs = [(C.c_int32 * max(n_layers, 1))() for _ in range(5)]
    n = C.c_int32(0)
    rc = lib().lckv_plan(n_layers, n_warmup, top_variant, *arrs, C.byref(n))
    _chk(rc, "lckv_plan")
    keys = ["is_warmup", "read_slot", "mode", "write_slot", "write_before"]
    out = {k: list(a)[:n_layers] for k, a in zip(keys, arrs)}
    out["n_slots"] = n.value
    return out


def make_config(n_layers, n_warmup, n_q_heads, n_kv_heads, head_dim, max_batch, max_seq,
                softmax_scale=0.0, top_variant=0, out_dtype=0, host_staging=0, use_graph=0,
                kernel_kind=0, stream_sink=0, page_rows=0, n_pages=0):
    return Config(C.sizeof(Config), n_layers, n_warmup, n_q_heads, n_kv_heads, head_dim,
                  max_batch, max_seq, softmax_scale, top_variant, out_dtype, host_staging,
                  use_graph, stream_sink, page_rows, n_pages, kernel_kind)


def lckv_cache_bytes(cfg):
    return int(lib().lckv_cache_bytes(C.byref(cfg)))


def lckv_decode_attention_static(k, v, lens, q, out, mode, lse=None, dev_status=None,
                                 softmax_scale=0.0, stream=None):
    """Decode attention for callers that must not allocate: k, v [B, H_kv, T_cap, d_h] bf16,
    lens [B] int32, q [B, H_q, d_h] bf16 and `out` (bf16 or fp32, caller-provided) are CUDA
    tensors; the library's scratch is a fixed array inside its device image, so nothing is
    allocated here or there.  One call at a time per GPU: all calls share that scratch."""
    B, Hkv, T_cap, d = k.shape
    Hq = q.shape[1]
    rc = lib().lckv_decode_attention_static(
        _ptr(k), _ptr(v), _ptr(lens), _ptr(q), _ptr(out), _ptr(lse), _ptr(dev_status), q.shape[0],
        Hq, Hkv, d, T_cap, mode, softmax_scale, 1 if out.dtype == torch.float32 else 0,
        _stream(stream))
    _chk(rc, "lckv_decode_attention_static")
    return out


def lckv_read_stream_probe(src, nbytes, kind, dev_sum, dev_status, repeats=1, l2_keep=0.0, stream=None):
    """Read-only stream over the first nbytes of the CUDA tensor `src`, `repeats` passes in one launch;
    dev_sum (uint32/int32 [1]) and dev_status (int32 [1]) are CUDA tensors."""
    _chk(lib().lckv_read_stream_probe(_ptr(src), nbytes, kind, repeats, l2_keep, _ptr(dev_sum),
                                      _ptr(dev_status), _stream(stream)), "lckv_read_stream_probe")


class Cache:
    """Owner of one lckv_cache_t and of the torch buffer behind it."""

    def __init__(self, cfg, device="cuda:0"):
        self.cfg = cfg
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            nbytes = lckv_cache_bytes(cfg)
            if nbytes == 0:
                raise LckvError(EINVAL, "lckv_cache_bytes")
            self.buf = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            h = C.c_void_p()
            _chk(lib().lckv_cache_alloc(C.byref(h), C.byref(cfg), _ptr(self.buf), nbytes),
                 "lckv_cache_alloc")
        self.h = h
        info = Info()
        _chk(lib().lckv_cache_info(self.h, C.byref(info)), "lckv_cache_info")
        self.info = info
        self.out_torch_dtype = torch.float32 if cfg.out_dtype else torch.bfloat16

    def close(self):
        if getattr(self, "h", None):
            lib().lckv_cache_free(self.h)
            self.h = None
            self.buf = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C entry points, same names ---------------------------------------------------------
    def lckv_cache_reset(self, host_lens=None, batch=None, stream=None):
        if host_lens is not None:
            arr = (C.c_int32 * len(host_lens))(*[int(x) for x in host_lens])
            batch = len(host_lens) if batch is None else batch
            rc = lib().lckv_cache_reset(self.h, arr, batch, _stream(stream))
        else:
            rc = lib().lckv_cache_reset(self.h, None, batch or self.cfg.max_batch, _stream(stream))
        _chk(rc, "lckv_cache_reset")

    def lckv_cache_lengths(self, batch=None, stream=None):
        batch = batch or self.cfg.max_batch
        arr = (C.c_int32 * batch)()
        _chk(lib().lckv_cache_lengths(self.h, arr, batch, _stream(stream)), "lckv_cache_lengths")
        return list(arr)

    def lckv_cache_status(self, stream=None):
        s = C.c_int32(0)
        _chk(lib().lckv_cache_status(self.h, C.byref(s), _stream(stream)), "lckv_cache_status")
        return s.value

    def lckv_cache_set_wait_limit(self, polls):
        _chk(lib().lckv_cache_set_wait_limit(self.h, polls), "lckv_cache_set_wait_limit")

    def lckv_cache_set_worker_limit(self, workers):
        _chk(lib().lckv_cache_set_worker_limit(self.h, workers), "lckv_cache_set_worker_limit")

    def lckv_cache_slot_ptrs(self, slot):
        k, v = C.c_void_p(), C.c_void_p()
        _chk(lib().lckv_cache_slot_ptrs(self.h, slot, C.byref(k), C.byref(v)),
             "lckv_cache_slot_ptrs")
        return k.value, v.value

    def lckv_cache_page_table(self):
        """Paged caches: torch int64 tensor [B_max, entries_per_seq] of page ids (-1 = none)."""
        n = C.c_int32(0)
        _chk(lib().lckv_cache_page_table(self.h, None, C.byref(n)), "lckv_cache_page_table")
        arr = (C.c_int32 * (self.cfg.max_batch * n.value))()
        _chk(lib().lckv_cache_page_table(self.h, arr, C.byref(n)), "lckv_cache_page_table")
        return torch.tensor(list(arr), dtype=torch.int64).view(self.cfg.max_batch, n.value)

    def slot_tensors(self, slot):
        """torch views of a slot's K and V (same memory): [B_max, H_kv, T_cap, d_h] bf16, or
        [n_pages, H_kv, page_rows, d_h] for a paged cache."""
        k, v = self.lckv_cache_slot_ptrs(slot)
        c = self.cfg
        shape = (c.max_batch, c.n_kv_heads, c.max_seq, c.head_dim)
        if c.page_rows:
            shape = (c.n_pages, c.n_kv_heads, c.page_rows, c.head_dim)
        n = 2 * shape[0] * shape[1] * shape[2] * shape[3]
        base = self.buf.data_ptr()
        kt = self.buf[k - base:k - base + n].view(torch.bfloat16).view(shape)
        vt = self.buf[v - base:v - base + n].view(torch.bfloat16).view(shape)
        return kt, vt

    def lckv_append_kv(self, slot, k_new, v_new, batch=None, advance_len=0, stream=None):
        batch = k_new.shape[0] if batch is None else batch
        _chk(lib().lckv_append_kv(self.h, slot, _ptr(k_new), _ptr(v_new), batch, advance_len,
                                  _stream(stream)), "lckv_append_kv")

    def lckv_project_append_kv(self, slot, x, w_k, w_v, rope_cos=None, rope_sin=None, batch=None,
                               advance_len=0, stream=None):
        """x [batch, d_model], w_k / w_v [H_kv*d_h, d_model] bf16 device tensors; optional rotary
        tables [positions, d_h/2] fp32."""
        batch = x.shape[0] if batch is None else batch
        n_pos = 0 if rope_cos is None else rope_cos.shape[0]
        _chk(lib().lckv_project_append_kv(self.h, slot, _ptr(x), x.shape[1], _ptr(w_k), _ptr(w_v),
                                          _ptr(rope_cos), _ptr(rope_sin), n_pos, batch, advance_len,
                                          _stream(stream)), "lckv_project_append_kv")

    def lckv_decode_attention(self, slot, mode, q, out=None, lse=None, batch=None, stream=None):
        batch = q.shape[0] if batch is None else batch
        if out is None:
            out = torch.empty(q.shape, dtype=self.out_torch_dtype, device=q.device)
        _chk(lib().lckv_decode_attention(self.h, slot, mode, _ptr(q), _ptr(out), _ptr(lse), batch,
                                         _stream(stream)), "lckv_decode_attention")
        return out

    def lckv_layer_stack_step(self, q_layers, out_layers, k_new_layers, v_new_layers, batch=None,
                              stream=None):
        batch = q_layers[0].shape[0] if batch is None else batch
        _chk(lib().lckv_layer_stack_step(self.h, _ptr_array(q_layers), _ptr_array(out_layers),
                                         _ptr_array(k_new_layers), _ptr_array(v_new_layers),
                                         batch, _stream(stream)), "lckv_layer_stack_step")

    def lckv_layer_stack_step_host(self, q_layers, out_layers, k_new_layers, v_new_layers,
                                   batch=None, stream=None):
        """Same, with HOST (ideally pinned) torch tensors."""
        batch = q_layers[0].shape[0] if batch is None else batch
        _chk(lib().lckv_layer_stack_step_host(self.h, _ptr_array(q_layers),
                                              _ptr_array(out_layers), _ptr_array(k_new_layers),
                                              _ptr_array(v_new_layers), batch, _stream(stream)),
             "lckv_layer_stack_step_host")

    # -- prompt encoding (token-major tensors [B, n_max, H, d_h]) -------------------------------
    def lckv_prefill_write_kv(self, slot, k, v, stream=None):
        _chk(lib().lckv_prefill_write_kv(self.h, slot, _ptr(k), _ptr(v), k.shape[1], k.shape[0],
                                         _stream(stream)), "lckv_prefill_write_kv")

    def lckv_prefill_attention(self, slot, mode, q, out=None, stream=None):
        if out is None:
            out = torch.zeros(q.shape, dtype=self.out_torch_dtype, device=q.device)
        _chk(lib().lckv_prefill_attention(self.h, slot, mode, _ptr(q), _ptr(out), q.shape[1],
                                          q.shape[0], _stream(stream)), "lckv_prefill_attention")
        return out

    def lckv_prefill_iteration(self, q_layers, out_layers, k_layers, v_layers, stream=None):
        q0 = q_layers[0]
        _chk(lib().lckv_prefill_iteration(self.h, _ptr_array(q_layers), _ptr_array(out_layers),
                                          _ptr_array(k_layers), _ptr_array(v_layers), q0.shape[1],
                                          q0.shape[0], _stream(stream)), "lckv_prefill_iteration")
