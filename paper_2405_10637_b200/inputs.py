"""Seeded synthetic inputs for the LCKV decode path: shapes, lengths and Gaussian tensors.

This module holds no arithmetic of the method.  It only draws random numbers and
describes workload shapes, so the CUDA library's tests, the benchmark and the CPU
checker can all be fed the same bits.  Shapes follow the paper's model table
(Appendix B: 1.1B, 7B and 30B Llama configurations) and the prompt+generation
length pairs of its throughput table (Section 3.1).
"""
from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    cfg_id: int          # seeds are 1000 * cfg_id + tensor id
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_warmup: int
    std: float           # standard deviation of q, k, v entries

    def with_(self, **kw):
        return replace(self, **kw)


# tensor ids for seeding
T_LENS, T_K, T_V, T_Q, T_KNEW, T_VNEW = range(6)

WORKLOADS = {
    # 4-layer toy stack, MHA, w = 0
    "toy": Workload("toy", 1, 4, 4, 4, 64, 0, 1.0),
    # TinyLlama-1.1B shape: 22 layers, 32 q heads, 4 kv heads, d_h 64
    "tinyllama": Workload("tinyllama", 2, 22, 32, 4, 64, 2, 64 ** -0.5),
    # Llama-7B shape: 32 layers, 32 heads, d_h 128
    "llama7b": Workload("llama7b", 3, 32, 32, 32, 128, 2, 1.0),
    # Llama-30B shape: 60 layers, 52 heads, d_h 128
    "llama30b": Workload("llama30b", 4, 60, 52, 52, 128, 2, 1.0),
    # warmup-count / long-context sweep on the 7B shape
    "sweep7b": Workload("sweep7b", 5, 32, 32, 32, 128, 2, 1.0),
    # a grouped-query layout outside the paper's models (groups of 4: 32 q heads, 8 kv heads, d_h 128),
    # to time query groups smaller than the 8-wide tensor-core tile
    "gqa4": Workload("gqa4", 6, 32, 32, 8, 128, 2, 1.0),
}


def seed_for(wl: Workload, tensor_id: int, extra: int = 0) -> int:
    """Seed of one tensor of a workload.  The toy case draws everything from seed 0
    (one generator, tensors in the order K, V, q, k_new, v_new: see draw_sequence)."""
    if wl.cfg_id == 1:
        return 0
    return 1000 * wl.cfg_id + tensor_id + 100000 * extra


def draw_sequence(shapes, seed: int, device="cpu", std: float = 1.0):
    """Several bf16 Gaussian tensors drawn one after another from ONE seeded generator."""
    g = torch.Generator(device=device).manual_seed(seed)
    out = []
    for shp in shapes:
        x = torch.randn(shp, generator=g, device=device, dtype=torch.float32)
        if std != 1.0:
            x = x * std
        out.append(x.to(torch.bfloat16))
    return out


def ragged_lengths(batch: int, lo: int, hi: int, seed: int) -> torch.Tensor:
    """Per-sequence cached lengths, integers uniform in [lo, hi], int32 on the CPU."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    return torch.randint(lo, hi + 1, (batch,), generator=g, dtype=torch.int64).to(torch.int32)


def randn_bf16(shape, seed: int, device="cpu", std: float = 1.0) -> torch.Tensor:
    """N(0, std^2) in bf16 (drawn in fp32, scaled, rounded to nearest even)."""
    g = torch.Generator(device=device).manual_seed(seed)
    x = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if std != 1.0:
        x = x * std
    return x.to(torch.bfloat16)


def fill_randn_bf16_(dst: torch.Tensor, seed: int, std: float = 1.0, chunk_elems: int = 1 << 28):
    """Fill a (possibly huge) bf16 tensor in place, chunked along dim 0 to bound temporaries."""
    assert dst.dtype == torch.bfloat16
    g = torch.Generator(device=dst.device).manual_seed(seed)
    flat = dst.view(-1) if dst.is_contiguous() else None
    if flat is None:
        raise ValueError("fill_randn_bf16_ needs a contiguous tensor")
    n = flat.numel()
    for s in range(0, n, chunk_elems):
        e = min(n, s + chunk_elems)
        x = torch.randn(e - s, generator=g, device=dst.device, dtype=torch.float32)
        if std != 1.0:
            x = x * std
        flat[s:e].copy_(x)
    return dst


def bits(t: torch.Tensor) -> np.ndarray:
    """Raw bf16 bits of a tensor as a numpy uint16 array on the host."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    """Inverse of bits()."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)


def shard_batch(total_batch: int, rank: int, world: int):
    """Contiguous batch shard [start, stop) of this rank: sequences are independent."""
    base, rem = divmod(total_batch, world)
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)


def shard_heads(n_kv_heads: int, rank: int, world: int):
    """Contiguous kv-head shard [start, stop) of this rank; a rank takes whole kv heads, hence whole
    query groups (q heads [start * g, stop * g)), so no rank needs another's keys or values."""
    if n_kv_heads % world:
        raise ValueError(f"{n_kv_heads} kv heads do not split evenly over {world} ranks")
    per = n_kv_heads // world
    return rank * per, (rank + 1) * per
