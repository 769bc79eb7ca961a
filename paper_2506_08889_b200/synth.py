"""Seeded synthetic inputs shaped like the decode workloads the library is measured on.

This module only *draws* data (tensors, lengths, index lists, page tables) and names
the workload shapes.  It holds none of the method's arithmetic, so that both the GPU
path and the CPU checker can be fed from it without sharing any computation.

Everything is a pure function of ``(seed, tensor name)``; values are drawn once (on the
device asked for) and handed to whoever needs them, so the two sides of a comparison
always see the same bits.
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import List, Optional

import numpy as np
import torch

BASE_SEED = 20250608


def _gen(seed: int, name: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + zlib.crc32(name.encode())) % (2 ** 63 - 1))
    return g


def normal_bf16(shape, seed: int, name: str, device="cpu", std: float = 1.0,
                chunk_elems: int = 1 << 28) -> torch.Tensor:
    """i.i.d. N(0, std^2) rounded to bf16, drawn in bounded chunks."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    g = _gen(seed, name, device)
    n = flat.numel()
    for s in range(0, n, chunk_elems):
        e = min(n, s + chunk_elems)
        tmp = torch.randn(e - s, generator=g, device=device, dtype=torch.float32)
        if std != 1.0:
            tmp.mul_(std)
        flat[s:e] = tmp.to(torch.bfloat16)
    return out


def normal_f32(shape, seed: int, name: str, device="cpu") -> torch.Tensor:
    return torch.randn(shape, generator=_gen(seed, name, device), device=device,
                       dtype=torch.float32)


def np_rng(seed: int, name: str) -> np.random.Generator:
    return np.random.default_rng([seed, zlib.crc32(name.encode())])


def ragged_lengths(batch: int, lo: int, hi: int, multiple: int, seed: int,
                   name: str = "seq_lens") -> np.ndarray:
    """Lengths uniform in [lo, hi], each a multiple of ``multiple``."""
    r = np_rng(seed, name)
    return (r.integers(lo // multiple, hi // multiple + 1, size=batch) * multiple).astype(np.int32)


def random_block_lists(seq_lens, num_kv_heads: int, block_size: int, k_per_unit,
                       max_sel: int, seed: int, name: str = "block_idx",
                       shuffle: bool = False):
    """Per (sequence, KV head): ``k`` distinct blocks, the last block always among them.

    Returns (block_idx [B,Hkv,max_sel] int32 padded with -1, block_cnt [B,Hkv] int32).
    Lists are ascending unless ``shuffle``.
    """
    r = np_rng(seed, name)
    B = len(seq_lens)
    idx = np.full((B, num_kv_heads, max_sel), -1, np.int32)
    cnt = np.zeros((B, num_kv_heads), np.int32)
    for i in range(B):
        n = (int(seq_lens[i]) + block_size - 1) // block_size
        k = int(k_per_unit[i] if np.ndim(k_per_unit) else k_per_unit)
        k = max(0, min(k, n, max_sel))
        for h in range(num_kv_heads):
            if k == 0 or n == 0:
                continue
            others = r.choice(n - 1, size=k - 1, replace=False) if k > 1 else np.empty(0, np.int64)
            sel = np.concatenate([others, [n - 1]]).astype(np.int32)
            sel = r.permutation(sel) if shuffle else np.sort(sel)
            idx[i, h, :k] = sel
            cnt[i, h] = k
    return idx, cnt


def page_permutation(num_pages: int, seed: int, name: str = "page_table") -> np.ndarray:
    return np_rng(seed, name).permutation(num_pages).astype(np.int32)


def keep_count(n_blocks: int, sparsity: float) -> int:
    """Blocks kept when a fraction ``sparsity`` of a sequence's blocks is skipped."""
    return int(n_blocks - int(np.floor(sparsity * n_blocks + 1e-9)))


@dataclasses.dataclass
class Workload:
    """Shape of one synthetic decode workload (one attention layer, one new token)."""
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    block_size: int
    seq_len: int                      # fixed length, or the maximum when ragged
    seq_len_min: Optional[int] = None  # set -> ragged lengths in [min, seq_len]
    ragged_multiple: int = 128
    token_budget: Optional[int] = None
    sparsity: Optional[float] = None
    selected_blocks: Optional[int] = None
    d_gate: int = 128
    rope_theta: float = 1.0e6
    gate_weight_std: float = 0.02

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def sm_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))

    def lengths(self, seed: int = BASE_SEED) -> np.ndarray:
        if self.seq_len_min is None:
            return np.full(self.batch, self.seq_len, np.int32)
        return ragged_lengths(self.batch, self.seq_len_min, self.seq_len,
                              self.ragged_multiple, seed, self.name + ":lens")

    def keep(self, n_blocks: int) -> int:
        if self.selected_blocks is not None:
            return min(self.selected_blocks, n_blocks)
        if self.token_budget is not None:
            return min(max(1, self.token_budget // self.block_size), n_blocks)
        if self.sparsity is not None:
            return keep_count(n_blocks, self.sparsity)
        return n_blocks


# The five workloads the library is specified on.  Head counts follow Qwen3-4B/8B/14B
# attention layers; the kernel benchmark they stand in for is the paper's Sec. 4.4 grid
# (random selections at a sparsity ratio over fixed shapes).
def workloads() -> List[Workload]:
    return [
        Workload("tiny", 1, 4, 1, 128, 64, 4096, selected_blocks=8),
        Workload("qwen3_8b_l32k_budget4k", 1, 32, 8, 128, 64, 32768, token_budget=4096),
        Workload("qwen3_14b_l64k_gate_budget4k", 1, 40, 8, 128, 64, 65536, token_budget=4096),
        Workload("qwen3_4b_b16_ragged_s90", 16, 32, 8, 128, 128, 65536, seq_len_min=8192,
                 sparsity=0.9),
        Workload("qwen3_14b_b8_l128k_sweep", 8, 40, 8, 128, 64, 131072, sparsity=0.9),
    ]


def workload(name_or_index) -> Workload:
    ws = workloads()
    if isinstance(name_or_index, int):
        return ws[name_or_index]
    for w in ws:
        if w.name == name_or_index:
            return w
    raise KeyError(name_or_index)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """Raw bit patterns of a bf16 tensor as a numpy uint16 array (host copy, same strides)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
