"""Seeded synthetic inputs for the speculative-step attention path.

This module holds only input construction -- none of the attention arithmetic -- so the CUDA path,
the CPU oracle's tests and the benchmark can all draw the same tensors from it.  Everything is a
pure function of (seed, tensor id, element index): a counter-based splitmix64 stream evaluated with
integer torch ops, which give bit-identical results on CPU and on a CUDA device.  N(0,1) values come
from a 65,536-entry inverse-CDF table of bf16 values indexed by the top 16 bits of the stream (the
tails are therefore clipped near +-4.2 sigma).

The shapes follow a Qwen2-VL-7B-like decoder (28 query heads, 4 KV heads, head_dim 128) at the
paper's long-video sequence lengths (about 25k visual tokens, more than 99 % of the context), with
draft trees of a few dozen nodes.  These synthetic tensors stand in for the video benchmarks the
paper evaluates on; no benchmark item is reproduced.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

BASE_SEED = 260215318
HQ, HKV, D = 28, 4, 128
GROUP = HQ // HKV
SCALE = 1.0 / math.sqrt(D)

_M64 = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _s64(x: int) -> int:
    """Two's-complement reinterpretation of an unsigned 64-bit value."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def splitmix64(x: int) -> int:
    """One splitmix64 output for the 64-bit state ``x`` (host integers)."""
    z = (x + _GOLD) & _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, tensor_id: int) -> int:
    """Per-tensor key: every tensor of a case gets its own stream."""
    return splitmix64((seed & _M64) ^ ((tensor_id & 0xFF) << 56))


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def splitmix64_tensor(key: int, start: int, n: int, device) -> torch.Tensor:
    """splitmix64(key + i) for i in [start, start+n) as int64 bit patterns."""
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    z = idx + _s64(key) + _s64(_GOLD)
    z = (z ^ _lsr(z, 30)) * _s64(_C1)
    z = (z ^ _lsr(z, 27)) * _s64(_C2)
    return z ^ _lsr(z, 31)


_TABLE_CPU: Optional[torch.Tensor] = None
_TABLES = {}


def normal_table(device) -> torch.Tensor:
    """bf16 inverse-CDF table: entry i is the N(0,1) quantile at (i + 1/2) / 65536."""
    global _TABLE_CPU
    if _TABLE_CPU is None:
        from scipy.special import ndtri
        p = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
        _TABLE_CPU = torch.from_numpy(ndtri(p).astype(np.float32)).to(torch.bfloat16)
    key = str(device)
    if key not in _TABLES:
        _TABLES[key] = _TABLE_CPU.to(device)
    return _TABLES[key]


def normal_bf16(seed: int, tensor_id: int, shape, device, chunk: int = 1 << 24) -> torch.Tensor:
    """bf16 tensor of the given shape, N(0,1) by table lookup of the counter-based stream."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    table = normal_table(device)
    key = stream_key(seed, tensor_id)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        u = splitmix64_tensor(key, s, m, device)
        out[s:s + m] = table[_lsr(u, 48)]
    return out.view(*shape)


def host_stream(seed: int, tensor_id: int):
    """Generator of 64-bit stream values on the host (for small integer structures)."""
    key = stream_key(seed, tensor_id)
    i = 0
    while True:
        yield splitmix64((key + i) & _M64)
        i += 1


def chain_parents(T: int) -> List[int]:
    return [-1] + list(range(T - 1))


def random_tree_parents(seed: int, tensor_id: int, T: int, max_depth: int = 8,
                        max_children: int = 4) -> List[int]:
    """Seeded draft tree in topological order: node 0 is the root (depth 1); each later node picks
    a parent among the earlier nodes that are above the depth limit and have a free child slot."""
    g = host_stream(seed, tensor_id)
    parents, depth, children = [-1], [1], [0]
    for i in range(1, T):
        cand = [j for j in range(i) if depth[j] < max_depth and children[j] < max_children]
        u = next(g)
        if not cand:            # cannot happen for T <= 64 with the default limits; keep total
            parents.append(-1); depth.append(1); children.append(0)
            continue
        p = cand[u % len(cand)]
        parents.append(p); depth.append(depth[p] + 1); children.append(0)
        children[p] += 1
    return parents


def ragged_lengths(seed: int, tensor_id: int, B: int, lo: int = 8192, hi: int = 32768) -> List[int]:
    g = host_stream(seed, tensor_id)
    return [lo + next(g) % (hi - lo + 1) for _ in range(B)]


def sample_without_replacement(seed: int, tensor_id: int, n: int, k: int) -> List[int]:
    g = host_stream(seed, tensor_id)
    chosen, seen = [], set()
    while len(chosen) < k:
        c = next(g) % n
        if c not in seen:
            seen.add(c); chosen.append(c)
    return chosen


# tensor ids within a case
_TID_Q, _TID_K, _TID_V, _TID_TREE, _TID_LEN, _TID_HEAVY = 1, 2, 3, 4, 5, 6


@dataclass
class VerifyCase:
    """Inputs of one verification-mode call.  Cache rows [kv_len[b], kv_len[b]+T) hold the draft
    tokens' K/V; rows past that are filled too (the path must ignore them)."""
    q: torch.Tensor            # [B, T, 28, 128] bf16
    k: torch.Tensor            # [B, 4, capacity, 128] bf16
    v: torch.Tensor
    kv_len: List[int]
    parents: torch.Tensor      # [B, T] int32 (same device as q)
    T: int
    capacity: int
    name: str = ""
    meta: dict = field(default_factory=dict)

    @property
    def B(self):
        return self.q.shape[0]

    def kv_bytes(self) -> int:
        """Algorithmic K+V bytes: every visible row once per KV head."""
        return sum((n + self.T) * HKV * D * 2 * 2 for n in self.kv_len)

    def io_bytes(self) -> int:
        """Q + out + lse bytes."""
        return self.B * self.T * HQ * (D * 2 * 2 + 4)

    def flops(self) -> int:
        return sum(4 * GROUP * self.T * (n + self.T) * D * HKV for n in self.kv_len)


@dataclass
class AnchorCase:
    q: torch.Tensor            # [B, T, 28, 128]
    k: torch.Tensor            # [B, 4, capacity, 128]
    v: torch.Tensor
    anchor_idx: torch.Tensor   # [B, n_anchor] int32
    n_anchor: int
    window: int
    T: int
    capacity: int
    name: str = ""

    @property
    def B(self):
        return self.q.shape[0]

    def kv_bytes(self) -> int:
        return self.B * self.n_anchor * HKV * D * 2 * 2

    def io_bytes(self) -> int:
        return self.B * self.T * HQ * (D * 2 * 2 + 4) + self.B * self.n_anchor * 4


def make_verify_case(seed: int, kv_len: List[int], T: int, tree: str = "chain", device="cpu",
                     capacity: Optional[int] = None, heavy_frac: float = 0.0,
                     n_visual: Optional[List[int]] = None, name: str = "", hq: int = HQ, hkv: int = HKV) -> VerifyCase:
    """tree: "chain", "random" (seeded, depth <= 8, <= 4 children) or "forest" (all roots).
    hq / hkv: query and KV heads (28 / 4 unless a test asks for another GQA ratio)."""
    B = len(kv_len)
    cap = capacity if capacity is not None else max(kv_len) + T
    assert cap >= max(kv_len) + T
    q = normal_bf16(seed, _TID_Q, (B, T, hq, D), device)
    k = normal_bf16(seed, _TID_K, (B, hkv, cap, D), device)
    v = normal_bf16(seed, _TID_V, (B, hkv, cap, D), device)
    par = []
    for b in range(B):
        if tree == "chain":
            par.append(chain_parents(T))
        elif tree == "forest":
            par.append([-1] * T)
        elif tree == "random":
            par.append(random_tree_parents(seed + 7919 * b, _TID_TREE, T))
        else:
            raise ValueError(tree)
    if heavy_frac > 0.0:
        # Mimic attention-heavy visual tokens: shift a seeded subset of visual key rows of each
        # KV head by twice the mean query vector of that head's group.
        for b in range(B):
            nv = n_visual[b] if n_visual is not None else kv_len[b]
            n_heavy = int(math.floor(heavy_frac * nv))
            for h in range(hkv):
                qbar = q[b, :, h * (hq // hkv):(h + 1) * (hq // hkv), :].float().mean(dim=(0, 1))
                rows = sample_without_replacement(seed + 104729 * b + h, _TID_HEAVY, nv, n_heavy)
                ridx = torch.tensor(rows, dtype=torch.long, device=device)
                k[b, h, ridx, :] = (k[b, h, ridx, :].float() + 2.0 * qbar).to(torch.bfloat16)
    parents = torch.tensor(par, dtype=torch.int32, device=device)
    return VerifyCase(q=q, k=k, v=v, kv_len=list(kv_len), parents=parents, T=T, capacity=cap,
                      name=name)


def make_anchor_case(seed: int, anchor_list: Sequence[int], window: int, T: int, B: int = 1,
                     device="cpu", capacity: Optional[int] = None, name: str = "") -> AnchorCase:
    """Inputs of one anchored-mode call.  ``anchor_list`` is the caller's list of anchored rows
    (strictly increasing, the last T entries being the draft tokens' rows); which rows are anchors
    is decided by the caller -- this module only draws the tensors."""
    idx = [int(x) for x in anchor_list]
    cap = capacity if capacity is not None else idx[-1] + 1
    assert len(idx) >= T and cap > idx[-1]
    q = normal_bf16(seed, _TID_Q, (B, T, HQ, D), device)
    k = normal_bf16(seed, _TID_K, (B, HKV, cap, D), device)
    v = normal_bf16(seed, _TID_V, (B, HKV, cap, D), device)
    anchor = torch.tensor([idx] * B, dtype=torch.int32, device=device)
    return AnchorCase(q=q, k=k, v=v, anchor_idx=anchor, n_anchor=len(idx), window=window, T=T,
                      capacity=cap, name=name)


# The anchored configuration, written out: 26,112 positions, visual span [64, 25,664), the text
# rows inside the last 1024 positions (25,664 .. 26,111: 448 of them), then the draft rows.
C4_SEQ_LEN, C4_VIS_SPANS, C4_WINDOW = 26112, [[64, 25664]], 1024


def c4_anchor_list(T: int) -> List[int]:
    return list(range(25664, 26112)) + list(range(26112, 26112 + T))


# ---- the five benchmark configurations --------------------------------------------------------

def config_seed(c: int, layer: int = 0) -> int:
    return BASE_SEED + c + 1000 * layer


def make_config(c: int, device="cpu", layer: int = 0):
    """c = 0..4 -> the five workload configurations (c = 4 builds ONE of its 28 layers)."""
    s = config_seed(c, layer)
    if c == 0:
        return make_verify_case(s, [2048], 8, "chain", device, name="C1 verify kv2048 T8 chain")
    if c == 1:
        return make_verify_case(s, [26112], 16, "chain", device, heavy_frac=0.01,
                                n_visual=[25600], name="C2 verify kv26112 T16 chain")
    if c == 2:
        return make_verify_case(s, [16384], 64, "random", device, name="C3 verify kv16384 T64 tree")
    if c == 3:
        return make_anchor_case(s, c4_anchor_list(8), C4_WINDOW, 8, 1, device,
                                name="C4 anchor L26112 W1024 T8")
    if c == 4:
        # lengths and trees are per sequence and shared by all layers; K/V/Q differ per layer
        lens = ragged_lengths(config_seed(4, 0), _TID_LEN, 8)
        case = make_verify_case(s, lens, 32, "chain", device, capacity=32768 + 32,
                                name=f"C5 batch8 ragged T32 tree layer{layer}")
        par = [random_tree_parents(config_seed(4, 0) + 7919 * b, _TID_TREE, 32) for b in range(8)]
        case.parents = torch.tensor(par, dtype=torch.int32, device=device)
        return case
    raise ValueError(c)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 numpy array of its bit patterns (on the host)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)
