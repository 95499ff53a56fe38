"""Seeded synthetic workloads: example lengths, position ids and bf16 values.

This module holds no attention arithmetic.  It only draws example lengths,
arranges them into packed streams the way the paper's packing variants do
(Sec. 3.1 online mini-batch collating, Sec. 3.2 offline flat packs, Sec. 3.3
bin-packed / sorted sample selection), writes the matching ``position_ids``
(restart at 0 for every example, Sec. 3.1 / Sec. 3.5) and draws N(0,1) values
rounded once to bf16.  Both the CUDA path and the CPU oracle are fed from here
so that they see identical bytes.

The paper's datasets (FLAN, OrcaMath, the Stack) are not available; the length
distributions below stand in for their shape (short-mode instruction data,
longer-mode maths data, long high-variance code).
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """One configuration: head shapes plus a list of independent packed streams."""

    name: str
    seed: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    rope_theta: float            # <= 0: no rotary embedding
    streams: List[List[int]]     # example lengths of every stream, in stream order
    packing: str                 # which of the paper's packing variants it mimics
    window: int = 0              # > 0: sliding-window attention, keys visible per row

    @property
    def softmax_scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    @property
    def total_tokens(self) -> int:
        return sum(sum(s) for s in self.streams)

    @property
    def causal_pairs(self) -> int:
        """Sum over examples of L(L+1)/2 (diagonal included); with a sliding window W every
        row counts min(position + 1, W) keys."""
        def pairs(l: int) -> int:
            w = self.window
            if w <= 0 or l <= w:
                return l * (l + 1) // 2
            return w * (w + 1) // 2 + (l - w) * w
        return sum(pairs(l) for s in self.streams for l in s)

    @property
    def useful_flops_fwd(self) -> int:
        return 4 * self.head_dim * self.num_q_heads * self.causal_pairs

    @property
    def useful_flops_bwd(self) -> int:
        return 10 * self.head_dim * self.num_q_heads * self.causal_pairs

    def flat_lengths(self) -> List[int]:
        """All streams joined into one stream (pack edges are example edges)."""
        return [l for s in self.streams for l in s]


def position_ids_from_lengths(lengths, start_offsets=None) -> np.ndarray:
    """``[0..L_1-1, 0..L_2-1, ...]`` as int32 (Sec. 3.1).  ``start_offsets[i]``
    optionally makes example ``i`` count from that value instead of 0."""
    parts = []
    for i, l in enumerate(lengths):
        o = 0 if start_offsets is None else int(start_offsets[i])
        parts.append(np.arange(o, o + l, dtype=np.int32))
    if not parts:
        return np.zeros((0,), dtype=np.int32)
    return np.concatenate(parts)


# ----------------------------------------------------------------------------
# length recipes
# ----------------------------------------------------------------------------

def _tiny_lengths(seed: int) -> List[List[int]]:
    rng = np.random.default_rng(seed)
    lens: List[int] = []
    while sum(lens) < 512:
        lens.append(int(rng.integers(16, 129)))
    lens[-1] -= sum(lens) - 512
    return [lens]


def _fixed_length_packs(seed: int, n_packs: int = 8, msl: int = 4096) -> List[List[int]]:
    """Examples concatenated in draw order and cut every ``msl`` tokens; the
    fragment after a cut restarts its ids at 0 (it becomes its own example)."""
    rng = np.random.default_rng(seed)
    total = n_packs * msl
    lens: List[int] = []
    while sum(lens) < total:
        x = rng.lognormal(math.log(256.0), 1.0)
        lens.append(int(np.clip(np.rint(x), 8, 4096)))
    lens[-1] -= sum(lens) - total
    packs: List[List[int]] = [[] for _ in range(n_packs)]
    pos = 0
    for l in lens:
        while l > 0:
            p = pos // msl
            room = (p + 1) * msl - pos
            take = min(l, room)
            packs[p].append(take)
            pos += take
            l -= take
    return packs


def _minibatch_streams(seed: int, n_batches: int = 64, bs: int = 16) -> List[List[int]]:
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n_batches):
        row = []
        for _ in range(bs):
            x = rng.lognormal(math.log(200.0), 1.2)
            row.append(int(np.clip(np.rint(x), 8, 4096)))
        out.append(row)
    return out


def _multipack_bins(seed: int, n_bins: int = 16, cap: int = 8192) -> List[List[int]]:
    """First-fit-decreasing bin packing of a 70/30 short/long mixture."""
    rng = np.random.default_rng(seed)
    pool: List[int] = []
    while sum(pool) < n_bins * cap:
        if rng.random() < 0.7:
            pool.append(int(rng.integers(16, 257)))
        else:
            pool.append(int(rng.integers(1024, 8193)))
    order = sorted(range(len(pool)), key=lambda i: (-pool[i], i))
    bins: List[List[int]] = []
    room: List[int] = []
    for i in order:
        l = pool[i]
        for b in range(len(bins)):
            if room[b] >= l:
                bins[b].append(l)
                room[b] -= l
                break
        else:
            bins.append([l])
            room.append(cap - l)
    return bins[:n_bins]


def _sorted_packs(seed: int, n_packs: int = 4, cap: int = 16384) -> List[List[int]]:
    """Lengths sorted long to short, then filled first-come-first-served without
    breaking examples (Sec. 3.3, the sorted baseline)."""
    rng = np.random.default_rng(seed)
    pool: List[int] = []
    while sum(pool) < n_packs * cap:
        x = math.exp(rng.uniform(math.log(32.0), math.log(16384.0)))
        pool.append(int(np.clip(np.rint(x), 32, 16384)))
    pool.sort(reverse=True)
    packs: List[List[int]] = [[]]
    used = 0
    for l in pool:
        if used + l > cap:
            packs.append([])
            used = 0
        packs[-1].append(l)
        used += l
    return packs[:n_packs]


def workload(name: str) -> Workload:
    """The five configurations (``c1`` .. ``c5``) and the padded twin of ``c3``."""
    if name == "c1":
        return Workload("c1", 0, 4, 4, 64, 0.0, _tiny_lengths(0), "tiny pack")
    if name == "c2":
        return Workload("c2", 1, 32, 32, 128, 1.0e4, _fixed_length_packs(1),
                        "FixedLengthPacking+PosID")
    if name == "c3":
        return Workload("c3", 2, 32, 8, 128, 5.0e5, _minibatch_streams(2),
                        "MiniBatchPacking+PosID")
    if name == "c3_padded":
        packed = _minibatch_streams(2)
        padded = [[max(row)] * len(row) for row in packed]
        return Workload("c3_padded", 2, 32, 8, 128, 5.0e5, padded,
                        "RandomSampling+Padding")
    if name == "c4":
        return Workload("c4", 3, 32, 8, 128, 0.0, _multipack_bins(3), "Multipack+PosID")
    if name == "c5":
        return Workload("c5", 4, 64, 8, 128, 0.0, _sorted_packs(4), "SortedPacking+PosID")
    raise KeyError(name)


WORKLOAD_NAMES = ("c1", "c2", "c3", "c4", "c5")


# ----------------------------------------------------------------------------
# values
# ----------------------------------------------------------------------------

def normal_bf16(shape, seed: int, device: str = "cpu") -> torch.Tensor:
    """N(0,1) values rounded once to bf16, from a seeded generator on ``device``."""
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    x = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    return x.to(torch.bfloat16)


@dataclasses.dataclass
class StreamTensors:
    position_ids: torch.Tensor   # int32 [T]
    q: torch.Tensor              # bf16 [T, Hq, D]
    k: torch.Tensor              # bf16 [T, Hkv, D]
    v: torch.Tensor              # bf16 [T, Hkv, D]
    dout: torch.Tensor           # bf16 [T, Hq, D]
    lengths: List[int]


def stream_tensors(w: Workload, lengths: List[int], stream_index: int = 0,
                   device: str = "cpu",
                   start_offsets: Optional[List[int]] = None) -> StreamTensors:
    """Tensors of one packed stream of workload ``w`` (seed derived from the
    workload seed and the stream index)."""
    T = int(sum(lengths))
    base = 1000003 * (w.seed + 1) + 7919 * stream_index
    pos = torch.from_numpy(position_ids_from_lengths(lengths, start_offsets)).to(device)
    q = normal_bf16((T, w.num_q_heads, w.head_dim), base + 1, device)
    k = normal_bf16((T, w.num_kv_heads, w.head_dim), base + 2, device)
    v = normal_bf16((T, w.num_kv_heads, w.head_dim), base + 3, device)
    do = normal_bf16((T, w.num_q_heads, w.head_dim), base + 4, device)
    return StreamTensors(pos, q, k, v, do, list(lengths))
