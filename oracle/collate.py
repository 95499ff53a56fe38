"""CPU oracle for the collation and sample-selection steps around the attention path --
TEST INFRASTRUCTURE (same rules as packed_attention.py: only tests may use it).

Plain Python from the paper's description: the padding-free collator of Sec. 3.4 / 3.5
(concatenate the examples, first label of every example becomes -100, position ids restart at
0 per example), its fixed-length variant that cuts the stream into packs, and the sample-selection baselines of Sec. 3.3 (first-fit-decreasing bin
packing as in Multipack, and first-come-first-served filling of a given or sorted order).
Pinned by the worked example of Sec. 3.5 and by brute force on tiny inputs.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def collate_padding_free(examples: Sequence[Sequence[int]], ignore_index: int = -100):
    """Returns (input_ids, labels, position_ids, cu_seqlens) of the flattened mini-batch."""
    input_ids: List[int] = []
    labels: List[int] = []
    position_ids: List[int] = []
    cu = [0]
    for ex in examples:
        for p, tok in enumerate(ex):
            input_ids.append(int(tok))
            labels.append(ignore_index if p == 0 else int(tok))
            position_ids.append(p)
        cu.append(len(input_ids))
    return input_ids, labels, position_ids, cu


def collate_fixed_length(examples: Sequence[Sequence[int]], msl: int, ignore_index: int = -100):
    """Fixed-length packing with position ids (Sec. 3.3, Table 1: the variant that uses position
    ids and still breaks examples): the concatenated stream is chopped into packs of msl tokens.
    The paper does not say which ids the tail of a broken example gets; the reading taken here is
    that a pack is a sequence of its own, so the fragment that opens a pack is treated as a new
    example: its position ids restart at 0 and its first label is ignored.
    Returns (input_ids, labels, position_ids, fragment_starts + [T])."""
    if msl <= 0:
        raise ValueError("msl must be positive")
    input_ids: List[int] = []
    labels: List[int] = []
    position_ids: List[int] = []
    starts: List[int] = []
    for ex in examples:
        p = 0
        for tok in ex:
            t = len(input_ids)
            if t % msl == 0:          # a pack begins here, whether or not an example does
                p = 0
            if p == 0:
                starts.append(t)
            input_ids.append(int(tok))
            labels.append(ignore_index if p == 0 else int(tok))
            position_ids.append(p)
            p += 1
    return input_ids, labels, position_ids, starts + [len(input_ids)]


def pack_first_fit_decreasing(lengths: Sequence[int], capacity: int) -> Tuple[List[int], int]:
    """Bin index of every example: examples are taken from long to short (ties in the given
    order) and put into the first bin with room; a new bin is opened when none has."""
    order = sorted(range(len(lengths)), key=lambda i: -lengths[i])      # stable
    room: List[int] = []
    bin_of = [-1] * len(lengths)
    for i in order:
        for b in range(len(room)):
            if room[b] >= lengths[i]:
                bin_of[i] = b
                room[b] -= lengths[i]
                break
        else:
            bin_of[i] = len(room)
            room.append(capacity - lengths[i])
    return bin_of, len(room)


def pack_next_fit(lengths: Sequence[int], capacity: int, sort_descending: bool) -> Tuple[List[int], int]:
    """First-come-first-served: walk the examples in the given order (or from long to short) and
    start a new pack whenever the next example does not fit into the current one."""
    order = list(range(len(lengths)))
    if sort_descending:
        order.sort(key=lambda i: -lengths[i])
    bin_of = [-1] * len(lengths)
    b, used = 0, 0
    started = False
    for i in order:
        if started and used + lengths[i] > capacity:
            b += 1
            used = 0
        bin_of[i] = b
        used += lengths[i]
        started = True
    return bin_of, (b + 1 if started else 0)
