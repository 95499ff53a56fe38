"""Collator and sample selection (the scope's "next" rows): oracle pins, host packers against the
oracle (no GPU needed: they are host code), device collator against the oracle (GPU)."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import collate as orc
from oracle import packed_attention as orc_attn
from paper_2407_09105_b200 import api

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example_sec3_5.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split(":")
        out[k.strip()] = [int(x) for x in v.split()]
    return out


EXAMPLES = [[10, 11, 12, 13], [20, 21, 22, 23, 24, 25, 26, 27], [30, 31, 32, 33, 34],
            [40, 41, 42, 43, 44, 45, 46, 47, 48, 49, 410]]


# ------------------------------------------------------------------ oracle pins
def test_collator_reproduces_the_papers_example():
    g = _golden()
    ids, labels, pos, cu = orc.collate_padding_free(EXAMPLES)
    assert ids == g["input_ids"] and labels == g["labels"] and pos == g["position_ids"]
    assert cu == g["cu_seqlens"]
    # and the boundary recovery of the attention path inverts it
    cu2, E, _ = orc_attn.seqlens_from_posids(pos)
    assert cu2[:E + 1].tolist() == cu


def _optimal_bins(lengths, cap):
    """Brute force: smallest number of bins over all assignments (tiny inputs only)."""
    n = len(lengths)
    for k in range(1, n + 1):
        for assign in itertools.product(range(k), repeat=n):
            load = [0] * k
            for l, b in zip(lengths, assign):
                load[b] += l
            if max(load) <= cap:
                return k
    return n


def test_ffd_hand_worked_and_bound():
    # capacity 10: sorted 7 6 5 5 4 2 2 1 -> bins [7,2,1] [6,4] [5,5] [2]
    lengths = [5, 7, 5, 2, 4, 2, 6, 1]
    bin_of, nb = orc.pack_first_fit_decreasing(lengths, 10)
    assert nb == 4
    groups = [sorted(lengths[i] for i in range(len(lengths)) if bin_of[i] == b) for b in range(nb)]
    assert groups == [[1, 2, 7], [4, 6], [5, 5], [2]]
    rng = np.random.default_rng(0)
    for _ in range(30):
        ls = [int(x) for x in rng.integers(1, 9, size=rng.integers(1, 7))]
        bin_of, nb = orc.pack_first_fit_decreasing(ls, 8)
        load = [sum(l for l, b in zip(ls, bin_of) if b == k) for k in range(nb)]
        assert max(load) <= 8 and min(load) > 0
        opt = _optimal_bins(ls, 8)
        assert opt <= nb <= (11 * opt + 6) // 9 + 1       # the classic FFD guarantee (loosely)


def test_next_fit_hand_worked():
    lengths = [4, 5, 3, 6, 2]
    assert orc.pack_next_fit(lengths, 8, False) == ([0, 1, 1, 2, 2], 3)
    # sorted long to short: 6 5 4 3 2 -> [6] [5] [4,3] [2]
    assert orc.pack_next_fit(lengths, 8, True) == ([2, 1, 2, 0, 3], 4)
    assert orc.pack_next_fit([], 8, True) == ([], 0)


# ------------------------------------------------------------------ host packers vs oracle
@pytest.mark.parametrize("seed", range(6))
def test_host_packers_match_the_oracle(seed):
    rng = np.random.default_rng(seed)
    cap = int(rng.integers(64, 8193))
    ls = [int(x) for x in rng.integers(1, cap + 1, size=rng.integers(1, 400))]
    assert api.pk_pack_first_fit_decreasing(ls, cap) == orc.pack_first_fit_decreasing(ls, cap)
    for srt in (False, True):
        assert api.pk_pack_next_fit(ls, cap, srt) == orc.pack_next_fit(ls, cap, srt)


def test_host_packers_reject_bad_lengths():
    with pytest.raises(api.PkError):
        api.pk_pack_first_fit_decreasing([3, 9], 8)
    with pytest.raises(api.PkError):
        api.pk_pack_next_fit([0, 2], 8, False)


def test_multipack_workload_is_reproduced_by_the_library_packer():
    from paper_2407_09105_b200 import workloads as wl
    rng = np.random.default_rng(3)              # the c4 pool, drawn as the workload does
    pool = []
    while sum(pool) < 16 * 8192:
        pool.append(int(rng.integers(16, 257)) if rng.random() < 0.7 else int(rng.integers(1024, 8193)))
    bin_of, nb = api.pk_pack_first_fit_decreasing(pool, 8192)
    bins = [[] for _ in range(nb)]
    for i in sorted(range(len(pool)), key=lambda i: -pool[i]):
        bins[bin_of[i]].append(pool[i])
    assert bins[:16] == wl.workload("c4").streams


# ------------------------------------------------------------------ device collator
@pytest.mark.gpu
def test_device_collator_matches_the_papers_example_and_the_oracle():
    for examples in (EXAMPLES, [[7]], [list(range(1, 3001)), [5], list(range(9))]):
        ids, labels, pos, cu = orc.collate_padding_free(examples)
        d_ids = torch.tensor(ids, dtype=torch.int32, device="cuda")
        d_len = torch.tensor([len(e) for e in examples], dtype=torch.int32, device="cuda")
        d_pos = torch.full_like(d_ids, -7)
        d_lab = torch.full_like(d_ids, -7)
        d_cu = torch.full((len(examples) + 1,), -7, dtype=torch.int32, device="cuda")
        api.pk_collate_padding_free(d_ids, d_len, d_pos, d_lab, d_cu)
        assert d_pos.tolist() == pos and d_lab.tolist() == labels and d_cu.tolist() == cu


@pytest.mark.gpu
def test_collate_then_boundary_recovery_roundtrip():
    rng = np.random.default_rng(1)
    lens = [int(x) for x in rng.integers(1, 700, size=2500)]
    T = sum(lens)
    d_ids = torch.arange(T, dtype=torch.int32, device="cuda")
    d_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
    d_pos = torch.empty_like(d_ids)
    d_cu = torch.empty((len(lens) + 1,), dtype=torch.int32, device="cuda")
    api.pk_collate_padding_free(d_ids, d_len, d_pos, None, d_cu)
    ws = api.alloc_workspace(T, 1, 1, 64)
    cu2 = torch.empty((T + 1,), dtype=torch.int32, device="cuda")
    ne = torch.empty((1,), dtype=torch.int32, device="cuda")
    mx = torch.empty((1,), dtype=torch.int32, device="cuda")
    api.pk_seqlens_from_posids(d_pos, cu2, ne, mx, ws)
    assert int(ne) == len(lens) and int(mx) == max(lens)
    assert torch.equal(cu2[:len(lens) + 1], d_cu)
