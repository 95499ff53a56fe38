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


def test_fixed_length_collator_pins():
    g = _golden()
    T = len(g["input_ids"])
    # a pack at least as long as the stream cuts nothing: the paper's worked example again
    for msl in (T, T + 1, 1000):
        ids, labels, pos, starts = orc.collate_fixed_length(EXAMPLES, msl)
        assert ids == g["input_ids"] and labels == g["labels"] and pos == g["position_ids"]
        assert starts == g["cu_seqlens"]
    # hand-worked: lengths 4, 8, 5, 11 cut every 10 tokens -> boundaries at the example starts
    # 0 4 12 17 and at the pack starts 10 20
    ids, labels, pos, starts = orc.collate_fixed_length(EXAMPLES, 10)
    assert starts == [0, 4, 10, 12, 17, 20, 28]
    assert pos == [0, 1, 2, 3, 0, 1, 2, 3, 4, 5, 0, 1, 0, 1, 2, 3, 4, 0, 1, 2, 0, 1, 2, 3, 4, 5, 6, 7]
    assert [t for t, l in enumerate(labels) if l == -100] == starts[:-1]
    assert all(l == i for l, i in zip(labels, ids) if l != -100) and ids == g["input_ids"]
    # every pack taken alone is a well-formed padding-free stream: it equals the padding-free
    # collation of the pieces that fall into it (random lengths, several pack sizes)
    rng = np.random.default_rng(11)
    for msl in (1, 7, 64):
        examples = [list(rng.integers(0, 1000, size=n)) for n in rng.integers(1, 40, size=30)]
        ids, labels, pos, starts = orc.collate_fixed_length(examples, msl)
        flat = [t for e in examples for t in e]
        ex_of = [i for i, e in enumerate(examples) for _ in e]
        for k in range(0, len(flat), msl):
            piece_ids = flat[k:k + msl]
            pieces = [[t for t, _ in grp] for _, grp in
                      itertools.groupby(zip(piece_ids, ex_of[k:k + msl]), key=lambda x: x[1])]
            i2, l2, p2, _ = orc.collate_padding_free(pieces)
            assert ids[k:k + msl] == i2 and labels[k:k + msl] == l2 and pos[k:k + msl] == p2
        # and the boundary recovery of the attention path finds exactly these fragments
        cu2, E, _ = orc_attn.seqlens_from_posids(pos)
        assert cu2[:E + 1].tolist() == starts


def test_fixed_length_collator_gives_the_fragments_of_the_fixed_length_workload():
    # the c2 generator cuts its drawn lengths into fragments per pack; the collator's boundaries
    # on the same lengths must be those fragments
    from paper_2407_09105_b200 import workloads as wl
    w = wl.workload("c2")
    frags = [l for pack in w.streams for l in pack]
    # undo the cuts: a fragment that starts at a multiple of 4096 may continue an example, which the
    # generator does not record, so feed the fragments themselves (cutting is idempotent)
    examples = [[0] * l for l in frags]
    _, _, pos, starts = orc.collate_fixed_length(examples, 4096)
    assert np.diff(starts).tolist() == frags
    assert pos == wl.position_ids_from_lengths(frags).tolist()


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
def test_device_fixed_length_collator_matches_the_oracle():
    rng = np.random.default_rng(5)
    cases = [(EXAMPLES, 10), (EXAMPLES, 28), (EXAMPLES, 1), ([[7]], 4),
             ([list(range(1, 3001)), [5], list(range(9))], 256),
             ([list(rng.integers(0, 9999, size=n)) for n in rng.integers(1, 900, size=400)], 4096)]
    for examples, msl in cases:
        ids, labels, pos, starts = orc.collate_fixed_length(examples, msl)
        lens = [len(e) for e in examples]
        d_ids = torch.tensor(ids, dtype=torch.int32, device="cuda")
        d_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
        d_pos = torch.full_like(d_ids, -7)
        d_lab = torch.full_like(d_ids, -7)
        d_cu = torch.full((len(examples) + 1,), -7, dtype=torch.int32, device="cuda")
        api.pk_collate_fixed_length(d_ids, d_len, msl, d_pos, d_lab, d_cu)
        assert d_pos.tolist() == pos and d_lab.tolist() == labels
        assert d_cu.tolist() == [0] + list(np.cumsum(lens))
        # the attention path's scan recovers the fragments
        T = len(ids)
        ws = api.alloc_workspace(T, 1, 1, 64)
        cu2 = torch.empty((T + 1,), dtype=torch.int32, device="cuda")
        ne = torch.empty((1,), dtype=torch.int32, device="cuda")
        mx = torch.empty((1,), dtype=torch.int32, device="cuda")
        api.pk_seqlens_from_posids(d_pos, cu2, ne, mx, ws)
        assert cu2[:int(ne) + 1].tolist() == starts
    with pytest.raises(api.PkError):
        api.pk_collate_fixed_length(d_ids, d_len, 0, d_pos, d_lab, d_cu)


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
