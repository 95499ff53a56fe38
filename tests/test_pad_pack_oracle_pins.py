"""Pins for the padded <-> packed oracle (CPU): the paper's worked example (Sec. 3.5), round trips,
fill values."""
import os

import numpy as np

from oracle import pad_pack as pp

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example_sec3_5.txt")


def _golden():
    rows = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split(":", 1)
            rows[k.strip()] = [int(x) for x in v.split()]
    return rows


def test_worked_example_padded_batch_packs_to_the_printed_stream():
    g = _golden()
    cu = g["cu_seqlens"]
    lengths = np.diff(cu)                                   # 4, 8, 5, 11
    ids = np.asarray(g["input_ids"])
    # the padded batch of the example: 4 rows of 11, padding id 0 appended on the right
    padded = np.zeros((4, 11), dtype=np.int64)
    for b in range(4):
        padded[b, :lengths[b]] = ids[cu[b]:cu[b + 1]]
    assert padded[0].tolist() == [10, 11, 12, 13, 0, 0, 0, 0, 0, 0, 0]
    assert padded[3].tolist() == [40, 41, 42, 43, 44, 45, 46, 47, 48, 49, 410]
    packed = pp.pack_rows(padded, lengths)
    assert packed.tolist() == ids.tolist()                  # the input_ids the paper prints
    back = pp.unpack_rows(packed, lengths, 11, fill=0)
    assert np.array_equal(back, padded)
    # 28 real tokens in a 44-slot batch: the padding the method removes
    assert packed.shape[0] == 28 and padded.size == 44


def test_round_trip_with_feature_rows_and_fill():
    rng = np.random.default_rng(0)
    lengths = [3, 0, 7, 1]
    packed = rng.standard_normal((sum(lengths), 5)).astype(np.float32)
    padded = pp.unpack_rows(packed, lengths, 9, fill=-1)
    assert padded.shape == (4, 9, 5)
    assert (padded[1] == -1).all() and (padded[0, 3:] == -1).all() and (padded[2, 7:] == -1).all()
    assert np.array_equal(pp.pack_rows(padded, lengths), packed)
    assert pp.pack_rows(np.zeros((0, 4, 2)), []).shape == (0, 2)
