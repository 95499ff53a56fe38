"""Padded <-> packed row movement on the GPU against the oracle: byte work, so bit-exact."""
import numpy as np
import pytest
import torch

from oracle import pad_pack as pp
from paper_2407_09105_b200 import api

pytestmark = pytest.mark.gpu


def _case(lengths, l_max, tail, dtype, seed=0, misalign=0):
    rng = np.random.default_rng(seed)
    B, T = len(lengths), int(sum(lengths))
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lengths)]), dtype=torch.int32, device="cuda")
    shape_p = (B, l_max) + tail
    if dtype.is_floating_point:
        padded = torch.tensor(rng.standard_normal(shape_p), dtype=dtype)
    else:
        padded = torch.tensor(rng.integers(-1000, 1000, size=shape_p), dtype=dtype)
    as_np = (lambda x: x.float().cpu().numpy()) if dtype.is_floating_point else (lambda x: x.cpu().numpy())
    ref_packed = pp.pack_rows(as_np(padded), lengths)
    dev_padded = padded.cuda()
    # optional misalignment of the packed buffer to force the narrower copy paths
    n_el = int(np.prod((T,) + tail))
    store = torch.zeros(n_el + 8, dtype=dtype, device="cuda")
    packed = store[misalign:misalign + n_el].view((T,) + tail)
    api.pk_pack_rows(dev_padded, cu, packed)
    torch.cuda.synchronize()
    got = as_np(packed)
    assert np.array_equal(got, ref_packed)
    # and back: padding rows must come out as zeros whatever was there before
    back = torch.full(shape_p, 7, dtype=dtype, device="cuda")
    api.pk_unpack_rows(packed, cu, back)
    torch.cuda.synchronize()
    ref_back = pp.unpack_rows(ref_packed, lengths, l_max, fill=0)
    got_back = as_np(back)
    assert np.array_equal(got_back, ref_back)


def test_worked_example_ids():
    # the paper's example (Sec. 3.5): lengths 4, 8, 5, 11 in a 4 x 11 batch of token ids
    _case([4, 8, 5, 11], 11, (), torch.int32)


@pytest.mark.parametrize("tail,dtype,misalign", [((), torch.int32, 0), ((), torch.int64, 0),
                                                 ((3,), torch.bfloat16, 0), ((8,), torch.bfloat16, 0),
                                                 ((8,), torch.bfloat16, 1), ((4, 128), torch.bfloat16, 0),
                                                 ((5,), torch.float32, 0), ((1,), torch.int8, 0),
                                                 ((1,), torch.int8, 3)])
def test_row_sizes_and_alignments(tail, dtype, misalign):
    _case([7, 0, 1, 130, 64, 0, 33], 130, tail, dtype, seed=1, misalign=misalign)


def test_degenerate_batches():
    _case([0, 0], 5, (4,), torch.float32)
    _case([5], 5, (2,), torch.float32)
    _case([], 0, (2,), torch.float32)


def test_hidden_state_sized_rows():
    # a mini-batch of c3's shape: 16 examples, hidden size 4096 in bf16 (8 KB rows)
    rng = np.random.default_rng(2)
    lengths = [int(x) for x in rng.integers(1, 1500, size=16)]
    _case(lengths, max(lengths), (4096,), torch.bfloat16, seed=3)
