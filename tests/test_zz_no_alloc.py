"""The no-allocation entry point (pk_seqlens_from_posids_noalloc) against the regular one.

It serves callers that cannot allocate device memory (the framework's allocator owns the
GPU, or an implicit device synchronisation is unacceptable), so its scratch is a fixed array
inside the library that every call shares.  Two calls in a row on different inputs check that
nothing stale from the first call leaks into the second.  This file sorts last so that a run
stopping at the first failure has already been through every other test."""
import numpy as np
import pytest
import torch

from paper_2407_09105_b200 import api, workloads as wl
from helpers import run_plan

pytestmark = pytest.mark.gpu


def _both(lens):
    pos = torch.from_numpy(wl.position_ids_from_lengths(lens)).cuda()
    T = pos.numel()
    _, cu_ref, ne_ref, mx_ref = run_plan(pos)
    cu = torch.full((T + 1,), -7, dtype=torch.int32, device="cuda")
    ne = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    mx = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    api.pk_seqlens_from_posids_noalloc(pos, cu, ne, mx)
    torch.cuda.synchronize()
    assert torch.equal(cu, cu_ref)
    assert int(ne) == int(ne_ref) and int(mx) == int(mx_ref)


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    w = wl.workload("c2")
    _both(w.flat_lengths())                 # 32768 tokens: the built-in capacity exactly
    _both([5, 300, 1, 1, 129, 4000, 17])    # shorter, different layout, same shared scratch
    _both(wl.workload("c1").streams[0])


def test_rejects_streams_beyond_the_built_in_capacity():
    T = api.PK_NOALLOC_MAX_TOKENS + 1
    pos = torch.zeros((T,), dtype=torch.int32, device="cuda")
    cu = torch.zeros((T + 1,), dtype=torch.int32, device="cuda")
    ne = torch.zeros((1,), dtype=torch.int32, device="cuda")
    mx = torch.zeros((1,), dtype=torch.int32, device="cuda")
    with pytest.raises(api.PkError) as e:
        api.pk_seqlens_from_posids_noalloc(pos, cu, ne, mx)
    assert e.value.code == api.PK_ERR_TOO_LARGE
