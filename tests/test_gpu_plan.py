"""GPU parity, integer part: cu_seqlens, counts and work lists are bit-exact."""
import numpy as np
import pytest
import torch

from oracle import packed_attention as orc
from paper_2407_09105_b200 import api, workloads as wl
from helpers import run_plan

pytestmark = pytest.mark.gpu


def _check(pos_np):
    pos = torch.from_numpy(np.asarray(pos_np, dtype=np.int32)).cuda()
    T = pos.numel()
    ws, cu, ne, mx = run_plan(pos)
    code, detail = api.pk_status_read(ws)
    assert code == api.PK_OK, (code, detail)
    ecu, eE, emx = orc.seqlens_from_posids(pos_np)
    assert np.array_equal(cu.cpu().numpy(), ecu)
    assert int(ne) == eE and int(mx) == emx
    bm, bn = api.pk_tile_shape()
    fwd, bwd, fo, bo = orc.work_lists(ecu, eE, bm, bn)
    hdr = api.workspace_view(ws, api.PK_WS_HEADER, T, 1, 1, 64).cpu().numpy()
    N = len(fwd)
    assert hdr[api.PK_HDR_N_ITEMS] == N and hdr[api.PK_HDR_N_EXAMPLES] == eE
    assert hdr[api.PK_HDR_MAX_SEQLEN] == emx and hdr[api.PK_HDR_PLAN_T] == T
    gf = api.workspace_view(ws, api.PK_WS_FWD_ITEMS, T, 1, 1, 64).cpu().numpy().reshape(-1, 4)[:N]
    gb = api.workspace_view(ws, api.PK_WS_BWD_ITEMS, T, 1, 1, 64).cpu().numpy().reshape(-1, 4)[:N]
    gfo = api.workspace_view(ws, api.PK_WS_FWD_ORDER, T, 1, 1, 64).cpu().numpy()[:N]
    gbo = api.workspace_view(ws, api.PK_WS_BWD_ORDER, T, 1, 1, 64).cpu().numpy()[:N]
    assert np.array_equal(gf, fwd) and np.array_equal(gb, bwd)
    assert np.array_equal(gfo, fo) and np.array_equal(gbo, bo)


def test_worked_example():
    _check([0, 1, 2, 3, 0, 1, 2, 3, 4, 5, 6, 7, 0, 1, 2, 3, 4, 0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10])


@pytest.mark.parametrize("lens", [
    [1], [1, 1, 1, 1], [127, 128, 129], [128] * 9, [5000], [1] * 3000,
    [300, 1, 1, 1025, 2, 4097, 127], [1023, 1, 1024, 1025]])
def test_edge_layouts(lens):
    _check(wl.position_ids_from_lengths(lens))


def test_irregular_ids():
    _check([5, 6, 7, 3, 4])
    _check([0, 2, 4, 4, 9, 1])
    _check([7] * 2500)


@pytest.mark.parametrize("name", wl.WORKLOAD_NAMES)
def test_configs(name):
    w = wl.workload(name)
    _check(wl.position_ids_from_lengths(w.streams[0]))
    _check(wl.position_ids_from_lengths(w.flat_lengths()))


@pytest.mark.parametrize("seed", range(4))
def test_random_layouts(seed):
    rng = np.random.default_rng(seed)
    lens = [int(x) for x in np.clip(np.rint(rng.lognormal(4.0, 1.5, size=400)), 1, 3000)]
    _check(wl.position_ids_from_lengths(lens))


def test_empty_stream():
    ws = api.alloc_workspace(0, 1, 1, 64)
    cu = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    ne = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    mx = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    pos = torch.zeros((0,), dtype=torch.int32, device="cuda")
    api.pk_seqlens_from_posids(pos, cu, ne, mx, ws)
    assert cu.tolist() == [0] and int(ne) == 0 and int(mx) == 0


def test_negative_id_sets_status():
    pos = torch.tensor([0, 1, 2, -1, 0, 1], dtype=torch.int32, device="cuda")
    ws, cu, ne, mx = run_plan(pos)
    code, detail = api.pk_status_read(ws)
    assert code == api.PK_ERR_BAD_POSIDS and detail == 3
    hdr = api.workspace_view(ws, api.PK_WS_HEADER, 6, 1, 1, 64).cpu().numpy()
    assert hdr[api.PK_HDR_N_ITEMS] == 0


def test_bounded_wait_expires_and_reports_timeout():
    """A wait that nothing satisfies gives up after its budget, records PK_ERR_TIMEOUT and
    returns; the context stays usable (the next planning call succeeds)."""
    pos = torch.from_numpy(wl.position_ids_from_lengths([40, 9])).cuda()
    ws, cu, ne, mx = run_plan(pos)
    assert api.pk_status_read(ws) == (api.PK_OK, 0)
    api.pk_selftest_bounded_wait(ws, 2_000_000)          # about a millisecond
    assert api.pk_status_read(ws) == (api.PK_ERR_TIMEOUT, 99)
    ws, cu, ne, mx = run_plan(pos)
    assert api.pk_status_read(ws) == (api.PK_OK, 0) and int(ne) == 2
