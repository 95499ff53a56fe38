"""Sliding-window attention on the GPU against the fp64 oracle (forward and backward), through
the C-ABI.  Same tolerances as the unwindowed tests: O, lse 1e-2; gradients 2e-2 (+ 2^-8 |ref|
for bf16 outputs)."""
import numpy as np
import pytest
import torch

from oracle import packed_attention as orc
from paper_2407_09105_b200 import api, workloads as wl
from helpers import f64, max_abs, run_bwd, run_fwd, to_cuda

pytestmark = pytest.mark.gpu

TOL_O = 1e-2
TOL_G = 2e-2


def _case(lens, Hq, Hkv, D, theta, window, seed=0, dtype=torch.float32):
    w = wl.Workload("t", seed, Hq, Hkv, D, theta, [list(lens)], "test")
    st = to_cuda(wl.stream_tensors(w, list(lens), 0, "cpu"))
    out, lse, ws = run_fwd(st, w, dtype, window=window)
    dq, dk, dv = run_bwd(st, w, out, lse, ws, dtype, window=window)
    pos = st.position_ids.cpu().numpy()
    eo, el = orc.attn_fwd(f64(st.q), f64(st.k), f64(st.v), pos, w.softmax_scale, theta, window=window)
    edq, edk, edv = orc.attn_bwd(f64(st.dout), f64(st.q), f64(st.k), f64(st.v), pos,
                                 w.softmax_scale, theta, window=window)
    extra = (lambda e: 2.0 ** -8 * np.abs(e)) if dtype == torch.bfloat16 else (lambda e: 0.0)
    for name, g, e, tol in (("out", out, eo, TOL_O), ("lse", lse, el, TOL_O), ("dq", dq, edq, TOL_G),
                            ("dk", dk, edk, TOL_G), ("dv", dv, edv, TOL_G)):
        g = f64(g)
        assert not np.isnan(g).any(), name
        bound = tol + (extra(e) if name != "lse" else 0.0)
        assert (np.abs(g - e) <= bound).all(), (name, window, max_abs(g, e))


@pytest.mark.parametrize("window", [1, 2, 100, 128, 129, 200, 256, 300, 1000])
def test_window_sizes_across_tile_edges(window):
    # examples of 1 .. 6 tiles; windows below, at and above the 128-row tile, so that whole key
    # tiles are skipped, edge tiles are partly masked and some rows see nothing in a tile
    _case([700, 1, 130, 385, 128, 64], 4, 2, 128, 0.0, window, seed=40)


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (3, 1), (8, 1)])
def test_window_with_block_pairs_and_mqa(Hq, Hkv):
    # odd group sizes pair two query blocks per unit: their windows start at different key tiles
    for window in (90, 257, 512):
        _case([641, 300, 129], Hq, Hkv, 128, 0.0, window, seed=41)


@pytest.mark.parametrize("D", [64, 128])
def test_window_with_rope_and_bf16(D):
    _case([513, 77, 260], 4, 2, D, 1e4, 192, seed=42, dtype=torch.bfloat16)
    _case([400, 131], 4, 4, D, 5e5, 130, seed=43)


def test_window_longer_than_every_example_is_bitwise_the_unwindowed_result():
    lens = [300, 129, 5]
    w = wl.Workload("t", 44, 4, 2, 128, 0.0, [lens], "test")
    st = to_cuda(wl.stream_tensors(w, lens, 0, "cpu"))
    res = []
    for window in (0, 300, 4096):
        out, lse, ws = run_fwd(st, w, window=window)
        dq, dk, dv = run_bwd(st, w, out, lse, ws, window=window)
        res.append([x.cpu().numpy().tobytes() for x in (out, lse, dq, dk, dv)])
    assert res[0] == res[1] == res[2]


def test_window_is_refused_with_in_tile_rope():
    lens = [200]
    w = wl.Workload("t", 45, 2, 2, 128, 1e4, [lens], "test")
    st = to_cuda(wl.stream_tensors(w, lens, 0, "cpu"))
    api.pk_set_rope_mode(api.PK_ROPE_IN_TILE)
    try:
        with pytest.raises(api.PkError) as e:
            run_fwd(st, w, window=64)
        assert e.value.code == api.PK_ERR_UNSUPPORTED
    finally:
        api.pk_set_rope_mode(api.PK_ROPE_ROTATED_COPIES)


def test_mistral_shaped_pack_with_its_window():
    # one 8192-token pack of c4's shape (GQA 32/8, D 128) with the 4096-token window of Mistral-7B:
    # sampled rows against the oracle's single-row routine would not know the window, so a short
    # head count keeps the full oracle affordable
    lens = [5000, 3000, 192]
    _case(lens, 4, 1, 128, 0.0, 4096, seed=46, dtype=torch.bfloat16)
