"""GPU parity of the forward against the fp64 oracle (same seeded bf16 inputs).

Tolerances: fp32 outputs are held to the stated max-abs 1e-2 (O and lse); bf16 outputs to
1e-2 + 2^-8 |ref| (half a bf16 ulp of the exact value on top of the bound)."""
import numpy as np
import pytest
import torch

from oracle import packed_attention as orc
from paper_2407_09105_b200 import api, workloads as wl
from helpers import f64, max_abs, run_fwd, to_cuda

pytestmark = pytest.mark.gpu

TOL_O = 1e-2
TOL_LSE = 1e-2


def _case(lens, Hq, Hkv, D, theta, seed=0, out_dtype=torch.float32, offsets=None):
    w = wl.Workload("t", seed, Hq, Hkv, D, theta, [list(lens)], "test")
    st = to_cuda(wl.stream_tensors(w, list(lens), 0, "cpu", offsets))
    out, lse, _ = run_fwd(st, w, out_dtype)
    eo, el = orc.attn_fwd(f64(st.q), f64(st.k), f64(st.v), st.position_ids.cpu().numpy(),
                          w.softmax_scale, theta)
    go, gl = f64(out), f64(lse)
    assert not np.isnan(go).any() and not np.isnan(gl).any()
    if out_dtype == torch.float32:
        assert max_abs(go, eo) <= TOL_O, max_abs(go, eo)
    else:
        assert (np.abs(go - eo) <= TOL_O + 2.0 ** -8 * np.abs(eo)).all()
    assert max_abs(gl, el) <= TOL_LSE, max_abs(gl, el)
    return max_abs(go, eo), max_abs(gl, el)


def test_c1_tiny_pack():
    w = wl.workload("c1")
    _case(w.streams[0], w.num_q_heads, w.num_kv_heads, w.head_dim, w.rope_theta)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("lens", [[1], [128], [129], [127, 1, 130], [300, 5, 5, 700, 1]])
def test_tile_edges(D, lens):
    _case(lens, 2, 2, D, 0.0, seed=3)


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (3, 1), (6, 2)])
def test_odd_group_sizes_pair_query_blocks(Hq, Hkv):
    # with an odd number of query heads per kv head a unit is two consecutive query blocks of one
    # example: block counts 1 .. 7 cover the left-over block 0, the masked last step of the
    # shorter block, and ragged last blocks
    _case([1, 128, 129, 256, 257, 384, 385, 641, 896, 100], Hq, Hkv, 128, 0.0, seed=21)
    _case([513, 2, 300], Hq, Hkv, 64, 0.0, seed=22, out_dtype=torch.bfloat16)
    _case([385, 130], Hq, Hkv, 128, 1e4, seed=23)         # rotated copies


@pytest.mark.parametrize("D", [64, 128])
def test_gqa(D):
    _case([200, 77, 400], 8, 2, D, 0.0, seed=4)


@pytest.mark.parametrize("mode", [api.PK_ROPE_ROTATED_COPIES, api.PK_ROPE_IN_TILE])
@pytest.mark.parametrize("D,theta", [(64, 1e4), (128, 1e4), (128, 5e5)])
def test_fused_rope(D, theta, mode):
    api.pk_set_rope_mode(mode)
    try:
        _case([150, 260, 3, 129], 4, 2, D, theta, seed=5)
        _case([300, 40], 4, 4, D, theta, seed=15)          # MHA: block pairs share K/V tiles
    finally:
        api.pk_set_rope_mode(api.PK_ROPE_ROTATED_COPIES)


def test_rope_uses_given_ids_of_a_fragment():
    _case([100, 50], 2, 2, 128, 1e4, seed=6, offsets=[1000, 0])


def test_bf16_output():
    _case([300, 5, 200], 4, 2, 128, 0.0, seed=7, out_dtype=torch.bfloat16)
    _case([300, 5, 200], 4, 4, 64, 1e4, seed=7, out_dtype=torch.bfloat16)


def test_long_example_many_tiles():
    _case([2100, 37], 2, 1, 128, 0.0, seed=8)
