"""Head sizes other than 64 and 128 (they run on zero-padded copies): parity with the fp64 oracle
at the tolerances of the native sizes (O, lse 1e-2; gradients 2e-2; bf16 outputs get half a bf16
ulp of the exact value on top)."""
import numpy as np
import pytest
import torch

from oracle import packed_attention as orc
from paper_2407_09105_b200 import api, workloads as wl
from helpers import f64, max_abs, run_bwd, run_fwd, to_cuda

pytestmark = pytest.mark.gpu


def _case(lens, Hq, Hkv, D, theta, seed, out_dtype=torch.float32, grad_dtype=torch.float32, window=0):
    w = wl.Workload("t", seed, Hq, Hkv, D, theta, [list(lens)], "test")
    st = to_cuda(wl.stream_tensors(w, list(lens), 0, "cpu"))
    pos = st.position_ids.cpu().numpy()
    out, lse, ws = run_fwd(st, w, out_dtype, window=window)
    kw = {"window": window} if window else {}
    o_ref, l_ref = orc.attn_fwd(f64(st.q), f64(st.k), f64(st.v), pos, w.softmax_scale, theta, **kw)
    assert not np.isnan(f64(out)).any()
    assert max_abs(f64(lse), l_ref) <= 1e-2
    extra = 2.0 ** -8 * np.abs(o_ref) if out_dtype == torch.bfloat16 else 0.0
    assert (np.abs(f64(out) - o_ref) <= 1e-2 + extra).all()
    grads = run_bwd(st, w, out, lse, ws, grad_dtype, window=window)
    refs = orc.attn_bwd(f64(st.dout), f64(st.q), f64(st.k), f64(st.v), pos, w.softmax_scale, theta, **kw)
    for name, g, e in zip(("dq", "dk", "dv"), grads, refs):
        g = f64(g)
        assert g.shape == e.shape and not np.isnan(g).any(), name
        extra = 2.0 ** -8 * np.abs(e) if grad_dtype == torch.bfloat16 else 0.0
        assert (np.abs(g - e) <= 2e-2 + extra).all(), (name, max_abs(g, e))


@pytest.mark.parametrize("theta", [0.0, 1e4])
@pytest.mark.parametrize("D", [16, 32, 48, 80, 96, 112])
def test_head_sizes(D, theta):
    _case([150, 260, 3, 129], 4, 2, D, theta, seed=40 + D)


@pytest.mark.parametrize("D", [80, 96])
def test_bf16_outputs_mha_and_window(D):
    _case([300, 5, 200], 4, 4, D, 5e5, seed=50, out_dtype=torch.bfloat16, grad_dtype=torch.bfloat16)
    _case([400, 77], 6, 2, D, 0.0, seed=51, window=100)
    _case([1], 2, 1, D, 1e4, seed=52)


def test_rope_uses_the_callers_head_size_and_position_ids():
    # a fragment whose ids start at 1000: the frequencies are theta^(-2i/96), not the padded size's
    w = wl.Workload("t", 53, 2, 2, 96, 1e4, [[100, 50]], "test")
    st = to_cuda(wl.stream_tensors(w, [100, 50], 0, "cpu", [1000, 0]))
    out, lse, ws = run_fwd(st, w)
    o_ref, _ = orc.attn_fwd(f64(st.q), f64(st.k), f64(st.v), st.position_ids.cpu().numpy(),
                            w.softmax_scale, 1e4)
    assert max_abs(f64(out), o_ref) <= 1e-2


def test_backward_reusing_the_forwards_padded_copies_is_bitwise_the_same():
    lens = [300, 5, 200, 131]
    w = wl.Workload("t", 54, 8, 2, 80, 1e4, [lens], "test")
    st = wl.stream_tensors(w, lens, 0, device="cuda")
    T, Hq, D = st.q.shape
    ws = api.alloc_workspace(T, Hq, 2, D)
    out = torch.empty_like(st.q)
    lse = torch.empty((Hq, T), dtype=torch.float32, device="cuda")
    res = []
    for reuse in (False, True):
        api.pk_attn_fwd(st.q, st.k, st.v, st.position_ids, w.softmax_scale, w.rope_theta, out, lse, ws)
        dq, dk, dv = torch.empty_like(st.q), torch.empty_like(st.k), torch.empty_like(st.v)
        api.pk_attn_bwd(st.dout, st.q, st.k, st.v, out, lse, st.position_ids, w.softmax_scale,
                        w.rope_theta, dq, dk, dv, ws, reuse_plan=True, reuse_rotated=reuse)
        torch.cuda.synchronize()
        res.append([x.float().cpu().numpy().tobytes() for x in (dq, dk, dv)])
    assert res[0] == res[1]
    assert api.pk_status_read(ws) == (api.PK_OK, 0)
