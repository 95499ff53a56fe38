"""Shared helpers of the GPU parity tests."""
import numpy as np
import torch

from oracle import packed_attention as orc
from paper_2407_09105_b200 import api, workloads as wl


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def run_plan(pos: torch.Tensor, Hq=1, Hkv=1, D=64):
    T = pos.numel()
    ws = api.alloc_workspace(T, Hq, Hkv, D)
    cu = torch.full((T + 1,), -7, dtype=torch.int32, device="cuda")
    ne = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    mx = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    api.pk_seqlens_from_posids(pos, cu, ne, mx, ws)
    return ws, cu, ne, mx


def run_fwd(st, w, out_dtype=torch.float32, theta=None, scale=None, window=0):
    T, Hq, D = st.q.shape
    Hkv = st.k.shape[1]
    theta = w.rope_theta if theta is None else theta
    scale = w.softmax_scale if scale is None else scale
    ws = api.alloc_workspace(T, Hq, Hkv, D)
    out = torch.full((T, Hq, D), float("nan"), dtype=out_dtype, device="cuda")
    lse = torch.full((Hq, T), float("nan"), dtype=torch.float32, device="cuda")
    api.pk_attn_fwd(st.q, st.k, st.v, st.position_ids, scale, theta, out, lse, ws, window=window)
    code, detail = api.pk_status_read(ws)
    assert code == api.PK_OK, (code, detail)
    return out, lse, ws


def run_bwd(st, w, out, lse, ws, grad_dtype=torch.float32, theta=None, scale=None, window=0):
    T, Hq, D = st.q.shape
    theta = w.rope_theta if theta is None else theta
    scale = w.softmax_scale if scale is None else scale
    dq = torch.full_like(st.q, float("nan"), dtype=grad_dtype)
    dk = torch.full_like(st.k, float("nan"), dtype=grad_dtype)
    dv = torch.full_like(st.v, float("nan"), dtype=grad_dtype)
    api.pk_attn_bwd(st.dout, st.q, st.k, st.v, out, lse, st.position_ids, scale, theta,
                    dq, dk, dv, ws, reuse_plan=True, window=window)
    code, detail = api.pk_status_read(ws)
    assert code == api.PK_OK, (code, detail)
    return dq, dk, dv


def to_cuda(st):
    return wl.StreamTensors(*(x.cuda() if isinstance(x, torch.Tensor) else x
                              for x in (st.position_ids, st.q, st.k, st.v, st.dout, st.lengths)))


def max_abs(a, b):
    return float(np.abs(np.asarray(a) - np.asarray(b)).max()) if np.asarray(a).size else 0.0
