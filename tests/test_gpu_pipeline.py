"""The host-to-host pipeline (copy-in, kernels and copy-out of different packs overlapped on three
streams) must deliver exactly what direct per-pack calls deliver, pass after pass."""
import numpy as np
import pytest
import torch

from paper_2407_09105_b200 import api, pipeline, workloads as wl

pytestmark = pytest.mark.gpu


def test_pipeline_matches_direct_calls_bitwise():
    packs = [[300, 40, 172], [512], [7, 130, 129, 246], [90, 422]]
    w = wl.Workload("t", 31, 4, 2, 128, 1e4, packs, "test")
    lens = w.flat_lengths()
    st = wl.stream_tensors(w, lens, 0, device="cuda")
    T, Hq, D = st.q.shape
    Hkv = st.k.shape[1]
    bounds = np.concatenate([[0], np.cumsum([sum(p) for p in packs])]).tolist()
    spans = list(zip(bounds, bounds[1:]))
    ws = api.alloc_workspace(max(b - a for a, b in spans), Hq, Hkv, D)

    def run_pack(i, tensors, outs, stream):
        q, k, v, do, pos = tensors
        out, dq, dk, dv = outs
        a, b = spans[i]
        lse = torch.empty((Hq, b - a), dtype=torch.float32, device="cuda")
        api.pk_attn_fwd(q[a:b], k[a:b], v[a:b], pos[a:b], w.softmax_scale, w.rope_theta, out[a:b], lse,
                        ws, reuse_plan=False, stream=stream)
        api.pk_attn_bwd(do[a:b], q[a:b], k[a:b], v[a:b], out[a:b], lse, pos[a:b], w.softmax_scale,
                        w.rope_theta, dq[a:b], dk[a:b], dv[a:b], ws, reuse_plan=True,
                        reuse_rotated=True, stream=stream)

    dev_in = [st.q, st.k, st.v, st.dout, st.position_ids]
    ref_out = [torch.empty_like(st.q), torch.empty_like(st.q), torch.empty_like(st.k), torch.empty_like(st.v)]
    cur = torch.cuda.current_stream()
    for i in range(len(spans)):
        run_pack(i, dev_in, ref_out, cur)
    torch.cuda.synchronize()
    ref = [x.float().cpu().numpy() for x in ref_out]

    host_in = [x.cpu().pin_memory() for x in dev_in]
    work_in = [torch.zeros_like(x) for x in dev_in]          # the pipeline fills these
    work_out = [torch.zeros_like(x) for x in ref_out]
    host_out = [torch.zeros(x.shape, dtype=x.dtype).pin_memory() for x in ref_out]
    cut = lambda ts: [[x[a:b] for x in ts] for a, b in spans]
    pipe = pipeline.HostPipeline(cut(host_in), cut(work_in), cut(work_out), cut(host_out),
                                 lambda i, s: run_pack(i, work_in, work_out, s))
    for _ in range(3):                                       # buffers are reused pass after pass
        for h in host_out:
            h.zero_()
        pipe.step(cur)
        torch.cuda.synchronize()
        for h, r in zip(host_out, ref):
            assert h.float().numpy().tobytes() == r.tobytes()
