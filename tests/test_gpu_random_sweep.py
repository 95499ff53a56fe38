"""A seeded sweep over random small problems: lengths, head layouts, head size, RoPE, sliding window
and output types are drawn together, forward and backward are compared with the fp64 oracle.
Tolerances as everywhere: O, lse 1e-2; gradients 2e-2 (+ 2^-8 |ref| for bf16 outputs)."""
import numpy as np
import pytest
import torch

from oracle import packed_attention as orc
from paper_2407_09105_b200 import workloads as wl
from helpers import f64, max_abs, run_bwd, run_fwd, to_cuda

pytestmark = pytest.mark.gpu


def _draw(rng):
    n_ex = int(rng.integers(1, 7))
    kinds = rng.integers(0, 4, size=n_ex)
    lens = []
    for k in kinds:
        if k == 0:
            lens.append(int(rng.integers(1, 20)))                 # tiny
        elif k == 1:
            lens.append(int(128 * rng.integers(1, 4) + rng.integers(-1, 2)))   # next to a tile edge
        elif k == 2:
            lens.append(int(rng.integers(20, 400)))
        else:
            lens.append(int(rng.integers(400, 900)))
    Hkv = int(rng.choice([1, 2, 3]))
    G = int(rng.choice([1, 2, 3, 4]))
    D = int(rng.choice([64, 128]))
    theta = float(rng.choice([0.0, 0.0, 1e4, 5e5]))
    window = int(rng.choice([0, 0, 1, 17, 128, 200, 333]))
    dtype = torch.bfloat16 if rng.integers(0, 2) else torch.float32
    return lens, Hkv * G, Hkv, D, theta, window, dtype


@pytest.mark.parametrize("seed", range(24))
def test_random_problem(seed):
    rng = np.random.default_rng(1000 + seed)
    lens, Hq, Hkv, D, theta, window, dtype = _draw(rng)
    w = wl.Workload("sweep", 2000 + seed, Hq, Hkv, D, theta, [lens], "test", window)
    st = to_cuda(wl.stream_tensors(w, lens, 0, "cpu"))
    out, lse, ws = run_fwd(st, w, dtype, window=window)
    dq, dk, dv = run_bwd(st, w, out, lse, ws, dtype, window=window)
    pos = st.position_ids.cpu().numpy()
    eo, el = orc.attn_fwd(f64(st.q), f64(st.k), f64(st.v), pos, w.softmax_scale, theta, window=window)
    edq, edk, edv = orc.attn_bwd(f64(st.dout), f64(st.q), f64(st.k), f64(st.v), pos,
                                 w.softmax_scale, theta, window=window)
    what = (lens, Hq, Hkv, D, theta, window, dtype)
    extra = (lambda e: 2.0 ** -8 * np.abs(e)) if dtype == torch.bfloat16 else (lambda e: 0.0)
    for name, g, e, tol in (("out", out, eo, 1e-2), ("dq", dq, edq, 2e-2), ("dk", dk, edk, 2e-2),
                            ("dv", dv, edv, 2e-2)):
        g = f64(g)
        assert not np.isnan(g).any(), (name, what)
        assert (np.abs(g - e) <= tol + extra(e)).all(), (name, what, max_abs(g, e))
    assert max_abs(f64(lse), el) <= 1e-2, ("lse", what)
