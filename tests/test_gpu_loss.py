"""GPU parity of the packed-stream loss kernels against the fp64 oracle, through the C-ABI.

Tolerances (written here, derived from the arithmetic): the kernels read the same bf16 / fp32
logits as the oracle and work in fp32 with exp2/log2 approximations of a few ulp, accumulated
over V terms in a tree of 256 partial sums: per-row loss and logsumexp within 2e-4 absolute
(values are of order log V ~ 10; rows with huge logits add 4e-7 of the largest |logit|, the
fp32 spacing of the result), the mean within 2e-5 relative (plus that term); gradients are written in the
logits' dtype: |err| <= 2^-8 |ref| + 1e-7 for bf16, 4e-6 relative + 1e-9 for fp32 (plus the
relative term explained in _check for rows with huge logits)."""
import numpy as np
import pytest
import torch

from oracle import collate as col
from oracle import packed_loss as pl

pytestmark = pytest.mark.gpu


def _api():
    from paper_2407_09105_b200 import api
    return api


def _stream(lengths, V, seed):
    rng = np.random.default_rng(seed)
    examples = [list(rng.integers(0, V, size=n)) for n in lengths]
    ids, labels, pos, cu = col.collate_padding_free(examples)
    return np.asarray(labels, dtype=np.int32)


def _run(logits_t, labels_np, grad_out=1.0):
    api = _api()
    T, V = logits_t.shape
    dev = logits_t.device
    labels = torch.tensor(labels_np, dtype=torch.int32, device=dev)
    token_loss = torch.full((max(T, 1),), 7.0, device=dev)
    lse = torch.full((max(T, 1),), 7.0, device=dev)
    result = torch.full((2,), -1.0, device=dev)
    n_valid = torch.full((1,), -1, dtype=torch.int32, device=dev)
    api.pk_packed_loss_fwd(logits_t, labels, token_loss[:T], lse[:T], result, n_valid)
    dlogits = torch.empty_strided(logits_t.shape, logits_t.stride(), dtype=logits_t.dtype, device=dev)
    dlogits.fill_(3.0)
    api.pk_packed_loss_bwd(logits_t, labels, lse[:T], n_valid, grad_out, dlogits)
    torch.cuda.synchronize()
    return result.cpu().numpy(), int(n_valid.item()), token_loss[:T].cpu().numpy(), \
        lse[:T].cpu().numpy(), dlogits.float().cpu().numpy()


def _check(logits_t, labels_np, grad_out=1.0):
    x64 = logits_t.float().cpu().numpy().astype(np.float64)
    res, n, tok, lse, dl = _run(logits_t, labels_np, grad_out)
    mean, total, n_ref, tok_ref, lse_ref = pl.loss_fwd(x64, labels_np)
    assert n == n_ref                                            # integer work: exact
    row_tol = 2e-4 + 4e-7 * np.abs(x64).max(axis=1, initial=0)
    assert (np.abs(tok - tok_ref) <= row_tol).all()
    assert (np.abs(lse - lse_ref) <= row_tol).all()
    assert abs(res[0] - mean) <= 2e-5 * max(1.0, abs(mean)) + row_tol.max(initial=0)
    assert abs(res[1] - total) <= 2e-5 * max(1.0, abs(total)) + row_tol.sum()
    g_ref = pl.loss_bwd(x64, labels_np, grad_out)
    # the stored fp32 logsumexp is a few ulp off, which the exponential turns into a relative error
    # of that size in every probability of the row: 5e-7 of the largest |logit| (nothing for
    # ordinary logits, percents for offsets of 1e4 and more)
    rel = (5e-7 * np.abs(x64).max(axis=1, initial=0))[:, None]
    if logits_t.dtype == torch.bfloat16:
        tol = (2.0 ** -8 + rel) * np.abs(g_ref) + 1e-7
    else:
        tol = (4e-6 + rel) * np.abs(g_ref) + 1e-9           # exp2 approximation: a few ulp
    assert (np.abs(dl - g_ref) <= tol).all()
    ignored = pl.shifted_targets(labels_np) == pl.IGNORE
    assert (dl[ignored] == 0).all() and (tok[ignored] == 0).all()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_worked_example_stream(dtype):
    # the label pattern of the paper's worked example (lengths 4, 8, 5, 11), V spans several
    # 16-byte vectors per thread and a ragged number of them
    lengths = (4, 8, 5, 11)
    V = 32000 if dtype == torch.bfloat16 else 5000
    labels = _stream(lengths, V, 0)
    g = torch.Generator(device="cuda").manual_seed(1)
    x = (torch.randn((sum(lengths), V), generator=g, device="cuda") * 3).to(dtype)
    _check(x, labels, grad_out=0.5)


@pytest.mark.parametrize("V,stride", [(1000, 1000), (1003, 1003), (1003, 1008), (50, 64), (8, 8), (1, 1)])
def test_vocab_shapes_vector_and_scalar_paths(V, stride):
    # V % 8 != 0 or an odd stride takes the scalar path; a padded stride leaves the padding alone
    lengths = (3, 1, 6, 2, 9)
    T = sum(lengths)
    labels = _stream(lengths, V, 2)
    g = torch.Generator(device="cuda").manual_seed(3)
    buf = (torch.randn((T, stride), generator=g, device="cuda") * 4).to(torch.bfloat16)
    x = buf[:, :V]
    _check(x, labels)


def test_extreme_logits_do_not_overflow():
    lengths = (5, 7)
    V = 4096
    labels = _stream(lengths, V, 4)
    g = torch.Generator(device="cuda").manual_seed(5)
    x = torch.randn((12, V), generator=g, device="cuda") * 2
    x[3] += 3.0e4          # huge common offset
    x[7, 11] = 8.0e4       # one dominant entry
    x[9] -= 6.0e4
    _check(x.float(), labels)


def test_degenerate_streams():
    api = _api()
    V = 64
    # only one-token examples: nothing to predict, mean 0, gradient 0
    labels = _stream((1, 1, 1), V, 6)
    x = torch.randn((3, V), device="cuda").to(torch.bfloat16)
    res, n, tok, lse, dl = _run(x, labels)
    assert n == 0 and res[0] == 0 and res[1] == 0 and (dl == 0).all()
    # empty stream
    result = torch.full((2,), -1.0, device="cuda")
    n_valid = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    empty = torch.empty((0, V), dtype=torch.bfloat16, device="cuda")
    api.pk_packed_loss_fwd(empty, torch.empty((0,), dtype=torch.int32, device="cuda"),
                           torch.empty((0,), device="cuda"), torch.empty((0,), device="cuda"),
                           result, n_valid)
    torch.cuda.synchronize()
    assert n_valid.item() == 0 and result[0].item() == 0 and result[1].item() == 0


def test_loss_is_bitwise_reproducible_and_independent_of_ignored_rows():
    lengths = (40, 3, 77, 8)
    V = 8192
    T = sum(lengths)
    labels = _stream(lengths, V, 7)
    g = torch.Generator(device="cuda").manual_seed(8)
    x = (torch.randn((T, V), generator=g, device="cuda") * 2).to(torch.bfloat16)
    a = _run(x, labels)
    b = _run(x, labels)
    assert a[0].tobytes() == b[0].tobytes() and a[4].tobytes() == b[4].tobytes()
    y = x.clone()
    ends = np.cumsum(lengths) - 1
    y[torch.tensor(ends, device="cuda")] = 9.0
    c = _run(y, labels)
    assert a[0].tobytes() == c[0].tobytes()


def test_sampled_rows_at_benchmark_size():
    # the launch configuration bench.py times (bf16, V = 32000, 16384 rows); the oracle checks a sample
    V, T = 32000, 16384
    lengths = []
    rng = np.random.default_rng(9)
    while sum(lengths) < T:
        lengths.append(int(min(T - sum(lengths), rng.integers(1, 3000))))
    labels = np.concatenate([np.r_[-100, rng.integers(0, V, size=n - 1)] for n in lengths]).astype(np.int32)
    g = torch.Generator(device="cuda").manual_seed(10)
    x = torch.empty((T, V), dtype=torch.bfloat16, device="cuda")
    for i in range(0, T, 2048):
        x[i:i + 2048] = (torch.randn((2048, V), generator=g, device="cuda") * 2.5).to(torch.bfloat16)
    res, n, tok, lse, dl = _run(x, labels, grad_out=1.0)
    tgt = pl.shifted_targets(labels)
    assert n == int((tgt != pl.IGNORE).sum())
    rows = sorted(set([0, 1, T - 2, T - 1] + list(np.cumsum(lengths)[:3] - 1) +
                      list(rng.integers(0, T, size=24))))
    x_rows = x[torch.tensor(rows, device="cuda")].float().cpu().numpy().astype(np.float64)
    for r, row in zip(rows, x_rows):
        if tgt[r] == pl.IGNORE:
            assert tok[r] == 0 and (dl[r] == 0).all()
            continue
        m = row.max()
        l = m + np.log(np.exp(row - m).sum())
        assert abs(lse[r] - l) <= 2e-4 and abs(tok[r] - (l - row[tgt[r]])) <= 2e-4
        p = np.exp(row - l)
        p[tgt[r]] -= 1.0
        gref = p / n
        assert (np.abs(dl[r] - gref) <= 2.0 ** -8 * np.abs(gref) + 1e-7).all()
    # the mean is the fixed-order sum of the per-row values the kernel wrote
    assert abs(res[0] - tok.astype(np.float64).sum() / n) <= 2e-5 * res[0]
