"""Pins for the packed-stream loss oracle (CPU only): closed forms, the label pattern of the
paper's worked example (Sec. 3.5), a library routine applied to the unpacked examples, and
finite differences for the gradient."""
import os

import numpy as np
import torch

from oracle import collate as col
from oracle import packed_loss as pl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example_sec3_5.txt")


def _worked_example():
    rows = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split(":", 1)
        rows[k.strip()] = [int(x) for x in v.split()]
    return rows


def test_uniform_logits_give_log_vocab():
    T, V = 7, 50
    labels = np.arange(T) % V
    mean, total, n, tok, lse = pl.loss_fwd(np.zeros((T, V)), labels)
    assert n == T - 1
    assert np.allclose(tok[:-1], np.log(V), atol=1e-12) and tok[-1] == 0.0
    assert abs(mean - np.log(V)) < 1e-12 and abs(total - (T - 1) * np.log(V)) < 1e-10
    # adding a constant to a row changes nothing (softmax is shift invariant)
    x = np.random.default_rng(0).normal(size=(T, V))
    a = pl.loss_fwd(x, labels)[0]
    b = pl.loss_fwd(x + np.arange(T)[:, None] * 3.0, labels)[0]
    assert abs(a - b) < 1e-12


def test_confident_row_has_vanishing_or_linear_loss():
    V = 11
    x = np.zeros((2, V))
    x[0, 4] = 40.0
    # right answer: loss -> 0 ; wrong answer: loss -> the margin
    assert pl.loss_fwd(x, [0, 4])[0] < 1e-15 + 11 * np.exp(-40.0)
    assert abs(pl.loss_fwd(x, [0, 5])[0] - 40.0) < 1e-12


def test_worked_example_label_pattern():
    ex = _worked_example()
    labels = ex["labels"]
    T = len(labels)
    tgt = pl.shifted_targets(labels)
    # 28 tokens, 4 examples: every example loses its first label, the stream loses the last row
    assert T == 28 and (tgt != pl.IGNORE).sum() == 24
    ends = [3, 11, 16, 27]                      # last token of every example
    assert [t for t in range(T) if tgt[t] == pl.IGNORE] == ends
    # the loss does not depend on the logits of those rows ...
    rng = np.random.default_rng(1)
    V = 500
    x = rng.normal(size=(T, V))
    base = pl.loss_fwd(x, labels)
    y = x.copy()
    y[ends] = rng.normal(size=(4, V)) * 10
    assert pl.loss_fwd(y, labels)[0] == base[0]
    # ... and their gradient rows are exactly zero
    g = pl.loss_bwd(x, labels)
    assert (g[ends] == 0).all() and (np.abs(g).sum(axis=1)[[0, 5, 20]] > 0).all()


def test_packed_loss_equals_examples_one_by_one_with_a_library_routine():
    # the packed stream against torch's cross entropy on every example alone (shifted by hand)
    rng = np.random.default_rng(2)
    V = 97
    examples = [list(rng.integers(0, V, size=n)) for n in (5, 1, 9, 2, 14)]
    ids, labels, pos, cu = col.collate_padding_free(examples)
    T = len(ids)
    x = rng.normal(size=(T, V)) * 2
    mean, total, n, tok, lse = pl.loss_fwd(x, labels)
    s, cnt = 0.0, 0
    for e in range(len(examples)):
        a, b = cu[e], cu[e + 1]
        if b - a < 2:
            continue
        lg = torch.tensor(x[a:b - 1], dtype=torch.float64)
        tg = torch.tensor(ids[a + 1:b], dtype=torch.int64)
        s += float(torch.nn.functional.cross_entropy(lg, tg, reduction="sum"))
        cnt += b - a - 1
    assert n == cnt == sum(len(e) - 1 for e in examples)
    assert abs(total - s) < 1e-9 and abs(mean - s / cnt) < 1e-12
    # logsumexp against the library's
    ref = torch.logsumexp(torch.tensor(x), dim=1).numpy()
    valid = pl.shifted_targets(labels) != pl.IGNORE
    assert np.allclose(lse[valid], ref[valid], atol=1e-12) and (lse[~valid] == 0).all()


def test_gradient_matches_finite_differences_and_sums_to_zero():
    rng = np.random.default_rng(3)
    V, lens = 13, (3, 4, 2)
    examples = [list(rng.integers(0, V, size=n)) for n in lens]
    _, labels, _, _ = col.collate_padding_free(examples)
    T = len(labels)
    x = rng.normal(size=(T, V))
    g = pl.loss_bwd(x, labels, grad_out=0.7)
    assert np.allclose(g.sum(axis=1), 0.0, atol=1e-15)       # softmax minus one-hot
    h = 1e-6
    for (t, v) in [(0, 0), (1, 5), (4, 12), (6, 3), (2, 7), (8, 1)]:
        xp, xm = x.copy(), x.copy()
        xp[t, v] += h
        xm[t, v] -= h
        fd = 0.7 * (pl.loss_fwd(xp, labels)[0] - pl.loss_fwd(xm, labels)[0]) / (2 * h)
        assert abs(fd - g[t, v]) < 1e-8
    # against autograd of the library routine on the whole stream with ignore_index
    xt = torch.tensor(x, requires_grad=True)
    tgt = torch.tensor(pl.shifted_targets(labels))
    loss = torch.nn.functional.cross_entropy(xt, tgt, ignore_index=pl.IGNORE)
    (0.7 * loss).backward()
    assert np.allclose(xt.grad.numpy(), g, atol=1e-14)


def test_degenerate_streams():
    V = 5
    # one token, or only one-token examples: nothing to predict
    assert pl.loss_fwd(np.zeros((1, V)), [-100])[:3] == (0.0, 0.0, 0)
    _, labels, _, _ = col.collate_padding_free([[1], [2], [3]])
    assert pl.loss_fwd(np.ones((3, V)), labels)[2] == 0
    assert (pl.loss_bwd(np.ones((3, V)), labels) == 0).all()
