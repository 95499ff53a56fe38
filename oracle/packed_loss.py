"""CPU oracle for the loss over a packed stream -- TEST INFRASTRUCTURE (same rules as
packed_attention.py: only tests, the smoke check and the benchmark's CPU leg may use it).

The padding-free collator of Sec. 3.4 hands the model ``labels`` in which the first label of
every example is -100 (worked example in Sec. 3.5).  A causal language model scores position t
against the label of position t + 1, so with those labels the last token of an example is never
asked to predict the first token of the next one, and the loss of the packed stream equals the
loss of the examples taken one by one.  This file writes that definition out in fp64:

    target[t] = labels[t + 1]   for t < T - 1,   ignore for t = T - 1
    loss_t    = log(sum_v exp(logits[t, v])) - logits[t, target[t]]      (target[t] != ignore)
    loss      = sum_t loss_t / n_valid,    n_valid = number of rows with a target

and its gradient  d loss / d logits[t, v] = (softmax(logits[t])[v] - [v == target[t]]) / n_valid
for rows with a target, 0 for the others.  Pinned in tests/test_loss_oracle_pins.py by closed
forms, the worked example's label pattern, a library routine on the unpacked examples and
finite differences.
"""
from __future__ import annotations

import numpy as np

IGNORE = -100


def shifted_targets(labels, ignore_index: int = IGNORE):
    """target[t] = labels[t + 1]; the last row has none."""
    labels = np.asarray(labels, dtype=np.int64).reshape(-1)
    T = labels.shape[0]
    out = np.full((T,), ignore_index, dtype=np.int64)
    if T > 1:
        out[:-1] = labels[1:]
    return out


def loss_fwd(logits, labels, ignore_index: int = IGNORE):
    """Returns (mean loss, loss sum, n_valid, per-row loss [T], per-row logsumexp [T]).
    Rows without a target have loss 0 and logsumexp 0; an empty selection has mean 0."""
    x = np.asarray(logits, dtype=np.float64)
    T, V = x.shape
    tgt = shifted_targets(labels, ignore_index)
    token_loss = np.zeros((T,), dtype=np.float64)
    lse = np.zeros((T,), dtype=np.float64)
    n_valid = 0
    for t in range(T):
        c = int(tgt[t])
        if c == ignore_index:
            continue
        assert 0 <= c < V, "labels must be the ignore value or a vocabulary index"
        row = x[t]
        m = row.max()
        lse[t] = m + np.log(np.exp(row - m).sum())
        token_loss[t] = lse[t] - row[c]
        n_valid += 1
    total = float(token_loss.sum())
    mean = total / n_valid if n_valid > 0 else 0.0
    return mean, total, n_valid, token_loss, lse


def loss_bwd(logits, labels, grad_out: float = 1.0, ignore_index: int = IGNORE):
    """d (grad_out * mean loss) / d logits, shape [T, V]."""
    x = np.asarray(logits, dtype=np.float64)
    T, V = x.shape
    tgt = shifted_targets(labels, ignore_index)
    n_valid = int((tgt != ignore_index).sum())
    g = np.zeros((T, V), dtype=np.float64)
    if n_valid == 0:
        return g
    for t in range(T):
        c = int(tgt[t])
        if c == ignore_index:
            continue
        row = x[t]
        p = np.exp(row - row.max())
        p /= p.sum()
        p[c] -= 1.0
        g[t] = p * (grad_out / n_valid)
    return g
