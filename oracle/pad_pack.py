"""CPU oracle for moving between a padded batch and the packed stream -- TEST INFRASTRUCTURE
(same rules as packed_attention.py).

The padded layout is the one the paper starts from (Sec. 3: every example of a mini-batch
extended with padding tokens to the longest one, appended on the right); the packed layout is the
concatenation of the examples without padding (Sec. 3.4).  Both directions are plain indexing:

    packed[cu[b] + i] = padded[b][i]          for i < length[b]
    padded[b][i]      = packed[cu[b] + i]     for i < length[b],  fill otherwise
"""
from __future__ import annotations

import numpy as np


def pack_rows(padded, lengths):
    padded = np.asarray(padded)
    out = [padded[b, :int(n)] for b, n in enumerate(lengths)]
    return np.concatenate(out, axis=0) if out else padded.reshape((0,) + padded.shape[2:])


def unpack_rows(packed, lengths, l_max, fill=0):
    packed = np.asarray(packed)
    out = np.full((len(lengths), int(l_max)) + packed.shape[1:], fill, dtype=packed.dtype)
    t = 0
    for b, n in enumerate(lengths):
        out[b, :int(n)] = packed[t:t + int(n)]
        t += int(n)
    return out
