"""Second opinions for the oracle - TEST INFRASTRUCTURE ONLY, tiny inputs.

Two routines written differently from ``reference.py`` / ``kvp_oracle.c`` on purpose:

* ``dense_mask_attention`` - materialise the whole concatenated sequence, build the dense boolean
  attention map of Fig. 2(d) (packets block-diagonal and causal inside; query rows see every
  earlier token), run masked softmax attention for *all* rows with library matmuls, and keep the
  query rows.
* ``ordinary_causal_prefill`` - textbook causal self-attention of one contiguous sequence in pure
  Python floats (sequential sums, ``math.exp``), the thing the composed path must reduce to when
  there is one packet, no adapters and no position shift.
"""
from __future__ import annotations

import math
from typing import Sequence

import numpy as np


def fig2d_mask(segment_lens: Sequence[int], q_len: int) -> np.ndarray:
    """Boolean [T][T] attention map, T = sum(segment_lens) + q_len.  Row t may look at column c iff
    mask[t, c].  Each packet (header+doc+trailer = one entry of ``segment_lens``) is causal within
    itself and blind to other packets; query rows see all packet tokens and query tokens <= self."""
    P = int(sum(segment_lens))
    T = P + q_len
    m = np.zeros((T, T), dtype=bool)
    o = 0
    for n in segment_lens:
        m[o:o + n, o:o + n] = np.tril(np.ones((n, n), dtype=bool))
        o += n
    m[P:, :P] = True
    m[P:, P:] = np.tril(np.ones((q_len, q_len), dtype=bool))
    return m


def dense_mask_attention(K_cat: np.ndarray, V_cat: np.ndarray, Q_all: np.ndarray, mask: np.ndarray,
                         scale: float, group: int) -> np.ndarray:
    """K_cat, V_cat: fp64 [T][Hkv][d]; Q_all: fp64 [T][Hq][d] (rows of packet positions are
    arbitrary fillers); mask [T][T].  Returns out [T][Hq][d] for every row."""
    T, Hq, d = Q_all.shape
    out = np.empty((T, Hq, d), dtype=np.float64)
    for h in range(Hq):
        hk = h // group
        S = (Q_all[:, h, :] @ K_cat[:, hk, :].T) * scale          # [T][T]
        S = np.where(mask, S, -np.inf)
        S = S - S.max(axis=1, keepdims=True)
        Pm = np.exp(S)
        Pm = Pm / Pm.sum(axis=1, keepdims=True)
        out[:, h, :] = Pm @ V_cat[:, hk, :]
    return out


def ordinary_causal_prefill(K: np.ndarray, V: np.ndarray, Q: np.ndarray, n_ctx: int, scale: float,
                            group: int) -> np.ndarray:
    """Causal attention of the last ``len(Q)`` tokens of one contiguous sequence.
    K, V: fp64 [n_ctx + q_len][Hkv][d]; Q: fp64 [q_len][Hq][d].  Query token i sits at sequence
    index n_ctx + i and sees indices <= its own.  Pure Python, left-to-right sums."""
    q_len, Hq, d = Q.shape
    out = np.empty((q_len, Hq, d), dtype=np.float64)
    for i in range(q_len):
        for h in range(Hq):
            hk = h // group
            qv = [float(x) for x in Q[i, h]]
            s = []
            for j in range(n_ctx + i + 1):
                kv = K[j, hk]
                acc = 0.0
                for c in range(d):
                    acc += qv[c] * float(kv[c])
                s.append(acc * scale)
            m = max(s)
            p = [math.exp(x - m) for x in s]
            l = 0.0
            for x in p:
                l += x
            o = [0.0] * d
            for j, pj in enumerate(p):
                w = pj / l
                vv = V[j, hk]
                for c in range(d):
                    o[c] += w * float(vv[c])
            out[i, h] = o
    return out
