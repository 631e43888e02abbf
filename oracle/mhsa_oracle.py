"""Oracle for multi-head self-attention.  TEST INFRASTRUCTURE ONLY: tests, the smoke check and
the benchmark's CPU baseline may call it; the CUDA package never does and shares no code with it.

What it computes (paper: Prompts appendix, task 6 "Multi-Head Self-Attention").  Q, K, V are
N x d_model, row-major.  With h heads and d_k = d_model / h, head i owns columns
[i d_k, (i+1) d_k) of each matrix (the i-th contiguous partition), and

    head_i = softmax(Q_i K_i^T / sqrt(d_k)) V_i          (softmax over each row, i.e. over keys)
    MultiHead(Q, K, V) = Concat(head_1, ..., head_h)      (N x d_model, head i back in its columns)

There is no mask and no output projection in the task.  Everything is fp64; the softmax is the
definition exp(s_j) / sum_j exp(s_j), evaluated after subtracting the row maximum (which cancels
exactly in the quotient and keeps exp in range).  bf16 tensors arrive as uint16 bit patterns and
are widened exactly (a bf16 is the upper half of an fp32).

The only library routine in the arithmetic is numpy's matrix product `@` (fp64), used for the two
products per head; tests/test_mhsa_oracle.py replaces it by explicit loops over queries, keys and
columns (an element-by-element brute force of the task's formula) and demands agreement.
"""
from __future__ import annotations

import numpy as np


def widen(x) -> np.ndarray:
    """Exact fp64 copy of a float array, or of bf16 bit patterns given as uint16."""
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return x.astype(np.float64)


def softmax_rows(S: np.ndarray) -> np.ndarray:
    E = np.exp(S - S.max(axis=1, keepdims=True))
    return E / E.sum(axis=1, keepdims=True)


def mhsa(Q, K, V, n: int, d_model: int, h: int, rows=None) -> np.ndarray:
    """MultiHead(Q, K, V) as an fp64 array of shape (n, d_model), or (len(rows), d_model) for the
    query rows listed in `rows` (every key still takes part)."""
    if d_model % h != 0:
        raise ValueError("d_model must be a multiple of h")
    dk = d_model // h
    Qf, Kf, Vf = (widen(t).reshape(n, d_model) for t in (Q, K, V))
    if rows is not None:
        Qf = Qf[np.asarray(rows, dtype=np.int64)]
    out = np.empty((Qf.shape[0], d_model), dtype=np.float64)
    for i in range(h):
        cols = slice(i * dk, (i + 1) * dk)
        S = (Qf[:, cols] @ Kf[:, cols].T) / np.sqrt(float(dk))
        out[:, cols] = softmax_rows(S) @ Vf[:, cols]
    return out
