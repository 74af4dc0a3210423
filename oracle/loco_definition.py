"""Double-precision statement of LoCo's definitions (arXiv 2407.04480).  Test infrastructure only.

The C oracle pins every fp32 rounding; this file is the same mathematics in
float64 numpy, one line per line of Algorithm 1, and serves on tiny vectors to
check the invariants that the paper's lemmas state about real numbers.  It is
not used by the CUDA library, and it covers the paper's own scale rule only
(global s and s_e, Eq. 1); the block-scaled extension has no twin.
"""
from __future__ import annotations

import numpy as np


def compressor(h, s, p):
    """Eq. 1: round_p-bit(h x s), nearest integer (ties to even) within [-2^(p-1), 2^(p-1)-1]."""
    return np.clip(np.rint(np.asarray(h, dtype=np.float64) * s), -(2 ** (p - 1)), 2 ** (p - 1) - 1)


def decompressor(q, s):
    """Eq. 1: float(q) / s."""
    return np.asarray(q, dtype=np.float64) / s


def loco_step(g, e_tilde, e_code, k, *, s, s_e, beta, T_c, p=4, p_e=8, state="int8"):
    """One pass of Algorithm 1, steps 1 and 2, for one worker.

    state = "int8": only the 8-bit e_k exists, and e~_k of Eq. 5 is dec(e_k; s_e);
    state = "fp32": e~_k is kept and used for compensation as it is;
    state = "fp32_q8comp": e~_k is kept, compensation uses dec(comp(e~_k; s_e, 8); s_e).
    Returns (codes, d, h, e~_{k+1} before reset, e~_{k+1} as kept, e_{k+1} codes).
    """
    g = np.asarray(g, dtype=np.float64)
    if state == "int8":
        c = decompressor(e_code, s_e)
        prev = c
    elif state == "fp32":
        c = np.asarray(e_tilde, dtype=np.float64)
        prev = c
    elif state == "fp32_q8comp":
        prev = np.asarray(e_tilde, dtype=np.float64)
        c = decompressor(compressor(prev, s_e, p_e), s_e)
    else:
        raise ValueError(state)
    h = g + c                                           # Algorithm 1, step 1 / Eq. 2
    q = compressor(h, s, p)                             # Eq. 3
    d = decompressor(q, s)                              # step 2
    e_next = (1.0 - beta) * prev + beta * (h - d)       # Eq. 5
    if T_c > 0 and k % T_c == 0:                        # Eq. 7
        e_code_next = np.zeros_like(g)
        e_next_kept = np.zeros_like(g)
    else:
        e_code_next = compressor(e_next, s_e, p_e)
        e_next_kept = e_next
    return q, d, h, e_next, e_next_kept, e_code_next


def average(ds):
    """Eq. 8: the mean of the workers' dequantised vectors."""
    return np.mean(np.asarray(ds, dtype=np.float64), axis=0)


def adam_family_step(g, m, v, theta, *, lr, beta1, beta2, delta):
    """The paper's Adam-family equations with Adam's pre-conditioner: m = (1-b1) m + b1 g, v = (1-b2) v + b2 g^2,
    theta = theta - lr / sqrt(v + delta) * m  (no bias correction, delta inside the root).  Returns (m, v, theta)."""
    g, m, v, theta = (np.asarray(a, dtype=np.float64) for a in (g, m, v, theta))
    m = (1.0 - beta1) * m + beta1 * g
    v = (1.0 - beta2) * v + beta2 * g * g
    theta = theta - lr / np.sqrt(v + delta) * m
    return m, v, theta
