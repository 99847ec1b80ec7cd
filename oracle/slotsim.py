"""Slot-level simulator of the diagonal / baby-step giant-step matrix-vector product.

TEST INFRASTRUCTURE ONLY.  No cryptography: slot vectors are plain fp64 arrays, a rotation is
np.roll.  It exists to check the packing map and the BSGS identity used by oracle/ckks.py against
the plain definition y = W x, for any tile side D, replica split tau and split b*g = D/tau.
"""
from __future__ import annotations

import numpy as np

from .ckks import Plan, fold_output, pack_input, plain_slots


def rot_left(v: np.ndarray, steps: int) -> np.ndarray:
    """out[s] = v[(s + steps) mod n]."""
    return np.roll(v, -steps)


def linear_slots(W: np.ndarray, x: np.ndarray, plan: Plan, n: int) -> np.ndarray:
    """Evaluate the encrypted algorithm's dataflow on plain slot vectors and fold: returns y[d_out]."""
    plan.check(n)
    d_out, d_in = W.shape
    D = plan.D
    n_in, n_out = -(-d_in // D), plan.n_out(d_out)
    xp = np.zeros(n_in * D)
    xp[:d_in] = x
    packed = [pack_input(xp[q * D:(q + 1) * D], plan, n) for q in range(n_in)]
    y = np.zeros(d_out)
    for p in range(n_out):
        Y = np.zeros(n, dtype=np.complex128 if plan.pack == "complex" else np.float64)
        for j in range(plan.g):
            inner = np.zeros_like(Y)
            for q in range(n_in):
                for k in range(plan.b):
                    inner += plain_slots(W, plan, p, q, j, k, n) * rot_left(packed[q], k * plan.tau)
            Y += rot_left(inner, j * plan.b * plan.tau)
        part = fold_output(Y, plan, p, d_out)
        y[p * plan.rows_per_ct:p * plan.rows_per_ct + len(part)] = part
    return y
