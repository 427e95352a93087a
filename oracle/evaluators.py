"""ORACLE - test infrastructure only: independent numpy evaluators (fp64).

Cross-checks for oracle A (``gdn_fullstate.c``).  Each evaluates the same
quantity, the output of one (beam, head) unit, by a different route, so that a
mistake in one shows as a disagreement:

* :func:`forward_projection_replay` - the paper's own route: transition records
  (alpha, delta, k) of Eq. 2 replayed forward on the two projection accumulators
  of Eq. 3, closed by Eq. 4.
* :func:`backward_fold` - the adjoint route: fold the query through the chain
  newest-first, then meet S_0 once.
* :func:`ancestry_table` - Eq. 5, the flattened ancestry index, against which the
  linked parent-pointer walk of oracle A is compared.

All inputs are for ONE head: S0 [dv, dk]; chain = list of (k [dk], v [dv], alpha, beta)
oldest first; q [dk].
"""
from __future__ import annotations

import numpy as np


def forward_projection_replay(S0, chain, q):
    """Eq. 2-4.  First turn the raw tokens into transition records (alpha_j, delta_j, k_j), each
    delta_j from the key projection u_k = S_{j-1} k_j obtained by replay (never from a state
    matrix); then replay the records on the query projection and close with Eq. 4."""
    S0 = np.asarray(S0, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    gtr = []                                    # (alpha, delta, k)
    for (k, v, a, b) in chain:
        k = np.asarray(k, dtype=np.float64)
        v = np.asarray(v, dtype=np.float64)
        u_k = S0 @ k                            # Eq. 3, u_k^(-1)
        for (ai, di, ki) in gtr:                # Eq. 3, 0 <= i < j
            u_k = ai * u_k + di * (ki @ k)
        delta = b * (v - a * u_k)               # Eq. 4, first line
        gtr.append((float(a), delta, k))
    if not gtr:
        return S0 @ q
    u_q = S0 @ q                                # Eq. 3, u_q^(-1)
    for (ai, di, ki) in gtr[:-1]:
        u_q = ai * u_q + di * (ki @ q)
    at, dt, kt = gtr[-1]
    return at * u_q + dt * (kt @ q)             # Eq. 4, second line


def backward_fold(S0, chain, q):
    """Adjoint of Eq. 1: with A_j = alpha_j (I - beta_j k_j k_j^T), S_j r = S_{j-1}(A_j r) + beta_j (k_j.r) v_j,
    so o = S_0 r_final + sum_j beta_j (k_j.r_j) v_j, folding newest -> oldest."""
    S0 = np.asarray(S0, dtype=np.float64)
    r = np.asarray(q, dtype=np.float64).copy()
    corr = np.zeros(S0.shape[0], dtype=np.float64)
    for (k, v, a, b) in reversed(chain):
        k = np.asarray(k, dtype=np.float64)
        c = k @ r
        corr += b * c * np.asarray(v, dtype=np.float64)
        r = a * (r - b * c * k)
    return S0 @ r + corr


def ancestry_table(parents, widths):
    """Eq. 5 as a table.  parents[t] (t >= 1) maps beams of call t to beams of call t-1.
    Returns, for the last call T-1, h [W_{T-1}, T] with h[b, j] = beam index at call j on b's
    ancestry (the paper's h_t(b, j) for j < t) and h[b, T-1] = b (the beam's own new record)."""
    T = len(widths)
    h = np.arange(widths[0], dtype=np.int64).reshape(-1, 1)
    for t in range(1, T):
        p = np.asarray(parents[t], dtype=np.int64)
        assert p.shape == (widths[t],)
        new = np.empty((widths[t], t + 1), dtype=np.int64)
        new[:, : t - 1] = h[p, : t - 1]          # 0 <= j < t-1: inherit the parent's row
        new[:, t - 1] = p                        # j = t-1: the parent's own slot
        new[:, t] = np.arange(widths[t])         # the record written at call t
        h = new
    return h
