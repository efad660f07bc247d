"""Second formulation of the compression-phase step, used only to check the first.

The un-chunked parameter-server form of Supplement Section A, in binary64 with
numpy: every worker forms beta*m + (1-beta)*g_i, compresses it with error
compensation, the server averages the n compressed vectors, compresses the
average with its own error compensation and broadcasts it; the model moves by
-lr * m_new / (sqrt(v) + eps).  The paper notes (Supplement A, first sentence)
that the chunked algorithm equals this form run on every chunk by itself; the
test-suite relies on that to cross-check the C oracle's chunk and exchange
indexing.  Test infrastructure only.
"""
from __future__ import annotations

import numpy as np


def compress(z: np.ndarray) -> np.ndarray:
    """C[z] for the 1-bit compressor of Section 5.1, returned already decompressed."""
    scale = np.sqrt(np.sum(z * z) / z.size)          # ||z|| / ||sign vector||
    return np.where(z >= 0.0, scale, -scale)


def parameter_server_step(m, x, v, worker_err, server_err, grads, beta, lr, eps):
    """One step of Supplement A on one vector.  All arrays float64; returns new state."""
    n = len(grads)
    sent = []
    new_worker_err = []
    for i in range(n):
        m_i = beta * m + (1.0 - beta) * grads[i]
        half = compress(m_i + worker_err[i])
        new_worker_err.append(m_i + worker_err[i] - half)
        sent.append(half)
    m_half = sum(sent) / n
    m_new = compress(m_half + server_err)
    new_server_err = m_half + server_err - m_new
    x_new = x - lr * m_new / (np.sqrt(v) + eps)
    return m_new, x_new, new_worker_err, new_server_err


def chunked_step(m, x, v, worker_err, server_err, grads, beta, lr, eps, chunk):
    """The same step applied to every block of `chunk` elements as its own problem."""
    d = m.size
    m2, x2 = np.empty(d), np.empty(d)
    se2 = np.empty(d)
    we2 = [np.empty(d) for _ in grads]
    for lo in range(0, d, chunk):
        sl = slice(lo, min(d, lo + chunk))
        mm, xx, we, se = parameter_server_step(
            m[sl], x[sl], v[sl], [e[sl] for e in worker_err], server_err[sl],
            [g[sl] for g in grads], beta, lr, eps)
        m2[sl], x2[sl], se2[sl] = mm, xx, se
        for i, e in enumerate(we):
            we2[i][sl] = e
    return m2, x2, we2, se2
