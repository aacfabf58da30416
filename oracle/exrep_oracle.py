"""CPU checker for the expert-replacement metric.  TEST INFRASTRUCTURE ONLY.

hard_replacements / exrep follow Eq. 4 and Eq. 5 (Section 2.3) on 0/1 expert
activity; pinned by the paper's worked example (Fig. 5: 11 and 21 replacements).
delta_uniform is one reading of "delta between the uniform distribution and the
realised expert balance" (Section 3.3): parity unpinned (the paper gives no formula).
"""
from __future__ import annotations

import numpy as np


def activity_from_topk(S, n_experts: int) -> np.ndarray:
    """A[b, t, e] = 1 if expert e is among token t's selected experts.  S: [B, T, K]."""
    S = np.asarray(S)
    B, T, K = S.shape
    A = np.zeros((B, T, n_experts), dtype=np.int64)
    for b in range(B):
        for t in range(T):
            for j in range(K):
                A[b, t, S[b, t, j]] = 1
    return A


def hard_replacements(A: np.ndarray):
    """Eq. 4: H_e = sum_b sum_{t=1}^{T-1} |A[b,t+1,e] - A[b,t,e]|, H = sum_e H_e."""
    B, T, E = A.shape
    H_e = np.zeros(E, dtype=np.int64)
    for e in range(E):
        for b in range(B):
            for t in range(T - 1):
                H_e[e] += abs(int(A[b, t + 1, e]) - int(A[b, t, e]))
    return H_e, int(H_e.sum())


def exrep(A: np.ndarray, K: int):
    """Eq. 5: every replacement is counted twice in H, so replacements = floor(H/2),
    normalised by B * K * (T - 1).  Returns (replacements, H_norm)."""
    B, T, _ = A.shape
    _, H = hard_replacements(A)
    repl = H // 2
    return repl, repl / (B * K * (T - 1))


def delta_uniform(A: np.ndarray) -> float:
    """Mean over experts of |share_e - 1/E|, in percent, share_e = fraction of all
    activations that went to expert e.  Parity unpinned."""
    E = A.shape[-1]
    share = A.reshape(-1, E).sum(axis=0) / A.sum()
    return float(np.mean(np.abs(share - 1.0 / E)) * 100.0)
