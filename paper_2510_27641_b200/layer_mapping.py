"""Offline utilities that produce the `layer_map` input of a verification step (CPU, numpy).

Not part of the per-step path: the map from verifier layers to draft layers is computed once,
from attention distributions collected on a representative data set (Sec. 3.3), and then fixed.

  kl_similarity   S[i, j] = -D_KL(A^v_j || A^d_i)                      (Sec. 3.3, the equation of S_ij)
  monotonic_dtw   f maximising sum_j S[f(j), j] over non-decreasing f  (App. B, Alg. 3)

Alg. 3's recurrence takes, for draft layer i and verifier layer j, the best of "diagonal", "left"
and "min over k <= i of dp[k, j-1]"; the third option contains the first two, so the table below
carries exactly that prefix optimum.  Draft layers may be skipped or repeated.
"""
from __future__ import annotations

import numpy as np

__all__ = ["kl_similarity", "monotonic_dtw"]


def kl_similarity(attn_verifier: np.ndarray, attn_draft: np.ndarray) -> np.ndarray:
    """attn_verifier [n, L], attn_draft [m, L]: one attention distribution per layer (rows sum to
    1).  Returns S [m, n] with S[i, j] = -sum_k A^v_j[k] * log(A^v_j[k] / A^d_i[k]); terms with
    A^v_j[k] == 0 contribute 0, and a verifier mass on a position where the draft has none gives
    -inf (the divergence is infinite)."""
    av = np.asarray(attn_verifier, np.float64)
    ad = np.asarray(attn_draft, np.float64)
    if av.ndim != 2 or ad.ndim != 2 or av.shape[1] != ad.shape[1]:
        raise ValueError("expected [n, L] and [m, L]")
    if (av < 0).any() or (ad < 0).any():
        raise ValueError("attention distributions must be non-negative")
    m, n = ad.shape[0], av.shape[0]
    S = np.empty((m, n), np.float64)
    with np.errstate(divide="ignore", invalid="ignore"):
        log_av = np.where(av > 0, np.log(av), 0.0)
        log_ad = np.log(ad)  # -inf where the draft has no mass
        for i in range(m):
            for j in range(n):
                pos = av[j] > 0
                S[i, j] = -np.sum(av[j][pos] * (log_av[j][pos] - log_ad[i][pos]))
    return S


def monotonic_dtw(S: np.ndarray):
    """S [m, n]: similarity of draft layer i and verifier layer j.  Returns (f, total) where f is
    an int32 array of length n with f[0] <= f[1] <= ... (0-based draft layers) maximising
    total = sum_j S[f[j], j].  Among maps of equal total the one that takes the smallest draft
    layer at the last verifier layer, then at the one before it, and so on, is returned.
    -inf entries are allowed (never chosen unless a column has nothing else); NaN is rejected."""
    S = np.asarray(S, np.float64)
    if S.ndim != 2 or S.shape[0] < 1:
        raise ValueError("expected a non-empty [m, n] matrix")
    if np.isnan(S).any():
        raise ValueError("NaN in the similarity matrix")
    m, n = S.shape
    if n == 0:
        return np.zeros(0, np.int32), 0.0
    # best[i] = best total of verifier layers 0..j with f(j) == i;  pre[i] = max_{k <= i} best[k] of
    # the previous column, arg[i] = smallest k attaining it
    best = S[:, 0].copy()
    back = np.zeros((n, m), np.int32)
    for j in range(1, n):
        pre = np.empty(m)
        arg = np.empty(m, np.int32)
        run, run_k = -np.inf, 0
        for k in range(m):
            if best[k] > run or k == 0:
                run, run_k = best[k], k
            pre[k], arg[k] = run, run_k
        best = pre + S[:, j]
        back[j] = arg
    f = np.empty(n, np.int32)
    f[n - 1] = int(np.argmax(best))          # first maximum = smallest draft layer
    total = float(best[f[n - 1]])
    for j in range(n - 1, 0, -1):
        f[j - 1] = back[j][f[j]]
    return f, total
