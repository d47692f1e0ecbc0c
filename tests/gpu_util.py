"""Helpers shared by the GPU parity tests: comparison of index lists and attention outputs
against the CPU oracle under the gates of the task (bit-exact lists except rows whose boundary
mass is within 1e-5 of p; outputs within 2e-3 max-abs; LSE within 1e-4 relative)."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from workloads import bf16

OUT_TOL = 2e-3
LSE_TOL = 1e-4
NEAR = 1e-5


def dev():
    return torch.device("cuda:0")


def to_dev(a: np.ndarray, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(dev())


def bf16_to_dev(bits: np.ndarray):
    return bf16.bits_to_torch(bits).to(dev())


def compare_lists(a_rows, p, g_idx, g_counts, g_status, o_idx, o_counts, o_status, o_diag):
    """Compares every list (flattened leading dims).  ``a_rows`` maps a flat list id to its
    aggregated row (callable) for validating near-boundary rows.  Returns
    dict(n, exact, near_boundary, near_boundary_exact)."""
    g_idx = g_idx.reshape(-1, g_idx.shape[-1])
    o_idx = o_idx.reshape(-1, o_idx.shape[-1])
    g_counts, o_counts = g_counts.reshape(-1), o_counts.reshape(-1)
    g_status, o_status = g_status.reshape(-1), o_status.reshape(-1)
    o_diag = o_diag.reshape(-1, o_diag.shape[-1])
    stats = dict(n=0, exact=0, near_boundary=0, near_boundary_exact=0)
    for i in range(len(o_counts)):
        if o_counts[i] < 0:      # list of an unmapped draft layer: untouched on both sides
            continue
        stats["n"] += 1
        assert g_status[i] == o_status[i], f"list {i}: status {g_status[i]} vs oracle {o_status[i]}"
        if o_status[i] == oracle.INVALID_PROB:
            assert g_counts[i] == 0
            stats["exact"] += 1
            continue
        near = o_diag[i, 4] <= NEAR
        stats["near_boundary"] += int(near)
        n = min(int(o_counts[i]), o_idx.shape[1])
        same = g_counts[i] == o_counts[i] and np.array_equal(g_idx[i, :n], o_idx[i, :n])
        if same:
            stats["exact"] += 1
            stats["near_boundary_exact"] += int(near)
            continue
        assert near, (f"list {i}: GPU list differs from the oracle (count {g_counts[i]} vs "
                      f"{o_counts[i]}) and the row is not near-boundary (margin {o_diag[i, 4]:.3e})")
        # a near-boundary row may take a neighbouring threshold, but must still be a threshold
        # set whose mass is within the band around the target
        a = a_rows(i)
        gc = int(g_counts[i])
        kept = g_idx[i, :gc]
        assert np.all(np.diff(kept) > 0)
        mask = np.zeros(len(a), bool)
        mask[kept] = True
        assert a[mask].min() > a[~mask].max() if (~mask).any() and mask.any() else True
        total, target = o_diag[i, 0], o_diag[i, 1]
        m_ge = a[mask].astype(np.float64).sum()
        m_gt = a[a > a[mask].min()].astype(np.float64).sum()
        assert m_ge >= target - NEAR * total and m_gt < target + NEAR * total
    return stats


def lse_err(got: np.ndarray, ref: np.ndarray) -> float:
    both_inf = np.isneginf(got) & np.isneginf(ref)
    with np.errstate(invalid="ignore"):
        diff = got - ref
    d = np.abs(np.where(both_inf, 0.0, diff)) / np.maximum(1.0, np.abs(np.where(both_inf, 0.0, ref)))
    return float(np.max(d)) if d.size else 0.0


def check_attention(out_g: torch.Tensor, lse_g: torch.Tensor, out_o: np.ndarray, lse_o: np.ndarray):
    og = out_g.detach().cpu().numpy().astype(np.float64)
    lg = lse_g.detach().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(og))
    e_out = float(np.max(np.abs(og - out_o))) if og.size else 0.0
    e_lse = lse_err(lg, lse_o)
    assert e_out <= OUT_TOL, f"attention output max-abs error {e_out:.3e} > {OUT_TOL}"
    assert e_lse <= LSE_TOL, f"LSE relative error {e_lse:.3e} > {LSE_TOL}"
    return e_out, e_lse
