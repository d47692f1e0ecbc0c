"""Seeded generators: draft attention rows, top-p row families, queries, hashed K/V pools,
block tables and layer maps.  Inputs only -- nothing of the method is computed here."""
from __future__ import annotations

import numpy as np

from . import bf16

__all__ = ["draft_probs", "topp_rows", "queries", "kv_values", "kv_pool", "kv_strides",
           "block_table", "layer_map", "ragged_lengths", "round_up"]

_M64 = (1 << 64) - 1


def round_up(x: int, m: int) -> int:
    return (x + m - 1) // m * m


def _rng(seed: int, *ids: int) -> np.random.Generator:
    k = 0x9E3779B97F4A7C15
    for v in ids:
        k = ((k ^ (int(v) & _M64)) * 0xBF58476D1CE4E5B9 + 0x94D049BB133111EB) & _M64
    return np.random.Generator(np.random.Philox(key=np.array([seed & _M64, k], dtype=np.uint64)))


# --------------------------------------------------------------------------- draft attention rows
def draft_probs(seed: int, layer: int, kv_len, n_heads: int, gamma: int, L_stride: int | None = None,
                sink=8.0, slope=0.002) -> np.ndarray:
    """Draft attention maps of one draft layer: float32 [B, n_heads, gamma, L_stride].

    Row (b, h, s) is the float32 softmax over positions i < kv_len[b] of
    logit = 3 z + sink [i < 4] + slope i with z ~ N(0, 1) iid; zero beyond kv_len[b].
    ``sink`` and ``slope`` are scalars or per-sequence arrays.
    """
    kv_len = np.asarray(kv_len, dtype=np.int64)
    B = len(kv_len)
    Ls = round_up(int(kv_len.max()), 4) if L_stride is None else int(L_stride)
    sink = np.broadcast_to(np.asarray(sink, dtype=np.float32), (B,))
    slope = np.broadcast_to(np.asarray(slope, dtype=np.float32), (B,))
    out = np.zeros((B, n_heads, gamma, Ls), dtype=np.float32)
    for b in range(B):
        L = int(kv_len[b])
        if L == 0:
            continue
        rng = _rng(seed, 1, layer, b)
        z = rng.standard_normal((n_heads, gamma, L), dtype=np.float32)
        pos = np.arange(L, dtype=np.float32)
        logit = np.float32(3.0) * z + slope[b] * pos
        logit[..., :4] += sink[b]
        logit -= logit.max(axis=-1, keepdims=True)
        np.exp(logit, out=logit)
        logit /= logit.sum(axis=-1, keepdims=True, dtype=np.float32)
        out[b, :, :, :L] = logit
    return out


def topp_rows(family: str, n_rows: int, n: int, seed: int) -> np.ndarray:
    """Probability rows of the selection micro-benchmark: float32 [n_rows, n], each summing to 1.

    uniform   iid U(0,1) values (flat)
    zipf      rank^-1.2 under a random permutation (peaked)
    quantised 2^(-j/4), j iid in 0..63: 64 distinct values, heavy ties
    """
    fam = {"uniform": 0, "zipf": 1, "quantised": 2}[family]
    rng = _rng(seed, 2, fam, n)
    if family == "uniform":
        a = rng.random((n_rows, n), dtype=np.float32)
    elif family == "zipf":
        base = (np.arange(1, n + 1, dtype=np.float64) ** -1.2).astype(np.float32)
        a = np.empty((n_rows, n), dtype=np.float32)
        for r in range(n_rows):
            a[r] = base[rng.permutation(n)]
    else:
        j = rng.integers(0, 64, size=(n_rows, n))
        a = np.exp2(-j / 4.0).astype(np.float32)
    a /= a.sum(axis=1, keepdims=True, dtype=np.float32)
    return a


def queries(seed: int, layer: int, B: int, T: int, n_q_heads: int, d: int) -> np.ndarray:
    """Verification queries, bf16 bits [B, T, H_q, d], ~N(0, 1)."""
    rng = _rng(seed, 3, layer)
    return bf16.from_f32(rng.standard_normal((B, T, n_q_heads, d), dtype=np.float32))


# --------------------------------------------------------------------------- hashed K/V pool
def _mix64(x):
    """A 64-bit finaliser (xor-shift-multiply rounds) on torch int64 tensors, wrap-around."""
    x = (x ^ ((x >> 30) & 0x3FFFFFFFF)) * (-4658895280553007687)   # 0xBF58476D1CE4E5B9
    x = (x ^ ((x >> 27) & 0x1FFFFFFFFF)) * (-7723592293110705685)  # 0x94D049BB133111EB
    return x ^ ((x >> 31) & 0x1FFFFFFFF)


def kv_values(seed: int, layer: int, flat_index):
    """bf16 K/V values as an integer-only function of (seed, layer, flat element index).

    Twelve 16-bit hash lanes are summed (Irwin-Hall, variance 1 after scaling), centred and
    divided by 65536, then rounded to bf16: bit-identical on CPU and CUDA tensors.
    ``flat_index`` is a torch int64 tensor of element offsets into the layer's pool.
    """
    import torch
    base = (int(seed) * 0x9E3779B97F4A7C15 + (int(layer) + 1) * 0xD1B54A32D192ED03) & _M64
    if base >= 1 << 63:
        base -= 1 << 64
    x = flat_index.to(torch.int64) * 3 + base
    acc = torch.zeros_like(x)
    for k in range(3):
        h = _mix64(x + k)
        acc += (h & 0xFFFF) + ((h >> 16) & 0xFFFF) + ((h >> 32) & 0xFFFF) + ((h >> 48) & 0xFFFF)
    val = (acc - 393210).to(torch.float32) / 65536.0
    return val.to(torch.bfloat16)


def kv_strides(page_size: int, n_kv_heads: int, d: int):
    """Element strides (page, kv, slot, head) of a pool laid out [n_pages, 2, page, H_kv, d]."""
    return (2 * page_size * n_kv_heads * d, page_size * n_kv_heads * d, n_kv_heads * d, d)


def kv_pool(seed: int, layer: int, n_pages: int, page_size: int, n_kv_heads: int, d: int,
            device="cpu", chunk_elems: int = 1 << 26, out=None):
    """One target layer's paged pool: torch bf16 [n_pages, 2, page_size, H_kv, d]."""
    import torch
    n = n_pages * 2 * page_size * n_kv_heads * d
    if out is None:
        out = torch.empty(n, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    for lo in range(0, n, chunk_elems):
        hi = min(n, lo + chunk_elems)
        flat[lo:hi] = kv_values(seed, layer, torch.arange(lo, hi, dtype=torch.int64, device=flat.device))
    return flat.view(n_pages, 2, page_size, n_kv_heads, d)


def block_table(seed: int, B: int, pages_per_seq: int, n_pages: int | None = None,
                shuffle: bool = True) -> np.ndarray:
    """int32 [B, pages_per_seq]: a seeded shuffle of the pool's page ids (identity if not shuffle)."""
    n_pages = B * pages_per_seq if n_pages is None else n_pages
    ids = _rng(seed, 4).permutation(n_pages) if shuffle else np.arange(n_pages)
    return ids[:B * pages_per_seq].reshape(B, pages_per_seq).astype(np.int32)


def layer_map(seed: int, n_target_layers: int, n_draft_layers: int, n_dense_first: int = 0) -> np.ndarray:
    """Monotone many-to-one map target layer -> draft layer (sorted iid draws); the first
    ``n_dense_first`` entries are -1 (dense layers)."""
    m = np.sort(_rng(seed, 5).integers(0, n_draft_layers, size=n_target_layers)).astype(np.int32)
    m[:n_dense_first] = -1
    return m


def ragged_lengths(seed: int, B: int, lo: int, hi: int):
    """Log-uniform context lengths in [lo, hi] plus per-sequence sink / slope strengths."""
    rng = _rng(seed, 6)
    L = np.rint(np.exp(rng.uniform(np.log(lo), np.log(hi), size=B))).astype(np.int32)
    sink = rng.uniform(4.0, 12.0, size=B).astype(np.float32)
    slope = (rng.uniform(0.0, 16.0, size=B) / L).astype(np.float32)
    return L, sink, slope
