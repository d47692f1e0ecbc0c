"""CPU oracle of the SpecAttn verification hot path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes binding over ``specattn_oracle.cpp`` (plain C++, binary64 masses and
attention, fixed-order binary32 aggregation).  Only the tests, the smoke check
and the benchmark's CPU-baseline leg may import this package; the CUDA library
and its Python binding never do, and this package never imports them.

Arrays are numpy; bf16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "specattn_oracle.cpp"
_LIB = _HERE / "libspecattn_oracle.so"

OK, INVALID_PROB, OVERFLOW = 0, 1, 2


def build(force: bool = False) -> Path:
    """Compile the oracle with g++ (no fast-math, no FMA contraction)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", str(_SRC), "-o", str(_LIB)]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(str(_LIB))
        _lib.specattn_oracle_nucleus.restype = C.c_int64
        _lib.specattn_oracle_aggregate.restype = C.c_int
        _lib.specattn_oracle_num_threads.restype = C.c_int
        _lib.specattn_oracle_select_topp.restype = None
        _lib.specattn_oracle_bisect.restype = C.c_int64
        _lib.specattn_oracle_select_variant.restype = None
        _lib.specattn_oracle_attend_rows.restype = None
        _lib.specattn_oracle_sparse_verify.restype = None
    return _lib


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    return int(lib().specattn_oracle_num_threads())


def aggregate(A: np.ndarray, L: int | None = None, head_group=None, g: int = 0):
    """O1 for one (layer, sequence, group).  A: [H_d, gamma, L_stride] float32."""
    A = _chk(A, np.float32)
    H, gamma, Ls = A.shape
    L = Ls if L is None else L
    hg = None if head_group is None else _chk(head_group, np.int32)
    out = np.zeros(L, dtype=np.float32)
    st = lib().specattn_oracle_aggregate(_p(A), H, gamma, C.c_int64(Ls), L, _p(hg), g, _p(out))
    return out, int(st)


def nucleus(a: np.ndarray, p: float, idx_cap: int | None = None):
    """O2 for one row.  Returns (idx[int32, ascending], count, diag dict)."""
    a = _chk(a, np.float32)
    L = a.shape[0]
    cap = L if idx_cap is None else idx_cap
    idx = np.full(max(cap, 1), -1, dtype=np.int32)
    diag = np.zeros(6, dtype=np.float64)
    n = lib().specattn_oracle_nucleus(_p(a), L, C.c_float(p), _p(idx), C.c_int64(cap), _p(diag))
    n = int(n)
    d = dict(total=diag[0], target=diag[1], m_gt=diag[2], m_ge=diag[3], margin=diag[4],
             theta=diag[5])
    return idx[:min(n, cap)].copy(), n, d


def select_topp(draft_probs, layer_map, kv_len, p, n_groups=1, head_group=None, idx_stride=None):
    """O1+O2 over a step.

    draft_probs: list (one per draft layer) of float32 [B, H_d, gamma, L_stride] or None.
    Returns idx [n_d, B, G, idx_stride] (-1 filled), counts, status, diag [n_d, B, G, 6].
    """
    n_d = len(draft_probs)
    ref = next(x for x in draft_probs if x is not None)
    B, H, gamma, Ls = ref.shape
    arrs = [None if x is None else _chk(x, np.float32) for x in draft_probs]
    for x in arrs:
        assert x is None or x.shape == (B, H, gamma, Ls)
    ptrs = (C.c_void_p * n_d)(*[None if x is None else x.ctypes.data for x in arrs])
    layer_map = _chk(layer_map, np.int32)
    kv_len = _chk(kv_len, np.int32)
    hg = None if head_group is None else _chk(head_group, np.int32)
    G = n_groups
    stride = int(Ls if idx_stride is None else idx_stride)
    idx = np.full((n_d, B, G, max(stride, 1)), -1, dtype=np.int32)
    counts = np.full((n_d, B, G), -1, dtype=np.int32)
    status = np.full((n_d, B, G), -1, dtype=np.int32)
    diag = np.zeros((n_d, B, G, 6), dtype=np.float64)
    lib().specattn_oracle_select_topp(ptrs, n_d, _p(layer_map), len(layer_map), B, H, gamma, G,
                                      C.c_int64(Ls), _p(kv_len), _p(hg), C.c_float(p), _p(idx),
                                      C.c_int64(stride), _p(counts), _p(status), _p(diag))
    return idx, counts, status, diag


def bisect(a: np.ndarray, p: float, n_iters: int = 10, idx_cap: int | None = None):
    """O2b for one row: Alg. 2's bisection with a fixed number of iterations.
    Returns (idx[int32, ascending], count, diag dict)."""
    a = _chk(a, np.float32)
    L = a.shape[0]
    cap = L if idx_cap is None else idx_cap
    idx = np.full(max(cap, 1), -1, dtype=np.int32)
    diag = np.zeros(6, dtype=np.float64)
    n = int(lib().specattn_oracle_bisect(_p(a), L, C.c_float(p), int(n_iters), _p(idx), C.c_int64(cap), _p(diag)))
    d = dict(total=diag[0], target=diag[1], kept_mass=diag[2], theta_mid=diag[3], margin=diag[4], max=diag[5])
    return idx[:min(n, cap)].copy(), n, d


def select_variant(draft_probs, layer_map, kv_len, p, *, per_step=False, n_iters=0, chunk=1, n_groups=1,
                   head_group=None, idx_stride=None):
    """O1+O2 over a step with Alg. 2's variants: per_step = one nucleus per speculated query,
    unioned; n_iters >= 1 = literal bisection; chunk > 1 = selection over per-chunk sums, kept
    chunks keep all their positions.  Same outputs as select_topp; diag[..., 4] is the
    smallest margin over the rows of a list."""
    n_d = len(draft_probs)
    ref = next(x for x in draft_probs if x is not None)
    B, H, gamma, Ls = ref.shape
    arrs = [None if x is None else _chk(x, np.float32) for x in draft_probs]
    ptrs = (C.c_void_p * n_d)(*[None if x is None else x.ctypes.data for x in arrs])
    layer_map = _chk(layer_map, np.int32)
    kv_len = _chk(kv_len, np.int32)
    hg = None if head_group is None else _chk(head_group, np.int32)
    G = n_groups
    stride = int(Ls if idx_stride is None else idx_stride)
    idx = np.full((n_d, B, G, max(stride, 1)), -1, dtype=np.int32)
    counts = np.full((n_d, B, G), -1, dtype=np.int32)
    status = np.full((n_d, B, G), -1, dtype=np.int32)
    diag = np.zeros((n_d, B, G, 6), dtype=np.float64)
    lib().specattn_oracle_select_variant(ptrs, n_d, _p(layer_map), len(layer_map), B, H, gamma, G,
                                         C.c_int64(Ls), _p(kv_len), _p(hg), C.c_float(p),
                                         int(bool(per_step)), int(n_iters), int(chunk), _p(idx), C.c_int64(stride),
                                         _p(counts), _p(status), _p(diag))
    return idx, counts, status, diag


def attend_rows(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float | None = None):
    """O3 core.  q [M, d], K/V [c, d] as uint16 bf16 bits.  Returns (out f64 [M,d], lse f64 [M])."""
    q = _chk(q, np.uint16)
    K = _chk(K, np.uint16)
    V = _chk(V, np.uint16)
    M, d = q.shape
    c = K.shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((M, d), dtype=np.float64)
    lse = np.zeros(M, dtype=np.float64)
    lib().specattn_oracle_attend_rows(_p(q), C.c_int64(d), _p(K), C.c_int64(d), _p(V),
                                      C.c_int64(d), M, C.c_int64(c), d, C.c_double(scale), _p(out),
                                      _p(lse))
    return out, lse


def sparse_verify(q, kv_pages, kv_strides, block_table, kv_len, idx, counts, *, n_kv_heads,
                  page_size, n_groups=1, dense=False, scale=0.0, pages_per_seq=None, tail_len=0):
    """O3 over one target layer.

    q [B,T,H_q,d] uint16; kv_pages any-shaped uint16 buffer with element strides
    kv_strides = (page, kv, slot, head); block_table [B, max_pages] int32 or None
    (contiguous; pages_per_seq then required); idx [B,G,idx_stride], counts [B,G].
    tail_len > 0: the in-flight tokens at positions kv_len[b] + j are attended causally.
    """
    q = _chk(q, np.uint16)
    B, T, Hq, d = q.shape
    kv_pages = _chk(kv_pages, np.uint16)
    kv_len = _chk(kv_len, np.int32)
    if block_table is not None:
        block_table = _chk(block_table, np.int32)
        bts = block_table.shape[1]
    else:
        bts = int(pages_per_seq)
    if dense:
        idx_a, cnt_a, istride = None, None, 0
    else:
        idx_a = _chk(idx, np.int32)
        cnt_a = _chk(counts, np.int32)
        istride = idx_a.shape[-1]
    out = np.zeros((B, T, Hq, d), dtype=np.float64)
    lse = np.zeros((B, T, Hq), dtype=np.float64)
    sp, sk, ss, sh = (int(x) for x in kv_strides)
    lib().specattn_oracle_sparse_verify(B, T, Hq, n_kv_heads, d, page_size, n_groups, _p(q),
                                        _p(kv_pages), C.c_int64(sp), C.c_int64(sk), C.c_int64(ss),
                                        C.c_int64(sh), _p(block_table), C.c_int64(bts), _p(kv_len),
                                        _p(idx_a), C.c_int64(istride), _p(cnt_a), int(bool(dense)),
                                        C.c_double(scale), int(tail_len), _p(out), _p(lse))
    return out, lse
