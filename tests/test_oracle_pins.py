"""Pins for the CPU oracle: each check ties it to something other than itself.

O1 (aggregate): exact dyadic sums, an order-sensitive binary32 chain, the R = 1 identity.
O2 (nucleus, App. A Eq. 7 / Alg. 2): hand-worked rows, brute force over all subsets,
    Alg. 2's bisection run to convergence, a numpy sort+cumsum reduction, closed forms and
    the set invariants.
O3 (attention, Eq. 1 restricted to I): a dense fp64 library softmax attention, one-token,
    zero-key, score-shift, permutation and LSE-merge identities, and the App. A error bound.
"""
import itertools
from pathlib import Path

import numpy as np
import pytest

import oracle
from workloads import bf16

GOLDEN = Path(__file__).resolve().parent / "golden"


# ----------------------------------------------------------------------------- O1
def test_aggregate_dyadic_exact():
    rng = np.random.default_rng(1)
    A = rng.integers(0, 1 << 10, size=(5, 3, 40)).astype(np.float32) / 1024.0
    a, st = oracle.aggregate(A)
    assert st == oracle.OK
    assert np.array_equal(a, A.astype(np.float64).sum(axis=(0, 1)).astype(np.float32))


def test_aggregate_order_is_heads_then_queries_in_binary32():
    # 2^24 + 1 rounds back to 2^24 in binary32 (ties to even); 1 + 1 + 2^24 is exact.
    big = np.float32(2.0 ** 24)
    A = np.zeros((2, 2, 1), dtype=np.float32)
    A[0, 0, 0], A[0, 1, 0], A[1, 0, 0], A[1, 1, 0] = big, 1.0, 1.0, 0.0
    a, _ = oracle.aggregate(A)
    assert a[0] == np.float32(16777216.0)  # ((2^24 + 1) + 1) + 0, every add rounded to binary32
    A[0, 0, 0], A[0, 1, 0], A[1, 0, 0], A[1, 1, 0] = 1.0, 1.0, big, 0.0
    a, _ = oracle.aggregate(A)
    assert a[0] == np.float32(16777218.0)
    # query index runs inside the head index
    A[0, 0, 0], A[0, 1, 0], A[1, 0, 0], A[1, 1, 0] = 1.0, big, 1.0, 0.0
    a, _ = oracle.aggregate(A)
    assert a[0] == np.float32(16777216.0)  # (1 + 2^24) -> 2^24, + 1 -> 2^24
    # a binary64 accumulator would have produced 2^24 + 2 in all three cases


def test_aggregate_identity_groups_and_validity():
    rng = np.random.default_rng(2)
    A = rng.random((1, 1, 33), dtype=np.float32)
    a, st = oracle.aggregate(A)
    assert st == oracle.OK and np.array_equal(a, A[0, 0])
    A = rng.integers(0, 64, size=(4, 2, 9)).astype(np.float32) / 64
    hg = np.array([1, 0, 1, 0], dtype=np.int32)
    a0, _ = oracle.aggregate(A, head_group=hg, g=0)
    a1, _ = oracle.aggregate(A, head_group=hg, g=1)
    assert np.array_equal(a0, A[[1, 3]].sum(axis=(0, 1)))
    assert np.array_equal(a1, A[[0, 2]].sum(axis=(0, 1)))
    for bad in (-0.25, np.nan, np.inf):
        B = A.copy()
        B[2, 1, 5] = bad
        assert oracle.aggregate(B)[1] == oracle.INVALID_PROB
    B = A.copy()
    B[0, 0, 0] = -0.0
    a, st = oracle.aggregate(B[:1, :1])
    assert st == oracle.OK and a[0] == 0.0 and not np.signbit(a[0])


# ----------------------------------------------------------------------------- O2
def _worked_rows():
    rows = []
    for line in (GOLDEN / "nucleus_worked_rows.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        p, vals, kept = (s.strip() for s in line.split("|"))
        rows.append((float(p), [float(v) for v in vals.split()], [int(k) for k in kept.split()]))
    return rows


@pytest.mark.parametrize("p,vals,kept", _worked_rows())
def test_nucleus_worked_rows(p, vals, kept):
    idx, n, d = oracle.nucleus(np.array(vals, dtype=np.float32), p)
    assert n == len(kept) and idx.tolist() == kept


def _brute_force_kept(a, target):
    """Union of all maximum-mass subsets among the smallest feasible cardinality (exact ints)."""
    n = len(a)
    for k in range(1, n + 1):
        best, sets = None, []
        for comb in itertools.combinations(range(n), k):
            m = sum(int(a[i]) for i in comb)
            if best is None or m > best:
                best, sets = m, [comb]
            elif m == best:
                sets.append(comb)
        if best >= target:
            return k, best, sorted(set().union(*[set(s) for s in sets]))
    raise AssertionError("infeasible")


@pytest.mark.parametrize("seed", range(12))
def test_nucleus_equals_brute_force_subset_enumeration(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(3, 13))
    levels = int(rng.choice([3, 8, 1 << 12]))  # few levels -> many ties
    a_int = rng.integers(0, levels, size=n).astype(np.int64)
    if a_int.sum() == 0:
        a_int[0] = 1
    # p = j/64 and integer values: p * total and every partial sum are exact
    for j in (1, 13, 32, 47, 60, 63):
        p = j / 64.0
        target_times_64 = j * int(a_int.sum())
        a = a_int.astype(np.float32) / np.float32(1 << 12)
        k, best, kept = _brute_force_kept(a_int * 64, target_times_64)
        idx, cnt, d = oracle.nucleus(a, p)
        assert idx.tolist() == kept
        # the minimal cardinality is the largest-first prefix length; ties only add positions
        srt = np.sort(a_int)[::-1]
        assert int(srt[:k].sum()) * 64 >= target_times_64 > (int(srt[:k - 1].sum()) * 64 if k > 1 else -1)
        assert cnt >= k


def _alg2_bisection(a, p, iters=200):
    """Alg. 2 for one row, run until the bracket stops moving; the returned set uses the
    lower bound, the bracket end that always satisfies the mass constraint."""
    a64 = a.astype(np.float64)
    target = np.float64(np.float32(p)) * a64.sum()
    lo, hi = np.float32(0.0), a.max()
    if a64[a >= hi].sum() >= target:  # the maximum alone (with its ties) already suffices
        return np.nonzero(a >= hi)[0]
    for _ in range(iters):
        mid = np.float32((np.float64(lo) + np.float64(hi)) / 2)
        if mid == lo or mid == hi:
            break
        if a64[a >= mid].sum() < target:
            hi = mid
        else:
            lo = mid
    return np.nonzero(a >= lo)[0] if lo > 0 else np.arange(len(a))[a >= lo]


@pytest.mark.parametrize("seed", range(8))
def test_nucleus_equals_alg2_bisection_at_convergence(seed):
    rng = np.random.default_rng(200 + seed)
    n = int(rng.integers(50, 3000))
    kind = seed % 4
    if kind == 0:
        a = rng.random(n, dtype=np.float32)
    elif kind == 1:
        a = (1.0 / np.arange(1, n + 1) ** 1.2).astype(np.float32)[rng.permutation(n)]
    elif kind == 2:
        a = np.exp2(-rng.integers(0, 64, size=n) / 4.0).astype(np.float32)
    else:
        z = rng.standard_normal(n).astype(np.float32) * 3
        a = np.exp(z - z.max()).astype(np.float32)
    a = (a / a.sum(dtype=np.float32)).astype(np.float32)
    for p in (0.5, 0.9, 0.99):
        idx, cnt, d = oracle.nucleus(a, p)
        if d["margin"] < 1e-12:
            continue  # the two summation orders may legitimately disagree in the last ulp
        assert np.array_equal(idx, _alg2_bisection(a, p).astype(np.int32))


@pytest.mark.parametrize("seed", range(6))
def test_nucleus_equals_numpy_sort_cumsum(seed):
    rng = np.random.default_rng(300 + seed)
    n = int(rng.integers(10, 5000))
    a = rng.random(n, dtype=np.float32) ** 4
    p = float(rng.choice([0.3, 0.8, 0.95, 0.999]))
    order = np.argsort(-a, kind="stable")
    csum = np.cumsum(a[order].astype(np.float64))
    target = np.float64(np.float32(p)) * a.astype(np.float64).sum()
    k = int(np.searchsorted(csum, target, side="left")) + 1
    theta = a[order[k - 1]]
    idx, cnt, d = oracle.nucleus(a, p)
    if d["margin"] < 1e-12:
        pytest.skip("decision within rounding of the summation order")
    assert np.array_equal(idx, np.nonzero(a >= theta)[0])
    assert d["theta"] == float(theta)


def test_nucleus_closed_forms():
    # geometric row 2^-(i+1), last element doubled so the row sums to 1: p = 1 - 2^-k keeps k
    n = 20
    a = np.exp2(-(np.arange(n) + 1.0)).astype(np.float32)
    a[-1] *= 2
    for k in range(1, n - 1):
        idx, cnt, _ = oracle.nucleus(a, float(np.float32(1 - 2.0 ** -k)))
        assert cnt == k and idx.tolist() == list(range(k))
    # constant row keeps everything for any p
    assert oracle.nucleus(np.full(37, 0.25, np.float32), 0.01)[1] == 37
    # one-hot
    a = np.zeros(100, np.float32)
    a[42] = 1
    assert oracle.nucleus(a, 0.999)[0].tolist() == [42]
    # empty row
    assert oracle.nucleus(np.zeros(0, np.float32), 0.5)[1] == 0
    # iid U(0,1): kept fraction -> 1 - sqrt(1 - p)
    rng = np.random.default_rng(7)
    a = rng.random(200000, dtype=np.float32)
    for p in (0.5, 0.9, 0.99):
        frac = oracle.nucleus(a, p)[1] / a.size
        assert abs(frac - (1 - np.sqrt(1 - p))) < 5e-3


@pytest.mark.parametrize("seed", range(6))
def test_nucleus_invariants(seed):
    rng = np.random.default_rng(400 + seed)
    n = int(rng.integers(5, 4000))
    a = (rng.random(n, dtype=np.float32) ** 6).astype(np.float32)
    a[rng.integers(0, n, size=n // 5)] = 0.0
    a[rng.integers(0, n, size=n // 7)] = a[0]  # ties
    prev = set()
    for p in (0.1, 0.5, 0.9, 0.97, 0.999):
        idx, cnt, d = oracle.nucleus(a, p)
        assert d["m_ge"] >= d["target"] > d["m_gt"] or d["total"] == 0
        assert d["target"] == np.float64(np.float32(p)) * d["total"]
        kept = set(idx.tolist())
        assert prev <= kept and np.all(np.diff(idx) > 0)
        prev = kept
        # mass bookkeeping against an independent fp64 sum
        assert np.isclose(d["m_ge"], a[idx].astype(np.float64).sum(), rtol=1e-12)
        # removing the whole tie group at the threshold drops the mass below the target
        th = np.float32(d["theta"])
        assert a[a > th].astype(np.float64).sum() < d["target"]
        # every kept value >= every dropped value
        dropped = np.setdiff1d(np.arange(n), idx)
        if dropped.size and idx.size:
            assert a[idx].min() > a[dropped].max()
        # permutation equivariance and power-of-two scaling
        perm = rng.permutation(n)
        idx_p, _, _ = oracle.nucleus(a[perm], p)
        assert set(perm[idx_p].tolist()) == kept
        idx_s, _, _ = oracle.nucleus(a * np.float32(2.0 ** -9), p)
        assert np.array_equal(idx_s, idx)
    idx, cnt, d = oracle.nucleus(a, 1.0)
    assert cnt == n and np.array_equal(idx, np.arange(n))


def test_nucleus_capacity_and_select_wrapper():
    rng = np.random.default_rng(5)
    B, H, g, L = 3, 4, 2, 257
    probs = [rng.random((B, H, g, L), dtype=np.float32), None, rng.random((B, H, g, L), dtype=np.float32)]
    kv_len = np.array([257, 100, 0], np.int32)
    layer_map = np.array([-1, 0, 0, 2], np.int32)
    idx, counts, status, diag = oracle.select_topp(probs, layer_map, kv_len, 0.7)
    assert np.all(counts[1] == -1) and np.all(status[1] == -1)  # unmapped layer untouched
    for u in (0, 2):
        for b in range(B):
            a, _ = oracle.aggregate(probs[u][b], L=int(kv_len[b]))
            ref, n, _ = oracle.nucleus(a, 0.7)
            assert counts[u, b, 0] == n and np.array_equal(idx[u, b, 0, :n], ref)
            assert status[u, b, 0] == oracle.OK
    idx, counts, status, _ = oracle.select_topp(probs, layer_map, kv_len, 0.7, idx_stride=16)
    assert status[0, 0, 0] == oracle.OVERFLOW and counts[0, 0, 0] > 16
    full, _, _ = oracle.nucleus(oracle.aggregate(probs[0][0])[0], 0.7)
    assert np.array_equal(idx[0, 0, 0], full[:16])
    # per-group lists
    hg = np.array([0, 0, 1, 1], np.int32)
    idx, counts, status, _ = oracle.select_topp(probs, layer_map, kv_len, 0.7, n_groups=2, head_group=hg)
    a, _ = oracle.aggregate(probs[2][1], L=100, head_group=hg, g=1)
    ref, n, _ = oracle.nucleus(a, 0.7)
    assert counts[2, 1, 1] == n and np.array_equal(idx[2, 1, 1, :n], ref)


# ----------------------------------------------------------------------------- O3
def _rand_bf16(rng, shape, scale=1.0):
    return bf16.from_f32(rng.standard_normal(shape).astype(np.float32) * scale)


def _torch_dense(qb, Kb, Vb):
    import torch
    q = torch.from_numpy(bf16.to_f32(qb).astype(np.float64))
    K = torch.from_numpy(bf16.to_f32(Kb).astype(np.float64))
    V = torch.from_numpy(bf16.to_f32(Vb).astype(np.float64))
    s = q @ K.T / np.sqrt(q.shape[1])
    return (torch.softmax(s, dim=-1) @ V).numpy(), torch.logsumexp(s, dim=-1).numpy()


def test_attend_rows_equals_library_dense_attention():
    rng = np.random.default_rng(11)
    for (M, c, d) in ((1, 1, 128), (5, 77, 128), (3, 500, 64)):
        q, K, V = _rand_bf16(rng, (M, d)), _rand_bf16(rng, (c, d)), _rand_bf16(rng, (c, d))
        out, lse = oracle.attend_rows(q, K, V)
        ro, rl = _torch_dense(q, K, V)
        assert np.allclose(out, ro, rtol=1e-12, atol=1e-13) and np.allclose(lse, rl, rtol=1e-12)


def test_attend_rows_identities():
    rng = np.random.default_rng(12)
    d = 128
    q = _rand_bf16(rng, (4, d))
    K, V = _rand_bf16(rng, (64, d)), _rand_bf16(rng, (64, d))
    # one token: output is that value row, LSE is its score
    out, lse = oracle.attend_rows(q, K[:1], V[:1])
    assert np.array_equal(out, np.broadcast_to(bf16.to_f32(V[:1]).astype(np.float64), out.shape))
    s0 = bf16.to_f32(q).astype(np.float64) @ bf16.to_f32(K[0]).astype(np.float64) / np.sqrt(d)
    assert np.allclose(lse, s0, rtol=1e-14)
    # all keys zero: uniform weights, LSE = ln c
    out, lse = oracle.attend_rows(q, np.zeros_like(K), V)
    assert np.allclose(out, bf16.to_f32(V).astype(np.float64).mean(0), rtol=1e-13)
    assert np.allclose(lse, np.log(64.0))
    # empty list
    out, lse = oracle.attend_rows(q, K[:0], V[:0])
    assert np.all(out == 0) and np.all(np.isneginf(lse))
    # permutation of the list changes nothing beyond rounding
    perm = rng.permutation(64)
    o1, l1 = oracle.attend_rows(q, K, V)
    o2, l2 = oracle.attend_rows(q, K[perm], V[perm])
    assert np.allclose(o1, o2, rtol=1e-12, atol=1e-14) and np.allclose(l1, l2, rtol=1e-13)
    # merging two disjoint sub-lists through their LSE gives the union
    oa, la = oracle.attend_rows(q, K[:20], V[:20])
    ob, lb = oracle.attend_rows(q, K[20:], V[20:])
    lm = np.logaddexp(la, lb)
    om = oa * np.exp(la - lm)[:, None] + ob * np.exp(lb - lm)[:, None]
    assert np.allclose(om, o1, rtol=1e-12, atol=1e-14) and np.allclose(lm, l1, rtol=1e-13)
    # explicit scale: doubling the scale equals doubling q (exact in bf16)
    q2 = bf16.from_f32(bf16.to_f32(q) * 2)
    o3, l3 = oracle.attend_rows(q2, K, V)
    o4, l4 = oracle.attend_rows(q, K, V, scale=2 / np.sqrt(d))
    assert np.allclose(o3, o4, rtol=1e-13) and np.allclose(l3, l4, rtol=1e-13)


def _paged_case(rng, B, T, Hq, Hkv, d, page, lens, shuffle=True):
    max_pages = (max(lens) + page - 1) // page
    n_pages = B * max_pages
    kv = _rand_bf16(rng, (n_pages, 2, page, Hkv, d))
    ids = rng.permutation(n_pages) if shuffle else np.arange(n_pages)
    bt = ids.reshape(B, max_pages).astype(np.int32)
    q = _rand_bf16(rng, (B, T, Hq, d))
    strides = (2 * page * Hkv * d, page * Hkv * d, Hkv * d, d)
    return q, kv, bt, strides


def test_sparse_verify_paged_matches_gathered_library_attention():
    rng = np.random.default_rng(13)
    B, T, Hq, Hkv, d, page = 3, 5, 8, 2, 128, 16
    lens = [45, 16, 130]
    q, kv, bt, strides = _paged_case(rng, B, T, Hq, Hkv, d, page, lens)
    kv_len = np.array(lens, np.int32)
    G = 1
    idx = np.full((B, G, 64), -1, np.int32)
    counts = np.zeros((B, G), np.int32)
    for b in range(B):
        sel = np.sort(rng.choice(lens[b], size=min(lens[b], 11 + 7 * b), replace=False))
        idx[b, 0, :len(sel)] = sel
        counts[b, 0] = len(sel)
    out, lse = oracle.sparse_verify(q, kv, strides, bt, kv_len, idx, counts, n_kv_heads=Hkv,
                                    page_size=page)
    for b in range(B):
        sel = idx[b, 0, :counts[b, 0]]
        for h in range(Hq):
            hk = h // (Hq // Hkv)
            K = np.stack([kv[bt[b, i // page], 0, i % page, hk] for i in sel])
            V = np.stack([kv[bt[b, i // page], 1, i % page, hk] for i in sel])
            ro, rl = _torch_dense(q[b, :, h], K, V)
            assert np.allclose(out[b, :, h], ro, rtol=1e-12, atol=1e-13)
            assert np.allclose(lse[b, :, h], rl, rtol=1e-12)
    # dense flag = every position below kv_len, lists unread; also the p = 1 list
    od, ld = oracle.sparse_verify(q, kv, strides, bt, kv_len, None, None, n_kv_heads=Hkv,
                                  page_size=page, dense=True)
    full = np.full((B, G, 130), -1, np.int32)
    fc = np.zeros((B, G), np.int32)
    for b in range(B):
        full[b, 0, :lens[b]] = np.arange(lens[b])
        fc[b, 0] = lens[b]
    of, lf = oracle.sparse_verify(q, kv, strides, bt, kv_len, full, fc, n_kv_heads=Hkv, page_size=page)
    assert np.array_equal(od, of) and np.array_equal(ld, lf)
    b, h = 2, 5
    K = np.stack([kv[bt[b, i // page], 0, i % page, h // 4] for i in range(lens[b])])
    V = np.stack([kv[bt[b, i // page], 1, i % page, h // 4] for i in range(lens[b])])
    ro, rl = _torch_dense(q[b, :, h], K, V)
    assert np.allclose(od[b, :, h], ro, rtol=1e-12, atol=1e-13)
    # contiguous cache (no block table) and per-kv-head lists
    qc, kvc, btc, strides = _paged_case(rng, 2, 2, 4, 2, 64, 8, [24, 24], shuffle=False)
    idx2 = np.array([[[0, 5, 23, -1], [1, 2, -1, -1]], [[7, -1, -1, -1], [3, 4, 5, 6]]], np.int32)
    cnt2 = np.array([[3, 2], [1, 4]], np.int32)
    o1, l1 = oracle.sparse_verify(qc, kvc, strides, btc, np.array([24, 24], np.int32), idx2, cnt2,
                                  n_kv_heads=2, page_size=8, n_groups=2)
    o2, l2 = oracle.sparse_verify(qc, kvc, strides, None, np.array([24, 24], np.int32), idx2, cnt2,
                                  n_kv_heads=2, page_size=8, n_groups=2, pages_per_seq=3)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)
    K = np.stack([kvc[3 + i // 8, 0, i % 8, 1] for i in (3, 4, 5, 6)])
    V = np.stack([kvc[3 + i // 8, 1, i % 8, 1] for i in (3, 4, 5, 6)])
    ro, rl = _torch_dense(qc[1, :, 3], K, V)
    assert np.allclose(o1[1, :, 3], ro, rtol=1e-12, atol=1e-13)


def test_joint_error_bound_of_appendix_a():
    """App. A: with the nucleus taken on the query's own attention weights, the masked,
    un-renormalised output is within (1 - kept mass) * max ||v|| <= (1 - p) * max ||v||."""
    rng = np.random.default_rng(14)
    d, L = 128, 600
    q = _rand_bf16(rng, (1, d), 2.0)
    K, V = _rand_bf16(rng, (L, d)), _rand_bf16(rng, (L, d))
    dense_o, dense_lse = oracle.attend_rows(q, K, V)
    s = bf16.to_f32(q).astype(np.float64) @ bf16.to_f32(K).astype(np.float64).T / np.sqrt(d)
    W = np.exp(s[0] - dense_lse[0]).astype(np.float32)
    vmax = np.linalg.norm(bf16.to_f32(V).astype(np.float64), axis=1).max()
    for p in (0.5, 0.8, 0.95, 0.99):
        idx, cnt, dg = oracle.nucleus(W, p)
        o, lse = oracle.attend_rows(q, K[idx], V[idx])
        masked = o * np.exp(lse - dense_lse)  # W Lambda_I V of Eq. 2
        err = np.linalg.norm(dense_o - masked)
        kept = dg["m_ge"] / dg["total"]
        assert err <= (1 - kept) * vmax * (1 + 1e-6) + 1e-9
        assert (1 - kept) <= (1 - p) + 1e-6


def test_sparse_verify_causal_tail_matches_library_attention_per_query():
    """The in-flight tokens (Alg. 1, "Verification with Sparse Attention": the gamma+1 tokens are
    verified in one pass) are attended causally on top of the list: query t sees tail tokens
    j <= t + tail_len - T.  Checked per query against a dense library softmax over that set."""
    rng = np.random.default_rng(15)
    B, T, Hq, Hkv, d, page = 2, 4, 4, 2, 128, 16
    lens = [40, 23]
    for tail in (4, 2, 6):
        q, kv, bt, strides = _paged_case(rng, B, T, Hq, Hkv, d, page, [x + tail for x in lens])
        kv_len = np.array(lens, np.int32)
        idx = np.full((B, 1, 16), -1, np.int32)
        counts = np.zeros((B, 1), np.int32)
        for b in range(B):
            sel = np.sort(rng.choice(lens[b], size=5 + 3 * b, replace=False))
            idx[b, 0, :len(sel)] = sel
            counts[b, 0] = len(sel)
        out, lse = oracle.sparse_verify(q, kv, strides, bt, kv_len, idx, counts, n_kv_heads=Hkv,
                                        page_size=page, tail_len=tail)
        for b in range(B):
            for t in range(T):
                n_tail = max(0, min(tail, t + tail - T + 1))
                pos = list(idx[b, 0, :counts[b, 0]]) + [lens[b] + j for j in range(n_tail)]
                for h in range(Hq):
                    hk = h // (Hq // Hkv)
                    K = np.stack([kv[bt[b, i // page], 0, i % page, hk] for i in pos])
                    V = np.stack([kv[bt[b, i // page], 1, i % page, hk] for i in pos])
                    ro, rl = _torch_dense(q[b, t:t + 1, h], K, V)
                    assert np.allclose(out[b, t, h], ro[0], rtol=1e-12, atol=1e-13)
                    assert np.allclose(lse[b, t, h], rl[0], rtol=1e-12)
    # tail_len = 0 is the plain call
    o0, l0 = oracle.sparse_verify(q, kv, strides, bt, kv_len, idx, counts, n_kv_heads=Hkv, page_size=page)
    o1, l1 = oracle.sparse_verify(q, kv, strides, bt, kv_len, idx, counts, n_kv_heads=Hkv, page_size=page, tail_len=0)
    assert np.array_equal(o0, o1) and np.array_equal(l0, l1)


# ---------------------------------------------------------------------------------------------
# O2b: Alg. 2's bisection taken literally (fixed iterations), and the per-step union
# ---------------------------------------------------------------------------------------------
def _bisection_rows():
    rows = []
    for line in (Path(__file__).parent / "golden" / "bisection_worked_rows.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        p, k, vals, kept, theta = [x.strip() for x in line.split("|")]
        rows.append((float(p), int(k), [float(v) for v in vals.split()], [int(v) for v in kept.split()], float(theta)))
    return rows


@pytest.mark.parametrize("p,k,vals,kept,theta", _bisection_rows())
def test_bisection_worked_rows(p, k, vals, kept, theta):
    idx, cnt, d = oracle.bisect(np.asarray(vals, np.float32), p, k)
    assert idx.tolist() == kept and cnt == len(kept)
    if p < 1.0:
        assert d["theta_mid"] == theta


def _rows_for_bisection(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(20, 4000))
    kind = seed % 3
    if kind == 0:
        a = rng.random(n, dtype=np.float32) ** 3
    elif kind == 1:
        a = (1.0 / np.arange(1, n + 1) ** 1.1).astype(np.float32)[rng.permutation(n)]
    else:
        z = rng.standard_normal(n).astype(np.float32) * 4
        a = np.exp(z - z.max()).astype(np.float32)
    return (a / a.sum(dtype=np.float32)).astype(np.float32)


@pytest.mark.parametrize("seed", range(9))
def test_bisection_is_a_scalar_bisection_against_the_exact_threshold(seed):
    # M(theta) = mass of {a >= theta} is non-increasing in theta, so "M(theta_mid) < target" holds
    # exactly when theta_mid lies above the exact threshold theta* of the sorted-prefix definition:
    # the literal loop must walk the same midpoints as a bisection that only knows theta* --
    # derived here from numpy's sort, not from the oracle's loop.
    a = _rows_for_bisection(400 + seed)
    for p in (0.5, 0.9, 0.97):
        order = np.argsort(-a, kind="stable")
        csum = np.cumsum(a[order].astype(np.float64))
        target = np.float64(np.float32(p)) * a.astype(np.float64).sum()
        theta_star = a[order[int(np.searchsorted(csum, target, side="left"))]]
        for k in (1, 3, 10, 30):
            idx, cnt, d = oracle.bisect(a, p, k)
            if d["margin"] < 1e-12:
                continue
            lo, hi, mid = np.float32(0), a.max(), np.float32(0)
            for _ in range(k):
                mid = np.float32((hi + lo) / np.float32(2))
                if mid > theta_star:
                    hi = mid
                else:
                    lo = mid
            assert d["theta_mid"] == float(mid)
            assert np.array_equal(idx, np.nonzero(a >= mid)[0])
            # the bracket halves every iteration and always holds theta*
            # (plus the rounding of k binary32 midpoints)
            assert abs(float(mid) - float(theta_star)) <= float(a.max()) * 2.0 ** (-k) + (k + 1) * float(np.spacing(a.max()))


@pytest.mark.parametrize("seed", range(6))
def test_bisection_at_convergence_is_the_nucleus_with_or_without_its_threshold_ties(seed):
    a = _rows_for_bisection(500 + seed)
    for p in (0.6, 0.95):
        nuc, _, dn = oracle.nucleus(a, p)
        idx, _, d = oracle.bisect(a, p, 60)
        if min(d["margin"], dn["margin"]) < 1e-12:
            continue
        theta = np.float32(dn["theta"])
        assert np.array_equal(idx, nuc) or np.array_equal(idx, np.nonzero(a > theta)[0])
        # short of the target by at most the mass tied at the threshold
        assert d["kept_mass"] >= dn["m_gt"] - 1e-12


def _numpy_nucleus(a, p):
    order = np.argsort(-a, kind="stable")
    csum = np.cumsum(a[order].astype(np.float64))
    target = np.float64(np.float32(p)) * a.astype(np.float64).sum()
    theta = a[order[int(np.searchsorted(csum, target, side="left"))]]
    return np.nonzero(a >= theta)[0]


@pytest.mark.parametrize("seed", range(5))
def test_per_step_union_equals_the_union_of_per_row_nuclei(seed):
    rng = np.random.default_rng(600 + seed)
    B, H, gamma, L = 2, 3, 4, int(rng.integers(40, 900))
    x = rng.random((B, H, gamma, L), dtype=np.float32) ** 4
    x /= x.sum(axis=-1, keepdims=True)
    x = x.astype(np.float32)
    kv_len = np.array([L, max(1, L // 3)], np.int32)
    p = 0.85
    idx, cnt, st, dg = oracle.select_variant([x], [0], kv_len, p, per_step=True)
    for b in range(B):
        Lb = int(kv_len[b])
        union = set()
        sizes = []
        for s in range(gamma):
            row = np.zeros(Lb, np.float32)
            for h in range(H):                      # heads ascending, binary32
                row = (row + x[b, h, s, :Lb]).astype(np.float32)
            kept = _numpy_nucleus(row, p)
            sizes.append(len(kept))
            union |= set(kept.tolist())
        if dg[0, b, 0, 4] < 1e-12:
            continue
        assert st[0, b, 0] == 0
        assert idx[0, b, 0, :cnt[0, b, 0]].tolist() == sorted(union)
        assert max(sizes) <= cnt[0, b, 0] <= sum(sizes)


def test_variant_special_cases():
    rng = np.random.default_rng(7)
    x = rng.random((1, 2, 1, 64), dtype=np.float32)
    kv = np.array([64], np.int32)
    # one speculated query: per-step selection is the aggregated selection
    a = oracle.select_topp([x], [0], kv, 0.9)
    b = oracle.select_variant([x], [0], kv, 0.9, per_step=True)
    c = oracle.select_variant([x], [0], kv, 0.9, per_step=False)
    for u, v in zip(a[:3], b[:3]):
        assert np.array_equal(u, v)
    for u, v in zip(a[:3], c[:3]):
        assert np.array_equal(u, v)
    # p >= 1 keeps everything in every variant; an invalid probability voids the list
    for per_step in (False, True):
        for it in (0, 10):
            i, n, s, _ = oracle.select_variant([x], [0], kv, 1.0, per_step=per_step, n_iters=it)
            assert n[0, 0, 0] == 64 and s[0, 0, 0] == 0
    y = np.tile(x, (1, 1, 3, 1)).copy()
    y[0, 1, 2, 5] = -0.25
    for per_step in (False, True):
        i, n, s, _ = oracle.select_variant([y], [0], kv, 0.9, per_step=per_step, n_iters=10)
        assert n[0, 0, 0] == 0 and s[0, 0, 0] == 1
    # truncation keeps the true count
    i, n, s, _ = oracle.select_variant([x], [0], kv, 0.99, per_step=True, idx_stride=4)
    assert n[0, 0, 0] > 4 and s[0, 0, 0] == 2 and np.all(np.diff(i[0, 0, 0]) > 0)


# ---------------------------------------------------------------------------------------------
# selection at chunk granularity
# ---------------------------------------------------------------------------------------------
def _chunk_rows():
    rows = []
    for line in (Path(__file__).parent / "golden" / "chunk_worked_rows.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        p, c, vals, kept = [x.strip() for x in line.split("|")]
        rows.append((float(p), int(c), [float(v) for v in vals.split()], [int(v) for v in kept.split()]))
    return rows


@pytest.mark.parametrize("p,chunk,vals,kept", _chunk_rows())
def test_chunk_selection_worked_rows(p, chunk, vals, kept):
    x = np.asarray(vals, np.float32).reshape(1, 1, 1, -1)
    idx, cnt, st, _ = oracle.select_variant([x], [0], np.array([x.shape[-1]], np.int32), p, chunk=chunk)
    assert st[0, 0, 0] == 0 and idx[0, 0, 0, :cnt[0, 0, 0]].tolist() == kept


@pytest.mark.parametrize("seed", range(5))
def test_chunk_selection_equals_numpy_nucleus_over_chunk_sums(seed):
    rng = np.random.default_rng(700 + seed)
    H, gamma, L = 2, 3, int(rng.integers(50, 2000))
    chunk = int(rng.choice([4, 16, 64]))
    x = (rng.random((1, H, gamma, L), dtype=np.float32) ** 5).astype(np.float32)
    kv = np.array([L - int(rng.integers(0, chunk))], np.int32)       # usually a cut last chunk
    Lb = int(kv[0])
    for per_step in (False, True):
        idx, cnt, st, dg = oracle.select_variant([x], [0], kv, 0.9, per_step=per_step, chunk=chunk)
        if dg[0, 0, 0, 4] < 1e-12:
            continue
        rows = []
        for s in (range(gamma) if per_step else [None]):
            row = np.zeros(Lb, np.float32)
            for h in range(H):                                  # heads ascending, queries inside
                for ss in ([s] if per_step else range(gamma)):
                    row = (row + x[0, h, ss, :Lb]).astype(np.float32)
            rows.append(row)
        want = set()
        for row in rows:
            nc = (Lb + chunk - 1) // chunk
            score = np.zeros(nc, np.float32)
            for j in range(nc):
                acc = np.float32(0)
                for v in row[j * chunk:(j + 1) * chunk]:
                    acc = np.float32(acc + v)
                score[j] = acc
            for j in _numpy_nucleus(score, 0.9):
                want |= set(range(j * chunk, min(Lb, (j + 1) * chunk)))
        got = idx[0, 0, 0, :cnt[0, 0, 0]].tolist()
        assert got == sorted(want)
        # whole chunks only
        kept = np.zeros(Lb, bool)
        kept[got] = True
        for j in range((Lb + chunk - 1) // chunk):
            seg = kept[j * chunk:(j + 1) * chunk]
            assert seg.all() or not seg.any()


def test_chunk_one_is_per_position_selection():
    rng = np.random.default_rng(9)
    x = rng.random((2, 2, 2, 300), dtype=np.float32)
    kv = np.array([300, 123], np.int32)
    for per_step, it in ((False, 0), (True, 0), (False, 10)):
        a = oracle.select_variant([x], [0], kv, 0.85, per_step=per_step, n_iters=it, chunk=1)
        b = oracle.select_variant([x], [0], kv, 0.85, per_step=per_step, n_iters=it)
        assert all(np.array_equal(u, v) for u, v in zip(a[:3], b[:3]))


# ---------------------------------------------------------------------------------------------
# the binary32 chain of an aggregated value must stay finite (reading of the input domain: Alg. 2
# and App. A Eq. 7 take attention probabilities; a sum that leaves binary32 is no such row)
# ---------------------------------------------------------------------------------------------
def _numpy_chain(values):
    """The defining chain ((+0 + x1) + x2) + ... with numpy's binary32 adds."""
    acc = np.float32(0.0)
    with np.errstate(over="ignore"):
        for v in values:
            acc = np.float32(acc + np.float32(v))
    return acc


FMAX = np.finfo(np.float32).max


@pytest.mark.parametrize("vals,finite", [
    ([3e38, 3e38], False),                 # two finite inputs whose binary32 sum is +inf
    ([FMAX, 0.0], True),                   # the largest finite value itself is a valid sum
    ([FMAX, FMAX * 2.0 ** -26], True),     # rounds back to FLT_MAX: still finite, still valid
    ([FMAX, FMAX * 2.0 ** -24], False),    # rounds up past FLT_MAX
    ([1e38, 1e38, 1e38], True),
    ([1e38, 1e38, 1e38, 1e38], False),
])
def test_aggregate_sum_overflow_marks_the_row_invalid(vals, finite):
    # what IEEE binary32 says about the chain, independent of the oracle
    assert bool(np.isfinite(_numpy_chain(vals))) == finite
    n = len(vals)
    A = np.zeros((n, 1, 8), dtype=np.float32)
    A[:, 0, 3] = np.array(vals, dtype=np.float32)
    A[0, 0, 1] = 0.5  # an ordinary position beside the overflowing one
    a, st = oracle.aggregate(A)
    assert st == (oracle.OK if finite else oracle.INVALID_PROB)
    assert a[3] == _numpy_chain(vals)      # the row is written either way
    # through the step-level entry points: the list is voided exactly when the chain overflows
    kv = np.array([8], np.int32)
    x = A[None]                            # [B=1, H=n, gamma=1, L]
    for call in (lambda: oracle.select_topp([x], [0], kv, 0.9),
                 lambda: oracle.select_variant([x], [0], kv, 0.9, per_step=True)):
        _, cnt, status, _ = call()
        assert status[0, 0, 0] == (oracle.OK if finite else oracle.INVALID_PROB)
        assert (cnt[0, 0, 0] > 0) == finite
    # heads as speculated queries: per_step sums over heads only, so each query's row is one value
    y = np.ascontiguousarray(np.transpose(x, (0, 2, 1, 3)))   # [1, 1, gamma=n, L]
    _, cnt, status, _ = oracle.select_variant([y], [0], kv, 0.9, per_step=True)
    assert status[0, 0, 0] == oracle.OK and cnt[0, 0, 0] > 0   # no chain is longer than one value
    _, cnt, status, _ = oracle.select_topp([y], [0], kv, 0.9)
    assert status[0, 0, 0] == (oracle.OK if finite else oracle.INVALID_PROB)


def test_chunk_score_overflow_marks_the_list_invalid():
    # positions stay finite, the binary32 sum of one chunk does not
    x = np.zeros((1, 1, 1, 16), dtype=np.float32)
    x[0, 0, 0, 4:8] = 1e38
    kv = np.array([16], np.int32)
    assert not np.isfinite(_numpy_chain(x[0, 0, 0, 4:8]))
    _, cnt, status, _ = oracle.select_variant([x], [0], kv, 0.9, chunk=4)
    assert status[0, 0, 0] == oracle.INVALID_PROB and cnt[0, 0, 0] == 0
    _, cnt, status, _ = oracle.select_variant([x], [0], kv, 0.9, chunk=1)
    assert status[0, 0, 0] == oracle.OK and cnt[0, 0, 0] == 4
    x[0, 0, 0, 7] = 0.0                     # three of them fit
    assert np.isfinite(_numpy_chain(x[0, 0, 0, 4:8]))
    idx, cnt, status, _ = oracle.select_variant([x], [0], kv, 0.9, chunk=4)
    assert status[0, 0, 0] == oracle.OK and idx[0, 0, 0, :cnt[0, 0, 0]].tolist() == [4, 5, 6, 7]
