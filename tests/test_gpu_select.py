"""GPU parity of specattn_select_topp (through the C ABI) against the CPU oracle.

Index lists must match the sorted-prefix nucleus of App. A Eq. 7 / Alg. 2 bit for bit; rows whose
boundary mass lies within 1e-5 of p are counted apart and may only differ by a neighbouring
threshold."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from gpu_util import compare_lists, dev, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(params=["two_launch", "cluster"], autouse=True)
def form(request, monkeypatch):
    """Every case runs once per form of the call: with a workspace (aggregation launch + search
    launch, where the shape allows it) and without (one cluster per list)."""
    import functools
    import paper_2510_27641_b200 as sa
    monkeypatch.setattr(sa, "select_topp", functools.partial(sa.select_topp, workspace=request.param == "two_launch"))
    return request.param


def _run_rows(rows: np.ndarray, kv_len, p, idx_stride=None):
    """R = 1: each row is its own list.  rows [n_rows, L_stride] float32."""
    import paper_2510_27641_b200 as sa
    n_rows, Ls = rows.shape
    kv = np.asarray(kv_len, np.int32) if np.ndim(kv_len) else np.full(n_rows, kv_len, np.int32)
    probs = rows.reshape(n_rows, 1, 1, Ls)
    gi, gc, gs, gd = sa.select_topp([to_dev(probs)], to_dev(kv), [0], p, idx_stride=idx_stride,
                                    want_diag=True)
    torch.cuda.synchronize()
    oi, oc, os_, od = oracle.select_topp([probs], np.zeros(1, np.int32), kv, p, idx_stride=idx_stride)
    st = compare_lists(lambda i: rows[i, :kv[i]], p, gi.cpu().numpy(), gc.cpu().numpy(),
                       gs.cpu().numpy(), oi, oc, os_, od)
    return st, gd.cpu().numpy(), od


@pytest.mark.parametrize("family", wl.TOPP_FAMILIES)
@pytest.mark.parametrize("n", [1024, 8192, 40000])
def test_row_families_match_oracle(family, n):
    rows = wl.topp_rows(family, 24, n, seed=n)
    for p in wl.TOPP_PS:
        st, gd, od = _run_rows(rows, n, p)
        assert st["n"] == 24
        # masses reported by the kernel agree with the oracle's binary64 sums
        assert np.allclose(gd.reshape(-1, 4), od.reshape(-1, 6)[:, :4], rtol=1e-9, atol=0)


def test_long_rows_span_a_full_cluster():
    rows = wl.topp_rows("uniform", 3, 131072, seed=5)
    rows = np.concatenate([rows, wl.topp_rows("quantised", 3, 131072, seed=6),
                           wl.topp_rows("zipf", 2, 131072, seed=7)])
    for p in (0.5, 0.99):
        st, _, _ = _run_rows(rows, 131072, p)
        assert st["n"] == 8


def test_ragged_lengths_and_tails():
    rng = np.random.default_rng(0)
    Ls = 5000
    lens = np.array([0, 1, 2, 3, 4, 5, 31, 32, 33, 1023, 1025, 4093, 4999, 5000], np.int32)
    rows = np.zeros((len(lens), Ls), np.float32)
    for i, L in enumerate(lens):
        rows[i, :L] = rng.random(L, dtype=np.float32) ** 3
        rows[i, L:] = 7.0      # beyond kv_len: must be ignored entirely
    for p in (0.3, 0.9):
        st, _, _ = _run_rows(rows, lens, p)
        assert st["n"] == len(lens)


def test_degenerate_rows():
    n = 4096
    rows = np.zeros((8, n), np.float32)
    rows[0] = 0.25                       # constant: everything ties
    rows[1, 1234] = 1.0                  # one-hot
    # row 2 all zero: everything ties at zero
    rows[3] = np.float32(1e-42)          # denormal constant
    rows[4, :] = np.where(np.arange(n) % 2 == 0, 0.5, 0.0)
    rows[5, :100] = np.exp2(-np.arange(100, dtype=np.float32))  # spans 100 exponents
    rows[6, :] = 1.0
    rows[6, 7] = 3.0e38                  # huge dynamic range
    rows[7, :] = np.float32(np.nextafter(np.float32(1), np.float32(2)))
    rows[7, ::3] = 1.0                   # two values one ulp apart
    for p in (0.001, 0.5, 0.999):
        st, _, _ = _run_rows(rows, n, p)
        assert st["n"] == 8
    import paper_2510_27641_b200 as sa
    gi, gc, gs, _ = sa.select_topp([to_dev(rows.reshape(8, 1, 1, n))], to_dev(np.full(8, n, np.int32)), [0], 0.5)
    assert gc.cpu().numpy().ravel().tolist()[:3] == [n, 1, n]


def test_p_one_keeps_everything_and_zeros():
    rows = wl.topp_rows("zipf", 4, 3000, seed=1)
    rows[:, ::7] = 0.0
    st, _, _ = _run_rows(rows, np.array([3000, 2999, 17, 0], np.int32), 1.0)
    assert st["exact"] == 4


def test_invalid_probabilities_are_flagged_per_list():
    import paper_2510_27641_b200 as sa
    rows = wl.topp_rows("uniform", 6, 9000, seed=2)
    rows[1, 8999] = np.nan
    rows[2, 0] = -1e-30
    rows[3, 4500] = np.inf
    rows[4, 100] = -0.0          # minus zero is a valid zero
    rows[5, 8000] = -1.0         # beyond kv_len below: not an input
    kv = np.array([9000, 9000, 9000, 9000, 9000, 7000], np.int32)
    st, _, _ = _run_rows(rows, kv, 0.9)
    assert st["n"] == 6
    _, _, gs, _ = sa.select_topp([to_dev(rows.reshape(6, 1, 1, 9000))], to_dev(kv), [0], 0.9)
    assert gs.cpu().numpy().ravel().tolist() == [0, sa.ROW_INVALID_PROB, sa.ROW_INVALID_PROB,
                                                 sa.ROW_INVALID_PROB, 0, 0]


def test_capacity_overflow_truncates_and_reports_true_count():
    rows = wl.topp_rows("uniform", 5, 4096, seed=3)
    st, _, _ = _run_rows(rows, 4096, 0.9, idx_stride=100)
    assert st["n"] == 5


@pytest.mark.parametrize("G", [1, 2, 4])
def test_aggregation_over_heads_queries_layers_and_groups(G):
    import paper_2510_27641_b200 as sa
    B, H, gamma, n_d = 3, 12, 5, 3
    kv_len = np.array([4096, 1000, 2731], np.int32)
    Ls = 4096
    probs = [wl.draft_probs(7, u, kv_len, H, gamma, Ls, sink=6.0, slope=0.004) if u != 1 else None
             for u in range(n_d)]
    layer_map = np.array([-1, 0, 0, 2, 2, 2], np.int32)
    hg = None if G == 1 else (np.arange(H) * G // H).astype(np.int32)
    for p in (0.9, 0.95):
        gi, gc, gs, gd = sa.select_topp([None if x is None else to_dev(x) for x in probs], to_dev(kv_len),
                                        layer_map.tolist(), p, n_groups=G,
                                        head_group=None if hg is None else hg.tolist(), want_diag=True)
        torch.cuda.synchronize()
        oi, oc, os_, od = oracle.select_topp(probs, layer_map, kv_len, p, n_groups=G, head_group=hg)

        def row(i):
            u, b, g = i // (B * G), (i // G) % B, i % G
            return oracle.aggregate(probs[u][b], L=int(kv_len[b]), head_group=hg, g=g)[0]

        st = compare_lists(row, p, gi.cpu().numpy(), gc.cpu().numpy(), gs.cpu().numpy(), oi, oc, os_, od)
        assert st["n"] == 2 * B * G
        assert np.all(gc.cpu().numpy()[1] == -1)      # unmapped layer untouched


def test_order_of_the_binary32_adds_is_heads_then_queries():
    import paper_2510_27641_b200 as sa
    big = np.float32(2.0 ** 24)
    A = np.zeros((1, 2, 2, 8), np.float32)
    A[0, :, :, 0] = [[big, 1.0], [1.0, 0.0]]    # ((2^24 + 1) + 1) + 0 = 2^24 in binary32
    A[0, :, :, 1] = [[1.0, 1.0], [big, 0.0]]    # exact 2^24 + 2
    A[0, :, :, 2] = 16777217.5                  # rounds per add; just another large value
    A[0, :, :, 3:] = 1.0
    kv = np.array([8], np.int32)
    gi, gc, _, gd = sa.select_topp([to_dev(A)], to_dev(kv), [0], 0.2, want_diag=True)
    oi, oc, _, od = oracle.select_topp([A], np.zeros(1, np.int32), kv, 0.2)
    assert gc.item() == oc.item() and np.array_equal(gi.cpu().numpy()[0, 0, 0, :oc.item()], oi[0, 0, 0, :oc.item()])
    assert gd.cpu().numpy()[0, 0, 0, 0] == od[0, 0, 0, 0]   # totals equal bit for bit: same a_bar


def test_argument_errors_are_synchronous_and_launch_nothing():
    import paper_2510_27641_b200 as sa
    probs = to_dev(wl.topp_rows("uniform", 2, 1024, 0).reshape(2, 1, 1, 1024))
    kv = to_dev(np.full(2, 1024, np.int32))
    before = sa.kernel_launch_count()
    for bad_p in (0.0, -0.5, float("nan")):
        with pytest.raises(sa.SpecAttnError) as e:
            sa.select_topp([probs], kv, [0], bad_p)
        assert e.value.code == -3
    with pytest.raises(sa.SpecAttnError) as e:
        sa.select_topp([probs], kv, [1], 0.5)          # layer_map out of range
    assert e.value.code == -3
    with pytest.raises(sa.SpecAttnError) as e:
        sa.select_topp([probs[:, :, :, :1022].contiguous()], kv, [0], 0.5)   # L_stride % 4 != 0
    assert e.value.code == -4
    assert sa.kernel_launch_count() == before
    # repeated calls are deterministic
    a = sa.select_topp([probs], kv, [0], 0.7)
    b = sa.select_topp([probs], kv, [0], 0.7)
    torch.cuda.synchronize()
    assert torch.equal(a[1], b[1])
    n = int(a[1][0, 0, 0])
    assert torch.equal(a[0][0, 0, 0, :n], b[0][0, 0, 0, :n])
    assert sa.kernel_launch_count() == before + 2


# ---------------------------------------------------------------------------------------------
# Alg. 2's variants: one nucleus per speculated query, unioned; fixed-iteration bisection
# ---------------------------------------------------------------------------------------------
def _compare_variant(gi, gc, gs, oi, oc, os_, od):
    """Lists must equal the oracle's bit for bit unless one of the oracle's comparisons was
    within NEAR of flipping (a binary64 sum in another order may then decide otherwise)."""
    from gpu_util import NEAR
    gi, gc, gs = gi.cpu().numpy(), gc.cpu().numpy(), gs.cpu().numpy()
    n = near = 0
    for i in np.ndindex(oc.shape):
        if oc[i] < 0:
            assert gc[i] == -1
            continue
        n += 1
        assert gs[i] == os_[i]
        k = min(int(oc[i]), oi.shape[-1])
        if gc[i] == oc[i] and np.array_equal(gi[i][:k], oi[i][:k]):
            continue
        assert od[i][4] <= NEAR, f"list {i}: count {gc[i]} vs oracle {oc[i]}, margin {od[i][4]:.3e}"
        near += 1
    assert near <= max(1, n // 20)
    return n


@pytest.mark.parametrize("per_step,iters", [(True, 0), (False, 10), (True, 10), (False, 3), (True, 1), (False, 40)])
def test_selection_variants_match_oracle(per_step, iters):
    import paper_2510_27641_b200 as sa
    # (a) ragged lengths, two draft layers, per-group head sets; (b) rows that span a cluster
    cases = [(3, 8, 5, 4096, np.array([4096, 1000, 2731], np.int32), 2),
             (2, 3, 4, 40000, np.array([40000, 33333], np.int32), 1)]
    for B, H, gamma, Ls, kv_len, G in cases:
        probs = [wl.draft_probs(11, u, kv_len, H, gamma, Ls, sink=6.0, slope=0.004) for u in range(2)]
        hg = None if G == 1 else (np.arange(H) * G // H).astype(np.int32)
        for p in (0.8, 0.95):
            gi, gc, gs, _ = sa.select_topp([to_dev(x) for x in probs], to_dev(kv_len), [0, 1, 1], p, n_groups=G,
                                           head_group=None if hg is None else hg.tolist(),
                                           per_step=per_step, bisect_iters=iters)
            torch.cuda.synchronize()
            oi, oc, os_, od = oracle.select_variant(probs, [0, 1, 1], kv_len, p, per_step=per_step, n_iters=iters,
                                                    n_groups=G, head_group=hg)
            assert _compare_variant(gi, gc, gs, oi, oc, os_, od) == 2 * B * G


def test_selection_variants_special_cases():
    import paper_2510_27641_b200 as sa
    kv = np.array([3000, 17], np.int32)
    probs = wl.draft_probs(12, 0, kv, 4, 3, 3008, sink=6.0, slope=0.004)
    d = to_dev(probs)
    # p >= 1 keeps everything whatever the variant
    for per_step, iters in ((True, 0), (False, 10), (True, 10)):
        gi, gc, gs, _ = sa.select_topp([d], to_dev(kv), [0], 1.0, per_step=per_step, bisect_iters=iters)
        assert gc.cpu().numpy().reshape(-1).tolist() == [3000, 17] and int(gs.abs().sum()) == 0
    # a negative probability in any query's row voids the list in the per-step variant too
    bad = probs.copy()
    bad[0, 2, 1, 77] = -1e-3
    gi, gc, gs, _ = sa.select_topp([to_dev(bad)], to_dev(kv), [0], 0.9, per_step=True, bisect_iters=10)
    oi, oc, os_, od = oracle.select_variant([bad], [0], kv, 0.9, per_step=True, n_iters=10)
    assert gs.cpu().numpy().reshape(-1).tolist() == os_.reshape(-1).tolist() == [sa.ROW_INVALID_PROB, 0]
    assert gc.cpu().numpy().reshape(-1).tolist() == oc.reshape(-1).tolist()
    # a single long row (read in place) with the literal bisection
    row = wl.topp_rows("zipf", 2, 65536, 3).reshape(2, 1, 1, 65536)
    kv1 = np.array([65536, 50001], np.int32)
    gi, gc, gs, _ = sa.select_topp([to_dev(row)], to_dev(kv1), [0], 0.9, bisect_iters=10)
    oi, oc, os_, od = oracle.select_variant([row], [0], kv1, 0.9, n_iters=10)
    _compare_variant(gi, gc, gs, oi, oc, os_, od)
    # out-of-range variant arguments are refused synchronously
    a, keep = sa.make_select_args([d], to_dev(kv), [0], 0.9, idx=gi.new_zeros((1, 2, 1, 8)), counts=gc.new_zeros((1, 2, 1)),
                                  row_status=gs.new_zeros((1, 2, 1)), bisect_iters=65)
    assert sa.lib().specattn_select_topp(C.byref(a), None) == -3


@pytest.mark.parametrize("chunk,per_step,iters", [(16, False, 0), (16, True, 0), (16, False, 10), (4, True, 10),
                                                  (64, False, 0), (8, True, 0), (32, False, 5)])
def test_chunk_granular_selection_matches_oracle(chunk, per_step, iters):
    import paper_2510_27641_b200 as sa
    # lengths that are not multiples of the chunk; rows that span a cluster; per-group head sets
    cases = [(3, 8, 5, 4096, np.array([4096, 1000, 2731], np.int32), 2),
             (2, 3, 4, 40000, np.array([40000, 33333], np.int32), 1),
             (2, 2, 2, 64, np.array([3, 64], np.int32), 1)]
    for B, H, gamma, Ls, kv_len, G in cases:
        probs = [wl.draft_probs(13, u, kv_len, H, gamma, Ls, sink=6.0, slope=0.004) for u in range(2)]
        hg = None if G == 1 else (np.arange(H) * G // H).astype(np.int32)
        for p in (0.8, 0.95):
            gi, gc, gs, _ = sa.select_topp([to_dev(x) for x in probs], to_dev(kv_len), [1, 0], p, n_groups=G,
                                           head_group=None if hg is None else hg.tolist(),
                                           per_step=per_step, bisect_iters=iters, chunk=chunk)
            torch.cuda.synchronize()
            oi, oc, os_, od = oracle.select_variant(probs, [1, 0], kv_len, p, per_step=per_step, n_iters=iters,
                                                    chunk=chunk, n_groups=G, head_group=hg)
            assert _compare_variant(gi, gc, gs, oi, oc, os_, od) == 2 * B * G
            # whole chunks only (the last one cut at kv_len)
            g_idx, g_cnt = gi.cpu().numpy(), gc.cpu().numpy()
            for b in range(B):
                kept = np.zeros(int(kv_len[b]), bool)
                kept[g_idx[0, b, 0, :g_cnt[0, b, 0]]] = True
                for j in range(0, int(kv_len[b]), chunk):
                    assert kept[j:j + chunk].all() or not kept[j:j + chunk].any()


def test_chunk_selection_overflow_single_row_and_arguments():
    import paper_2510_27641_b200 as sa
    kv = np.array([5000], np.int32)
    probs = wl.draft_probs(14, 0, kv, 2, 2, 5000, sink=6.0, slope=0.004)
    # the list is cut to idx_stride positions (in the middle of a chunk), the count stays true
    gi, gc, gs, _ = sa.select_topp([to_dev(probs)], to_dev(kv), [0], 0.99, chunk=16, idx_stride=40)
    oi, oc, os_, od = oracle.select_variant([probs], [0], kv, 0.99, chunk=16, idx_stride=40)
    assert gc.item() == oc.item() > 40 and gs.item() == os_.item() == sa.ROW_OVERFLOW
    assert np.array_equal(gi.cpu().numpy()[0, 0, 0], oi[0, 0, 0])
    # one long row: chunked selection does not take the in-place path
    row = wl.topp_rows("zipf", 1, 65536, 5).reshape(1, 1, 1, 65536)
    kv1 = np.array([65530], np.int32)
    gi, gc, gs, _ = sa.select_topp([to_dev(row)], to_dev(kv1), [0], 0.9, chunk=16)
    oi, oc, os_, od = oracle.select_variant([row], [0], kv1, 0.9, chunk=16)
    _compare_variant(gi, gc, gs, oi, oc, os_, od)
    for bad_chunk in (2, 3, 12, 128, -1):
        a, keep = sa.make_select_args([to_dev(probs)], to_dev(kv), [0], 0.9, idx=gi.new_zeros((1, 1, 1, 8)),
                                      counts=gc.new_zeros((1, 1, 1)), row_status=gs.new_zeros((1, 1, 1)), chunk=bad_chunk)
        assert sa.lib().specattn_select_topp(C.byref(a), None) == -3


def test_both_forms_give_the_same_bits_and_flag_hidden_negative_inputs(form):
    """Multi-row lists: the two-launch form (workspace) and the cluster form must agree bit for
    bit (lists, counts, status, diag), also for ragged lengths, head groups and invalid inputs --
    a negative input that the sum hides, NaN, Inf, and garbage beyond kv_len."""
    import paper_2510_27641_b200 as sa
    B, H, gamma, Ls = 5, 6, 3, 6144
    kv_len = np.array([6144, 2049, 5000, 6144, 3000], np.int32)
    probs = wl.draft_probs(11, 0, kv_len, H, gamma, Ls, sink=6.0, slope=0.004)
    probs[1, 2, 1, 700] = -1e-30        # hidden by the other 17 rows' mass
    probs[2, 0, 0, 4999] = np.nan
    probs[3, 5, 2, 6143] = np.inf
    probs[4, :, :, 3000:] = -5.0        # beyond kv_len: not inputs
    hg = (np.arange(H) * 2 // H).astype(np.int32)
    d = to_dev(probs)
    res = {}
    for ws in (True, False):
        n0 = sa.lib().specattn_kernel_launch_count()
        gi, gc, gs, gd = sa.select_topp.func([d], to_dev(kv_len), [0], 0.9, n_groups=2, head_group=hg.tolist(),
                                             want_diag=True, workspace=ws)
        torch.cuda.synchronize()
        assert sa.lib().specattn_kernel_launch_count() - n0 == (2 if ws else 1)   # the form asked for ran
        res[ws] = (gi.cpu().numpy(), gc.cpu().numpy(), gs.cpu().numpy(), gd.cpu().numpy())
    (i1, c1, s1, d1), (i0, c0, s0, d0) = res[True], res[False]
    assert np.array_equal(c1, c0) and np.array_equal(s1, s0)
    ok = s0 == 0
    assert np.array_equal(d1[ok], d0[ok])
    for b in range(B):
        for g in range(2):
            assert np.array_equal(i1[0, b, g, :c0[0, b, g]], i0[0, b, g, :c0[0, b, g]])
    bad = sa.ROW_INVALID_PROB
    assert s0[0, :, 0].tolist() == [0, bad if hg[2] == 0 else 0, bad, 0, 0]
    assert s0[0, :, 1].tolist() == [0, bad if hg[2] == 1 else 0, 0, bad, 0]
    oi, oc, os_, od = oracle.select_topp([probs], np.zeros(1, np.int32), kv_len, 0.9, n_groups=2, head_group=hg)
    assert np.array_equal(os_, s0)
    assert np.array_equal(oc[os_ == 0], c0[os_ == 0])


@pytest.mark.parametrize("n", [1024, 4096, 40000])
@pytest.mark.parametrize("n_bin", [1, 37, 128, 129, 512, 513])
def test_threshold_bin_population_around_the_short_cut_capacity(n, n_bin):
    """The search takes a short cut when the level-1 threshold bin can hold at most 512 values
    (it gathers them instead of refining with two more histogram levels over the row; up to 128
    gathered values are searched directly, more through two histogram levels over the gathered
    values).  Rows whose threshold
    bin holds exactly n_bin distinct values just above 2^-10 (so the bin's mantissa sum >> 23
    equals n_bin), for populations on both sides of that capacity, in a shared-memory slice
    (n = 1024), a row read in place by one CTA and one read by a cluster."""
    rng = np.random.default_rng(n + n_bin)
    rows = np.full((3, n), 1e-9, np.float32)
    for r in range(3):
        pos = rng.permutation(n)
        rows[r, pos[:n_bin]] = (np.float32(2.0 ** -10) * (1 + np.arange(n_bin, dtype=np.float64) * 2.0 ** -23)).astype(np.float32)
        rows[r, pos[n_bin:n_bin + 4]] = 0.1
    bin_mass = n_bin * 2.0 ** -10
    total = 0.4 + bin_mass + (n - n_bin - 4) * 1e-9
    for frac in (0.01, 0.5, 0.999):       # threshold at the top, in the middle and at the bottom of the bin
        p = (0.4 + frac * bin_mass) / total
        st, gd, od = _run_rows(rows, n, float(p))
        assert st["n"] == 3


@pytest.mark.parametrize("n", wl.TOPP_SIZES)
@pytest.mark.parametrize("family", wl.TOPP_FAMILIES)
def test_config2_full_size_in_the_benchmarks_launch_shape(family, n, form):
    """Config 2 as the benchmark launches it: 256 rows per call (which decides how many CTAs a row
    gets), every row length and every p of the configuration.  The GPU selects all 256 rows; the
    oracle checks a sample of them row by row, and every row against the mass invariant
    M_> < target <= M_>=."""
    if form == "cluster":
        pytest.skip("single-row lists take the same path with and without a workspace")
    import paper_2510_27641_b200 as sa
    rows = wl.topp_rows(family, 256, n, seed=2)
    d = to_dev(rows.reshape(256, 1, 1, n))
    kv = np.full(256, n, np.int32)
    sample = np.random.default_rng(n).choice(256, size=12, replace=False)
    sub = rows[sample]
    for p in wl.TOPP_PS:
        gi, gc, gs, gd = sa.select_topp.func([d], to_dev(kv), [0], p, want_diag=True)
        torch.cuda.synchronize()
        gc_h, gs_h, gd_h = gc.cpu().numpy().ravel(), gs.cpu().numpy().ravel(), gd.cpu().numpy().reshape(256, 4)
        assert np.all(gs_h == 0)
        assert np.all(gd_h[:, 3] >= gd_h[:, 1]) and np.all(gd_h[:, 2] < gd_h[:, 1])   # M_>= >= target > M_>
        oi, oc, os_, od = oracle.select_topp([sub.reshape(12, 1, 1, n)], np.zeros(1, np.int32), kv[:12], p)
        gi_h = gi.cpu().numpy()[0, sample]
        st = compare_lists(lambda i: sub[i], p, gi_h[None], gc_h[sample].reshape(1, 12, 1),
                           gs_h[sample].reshape(1, 12, 1), oi, oc, os_, od)
        assert st["n"] == 12


FMAX = float(np.finfo(np.float32).max)


@pytest.mark.parametrize("variant", ["exact", "per_step", "chunk"])
def test_sum_overflow_voids_the_list_like_the_oracle(variant):
    """Finite inputs whose binary32 sum leaves the format: the list is invalid, as in the oracle;
    a sum that lands exactly on the largest finite value is valid.  Multi-row lists (both forms
    of the call through the fixture), and the same rule for chunk scores."""
    import paper_2510_27641_b200 as sa
    B, H, gamma, Ls = 4, 2, 2, 4096
    rng = np.random.default_rng(5)
    probs = (rng.random((B, H, gamma, Ls), dtype=np.float32) * 1e-3).astype(np.float32)
    probs[0, :, :, 100] = [[3e38, 0.0], [3e38, 0.0]]        # heads sum to +inf (also per query)
    probs[1, :, :, 200] = [[FMAX, 0.0], [0.0, 0.0]]         # exactly FLT_MAX: valid
    probs[2, :, :, 300] = [[3e38, 3e38], [0.0, 0.0]]        # overflows across queries only
    probs[3, :, :, 64:68] = 1e38 * 0.6                      # each position finite, a 4-chunk of them not
    kv = np.array([Ls, Ls, 3000, Ls], np.int32)
    kw = dict(per_step=variant == "per_step", chunk=4 if variant == "chunk" else 1)
    gi, gc, gs, _ = sa.select_topp([to_dev(probs)], to_dev(kv), [0], 0.9, **kw)
    torch.cuda.synchronize()
    if variant == "exact":
        oi, oc, os_, od = oracle.select_topp([probs], [0], kv, 0.9)
    else:
        oi, oc, os_, od = oracle.select_variant([probs], [0], kv, 0.9, **kw)
    assert gs.cpu().numpy().ravel().tolist() == os_.ravel().tolist()
    assert gc.cpu().numpy().ravel().tolist() == oc.ravel().tolist()
    bad, ok = sa.ROW_INVALID_PROB, 0
    expect = {"exact": [bad, ok, bad, ok], "per_step": [bad, ok, ok, ok], "chunk": [bad, ok, bad, bad]}[variant]
    assert os_.ravel().tolist() == expect
    for b in range(B):
        c = int(oc[0, b, 0])
        assert np.array_equal(gi.cpu().numpy()[0, b, 0, :c], oi[0, b, 0, :c])


def test_single_rows_at_the_edge_of_binary32():
    """R = 1 (a row read in place from 2048 positions on, and the shared-memory path below that):
    FLT_MAX is a valid value, +inf is not."""
    for n in (1024, 4096):
        rows = np.full((3, n), 1e-3, np.float32)
        rows[0, 17] = FMAX
        rows[1, 17] = np.inf
        rows[2, 17] = FMAX
        rows[2, 18] = FMAX          # the row total exceeds binary32 but not the binary64 masses
        st, gd, od = _run_rows(rows, n, 0.9)
        assert st["n"] == 3


def test_few_lists_wide_clusters_thresholds_above_two():
    """The two-launch form on very few lists (the search then runs eight CTAs per list) with
    aggregated values of 2.0 and more around the threshold -- level-1 bins in the upper half of
    the histogram -- for bins that take the short cut (few values per bin) and bins that do not."""
    import paper_2510_27641_b200 as sa
    B, H, gamma, Ls = 2, 16, 4, 32768
    rng = np.random.default_rng(9)
    kv = np.array([Ls, 30001], np.int32)
    flat = rng.random((B, H, gamma, Ls), dtype=np.float32)                       # sums ~ 32
    spread = np.exp(3.0 * rng.standard_normal((B, H, gamma, Ls))).astype(np.float32)  # sums spread over octaves
    for probs in (flat, spread):
        for p in (0.3, 0.9):
            gi, gc, gs, gd = sa.select_topp([to_dev(probs)], to_dev(kv), [0], p, want_diag=True)
            torch.cuda.synchronize()
            oi, oc, os_, od = oracle.select_topp([probs], [0], kv, p)
            theta = od[0, :, 0, 5]
            assert np.all(theta >= 2.0)
            st = compare_lists(lambda i: oracle.aggregate(probs[i], L=int(kv[i]))[0], p, gi.cpu().numpy(),
                               gc.cpu().numpy(), gs.cpu().numpy(), oi, oc, os_, od)
            assert st["n"] == B
