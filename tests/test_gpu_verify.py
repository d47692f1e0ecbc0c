"""GPU parity of specattn_sparse_verify (through the C ABI) against the CPU oracle's fp64
attention restricted to the listed rows (Eq. 1 over the index set of Eq. 2-3)."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from gpu_util import bf16_to_dev, check_attention, dev, to_dev
from workloads import bf16

pytestmark = pytest.mark.gpu

_ENGINE = {"flags": 0}


@pytest.fixture(params=["mma_sync", "tcgen05"], autouse=True)
def engine(request):
    """Every case runs once per implementation of the operation (forced through the flags)."""
    import paper_2510_27641_b200 as sa
    _ENGINE["flags"] = sa.VERIFY_ENGINE_MMA_SYNC if request.param == "mma_sync" else sa.VERIFY_ENGINE_TCGEN05
    yield request.param
    _ENGINE["flags"] = 0


def _make_case(seed, B, T, Hq, Hkv, page, lens, G=1, counts=None, shuffle=True, d=128, tail=0):
    rng = np.random.default_rng(seed)
    lens = np.asarray(lens, np.int32)
    pages_per_seq = max(1, (int(lens.max()) + tail + page - 1) // page)   # room for the in-flight tokens
    n_pages = B * pages_per_seq
    kv = wl.kv_pool(seed, 0, n_pages, page, Hkv, d)                      # torch bf16 on CPU
    bt = wl.block_table(seed, B, pages_per_seq, n_pages, shuffle=shuffle)
    q = wl.queries(seed, 0, B, T, Hq, d)
    stride = max(1, int(lens.max()))
    idx = np.zeros((B, G, stride), np.int32)
    cnt = np.zeros((B, G), np.int32)
    for b in range(B):
        for g in range(G):
            c = int(counts[b][g]) if counts is not None else int(rng.integers(0, lens[b] + 1))
            c = min(c, int(lens[b]))
            sel = np.sort(rng.choice(int(lens[b]), size=c, replace=False)) if c else np.zeros(0, np.int64)
            idx[b, g, :c] = sel
            cnt[b, g] = c
    return dict(q=q, kv=kv, bt=bt, lens=lens, idx=idx, cnt=cnt, page=page, Hkv=Hkv, G=G,
                pages_per_seq=pages_per_seq, tail=tail)


def _run(case, dense=False, use_bt=True, sm_scale=0.0, workspace=None):
    import paper_2510_27641_b200 as sa
    kv_d = case["kv"].to(dev())
    out, lse, status = sa.sparse_verify(
        bf16_to_dev(case["q"]), kv_d, to_dev(case["lens"]),
        block_table=to_dev(case["bt"]) if use_bt else None, pages_per_seq=case["pages_per_seq"],
        idx=None if dense else to_dev(case["idx"]), counts=None if dense else to_dev(case["cnt"]),
        n_groups=case["G"], dense=dense, sm_scale=sm_scale, workspace=workspace, tail_len=case.get("tail", 0),
        flags=_ENGINE["flags"])
    torch.cuda.synchronize()
    return out, lse, status


def _oracle(case, dense=False, use_bt=True, scale=0.0):
    kv_bits = bf16.torch_to_bits(case["kv"])
    page, Hkv = case["page"], case["Hkv"]
    return oracle.sparse_verify(case["q"], kv_bits, wl.kv_strides(page, Hkv, 128),
                                case["bt"] if use_bt else None, case["lens"], case["idx"], case["cnt"],
                                n_kv_heads=Hkv, page_size=page, n_groups=case["G"], dense=dense,
                                scale=scale, pages_per_seq=case["pages_per_seq"], tail_len=case.get("tail", 0))


@pytest.mark.parametrize("T,Hq,Hkv", [(5, 32, 8), (6, 32, 8), (5, 64, 8), (2, 8, 2), (8, 16, 2), (1, 4, 4)])
def test_query_block_shapes(T, Hq, Hkv):
    case = _make_case(10 + T, 3, T, Hq, Hkv, 16, [700, 130, 1], counts=[[300], [130], [1]])
    out, lse, status = _run(case)
    check_attention(out, lse, *_oracle(case))
    assert status.cpu().numpy().tolist() == [0, 0, 0]


def test_list_lengths_around_tile_edges_and_empty_lists():
    lens = [2000] * 14
    counts = [[c] for c in (0, 1, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129)]
    case = _make_case(20, 14, 5, 32, 8, 16, lens, counts=counts)
    out, lse, _ = _run(case)
    check_attention(out, lse, *_oracle(case))
    assert torch.all(out[0] == 0) and torch.all(torch.isneginf(lse[0]))


def test_long_lists_are_split_across_ctas_and_merged():
    # one sequence, 2 kv heads: every unit is cut among ~74 CTAs and merged by the last arriver
    case = _make_case(21, 1, 6, 8, 2, 16, [40000], counts=[[33333]])
    out, lse, _ = _run(case)
    check_attention(out, lse, *_oracle(case))
    # bitwise reproducible regardless of which CTA happens to arrive last
    out2, lse2, _ = _run(case)
    assert torch.equal(out, out2) and torch.equal(lse, lse2)


@pytest.mark.parametrize("T,Hq,counts", [
    (5, 64, [700, 1250, 2100]),      # 40 query rows (two warps per slab): units of 44 - 132 atoms, cut in 2 - 8 parts
    (6, 32, [1100, 1700, 2600]),     # 24 rows (CTA pairs): units above 64 atoms, cut in three or more parts
    (6, 32, [300, 640, 1000]),       # 24 rows: units of up to 64 atoms take the pair's path, cut in two
])
def test_units_cut_in_few_parts_merge_like_the_oracle(T, Hq, counts):
    """Short lists on few sequences: every unit is cut into a handful of parts (odd and even
    numbers of them), merged by the CTA that arrives last -- alone, with the slab's second warp,
    or through the pair's shared memory, depending on the shape.  Results are the oracle's and do
    not depend on who arrives last."""
    case = _make_case(31, 3, T, Hq, 8, 16, [9000, 9000, 9000], counts=[[c] for c in counts])
    out, lse, status = _run(case)
    assert int(status.abs().sum()) == 0
    check_attention(out, lse, *_oracle(case))
    for _ in range(3):
        out2, lse2, _ = _run(case)
        assert torch.equal(out, out2) and torch.equal(lse, lse2)


def test_ragged_batch_with_shared_workspace_reuse():
    import paper_2510_27641_b200 as sa
    rng = np.random.default_rng(3)
    lens = rng.integers(1, 6000, size=12).tolist()
    case = _make_case(22, 12, 5, 32, 8, 16, lens)
    out, lse, _ = _run(case)
    ref = _oracle(case)
    check_attention(out, lse, *ref)
    # the same workspace serves consecutive calls on a stream
    kv_d = case["kv"].to(dev())
    q_d, len_d, bt_d = bf16_to_dev(case["q"]), to_dev(case["lens"]), to_dev(case["bt"])
    idx_d, cnt_d = to_dev(case["idx"]), to_dev(case["cnt"])
    o = torch.empty_like(out)
    l = torch.empty_like(lse)
    args = sa.make_verify_args(q_d, kv_d, len_d, block_table=bt_d, idx=idx_d, counts=cnt_d, out=o, lse=l)
    ws = sa.verify_workspace(args)
    for _ in range(3):
        o.fill_(float("nan"))
        sa.sparse_verify(q_d, kv_d, len_d, block_table=bt_d, idx=idx_d, counts=cnt_d, out=o, lse=l, workspace=ws,
                         flags=_ENGINE["flags"])
        torch.cuda.synchronize()
        assert torch.equal(o, out) and torch.equal(l, lse)


def test_dense_flag_equals_full_list_and_contiguous_cache():
    lens = [1000, 37, 2048]
    case = _make_case(23, 3, 5, 32, 8, 16, lens, counts=[[1000], [37], [2048]], shuffle=False)
    o_d, l_d, _ = _run(case, dense=True)
    check_attention(o_d, l_d, *_oracle(case, dense=True))
    o_f, l_f, _ = _run(case)                      # the p = 1 list
    assert torch.equal(o_d, o_f) and torch.equal(l_d, l_f)
    o_c, l_c, _ = _run(case, use_bt=False)        # identity block table == contiguous addressing
    assert torch.equal(o_c, o_f) and torch.equal(l_c, l_f)
    check_attention(o_c, l_c, *_oracle(case, use_bt=False))


def test_per_kv_head_lists_page_sizes_and_scale():
    for page in (1, 8, 16, 48):
        case = _make_case(24 + page, 2, 5, 16, 4, page, [900, 333], G=4)
        out, lse, _ = _run(case, sm_scale=0.05)
        check_attention(out, lse, *_oracle(case, scale=0.05))


@pytest.mark.parametrize("T,tail", [(5, 5), (6, 6), (5, 2), (4, 7), (6, 1)])
def test_causal_tail_of_in_flight_tokens(T, tail):
    # list lengths chosen so that the tail starts at every offset of a 64-token tile, straddles
    # tiles, follows an empty list, and follows lists cut between CTAs
    lens = [300, 300, 300, 300, 300, 300, 3000, 5000]
    counts = [[0], [1], [31], [60], [63], [64], [2999], [4097]]
    case = _make_case(40 + T, 8, T, 32, 8, 16, lens, counts=counts, tail=tail)
    out, lse, status = _run(case)
    check_attention(out, lse, *_oracle(case))
    assert int(status.abs().sum()) == 0
    # dense context + tail = ordinary causal decode attention of the verified tokens
    case_d = _make_case(50 + T, 2, T, 16, 2, 16, [130, 64], counts=[[130], [64]], tail=tail)
    o_d, l_d, _ = _run(case_d, dense=True)
    check_attention(o_d, l_d, *_oracle(case_d, dense=True))
    o_f, l_f, _ = _run(case_d)
    assert torch.equal(o_d, o_f) and torch.equal(l_d, l_f)


def test_precision_when_few_tokens_dominate():
    # two nearly tied dominant keys with large opposite values: exposes bf16 rounding of P
    case = _make_case(30, 1, 5, 32, 8, 16, [64], counts=[[2]])
    kvb = bf16.torch_to_bits(case["kv"]).copy()
    vals = bf16.to_f32(kvb)
    pages = case["bt"][0]
    for k, pos in enumerate(case["idx"][0, 0, :2]):
        vals[pages[pos // 16], 1, pos % 16] = 4.0 if k == 0 else -4.0
        vals[pages[pos // 16], 0, pos % 16] *= 0.01
    case["kv"] = bf16.bits_to_torch(bf16.from_f32(vals)).reshape(case["kv"].shape)
    out, lse, _ = _run(case)
    check_attention(out, lse, *_oracle(case))


def test_bad_positions_and_pages_are_flagged_not_followed():
    import paper_2510_27641_b200 as sa
    case = _make_case(31, 3, 5, 32, 8, 16, [500, 500, 500], counts=[[100], [100], [100]])
    case["idx"][1, 0, 5] = 500          # == kv_len: out of range
    case["idx"][1, 0, 6] = -3
    case["bt"][2, 0:32] = 10 ** 6       # page id far outside the pool
    out, lse, status = _run(case)
    st = status.cpu().numpy()
    assert st[0] == 0 and st[1] == sa.ROW_BAD_INDEX and st[2] == sa.ROW_BAD_INDEX
    assert torch.all(torch.isfinite(out))
    ref_o, ref_l = _oracle(dict(case, idx=case["idx"][:1], cnt=case["cnt"][:1], lens=case["lens"][:1],
                                bt=case["bt"][:1], q=case["q"][:1]))
    check_attention(out[:1], lse[:1], ref_o, ref_l)


def test_argument_errors():
    import paper_2510_27641_b200 as sa
    case = _make_case(32, 1, 5, 32, 8, 16, [64], counts=[[10]])
    q_d, kv_d = bf16_to_dev(case["q"]), case["kv"].to(dev())
    len_d, bt_d = to_dev(case["lens"]), to_dev(case["bt"])
    idx_d, cnt_d = to_dev(case["idx"]), to_dev(case["cnt"])
    with pytest.raises(sa.SpecAttnError) as e:     # 9 queries x group 8 = 72 rows > 64
        q9 = torch.zeros((1, 9, 64, 128), dtype=torch.bfloat16, device=dev())
        sa.sparse_verify(q9, kv_d, len_d, block_table=bt_d, idx=idx_d, counts=cnt_d)
    assert e.value.code == -6
    tiny = torch.zeros(1024, dtype=torch.uint8, device=dev())
    with pytest.raises(sa.SpecAttnError) as e:
        sa.sparse_verify(q_d, kv_d, len_d, block_table=bt_d, idx=idx_d, counts=cnt_d, workspace=tiny)
    assert e.value.code == -5
    with pytest.raises(sa.SpecAttnError) as e:     # misaligned K/V base
        kv_off = kv_d.view(-1)[4:4 + 3 * 32768].view(3, 2, 16, 8, 128)
        sa.sparse_verify(q_d, kv_off, len_d, block_table=bt_d, idx=idx_d, counts=cnt_d)
    assert e.value.code == -4


def test_back_to_back_launches_with_many_segments_per_cta():
    # 256 units of ~125 atoms: every CTA walks several units, launches overlap through programmatic
    # stream serialization, and short last tiles make consecutive completion signals arrive within
    # nanoseconds of each other -- the case in which a completion barrier must not be missed
    import paper_2510_27641_b200 as sa
    case = _make_case(60, 32, 8, 64, 8, 16, [2100] * 32, counts=[[2000]] * 32)
    kv_d = case["kv"].to(dev())
    q_d, len_d, bt_d = bf16_to_dev(case["q"]), to_dev(case["lens"]), to_dev(case["bt"])
    idx_d, cnt_d = to_dev(case["idx"]), to_dev(case["cnt"])
    out, lse, status = _run(case)
    assert int(status.abs().sum()) == 0
    o, l = torch.empty_like(out), torch.empty_like(lse)
    st = torch.zeros_like(status)
    args = sa.make_verify_args(q_d, kv_d, len_d, block_table=bt_d, idx=idx_d, counts=cnt_d, out=o, lse=l)
    ws = sa.verify_workspace(args)
    for _ in range(100):
        sa.sparse_verify(q_d, kv_d, len_d, block_table=bt_d, idx=idx_d, counts=cnt_d, out=o, lse=l, status=st,
                         workspace=ws, flags=_ENGINE["flags"])
    torch.cuda.synchronize()
    assert int(st.abs().sum()) == 0
    assert torch.equal(o, out) and torch.equal(l, lse)


def test_precomputed_work_partition_gives_the_same_results_and_is_ignored_when_it_does_not_fit():
    import ctypes as C
    import paper_2510_27641_b200 as sa
    if _ENGINE["flags"] != sa.VERIFY_ENGINE_MMA_SYNC:
        pytest.skip("only the mma.sync engine reads plans")
    rng = np.random.default_rng(5)
    lens = rng.integers(1, 5000, size=10).tolist()
    case = _make_case(70, 10, 5, 32, 8, 16, lens)
    kv_d = case["kv"].to(dev())
    q_d, len_d, bt_d = bf16_to_dev(case["q"]), to_dev(case["lens"]), to_dev(case["bt"])
    idx_d, cnt_d = to_dev(case["idx"]), to_dev(case["cnt"])
    ref_o, ref_l, _ = _run(case)

    def run(plan, tail_len=0, cnt=cnt_d):
        o = torch.full_like(ref_o, float("nan"))
        l = torch.full_like(ref_l, float("nan"))
        a = sa.make_verify_args(q_d, kv_d, len_d, block_table=bt_d, idx=idx_d, counts=cnt, out=o, lse=l,
                                flags=_ENGINE["flags"], tail_len=tail_len)
        a.workspace_t = sa.verify_workspace(a)
        a.workspace, a.workspace_bytes = a.workspace_t.data_ptr(), a.workspace_t.numel()
        a.plan = None if plan is None else plan.data_ptr()
        rc = sa.lib().specattn_sparse_verify(C.byref(a), None)
        assert rc == 0
        torch.cuda.synchronize()
        return o, l, a

    o0, l0, a0 = run(None)
    plan = sa.verify_plan_buffer(a0)
    sa.verify_plan(a0, plan)
    torch.cuda.synchronize()
    hdr = plan[:8].cpu().tolist()
    assert hdr[1] == 10 * 8 and hdr[6] == 0 and hdr[7] == 0 and hdr[4] >= 1
    o1, l1, _ = run(plan)
    assert torch.equal(o0, o1) and torch.equal(l0, l1) and torch.equal(o0, ref_o)
    # a plan made for other lists of the same shape is the caller's mistake; one whose header
    # does not fit the launch (here: another tail_len) is ignored and the kernel partitions itself
    case_t = _make_case(70, 10, 5, 32, 8, 16, lens, tail=3)
    ref_t = _oracle(case_t)
    kv_t = case_t["kv"].to(dev())
    o = torch.empty_like(ref_o)
    l = torch.empty_like(ref_l)
    at = sa.make_verify_args(bf16_to_dev(case_t["q"]), kv_t, to_dev(case_t["lens"]), block_table=to_dev(case_t["bt"]),
                             idx=to_dev(case_t["idx"]), counts=to_dev(case_t["cnt"]), out=o, lse=l,
                             flags=_ENGINE["flags"], tail_len=3)
    ws = sa.verify_workspace(at)
    at.workspace, at.workspace_bytes = ws.data_ptr(), ws.numel()
    at.plan = plan.data_ptr()
    assert sa.lib().specattn_sparse_verify(C.byref(at), None) == 0
    torch.cuda.synchronize()
    check_attention(o, l, *ref_t)
    # several plans in one launch: the same bits as one launch each (here 11: two launches of <= 8)
    variants = []
    for k in range(11):
        cnt_k = torch.clamp(cnt_d - 3 * k, min=0)
        _, _, ak = run(None, cnt=cnt_k)
        variants.append((ak, cnt_k))
    singles = []
    for ak, _ in variants:
        pk = sa.verify_plan_buffer(ak)
        sa.verify_plan(ak, pk)
        singles.append(pk)
    many = [sa.verify_plan_buffer(ak) for ak, _ in variants]
    n0 = sa.kernel_launch_count()
    sa.verify_plan_many([ak for ak, _ in variants], many)
    torch.cuda.synchronize()
    assert sa.kernel_launch_count() - n0 == 2
    for pk, pm in zip(singles, many):
        assert torch.equal(pk, pm)
    # argument errors
    small = torch.zeros(4, dtype=torch.int32, device=dev())
    with pytest.raises(sa.SpecAttnError):
        sa.verify_plan_many([a0], [small])
    assert sa.lib().specattn_verify_plan(C.byref(a0), small.data_ptr(), 16, None) == -5
    assert sa.lib().specattn_verify_plan(C.byref(a0), None, 1 << 20, None) == -1


def test_kv_len_beyond_the_block_table_is_flagged_not_followed():
    """A device-side kv_len (dense call) or a listed position that lies beyond what the
    sequence's row of the block table covers must not index the table out of its row: those
    positions are flagged SPECATTN_ROW_BAD_INDEX and read position 0 instead; the other
    sequences are unaffected."""
    import paper_2510_27641_b200 as sa
    case = _make_case(33, 3, 5, 32, 8, 16, [480, 480, 480], counts=[[100], [100], [100]])
    assert case["pages_per_seq"] == 30
    # dense: sequence 1 claims one page more than its block-table row holds
    over = dict(case, lens=np.array([480, 496, 480], np.int32))
    for use_bt in (True, False):
        out, lse, status = _run(over, dense=True, use_bt=use_bt)
        st = status.cpu().numpy()
        assert st[0] == 0 and st[1] == sa.ROW_BAD_INDEX and st[2] == 0
        assert torch.all(torch.isfinite(out))
        ref_o, ref_l = _oracle(case, dense=True, use_bt=use_bt)
        check_attention(out[[0, 2]], lse[[0, 2]], ref_o[[0, 2]], ref_l[[0, 2]])
    # listed: the same claim lets position 485 through the kv_len check, not through the table's
    over["idx"] = case["idx"].copy()
    over["idx"][1, 0, 99] = 485
    out, lse, status = _run(over)
    st = status.cpu().numpy()
    assert st[0] == 0 and st[1] == sa.ROW_BAD_INDEX and st[2] == 0
    ref_o, ref_l = _oracle(case)
    check_attention(out[[0, 2]], lse[[0, 2]], ref_o[[0, 2]], ref_l[[0, 2]])


def test_a_bounded_wait_that_runs_out_is_reported_and_the_next_call_is_correct():
    """Failure path of the device-side waits, without faulting anything: with the test-only flag
    one producer warp of CTA 0 withholds the completion signal of its first tile; the waits on it
    give up at their poll limit, the kernel returns normally with SPECATTN_ROW_TIMEOUT in
    status[0], and -- after the workspace is re-initialised -- the next ordinary call on the same
    buffers is correct."""
    import ctypes as C
    import time
    import paper_2510_27641_b200 as sa
    case = _make_case(34, 2, 5, 32, 8, 16, [3000, 2000], counts=[[2500], [1500]])
    kv_d = case["kv"].to(dev())
    q_d, len_d, bt_d = bf16_to_dev(case["q"]), to_dev(case["lens"]), to_dev(case["bt"])
    idx_d, cnt_d = to_dev(case["idx"]), to_dev(case["cnt"])
    o = torch.zeros((2, 5, 32, 128), dtype=torch.float32, device=dev())
    l = torch.zeros((2, 5, 32), dtype=torch.float32, device=dev())
    st = torch.zeros(2, dtype=torch.int32, device=dev())
    a = sa.make_verify_args(q_d, kv_d, len_d, block_table=bt_d, idx=idx_d, counts=cnt_d, out=o, lse=l, status=st,
                            flags=_ENGINE["flags"] | sa.VERIFY_TEST_LOSE_ARRIVAL)
    ws = sa.verify_workspace(a)
    a.workspace, a.workspace_bytes = ws.data_ptr(), ws.numel()
    torch.cuda.synchronize()
    t0 = time.time()
    assert sa.lib().specattn_sparse_verify(C.byref(a), None) == 0
    torch.cuda.synchronize()           # returns: the kernel gave up instead of spinning for ever
    elapsed = time.time() - t0
    assert int(st[0]) & sa.ROW_TIMEOUT
    assert elapsed < 30.0
    # recovery: fresh counters, same buffers, no test flag
    assert sa.lib().specattn_verify_workspace_init(ws.data_ptr(), ws.numel(), None) == 0
    st.zero_()
    a.flags = _ENGINE["flags"]
    assert sa.lib().specattn_sparse_verify(C.byref(a), None) == 0
    torch.cuda.synchronize()
    assert int(st.abs().sum()) == 0
    check_attention(o, l, *_oracle(case))


def _chunk_lists(case, rng, chunk=16, frac=0.4):
    """Replaces the case's lists by lists of whole aligned chunks (the form specattn_select_topp
    emits with chunk = 16, 32 or 64): a random subset of each sequence's chunks, always including
    the last one (cut at kv_len) for half of the lists."""
    B, G = case["cnt"].shape
    for b in range(B):
        L = int(case["lens"][b])
        n_chunks = (L + chunk - 1) // chunk
        for g in range(G):
            take = rng.random(n_chunks) < frac
            if n_chunks and (b + g) % 2 == 0:
                take[-1] = True
            pos = np.concatenate([np.arange(j * chunk, min(L, (j + 1) * chunk)) for j in np.flatnonzero(take)]
                                 or [np.zeros(0, np.int64)])
            case["idx"][b, g, :len(pos)] = pos
            case["idx"][b, g, len(pos):] = 0
            case["cnt"][b, g] = len(pos)


@pytest.mark.parametrize("page,chunk", [(16, 16), (32, 16), (16, 64), (64, 32)])
def test_page_granular_lists_and_dense_calls(page, chunk):
    """Lists of whole aligned chunks flagged SPECATTN_VERIFY_PAGE_LISTS, and dense calls, read K/V
    page-wise (tiled bulk tensor copies in the tcgen05 engine): page sizes 16 to 64, partial last
    pages and chunks, shuffled block table, per-kv-head lists, lists cut between CTAs.  The slots
    of a last page beyond kv_len are poisoned with NaN: they must not reach the result."""
    import paper_2510_27641_b200 as sa
    rng = np.random.default_rng(page * 100 + chunk)
    lens = [5000, 777, 16, 1, 4096, 3333]
    case = _make_case(80 + page, 6, 5, 32, 8, page, lens, G=1)
    _chunk_lists(case, rng, chunk)
    kv = case["kv"].clone()
    for b, L in enumerate(lens):                       # poison what lies beyond kv_len in the last page
        if L % page:
            pg = int(case["bt"][b, L // page])
            kv[pg, :, L % page:] = float("nan")
    poisoned = dict(case, kv=kv)
    flags0 = _ENGINE["flags"]
    try:
        _ENGINE["flags"] = flags0 | sa.VERIFY_PAGE_LISTS
        out, lse, status = _run(poisoned)
        assert int(status.abs().sum()) == 0
        check_attention(out, lse, *_oracle(case))
        o_d, l_d, status = _run(poisoned, dense=True)
        assert int(status.abs().sum()) == 0
        check_attention(o_d, l_d, *_oracle(case, dense=True))
        # the flag changes how rows are fetched, not the results
        _ENGINE["flags"] = flags0
        out0, lse0, _ = _run(case)
        assert float((out - out0).abs().max()) <= 2e-5
        assert float(torch.nan_to_num(lse - lse0, nan=0.0).abs().max()) <= 2e-5    # (-inf) - (-inf): empty lists
    finally:
        _ENGINE["flags"] = flags0


def test_page_granular_per_head_lists_tails_and_contiguous_cache():
    import paper_2510_27641_b200 as sa
    rng = np.random.default_rng(7)
    flags0 = _ENGINE["flags"]
    try:
        _ENGINE["flags"] = flags0 | sa.VERIFY_PAGE_LISTS
        # per-kv-head lists; in-flight tokens behind the lists (they start in the middle of a page)
        case = _make_case(90, 3, 5, 16, 4, 16, [2000, 1000, 37], G=4, tail=5)
        _chunk_lists(case, rng, 16)
        out, lse, status = _run(case)
        assert int(status.abs().sum()) == 0
        check_attention(out, lse, *_oracle(case))
        # dense + tail: ordinary causal decode attention of the verified tokens, page-wise
        o_d, l_d, _ = _run(case, dense=True)
        check_attention(o_d, l_d, *_oracle(case, dense=True))
        # contiguous cache (no block table), one long sequence cut among all CTAs
        case = _make_case(91, 1, 6, 8, 2, 32, [40000], shuffle=False)
        _chunk_lists(case, rng, 32, frac=0.8)
        out, lse, _ = _run(case, use_bt=False)
        check_attention(out, lse, *_oracle(case, use_bt=False))
        o_d, l_d, _ = _run(case, dense=True, use_bt=False)
        check_attention(o_d, l_d, *_oracle(case, dense=True, use_bt=False))
        # a list that breaks the promise is flagged, and nothing faults
        case = _make_case(92, 2, 5, 32, 8, 16, [3000, 3000])
        _chunk_lists(case, rng, 16)
        case["idx"][1, 0, 16 * 3] += 5
        out, lse, status = _run(case)
        st = status.cpu().numpy()
        assert st[0] == 0 and torch.all(torch.isfinite(out))
        if flags0 == sa.VERIFY_ENGINE_TCGEN05:
            assert st[1] == sa.ROW_BAD_INDEX
    finally:
        _ENGINE["flags"] = flags0
