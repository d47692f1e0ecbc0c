"""The seeded input generators: determinism, shapes and value laws."""
import numpy as np
import torch

import workloads as wl


def test_draft_probs_rows_are_softmax_rows():
    kv_len = np.array([100, 37, 0], np.int32)
    a = wl.draft_probs(0, 2, kv_len, 3, 2, 128)
    b = wl.draft_probs(0, 2, kv_len, 3, 2, 128)
    assert a.dtype == np.float32 and a.shape == (3, 3, 2, 128) and np.array_equal(a, b)
    assert np.allclose(a[0].sum(-1), 1, atol=1e-5) and np.allclose(a[1].sum(-1), 1, atol=1e-5)
    assert np.all(a[1, :, :, 37:] == 0) and np.all(a[2] == 0) and np.all(a >= 0)
    assert not np.array_equal(a, wl.draft_probs(1, 2, kv_len, 3, 2, 128))
    # sink positions carry visibly more mass than their neighbours
    assert a[0, :, :, :4].mean() > 20 * a[0, :, :, 4:20].mean()


def test_topp_row_families():
    for fam in wl.TOPP_FAMILIES:
        a = wl.topp_rows(fam, 4, 1024, 0)
        assert a.shape == (4, 1024) and a.dtype == np.float32
        assert np.allclose(a.sum(1), 1, atol=1e-5) and np.all(a > 0)
        assert np.array_equal(a, wl.topp_rows(fam, 4, 1024, 0))
    assert len(np.unique(wl.topp_rows("quantised", 1, 8192, 0))) <= 64


def test_kv_values_are_reproducible_and_standard_normal():
    pool = wl.kv_pool(3, 1, 8, 16, 2, 128, chunk_elems=5000)
    again = wl.kv_pool(3, 1, 8, 16, 2, 128)
    assert pool.dtype == torch.bfloat16 and tuple(pool.shape) == (8, 2, 16, 2, 128)
    assert torch.equal(pool.view(torch.int16), again.view(torch.int16))
    x = pool.float()
    assert abs(x.mean().item()) < 0.02 and abs(x.std().item() - 1) < 0.02
    sp, sk, ss, sh = wl.kv_strides(16, 2, 128)
    flat = 5 * sp + 1 * sk + 7 * ss + 1 * sh + torch.arange(128)
    row = wl.kv_values(3, 1, flat)
    assert torch.equal(row.view(torch.int16), pool[5, 1, 7, 1].view(torch.int16))
    assert not torch.equal(wl.kv_values(3, 2, flat), row)


def test_block_table_layer_map_and_lengths():
    bt = wl.block_table(1, 4, 10)
    assert bt.shape == (4, 10) and sorted(bt.ravel().tolist()) == list(range(40))
    assert not np.array_equal(bt.ravel(), np.arange(40))
    m = wl.layer_map(1, 32, 4, n_dense_first=2)
    assert np.all(m[:2] == -1) and np.all(np.diff(m[2:]) >= 0) and m.max() < 4
    L, sink, slope = wl.ragged_lengths(3, 32, 2048, 65536)
    assert L.min() >= 2048 and L.max() <= 65536 and len(set(L.tolist())) > 20


def test_step_inputs_of_a_shrunken_config():
    cfg = wl.config1().scaled(n_target_layers=3, n_draft_layers=2, batch=2, ctx=200)
    si = wl.make_step_inputs(cfg)
    assert si.L_stride == 200 and si.pages_per_seq == 13 and si.block_table.shape == (2, 13)
    assert len(si.q) == 3 and si.q[0].shape == (2, 6, 32, 128) and si.q[0].dtype == np.uint16
    used = set(si.layer_map.tolist())
    for u in range(2):
        assert (si.draft_probs[u] is not None) == (u in used)
