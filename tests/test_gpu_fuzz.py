"""Seeded random sweeps over shapes, lengths, value families and call options, each case compared
with the CPU oracle under the same gates as the targeted tests.  (Longer runs of the same generators
-- tens of thousands of selection cases, hundreds of attention cases -- found the bugs that the
targeted tests now pin; these short runs keep the generators alive.)"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from gpu_util import check_attention, compare_lists, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [0, 1])
def test_random_selection_cases(seed):
    import paper_2510_27641_b200 as sa
    rng = np.random.default_rng(seed)
    n_lists = 0
    for _ in range(150):
        B = int(rng.integers(1, 7))
        H = int(rng.choice([1, 1, 2, 3, 6]))
        gamma = int(rng.choice([1, 1, 2, 4]))
        Ls = int(rng.choice([260, 1024, 2048, 2052, 4096, 9000, 20000, 40000])) // 4 * 4
        if H * gamma * Ls * B > 8_000_000:
            continue
        kv_len = rng.integers(0, Ls + 1, size=B).astype(np.int32)
        if rng.random() < 0.5:
            kv_len[rng.integers(0, B)] = Ls
        fam = rng.choice(["draft", "uniform", "quantised", "zipf", "bin"])
        if fam == "draft":
            probs = wl.draft_probs(int(rng.integers(1 << 30)), 0, np.maximum(kv_len, 1), H, gamma, Ls,
                                   sink=float(rng.uniform(2, 12)), slope=float(rng.uniform(0, 16)) / Ls)
            for b in range(B):
                probs[b, :, :, kv_len[b]:] = 0
        elif fam == "bin":   # many values inside one level-1 bin, around the capacities of the short cut
            probs = np.full((B, H, gamma, Ls), 1e-9, np.float32)
            for b in range(B):
                nb = min(int(rng.choice([1, 5, 100, 127, 128, 129, 300, 511, 512, 513, 700])), Ls - 8)
                pos = rng.permutation(Ls)
                vals = (np.float32(2.0 ** -10) * (1 + rng.integers(0, 1 << 19, size=nb) * 2.0 ** -23)).astype(np.float32)
                probs[b, :, :, pos[:nb]] = vals[:, None, None] / (H * gamma)
                probs[b, :, :, pos[nb:nb + 4]] = 0.1 / (H * gamma)
        else:
            probs = np.stack([wl.topp_rows(fam, H * gamma, Ls, int(rng.integers(1 << 30))).reshape(H, gamma, Ls)
                              for _ in range(B)])
            for b in range(B):
                probs[b, :, :, kv_len[b]:] = 7.0      # beyond kv_len: not an input
        probs = np.ascontiguousarray(probs, np.float32)
        p = float(rng.choice([0.3, 0.5, 0.9, 0.95, 0.99, 1.0, rng.uniform(0.01, 0.999)]))
        G, hg = 1, None
        if H >= 2 and rng.random() < 0.3:
            G, hg = 2, (np.arange(H) * 2 // H).astype(np.int32)
        gi, gc, gs, _ = sa.select_topp([to_dev(probs)], to_dev(kv_len), [0], p, n_groups=G,
                                       head_group=None if hg is None else hg.tolist(),
                                       workspace=bool(rng.random() < 0.5))
        torch.cuda.synchronize()
        oi, oc, os_, od = oracle.select_topp([probs], np.zeros(1, np.int32), kv_len, p, n_groups=G, head_group=hg)

        def row(i):
            return oracle.aggregate(probs[i // G], L=int(kv_len[i // G]), head_group=hg, g=i % G)[0]

        st = compare_lists(row, p, gi.cpu().numpy(), gc.cpu().numpy(), gs.cpu().numpy(), oi, oc, os_, od)
        n_lists += st["n"]
    assert n_lists > 200


@pytest.mark.parametrize("seed", [0])
def test_random_attention_cases(seed):
    import paper_2510_27641_b200 as sa
    import test_gpu_verify as tv
    rng = np.random.default_rng(seed)
    shapes = [(5, 32, 8), (6, 32, 8), (5, 64, 8), (2, 8, 2), (8, 16, 2), (1, 4, 4), (6, 8, 1), (4, 16, 8)]
    try:
        for _ in range(14):
            eng = rng.choice(["mma_sync", "tcgen05"], p=[0.7, 0.3])
            tv._ENGINE["flags"] = sa.VERIFY_ENGINE_MMA_SYNC if eng == "mma_sync" else sa.VERIFY_ENGINE_TCGEN05
            T, Hq, Hkv = shapes[rng.integers(0, len(shapes))]
            B = int(rng.integers(1, 10))
            page = int(rng.choice([16, 16, 32, 24, 1]))
            lens = rng.integers(1, int(rng.choice([40, 300, 1500, 5000])) + 1, size=B).tolist()
            G = 1 if rng.random() < 0.7 else Hkv
            tail = int(rng.choice([0, 0, 0, 1, T]))
            counts = None
            if rng.random() < 0.5:
                counts = [[min(int(rng.choice([0, 1, 15, 16, 17, 63, 64, 65, lens[b] // 2, lens[b]])), lens[b])
                           for _ in range(G)] for b in range(B)]
            dense = bool(rng.random() < 0.15) and tail == 0
            use_bt = bool(rng.random() < 0.85)
            case = tv._make_case(int(rng.integers(1 << 30)), B, T, Hq, Hkv, page, lens, G=G, counts=counts,
                                 shuffle=use_bt and bool(rng.random() < 0.8), tail=tail)
            out, lse, status = tv._run(case, dense=dense, use_bt=use_bt)
            check_attention(out, lse, *tv._oracle(case, dense=dense, use_bt=use_bt)[:2])
            assert int(status.abs().sum()) == 0
    finally:
        tv._ENGINE["flags"] = 0
