#!/usr/bin/env python
"""Benchmark of the SpecAttn verification hot path on B200.

A step = one pass of the whole hot path over one synthetic batch: one specattn_select_topp over
the mapped draft layers, one launch for the work partitions (plans) of the list sets, and one
specattn_sparse_verify per target layer (34 launches on the default workload).  Default workload: the Llama-3-8B-shaped configuration -- 32 target
layers, 4-layer 12-head draft, batch 8, context 32768, paged bf16 KV (page 16, shuffled block
table), gamma = 5, p = 0.95.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--no-topp-sweep] [--no-long-context] [--no-cpu-baseline]

Prints ONE JSON line (rank 0).  `value` is microseconds per step with all inputs resident in
HBM (CUDA-graph replay of the step, CUDA events, max over ranks); `e2e` is the same step issued
through specattn_verify_step_host from pinned host buffers (draft probabilities and queries go
host->device, outputs and LSE come back, inside the timed region); `roofline` describes the
dominant kernel (sparse verify) against the measured HBM copy bandwidth; `cpu_baseline` is the
CPU oracle timed on a bounded sample of the same workload and scaled to a step.  `extra` adds
context measured in the same run: the selection variants of Alg. 2, the attention of all layers
in one launch (an upper bound, labelled so), the selection micro-benchmark of config 2
(256 rows x {1k, 8k, 64k, 128k} x 3 p x 3 families, rows/s) and config 4 (ctx 131072, 64 q / 8 kv
heads: p in {0.8, 0.9, 0.95} against the same kernel at p = 1).
With N > 1 every rank runs its own batch of 8 sequences (batch sharding, no collective).
`--impl reference` times the CPU oracle alone (rank 0) and prints the same line.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "sparse_verify_step_time"
UNIT = "us/step"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum per sparse_verify launch on this workload, from
# the ncu capture summarised in profiles/sparse_verify_cfg1.md.
NCU_VERIFY_TRAFFIC_BYTES = 40.9e6


# ----------------------------------------------------------------------------------------------
def _rank_env():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def _measured_peaks():
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        try:
            d = json.loads(f.read_text())
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def rank_config(cfg, rank: int, world: int):
    """The workload of one rank: with N > 1 every rank owns a batch of its own (sharding by
    sequence, no collective on the data path) -- same shapes, rank-specific seed."""
    return cfg.scaled(seed=cfg.seed + 1000 * rank) if world > 1 else cfg


def reduce_max(values, world: int, device="cuda"):
    """Element-wise MAX over ranks of a list of timings (identity for one rank)."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x2: "applications_clocks_setting"}

    def __init__(self, index: int, uuid: str | None = None, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------------------------
def build_step(cfg, dev, verify_flags=0, select_workspace=True, select_form=0):
    import torch
    import workloads as wl
    from paper_2510_27641_b200.step import VerifyStep
    from workloads import bf16
    si = wl.make_step_inputs(cfg)
    # one allocation for all layers' pools (each layer's pool is a slice of it), so that the
    # layer-batched upper bound below can address every layer through one block table
    per_layer = si.n_pages * 2 * cfg.page_size * cfg.n_kv_heads * cfg.head_dim
    big = torch.empty(cfg.n_target_layers * per_layer, dtype=torch.bfloat16, device=dev)
    pools = [wl.kv_pool(cfg.seed, j, si.n_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim, device=dev,
                        out=big[j * per_layer:(j + 1) * per_layer]) for j in range(cfg.n_target_layers)]
    step = VerifyStep(layer_map=si.layer_map.tolist(), n_draft_layers=cfg.n_draft_layers, batch=cfg.batch,
                      n_draft_heads=cfg.n_draft_heads, gamma=cfg.gamma, L_stride=si.L_stride,
                      n_q_heads=cfg.n_q_heads, p=cfg.p, kv_pools=pools,
                      kv_len=torch.from_numpy(si.kv_len).to(dev),
                      block_table=None if si.block_table is None else torch.from_numpy(si.block_table).to(dev),
                      pages_per_seq=si.pages_per_seq, verify_flags=verify_flags, select_workspace=select_workspace,
                      select_form=select_form)
    dp_host = [None if x is None else torch.from_numpy(x).pin_memory() for x in si.draft_probs]
    q_host = [bf16.bits_to_torch(q).pin_memory() for q in si.q]
    step.load_inputs(dp_host, q_host)
    step.kv_big = big.view(cfg.n_target_layers * si.n_pages, 2, cfg.page_size, cfg.n_kv_heads, cfg.head_dim)
    torch.cuda.synchronize()
    return si, pools, step, dp_host, q_host


def capture(fn):
    import torch
    import paper_2510_27641_b200 as sa
    g = torch.cuda.CUDAGraph()
    n0 = sa.kernel_launch_count()
    with torch.cuda.graph(g):
        fn()
    return g, sa.kernel_launch_count() - n0


def time_replays(g, steps, warmup, barrier=None, stats=None):
    """Microseconds per replay, CUDA events on the replaying (current) stream.  The `steps`
    replays run back to back inside one bracket (barrier + synchronize on both sides); events
    recorded between them, without any synchronisation, cut the bracket into up to ten batches
    whose per-replay times give a median and a minimum (returned through `stats`)."""
    import torch
    for _ in range(warmup):
        g.replay()
    torch.cuda.synchronize()
    if barrier is not None:
        barrier()
    nb = max(1, min(10, steps))
    edges = [round(k * steps / nb) for k in range(nb + 1)]
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(nb + 1)]
    ev[0].record()
    for k in range(nb):
        for _ in range(edges[k + 1] - edges[k]):
            g.replay()
        ev[k + 1].record()
    torch.cuda.synchronize()
    if barrier is not None:
        barrier()
    if stats is not None:
        per = [ev[k].elapsed_time(ev[k + 1]) * 1e3 / (edges[k + 1] - edges[k]) for k in range(nb)]
        stats.update(batches=nb, median=round(float(np.median(per)), 3), min=round(float(np.min(per)), 3),
                     max=round(float(np.max(per)), 3))
    return ev[0].elapsed_time(ev[nb]) * 1e3 / steps


def verify_bytes(cfg, si, counts_layer):
    """Algorithmic bytes of ONE sparse_verify launch: selected K and V rows, their indices, the
    block-table entries of the touched pages, the queries and the outputs."""
    c = counts_layer.astype(np.int64)          # [B, G]
    kv = int(c.sum()) * cfg.n_kv_heads * cfg.head_dim * 2 * 2 if c.shape[1] == 1 \
        else int(c.sum()) * cfg.head_dim * 2 * 2
    idx_b = 4 * int(c.sum())
    bt_b = 4 * int(np.minimum(c, (si.kv_len[:, None] + cfg.page_size - 1) // cfg.page_size).sum())
    q_b = 2 * cfg.batch * cfg.n_q * cfg.n_q_heads * cfg.head_dim
    o_b = 4 * cfg.batch * cfg.n_q * cfg.n_q_heads * (cfg.head_dim + 1)
    return kv + idx_b + bt_b + q_b + o_b, kv


def select_bytes(cfg, si, n_used, counts):
    R = cfg.n_draft_heads * cfg.gamma
    read = 4 * R * int(si.kv_len.astype(np.int64).sum()) * n_used
    return read + 4 * int(counts[counts >= 0].sum())


# ----------------------------------------------------------------------------------------------
class OracleSample:
    """The CPU oracle on a bounded sample of the workload, scaled to one step: selection
    (O1 + O2) for every list of the step, attention (O3) for `n_attn_layers` target layers (all
    sequences and heads), scaled by n_target_layers / n_attn_layers.  The K/V rows the oracle
    reads come from the device pools when those exist (one device->host copy per sampled
    layer, untimed); otherwise only the listed rows are regenerated on the CPU from the hashed
    pool definition into a compact pool of the touched pages."""

    def __init__(self, cfg, si, n_attn_layers, pools=None):
        import torch
        import oracle
        import workloads as wl
        from workloads import bf16
        self.cfg, self.si, self.oracle = cfg, si, oracle
        self.strides = wl.kv_strides(cfg.page_size, cfg.n_kv_heads, cfg.head_dim)
        sp, sk, ss, sh = self.strides
        oi, oc, _, _ = oracle.select_topp(si.draft_probs, si.layer_map, si.kv_len, cfg.p)
        # evenly spread, first and last target layer included
        n_take = max(1, min(n_attn_layers, cfg.n_target_layers))
        self.layers = sorted({int(round(x)) for x in np.linspace(0, cfg.n_target_layers - 1, n_take)})
        self.prepared = []
        for j in self.layers:
            u = int(si.layer_map[j])
            if pools is not None:
                self.prepared.append((bf16.torch_to_bits(pools[j].cpu()), si.block_table))
                continue
            bt_small = np.zeros_like(si.block_table)
            n_small, flats, dsts = 0, [], []
            for b in range(cfg.batch):
                pos = oi[u, b, 0, :int(oc[u, b, 0])].astype(np.int64)
                lps = np.unique(pos // cfg.page_size)
                bt_small[b, lps] = n_small + np.arange(len(lps))
                src_page = si.block_table[b, pos // cfg.page_size].astype(np.int64)
                dst_page = bt_small[b, pos // cfg.page_size].astype(np.int64)
                n_small += len(lps)
                row = np.arange(cfg.n_kv_heads * cfg.head_dim, dtype=np.int64)     # all heads of a slot
                for kvsel in (0, 1):
                    flats.append((src_page * sp + kvsel * sk + (pos % cfg.page_size) * ss)[:, None] + row[None, :])
                    dsts.append((dst_page * sp + kvsel * sk + (pos % cfg.page_size) * ss)[:, None] + row[None, :])
            flat = torch.from_numpy(np.concatenate([f.reshape(-1) for f in flats]))
            dst = np.concatenate([d.reshape(-1) for d in dsts])
            kv_small = np.zeros(n_small * sp, dtype=np.uint16)
            kv_small[dst] = bf16.torch_to_bits(wl.kv_values(cfg.seed, j, flat))
            self.prepared.append((kv_small, bt_small))
        self.oi, self.oc = oi, oc
        self.cores = oracle.num_threads()

    def step_us(self):
        cfg, si, oracle = self.cfg, self.si, self.oracle
        t0 = time.perf_counter()
        oi, oc, _, _ = oracle.select_topp(si.draft_probs, si.layer_map, si.kv_len, cfg.p)
        t_sel = time.perf_counter() - t0
        t0 = time.perf_counter()
        for j, (kv_bits, bt) in zip(self.layers, self.prepared):
            u = int(si.layer_map[j])
            oracle.sparse_verify(si.q[j], kv_bits, self.strides, bt, si.kv_len, oi[u], oc[u],
                                 n_kv_heads=cfg.n_kv_heads, page_size=cfg.page_size)
        t_attn = time.perf_counter() - t0
        scale = cfg.n_target_layers / len(self.layers)
        sample = (f"select: all {int((oc >= 0).sum())} lists of the step ({t_sel:.3f} s); attention: "
                  f"{len(self.layers)} of {cfg.n_target_layers} target layers (evenly spread, first and last "
                  f"included), all sequences and heads "
                  f"({t_attn:.3f} s), scaled x{scale:g}")
        return (t_sel + t_attn * scale) * 1e6, sample


def config_dict(cfg, world: int):
    """The `config` object of the JSON line: the same for both arms (--impl ours / reference)."""
    return {"workload": cfg.name, "n_target_layers": cfg.n_target_layers,
            "n_draft_layers": cfg.n_draft_layers, "batch_per_gpu": cfg.batch,
            "global_batch": cfg.batch * world, "ctx": cfg.ctx, "page_size": cfg.page_size,
            "gamma": cfg.gamma, "p": cfg.p, "q_heads": cfg.n_q_heads, "kv_heads": cfg.n_kv_heads,
            "head_dim": cfg.head_dim, "parallelism": f"batch-sharded x{world}, no collective",
            "l2": "inputs exceed L2: 252 MB of draft rows and 1.3 GB of gathered K/V per step"}


def run_reference(args, cfg):
    import workloads as wl
    rank, _, world = _rank_env()
    if rank != 0:
        return
    si = wl.make_step_inputs(cfg)
    smp = OracleSample(cfg, si, n_attn_layers=2)
    vals, sample = [], ""
    t_start = time.perf_counter()
    for k in range(args.warmup + args.steps):
        us, sample = smp.step_us()
        if k >= args.warmup:
            vals.append(us)
    v = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": round(v, 1), "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(v / 1e3, 3), "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(cfg, max(1, args.gpus)),
            "cpu_baseline": {"value": round(v, 1), "unit": UNIT, "cores": smp.cores, "kind": "oracle",
                             "sample": sample + f"; wall {time.perf_counter() - t_start:.1f} s for all steps"},
            "e2e": {"value": round(v, 1), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
def topp_sweep(dev, reps=5, families=None, sizes=None, ps=None, n_rows=256):
    """Selection micro-benchmark: 256 rows x n x p x family, rows/s per cell (R = 1).
    Each cell is timed as a CUDA graph of launches over rotating copies of the rows (at least
    256 MB in total, so every launch reads cold data), replayed `reps` times.  Bytes are the
    algorithmic ones: every row read once plus the index list written."""
    import ctypes as C
    import torch
    import paper_2510_27641_b200 as sa
    import workloads as wl
    out = {}
    R = n_rows
    for fam in (families or wl.TOPP_FAMILIES):
        for n in (sizes or wl.TOPP_SIZES):
            base = torch.from_numpy(wl.topp_rows(fam, R, n, seed=2)).to(dev).view(R, 1, 1, n)
            copies = max(2, min(64, (256 << 20) // (R * n * 4)))
            rows = [base.clone() for _ in range(copies)]
            kv = torch.full((R,), n, dtype=torch.int32, device=dev)
            idx = torch.empty((1, R, 1, n), dtype=torch.int32, device=dev)
            cnt = torch.empty((1, R, 1), dtype=torch.int32, device=dev)
            st = torch.empty((1, R, 1), dtype=torch.int32, device=dev)
            for p in (ps or wl.TOPP_PS):
                args = [sa.make_select_args([r], kv, [0], p, idx=idx, counts=cnt, row_status=st) for r in rows]

                def launch_all():
                    sp = sa._stream_ptr(None)
                    for a, _keep in args:
                        rc = sa.lib().specattn_select_topp(C.byref(a), sp)
                        assert rc == 0, rc
                launch_all()
                torch.cuda.synchronize()
                g, _ = capture(launch_all)
                us = time_replays(g, reps, 2) / copies
                assert int(st.abs().sum()) == 0, f"row_status not clean in cell {fam}/n={n}/p={p}"
                kept = float(cnt.float().mean().item())
                byts = R * (n * 4 + kept * 4)
                out[f"{fam}/n={n}/p={p}"] = {"us": round(us, 2), "rows_per_s": round(R / us * 1e6),
                                             "gbs": round(byts / us / 1e3, 1),
                                             "frac_of_measured": round(byts / us / 1e3 / _measured_peaks()[0], 3),
                                             "kept_mean": kept}
                del g
            del rows, idx, base
    return out


def overlapped_schedule(step, reps=20):
    """The step with one selection per used draft layer, all but the first on a second stream
    under the attention of earlier layers (VerifyStep(overlap_select=True)), on the step's own
    buffers: microseconds per step beside the default schedule's, and the outputs compared."""
    import torch
    from paper_2510_27641_b200.step import VerifyStep
    ref_out = [o.clone() for o in step.out]
    a0 = step.verify_args[0]
    ov = VerifyStep(layer_map=step.layer_map, n_draft_layers=len(step.draft_probs), batch=a0.batch,
                    n_draft_heads=step.select_args.n_draft_heads, gamma=step.select_args.gamma,
                    L_stride=step.select_args.L_stride, n_q_heads=a0.n_q_heads, p=step.select_args.p,
                    kv_pools=step.kv_pools, kv_len=step.kv_len, block_table=step.block_table,
                    pages_per_seq=a0.block_table_stride, overlap_select=True)
    ov.load_inputs(step.draft_probs, step.q)
    ov.run()
    torch.cuda.synchronize()
    same = all(torch.equal(a, b) for a, b in zip(ref_out, ov.out))
    g, n = capture(ov.run)
    us = time_replays(g, reps, 3)
    return {"us_per_step": round(us, 1), "launches_per_step": n, "outputs_identical": bool(same),
            "note": "not the default: the selections' CTAs take SMs from the attention launches"}


def select_variants(step, cfg, reps=5):
    """The selection variants of Alg. 2 on the step's own draft rows (separate output buffers):
    device time per launch and mean kept count, beside the default (aggregate, exact)."""
    import torch
    import paper_2510_27641_b200 as sa
    out = {}
    idx = torch.empty_like(step.idx)
    for name, kw in (("aggregate_exact", {}), ("per_step_union_exact", dict(per_step=True)),
                     ("aggregate_bisect10", dict(bisect_iters=10)),
                     ("per_step_union_bisect10", dict(per_step=True, bisect_iters=10)),
                     ("chunk16_aggregate_exact", dict(chunk=16)),
                     ("chunk16_per_step_union_bisect10", dict(chunk=16, per_step=True, bisect_iters=10))):
        counts = torch.full_like(step.counts, -1)
        status = torch.full_like(step.row_status, -1)
        f = lambda: sa.select_topp(step.draft_probs, step.kv_len, step.layer_map, cfg.p, idx=idx, counts=counts,
                                   row_status=status, **kw)
        for _ in range(2):
            f()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            f()
        e1.record()
        torch.cuda.synchronize()
        c = counts.cpu().numpy()
        out[name] = {"us": round(e0.elapsed_time(e1) * 1e3 / reps, 1), "kept_mean": round(float(c[c >= 0].mean()), 1)}
    return out


def verify_micro(dev, reps=10, flags=0, only=""):
    """sparse_verify alone on synthetic shapes: dense long context and sparse lists of several
    lengths (shuffled block table, page 16).  Returns {case: {us, gbs}}; bytes = K/V rows read."""
    import torch
    import paper_2510_27641_b200 as sa
    import workloads as wl
    out = {}
    cases = [("dense_b4_ctx131072_q6x32_kv8", 4, 131072, 6, 32, 8, None),
             ("dense_b4_ctx131072_q5x64_kv8", 4, 131072, 5, 64, 8, None),
             # a dense cache of the size of the long lists below: same units, tiles and partition
             ("dense_b8_ctx12288_q6x32_kv8", 8, 12288, 6, 32, 8, None),
             ("sparse1245_b8_ctx32768_q6x32_kv8", 8, 32768, 6, 32, 8, 1245),
             ("sparse12450_b8_ctx32768_q6x32_kv8", 8, 32768, 6, 32, 8, 12450),
             ("sparse1000_b4_ctx131072_q5x64_kv8", 4, 131072, 5, 64, 8, 1000),
             # the same number of positions as scattered tokens and as whole 16-position chunks
             # (the second with SPECATTN_VERIFY_PAGE_LISTS: page-wise K/V reads)
             ("tokens1536_b8_ctx32768_q6x32_kv8", 8, 32768, 6, 32, 8, 1536),
             ("chunks96x16_b8_ctx32768_q6x32_kv8", 8, 32768, 6, 32, 8, -96),
             ("tokens12288_b8_ctx32768_q6x32_kv8", 8, 32768, 6, 32, 8, 12288),
             ("chunks768x16_b8_ctx32768_q6x32_kv8", 8, 32768, 6, 32, 8, -768)]
    for name, B, L, T, Hq, Hkv, count in cases:
        if only and name != only:
            continue
        page = 16
        pps = (L + page - 1) // page
        kv = wl.kv_pool(9, 0, B * pps, page, Hkv, 128, device=dev)
        bt = torch.from_numpy(wl.block_table(9, B, pps)).to(dev)
        q = torch.randn((B, T, Hq, 128), device=dev).to(torch.bfloat16)
        kv_len = torch.full((B,), L, dtype=torch.int32, device=dev)
        o = torch.empty((B, T, Hq, 128), dtype=torch.float32, device=dev)
        l = torch.empty((B, T, Hq), dtype=torch.float32, device=dev)
        case_flags = flags
        if count is None:
            kw, c = dict(dense=True), L
        elif count < 0:
            nch = -count
            ch = torch.stack([torch.sort(torch.randperm(L // 16, device=dev)[:nch])[0] for _ in range(B)])
            idx = (ch[:, :, None] * 16 + torch.arange(16, device=dev)[None, None, :]).reshape(B, 1, nch * 16)
            kw = dict(idx=idx.to(torch.int32).contiguous(),
                      counts=torch.full((B, 1), nch * 16, dtype=torch.int32, device=dev))
            c = nch * 16
            case_flags = flags | sa.VERIFY_PAGE_LISTS
        else:
            idx = torch.stack([torch.sort(torch.randperm(L, device=dev)[:count])[0] for _ in range(B)])
            kw = dict(idx=idx.to(torch.int32).view(B, 1, count).contiguous(),
                      counts=torch.full((B, 1), count, dtype=torch.int32, device=dev))
            c = count
        a = sa.make_verify_args(q, kv, kv_len, block_table=bt, out=o, lse=l, idx=kw.get("idx"),
                                counts=kw.get("counts"), dense=kw.get("dense", False))
        ws = sa.verify_workspace(a)
        f = lambda: sa.sparse_verify(q, kv, kv_len, block_table=bt, out=o, lse=l, workspace=ws, flags=case_flags, **kw)
        for _ in range(3):
            f()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            f()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / reps
        byts = B * c * Hkv * 512
        out[name] = {"us": round(us, 1), "kv_mb": round(byts / 1e6, 1), "gbs": round(byts / us / 1e3)}
        del kv
    return out


def layer_batched(step, cfg, si, reps=20):
    """Secondary number, an upper bound and not something a model can do: the attention of ALL
    target layers in ONE launch, as if the layers did not depend on one another (layer j's
    queries exist only after layer j - 1 has run).  Every (layer, sequence) becomes a sequence of
    a batch of layers x batch: its lists are copied from its draft layer's, its block table
    points into its layer's slice of the pool allocation.  It shows what the per-launch start-up
    and merge of the per-layer launches cost."""
    import torch
    import paper_2510_27641_b200 as sa
    m, B = step.n_layers, cfg.batch
    if si.block_table is None or m * B * cfg.n_kv_heads > 2048 or any(u < 0 for u in step.layer_map):
        return {"skipped": "needs a paged cache, sparse layers only and layers x batch x kv heads <= 2048"}
    dev = step.kv_big.device
    bt = torch.from_numpy(si.block_table).to(dev)
    bt_all = torch.cat([bt + j * si.n_pages for j in range(m)]).contiguous()
    idx_all = torch.cat([step.idx[u] for u in step.layer_map]).contiguous()          # [m B, G, stride]
    cnt_all = torch.cat([step.counts[u] for u in step.layer_map]).contiguous()
    kv_len_all = step.kv_len.repeat(m).contiguous()
    q_all = torch.cat(step.q).contiguous()
    out = torch.empty((m * B,) + tuple(step.out[0].shape[1:]), dtype=torch.float32, device=dev)
    lse = torch.empty((m * B,) + tuple(step.lse[0].shape[1:]), dtype=torch.float32, device=dev)
    a = sa.make_verify_args(q_all, step.kv_big, kv_len_all, block_table=bt_all, idx=idx_all, counts=cnt_all,
                            out=out, lse=lse)
    ws = sa.verify_workspace(a)
    f = lambda: sa.sparse_verify(q_all, step.kv_big, kv_len_all, block_table=bt_all, idx=idx_all, counts=cnt_all,
                                 out=out, lse=lse, workspace=ws)
    f()
    torch.cuda.synchronize()
    close = max(float((out[j * B:(j + 1) * B] - step.out[j]).abs().max()) for j in range(m))
    g, _ = capture(f)
    us = time_replays(g, reps, 5)
    kept = int(cnt_all.clamp(min=0).sum())
    kv_bytes = kept * cfg.n_kv_heads * cfg.head_dim * 4
    return {"us_all_layers_one_launch": round(us, 1), "kv_gbs": round(kv_bytes / us / 1e3),
            "frac_of_measured": round(kv_bytes / us / 1e3 / _measured_peaks()[0], 3),
            "max_abs_diff_vs_per_layer_launches": close,
            "note": "upper bound: layers treated as independent; the per-layer launches are the result"}


def config_section(cfg, dev, copies, reps=20, select_form=0):
    """One whole step (select + plans + verify per target layer) of a small configuration, timed
    as a CUDA graph over `copies` independent copies of ALL its inputs (draft rows, K/V pools,
    queries), one step per copy in turn, so that every step reads data that is not in L2
    (config 0's footprint is far below L2; one copy suffices where a step reads more than L2
    holds).  Bytes are the algorithmic ones of select and verify."""
    import torch
    peak = _measured_peaks()[0]
    built = [build_step(cfg, dev, select_form=select_form) for _ in range(copies)]
    si, _, step0, _, _ = built[0]
    steps = [b[2] for b in built]
    for st in steps:
        st.run()
    torch.cuda.synchronize()
    assert all(int(st.status.abs().sum()) == 0 and int((st.row_status > 0).sum()) == 0 for st in steps)
    counts = step0.counts.cpu().numpy()
    g_step, n_launch = capture(lambda: [st.run() for st in steps])
    g_sel, _ = capture(lambda: [st.run_select() for st in steps])
    g_ver, _ = capture(lambda: [st.run_verify(j) for st in steps for j in range(st.n_layers)])
    stats = {}
    us = time_replays(g_step, reps, 5, stats=stats) / copies
    us_sel = time_replays(g_sel, reps, 5) / copies
    us_ver = time_replays(g_ver, reps, 5) / copies
    per_layer = [verify_bytes(cfg, si, counts[int(u)]) for u in si.layer_map]
    v_bytes = sum(b for b, _ in per_layer)
    kv_bytes = sum(k for _, k in per_layer)
    dense_kv = int(si.kv_len.astype(np.int64).sum()) * cfg.n_kv_heads * cfg.head_dim * 4 * cfg.n_target_layers
    s_bytes = select_bytes(cfg, si, len(step0.used), counts)
    kept = counts[counts >= 0]
    return {"workload": cfg.name, "us_per_step": round(us, 2),
            "us_per_step_median": round(stats["median"] / copies, 2), "us_per_step_min": round(stats["min"] / copies, 2),
            "us_select": round(us_sel, 2), "us_verify": round(us_ver, 2),
            "launches_per_step": n_launch // copies, "rotating_copies": copies,
            "algorithmic_bytes": int(s_bytes + v_bytes), "gbs": round((s_bytes + v_bytes) / us / 1e3, 1),
            "frac_of_measured": round((s_bytes + v_bytes) / us / 1e3 / peak, 4),
            "select_bytes": int(s_bytes), "select_gbs": round(s_bytes / us_sel / 1e3, 1),
            "verify_bytes": int(v_bytes), "verify_gbs": round(v_bytes / us_ver / 1e3, 1),
            "kv_bytes_touched": int(kv_bytes), "kv_bytes_dense": int(dense_kv),
            "kv_touched_fraction": round(kv_bytes / dense_kv, 4),
            "kept_min_mean_max": [int(kept.min()), round(float(kept.mean()), 1), int(kept.max())],
            "ctx_min_max": [int(si.kv_len.min()), int(si.kv_len.max())]}


def long_context_layers(dev, want=80, reserve_gb=6.0):
    """Target layers of config 4 that fit the free HBM: every layer holds its own 2.147 GB K/V
    pool (batch 4 x 131072 positions x 8 heads x 128 x K and V in bf16)."""
    import torch
    import workloads as wl
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info(dev)
    cfg = wl.config4(n_target_layers=1)
    per_layer = cfg.batch * cfg.ctx * cfg.n_kv_heads * cfg.head_dim * 2 * 2
    draft = cfg.n_draft_layers * cfg.batch * cfg.n_draft_heads * cfg.gamma * cfg.ctx * 4 * 2   # rows + sums
    return int(max(1, min(want, (free - reserve_gb * 1e9 - draft) // per_layer)))


def long_context(dev, reps=10, n_layers=8):
    """Config 4 (batch 4, ctx 131072, 64 q / 8 kv heads, gamma 4, 4 draft layers of 16 heads) on
    `n_layers` target layers of the 80 (each has its own 2.1 GB K/V pool, so nothing is served
    from L2): one selection over the mapped draft layers + plans + one sparse verify per layer,
    timed as CUDA graphs for p in {0.8, 0.9, 0.95}, and the same verify kernel over everything
    (dense, p = 1), on both verify engines.  Bytes are the algorithmic ones: draft rows read by
    the selection, K/V rows read by the attention."""
    import torch
    import paper_2510_27641_b200 as sa
    import workloads as wl
    from workloads import bf16
    from paper_2510_27641_b200.step import VerifyStep
    peak = _measured_peaks()[0]
    cfg = wl.config4(n_target_layers=n_layers, p=0.9)
    si = wl.make_step_inputs(cfg)
    pools = [wl.kv_pool(cfg.seed, j, si.n_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim, device=dev)
             for j in range(n_layers)]
    kv_len = torch.from_numpy(si.kv_len).to(dev)
    bt = torch.from_numpy(si.block_table).to(dev)
    dp_host = [None if x is None else torch.from_numpy(x) for x in si.draft_probs]
    q_host = [bf16.bits_to_torch(q) for q in si.q]
    lmap = si.layer_map.tolist()
    n_used = len(set(lmap))
    sel_bytes = n_used * cfg.batch * cfg.n_draft_heads * cfg.gamma * cfg.ctx * 4
    out = {"layers": n_layers, "draft_layers_used": n_used, "lists": n_used * cfg.batch}
    for p in (0.8, 0.9, 0.95, 1.0):
        for eng, flags in (("mma_sync", sa.VERIFY_ENGINE_MMA_SYNC), ("tcgen05", sa.VERIFY_ENGINE_TCGEN05)):
            dense = p == 1.0
            step = VerifyStep(layer_map=[-1] * n_layers if dense else lmap, n_draft_layers=cfg.n_draft_layers,
                              batch=cfg.batch, n_draft_heads=cfg.n_draft_heads, gamma=cfg.gamma,
                              L_stride=si.L_stride, n_q_heads=cfg.n_q_heads, p=p, kv_pools=pools, kv_len=kv_len,
                              block_table=bt, pages_per_seq=si.pages_per_seq, verify_flags=flags)
            step.load_inputs([None] * cfg.n_draft_layers if dense else dp_host, q_host)
            step.run()
            torch.cuda.synchronize()
            assert int(step.status.abs().sum()) == 0
            if dense:
                kept = n_layers * cfg.batch * cfg.ctx
            else:
                kept = sum(int(step.counts[u].clamp(min=0).sum()) for u in lmap)
            kv_bytes = kept * cfg.n_kv_heads * cfg.head_dim * 4          # all layers
            g_v, _ = capture(lambda: [step.run_verify(j) for j in range(n_layers)])
            v_us = time_replays(g_v, reps, 3)
            rec = {"kept_frac": round(kept / (n_layers * cfg.batch * cfg.ctx), 4),
                   "verify_us_per_layer": round(v_us / n_layers, 1), "verify_gbs": round(kv_bytes / v_us / 1e3),
                   "verify_frac_of_measured": round(kv_bytes / v_us / 1e3 / peak, 3)}
            if not dense:
                g_s, _ = capture(step.run)
                s_us = time_replays(g_s, reps, 3)
                rec.update(step_us=round(s_us, 1), select_us=round(s_us - v_us, 1),
                           select_gbs=round(sel_bytes / (s_us - v_us) / 1e3),
                           step_gbs=round((kv_bytes + sel_bytes) / s_us / 1e3),
                           step_frac_of_measured=round((kv_bytes + sel_bytes) / s_us / 1e3 / peak, 3))
                del g_s
            out[f"p={p}/{eng}"] = rec
            del g_v, step
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--topp-sweep", action="store_true", help="(default on) the 256-row selection micro-benchmark of config 2")
    ap.add_argument("--no-topp-sweep", action="store_true", help="skip the selection micro-benchmark")
    ap.add_argument("--verify-micro", action="store_true", help="only run the sparse_verify micro-benchmark")
    ap.add_argument("--verify-case", default="", help="with --verify-micro: run only the case of this name")
    ap.add_argument("--verify-engine", default="auto", choices=["auto", "mma_sync", "tcgen05"],
                    help="force one implementation of sparse_verify (default: the library picks by shape)")
    ap.add_argument("--long-context", action="store_true", help="only run the config-4 (ctx 131072) measurements")
    ap.add_argument("--no-long-context", action="store_true", help="skip the config-4 (ctx 131072) measurements")
    ap.add_argument("--long-context-layers", type=int, default=0,
                    help="target layers of config 4 held on the device (2.1 GB of K/V each); "
                         "0 = as many of the 80 as the free HBM holds")
    ap.add_argument("--no-small-configs", action="store_true", help="skip configs 0 and 3")
    ap.add_argument("--topp-case", default="",
                    help="only run one cell of the selection micro-benchmark: family,n,p,rows (e.g. zipf,131072,0.9,32)")
    ap.add_argument("--layers", type=int, default=0, help="override the number of target layers (debug)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-select-workspace", action="store_true",
                    help="selection without its optional workspace: one cluster per list whatever their number")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    import workloads as wl
    cfg = wl.config1()
    if args.layers:
        cfg = cfg.scaled(n_target_layers=args.layers)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    import paper_2510_27641_b200 as sa
    rank, local_rank, world = _rank_env()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    barrier = None
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        barrier = lambda: (dist.barrier(), torch.cuda.synchronize())

    vflags = {"auto": 0, "mma_sync": sa.VERIFY_ENGINE_MMA_SYNC, "tcgen05": sa.VERIFY_ENGINE_TCGEN05}[args.verify_engine]
    if args.verify_micro:
        print(json.dumps({"verify_micro": verify_micro(dev, reps=min(10, max(2, args.steps)), flags=vflags,
                                                       only=args.verify_case),
                          "engine": args.verify_engine}))
        return

    if args.long_context:
        nl = args.long_context_layers or long_context_layers(dev)
        print(json.dumps({"long_context": long_context(dev, reps=min(10, max(2, args.steps)), n_layers=nl)}))
        return

    if args.topp_case:
        fam, n, p, rows = args.topp_case.split(",")
        print(json.dumps({"topp_case": topp_sweep(dev, reps=min(5, max(1, args.steps)), families=[fam], sizes=[int(n)],
                                                   ps=[float(p)], n_rows=int(rows))}))
        return

    # every rank owns a batch of its own (batch sharding): same shapes, rank-specific seed
    cfg_r = rank_config(cfg, rank, world)
    si, pools, step, dp_host, q_host = build_step(cfg_r, dev, verify_flags=vflags,
                                                  select_workspace=not args.no_select_workspace)
    step.run()
    torch.cuda.synchronize()
    counts = step.counts.cpu().numpy()
    assert int(step.status.abs().sum()) == 0 and int((step.row_status.cpu().numpy() > 0).sum()) == 0

    g_step, n_step = capture(step.run)
    g_verify, n_verify = capture(lambda: [step.run_verify(j) for j in range(step.n_layers)])
    g_select, n_select = capture(step.run_select)

    try:
        uuid = str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        uuid = None
    sampler = ClockSampler(local_rank, uuid)
    with sampler:
        step_stats = {}
        us_step = time_replays(g_step, args.steps, args.warmup, barrier, stats=step_stats)
        us_verify_all = time_replays(g_verify, args.steps, args.warmup)
        us_select = time_replays(g_select, args.steps, args.warmup)
    clocks = sampler.summary()

    # eager launches (no graph) for comparison
    for _ in range(3):
        step.run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_eager = max(3, min(args.steps, 20))
    e0.record()
    for _ in range(n_eager):
        step.run()
    e1.record()
    torch.cuda.synchronize()
    us_eager = e0.elapsed_time(e1) * 1e3 / n_eager

    # end to end from pinned host buffers through the C ABI
    out_host = [torch.empty(o.shape, dtype=torch.float32).pin_memory() for o in step.out]
    lse_host = [torch.empty(l.shape, dtype=torch.float32).pin_memory() for l in step.lse]
    n_e2e = max(3, min(args.steps, 20))
    for _ in range(3):
        step.run_host(dp_host, q_host, out_host, lse_host)
    torch.cuda.synchronize()
    if barrier is not None:
        barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n_e2e):
        step.run_host(dp_host, q_host, out_host, lse_host)
    e1.record()
    torch.cuda.synchronize()
    us_e2e = e0.elapsed_time(e1) * 1e3 / n_e2e
    assert torch.equal(out_host[-1], step.out[-1].cpu())
    h2d = sum(t.numel() * 4 for t in dp_host if t is not None) + sum(t.numel() * 2 for t in q_host)
    d2h = sum(t.numel() * 4 for t in out_host) + sum(t.numel() * 4 for t in lse_host)

    us_step, us_e2e, us_verify_all, us_select = reduce_max([us_step, us_e2e, us_verify_all, us_select], world, dev)

    # ---- roofline of the dominant kernel (sparse verify) -------------------------------------
    per_layer = [verify_bytes(cfg_r, si, counts[int(u)]) for u in si.layer_map]
    bytes_launch = float(np.mean([b for b, _ in per_layer]))
    kv_bytes_step = sum(k for _, k in per_layer)
    dense_kv_step = int(si.kv_len.astype(np.int64).sum()) * cfg.n_kv_heads * cfg.head_dim * 4 * cfg.n_target_layers
    us_launch = us_verify_all / step.n_layers
    peak, peak_kind = _measured_peaks()
    achieved = bytes_launch / us_launch / 1e3
    n_used = len(step.used)
    sel_b = select_bytes(cfg_r, si, n_used, counts)
    roofline = {"kernel": "sparse_verify_kernel<2,4>", "bound": "hbm", "achieved": round(achieved, 1),
                "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4), "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
                "traffic": NCU_VERIFY_TRAFFIC_BYTES, "bytes_per_launch": round(bytes_launch),
                "us_per_launch": round(us_launch, 3),
                "select": {"kernel": "select_topp_kernel", "bytes_per_launch": sel_b, "us_per_launch": round(us_select, 3),
                           "achieved": round(sel_b / us_select / 1e3, 1),
                           "frac": round(sel_b / us_select / 1e3 / peak, 4)}}

    line = {"metric": METRIC, "value": round(us_step, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(us_step / 1e3, 6), "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_dict(cfg, world),
            "e2e": {"value": round(us_e2e, 1), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": int(n_step * args.steps),
            "clocks": clocks, "roofline": roofline,
            "extra": {"launch": f"CUDA graph of 1 select + 1 plan launch ({len(step.plans)} plans) + {step.n_layers} verify launches",
                      "us_step_batches": step_stats, "us_verify_per_step": round(us_verify_all, 3), "us_select_per_step": round(us_select, 3),
                      "us_step_eager_launches": round(us_eager, 3),
                      "topp_lists_per_s": round(n_used * cfg.batch / us_select * 1e6),
                      "topp_prob_rows_per_s": round(n_used * cfg.batch * cfg.n_draft_heads * cfg.gamma / us_select * 1e6),
                      "kept_mean": float(counts[counts >= 0].mean()),
                      "kv_bytes_touched_per_step": int(kv_bytes_step), "kv_bytes_dense_per_step": int(dense_kv_step),
                      "kv_touched_fraction": round(kv_bytes_step / dense_kv_step, 5),
                      "sequences_per_s": round(cfg.batch * world / us_step * 1e6, 1)}}

    # The sections below add context to the line; a failure in one of them (say, no memory left
    # for the long-context pools on a shared GPU) is recorded and must not lose the step's numbers.
    def extra(name, fn):
        try:
            line["extra"][name] = fn()
        except Exception as e:  # noqa: BLE001
            line["extra"][name] = {"error": f"{type(e).__name__}: {e}"[:300]}

    if rank == 0:
        extra("select_variants", lambda: select_variants(step, cfg_r))
        extra("overlapped_selection_schedule", lambda: overlapped_schedule(step))
        extra("layer_batched_upper_bound", lambda: layer_batched(step, cfg_r, si))
    if rank == 0 and not args.no_cpu_baseline:
        smp = OracleSample(cfg_r, si, n_attn_layers=8, pools=pools)
        us_cpu, sample = smp.step_us()
        line["cpu_baseline"] = {"value": round(us_cpu, 1), "unit": UNIT, "cores": smp.cores, "kind": "oracle",
                                "sample": sample}
    # the step's own buffers (34 GB of K/V pools) make room for the other configurations
    del g_step, g_verify, g_select, step, pools
    if "smp" in locals():
        del smp
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    if rank == 0 and not args.no_topp_sweep:
        extra("topp_sweep", lambda: topp_sweep(dev))
        sweep = line["extra"]["topp_sweep"]
        if "error" not in sweep:
            # the second half of the metric: rows/s of the selection alone, per row length
            # (geometric mean over the three families and three p of config 2)
            by_n = {}
            for k, v in sweep.items():
                by_n.setdefault(k.split("/")[1], []).append(v["rows_per_s"])
            line["extra"]["topp_rows_per_s"] = {n: round(float(np.exp(np.mean(np.log(v))))) for n, v in by_n.items()}
    if rank == 0 and not args.no_small_configs:
        # config 0 is latency-bound (0.8 MB of draft rows, 3 MB of K/V): 64 rotating copies of
        # all inputs keep every step's reads out of L2; config 3 reads more than L2 per step
        extra("config0", lambda: config_section(wl.config0(), dev, copies=64))
        torch.cuda.empty_cache()
        # (a ragged batch: the caller knows it and asks for the selection's two-launch form)
        extra("config3", lambda: config_section(wl.config3(), dev, copies=1,
                                                 select_form=sa.SELECT_FORM_TWO_LAUNCH))
        torch.cuda.empty_cache()
    if rank == 0 and not args.no_long_context:
        extra("long_context", lambda: long_context(dev, n_layers=args.long_context_layers or long_context_layers(dev)))
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
