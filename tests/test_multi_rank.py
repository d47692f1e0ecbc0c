"""The N > 1 path of the benchmark on CPU: two gloo ranks shard the workload by sequence batch
(rank-specific seeds, no data-path collective) and combine their timings with a MAX reduction."""
import os
import subprocess
import sys
import textwrap
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import numpy as np, torch, torch.distributed as dist
    import bench, workloads as wl
    rank, local_rank, world = bench._rank_env()
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = bench.rank_config(wl.config1().scaled(n_target_layers=2, n_draft_layers=2, batch=2, ctx=256), rank, world)
    si = wl.make_step_inputs(cfg)
    # each rank's batch is its own: different seeds give different draft rows, same shapes
    digest = float(np.sum([x.sum() for x in si.draft_probs if x is not None])) + 1e-3 * float(si.q[0].astype(np.float64).sum())
    t = bench.reduce_max([10.0 + rank, 100.0 - rank], world, device="cpu")
    gathered = [None] * world
    dist.all_gather_object(gathered, (cfg.seed, si.draft_probs[int(si.layer_map[0])].shape, digest))
    if rank == 0:
        print(json.dumps({"max": t, "ranks": gathered}))
    dist.barrier()
    dist.destroy_process_group()
""") % str(ROOT)


def test_two_gloo_ranks_shard_by_batch_and_reduce_with_max(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", WORLD_SIZE="2")
    procs = []
    for r in range(2):
        e = dict(env, RANK=str(r), LOCAL_RANK=str(r))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=e, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["max"] == [11.0, 100.0]                      # MAX over ranks, element-wise
    (s0, shape0, d0), (s1, shape1, d1) = res["ranks"]
    assert s0 != s1 and shape0 == shape1 and d0 != d1        # same shapes, different data


def test_single_rank_config_is_the_named_workload():
    sys.path.insert(0, str(ROOT))
    import bench
    import workloads as wl
    cfg = wl.config1()
    assert bench.rank_config(cfg, 0, 1) == cfg
    assert bench.rank_config(cfg, 3, 8).seed == cfg.seed + 3000
    assert bench.reduce_max([1.5, 2.5], 1) == [1.5, 2.5]
