"""The multi-GPU launch path on CPU: two `gloo` ranks run the host-side plumbing of `bench.py --gpus 2`
(per-rank batches, barrier, max/sum reduction of the timings).  The path has no data-path collective."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_21788_b200 import fcp, ranks, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = ranks.rank_workload("tiny", seed=0, rank=rank, world=world)
        # every rank plans its own batch on the host (no GPU needed for the plan)
        plan = fcp.fcp_plan_blocks(w.seqlens, w.cp_degrees, w.hq, w.hkv, w.head_dim)
        ms_local = 10.0 * (rank + 1)                      # rank 1 is the slow one
        dist.barrier()
        ms, flops = ranks.aggregate(ms_local, w.flops_fwd_bwd(), "cpu")
        out.put((rank, w.seqlens.tolist(), plan.info("n_pairs"), w.flops_fwd_bwd(), ms, flops))
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_different_batches_and_reduce_timings():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, len0, pairs0, f0, ms0, tot0), (r1, len1, pairs1, f1, ms1, tot1) = res
    assert (r0, r1) == (0, 1)
    assert len0 != len1                                   # seed = base seed + rank
    assert len0 == synth.make_workload("tiny", seed=0).seqlens.tolist()
    assert len1 == synth.make_workload("tiny", seed=1).seqlens.tolist()
    assert pairs0 > 0 and pairs1 > 0
    assert ms0 == ms1 == 20.0                             # max over ranks
    assert tot0 == tot1 == f0 + f1                        # whole-job FLOPs
    assert np.isclose(ranks.throughput_tflops(ms0, 4, tot0), (f0 + f1) / (5e-3) / 1e12)


def test_single_process_is_the_identity():
    assert ranks.aggregate(3.5, 7.0, "cpu") == (3.5, 7.0)
    w = ranks.rank_workload("tiny", seed=2, rank=0, world=1)
    assert w.seqlens.tolist() == synth.make_workload("tiny", seed=2).seqlens.tolist()


def test_bench_gpus_n_starts_its_own_ranks():
    """`python bench.py --gpus 2` run plainly (no WORLD_SIZE in the environment) starts two ranks through
    torch.distributed.run and rank 0 prints one JSON line with n_gpus = 2.  Here on CPU: `gloo` ranks and a
    sleep in place of the GPU step (`--selftest-launcher`), the same rank plumbing as the measured path."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "2", "--selftest-launcher"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["selftest"] == "launcher" and out["value"] is None
    f0 = synth.make_workload("tiny", 0).flops_fwd_bwd()
    f1 = synth.make_workload("tiny", 1).flops_fwd_bwd()
    assert out["flops_rank0"] == f0 and out["flops_all_ranks"] == f0 + f1      # seed = rank: different batches, summed
    assert out["max_ms_over_ranks"] >= 20.0                                    # rank 1 sleeps 20 ms: max over ranks
