"""The N > 1 path of bench.py on CPU: two gloo ranks.  The path shards by batch with no data-path
collective, so what there is to check is the plumbing: every rank gets its own batch (seed), the
job's time is the slowest rank's, the throughput counts all ranks' scale-steps, and the reference arm
prints from rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2505_19602_b200 import synth

    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = bench.rank_workload(synth.WORKLOADS["tiny"], rank, world)
    Q, K, V = synth.scale_inputs(wl, 0, 2)
    ms_local = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, world, "cpu")
    value = bench.job_throughput(wl.n_scales, 3, world, ms)
    dist.barrier()
    json.dump({"seed": wl.seed, "q0": float(Q.flatten()[0]), "ms": ms, "value": value},
              open(os.path.join(out_dir, f"rank{rank}.json"), "w"))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_batch_and_reduce_time(tmp_path):
    world, port = 2, 29611
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [json.load(open(tmp_path / f"rank{i}.json")) for i in range(world)]
    assert r[0]["seed"] != r[1]["seed"] and r[0]["q0"] != r[1]["q0"]          # different batches
    assert r[0]["ms"] == r[1]["ms"] == 15.0                                    # the slowest rank's time
    assert abs(r[0]["value"] - 4 * 3 * 2 / 0.015) < 1e-6 and r[0]["value"] == r[1]["value"]


def test_reference_arm_prints_from_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29612")
    outs = []
    for rank in (0, 1):
        res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                              "--steps", "1", "--warmup", "0", "--gpus", "2"], env=dict(env, RANK=str(rank)),
                             capture_output=True, text=True, timeout=300)
        assert res.returncode == 0, res.stderr
        outs.append(res.stdout.strip())
    line = json.loads(outs[0])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
    assert outs[1] == ""
