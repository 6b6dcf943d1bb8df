"""The N > 1 path of bench.py on CPU: two gloo ranks, whole-job throughput = units summed
over ranks / time maximised over ranks; the reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    import bench

    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank,
                            world_size=world)
    ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1), dist)
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, ms, units))


def test_aggregate_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29611, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    for _, ms, units in res:
        assert ms == 15.0 and units == 300.0


def test_aggregate_without_process_group_is_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.aggregate_over_ranks(3.0, 7.0, None) == (3.0, 7.0)


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, WORLD_SIZE="2")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "1",
           "--steps", "2", "--warmup", "1"]
    r1 = subprocess.run(cmd, env=dict(env, RANK="1"), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=dict(env, RANK="0", CUDA_VISIBLE_DEVICES=""), capture_output=True,
                        text=True, timeout=300)
    assert r0.returncode == 0, r0.stderr
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_both_arms_describe_the_workload_with_the_same_config_object():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2602_07878_b200 import workloads as wl

    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "1",
           "--steps", "1", "--warmup", "0"]
    r = subprocess.run(cmd, env=dict(os.environ, CUDA_VISIBLE_DEVICES=""), capture_output=True,
                       text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["config"] == bench.config_of(wl.config_spec(1), 1)   # what the GPU arm prints


def test_ncu_traffic_is_reported_only_for_the_captured_shape_and_partition_size():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2602_07878_b200 import workloads as wl

    spec = wl.config_spec(3)
    assert bench.ncu_traffic(spec, 512) == 1597484800
    assert bench.ncu_traffic(spec, 256) is None
    assert bench.ncu_traffic(wl.config_spec(3, scale_down=8), 512) is None   # same name, smaller
    other = wl.make_spec(spec.name, seq_lens=spec.seq_lens, num_q_heads=16, num_kv_heads=8,
                         head_dim=256, num_blocks=spec.num_blocks, seed=1)
    assert bench.ncu_traffic(other, 512) is None
    s = bench.spread([3.0, 1.0, 2.0])
    assert (s["median"], s["min"], s["max"], s["n"]) == (2.0, 1.0, 3.0, 3)
