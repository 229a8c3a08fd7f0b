"""The N > 1 bookkeeping of the benchmark on CPU: two gloo ranks, no GPU.

Rows are independent, so ranks share nothing on the data path; the only cross-rank step is the
maximum over the ranks' times, from which the whole-job rate is computed."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + rank, 3.0 - rank, 7.0]                 # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(mine, torch.device("cpu"), world)
    rate = bench.whole_job_rate(1000.0, world, got[0])
    if rank == 0:
        out.put((got, rate))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got, rate = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert got == [11.0, 3.0, 7.0]
    assert abs(rate - 2 * 1000.0 / 11e-3) < 1e-6


def _shard_worker(rank, world, port, out):
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    import oracle
    import synth_inputs as si
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    case = si.config3()
    x = case.x.reshape(-1, case.C)[:1000]                # 1000 rows: the last rank gets a ragged block
    wq = oracle.quantize_weight(case.w)                   # replicated on every rank
    lo, hi = bench.shard_rows(x.shape[0], rank, world)
    xa = oracle.quantize_act(x[lo:hi])
    y = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"])["y"]
    parts = [None] * world
    dist.all_gather_object(parts, (lo, hi, xa["codes"], xa["scale"], y))
    if rank == 0:
        parts.sort(key=lambda p: p[0])
        assert parts[0][0] == 0 and parts[-1][1] == x.shape[0]
        assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1)) and all(p[0] % 128 == 0 for p in parts)
        full = oracle.quantize_act(x)
        y_full = oracle.w4a4_linear(full["codes"], full["scale"], wq["codes"], wq["scale"])["y"]
        ok = (np.array_equal(np.concatenate([p[2] for p in parts]), full["codes"])
              and np.array_equal(np.concatenate([p[3] for p in parts]), full["scale"])
              and np.array_equal(np.concatenate([p[4] for p in parts]), y_full))
        out.put(ok)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_the_rows_and_reproduce_the_unsharded_result():
    """Row shards through the whole path (here the oracle stands in for it, on CPU) concatenate to the unsharded
    result bit for bit: the ranks exchange nothing but the finished outputs."""
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    assert out.get(timeout=300) is True
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    import bench
    for M, world in [(18464, 8), (256, 4), (100, 3), (1, 2)]:
        spans = [bench.shard_rows(M, r, world) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == M and all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))


def test_graph_steps_divides_the_step_count_and_respects_the_buffer_rotation():
    import bench
    for K, nsets in [(1000, 2), (50, 2), (7, 2), (64, 3), (97, 2), (128, 4), (3, 2)]:
        G = bench.graph_steps(K, nsets)
        assert K % G == 0 and 1 <= G <= max(K, 64)
        # either a whole number of rotations per graph, or one graph that holds every step
        assert G % nsets == 0 or G == K


def _run_reference_arm(extra_env):
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ)
    env.update(extra_env)
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "1",
                        "--workload", "cfg1"], capture_output=True, text=True, env=env, cwd=root, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    return [json.loads(l) for l in lines]


def test_reference_arm_prints_the_contract_line_on_the_host_cores():
    (line,) = _run_reference_arm({"RANK": "0", "WORLD_SIZE": "1"})
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0 and line["higher_is_better"] is True
    assert line["steps"] == 1 and line["warmup"] == 1 and line["ms_per_step"] > 0 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["cpu_baseline"]["value"] == line["value"] and line["cpu_baseline"]["sample"]
    assert line["e2e"] == dict(value=line["value"], unit="GB/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0)
    assert line["config"]["workload"].startswith("cfg1")


def test_reference_arm_is_silent_on_other_ranks():
    assert _run_reference_arm({"RANK": "1", "WORLD_SIZE": "2", "LOCAL_RANK": "1"}) == []
