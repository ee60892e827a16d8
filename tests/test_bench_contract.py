"""bench.py's CPU-only legs: the reference arm (the oracle timed on host cores) prints exactly one
JSON line with the contract's keys, alone and under a 2-rank torchrun launch (rank 0 prints, the
other rank exits 0 without work).  The path itself does not shard: N > 1 means independent replicas,
so the only exchange is the timed arm's maximum over the ranks' step times, which a two-rank gloo job checks
together with the whole-job throughput formula."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
KEYS = {"impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
        "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"}


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _check_line(out, n_gpus):
    lines = [l for l in out.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1, out
    d = json.loads(lines[0])
    assert KEYS <= set(d)
    assert d["impl"] == "reference" and d["n_gpus"] == n_gpus and d["unit"] == "TFLOP/s"
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] == d["e2e"]["value"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["config"]["workload"] == "config1" and d["vs_baseline"] is None


def test_reference_arm_prints_one_contract_line():
    out = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--workload", "config1", "--steps", "2",
                          "--warmup", "1"], cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr
    _check_line(out.stdout, 1)


def test_reference_arm_under_two_rank_torchrun():
    env = dict(os.environ, OMP_NUM_THREADS="2")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), "bench.py", "--gpus", "2",
                          "--impl", "reference", "--workload", "config1", "--steps", "1", "--warmup", "0"],
                         cwd=ROOT, capture_output=True, text=True, timeout=900, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    _check_line(out.stdout, 2)


def _aggregate_rank(rank, world, port, times_ms, flops, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        ms = bench.max_over_ranks(torch, times_ms[rank], world, torch.device("cpu"))
        out[rank] = (ms, bench.whole_job_tflops(flops, world, ms))
    finally:
        dist.destroy_process_group()


def test_job_time_is_the_slowest_rank_and_value_counts_every_replica():
    """The N > 1 path of the timed arm on two gloo ranks: every rank ends up with the maximum of the ranks' step
    times, and the reported throughput is both replicas' work over that time."""
    import torch.multiprocessing as mp
    world, flops, times = 2, 3.0e12, [2.0, 5.0]
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_aggregate_rank, args=(world, _free_port(), times, flops, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for ms, value in res.values():
        assert ms == 5.0
        assert abs(value - world * flops / 5.0e-3 / 1e12) < 1e-9
    import bench, torch
    assert bench.max_over_ranks(torch, 7.5, 1, torch.device("cpu")) == 7.5
    assert bench.whole_job_tflops(1.0e12, 1, 1000.0) == 1.0
