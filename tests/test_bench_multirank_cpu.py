"""The N > 1 path of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job aggregate,
and the reference arm printing on rank 0 only."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run_two_ranks(script: str, port: int):
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), PYTHONPATH=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", script], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    return [o for o, _ in outs]


def test_max_over_ranks_and_aggregate_with_gloo():
    script = textwrap.dedent("""
        import os, json, torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        rank = dist.get_rank()
        step_ms, fwd_ms = bench.max_over_ranks([1.0 + rank, 5.0 - rank], dist, "cpu")
        dist.barrier()
        if rank == 0:
            print(json.dumps({"step": step_ms, "fwd": fwd_ms, "value": bench.whole_job_tflops(2e12, 2, step_ms)}))
        dist.destroy_process_group()
    """)
    out0, out1 = _run_two_ranks(script, 29611)
    got = json.loads(out0.strip().splitlines()[-1])
    assert got["step"] == 2.0 and got["fwd"] == 5.0      # slowest rank decides
    assert abs(got["value"] - 2 * 2e12 / 2e-3 / 1e12) < 1e-9  # both replicas' work over the max time
    assert out1.strip() == ""                           # only rank 0 prints


def test_reference_arm_prints_on_rank0_only():
    outs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", PYTHONPATH=ROOT)
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "c1",
                            "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                           cwd=ROOT, timeout=300)
        assert r.returncode == 0, r.stderr
        outs.append(r.stdout.strip())
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2
    assert outs[1] == ""
