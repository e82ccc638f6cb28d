"""Host-side logic of the N > 1 benchmark path on CPU ranks (gloo, world size 2).

The path shards with no data-path collective: every rank runs the same per-GPU workload and the only
communication is the barrier and the max-over-ranks of the step time.  These tests run that logic in
two real processes over gloo, and check that under a two-rank launch the reference arm runs on rank 0
only."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, {root!r})
    import torch, torch.distributed as dist
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    local_ms = 2.0 + 3.0 * rank          # rank 1 is the slow one
    dist.barrier()
    ms = bench.max_over_ranks(local_ms, world, torch.device("cpu"))
    value = bench.whole_job_value(1e12, world, ms, 1e12)
    dist.barrier()
    dist.destroy_process_group()
    print(json.dumps({{"rank": rank, "ms": ms, "value": value}}))
""")


def test_max_over_ranks_and_whole_job_value_two_gloo_ranks(tmp_path):
    port = 29000 + os.getpid() % 2000
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, port=port))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["ms"] == 5.0                      # the slowest rank's time on every rank
        assert abs(o["value"] - 2 * 1.0 / 5e-3) < 1e-9   # both ranks' units over that time


def test_reference_arm_runs_on_rank_zero_only():
    base = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
            "--warmup", "1", "--workload", "cfg1", "--cpu-seconds", "1"]
    env1 = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r1 = subprocess.run(base, env=env1, capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    env0 = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    r0 = subprocess.run(base, env=env0, capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0, r0.stderr[-2000:]
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["config"]["workload"] == "cfg1"


def test_gpus_flag_starts_one_rank_per_gpu():
    """`bench.py --gpus 2` without a launcher re-executes itself under torchrun with two ranks (rendezvous on
    127.0.0.1).  Run on the reference arm, which needs no GPU: rank 0 alone times the oracle and prints the one JSON
    line, the other rank exits 0 without work."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference",
                        "--workload", "cfg1", "--steps", "1", "--warmup", "1", "--cpu-seconds", "0.2"],
                       capture_output=True, text=True, timeout=300, env=env, cwd=root)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["config"]["workload"] == "cfg1"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["cpu_baseline"]["kind"] == "oracle"
