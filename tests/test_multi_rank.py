"""The N > 1 host logic of bench.py on CPU: two gloo ranks, the slowest rank sets the time, the reference
arm runs on rank 0 only, and the batch is never split (independent matrices, one full batch per rank)."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run_ranks(script, world=2, port=29731):
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), PYTHONPATH=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", script], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_max_over_ranks_and_aggregate_with_gloo():
    script = textwrap.dedent("""
        import os, json
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        rank = dist.get_rank()
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist)       # rank 1 is slower
        val = bench.aggregate_throughput(1000.0, dist.get_world_size(), ms)
        print(json.dumps({"rank": rank, "ms": ms, "val": val}))
        dist.barrier()
        dist.destroy_process_group()
    """)
    outs = [json.loads(o.strip().splitlines()[-1]) for o in _run_ranks(script)]
    for o in outs:
        assert o["ms"] == 15.0                                   # the slowest rank's time on every rank
        assert abs(o["val"] - 2 * 1000.0 / 15e-3) < 1e-6         # whole-job units per second


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", PYTHONPATH=ROOT)
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--small", "--gpus", "2",
                        "--steps", "1"], env=env, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env["RANK"] = "0"
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--small", "--gpus", "2",
                        "--steps", "1"], env=env, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    assert line["metric"].startswith("deflated polar-filter")


def test_single_rank_helpers_need_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_throughput(10.0, 4, 2.0) == 4 * 10.0 / 2e-3
    # flops the method needs for one 1600 x 6400 matrix: the symmetric products once per pair, or in full
    filt, rest = bench.algorithmic_flops(1600, 6400, 32, 16, 2, 5, symmetric=False)
    assert abs(filt - 5 * (4 * 1600 ** 2 * 6400 + 2 * 1600 ** 3)) < 1
    assert abs(filt - bench.dense_filter_flops(1600, 6400, 5)) < 1
    fs, rs = bench.algorithmic_flops(1600, 6400, 32, 16, 2, 5, symmetric=True)
    assert abs(fs - 5 * (1600 * 1601 * 6400 + 1600 ** 2 * 1601 + 2 * 1600 ** 2 * 6400)) < 1
    # front end: six products with the 48-column panel and the rank-32 subtraction; the additive restore adds a rank-32 product
    assert abs(rest - (2 * 6400 * 1600 * 48 * 6 + 2 * 1600 * 6400 * 32)) < 1 and rs == rest
    assert bench.algorithmic_flops(1600, 6400, 32, 16, 2, 5, True, add_restore=True)[1] - rest == 2 * 1600 * 6400 * 32
    assert bench.algorithmic_flops(1600, 6400, 0, 0, 0, 5, True)[1] == 0


def test_gpus_flag_starts_its_own_ranks_when_no_launcher_did(monkeypatch):
    """`bench.py --gpus N` without an outer torchrun builds the launcher command itself (127.0.0.1 rendezvous, a free
    port, one process per GPU, the same arguments); under a launcher (WORLD_SIZE set) it does not."""
    import bench
    calls = []
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: calls.append(cmd) or 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "2"])
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    with __import__("pytest").raises(SystemExit) as e:
        bench.main()
    assert e.value.code == 0 and len(calls) == 1
    cmd = calls[0]
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4" and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "2"] and cmd[-5].endswith("bench.py")
