"""The multi-rank path of bench.py on CPU: two gloo ranks join, take the max of
their step times and the sum of their token counts, and rank 0 alone reports."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import torch
    import bench
    rank, local_rank, world = bench.dist_setup("gloo")
    assert world == 2 and rank == int(os.environ["RANK"])
    dev = torch.device("cpu")
    bench.dist_barrier(world)
    ms = bench.dist_max(10.0 + 5.0 * rank, world, dev)          # rank 1 is the slow one
    tokens = bench.dist_sum(1000.0, world, dev)
    value = bench.aggregate_throughput(1000.0, ms, 4, tokens)
    bench.dist_barrier(world)
    if rank == 0:
        print(json.dumps({"ms": ms, "tokens": tokens, "value": value}))
""") % ROOT


def test_two_gloo_ranks_reduce_time_and_tokens(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT="29533")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    assert outs[1][0].strip() == ""                    # only rank 0 prints
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["ms"] == 15.0 and line["tokens"] == 2000.0
    # 2000 tokens per layer pass, 4 layers in 15 ms -> tokens / (ms / layers)
    assert abs(line["value"] - 2000.0 / (15.0e-3 / 4)) < 1e-6


def test_reference_arm_on_non_zero_rank_exits_without_work():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_prints_the_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "tiny"], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
