"""The multi-rank plumbing of bench.py on CPU: two gloo ranks, no GPU.

With N > 1 the benchmark runs N independent replicas (the decode path has no exchange step), so
what the ranks share is only the timing reduction and who prints.
"""
import json
import os
import socket
import subprocess
import sys
import textwrap

REPO = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(code_or_args, world, as_code):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), PYTHONPATH=REPO + os.pathsep + os.environ.get("PYTHONPATH", ""))
        cmd = [sys.executable, "-c", code_or_args] if as_code else [sys.executable] + code_or_args
        procs.append(subprocess.Popen(cmd, env=env, cwd=REPO, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=600) for p in procs]
    return [(p.returncode, o, e) for p, (o, e) in zip(procs, outs)]


def test_timings_reduce_to_the_slowest_rank_and_throughput_sums_replicas():
    code = textwrap.dedent("""
        import os, json, torch, torch.distributed as dist
        import bench
        from paper_2503_00979_b200 import synth
        rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
        dist.init_process_group("gloo")
        ms, ms_e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 40.0 - 3.0 * rank], torch.device("cpu"), world)
        w = bench.replica_workload(synth.WORKLOADS["c0"], rank)
        print(json.dumps({"rank": rank, "ms": ms, "ms_e2e": ms_e2e, "seed": w.seed,
                          "value": bench.whole_job_tokens_per_s(world, 4, 100, ms)}))
        dist.barrier()
        dist.destroy_process_group()
    """)
    res = _spawn(code, 2, as_code=True)
    lines = []
    for rc, out, err in res:
        assert rc == 0, err[-2000:]
        lines.append(json.loads(out.strip().splitlines()[-1]))
    lines.sort(key=lambda r: r["rank"])
    for r in lines:
        assert r["ms"] == 15.0 and r["ms_e2e"] == 40.0               # max over ranks, element-wise
        assert abs(r["value"] - 2 * 4 * 100 / 15e-3) < 1e-6           # both replicas' tokens over the slowest time
    assert lines[0]["seed"] != lines[1]["seed"]                       # replicas decode different content


def test_reference_arm_prints_on_rank_zero_only():
    args = ["bench.py", "--impl", "reference", "--gpus", "2", "--workload", "c0", "--steps", "4", "--warmup", "3"]
    res = _spawn(args, 2, as_code=False)
    (rc0, out0, err0), (rc1, out1, err1) = res
    assert rc0 == 0, err0[-2000:]
    assert rc1 == 0, err1[-2000:]
    assert out1.strip() == ""                                          # the other rank exits without work
    line = json.loads(out0.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
