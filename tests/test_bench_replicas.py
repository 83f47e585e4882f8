"""The N > 1 path of bench.py on CPU: two gloo ranks, replicas only (no data-path collective).
Checks the max-over-ranks reduction of the device times, the whole-job value, per-rank seeds, and that
only rank 0 of the reference arm prints a line."""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(code, world=2, extra_env=None):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), PYTHONPATH=ROOT)
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable, "-c", code], cwd=ROOT, env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_max_over_ranks_and_whole_job_value_with_two_gloo_ranks():
    code = textwrap.dedent("""
        import os, json
        import torch.distributed as dist
        import bench
        rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
        dist.init_process_group("gloo")
        dist.barrier()
        mine = [10.0 * (rank + 1), 7.0 - rank]              # rank 1 is slower on the first, rank 0 on the second
        got = bench.max_over_ranks(mine, world)
        dist.barrier()
        print(json.dumps({"rank": rank, "got": got, "seed": bench.replica_seed("mixed_13b", rank),
                          "value": bench.whole_job_value(3 * 10**12, world, got[0])}))
        dist.destroy_process_group()
    """)
    outs = [json.loads(o.strip().splitlines()[-1]) for o in _launch(code)]
    for o in outs:
        assert o["got"] == [20.0, 7.0]                       # the slowest rank sets the time
        assert abs(o["value"] - 2 * 3.0 / 20e-3) < 1e-9      # 2 replicas x 3 TFLOP in 20 ms
    assert outs[0]["seed"] != outs[1]["seed"] and outs[0]["seed"] == 189895


def test_reference_arm_prints_on_rank_zero_only():
    code = textwrap.dedent("""
        import sys
        sys.argv = ["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                    "--workload", "tiny", "--cpu-budget", "1"]
        import bench
        bench.main()
    """)
    outs = _launch(code)
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    assert outs[1].strip() == ""
