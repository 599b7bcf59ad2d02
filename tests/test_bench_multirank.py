"""Host logic of the multi-rank benchmark path, run as two gloo ranks on the CPU: the
max-over-ranks timing reduction, the whole-job aggregate, the block sharding (disjoint
blocks per rank, no data-path collective), and the rule that only rank 0 prints."""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    from paper_2601_07396_b200 import streams
    rank, world, local = bench.dist_env()
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.reduce_max(10.0 + 5.0 * rank, world, torch.device("cpu"))
    blocks = bench.rank_blocks(streams.FLUX, rank, 57)
    value = bench.whole_job_value(1_000_000_000, 4, world, ms)
    dist.barrier()
    print(json.dumps({"rank": rank, "world": world, "ms": ms, "first": blocks[0], "last": blocks[-1],
                      "n": len(blocks), "value": value}))
    dist.destroy_process_group()
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(code, world, extra_args=()):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code, *extra_args], env=env, cwd=ROOT,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_two_ranks_reduce_time_by_max_and_own_disjoint_blocks():
    outs = _launch(WORKER, 2)
    rows = sorted((json.loads(o.strip().splitlines()[-1]) for o in outs), key=lambda r: r["rank"])
    assert [r["world"] for r in rows] == [2, 2]
    # the slowest rank's time is everybody's time
    assert rows[0]["ms"] == rows[1]["ms"] == 15.0
    # 57 blocks each, no overlap
    assert (rows[0]["first"], rows[0]["last"], rows[0]["n"]) == (0, 56, 57)
    assert (rows[1]["first"], rows[1]["last"], rows[1]["n"]) == (57, 113, 57)
    # whole job = both ranks' bytes over the slowest time
    assert rows[0]["value"] == rows[1]["value"] == 2 * 4 * 1.0 / 15e-3


def test_reference_arm_runs_on_rank_zero_only():
    code = "import sys; sys.argv = ['bench.py', '--impl', 'reference', '--steps', '1', '--warmup', '0', " \
           "'--workload', 'tiny', '--ref-rows', '64']; import runpy; runpy.run_path(%r, run_name='__main__')" \
           % os.path.join(ROOT, "bench.py")
    outs = _launch(code, 2)
    lines = [o.strip() for o in outs]
    printed = [l for l in lines if l]
    assert len(printed) == 1
    rec = json.loads(printed[0].splitlines()[-1])
    assert rec["impl"] == "reference" and rec["cpu_baseline"]["kind"] == "oracle" and rec["gpu_launches"] == 0
    assert rec["e2e"]["h2d_bytes_per_step"] == 0
