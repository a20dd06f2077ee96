"""The N > 1 logic of bench.py on CPU (gloo, world size 2): replicas only, step time = slowest rank,
whole-job throughput = tokens of all ranks / that time; the reference arm prints on rank 0 only."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 1.0 + rank            # rank 1 is the slow one
    job_ms = bench.max_over_ranks(ms, dist, torch.device("cpu"))
    out.put((rank, job_ms, bench.job_tokens_per_s(64, world, job_ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_job_throughput_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, job_ms, tps in res:
        assert job_ms == 2.0                       # the slowest rank's time, on every rank
        assert tps == pytest.approx(64 * 2 / 2.0e-3)


def test_single_process_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.job_tokens_per_s(64, 1, 0.5) == pytest.approx(128000.0)
    from paper_2504_15299_b200 import synth
    wl = synth.WORKLOADS["mixtral_decode"]
    K = len(wl.bits)
    # all 8 experts active at 8 bits: every plane of every expert + metadata
    group_off = [0]
    for e in range(wl.n_experts):
        for kk in range(K):
            group_off.append(group_off[-1] + (16 if kk == K - 1 else 0))
    b = bench.algorithmic_bytes(wl, 64, group_off)
    per_matrix = 14336 * 4096 + 14336 * 32 * 4
    assert b["active_experts"] == 8
    assert b["gate_up"] == 8 * 2 * per_matrix + 128 * 4096 * 2 + 128 * 14336 * 2
    # only expert 0 active, at 2 bits: a quarter of the code bytes
    group_off = [0, 5] + [5] * (wl.n_experts * K - 1)
    b = bench.algorithmic_bytes(wl, 64, group_off)
    assert b["active_experts"] == 1
    assert b["down"] == 14336 * 4096 // 4 + 4096 * 112 * 4 + 128 * 14336 * 2 + 128 * 4096 * 4


def test_gpus_flag_starts_the_replicas_itself():
    """`python bench.py --gpus 2` run as a plain script starts two ranks (torch.distributed.run, rendezvous on
    127.0.0.1) and passes rank 0's line on; the self-check arm stands in for the layer call (gloo, made-up step
    times 1 ms and 2 ms), so this runs without a GPU."""
    import json
    import subprocess
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.replica_command(2, ["--gpus", "2"], port=1234)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-2:] == ["--gpus", "2"]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "selfcheck"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["ms_per_step"] == 2.0 and d["value"] == pytest.approx(64 * 2 / 2.0e-3)
