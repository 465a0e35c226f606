"""Host-side logic of the benchmark: byte accounting, the replica aggregation over ranks (gloo, 2 ranks) and the
launch contract of the CPU reference arm."""
import json
import os
import socket
import subprocess
import sys

import pytest

import kg_inputs as ki
from paper_2404_18911_b200 import traffic

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_algorithmic_bytes_of_the_7b_shape():
    sh = ki.get_config("7b")
    d, F, V = 4096, 11008, 32000
    assert traffic.layer_weight_bytes(sh) == (4 * d * d + 3 * d * F) * 2 == 404_750_336
    assert traffic.head_weight_bytes(sh) == V * d * 2 == 262_144_000
    assert traffic.adapter_weight_bytes(sh) == 4 * d * d * 2
    assert traffic.kv_bytes_per_token_layer(sh) == 16_384
    # a draft step at KV length 512 is ~1.23 GB, a verify pass ~12.66 GB, a greedy step ~13.5 GB
    assert abs(traffic.draft_step_bytes(sh, 512) / 1e9 - 1.231) < 0.005
    assert abs(traffic.verify_bytes(sh, 512, 1) / 1e9 - 12.657) < 0.005
    assert abs(traffic.ar_step_bytes(sh, 512) / 1e9 - 13.485) < 0.005
    # verify bytes grow only by the K/V of the extra rows
    assert traffic.verify_bytes(sh, 512, 7) - traffic.verify_bytes(sh, 512, 1) == 30 * 12 * 16_384


def test_decode_bytes_follow_the_round_log():
    sh = ki.get_config("7b")
    log = [(3, 3, 3, 512), (2, 2, 0, 516)]        # round 1 accepts everything: the adapter lags in round 2
    b = traffic.decode_bytes(sh, log)
    r1 = traffic.round_bytes(sh, 3, 3, 512, 0)
    r2 = traffic.round_bytes(sh, 2, 2, 516, 1)
    assert b == r1 + r2
    assert r2 > traffic.round_bytes(sh, 2, 2, 516, 0)      # the catch-up row reads and writes one more K/V entry
    # n_d + 1 shallow passes, n_steps adapter + head passes, one verify pass
    expect = sum(traffic.shallow_pass_bytes(sh, 512 + j) for j in range(4)) + \
        sum(traffic.adapter_head_bytes(sh, 512 + j, 1) for j in range(3)) + traffic.verify_bytes(sh, 512, 4)
    assert r1 == expect


def _gloo_worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    vals = bench.max_over_ranks([10.0 + rank, 5.0 - rank], dist, "cpu")
    out.put((rank, vals))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_over_two_gloo_ranks():
    import torch.multiprocessing as mp
    sys.path.insert(0, ROOT)
    import bench
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gloo_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0] == got[1] == [11.0, 5.0]                  # every rank sees the slowest rank's time
    # two replicas that each make 256 tokens per step in 2 s -> 256 tokens/s for the job
    assert bench.job_throughput(256, 1, 2, 2000.0) == pytest.approx(256.0)
    assert bench.max_over_ranks([3.0], None, "cpu") == [3.0]


def test_reference_arm_prints_one_line_from_rank_zero_only():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny", "--gpus", "2",
           "--steps", "1", "--warmup", "0"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["n_gpus"] == 2 and j["value"] > 0
    assert j["cpu_baseline"]["kind"] == "oracle" and j["e2e"]["h2d_bytes_per_step"] == 0
    assert j["config"]["workload"].startswith("tiny")
