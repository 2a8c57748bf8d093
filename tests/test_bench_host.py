"""Host-side logic of bench.py that needs no GPU: the multi-rank aggregation (gloo, two CPU
ranks) and the reference arm's JSON line."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    bench.barrier(world)
    # rank r claims (10 + 5 r) ms for 100 (r + 1) units
    t, u = bench.reduce_max_time_sum_units(10.0 + 5.0 * rank, 100.0 * (rank + 1), world)
    q.put((rank, t, u))
    dist.destroy_process_group()


def test_two_rank_aggregation_takes_slowest_time_and_all_units():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0, 300.0), (1, 15.0, 300.0)]


def test_single_rank_aggregation_is_identity():
    import bench
    assert bench.reduce_max_time_sum_units(3.5, 42.0, 1) == (3.5, 42.0)


def test_reference_arm_prints_contract_line():
    env = dict(os.environ, OMP_NUM_THREADS="4")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--workload", "cfg0", "--steps", "2", "--warmup", "1"],
                         capture_output=True, text=True, env=env, timeout=600)
    assert res.returncode == 0, res.stderr
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "positions/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["higher_is_better"] is True
    # other ranks of a torchrun launch exit quietly
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--workload", "cfg0", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, env=dict(env, RANK="1", WORLD_SIZE="2"),
                         timeout=600)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_parity_helpers_count_planted_mismatches():
    """The in-run parity verdict of bench.py: bit-exact for the deterministic path, and for the
    stochastic path only decisions / draws that the oracle itself reports as close may differ."""
    import numpy as np
    import bench
    B = 5
    ref = {"accept_len": np.arange(B, dtype=np.int32), "out_tokens": np.arange(B * 6, dtype=np.int32).reshape(B, 6),
           "out_len": np.arange(1, B + 1, dtype=np.int32)}
    got = {k: v.copy() for k, v in ref.items()}
    keys = ("accept_len", "out_tokens", "out_len")
    assert bench.parity_deterministic(got, ref, B, keys)["mismatches"] == 0
    got["out_tokens"][3, 2] += 1
    got["accept_len"][1] += 1
    p = bench.parity_deterministic(got, ref, B, keys)
    assert p["mismatches"] == 2 and p["checked_sequences"] == B

    N = 4
    ref = {"accept_len": np.array([1, 2, 0], np.int32), "path_nodes": np.zeros((3, N), np.int32),
           "out_len": np.array([2, 3, 1], np.int32), "seq_status": np.zeros(3, np.int32),
           "node_how": np.ones((3, N), np.uint8), "out_tokens": np.array([[7, 9, -1, -1], [4, 5, 6, -1], [3, -1, -1, -1]], np.int32),
           "node_prob": np.full((3, N), 0.25), "margin": np.array([[1e-3, 1e-2], [1e-6, 1e-2], [1e-3, 1e-7]])}
    got = {k: v.copy() for k, v in ref.items() if k != "margin"}
    assert bench.parity_stochastic(got, ref, 3)["mismatches"] == 0
    got["accept_len"][1] = 1                 # a walk that differs, but its closest decision was within tolerance
    got["out_tokens"][2, 0] = 8              # another drawn token, the oracle's draw sat on a CDF step
    p = bench.parity_stochastic(got, ref, 3)
    assert p["mismatches"] == 0 and p["decisions_within_tolerance"] == 1 and p["draws_within_tolerance"] == 1
    got["out_tokens"][0, 1] = 1              # a clear draw that differs
    got["node_prob"][0, 0] *= 1.001
    assert bench.parity_stochastic(got, ref, 3)["mismatches"] == 2
