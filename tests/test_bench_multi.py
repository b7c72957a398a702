"""The N > 1 path of bench.py: replicas only, max over ranks, whole-job rate.

Runs as two gloo ranks on the CPU; no GPU and no compute.
"""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r measured (10 + r) ms device time and (1 + 2r) s end to end
        got = bench.max_over_ranks([10.0 + rank, 1.0 + 2.0 * rank], "cpu")
        dist.barrier()
        with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
            json.dump(got, f)
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_world2(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        got = json.load(open(tmp_path / f"r{r}.json"))
        assert got == [11.0, 3.0]   # the slowest rank's figures, on every rank


def test_whole_job_rate_counts_every_replica():
    sys.path.insert(0, ROOT)
    import bench
    one = bench.whole_job_rate(1, 64 * 1000, 10, 0.5)
    assert one == 64 * 1000 * 10 / 0.5
    assert bench.whole_job_rate(4, 64 * 1000, 10, 0.5) == 4 * one


@pytest.mark.parametrize("rank", [0, 1])
def test_reference_arm_runs_on_rank0_only(rank):
    env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
               MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "c1_ring4_topk", "--steps", "1", "--warmup", "3"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    if rank != 0:
        assert r.stdout.strip() == ""       # other ranks leave without work
        return
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0


def test_byte_model_of_the_step():
    """Minimum bytes a step must move: each dense array once, messages once per reader."""
    sys.path.insert(0, ROOT)
    import bench
    import workloads
    wl = workloads.WORKLOADS["c4_torus64_topk"]
    w = wl.mixing()
    N, k, nnz = 64 * 1_000_000, 10_000, 64 * 5
    assert bench.message_bytes(wl) == 8 * k
    want = 20 * N + 8 * k * 64 + 8 * k * (nnz - 64) + 4 * (64 * k + nnz * k)
    assert bench.step_min_bytes(wl, w) == want == 1_320_960_000
    assert bench.update_kernel_bytes(wl, w) == 20 * N + 8 * k * nnz + 4 * (64 * k + nnz * k)

    wl = workloads.WORKLOADS["c5_ring32_qsgd"]
    w = wl.mixing()
    d = 25_557_032
    per_worker = 4 * ((d + 511) // 512) + 4 * ((d + 31) // 32) + d // 2      # norms, sign plane, nibbles
    assert bench.message_bytes(wl) == per_worker
    assert bench.step_min_bytes(wl, w) == 28 * 32 * d + per_worker * 32 * 3  # written once, read by two neighbours
    assert abs(bench.step_min_bytes(wl, w) - 24.45e9) < 0.01e9

    # per layer: the entries kept and the message are sums over the layers
    wl = workloads.WORKLOADS["l3_ring8_topk_layers"]
    sizes = wl.layer_sizes()
    assert bench.entries_per_row(wl) == sum(max(1, s // 100) for s in sizes)
    assert bench.message_bytes(wl) == 8 * bench.entries_per_row(wl)
    wl = workloads.WORKLOADS["l3_ring8_sign_layers"]
    assert bench.message_bytes(wl) == sum(4 * ((s + 31) // 32) + 4 for s in sizes)
