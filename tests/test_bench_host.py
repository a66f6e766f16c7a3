"""Host logic of bench.py that a multi-GPU launch relies on, exercised with two gloo ranks on CPU:
the max-over-ranks reduction of the timings, and the reference arm's rank gating."""
import importlib.util
import json
import os
import socket
import subprocess
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bench = _bench()
    got = bench.max_over_ranks(torch, [1.0 + rank, 10.0 - rank, 5.0], dist, torch.device("cpu"))
    dist.barrier()
    dist.destroy_process_group()
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump(got, f)


def test_max_over_ranks_with_two_gloo_ranks(tmp_path):
    port = _free_port()
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        assert json.load(open(tmp_path / f"r{rank}.json")) == [2.0, 10.0, 5.0]


def test_max_over_ranks_single_process():
    bench = _bench()
    assert bench.max_over_ranks(torch, [3.5, 1.25], None, torch.device("cpu")) == [3.5, 1.25]


def test_reference_arm_is_silent_on_other_ranks():
    """Under a multi-rank launch only rank 0 runs and prints the reference line; the others exit 0."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0
    assert r.stdout.strip() == ""
