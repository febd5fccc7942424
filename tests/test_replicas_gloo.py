"""The multi-process side of the benchmark on CPU: two gloo ranks exercise the replica bookkeeping
(disjoint layers per rank, job time = slowest rank, aggregate throughput), and the reference arm run under
torchrun prints exactly one line, from rank 0."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2407_08454_b200 import replicas
from paper_2407_08454_b200 import synth_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str) -> None:
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        layers = replicas.layers_for_rank(rank, world, 3)
        mine = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        job_ms = replicas.slowest_rank_ms(mine, dist)
        gathered = [None] * world
        dist.all_gather_object(gathered, layers)
        # every rank's inputs differ: the generator is keyed by layer
        cfg = si.CONFIGS["C0"]
        k = si.make_layer(cfg, layer=layers[0])["K"]
        sums = [None] * world
        dist.all_gather_object(sums, float(k.double().sum()))
        dist.barrier()
        with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
            json.dump({"layers": gathered, "job_ms": job_ms, "sums": sums}, f)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_take_disjoint_layers_and_agree_on_the_slowest_time(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    assert res[0] == res[1]                                         # both ranks saw the same job-wide figures
    assert res[0]["layers"] == [[0, 1, 2], [3, 4, 5]]
    assert res[0]["job_ms"] == 15.0
    assert res[0]["sums"][0] != res[0]["sums"][1]
    assert replicas.aggregate_throughput(2, 10, 1000, 15.0) == pytest.approx(2 * 10 * 1000 / 0.015)


def test_single_process_helpers():
    assert replicas.layers_for_rank(0, 1, 3) == [0, 1, 2]
    assert replicas.slowest_rank_ms(7.5) == 7.5
    with pytest.raises(ValueError):
        replicas.layers_for_rank(2, 2, 3)
    with pytest.raises(ValueError):
        replicas.aggregate_throughput(1, 1, 1, 0.0)


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference",
           "--gpus", "2", "--steps", "1", "--warmup", "0"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
