"""Host-side logic of the multi-rank benchmark path, on CPU with the gloo backend (world size 2):
the max-over-ranks reduction, the per-rank layer seeds, and the reference arm under a two-rank
launch (rank 0 alone measures and prints, the other rank exits 0 without work)."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    import workloads as wl
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
    cfg = bench.rank_config(wl.CONFIGS["cfg1"], rank)
    W = wl.make_weight(cfg)
    gathered = [torch.zeros_like(W) for _ in range(world)]
    dist.all_gather(gathered, W)
    if rank == 0:
        json.dump({"ms": ms, "layers_differ": not torch.equal(gathered[0], gathered[1]),
                   "per_layer": bench.per_layer_ms(ms, world)}, open(out, "w"))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_per_rank_layers(tmp_path):
    out = str(tmp_path / "r0.json")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    res = json.load(open(out))
    assert res["ms"] == 15.0 and res["per_layer"] == 7.5 and res["layers_differ"]


def test_reference_arm_under_two_ranks_prints_once():
    """torchrun-style environment, two processes: one JSON line in total, from rank 0."""
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(
            [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--workload", "cfg1",
             "--steps", "1", "--warmup", "0"], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    lines0 = [l for l in outs[0][0].splitlines() if l.startswith("{")]
    lines1 = [l for l in outs[1][0].splitlines() if l.startswith("{")]
    assert len(lines0) == 1 and not lines1
    line = json.loads(lines0[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
