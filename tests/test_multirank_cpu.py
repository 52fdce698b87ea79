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


def _shard_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import numpy as np
    import workloads as wl
    from oracle import gptaq_oracle as orc
    from paper_2504_02692_b200 import sharded
    cfg = wl.scaled(wl.CONFIGS["cfg1"], n=48, m=70, batch_tokens=64, n_batches=5, group=0, blocksize=32)
    # this rank's share of the token batches, accumulated by the oracle into plain CPU tensors
    st = orc.new_stats(cfg.n)
    for b in sharded.token_shard(cfg.n_batches, rank, world):
        X, Xfp = wl.make_batch(cfg, b)
        orc.accumulate(st, X.numpy(), Xfp.numpy())
    H, D = torch.from_numpy(st.H.astype(np.float32)), torch.from_numpy(st.D.astype(np.float32))

    class HostState:
        """What allreduce_statistics needs of a LayerState, over plain CPU tensors."""
        def __init__(self, tokens): self._tokens, self.views = tokens, 0
        def H(self): self.views += 1; return H
        def D(self): self.views += 1; return D
        def tokens(self): return self._tokens
        def set_tokens(self, t): self._tokens = t

    hs = HostState(st.tokens)
    total = sharded.allreduce_statistics(hs)
    assert hs.tokens() == total and hs.views == 2
    full = orc.new_stats(cfg.n)
    for b in range(cfg.n_batches):
        X, Xfp = wl.make_batch(cfg, b)
        orc.accumulate(full, X.numpy(), Xfp.numpy())
    ok_stats = total == full.tokens and np.allclose(H.numpy(), full.H, rtol=1e-5) and np.allclose(D.numpy(), full.D, rtol=1e-4, atol=1e-3)
    # row slabs: quantizing a slab gives the slab of the full result (rows are independent)
    W = wl.make_weight(cfg).numpy().astype(np.float64)
    U, dead = orc.factor(full.H, full.tokens, cfg.damp)
    P = orc.build_P(full.D, full.tokens, U, cfg.alpha)
    r0, r1 = sharded.row_shard(cfg.m, rank, world)
    mine = orc.quantize(W[r0:r1], U, P, dead, cfg.bits, cfg.group, cfg.sym)
    whole = orc.quantize(W, U, P, dead, cfg.bits, cfg.group, cfg.sym)
    ok_rows = np.array_equal(mine.codes, whole.codes[r0:r1])
    spans = [None] * world
    dist.all_gather_object(spans, (r0, r1))
    if rank == 0:
        json.dump({"ok_stats": bool(ok_stats), "ok_rows": bool(ok_rows), "spans": spans}, open(out, "w"))
    dist.barrier()
    dist.destroy_process_group()


def test_token_sharded_statistics_and_row_sharded_quantize(tmp_path):
    """The one exchange step of a layer spread over ranks: all-reduced partial sums equal the full sums, and
    the row slabs tile the matrix and reproduce the full result."""
    from paper_2504_02692_b200 import sharded
    assert [list(sharded.token_shard(5, r, 2)) for r in range(2)] == [[0, 1, 2], [3, 4]]
    assert [list(sharded.token_shard(3, r, 4)) for r in range(4)] == [[0], [1], [2], []]
    assert [sharded.row_shard(70, r, 2) for r in range(2)] == [(0, 64), (64, 70)]
    assert [sharded.row_shard(4096, r, 8) for r in range(8)] == [(512 * r, 512 * r + 512) for r in range(8)]
    out = str(tmp_path / "shard.json")
    mp.spawn(_shard_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    res = json.load(open(out))
    assert res["ok_stats"] and res["ok_rows"] and res["spans"] == [[0, 64], [64, 70]]
