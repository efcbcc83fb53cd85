"""World-size-2 gloo test (CPU) of the multi-GPU host logic: row sharding without a data-path collective."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_04215_b200 import dist as D
from paper_2604_04215_b200 import inputs as I


def test_shard_rows_partition():
    for n in (1, 7, 16, 64, 65):
        for world in (1, 2, 3, 8):
            spans = [D.shard_rows(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    from oracle import dare_oracle as O
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = I.scaled(I.WORKLOADS["tiny"], batch=4, vocab=512, mask_id=511, hidden=64, prompt_len=16, mode=I.SELECT_TOPK, k=3)
    si = I.make_step(wl, step=0)
    lo, hi = D.shard_rows(wl.batch, rank, world)
    f = lambda t: None if t is None else t.to(torch.float64).numpy()
    L = wl.block_len
    # each rank runs the step on its own rollouts only: no exchange is needed for the result to be right
    res = O.denoise_step(f(si.q[lo:hi]), f(si.k_pre[lo:hi]), f(si.v_pre[lo:hi]), si.prefix_len[lo:hi].numpy(),
                         f(si.k_blk[lo:hi]), f(si.v_blk[lo:hi]), None, None, None, f(si.x[lo * L:hi * L]), f(si.w),
                         si.tokens[lo:hi].numpy(), si.block_start, L, wl.mask_id, wl.mode, wl.threshold, wl.k)
    mine = torch.from_numpy(res["tokens"])
    allt = D.gather_tokens(mine)
    ms, n = D.reduce_step_stats(10.0 + rank, float(res["n_committed"].sum()))
    if rank == 0:
        full = O.denoise_step(f(si.q), f(si.k_pre), f(si.v_pre), si.prefix_len.numpy(), f(si.k_blk), f(si.v_blk), None,
                              None, None, f(si.x), f(si.w), si.tokens.numpy(), si.block_start, L, wl.mask_id, wl.mode,
                              wl.threshold, wl.k)
        ok = bool((allt.numpy() == full["tokens"]).all()) and ms == 10.0 + world - 1 and n == float(full["n_committed"].sum())
        open(os.path.join(out_dir, "ok"), "w").write("1" if ok else "0")
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_rollouts_and_reduce(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert open(tmp_path / "ok").read() == "1"


def test_bench_starts_its_own_ranks_when_no_launcher_set_the_environment(tmp_path):
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment must start two ranks by itself (one process
    per GPU through torch.distributed.run on 127.0.0.1).  Checked on the CPU with the oracle arm standing in for the
    step: the two ranks meet over gloo, rank 0 alone prints the line, the other exits 0."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--workload", "tiny", "--steps", "2", "--warmup", "1"],
                         env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                              # rank 0 alone reports
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2 and lines[0]["value"] > 0
    # a rank count that contradicts the launcher's is refused instead of silently timing another job
    env1 = dict(env, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    bad = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--workload", "tiny", "--steps", "1", "--warmup", "0"],
                         env=env1, capture_output=True, text=True, timeout=600)
    assert bad.returncode != 0 and "does not match WORLD_SIZE" in bad.stderr
