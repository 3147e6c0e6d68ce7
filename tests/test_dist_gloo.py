"""World-size-2 CPU (gloo) test of the multi-process path: every rank plans its own replica, the
whole-job tile count is the sum over ranks, the step time is the maximum over ranks, and only
rank 0 reports."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_09385_b200 import binding as B
from paper_2607_09385_b200 import inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = inputs.Workload("replica", 1, 4, 2, 2048, 128, 128, inputs.MASK_CAUSAL | inputs.MASK_BITMAP,
                        keep_prob=0.3)
    bitmap = inputs.block_bitmap(w.heads_q, w.tiles, w.tiles, w.keep_prob, seed=inputs.DEFAULT_SEED + rank)
    p, keep = B.make_params(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                            w.block, w.block, 0, bitmap)
    st, stats, _ = B.steel_attn_plan_host(p)
    assert st == 0
    tiles = torch.tensor([float(stats["kept_tiles"])], dtype=torch.float64)
    fake_ms = torch.tensor([1.0 + rank], dtype=torch.float64)       # rank 1 is the slow one
    total = tiles.clone()
    dist.all_reduce(total, op=dist.ReduceOp.SUM)
    dist.all_reduce(fake_ms, op=dist.ReduceOp.MAX)
    dist.barrier()
    if rank == 0:
        out.put((float(tiles), float(total), float(fake_ms)))
    else:
        out.put((float(tiles), None, None))
    dist.destroy_process_group()


def test_two_rank_replicas_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    own = sorted(r[0] for r in results)
    reported = [r for r in results if r[1] is not None]
    assert len(reported) == 1
    assert reported[0][1] == sum(own) and reported[0][2] == 2.0
    assert own[0] != own[1]      # different seeds give different bitmaps per replica
