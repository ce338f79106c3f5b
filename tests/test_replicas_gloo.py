"""The N > 1 path on CPU: two gloo ranks take disjoint shares of a batch (replicas need no
exchange on the data path), each runs its share through the oracle, and the shares
concatenate to the single-rank result; the timing reduction is a max over ranks."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2609_14237_b200 import synth

    wl = synth.WORKLOADS["c1_tiny"]
    inp = synth.make_inputs(wl, device="cpu", growth=1, steps=1)
    rows = list(synth.shard_rows(wl.batch, rank, world))
    pool = oracle.as_u16(inp.pools[0]).copy()
    n = inp.kv_lens(0)
    out, lse, rc = oracle.decode_attention(pool, wl.num_q_heads, wl.num_kv_heads, wl.head_dim, 16, inp.q[0, 0], n,
                                           inp.page_tables[0], rows=rows)
    assert rc == 0
    mine = torch.from_numpy(out[rows])
    gathered = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)                      # test-only: compare with the single-rank result
    t = torch.tensor([1.0 + rank], dtype=torch.float64)  # stand-in for a per-rank step time
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    nbytes = torch.tensor([float(sum(int(n[r]) for r in rows) * wl.kv_bytes_per_token)], dtype=torch.float64)
    dist.all_reduce(nbytes, op=dist.ReduceOp.SUM)
    if rank == 0:
        full, _, _ = oracle.decode_attention(pool, wl.num_q_heads, wl.num_kv_heads, wl.head_dim, 16, inp.q[0, 0], n,
                                             inp.page_tables[0])
        ret["same"] = bool((torch.cat(gathered).numpy() == full).all())
        ret["tmax"] = float(t.item())
        ret["bytes"] = float(nbytes.item())
        ret["want_bytes"] = float(inp.kv_bytes(0))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_partition_the_batch_and_reduce_time_by_max():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_worker, args=(world, port, ret), nprocs=world, join=True)
        assert ret["same"] is True
        assert ret["tmax"] == 2.0
        assert ret["bytes"] == ret["want_bytes"]
