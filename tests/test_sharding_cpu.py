"""The head-sharded step on 2 gloo ranks on CPU: shards of the workload, the exchange of the cluster flags, and
that every rank then schedules the same union.  The kernels' part is played by the oracle here (a CPU machine has no
CUDA); the GPU tests run the library's two halves on shards of one device."""
import json
import os
import sys

import numpy as np
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _select(w):
    """Oracle stages 1-2 on a (shard of a) workload -> (sel, n_sel, flags over the global cluster ids)."""
    import oracle
    from paper_2603_17803_b200.workloads import bits_u16
    cfg = w.cfg
    pb, cl = w.page_base.numpy(), w.ctx_len.numpy()
    ksum = oracle.build_summaries(bits_u16(w.kv_pool), pb, cl, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    _, s32, _ = oracle.scores(bits_u16(w.q), ksum, pb, cl, cfg.n_kv_heads, cfg.page_size, cfg.max_pages())
    sel, n_sel = oracle.topk(s32, cl, cfg.page_size, cfg.top_k)
    flags = np.zeros(w.n_clusters, dtype=np.uint8)
    p2c, cb = w.page2cluster.numpy(), w.cluster_base.numpy()
    for b in range(cfg.batch):
        for h in range(cfg.n_q_heads):
            pages = sel[b, h, : n_sel[b, h]]
            flags[cb[b] + p2c[pb[b] + pages]] = 1
    return sel, n_sel, flags


def _workload():
    from paper_2603_17803_b200 import workloads as W
    cfg = W.scaled(W.CONFIGS["c3_batched"], batch=2, ctx_len=16 * 150 + 3, top_k=12, n_topics=6)
    return W.generate(cfg, seed=3)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(world), RANK=str(rank),
                      LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import torch.distributed as dist
    from paper_2603_17803_b200 import sharding
    dist.init_process_group("gloo")
    w = _workload()
    shard = sharding.shard_workload(w, rank, world)
    sel, n_sel, flags = _select(shard)
    mine = int(flags.sum())
    union = sharding.exchange_flags(torch.from_numpy(flags.copy())).numpy()
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"mine": mine, "union": union.tolist(), "sel": sel.tolist(), "heads": shard.cfg.n_q_heads}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_hold_the_union_of_the_activated_clusters(tmp_path):
    sys.path.insert(0, ROOT)
    import oracle
    world = 2
    mp.spawn(_worker, args=(world, 31000 + os.getpid() % 2000, str(tmp_path)), nprocs=world, join=True)
    r = [json.load(open(tmp_path / f"r{i}.json")) for i in range(world)]
    w = _workload()
    sel, n_sel, flags = _select(w)                           # the unsharded step
    assert r[0]["union"] == r[1]["union"] == flags.tolist()
    assert max(r[0]["mine"], r[1]["mine"]) < int(flags.sum())        # neither rank saw the whole union alone
    # the shards' selections are the unsharded selection's head blocks
    got = np.concatenate([np.array(r[i]["sel"]) for i in range(world)], axis=1)
    assert np.array_equal(got, sel)
    # and the schedule every rank derives from the union is the unsharded one
    uniq, queue_of, load = oracle.resolve(sel, n_sel, w.page_base.numpy(), w.page2cluster.numpy(), w.cluster_base.numpy(),
                                          w.cluster_replica_mask.numpy().view(np.uint32),
                                          w.cluster_size.numpy().view(np.uint16), w.cfg.n_queues)
    assert np.array_equal(uniq, np.flatnonzero(np.array(r[0]["union"])))


def test_shards_partition_the_heads():
    sys.path.insert(0, ROOT)
    from paper_2603_17803_b200 import sharding
    w = _workload()
    parts = [sharding.shard_workload(w, r, 4) for r in range(4)]
    assert torch.equal(torch.cat([p.q for p in parts], dim=1), w.q)
    assert torch.equal(torch.cat([p.kv_pool for p in parts], dim=1), w.kv_pool)
    assert all(p.cfg.n_q_heads // p.cfg.n_kv_heads == w.cfg.n_q_heads // w.cfg.n_kv_heads for p in parts)
    assert all(p.page2cluster is w.page2cluster and p.cluster_size is w.cluster_size for p in parts)
