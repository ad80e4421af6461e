"""A step whose query heads are spread over several GPUs, one process and one ctx per GPU.

Stages 1, 2 and 4 are independent per KV head, so rank r holds the K/V pool, the summaries and the queries of
its own KV heads only.  Stage 3 (Eq. 8: one I/O set per step over all heads) needs the union of the clusters
every rank activated: between the two halves of the step the ranks combine their cluster flag arrays by
maximum -- one all-reduce of max_clusters_total bytes -- after which every rank runs the same deterministic
queue assignment on the same union and keeps attending to its own heads.

    shard = shard_workload(w, rank, world)      # this rank's heads of a workload
    sess = Session(shard)
    sharded_step(sess)                          # begin, all-reduce(max) of the flags, end

Marshalling only: the kernels are the library's, the exchange is torch.distributed's (NCCL on GPUs).
"""
from __future__ import annotations

import dataclasses

import torch
import torch.distributed as dist

from .workloads import Workload


def shard_workload(w: Workload, rank: int, world: int) -> Workload:
    """Rank ``rank``'s KV heads (a contiguous block of n_kv_heads / world) with their query heads; every table of
    the clusters and requests is kept whole."""
    cfg = w.cfg
    if cfg.n_kv_heads % world != 0:
        raise ValueError("the KV heads do not divide over the ranks")
    hkv = cfg.n_kv_heads // world
    g = cfg.n_q_heads // cfg.n_kv_heads
    kv0, q0 = rank * hkv, rank * hkv * g
    shard_cfg = dataclasses.replace(cfg, n_q_heads=hkv * g, n_kv_heads=hkv)
    return dataclasses.replace(
        w, cfg=shard_cfg, q=w.q[:, q0:q0 + hkv * g].contiguous(), kv_pool=w.kv_pool[:, kv0:kv0 + hkv].contiguous(),
        centroids=None if w.centroids is None else w.centroids[:, kv0:kv0 + hkv].contiguous())


def exchange_flags(flags: torch.Tensor, group=None) -> torch.Tensor:
    """Element-wise maximum of the ranks' flag arrays, in place (no-op for a single process)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(flags, op=dist.ReduceOp.MAX, group=group)
    return flags


def sharded_step(sess, stream=None, group=None) -> None:
    """One step of a head-sharded session: selection, exchange of the cluster flags, attention + resolution."""
    sess.step_begin(stream)
    if stream is not None:
        with torch.cuda.stream(stream):
            exchange_flags(sess.cluster_flags(), group)
    else:
        exchange_flags(sess.cluster_flags(), group)
    sess.step_end(stream)
