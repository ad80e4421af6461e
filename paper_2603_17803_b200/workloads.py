"""Seeded synthetic workloads for the KVCache retrieval path.

This module only *draws inputs*: key/value pools, queries, page->cluster tables and replica
placements with the shapes and structure of the five benchmark configurations.  It contains
none of the method's arithmetic (no summaries, scores, selection, scheduling or attention),
so both the CUDA library's tests and the CPU oracle's tests can be fed from it.

Small tables are drawn on the host with numpy (identical on every device); the large bf16
pool is drawn with torch on the requested device, so a given (config, seed, device type)
always produces the same bytes.  Whoever needs the data on the other side copies the bytes.

Structure (synthetic stand-in for co-activation, Sec. 3.1): keys of a page are a per-topic
centroid plus noise, pages of one topic form the clusters, and queries point at a topic, so
pages of the same cluster tend to be selected together.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    batch: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    page_size: int
    top_k: int
    n_queues: int
    ctx_len: int = 0                                  # fixed context length (tokens) ...
    ctx_range: Optional[Tuple[int, int]] = None       # ... or uniform integer range [lo, hi]
    head_dim: int = 128
    n_topics: int = 0                                 # 0: iid N(0,1) keys and random clusters
    cluster_pages: int = 8                            # fixed cluster size (pages) ...
    cluster_pages_range: Optional[Tuple[int, int]] = None  # ... or seeded sizes in [lo, hi]
    replication: str = "two"                          # "two" | "half_two" | "hot_three" | "one" | "all"
    zipf_pages: float = 0.0                           # >0: topic of each page ~ Zipf over topic rank
    zipf_query: float = 0.0                           # >0: request topic ~ Zipf over topic rank
    noise: float = 0.3
    stay_prob: float = 0.75                           # a head follows its request's topic with this prob.

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def max_ctx(self) -> int:
        return self.ctx_range[1] if self.ctx_range else self.ctx_len

    def max_pages(self) -> int:
        return -(-self.max_ctx() // self.page_size)


CONFIGS = {
    # Tiny: iid keys, 2048 pages, 256 clusters of 8, D=4, two replicas each.
    "c1_tiny": WorkloadConfig("c1_tiny", batch=1, n_layers=1, n_q_heads=8, n_kv_heads=8, page_size=16, top_k=64,
                              n_queues=4, ctx_len=32768, n_topics=0, replication="two"),
    # Llama-3-8B-shaped layer at 128K: 64 topics x 128 pages, 1024 clusters of 8, D=8.
    "c2_128k": WorkloadConfig("c2_128k", batch=1, n_layers=1, n_q_heads=32, n_kv_heads=8, page_size=16, top_k=256,
                              n_queues=8, ctx_len=131072, n_topics=64, replication="two"),
    # Batched decode: 16 requests x 32 layers, 32 topics, half of the clusters have two replicas.
    "c3_batched": WorkloadConfig("c3_batched", batch=16, n_layers=32, n_q_heads=32, n_kv_heads=8, page_size=16,
                                 top_k=128, n_queues=8, ctx_len=32768, n_topics=32, replication="half_two"),
    # Long context: 512K tokens, page 32, g = 8, Zipf(1.1) topic popularity on the query side.
    "c4_long": WorkloadConfig("c4_long", batch=4, n_layers=1, n_q_heads=64, n_kv_heads=8, page_size=32, top_k=512,
                              n_queues=16, ctx_len=524288, n_topics=128, replication="two", zipf_query=1.1),
    # Skewed serving mix: ragged contexts, clusters of 4..16 pages, hot 10% of clusters on 3 queues.
    "c5_skewed": WorkloadConfig("c5_skewed", batch=64, n_layers=1, n_q_heads=32, n_kv_heads=8, page_size=16,
                                top_k=128, n_queues=12, ctx_range=(4096, 262144), n_topics=64,
                                cluster_pages_range=(4, 16), replication="hot_three", zipf_pages=1.2,
                                zipf_query=1.2),
}


def scaled(cfg: WorkloadConfig, **changes) -> WorkloadConfig:
    """A smaller (or otherwise altered) copy of a configuration, for tests."""
    return dataclasses.replace(cfg, **changes)


@dataclass
class Workload:
    cfg: WorkloadConfig
    seed: int
    q: torch.Tensor                     # bf16 [B][Hq][d]
    kv_pool: torch.Tensor               # bf16 [n_pool_pages][Hkv][2][S][d]   (0 = K, 1 = V)
    page_base: torch.Tensor             # int64 [B+1]
    ctx_len: torch.Tensor               # int32 [B]
    page2cluster: torch.Tensor          # int32 [n_pool_pages], cluster id local to the request
    cluster_base: torch.Tensor          # int64 [B+1]
    cluster_replica_mask: torch.Tensor  # int32 holding uint32 bits, [n_clusters]
    cluster_size: torch.Tensor          # int16 holding uint16 values, [n_clusters]
    topic_of_page: np.ndarray           # int32 [n_pool_pages]  (host; -1 when there are no topics)
    centroids: Optional[torch.Tensor]   # f32 [B][Hkv][n_topics][d] or None

    @property
    def n_pool_pages(self) -> int:
        return int(self.kv_pool.shape[0])

    @property
    def n_clusters(self) -> int:
        return int(self.cluster_size.shape[0])

    def tables_to(self, device) -> "Workload":
        """Same workload with every tensor on ``device``."""
        kw = {f.name: getattr(self, f.name) for f in dataclasses.fields(self)}
        for name, val in kw.items():
            if isinstance(val, torch.Tensor):
                kw[name] = val.to(device)
        return Workload(**kw)


def _rng(seed: int, *tags: int) -> np.random.Generator:
    return np.random.default_rng([int(seed) & 0x7FFFFFFF, *[int(t) & 0x7FFFFFFF for t in tags]])


def _zipf_weights(n: int, a: float) -> np.ndarray:
    w = 1.0 / np.arange(1, n + 1, dtype=np.float64) ** a if a > 0 else np.ones(n, dtype=np.float64)
    return w / w.sum()


def _cut_sizes(n: int, cfg: WorkloadConfig, rng: np.random.Generator) -> np.ndarray:
    """Cut a run of n pages into cluster sizes; a remainder below the minimum joins the previous cluster."""
    sizes = []
    left = n
    if cfg.cluster_pages_range:
        lo, hi = cfg.cluster_pages_range
        while left > 0:
            s = int(rng.integers(lo, hi + 1))
            if s > left:
                s = left
            if s < lo and sizes:
                sizes[-1] += s
            else:
                sizes.append(s)
            left -= s
    else:
        while left > 0:
            s = min(cfg.cluster_pages, left)
            sizes.append(s)
            left -= s
    return np.asarray(sizes, dtype=np.int64)


def _tables_for_request(cfg: WorkloadConfig, P: int, rng: np.random.Generator, cluster_id_offset: int):
    """topic_of_page [P], page2cluster [P] (local ids), cluster_size [C], replica_mask [C]."""
    D = cfg.n_queues
    if cfg.n_topics > 0:
        T = cfg.n_topics
        if cfg.zipf_pages > 0:
            topic = rng.choice(T, size=P, p=_zipf_weights(T, cfg.zipf_pages)).astype(np.int32)
        else:
            perm = rng.permutation(P)
            topic = np.empty(P, dtype=np.int32)
            topic[perm] = (np.arange(P, dtype=np.int64) * T // P).astype(np.int32)
        order = np.lexsort((np.arange(P), topic))        # pages sorted by (topic, id)
        if cfg.cluster_pages_range:
            sizes = _cut_sizes(P, cfg, rng)              # cut the topic-sorted run as one sequence
        else:
            counts = np.bincount(topic, minlength=T)
            sizes = np.concatenate([_cut_sizes(int(c), cfg, rng) for c in counts if c > 0])
    else:
        topic = np.full(P, -1, dtype=np.int32)
        order = rng.permutation(P)
        sizes = _cut_sizes(P, cfg, rng)
    C = len(sizes)
    cluster_of_sorted = np.repeat(np.arange(C, dtype=np.int32), sizes)
    page2cluster = np.empty(P, dtype=np.int32)
    page2cluster[order] = cluster_of_sorted

    # Placement: the primary copy walks round-robin over the queues in cluster order (Eq. 7 with the
    # cluster as placement unit); extra replicas sit on other, seeded queues.
    primary = (cluster_id_offset + np.arange(C)) % D
    n_rep = np.ones(C, dtype=np.int64)
    if cfg.replication == "two":
        n_rep[:] = min(2, D)
    elif cfg.replication == "all":
        n_rep[:] = D
    elif cfg.replication == "half_two":
        chosen = rng.permutation(C)[: C // 2]
        n_rep[chosen] = min(2, D)
    elif cfg.replication == "hot_three":
        start = np.concatenate([[0], np.cumsum(sizes)[:-1]])
        first_topic = topic[order[start]]                # popularity rank = topic index (0 is hottest)
        hot_order = np.lexsort((np.arange(C), first_topic))
        n_rep[hot_order[: max(1, C // 10)]] = min(3, D)
    elif cfg.replication != "one":
        raise ValueError(cfg.replication)
    mask = np.zeros(C, dtype=np.uint32)
    for c in range(C):
        m = 1 << int(primary[c])
        if n_rep[c] > 1:
            others = [x for x in range(D) if x != primary[c]]
            extra = rng.choice(len(others), size=int(n_rep[c]) - 1, replace=False)
            for e in extra:
                m |= 1 << others[int(e)]
        mask[c] = m
    return topic, page2cluster, sizes.astype(np.uint16), mask


def generate(cfg: WorkloadConfig, seed: int = 0, device="cpu", layer: int = 0, step: int = 0,
             poison_tail: bool = True, pages_per_chunk: int = 4096) -> Workload:
    """Draw one layer-step's inputs.  ``layer`` and ``step`` are folded into the seeds of the pool and of the
    query respectively.  Padding tokens of a partial last page are set to large finite constants so that
    any code that fails to mask them is caught."""
    device = torch.device(device)
    B, Hq, Hkv, d, S = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size
    r_len = _rng(seed, 1, layer)
    if cfg.ctx_range:
        ctx = r_len.integers(cfg.ctx_range[0], cfg.ctx_range[1] + 1, size=B).astype(np.int32)
    else:
        ctx = np.full(B, cfg.ctx_len, dtype=np.int32)
    pages = (ctx.astype(np.int64) + S - 1) // S
    page_base = np.concatenate([[0], np.cumsum(pages)]).astype(np.int64)
    n_pool = int(page_base[-1])

    topic_all = np.empty(n_pool, dtype=np.int32)
    p2c_all = np.empty(n_pool, dtype=np.int32)
    sizes_all, mask_all, cluster_base = [], [], [0]
    for b in range(B):
        topic, p2c, sizes, mask = _tables_for_request(cfg, int(pages[b]), _rng(seed, 2, layer, b), cluster_base[-1])
        topic_all[page_base[b]:page_base[b + 1]] = topic
        p2c_all[page_base[b]:page_base[b + 1]] = p2c
        sizes_all.append(sizes)
        mask_all.append(mask)
        cluster_base.append(cluster_base[-1] + len(sizes))
    sizes_all = np.concatenate(sizes_all)
    mask_all = np.concatenate(mask_all)

    gen = torch.Generator(device=device)
    gen.manual_seed((int(seed) * 1000003 + layer * 7919 + 17) & 0x7FFFFFFFFFFF)
    centroids = None
    if cfg.n_topics > 0:
        centroids = torch.randn((B, Hkv, cfg.n_topics, d), generator=gen, device=device, dtype=torch.float32)

    kv_pool = torch.empty((n_pool, Hkv, 2, S, d), dtype=torch.bfloat16, device=device)
    req_of_page = np.repeat(np.arange(B, dtype=np.int64), pages)
    for lo in range(0, n_pool, pages_per_chunk):
        hi = min(n_pool, lo + pages_per_chunk)
        x = torch.randn((hi - lo, Hkv, 2, S, d), generator=gen, device=device, dtype=torch.float32)
        if centroids is not None:
            rb = torch.from_numpy(req_of_page[lo:hi]).to(device)
            tp = torch.from_numpy(topic_all[lo:hi].astype(np.int64)).to(device)
            cen = centroids[rb, :, tp, :]                       # [chunk][Hkv][d]
            x[:, :, 0] = x[:, :, 0] * cfg.noise + cen[:, :, None, :]
        kv_pool[lo:hi] = x.to(torch.bfloat16)
    if poison_tail:
        for b in range(B):
            valid = int(ctx[b]) - S * (int(pages[b]) - 1)
            if valid < S:
                last = int(page_base[b + 1]) - 1
                kv_pool[last, :, 0, valid:, :] = 64.0
                kv_pool[last, :, 1, valid:, :] = -512.0

    # Queries: each request has a topic for this step; each head follows it or wanders.
    gq = torch.Generator(device=device)
    gq.manual_seed((int(seed) * 1000003 + layer * 7919 + step * 104729 + 5) & 0x7FFFFFFFFFFF)
    q = torch.randn((B, Hq, d), generator=gq, device=device, dtype=torch.float32)
    if centroids is not None:
        r_q = _rng(seed, 3, layer, step)
        w = _zipf_weights(cfg.n_topics, cfg.zipf_query)
        req_topic = r_q.choice(cfg.n_topics, size=B, p=w)
        wander = r_q.random((B, Hq)) >= cfg.stay_prob
        other = r_q.choice(cfg.n_topics, size=(B, Hq), p=w)
        head_topic = np.where(wander, other, req_topic[:, None]).astype(np.int64)
        bi = torch.arange(B, device=device)[:, None].expand(B, Hq)
        kvi = (torch.arange(Hq, device=device) // cfg.group)[None, :].expand(B, Hq)
        cen_q = centroids[bi, kvi, torch.from_numpy(head_topic).to(device), :]
        q = q * cfg.noise + cen_q
    q = q.to(torch.bfloat16)

    return Workload(
        cfg=cfg, seed=seed, q=q, kv_pool=kv_pool,
        page_base=torch.from_numpy(page_base).to(device),
        ctx_len=torch.from_numpy(ctx).to(device),
        page2cluster=torch.from_numpy(p2c_all).to(device),
        cluster_base=torch.from_numpy(np.asarray(cluster_base, dtype=np.int64)).to(device),
        cluster_replica_mask=torch.from_numpy(mask_all.view(np.int32)).to(device),
        cluster_size=torch.from_numpy(sizes_all.view(np.int16)).to(device),
        topic_of_page=topic_all, centroids=centroids,
    )


def subset_requests(w: "Workload", requests, device="cpu") -> "Workload":
    """The given requests of a workload as a workload of their own on ``device`` (their pages, cluster tables
    and queries copied and re-based; nothing is redrawn).  Used to hand the CPU oracle a bounded sample of a
    large batch."""
    requests = [int(b) for b in requests]
    page_base = w.page_base.cpu().numpy()
    cluster_base = w.cluster_base.cpu().numpy()
    pool, p2c, sizes, masks, topics = [], [], [], [], []
    pb, cb = [0], [0]
    for b in requests:
        lo, hi = int(page_base[b]), int(page_base[b + 1])
        clo, chi = int(cluster_base[b]), int(cluster_base[b + 1])
        pool.append(w.kv_pool[lo:hi].to(device))
        p2c.append(w.page2cluster[lo:hi].to(device))
        sizes.append(w.cluster_size[clo:chi].to(device))
        masks.append(w.cluster_replica_mask[clo:chi].to(device))
        topics.append(w.topic_of_page[lo:hi])
        pb.append(pb[-1] + hi - lo)
        cb.append(cb[-1] + chi - clo)
    idx = torch.tensor(requests, dtype=torch.long, device=w.q.device)
    cfg = dataclasses.replace(w.cfg, batch=len(requests))
    return Workload(
        cfg=cfg, seed=w.seed, q=w.q[idx].to(device), kv_pool=torch.cat(pool),
        page_base=torch.tensor(pb, dtype=torch.int64, device=device),
        ctx_len=w.ctx_len[idx].to(device), page2cluster=torch.cat(p2c),
        cluster_base=torch.tensor(cb, dtype=torch.int64, device=device),
        cluster_replica_mask=torch.cat(masks), cluster_size=torch.cat(sizes),
        topic_of_page=np.concatenate(topics),
        centroids=None if w.centroids is None else w.centroids[idx].to(device),
    )


def bits_u16(t: torch.Tensor) -> np.ndarray:
    """Raw bits of a bf16 (or 16-bit integer) tensor as a host uint16 array (the form the oracle takes)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def cluster_members(w: "Workload"):
    """Member lists of the clusters, derived from the page -> cluster table, and one medoid page per cluster.

    Returns (cluster_page_ptr int64 [C + 1], cluster_pages int32 [pages], medoid_page int32 [C]) on the workload's
    device: members in ascending page id (local to the request), clusters by global id.  The medoid is the middle
    member -- which member represents a cluster is decided by the offline clustering, which is not modelled here.
    """
    p2c = w.page2cluster.cpu().numpy()
    page_base = w.page_base.cpu().numpy()
    cluster_base = w.cluster_base.cpu().numpy()
    ctx = w.ctx_len.cpu().numpy()
    C = int(cluster_base[-1])
    S = w.cfg.page_size
    counts = np.zeros(C, dtype=np.int64)
    members = []
    for b in range(len(ctx)):
        P = -(-int(ctx[b]) // S)
        local = p2c[page_base[b]:page_base[b] + P].astype(np.int64)
        order = np.argsort(local, kind="stable")            # pages grouped by cluster, ascending page id inside
        members.append(order.astype(np.int32))
        counts[cluster_base[b]:cluster_base[b + 1]] = np.bincount(local, minlength=int(cluster_base[b + 1] - cluster_base[b]))
    ptr = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    pages = np.concatenate(members) if members else np.zeros(0, np.int32)
    medoid = np.where(counts > 0, pages[np.minimum(ptr[:-1] + counts // 2, max(len(pages) - 1, 0))], 0).astype(np.int32)
    dev = w.page2cluster.device
    return (torch.from_numpy(ptr).to(dev), torch.from_numpy(pages).to(dev), torch.from_numpy(medoid).to(dev))


def coactivation_distances(n: int, n_topics: int, seed: int, device="cpu", noise: float = 0.15,
                           bridge_frac: float = 0.1) -> torch.Tensor:
    """Synthetic distance matrix d = 1 - P for Algorithm 1: entries of one latent topic are co-activated with high
    probability (small distance), entries of different topics rarely; a fraction of "bridge" entries is also close
    to a second topic, which is what makes an entry join several clusters.  Symmetric, zero diagonal, float32 in
    [0, 1].  Stands in for the co-activation profile the paper measures on real models."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    topic = torch.randint(0, n_topics, (n,), generator=g)
    second = torch.where(torch.rand(n, generator=g) < bridge_frac, torch.randint(0, n_topics, (n,), generator=g), topic)
    same = (topic[:, None] == topic[None, :]) | (second[:, None] == topic[None, :]) | (topic[:, None] == second[None, :])
    base = torch.where(same, torch.tensor(0.25), torch.tensor(0.85))
    jitter = (torch.rand((n, n), generator=g) - 0.5) * 2.0 * noise
    d = (base + jitter).clamp_(0.0, 1.0)
    d = torch.minimum(d, d.T).contiguous()
    d.fill_diagonal_(0.0)
    return d.to(torch.float32).to(device)
