"""Convenience wrapper: owns a swarm ctx, its workspace and output tensors for one set of device inputs.

Allocation and marshalling only (torch supplies device memory and streams); all computing is done by
the library's kernels through ``binding``.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import torch

from . import binding as B


@dataclass
class StepOutputs:
    scores: Optional[torch.Tensor]
    sel: torch.Tensor
    n_sel: torch.Tensor
    uniq: torch.Tensor
    queue_of: torch.Tensor
    n_uniq: torch.Tensor
    queue_load: torch.Tensor
    k_out: Optional[torch.Tensor]
    v_out: Optional[torch.Tensor]
    n_tok: Optional[torch.Tensor]
    out: torch.Tensor
    lse: torch.Tensor


class Session:
    """One ctx bound to one resident KV pool (``workload`` tensors must live on a CUDA device)."""

    def __init__(self, workload, *, flags: int = 0, keep_scores: bool = False, keep_gathered: bool = False,
                 ksum: Optional[torch.Tensor] = None, local_window_pages: int = 0,
                 max_clusters_total: Optional[int] = None, scorer: int = B.SCORER_AUTO, tail_stream=None,
                 index_prefetch: bool = False):
        cfg = workload.cfg
        self.cfg = cfg
        self.w = workload
        dev = workload.kv_pool.device
        if dev.type != "cuda":
            raise ValueError("Session needs the workload on a CUDA device")
        self.device = dev
        self.Pmax = cfg.max_pages()
        self.shape = B.make_shape(batch=cfg.batch, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                                  page_size=cfg.page_size, top_k=cfg.top_k, n_queues=cfg.n_queues,
                                  max_pages_per_req=self.Pmax, max_clusters_total=max(1, workload.n_clusters, max_clusters_total or 0),
                                  n_pool_pages=workload.n_pool_pages, flags=flags,
                                  local_window_pages=local_window_pages)
        self.ctx = B.swarm_create(self.shape)
        self.workspace = torch.empty(B.swarm_workspace_bytes(self.shape), dtype=torch.uint8, device=dev)
        B.swarm_set_workspace(self.ctx, self.workspace)
        if scorer != B.SCORER_AUTO:
            B.swarm_set_scorer(self.ctx, scorer)
        if index_prefetch:                       # the workload's index and lengths are written once, before any step
            B.swarm_set_index_prefetch(self.ctx, True)
        self.tail_stream = tail_stream
        if tail_stream is not None:
            B.swarm_set_tail_stream(self.ctx, tail_stream)
        self.ksum = ksum if ksum is not None else torch.empty(
            (workload.n_pool_pages, cfg.n_kv_heads, 2, cfg.head_dim), dtype=torch.bfloat16, device=dev)
        self.inputs = self._inputs(workload.q)
        if ksum is None:
            B.swarm_build_summaries(self.ctx, self.inputs, self.ksum)
        Bq, Hq, k, S, d = cfg.batch, cfg.n_q_heads, cfg.top_k, cfg.page_size, cfg.head_dim
        i32 = dict(dtype=torch.int32, device=dev)
        self.o = StepOutputs(
            scores=torch.full((Bq, Hq, self.Pmax), float("-inf"), dtype=torch.float32, device=dev) if keep_scores else None,
            sel=torch.empty((Bq, Hq, k), **i32), n_sel=torch.empty((Bq, Hq), **i32),
            uniq=torch.empty(max(1, workload.n_clusters, max_clusters_total or 0), **i32),
            queue_of=torch.empty(max(16, workload.n_clusters, max_clusters_total or 0), dtype=torch.uint8, device=dev),
            n_uniq=torch.zeros(4, **i32), queue_load=torch.zeros(max(4, cfg.n_queues), **i32),
            k_out=torch.empty((Bq, Hq, k * S, d), dtype=torch.bfloat16, device=dev) if keep_gathered else None,
            v_out=torch.empty((Bq, Hq, k * S, d), dtype=torch.bfloat16, device=dev) if keep_gathered else None,
            n_tok=torch.empty((Bq, Hq), **i32) if keep_gathered else None,
            out=torch.empty((Bq, Hq, d), dtype=torch.float32, device=dev),
            lse=torch.empty((Bq, Hq), dtype=torch.float32, device=dev),
        )
        self.outputs = B.make_outputs(**{k_: getattr(self.o, k_) for k_ in self.o.__dataclass_fields__})

    def _inputs(self, q):
        w = self.w
        return B.make_inputs(q=q, ksum=self.ksum, kv_pool=w.kv_pool, page_base=w.page_base, ctx_len=w.ctx_len,
                             page2cluster=w.page2cluster, cluster_base=w.cluster_base,
                             cluster_replica_mask=w.cluster_replica_mask, cluster_size=w.cluster_size)

    def set_query(self, q: torch.Tensor) -> None:
        self._q = q
        self.inputs = self._inputs(q)

    # -- the five calls ---------------------------------------------------------------------------
    def select(self, stream=None):
        B.swarm_select(self.ctx, self.inputs, self.o.scores, self.o.sel, self.o.n_sel, stream)

    def resolve(self, sel=None, n_sel=None, stream=None):
        B.swarm_resolve_clusters(self.ctx, self.inputs, self.o.sel if sel is None else sel,
                                 self.o.n_sel if n_sel is None else n_sel, self.o.uniq, self.o.queue_of,
                                 self.o.n_uniq, self.o.queue_load, stream)

    def gather(self, sel=None, n_sel=None, stream=None):
        if self.o.k_out is None:
            raise ValueError("Session was created with keep_gathered=False")
        B.swarm_gather(self.ctx, self.inputs, self.o.sel if sel is None else sel,
                       self.o.n_sel if n_sel is None else n_sel, self.o.k_out, self.o.v_out, self.o.n_tok, stream)

    def sparse_attn(self, stream=None):
        B.swarm_sparse_attn(self.ctx, self.w.q if not hasattr(self, "_q") else self._q, self.o.k_out, self.o.v_out,
                            self.o.n_tok, self.o.out, self.o.lse, stream)

    def sparse_attn_paged(self, stream=None, reuse_last_selection=False):
        sel, n_sel = (None, None) if reuse_last_selection else (self.o.sel, self.o.n_sel)
        B.swarm_sparse_attn_paged(self.ctx, self.inputs, sel, n_sel, self.o.out, self.o.lse, stream)

    def step(self, stream=None):
        B.swarm_step(self.ctx, self.inputs, self.outputs, stream)

    def tail_join(self, stream=None):
        """Make `stream` wait for the cluster resolution of the last step (only needed with a tail stream)."""
        B.swarm_tail_join(self.ctx, stream)

    # -- the step in two halves (query heads spread over several ctxs) --------------------------------
    def step_begin(self, stream=None):
        B.swarm_step_begin(self.ctx, self.inputs, self.outputs, stream)

    def step_end(self, stream=None):
        B.swarm_step_end(self.ctx, self.inputs, self.outputs, stream)

    def cluster_flags(self) -> torch.Tensor:
        """The ctx's cluster flag array as a uint8 view of the workspace (what the ranks combine by maximum)."""
        addr, n = B.swarm_cluster_flags(self.ctx)
        off = addr - self.workspace.data_ptr()
        if off < 0 or off + n > self.workspace.numel():
            raise RuntimeError("cluster flags outside the workspace")
        return self.workspace[off:off + n]

    def step_host(self, q_host, out_host=None, lse_host=None, n_uniq_host=None, queue_load_host=None, stream=None):
        """swarm_step_host.  The call is synchronous and tens of microseconds long, so the marshalled arguments of
        the last call are kept and reused while the same tensor objects (and stream) are passed again; buffers
        must not be resized in place between calls."""
        if stream is None:                                  # the current stream may differ from call to call
            B.swarm_step_host(self.ctx, self.inputs, self.outputs, q_host, out_host, lse_host, n_uniq_host,
                              queue_load_host, None)
            return
        key = (id(q_host), id(out_host), id(lse_host), id(n_uniq_host), id(queue_load_host), id(stream), id(self.inputs))
        call = getattr(self, "_host_call", None)
        if call is None or call[0] != key:
            keep = (q_host, out_host, lse_host, n_uniq_host, queue_load_host, stream, self.inputs)   # ids stay unique while held
            call = (key, B.marshal_step_host(self.ctx, self.inputs, self.outputs, q_host, out_host, lse_host,
                                             n_uniq_host, queue_load_host, stream), keep)
            self._host_call = call
        B.swarm_step_host_marshalled(self.ctx, call[1])

    def enable_medoid_index(self, top_k_clusters: int, keep_scores: bool = False) -> None:
        """Builds the medoid index of the workload's clusters and the outputs of step_medoid()."""
        from .workloads import cluster_members
        w, cfg, dev = self.w, self.cfg, self.device
        self.cluster_page_ptr, self.cluster_pages, self.medoid_page = cluster_members(w)
        n_c = max(1, w.n_clusters)
        per_req = (w.cluster_base[1:] - w.cluster_base[:-1]).max().item()
        self.max_clusters_per_req = max(1, int(per_req))
        self.medoid_ksum = torch.empty((n_c, cfg.n_kv_heads, 2, cfg.head_dim), dtype=torch.bfloat16, device=dev)
        self.cluster_ctx_len = torch.empty(max(4, cfg.batch), dtype=torch.int32, device=dev)
        B.swarm_build_medoid_index(self.ctx, self.inputs, self.medoid_page, self.medoid_ksum, self.cluster_ctx_len)
        self.medoid_index = B.make_medoid_index(medoid_ksum=self.medoid_ksum, cluster_page_ptr=self.cluster_page_ptr,
                                                cluster_pages=self.cluster_pages, cluster_ctx_len=self.cluster_ctx_len,
                                                top_k_clusters=top_k_clusters,
                                                max_clusters_per_req=self.max_clusters_per_req)
        i32 = dict(dtype=torch.int32, device=dev)
        self.top_k_clusters = top_k_clusters
        self.sel_clusters = torch.empty((cfg.batch, cfg.n_q_heads, top_k_clusters), **i32)
        self.n_sel_clusters = torch.empty((cfg.batch, cfg.n_q_heads), **i32)
        self.cluster_scores = torch.full((cfg.batch, cfg.n_q_heads, self.max_clusters_per_req), float("-inf"),
                                         dtype=torch.float32, device=dev) if keep_scores else None
        o = self.o
        self.medoid_outputs = B.make_outputs(scores=self.cluster_scores, sel=self.sel_clusters,
                                             n_sel=self.n_sel_clusters, uniq=o.uniq, queue_of=o.queue_of,
                                             n_uniq=o.n_uniq, queue_load=o.queue_load, out=o.out, lse=o.lse)

    def enable_submit_order(self) -> None:
        """Attaches the outputs of the batched submission order (indices into uniq, and [batches, submitted])."""
        i32 = dict(dtype=torch.int32, device=self.device)
        self.submit_order = torch.full((max(4, self.o.uniq.numel()),), -1, **i32)
        self.submit_info = torch.zeros(4, **i32)
        B.swarm_set_submit_order(self.ctx, self.submit_order, self.submit_info)

    def step_medoid(self, stream=None):
        B.swarm_step_medoid(self.ctx, self.inputs, self.medoid_index, self.medoid_outputs, stream)

    def status(self) -> int:
        return B.swarm_device_status(self.ctx)

    def close(self):
        """Destroys the ctx.  Before that, checks the canaries between the workspace regions: a kernel that wrote
        outside its region is reported here (every test closes its sessions)."""
        if self.ctx is not None:
            torch.cuda.synchronize(self.device)
            damaged = B.swarm_check_workspace(self.ctx)
            B.swarm_destroy(self.ctx)
            self.ctx = None
            if damaged:
                raise RuntimeError(f"workspace canaries overwritten: mask {damaged:#x}")

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
