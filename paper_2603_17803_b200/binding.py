"""ctypes binding of libswarm.so: the same entry points as ``include/swarm.h``, taking torch tensors.

Argument marshalling only -- every step of the path runs in the CUDA kernels of the library.
There is no CPU fallback: if the library has not been built, or a call fails, an exception is raised.
torch is used for device memory and streams, nothing else.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libswarm.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA = 0, 1, 2, 3, 4
ERR_STATIC_SCRATCH_TOO_SMALL = 5
STATIC_MAX_HEADS = 2048
DEV_BAD_PAGE, DEV_BAD_CLUSTER, DEV_BAD_REPLICA, DEV_BAD_LENGTH, DEV_TIMEOUT = 1, 2, 4, 8, 16
ORDER_BY_ID, UNIT_LOAD = 1, 2
SCORER_AUTO, SCORER_TENSOR, SCORER_FP32 = 0, 1, 2
_ERR_NAMES = {1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "WORKSPACE_TOO_SMALL", 4: "CUDA",
              5: "STATIC_SCRATCH_TOO_SMALL"}

EXPORTS = (
    "swarm_version", "swarm_create", "swarm_destroy", "swarm_workspace_bytes", "swarm_set_workspace",
    "swarm_check_workspace", "swarm_set_attn_splits", "swarm_set_scorer", "swarm_set_index_prefetch", "swarm_set_tail_stream", "swarm_tail_join", "swarm_set_select_sms", "swarm_set_cache", "swarm_build_summaries", "swarm_select", "swarm_resolve_clusters", "swarm_gather",
    "swarm_sparse_attn", "swarm_sparse_attn_paged", "swarm_sparse_attn_static", "swarm_sparse_attn_static_status", "swarm_step", "swarm_step_host", "swarm_device_status", "swarm_last_cuda_error",
    "swarm_build_medoid_index", "swarm_step_medoid", "swarm_set_submit_order",
    "swarm_build_clusters_workspace_bytes", "swarm_build_clusters",
    "swarm_cache_admit_workspace_bytes", "swarm_cache_admit",
    "swarm_step_begin", "swarm_step_end", "swarm_cluster_flags",
)


class SwarmError(RuntimeError):
    def __init__(self, code: int, what: str, cuda_error: int = 0):
        self.code = code
        self.cuda_error = cuda_error
        extra = f" (cudaError {cuda_error})" if cuda_error else ""
        super().__init__(f"{what}: SWARM_ERR_{_ERR_NAMES.get(code, code)}{extra}")


class swarm_shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("batch", "n_q_heads", "n_kv_heads", "head_dim", "page_size", "top_k",
                                              "n_queues", "max_pages_per_req", "max_clusters_total")] + \
               [("flags", ctypes.c_uint32), ("n_pool_pages", ctypes.c_int64),
                ("local_window_pages", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class swarm_inputs(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("q", "ksum", "kv_pool", "page_base", "ctx_len", "page2cluster",
                                               "cluster_base", "cluster_replica_mask", "cluster_size")]


class swarm_outputs(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("scores", "sel", "n_sel", "uniq", "queue_of", "n_uniq", "queue_load",
                                               "k_out", "v_out", "n_tok", "out", "lse")]


class swarm_cache(ctypes.Structure):
    _fields_ = [("resident", ctypes.c_void_p), ("freq", ctypes.c_void_p), ("score", ctypes.c_void_p),
                ("n_hit", ctypes.c_void_p), ("t_base", ctypes.c_float), ("t_transfer", ctypes.c_float)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libswarm.so from the package directory; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2603_17803_b200.build` "
                               "(there is no fallback implementation)")
        lib = ctypes.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(lib, name).restype = ctypes.c_int32
        lib.swarm_workspace_bytes.restype = ctypes.c_int64
        lib.swarm_build_clusters_workspace_bytes.restype = ctypes.c_int64
        lib.swarm_cache_admit_workspace_bytes.restype = ctypes.c_int64
        _lib = lib
    return _lib


def _ptr(t: Optional[torch.Tensor], name: str = "tensor", device_check: bool = True):
    if t is None:
        return None
    if device_check and not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(rc: int, what: str, ctx=None):
    if rc != OK:
        cuda = load_library().swarm_last_cuda_error(ctx) if (ctx is not None and rc == ERR_CUDA) else 0
        raise SwarmError(rc, what, cuda)


class swarm_medoid_index(ctypes.Structure):
    _fields_ = [("medoid_ksum", ctypes.c_void_p), ("cluster_page_ptr", ctypes.c_void_p),
                ("cluster_pages", ctypes.c_void_p), ("entry_replica_mask", ctypes.c_void_p),
                ("cluster_ctx_len", ctypes.c_void_p), ("n_member_entries", ctypes.c_int64), ("top_k_clusters", ctypes.c_int32),
                ("max_clusters_per_req", ctypes.c_int32)]


def make_shape(*, batch, n_q_heads, n_kv_heads, page_size, top_k, n_queues, max_pages_per_req, max_clusters_total,
               n_pool_pages, head_dim=128, flags=0, local_window_pages=0) -> swarm_shape:
    return swarm_shape(batch, n_q_heads, n_kv_heads, head_dim, page_size, top_k, n_queues, max_pages_per_req,
                       max_clusters_total, flags, n_pool_pages, local_window_pages, 0)


def make_inputs(*, q=None, ksum=None, kv_pool=None, page_base=None, ctx_len=None, page2cluster=None,
                cluster_base=None, cluster_replica_mask=None, cluster_size=None) -> swarm_inputs:
    """Struct of device pointers.  The caller keeps the tensors alive while the struct is in use."""
    return swarm_inputs(*[_ptr(t, n) for n, t in (("q", q), ("ksum", ksum), ("kv_pool", kv_pool),
                                                  ("page_base", page_base), ("ctx_len", ctx_len),
                                                  ("page2cluster", page2cluster), ("cluster_base", cluster_base),
                                                  ("cluster_replica_mask", cluster_replica_mask),
                                                  ("cluster_size", cluster_size))])


def make_outputs(*, scores=None, sel=None, n_sel=None, uniq=None, queue_of=None, n_uniq=None, queue_load=None,
                 k_out=None, v_out=None, n_tok=None, out=None, lse=None) -> swarm_outputs:
    return swarm_outputs(*[_ptr(t, n) for n, t in (("scores", scores), ("sel", sel), ("n_sel", n_sel),
                                                   ("uniq", uniq), ("queue_of", queue_of), ("n_uniq", n_uniq),
                                                   ("queue_load", queue_load), ("k_out", k_out), ("v_out", v_out),
                                                   ("n_tok", n_tok), ("out", out), ("lse", lse))])


def swarm_version() -> int:
    return int(load_library().swarm_version())


def swarm_workspace_bytes(shape: swarm_shape) -> int:
    n = int(load_library().swarm_workspace_bytes(ctypes.byref(shape)))
    if n < 0:
        raise SwarmError(-n, "swarm_workspace_bytes")
    return n


def swarm_create(shape: swarm_shape) -> ctypes.c_void_p:
    ctx = ctypes.c_void_p()
    _check(load_library().swarm_create(ctypes.byref(shape), ctypes.byref(ctx)), "swarm_create")
    return ctx


def swarm_destroy(ctx) -> None:
    _check(load_library().swarm_destroy(ctx), "swarm_destroy")


def swarm_set_workspace(ctx, workspace: torch.Tensor, stream=None) -> None:
    _check(load_library().swarm_set_workspace(ctx, _ptr(workspace, "workspace"),
                                              ctypes.c_int64(workspace.numel() * workspace.element_size()),
                                              _stream(stream)), "swarm_set_workspace", ctx)


def swarm_check_workspace(ctx, stream=None) -> int:
    """Bit mask of the workspace canaries that were overwritten (0 = intact); synchronises the stream."""
    bits = ctypes.c_uint32(0)
    _check(load_library().swarm_check_workspace(ctx, _stream(stream), ctypes.byref(bits)), "swarm_check_workspace", ctx)
    return int(bits.value)


def swarm_set_attn_splits(ctx, n_splits: int) -> None:
    _check(load_library().swarm_set_attn_splits(ctx, ctypes.c_int32(n_splits)), "swarm_set_attn_splits", ctx)


def swarm_set_tail_stream(ctx, tail_stream) -> None:
    """Attach a torch.cuda.Stream on which swarm_step enqueues cluster resolution (None detaches)."""
    ptr = ctypes.c_void_p(tail_stream.cuda_stream) if tail_stream is not None else None
    _check(load_library().swarm_set_tail_stream(ctx, ptr), "swarm_set_tail_stream", ctx)


def swarm_tail_join(ctx, stream=None) -> None:
    _check(load_library().swarm_tail_join(ctx, _stream(stream)), "swarm_tail_join", ctx)


def swarm_set_select_sms(ctx, n_sms: int) -> None:
    _check(load_library().swarm_set_select_sms(ctx, ctypes.c_int32(n_sms)), "swarm_set_select_sms", ctx)


def swarm_set_scorer(ctx, kind: int) -> None:
    _check(load_library().swarm_set_scorer(ctx, ctypes.c_int32(kind)), "swarm_set_scorer", ctx)


def swarm_set_index_prefetch(ctx, on: bool) -> None:
    _check(load_library().swarm_set_index_prefetch(ctx, ctypes.c_int32(1 if on else 0)), "swarm_set_index_prefetch", ctx)


def swarm_set_cache(ctx, *, resident=None, freq=None, score=None, n_hit=None, t_base=0.0, t_transfer=0.0) -> None:
    """Attach cache state (uint8 resident, int32 freq, optional float32 score, optional int32 n_hit), or detach it
    when ``resident`` is None.  The caller keeps the tensors alive while they are attached."""
    if resident is None:
        _check(load_library().swarm_set_cache(ctx, None), "swarm_set_cache", ctx)
        return
    c = swarm_cache(_ptr(resident, "resident"), _ptr(freq, "freq"), _ptr(score, "score"), _ptr(n_hit, "n_hit"),
                    float(t_base), float(t_transfer))
    _check(load_library().swarm_set_cache(ctx, ctypes.byref(c)), "swarm_set_cache", ctx)


def swarm_cache_admit_workspace_bytes(n_clusters: int) -> int:
    n = int(load_library().swarm_cache_admit_workspace_bytes(ctypes.c_int32(n_clusters)))
    if n < 0:
        raise SwarmError(-n, "swarm_cache_admit_workspace_bytes")
    return n


def swarm_cache_admit(score: torch.Tensor, cluster_size: torch.Tensor, capacity_pages: int, resident: torch.Tensor,
                      info: Optional[torch.Tensor] = None, stream=None) -> None:
    """resident[c] = 1 for the clusters the fast tier holds: descending score while their sizes fit the capacity."""
    n = int(score.numel())
    ws = torch.empty(swarm_cache_admit_workspace_bytes(n), dtype=torch.uint8, device=score.device)
    _check(load_library().swarm_cache_admit(_ptr(score, "score"), _ptr(cluster_size, "cluster_size"), ctypes.c_int32(n),
                                            ctypes.c_int64(capacity_pages), _ptr(ws), ctypes.c_int64(ws.numel()),
                                            _ptr(resident, "resident"), _ptr(info, "info"), _stream(stream)),
           "swarm_cache_admit")
    if stream is None:
        torch.cuda.current_stream(score.device).synchronize()     # the scratch is freed when this returns


def swarm_build_clusters_workspace_bytes(n_entries: int) -> int:
    n = int(load_library().swarm_build_clusters_workspace_bytes(ctypes.c_int32(n_entries)))
    if n < 0:
        raise SwarmError(-n, "swarm_build_clusters_workspace_bytes")
    return n


def swarm_build_clusters(dist: torch.Tensor, tau: float, members_cap: Optional[int] = None, stream=None):
    """Algorithm 1 on a float32 [n][n] CUDA distance matrix.  Returns (density, cluster_ptr, cluster_members,
    medoid) as int32 CUDA tensors trimmed to the clusters found; raises if members_cap was too small."""
    n = int(dist.shape[0])
    if dist.dtype != torch.float32 or dist.dim() != 2 or dist.shape[1] != n:
        raise ValueError("dist must be a float32 [n][n] tensor")
    lib = load_library()
    ws_bytes = swarm_build_clusters_workspace_bytes(n)
    dev = dist.device
    cap = int(members_cap if members_cap is not None else 16 * n)
    i32 = dict(dtype=torch.int32, device=dev)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    density, ptr, medoid = torch.empty(n, **i32), torch.empty(n + 4, **i32), torch.empty(n, **i32)
    members, info = torch.empty(max(cap, 4), **i32), torch.zeros(8, **i32)
    _check(lib.swarm_build_clusters(_ptr(dist, "dist"), ctypes.c_int32(n), ctypes.c_float(tau), _ptr(ws),
                                    ctypes.c_int64(ws_bytes), _ptr(density), _ptr(ptr), _ptr(members),
                                    ctypes.c_int64(cap), _ptr(medoid), _ptr(info[0:4]), _ptr(info[4:8]),
                                    _stream(stream)), "swarm_build_clusters")
    n_clusters, status = int(info[0]), int(info[4])
    if status != 0:
        raise SwarmError(ERR_WORKSPACE_TOO_SMALL, "swarm_build_clusters (members_cap)")
    return density, ptr[: n_clusters + 1], members[: int(ptr[n_clusters])], medoid[:n_clusters]


def swarm_set_submit_order(ctx, submit_order=None, submit_info=None) -> None:
    """Attach int32 device tensors for the batched submission order (or detach with None)."""
    _check(load_library().swarm_set_submit_order(ctx, _ptr(submit_order, "submit_order"),
                                                 _ptr(submit_info, "submit_info")), "swarm_set_submit_order", ctx)


def swarm_build_summaries(ctx, inputs: swarm_inputs, ksum_out: torch.Tensor, stream=None) -> None:
    _check(load_library().swarm_build_summaries(ctx, ctypes.byref(inputs), _ptr(ksum_out, "ksum_out"),
                                                _stream(stream)), "swarm_build_summaries", ctx)


def swarm_select(ctx, inputs: swarm_inputs, scores, sel, n_sel, stream=None) -> None:
    _check(load_library().swarm_select(ctx, ctypes.byref(inputs), _ptr(scores, "scores"), _ptr(sel, "sel"),
                                       _ptr(n_sel, "n_sel"), _stream(stream)), "swarm_select", ctx)


def swarm_resolve_clusters(ctx, inputs: swarm_inputs, sel, n_sel, uniq, queue_of, n_uniq, queue_load,
                           stream=None) -> None:
    _check(load_library().swarm_resolve_clusters(ctx, ctypes.byref(inputs), _ptr(sel, "sel"), _ptr(n_sel, "n_sel"),
                                                 _ptr(uniq, "uniq"), _ptr(queue_of, "queue_of"),
                                                 _ptr(n_uniq, "n_uniq"), _ptr(queue_load, "queue_load"),
                                                 _stream(stream)), "swarm_resolve_clusters", ctx)


def swarm_gather(ctx, inputs: swarm_inputs, sel, n_sel, k_out, v_out, n_tok, stream=None) -> None:
    _check(load_library().swarm_gather(ctx, ctypes.byref(inputs), _ptr(sel, "sel"), _ptr(n_sel, "n_sel"),
                                       _ptr(k_out, "k_out"), _ptr(v_out, "v_out"), _ptr(n_tok, "n_tok"),
                                       _stream(stream)), "swarm_gather", ctx)


def swarm_sparse_attn(ctx, q, k_g, v_g, n_tok, out, lse, stream=None) -> None:
    _check(load_library().swarm_sparse_attn(ctx, _ptr(q, "q"), _ptr(k_g, "k_g"), _ptr(v_g, "v_g"),
                                            _ptr(n_tok, "n_tok"), _ptr(out, "out"), _ptr(lse, "lse"),
                                            _stream(stream)), "swarm_sparse_attn", ctx)


def swarm_sparse_attn_paged(ctx, inputs: swarm_inputs, sel, n_sel, out, lse, stream=None) -> None:
    _check(load_library().swarm_sparse_attn_paged(ctx, ctypes.byref(inputs), _ptr(sel, "sel"), _ptr(n_sel, "n_sel"),
                                                  _ptr(out, "out"), _ptr(lse, "lse"), _stream(stream)),
           "swarm_sparse_attn_paged", ctx)


def swarm_sparse_attn_static(q, k_g, v_g, n_tok, *, batch, n_q_heads, top_k, page_size, out, lse, stream=None) -> None:
    """swarm_sparse_attn without ctx or workspace, for callers that may not allocate device memory (a plugin
    inside another framework's allocator, a fixed memory budget): the split-K scratch is a fixed array inside
    the library.  At most STATIC_MAX_HEADS (batch * n_q_heads) heads; calls that overlap on the GPU race on
    that array; make the first call on a device outside stream capture."""
    _check(load_library().swarm_sparse_attn_static(_ptr(q, "q"), _ptr(k_g, "k_g"), _ptr(v_g, "v_g"),
                                                   _ptr(n_tok, "n_tok"), ctypes.c_int32(batch),
                                                   ctypes.c_int32(n_q_heads), ctypes.c_int32(top_k),
                                                   ctypes.c_int32(page_size), _ptr(out, "out"), _ptr(lse, "lse"),
                                                   _stream(stream)), "swarm_sparse_attn_static")


def swarm_sparse_attn_static_status(stream=None) -> int:
    """Reads and clears the device status word of swarm_sparse_attn_static (synchronises the stream)."""
    bits = ctypes.c_uint32(0)
    _check(load_library().swarm_sparse_attn_static_status(_stream(stream), ctypes.byref(bits)),
           "swarm_sparse_attn_static_status")
    return int(bits.value)


def swarm_step(ctx, inputs: swarm_inputs, outputs: swarm_outputs, stream=None) -> None:
    _check(load_library().swarm_step(ctx, ctypes.byref(inputs), ctypes.byref(outputs), _stream(stream)),
           "swarm_step", ctx)


def swarm_step_begin(ctx, inputs: swarm_inputs, outputs: swarm_outputs, stream=None) -> None:
    _check(load_library().swarm_step_begin(ctx, ctypes.byref(inputs), ctypes.byref(outputs), _stream(stream)),
           "swarm_step_begin", ctx)


def swarm_step_end(ctx, inputs: swarm_inputs, outputs: swarm_outputs, stream=None) -> None:
    _check(load_library().swarm_step_end(ctx, ctypes.byref(inputs), ctypes.byref(outputs), _stream(stream)),
           "swarm_step_end", ctx)


def swarm_cluster_flags(ctx):
    """(device address, number of bytes) of the ctx's cluster flag array."""
    ptr, n = ctypes.c_void_p(0), ctypes.c_int64(0)
    _check(load_library().swarm_cluster_flags(ctx, ctypes.byref(ptr), ctypes.byref(n)), "swarm_cluster_flags", ctx)
    return int(ptr.value or 0), int(n.value)


def make_medoid_index(*, medoid_ksum, cluster_page_ptr, cluster_pages, cluster_ctx_len, top_k_clusters,
                      max_clusters_per_req, entry_replica_mask=None) -> swarm_medoid_index:
    return swarm_medoid_index(_ptr(medoid_ksum, "medoid_ksum"), _ptr(cluster_page_ptr, "cluster_page_ptr"),
                              _ptr(cluster_pages, "cluster_pages"), _ptr(entry_replica_mask, "entry_replica_mask"),
                              _ptr(cluster_ctx_len, "cluster_ctx_len"), int(cluster_pages.numel()), top_k_clusters, max_clusters_per_req)


def swarm_build_medoid_index(ctx, inputs: swarm_inputs, medoid_page: torch.Tensor, medoid_ksum_out: torch.Tensor,
                             cluster_ctx_len_out: torch.Tensor, stream=None) -> None:
    _check(load_library().swarm_build_medoid_index(ctx, ctypes.byref(inputs), _ptr(medoid_page, "medoid_page"),
                                                   _ptr(medoid_ksum_out, "medoid_ksum_out"),
                                                   _ptr(cluster_ctx_len_out, "cluster_ctx_len_out"), _stream(stream)),
           "swarm_build_medoid_index", ctx)


def swarm_step_medoid(ctx, inputs: swarm_inputs, index: swarm_medoid_index, outputs: swarm_outputs,
                      stream=None) -> None:
    _check(load_library().swarm_step_medoid(ctx, ctypes.byref(inputs), ctypes.byref(index), ctypes.byref(outputs),
                                            _stream(stream)), "swarm_step_medoid", ctx)


def swarm_step_host(ctx, inputs: swarm_inputs, outputs: swarm_outputs, q_host, out_host=None, lse_host=None,
                    n_uniq_host=None, queue_load_host=None, stream=None) -> None:
    """Host tensors (pinned recommended) for the per-step data; blocks until the step has finished."""
    _check(load_library().swarm_step_host(ctx, ctypes.byref(inputs), ctypes.byref(outputs),
                                          _ptr(q_host, "q_host", False), _ptr(out_host, "out_host", False),
                                          _ptr(lse_host, "lse_host", False), _ptr(n_uniq_host, "n_uniq_host", False),
                                          _ptr(queue_load_host, "queue_load_host", False), _stream(stream)),
           "swarm_step_host", ctx)


def marshal_step_host(ctx, inputs: swarm_inputs, outputs: swarm_outputs, q_host, out_host=None, lse_host=None,
                      n_uniq_host=None, queue_load_host=None, stream=None) -> tuple:
    """The C arguments of swarm_step_host for these tensors, for callers that repeat the call with the same ones
    (the structures and tensors must stay alive and in place while the tuple is used)."""
    return (ctx, ctypes.byref(inputs), ctypes.byref(outputs), _ptr(q_host, "q_host", False),
            _ptr(out_host, "out_host", False), _ptr(lse_host, "lse_host", False),
            _ptr(n_uniq_host, "n_uniq_host", False), _ptr(queue_load_host, "queue_load_host", False), _stream(stream))


def swarm_step_host_marshalled(ctx, args: tuple) -> None:
    """swarm_step_host with arguments prepared by marshal_step_host."""
    rc = _step_host_fn()(*args)
    if rc != OK:
        _check(rc, "swarm_step_host", ctx)


_STEP_HOST_FN = None


def _step_host_fn():
    global _STEP_HOST_FN
    if _STEP_HOST_FN is None:
        _STEP_HOST_FN = load_library().swarm_step_host
    return _STEP_HOST_FN


def swarm_device_status(ctx, stream=None) -> int:
    bits = ctypes.c_uint32(0)
    _check(load_library().swarm_device_status(ctx, _stream(stream), ctypes.byref(bits)), "swarm_device_status", ctx)
    return int(bits.value)


def swarm_last_cuda_error(ctx) -> int:
    return int(load_library().swarm_last_cuda_error(ctx))
