"""Page selection against medoid (cluster) selection on one synthetic workload: what each one attends and
what it makes the queues fetch.

Two selectors share the rest of the step: the page selector keeps the k best pages of every head by the
per-page upper bound; the medoid selector (Sec. 4.2, Tier 1 (1)) keeps the k_c best clusters by the score of
their medoid and attends all of their pages.  Both then fetch whole clusters (Sec. 4.1), deduplicated and
spread over the queues (Sec. 5.1).  The report runs both through the library on the same inputs and gives,
per selector:

  attended_pages   pages a head attends, mean over heads
  mass_recall      share of the head's exact softmax mass (over the whole context) that lies on attended
                   pages, mean over heads
  topk_recall      share of the k pages of largest exact mass that are attended, mean over heads
  io_clusters      clusters fetched after deduplication (Eq. 8 without a resident set)
  io_pages/_bytes  their pages, and those pages' K and V bytes
  max_queue_load   pages on the fullest queue, and `imbalance` = that over the mean queue load

The exact attention mass is an evaluation quantity, computed here with torch on the device; the selections,
the cluster sets and the queue loads are the library's outputs.

    python -m paper_2603_17803_b200.selector_report --config c2_128k --seeds 4
"""
from __future__ import annotations

import argparse
import json
import math

import numpy as np
import torch

from . import workloads as W
from .session import Session


def page_mass(w: W.Workload, b: int) -> torch.Tensor:
    """Exact softmax mass of every page of request b for each query head: f32 [Hq][P], rows sum to 1."""
    cfg = w.cfg
    S, d, Hkv, g = cfg.page_size, cfg.head_dim, cfg.n_kv_heads, cfg.n_q_heads // cfg.n_kv_heads
    ctx = int(w.ctx_len[b])
    P = -(-ctx // S)
    pb = int(w.page_base[b])
    q = w.q[b].float().view(Hkv, g, d)
    mass = torch.empty((Hkv, g, P), dtype=torch.float32, device=w.q.device)
    for h in range(Hkv):                                    # one KV head at a time keeps the logits small
        keys = w.kv_pool[pb:pb + P, h, 0].float().reshape(P * S, d)
        logits = (q[h] @ keys.t()) / math.sqrt(d)           # [g][P*S]
        logits[:, ctx:] = float("-inf")                     # padding of the last page
        mass[h] = torch.softmax(logits, dim=-1).view(g, P, S).sum(-1)
    return mass.view(cfg.n_q_heads, P)


def attended_by_pages(sel: torch.Tensor, n_sel: torch.Tensor, P: int) -> torch.Tensor:
    """bool [Hq][P] from one request's page lists (sel [Hq][k], n_sel [Hq])."""
    Hq, k = sel.shape
    valid = torch.arange(k, device=sel.device)[None, :] < n_sel[:, None]
    att = torch.zeros((Hq, P + 1), dtype=torch.bool, device=sel.device)
    att.scatter_(1, torch.where(valid, sel, torch.full_like(sel, P)).long(), True)   # invalid slots land on column P
    return att[:, :P]


def attended_by_clusters(sel_c: torch.Tensor, n_sel_c: torch.Tensor, page2cluster: torch.Tensor, n_clusters: int) -> torch.Tensor:
    """bool [Hq][P]: pages whose cluster is in the head's cluster list (page2cluster holds request-local ids)."""
    chosen = attended_by_pages(sel_c, n_sel_c, n_clusters)   # [Hq][C_b]
    return chosen[:, page2cluster.long()]


def _recalls(mass: torch.Tensor, att: torch.Tensor, k: int):
    k_eff = min(k, mass.shape[1])
    top = torch.topk(mass, k_eff, dim=1).indices
    hit = torch.gather(att, 1, top).float().mean(1)
    return (mass * att).sum(1), hit


def _io(sess: Session, w: W.Workload):
    n = int(sess.o.n_uniq[0])
    uniq = sess.o.uniq[:n].long()
    sizes = W.bits_u16(w.cluster_size).astype(np.int64)
    pages = int(sizes[uniq.cpu().numpy()].sum())
    load = sess.o.queue_load[: w.cfg.n_queues].cpu().numpy().astype(np.int64)
    cfg = w.cfg
    page_bytes = cfg.page_size * cfg.n_kv_heads * 2 * cfg.head_dim * 2
    mean = load.sum() / max(1, cfg.n_queues)
    return dict(io_clusters=n, io_pages=pages, io_bytes=pages * page_bytes, max_queue_load=int(load.max()),
                imbalance=float(load.max() / mean) if mean > 0 else 0.0)


def compare(w: W.Workload, top_k_clusters: int, keep_lists: bool = False) -> dict:
    """Runs both selectors on workload ``w`` (on a CUDA device) and returns {"pages": {...}, "medoids": {...}}.
    ``keep_lists`` adds the selectors' own lists under "lists" (host arrays), for checking the figures."""
    cfg = w.cfg
    sess = Session(w)
    sess.enable_medoid_index(top_k_clusters)
    out = {}
    for name in ("pages", "medoids"):
        (sess.step if name == "pages" else sess.step_medoid)()
        torch.cuda.synchronize(w.q.device)
        if sess.status():
            raise RuntimeError(f"device status {sess.status():#x} after the {name} step")
        acc = dict(attended_pages=[], mass_recall=[], topk_recall=[])
        for b in range(cfg.batch):
            P = -(-int(w.ctx_len[b]) // cfg.page_size)
            pb = int(w.page_base[b])
            if name == "pages":
                att = attended_by_pages(sess.o.sel[b], sess.o.n_sel[b], P)
            else:
                n_c = int(w.cluster_base[b + 1] - w.cluster_base[b])
                att = attended_by_clusters(sess.sel_clusters[b], sess.n_sel_clusters[b], w.page2cluster[pb:pb + P], n_c)
            m, hit = _recalls(page_mass(w, b), att, cfg.top_k)
            acc["attended_pages"].append(att.sum(1).float())
            acc["mass_recall"].append(m)
            acc["topk_recall"].append(hit)
        row = {k_: float(torch.cat(v).mean()) for k_, v in acc.items()}
        row.update(_io(sess, w))
        if keep_lists:
            lists = (sess.o.sel, sess.o.n_sel) if name == "pages" else (sess.sel_clusters, sess.n_sel_clusters)
            row["lists"] = tuple(t.cpu().numpy().copy() for t in lists)
        out[name] = row
    sess.close()
    return out


def main(argv=None) -> None:
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--config", default="c2_128k", choices=sorted(W.CONFIGS))
    ap.add_argument("--seeds", type=int, default=4)
    ap.add_argument("--top-k-clusters", type=int, default=0,
                    help="clusters per head for the medoid selector (default: top_k pages / mean pages per cluster)")
    args = ap.parse_args(argv)
    cfg = W.CONFIGS[args.config]
    rows = []
    for seed in range(args.seeds):
        w = W.generate(cfg, seed=seed, device="cuda:0")
        k_c = args.top_k_clusters
        if k_c <= 0:
            mean_pages = float(W.bits_u16(w.cluster_size).astype(np.float64).mean())
            k_c = max(1, round(cfg.top_k / mean_pages))
        rows.append(compare(w, k_c))
        del w
        torch.cuda.empty_cache()
    mean = {sel: {key: float(np.mean([r[sel][key] for r in rows])) for key in rows[0][sel]} for sel in rows[0]}
    print(json.dumps({"config": cfg.name, "seeds": args.seeds, "top_k_pages": cfg.top_k, "top_k_clusters": k_c, **mean}))


if __name__ == "__main__":
    main()
