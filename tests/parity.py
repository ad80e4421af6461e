"""Parity rules between the CUDA library and the CPU oracle, written once and used by the GPU tests and
the smoke check.  The oracle sees host copies of the very bytes the GPU reads; its own inputs (the key
summaries included) never come from the CUDA path.

Rules
  scores      |gpu - s64| <= 1e-4*|s64| + 1e-6*cond           (cond = sum of |terms|: fp32 rounding floor)
  selection   with tau = k_eff-th largest s64 and band = {p: |s64_p - tau| <= 1e-4*|tau|}: every page above
              the band is selected, none below it, count = k_eff, ascending, no duplicates; and the GPU's
              selection equals the oracle's top-k run on the GPU's own scores bit for bit
  resolve     oracle run on the GPU's selection: uniq, queue_of, load, n_uniq bit-exact
  gather      oracle run on the GPU's selection: K/V buffers and n_tok bit-exact
  attention   oracle on the same gathered rows: max|d out| <= 2e-2 (the stated bar) and the tighter
              max|d out| <= 1e-3 + 1e-2*max|out|, |d lse| <= 1e-3
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2603_17803_b200.workloads import bits_u16

SCORE_RTOL, SCORE_COND = 1e-4, 1e-6
BAND_RTOL = 1e-4
ATTN_ATOL_STATED = 2e-2
ATTN_ATOL, ATTN_RTOL, LSE_ATOL = 1e-3, 1e-2, 1e-3


def host_tables(w):
    return dict(
        page_base=w.page_base.cpu().numpy(), ctx_len=w.ctx_len.cpu().numpy(),
        page2cluster=w.page2cluster.cpu().numpy(), cluster_base=w.cluster_base.cpu().numpy(),
        replica_mask=w.cluster_replica_mask.cpu().numpy().view(np.uint32),
        cluster_size=w.cluster_size.cpu().numpy().view(np.uint16),
    )


def check_scores(gpu_scores, s64, cond, P):
    g = np.asarray(gpu_scores, dtype=np.float64)[..., :P]
    ref, c = s64[..., :P], cond[..., :P]
    err = np.abs(g - ref)
    bound = SCORE_RTOL * np.abs(ref) + SCORE_COND * c
    assert np.all(err <= bound), f"score error {err.max():.3e} exceeds bound (worst ratio {(err / bound).max():.2f})"
    return float((err / np.maximum(np.abs(ref), 1e-30)).max())


def check_selection(sel_row, n_sel, s64_row, P, k, window=0):
    """Band rule for one (request, head).  Returns the number of band pages that differ from the exact top-k.
    With a local window the last `window` pages must all be there and the rule applies to the others."""
    k_eff = min(k, P)
    assert n_sel == k_eff
    chosen = sel_row[:k_eff]
    assert np.all(sel_row[k_eff:] == -1)
    assert np.all(chosen >= 0) and np.all(chosen < P)
    assert np.all(np.diff(chosen) > 0), "selection must be strictly ascending (no duplicates)"
    w_eff = min(window, P)
    if w_eff:
        assert np.array_equal(chosen[k_eff - w_eff:], np.arange(P - w_eff, P)), "local window pages missing"
        P, k_eff, chosen = P - w_eff, k_eff - w_eff, chosen[:k_eff - w_eff]
        if k_eff == 0:
            return 0
    s = s64_row[:P]
    order = np.lexsort((np.arange(P), -s))
    tau = s[order[k_eff - 1]]
    tol = BAND_RTOL * abs(tau)
    above = np.flatnonzero(s > tau + tol)
    below = np.flatnonzero(s < tau - tol)
    got = set(chosen.tolist())
    assert set(above.tolist()) <= got, "a page above the band is missing"
    assert not (set(below.tolist()) & got), "a page below the band was selected"
    return len(got ^ set(order[:k_eff].tolist())) // 2


def check_attention(out_gpu, lse_gpu, out_ref, lse_ref):
    d_out = np.abs(np.asarray(out_gpu, np.float64) - out_ref)
    scale = np.abs(out_ref).max()
    assert d_out.max() <= ATTN_ATOL_STATED, f"attention max-abs error {d_out.max():.3e} > 2e-2"
    assert d_out.max() <= ATTN_ATOL + ATTN_RTOL * scale, \
        f"attention error {d_out.max():.3e} > {ATTN_ATOL + ATTN_RTOL * scale:.3e} (output scale {scale:.3f})"
    d_lse = np.abs(np.asarray(lse_gpu, np.float64) - lse_ref)
    assert d_lse.max() <= LSE_ATOL, f"lse error {d_lse.max():.3e}"
    return float(d_out.max()), float(d_lse.max())


def check_resolve(w, tabs, sel, n_sel, uniq_gpu, queue_of_gpu, n_uniq_gpu, load_gpu, flags=0):
    uniq, qof, load = oracle.resolve(sel, n_sel, tabs["page_base"], tabs["page2cluster"], tabs["cluster_base"],
                                     tabs["replica_mask"], tabs["cluster_size"], w.cfg.n_queues, flags)
    n = int(n_uniq_gpu)
    assert n == len(uniq), f"n_uniq {n} != {len(uniq)}"
    assert np.array_equal(uniq_gpu[:n], uniq), "uniq differs"
    assert np.array_equal(queue_of_gpu[:n], qof), "queue assignment differs"
    assert np.array_equal(load_gpu[: w.cfg.n_queues], load), f"queue loads differ: {load_gpu} vs {load}"
    return uniq, qof, load


def check_request(w, sess, b, tabs, *, heads=None, check_gathered=True):
    """Stages 1, 2 and 4 for request b against the oracle run on that request alone (its slice of the pool).
    Returns a dict of diagnostics."""
    cfg = w.cfg
    S, k, Hkv, d, Hq = cfg.page_size, cfg.top_k, cfg.n_kv_heads, cfg.head_dim, cfg.n_q_heads
    lo, hi = int(tabs["page_base"][b]), int(tabs["page_base"][b + 1])
    ctx = int(tabs["ctx_len"][b])
    P = -(-ctx // S)
    pool_b = bits_u16(w.kv_pool[lo:hi])
    pb, cl = np.array([0, hi - lo], np.int64), np.array([ctx], np.int32)
    ksum_ref = oracle.build_summaries(pool_b, pb, cl, Hkv, d, S)
    ksum_gpu = sess.ksum[lo:lo + P].float().cpu().numpy()
    ref_f = (ksum_ref[:P].astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(ksum_gpu, ref_f), "key summaries differ"

    q_b = bits_u16(w.q[b:b + 1])
    s64, s32, cond = oracle.scores(q_b, ksum_ref, pb, cl, Hkv, S, P)
    o = sess.o
    W = int(sess.shape.local_window_pages)
    hs = range(Hq) if heads is None else heads
    info = dict(band_diffs=0, exact_heads=0, heads=0)
    sel_gpu = o.sel[b].cpu().numpy()
    nsel_gpu = o.n_sel[b].cpu().numpy()
    if o.scores is not None:
        sc_gpu = o.scores[b].cpu().numpy()
        info["score_rel_err"] = check_scores(sc_gpu[list(hs)], s64[0][list(hs)], cond[0][list(hs)], P)
        if P < sc_gpu.shape[-1]:
            assert np.all(np.isneginf(sc_gpu[:, P:])), "scores beyond the request's pages were written"
        sel_on_gpu_scores, _ = oracle.topk(sc_gpu[None, :, :P], cl, S, k, W)
        assert np.array_equal(sel_on_gpu_scores[0][list(hs)], sel_gpu[list(hs)]), \
            "selection is not the exact top-k of the GPU's own scores"
    sel_ref, nsel_ref = oracle.topk(s32, cl, S, k, W)
    for h in hs:
        info["band_diffs"] += check_selection(sel_gpu[h], int(nsel_gpu[h]), s64[0, h], P, k, W)
        info["exact_heads"] += int(np.array_equal(sel_gpu[h], sel_ref[0, h]))
        info["heads"] += 1

    # stage 4 on the GPU's selection
    kg, vg, n_tok = oracle.gather(pool_b, sel_gpu[None], nsel_gpu[None], pb, cl, Hkv, d, S)
    if check_gathered and o.k_out is not None:
        assert np.array_equal(bits_u16(o.k_out[b]), kg[0]), "gathered K differs"
        assert np.array_equal(bits_u16(o.v_out[b]), vg[0]), "gathered V differs"
        assert np.array_equal(o.n_tok[b].cpu().numpy(), n_tok[0]), "n_tok differs"
    hl = list(hs)
    out_ref, lse_ref = oracle.attention(q_b[:, hl], kg[:, hl], vg[:, hl], n_tok[:, hl])
    info["attn_err"], info["lse_err"] = check_attention(o.out[b].cpu().numpy()[hl], o.lse[b].cpu().numpy()[hl],
                                                        out_ref[0], lse_ref[0])
    return info


def check_step(w, sess, *, requests=None, heads=None, flags=0):
    """Everything for one executed step whose outputs sit in sess.o."""
    torch.cuda.synchronize()
    tabs = host_tables(w)
    o = sess.o
    status = sess.status()
    assert status == 0, f"device status bits {status:#x}"
    check_resolve(w, tabs, o.sel.cpu().numpy(), o.n_sel.cpu().numpy(), o.uniq.cpu().numpy(), o.queue_of.cpu().numpy(),
                  o.n_uniq.cpu().numpy()[0], o.queue_load.cpu().numpy(), flags)
    total = dict(band_diffs=0, exact_heads=0, heads=0, attn_err=0.0, lse_err=0.0, score_rel_err=0.0)
    for b in (range(w.cfg.batch) if requests is None else requests):
        info = check_request(w, sess, b, tabs, heads=heads)
        for key in ("band_diffs", "exact_heads", "heads"):
            total[key] += info[key]
        for key in ("attn_err", "lse_err", "score_rel_err"):
            total[key] = max(total[key], info.get(key, 0.0))
    return total
