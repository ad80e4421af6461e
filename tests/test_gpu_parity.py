"""GPU parity tests: every call goes through the C-ABI library and is compared with the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import parity
from helpers import to_bf16_bits
from paper_2603_17803_b200 import binding as B
from paper_2603_17803_b200 import workloads as W
from paper_2603_17803_b200.session import Session

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_separate_calls(sess):
    sess.select()
    sess.resolve()
    sess.gather()
    sess.sparse_attn()


def small(name, **kw):
    return W.scaled(W.CONFIGS[name], **kw)


CASES = {
    # several score tiles, a ragged tail, a partial last page; sized for an oracle run of seconds
    "c1_small": small("c1_tiny", ctx_len=16 * 700 + 5, top_k=48),
    "c2_small": small("c2_128k", ctx_len=16 * 1500 + 9, top_k=96, n_topics=12),
    "c3_small": small("c3_batched", batch=3, ctx_len=16 * 400 + 1, top_k=40, n_topics=8),
    "c4_small": small("c4_long", batch=2, ctx_len=32 * 900 + 17, top_k=64, n_topics=16),
    "c5_small": small("c5_skewed", batch=5, ctx_range=(16 * 20, 16 * 900), top_k=32, n_topics=10),
    "k_exceeds_pages": small("c5_skewed", batch=3, ctx_range=(1, 16 * 12), top_k=24, n_topics=3),
}


@pytest.mark.parametrize("name", list(CASES))
def test_separate_calls_match_oracle(name):
    w = W.generate(CASES[name], seed=11, device=DEV)
    sess = Session(w, keep_scores=True, keep_gathered=True)
    run_separate_calls(sess)
    info = parity.check_step(w, sess)
    assert info["heads"] == w.cfg.batch * w.cfg.n_q_heads
    sess.close()


@pytest.mark.parametrize("name", list(CASES))
def test_fused_step_equals_composition(name):
    w = W.generate(CASES[name], seed=12, device=DEV)
    a = Session(w, keep_scores=True, keep_gathered=True)
    run_separate_calls(a)
    torch.cuda.synchronize()
    b = Session(w, keep_scores=True, keep_gathered=True, ksum=a.ksum)
    b.step()
    info = parity.check_step(w, b)
    for f in ("sel", "n_sel", "n_tok", "k_out", "v_out", "queue_load"):
        assert torch.equal(getattr(a.o, f), getattr(b.o, f)), f
    n = int(a.o.n_uniq[0])
    assert int(b.o.n_uniq[0]) == n
    assert torch.equal(a.o.uniq[:n], b.o.uniq[:n]) and torch.equal(a.o.queue_of[:n], b.o.queue_of[:n])
    assert torch.equal(a.o.scores, b.o.scores)
    assert (a.o.out - b.o.out).abs().max().item() <= 1e-4
    assert (a.o.lse - b.o.lse).abs().max().item() <= 1e-4
    # fused step without the optional outputs gives the same required outputs
    c = Session(w, ksum=a.ksum)
    c.step()
    torch.cuda.synchronize()
    assert torch.equal(c.o.sel, b.o.sel) and torch.equal(c.o.out, b.o.out) and torch.equal(c.o.queue_load, b.o.queue_load)
    for s in (a, b, c):
        s.close()


def test_workspace_canaries_catch_a_stray_write():
    """Every Session.close() checks the canaries between the workspace regions (the stand-in for a memory checker
    on this path).  Here one canary byte is overwritten from the host side -- a torch fill, no kernel of the
    library involved -- to show that the check fires, and where."""
    w = W.generate(CASES["c1_small"], seed=3, device=DEV)
    sess = Session(w)
    sess.step()
    assert B.swarm_check_workspace(sess.ctx) == 0
    sess.workspace[7] = 0                                   # inside the canary in front of the first region
    assert B.swarm_check_workspace(sess.ctx) == 1
    sess.workspace[-3] = 1                                  # and inside the one behind the last region
    damaged = B.swarm_check_workspace(sess.ctx)
    assert damaged & 1 and damaged >> 1 and (damaged >> 1) & ((damaged >> 1) - 1) == 0
    with pytest.raises(RuntimeError, match="canaries"):
        sess.close()


@pytest.mark.parametrize("name", ["c2_small", "c3_small", "c5_small", "k_exceeds_pages"])
def test_overlapped_tail_gives_the_same_step(name):
    """Cluster resolution on a tail stream (swarm_set_tail_stream): consecutive steps with changing queries are
    enqueued without waiting in between, so a step's resolution runs beside the next step's scoring and
    selection; every step's outputs must equal those of the plain step bit for bit (integers) / within rounding
    (attention), and the last one must match the oracle."""
    w = W.generate(CASES[name], seed=14, device=DEV)
    plain = Session(w)
    tail_stream, stream = torch.cuda.Stream(), torch.cuda.Stream()
    tail = Session(w, ksum=plain.ksum, tail_stream=tail_stream)
    qs = [w.q, (w.q.float() * -1.0).to(torch.bfloat16), (w.q.float() * 0.5 + 0.125).to(torch.bfloat16), w.q]
    want = []
    for q in qs:
        plain.set_query(q)
        plain.step()
        torch.cuda.synchronize()
        n = int(plain.o.n_uniq[0])
        want.append(dict(sel=plain.o.sel.clone(), uniq=plain.o.uniq[:n].clone(), queue_of=plain.o.queue_of[:n].clone(),
                         load=plain.o.queue_load.clone(), out=plain.o.out.clone(), lse=plain.o.lse.clone()))
    # the tail session needs one set of outputs per step in flight: give every step its own
    outs = []
    with torch.cuda.stream(stream):
        for q in qs:
            o = type(tail.o)(**{f: (getattr(tail.o, f).clone() if getattr(tail.o, f) is not None else None)
                                for f in tail.o.__dataclass_fields__})
            outs.append(o)
            tail.o = o
            tail.outputs = B.make_outputs(**{k_: getattr(o, k_) for k_ in o.__dataclass_fields__})
            tail.set_query(q)
            tail.step(stream=stream)
        tail.tail_join(stream)
        stream.synchronize()
    assert tail.status() == 0
    for o, ref in zip(outs, want):
        n = len(ref["uniq"])
        assert int(o.n_uniq[0]) == n
        assert torch.equal(o.sel, ref["sel"]) and torch.equal(o.uniq[:n], ref["uniq"])
        assert torch.equal(o.queue_of[:n], ref["queue_of"]) and torch.equal(o.queue_load, ref["load"])
        assert (o.out - ref["out"]).abs().max().item() <= 1e-4 and (o.lse - ref["lse"]).abs().max().item() <= 1e-4
    parity.check_step(w, tail)
    # the same chain recorded into a CUDA graph (the capture has to join the tail stream) and replayed twice
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            for _ in range(3):
                tail.step(stream=stream)
            tail.tail_join(stream)
        g.replay()
        g.replay()
        stream.synchronize()
    parity.check_step(w, tail)
    plain.close()
    tail.close()


@pytest.mark.parametrize("hq,hkv", [(16, 2), (8, 2), (6, 3), (5, 5), (6, 2)])
def test_fp32_pipe_scorer_matches_oracle(hq, hkv):
    """The scorer on the fp32 pipes (what shapes beyond the streaming kernel's limits fall back to), forced by
    swarm_set_scorer: groups of 8, 4, 2 and 1 query heads per KV head (its four instantiations; a group of 3 runs
    the single-head one three times), ragged tails, requests of unequal length, then the whole step on top."""
    cfg = small("c5_skewed", batch=3, n_q_heads=hq, n_kv_heads=hkv, ctx_range=(16 * 9, 16 * 333), top_k=24, n_topics=5)
    w = W.generate(cfg, seed=31, device=DEV)
    ref = Session(w, keep_scores=True, keep_gathered=True)
    ref.step()
    sess = Session(w, keep_scores=True, keep_gathered=True, scorer=B.SCORER_FP32, ksum=ref.ksum)
    run_separate_calls(sess)
    info = parity.check_step(w, sess)
    assert info["heads"] == cfg.batch * hq
    sess.step()
    parity.check_step(w, sess)
    # the two scorers agree far inside the tolerance of the score rule
    torch.cuda.synchronize()
    a, b = ref.o.scores, sess.o.scores
    live = torch.isfinite(a)
    assert torch.equal(live, torch.isfinite(b))
    assert ((a[live] - b[live]).abs() <= 1e-5 * a[live].abs() + 1e-4).all()
    with pytest.raises(B.SwarmError):
        B.swarm_set_scorer(sess.ctx, 3)
    B.swarm_set_scorer(sess.ctx, B.SCORER_TENSOR)
    sess.step()
    parity.check_step(w, sess)
    ref.close()
    sess.close()


@pytest.mark.parametrize("name", ["c1_tiny", "c2_128k"])
def test_full_size_configs_match_oracle(name):
    """The two configurations the oracle handles whole, at full size, through the fused step."""
    w = W.generate(W.CONFIGS[name], seed=0, device=DEV)
    sess = Session(w, keep_scores=True, keep_gathered=True)
    sess.step()
    info = parity.check_step(w, sess)
    assert info["exact_heads"] >= info["heads"] - 4      # band differences are legal but rare
    sess.close()


@pytest.mark.parametrize("name,reqs,heads", [("c3_batched", [0, 9], [0, 5, 31]), ("c4_long", [1], [0, 17, 63])])
def test_full_size_sampled(name, reqs, heads):
    """Full-size launch configuration; stage 3 checked whole, the other stages on sampled requests/heads."""
    w = W.generate(W.CONFIGS[name], seed=0, device=DEV)
    sess = Session(w, keep_scores=True)
    sess.step()
    parity.check_step(w, sess, requests=reqs, heads=heads)
    sess.close()


def test_c5_full_size_sampled():
    w = W.generate(W.CONFIGS["c5_skewed"], seed=0, device=DEV)
    sess = Session(w, keep_scores=True)
    sess.step()
    lens = w.ctx_len.cpu().numpy()
    reqs = sorted({int(np.argmin(lens)), int(np.argmax(lens)), 7})
    parity.check_step(w, sess, requests=reqs, heads=[0, 13, 31])
    # more fetched clusters than the resolution kernel stages in shared memory: the submission order too
    sess.enable_submit_order()
    sess.step()
    assert check_submit_order(w, sess) > 20000
    sess.close()


def test_caller_supplied_selection_and_misplaced_partial_page():
    """swarm_gather / swarm_sparse_attn on a selection the caller wrote (ascending, a subset of the pages, the
    partial last page included): parity with the oracle; the same pages with the partial page NOT last are
    refused for that page (status bit, slot zero-filled) instead of attending its padding rows."""
    cfg = small("c2_128k", ctx_len=16 * 300 + 5, top_k=20, n_topics=4)
    w = W.generate(cfg, seed=17, device=DEV)
    sess = Session(w, keep_gathered=True)
    P = cfg.max_pages()
    rng = np.random.default_rng(2)
    sel = np.full((1, cfg.n_q_heads, cfg.top_k), -1, dtype=np.int32)
    n_sel = np.zeros((1, cfg.n_q_heads), dtype=np.int32)
    for h in range(cfg.n_q_heads):
        n = int(rng.integers(1, cfg.top_k + 1))
        pages = np.sort(rng.choice(P - 1, size=n - 1, replace=False)) if n > 1 else np.zeros(0, np.int64)
        sel[0, h, :n] = np.concatenate([pages, [P - 1]])     # the partial page, last
        n_sel[0, h] = n
    sel_t, n_sel_t = torch.from_numpy(sel).to(DEV), torch.from_numpy(n_sel).to(DEV)
    sess.gather(sel_t, n_sel_t)
    sess.sparse_attn()
    torch.cuda.synchronize()
    assert sess.status() == 0
    tabs = parity.host_tables(w)
    pool = parity.bits_u16(w.kv_pool)
    kg, vg, n_tok = oracle.gather(pool, sel, n_sel, tabs["page_base"], tabs["ctx_len"], cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    assert np.array_equal(parity.bits_u16(sess.o.k_out), kg) and np.array_equal(parity.bits_u16(sess.o.v_out), vg)
    assert np.array_equal(sess.o.n_tok.cpu().numpy(), n_tok)
    out_ref, lse_ref = oracle.attention(parity.bits_u16(w.q), kg, vg, n_tok)
    parity.check_attention(sess.o.out.cpu().numpy(), sess.o.lse.cpu().numpy(), out_ref, lse_ref)
    # the partial page first: flagged and skipped
    h = int(np.argmax(n_sel[0] >= 2))
    n = int(n_sel[0, h])
    sel[0, h, :n] = np.concatenate([[P - 1], sel[0, h, :n - 1]])
    sess.gather(torch.from_numpy(sel).to(DEV), n_sel_t)
    torch.cuda.synchronize()
    assert sess.status() == B.DEV_BAD_PAGE
    assert not sess.o.k_out[0, h, : cfg.page_size].any()
    sess.close()


@pytest.mark.parametrize("splits", [1, 2, 7, 64])
def test_split_count_is_unobservable(splits):
    w = W.generate(CASES["c2_small"], seed=5, device=DEV)
    sess = Session(w, keep_gathered=True)
    B.swarm_set_attn_splits(sess.ctx, splits)
    run_separate_calls(sess)
    parity.check_step(w, sess)
    sess.step()
    parity.check_step(w, sess)
    sess.close()


@pytest.mark.parametrize("flags", [B.ORDER_BY_ID, B.UNIT_LOAD, B.ORDER_BY_ID | B.UNIT_LOAD])
@pytest.mark.parametrize("name", ["c3_small", "c5_small"])
def test_scheduling_flags(name, flags):
    w = W.generate(CASES[name], seed=6, device=DEV)
    sess = Session(w, flags=flags)
    sess.step()
    parity.check_step(w, sess, flags=flags)
    sess.close()


@pytest.mark.parametrize("replication,D", [("one", 5), ("all", 7), ("all", 32), ("two", 32)])
def test_replication_extremes(replication, D):
    cfg = small("c3_batched", batch=2, ctx_len=16 * 300, top_k=50, n_topics=6, replication=replication, n_queues=D)
    w = W.generate(cfg, seed=7, device=DEV)
    sess = Session(w, flags=B.UNIT_LOAD if replication == "all" else 0)
    sess.step()
    parity.check_step(w, sess, flags=B.UNIT_LOAD if replication == "all" else 0)
    load = sess.o.queue_load.cpu().numpy()[:D]
    if replication == "all":
        assert load.max() - load.min() <= 1
    sess.close()


def test_all_equal_scores_pick_lowest_ids_and_signed_zero_ties():
    cfg = small("c1_tiny", ctx_len=16 * 300, top_k=20)
    w = W.generate(cfg, seed=8, device=DEV)
    w.q.zero_()                                          # every score is exactly 0
    sess = Session(w, keep_scores=True)
    sess.step()
    torch.cuda.synchronize()
    assert torch.equal(sess.o.sel[0, 3].cpu(), torch.arange(20, dtype=torch.int32))
    parity.check_step(w, sess)
    # planted duplicates straddling the k-th place: make the scorer reproduce chosen scores exactly
    # (q = e_0 and kmin = kmax = the wanted score in coordinate 0), then compare with the oracle's top-k
    P = cfg.max_pages()
    sc = torch.zeros((1, 8, P), device=DEV)
    sc[0, 1] = torch.arange(P, device=DEV) % 7
    sc[0, 2] = -(torch.arange(P, device=DEV) % 5).float()
    sc[0, 3] = (torch.arange(P, device=DEV) // 50).float()
    ref, _ = oracle.topk(sc.cpu().numpy(), w.ctx_len.cpu().numpy(), 16, 20)
    ksum = torch.zeros_like(sess.ksum)
    ksum[:, :, :, 0] = sc[0].t()[:, :, None].to(torch.bfloat16)
    w.q.zero_()
    w.q[..., 0] = 1.0
    sess2 = Session(w, keep_scores=True, ksum=ksum)
    sess2.select()
    torch.cuda.synchronize()
    assert torch.equal(sess2.o.scores[0, :, :P], sc[0])
    assert np.array_equal(sess2.o.sel.cpu().numpy()[0], ref[0])
    sess.close()
    sess2.close()


def test_structured_attention_outputs_of_order_one():
    """Dominant key and constant V: outputs of magnitude 1, so the tolerance is meaningful."""
    cfg = small("c1_tiny", ctx_len=16 * 200, top_k=30)
    w = W.generate(cfg, seed=9, device=DEV)
    q = w.q.float()
    # plant, for head 2, a key in page 77 aligned with q and strong enough to dominate
    w.kv_pool[77, 2, 0, 5] = (40.0 * q[0, 2] / q[0, 2].norm()).to(torch.bfloat16)
    w.kv_pool[:, 4, 1] = 1.5                              # head 4: constant V
    sess = Session(w, keep_gathered=True)
    sess.step()
    parity.check_step(w, sess)
    out = sess.o.out.cpu()
    assert (out[0, 2] - w.kv_pool[77, 2, 1, 5].float().cpu()).abs().max() < 2e-2
    assert (out[0, 4] - 1.5).abs().max() < 1e-5
    sess.close()


def test_corrupt_tables_set_status_bits_and_never_trap():
    cfg = small("c3_batched", batch=2, ctx_len=16 * 100, top_k=16, n_topics=4)
    w = W.generate(cfg, seed=10, device=DEV)
    sess = Session(w)
    sess.step()
    torch.cuda.synchronize()
    assert sess.status() == 0
    good_mask = w.cluster_replica_mask.clone()
    w.cluster_replica_mask.zero_()                        # no replica anywhere
    sess.step()
    assert sess.status() & B.DEV_BAD_REPLICA
    assert int(sess.o.queue_of[0]) == 0xFF
    w.cluster_replica_mask.copy_(good_mask)
    good_p2c = w.page2cluster.clone()
    w.page2cluster.fill_(10 ** 6)                         # cluster ids out of range
    sess.step()
    assert sess.status() & B.DEV_BAD_CLUSTER
    w.page2cluster.copy_(good_p2c)
    bad_sel = sess.o.sel.clone()
    bad_sel[0, 0, 0] = 10 ** 6                            # page id out of range, fed to the stage calls
    sess.resolve(sel=bad_sel)
    assert sess.status() & B.DEV_BAD_PAGE
    good_len = w.ctx_len.clone()
    w.ctx_len[0] = 0
    sess.select()
    assert sess.status() & B.DEV_BAD_LENGTH
    w.ctx_len.copy_(good_len)
    sess.step()                                           # the ctx is still usable
    torch.cuda.synchronize()
    assert sess.status() == 0
    parity.check_step(w, sess)
    sess.close()


def test_invalid_arguments_are_rejected_on_the_host():
    ok = dict(batch=1, n_q_heads=8, n_kv_heads=2, page_size=16, top_k=4, n_queues=4, max_pages_per_req=8,
              max_clusters_total=4, n_pool_pages=8)
    for bad, code in [(dict(head_dim=64), B.ERR_UNSUPPORTED), (dict(page_size=8), B.ERR_UNSUPPORTED),
                      (dict(n_queues=33), B.ERR_INVALID_ARG), (dict(n_kv_heads=3), B.ERR_INVALID_ARG),
                      (dict(top_k=0), B.ERR_INVALID_ARG), (dict(flags=64), B.ERR_INVALID_ARG)]:
        with pytest.raises(B.SwarmError) as e:
            B.swarm_create(B.make_shape(**{**ok, **bad}))
        assert e.value.code == code
    shape = B.make_shape(**ok)
    ctx = B.swarm_create(shape)
    t = torch.zeros(1024, dtype=torch.int32, device=DEV)
    with pytest.raises(B.SwarmError) as e:                # no workspace yet
        B.swarm_select(ctx, B.make_inputs(q=t, ksum=t, page_base=t, ctx_len=t), None, t, t)
    assert e.value.code == B.ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(B.SwarmError) as e:
        B.swarm_set_workspace(ctx, torch.empty(16, dtype=torch.uint8, device=DEV))
    assert e.value.code == B.ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(B.SwarmError) as e:                # the flag array lives in the workspace
        B.swarm_cluster_flags(ctx)
    assert e.value.code == B.ERR_WORKSPACE_TOO_SMALL
    ws = torch.empty(B.swarm_workspace_bytes(shape), dtype=torch.uint8, device=DEV)
    B.swarm_set_workspace(ctx, ws)
    with pytest.raises(B.SwarmError) as e:                # null input
        B.swarm_select(ctx, B.make_inputs(q=t, ksum=None, page_base=t, ctx_len=t), None, t, t)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.SwarmError) as e:                # misaligned pointer
        B.swarm_select(ctx, B.make_inputs(q=t[1:], ksum=t, page_base=t, ctx_len=t), None, t, t)
    assert e.value.code == B.ERR_INVALID_ARG
    addr, n = B.swarm_cluster_flags(ctx)
    assert n == 4 and ws.data_ptr() <= addr and addr + n <= ws.data_ptr() + ws.numel()
    for half in (B.swarm_step_begin, B.swarm_step_end):    # the halves validate like the whole step
        with pytest.raises(B.SwarmError) as e:
            half(ctx, B.make_inputs(q=t, ksum=t, page_base=t, ctx_len=t), B.make_outputs(sel=t, n_sel=t))
        assert e.value.code == B.ERR_INVALID_ARG
    B.swarm_destroy(ctx)


def test_step_host_round_trip():
    w = W.generate(CASES["c2_small"], seed=13, device=DEV)
    sess = Session(w)
    sess.step()
    torch.cuda.synchronize()
    want_out, want_load = sess.o.out.cpu().clone(), sess.o.queue_load.cpu().clone()
    q_host = w.q.cpu().pin_memory()
    out_host = torch.empty_like(want_out).pin_memory()
    lse_host = torch.empty((1, 32), dtype=torch.float32).pin_memory()
    n_host = torch.zeros(1, dtype=torch.int32).pin_memory()
    load_host = torch.zeros(w.cfg.n_queues, dtype=torch.int32).pin_memory()
    sess.o.out.zero_()
    sess.step_host(q_host, out_host, lse_host, n_host, load_host)
    assert torch.equal(out_host, want_out)
    assert torch.equal(load_host, want_load[: w.cfg.n_queues])
    assert int(n_host[0]) == int(sess.o.n_uniq[0])
    # on a stream of its own the call records a graph and replays it; repeated calls give the same bytes
    stream = torch.cuda.Stream()
    for _ in range(3):
        out_host.zero_(); lse_host.zero_(); n_host.zero_(); load_host.zero_()
        sess.step_host(q_host, out_host, lse_host, n_host, load_host, stream=stream)
        assert torch.equal(out_host, want_out) and torch.equal(load_host, want_load[: w.cfg.n_queues])
        assert torch.equal(lse_host.view(-1), sess.o.lse.cpu().view(-1)) and int(n_host[0]) == int(sess.o.n_uniq[0])
    # pageable (and odd-offset) destinations take the copy path and give the same bytes
    out_page = torch.empty(want_out.numel() + 1, dtype=torch.float32)[1:].view_as(want_out)
    lse_page = torch.empty((1, 32), dtype=torch.float32)
    n_page, load_page = torch.zeros(1, dtype=torch.int32), torch.zeros(w.cfg.n_queues, dtype=torch.int32)
    sess.step_host(q_host, out_page, lse_page, n_page, load_page)
    assert torch.equal(out_page, want_out) and torch.equal(load_page, want_load[: w.cfg.n_queues])
    assert int(n_page[0]) == int(sess.o.n_uniq[0])
    # a mix: pinned out, no lse, pageable counters
    out_host.zero_()
    sess.step_host(q_host, out_host, None, n_page, None)
    assert torch.equal(out_host, want_out)
    sess.close()


@pytest.mark.parametrize("name", ["c3_small", "c5_small", "k_exceeds_pages"])
def test_step_host_follows_a_query_buffer_rewritten_between_calls(name):
    """The same pinned buffers, new contents every call: every call's results are those of its own query and are
    complete in host memory when the call returns (the recorded graph, the fetch of q and the completion word
    are all reused from call to call)."""
    w = W.generate(CASES[name], seed=17, device=DEV)
    cfg = w.cfg
    sess = Session(w)
    ref = Session(w, ksum=sess.ksum)
    g = torch.Generator(device="cpu").manual_seed(5)
    q_host = torch.empty_like(w.q, device="cpu").pin_memory()
    out_host = torch.empty((cfg.batch, cfg.n_q_heads, cfg.head_dim), dtype=torch.float32).pin_memory()
    lse_host = torch.empty((cfg.batch, cfg.n_q_heads), dtype=torch.float32).pin_memory()
    n_host = torch.zeros(1, dtype=torch.int32).pin_memory()
    load_host = torch.zeros(cfg.n_queues, dtype=torch.int32).pin_memory()
    stream = torch.cuda.Stream()
    for it in range(40):
        q = (w.q.cpu().float() + 0.5 * torch.randn(w.q.shape, generator=g)).to(torch.bfloat16)
        q_host.copy_(q)
        out_host.fill_(float("nan")); lse_host.fill_(float("nan")); n_host.fill_(-1); load_host.fill_(-1)
        sess.step_host(q_host, out_host, lse_host, n_host, load_host, stream=stream)
        got = (out_host.clone(), lse_host.clone(), int(n_host[0]), load_host.clone())   # read at once, no synchronize
        ref.set_query(q.to(DEV))
        ref.step()
        torch.cuda.synchronize()
        assert torch.equal(got[0], ref.o.out.cpu()), f"call {it}"
        assert torch.equal(got[1], ref.o.lse.cpu()) and got[2] == int(ref.o.n_uniq[0])
        assert torch.equal(got[3], ref.o.queue_load.cpu()[: cfg.n_queues])
        assert torch.equal(sess.o.sel, ref.o.sel) and torch.equal(sess.o.uniq[: got[2]], ref.o.uniq[: got[2]])
    assert sess.status() == 0
    sess.close()
    ref.close()


def test_step_can_be_captured_in_a_cuda_graph():
    w = W.generate(CASES["c3_small"], seed=14, device=DEV)
    sess = Session(w)
    sess.step()
    torch.cuda.synchronize()
    n = int(sess.o.n_uniq[0])
    sess.o.uniq[n:].zero_()                               # entries beyond n_uniq are not written
    want = {f: getattr(sess.o, f).clone() for f in ("sel", "out", "lse", "queue_load", "uniq", "n_uniq")}
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        sess.step(stream=s)                               # warm-up on the capture stream
        s.synchronize()
        with torch.cuda.graph(graph, stream=s):
            sess.step(stream=s)
    for f in want:
        getattr(sess.o, f).zero_()
    graph.replay()
    torch.cuda.synchronize()
    for f, t in want.items():
        assert torch.equal(getattr(sess.o, f), t), f
    sess.close()


def test_paged_attention_alone_matches_gathered_attention():
    w = W.generate(CASES["c4_small"], seed=15, device=DEV)
    sess = Session(w, keep_gathered=True)
    run_separate_calls(sess)
    torch.cuda.synchronize()
    out, lse = sess.o.out.clone(), sess.o.lse.clone()
    sess.o.out.zero_()
    sess.sparse_attn_paged()
    torch.cuda.synchronize()
    assert (sess.o.out - out).abs().max().item() <= 1e-5 and (sess.o.lse - lse).abs().max().item() <= 1e-5
    parity.check_step(w, sess)
    out2 = sess.o.out.clone()
    sess.o.out.zero_()
    sess.sparse_attn_paged(reuse_last_selection=True)     # bitmaps left in the workspace by the calls above
    torch.cuda.synchronize()
    assert torch.equal(sess.o.out, out2)
    sess.close()


@pytest.mark.parametrize("name", ["c1_small", "c2_small", "c3_small", "c5_small"])
def test_paged_attention_reuses_the_bitmaps_a_step_left(name):
    """A fused step hands its page bitmaps to its own attention kernel in whichever form is fastest; whatever
    that is, a later swarm_sparse_attn_paged without a selection finds them in the workspace."""
    w = W.generate(CASES[name], seed=16, device=DEV)
    sess = Session(w)
    sess.step()
    sess.step()
    torch.cuda.synchronize()
    out, lse = sess.o.out.clone(), sess.o.lse.clone()
    sess.o.out.zero_()
    sess.o.lse.zero_()
    sess.sparse_attn_paged(reuse_last_selection=True)
    torch.cuda.synchronize()
    assert sess.status() == 0
    assert (sess.o.out - out).abs().max().item() <= 1e-5 and (sess.o.lse - lse).abs().max().item() <= 1e-5
    parity.check_step(w, sess)
    sess.close()


@pytest.mark.parametrize("name", ["c1_small", "c2_small", "c3_small", "c4_small", "c5_small"])
@pytest.mark.parametrize("tail", [False, True])
def test_index_prefetch_changes_no_result(name, tail):
    """swarm_set_index_prefetch: the scorer asks for its first index blocks before it waits for the previous
    step's attention kernel (which releases its SMs early for it).  Back-to-back steps with the switch on give the
    results of the switch off, bit for bit, and match the oracle."""
    w = W.generate(CASES[name], seed=17, device=DEV)
    tstream = torch.cuda.Stream() if tail else None
    ref = Session(w, tail_stream=tstream)
    for _ in range(2):
        ref.step()
    if tail:
        ref.tail_join()
    torch.cuda.synchronize()
    sess = Session(w, ksum=ref.ksum, tail_stream=tstream, index_prefetch=True)
    for _ in range(4):                                     # each step's scorer is launched behind the previous step's attention
        sess.step()
    if tail:
        sess.tail_join()
    torch.cuda.synchronize()
    assert sess.status() == 0
    for key in ("sel", "n_sel", "out", "lse"):
        assert torch.equal(getattr(ref.o, key), getattr(sess.o, key)), key
    n_q = w.cfg.n_queues
    assert int(ref.o.n_uniq[0]) == int(sess.o.n_uniq[0]) and torch.equal(ref.o.queue_load[:n_q], sess.o.queue_load[:n_q])
    parity.check_step(w, sess)
    B.swarm_set_index_prefetch(sess.ctx, False)            # and off again
    sess.step()
    if tail:
        sess.tail_join()
    torch.cuda.synchronize()
    assert sess.status() == 0 and torch.equal(ref.o.out, sess.o.out)
    sess.close()
    ref.close()


@pytest.mark.parametrize("name", ["c3_small", "c5_small"])
def test_resident_filter_and_cache_counters(name):
    """Eq. 8 with the resident term, activation frequencies and Eq. 6 scores, against the oracle on the GPU's
    own selection; two steps in a row so the counters accumulate; then detached again."""
    w = W.generate(CASES[name], seed=16, device=DEV)
    sess = Session(w)
    C = w.n_clusters
    g = torch.Generator(device="cpu").manual_seed(5)
    resident = (torch.rand(C, generator=g) < 0.3).to(torch.uint8).to(DEV)
    freq0 = torch.randint(-3, 10, (C,), generator=g, dtype=torch.int32)
    freq = freq0.to(DEV)
    score = torch.zeros(C, dtype=torch.float32, device=DEV)
    n_hit = torch.zeros(4, dtype=torch.int32, device=DEV)
    t_base, t_tr = 80.0, 2.5
    B.swarm_set_cache(sess.ctx, resident=resident, freq=freq, score=score, n_hit=n_hit, t_base=t_base, t_transfer=t_tr)
    tabs = parity.host_tables(w)
    want_freq = freq0.numpy().copy()
    for step_no in range(2):
        if step_no == 0:
            sess.step()
        else:                                             # the separate call takes the same path
            sess.resolve()
        torch.cuda.synchronize()
        assert sess.status() == 0
        uniq, qof, load, hits, want_freq, want_score = oracle.resolve_cached(
            sess.o.sel.cpu().numpy(), sess.o.n_sel.cpu().numpy(), tabs["page_base"], tabs["page2cluster"],
            tabs["cluster_base"], tabs["replica_mask"], tabs["cluster_size"], resident.cpu().numpy(), want_freq,
            w.cfg.n_queues, t_base, t_tr)
        n = int(sess.o.n_uniq[0])
        assert n == len(uniq) and hits > 0
        assert np.array_equal(sess.o.uniq[:n].cpu().numpy(), uniq)
        assert np.array_equal(sess.o.queue_of[:n].cpu().numpy(), qof)
        assert np.array_equal(sess.o.queue_load.cpu().numpy()[: w.cfg.n_queues], load)
        assert int(n_hit[0]) == hits
        assert np.array_equal(freq.cpu().numpy(), want_freq)
        assert np.allclose(score.cpu().numpy(), want_score, rtol=1e-6, atol=1e-6)
    B.swarm_set_cache(sess.ctx)                           # detached: plain merge again
    sess.step()
    parity.check_step(w, sess)
    assert np.array_equal(freq.cpu().numpy(), want_freq)
    sess.close()


EDGE_SHAPES = {
    # group of 16 heads per KV head (two head tiles in the scorer and in attention), 32-token pages
    "g16_s32": small("c4_long", batch=2, n_q_heads=32, n_kv_heads=2, ctx_len=32 * 300 + 5, top_k=24, n_topics=6),
    # odd number of KV heads, group of 2
    "hkv3_g2": small("c2_128k", batch=2, n_q_heads=6, n_kv_heads=3, ctx_len=16 * 500 + 3, top_k=33, n_topics=5),
    # more KV heads than one scorer block holds (two KV groups), MHA
    "hkv16_g1": small("c1_tiny", batch=1, n_q_heads=16, n_kv_heads=16, ctx_len=16 * 260, top_k=17),
    # a single page per head, a single queue
    "k1_d1": small("c3_batched", batch=3, ctx_len=16 * 150 + 1, top_k=1, n_topics=4, n_queues=1, replication="one"),
    # group of 12 heads: a full head tile of 8 plus a partial one of 4
    "g12": small("c2_128k", batch=1, n_q_heads=24, n_kv_heads=2, ctx_len=16 * 400, top_k=40, n_topics=6),
    # more (request, KV head) groups than fit one wave of attention CTAs with short page ranges: two waves, the
    # last groups cut into one range more than the others
    "two_waves": small("c3_batched", batch=12, ctx_len=16 * 300 + 7, top_k=128, n_topics=8),
}


@pytest.mark.parametrize("name", list(EDGE_SHAPES))
def test_unusual_shapes(name):
    w = W.generate(EDGE_SHAPES[name], seed=17, device=DEV)
    a = Session(w, keep_scores=True, keep_gathered=True)
    run_separate_calls(a)
    parity.check_step(w, a)
    b = Session(w, keep_scores=True, keep_gathered=True, ksum=a.ksum)
    b.step()
    parity.check_step(w, b)
    assert torch.equal(a.o.sel, b.o.sel) and (a.o.out - b.o.out).abs().max().item() <= 1e-4
    a.close()
    b.close()


# ---- local window (Sec. 4.2, Tier 1 (2)): the last W pages of every request are always selected ------------
@pytest.mark.parametrize("name,window", [("c1_small", 1), ("c2_small", 16), ("c3_small", 2), ("c4_small", 8), ("c5_small", 3),
                                         ("k_exceeds_pages", 8), ("k_exceeds_pages", 24)])
def test_local_window(name, window):
    cfg = CASES[name]
    window = min(window, cfg.top_k)
    w = W.generate(cfg, seed=23, device=DEV)
    a = Session(w, keep_scores=True, keep_gathered=True, local_window_pages=window)
    a.step()
    parity.check_step(w, a)
    sel, n_sel = a.o.sel.cpu().numpy(), a.o.n_sel.cpu().numpy()
    ctx = w.ctx_len.cpu().numpy()
    for b in range(cfg.batch):
        P = -(-int(ctx[b]) // cfg.page_size)
        w_eff = min(window, P)
        for h in range(cfg.n_q_heads):
            n = int(n_sel[b, h])
            assert list(sel[b, h, n - w_eff:n]) == list(range(P - w_eff, P))
    b_ = Session(w, keep_scores=True, keep_gathered=True, ksum=a.ksum, local_window_pages=window)
    run_separate_calls(b_)
    parity.check_step(w, b_)
    assert torch.equal(a.o.sel, b_.o.sel)
    a.close()
    b_.close()


def test_local_window_covering_all_of_k_and_longer_than_a_request():
    cfg = small("c3_batched", batch=3, ctx_len=16 * 40, top_k=12, n_topics=4)
    w = W.generate(cfg, seed=29, device=DEV)
    w.ctx_len[1] = 16 * 5 + 3                               # 6 pages < window
    a = Session(w, keep_scores=True, keep_gathered=True, local_window_pages=12)
    a.step()
    parity.check_step(w, a)
    a.close()
    with pytest.raises(B.SwarmError):
        Session(w, local_window_pages=13)


# ---- every list-length variant of the selection kernel, with and without a local window --------------------
@pytest.mark.parametrize("pages", [900, 2000, 4000, 8000, 16000, 30000, 45000])
@pytest.mark.parametrize("window", [0, 5])
def test_selection_at_every_list_length(pages, window):
    cfg = small("c1_tiny", batch=2, n_q_heads=2, n_kv_heads=1, ctx_len=16 * pages - 7, top_k=100, n_topics=8)
    w = W.generate(cfg, seed=31, device=DEV)
    w.ctx_len[1] = 16 * (pages // 3) + 1                    # a shorter request beside the long one
    sess = Session(w, keep_scores=True, local_window_pages=window)
    sess.select()
    torch.cuda.synchronize()
    assert sess.status() == 0
    sc = sess.o.scores.cpu().numpy()
    sel, n_sel = sess.o.sel.cpu().numpy(), sess.o.n_sel.cpu().numpy()
    ctx = w.ctx_len.cpu().numpy()
    want, n_want = oracle.topk(sc, ctx, cfg.page_size, cfg.top_k, window)
    assert np.array_equal(n_sel, n_want) and np.array_equal(sel, want)
    # the fused step marks the same pages and attends to them
    sess.step()
    torch.cuda.synchronize()
    assert np.array_equal(sess.o.sel.cpu().numpy(), want)
    parity.check_step(w, sess, requests=[1], heads=[1])
    sess.close()


# ---- medoid index (Sec. 4.2 Tier 1 (1)): clusters are scored by their medoid page and retrieved whole -------
def check_medoid_step(w, sess, k_c, flags=0, window=0):
    torch.cuda.synchronize()
    assert sess.status() == 0
    cfg = w.cfg
    tabs = parity.host_tables(w)
    ptr, members, medoid = (t.cpu().numpy() for t in (sess.cluster_page_ptr, sess.cluster_pages, sess.medoid_page))
    ksum = W.bits_u16(sess.ksum)
    rows_gpu = W.bits_u16(sess.medoid_ksum)
    rows_ref = oracle.medoid_rows(ksum, tabs["page_base"], tabs["cluster_base"], medoid)
    assert np.array_equal(rows_gpu[: len(rows_ref)], rows_ref), "medoid index rows differ"
    sel_c, n_sel_c = sess.sel_clusters.cpu().numpy(), sess.n_sel_clusters.cpu().numpy()
    r = oracle.medoid_step(W.bits_u16(w.q), ksum, W.bits_u16(w.kv_pool), tabs["page_base"], tabs["ctx_len"],
                           tabs["page2cluster"], tabs["cluster_base"], tabs["replica_mask"], tabs["cluster_size"],
                           ptr, members, medoid, Hkv=cfg.n_kv_heads, S=cfg.page_size, k_c=k_c, D=cfg.n_queues,
                           flags=flags, sel_override=(sel_c, n_sel_c), window=window)
    cb = tabs["cluster_base"]
    exact = 0
    for b in range(cfg.batch):
        n_c = int(cb[b + 1] - cb[b])
        if sess.cluster_scores is not None:
            sc = sess.cluster_scores[b].cpu().numpy()
            parity.check_scores(sc, r.score64[b], r.cond[b], n_c)
            on_gpu_scores, _ = oracle.topk(sc[None, :, :n_c], np.array([n_c * cfg.page_size], np.int32),
                                           cfg.page_size, k_c)
            assert np.array_equal(on_gpu_scores[0], sel_c[b]), "not the exact top-k of the GPU's own cluster scores"
        for h in range(cfg.n_q_heads):
            parity.check_selection(sel_c[b, h], int(n_sel_c[b, h]), r.score64[b, h], n_c, k_c)
            exact += int(np.array_equal(sel_c[b, h], r.sel_clusters[b, h]))
    o = sess.o
    n = int(o.n_uniq.cpu().numpy()[0])
    assert n == len(r.uniq) and np.array_equal(o.uniq.cpu().numpy()[:n], r.uniq)
    assert np.array_equal(o.queue_of.cpu().numpy()[:n], r.queue_of)
    assert np.array_equal(o.queue_load.cpu().numpy()[: cfg.n_queues], r.load)
    parity.check_attention(o.out.cpu().numpy(), o.lse.cpu().numpy(), r.out, r.lse)
    return exact


@pytest.mark.parametrize("name,k_c", [("c1_small", 6), ("c2_small", 12), ("c3_small", 5), ("c4_small", 9),
                                      ("c5_small", 4), ("k_exceeds_pages", 7)])
def test_medoid_step_matches_oracle(name, k_c):
    w = W.generate(CASES[name], seed=37, device=DEV)
    sess = Session(w)
    sess.enable_medoid_index(k_c, keep_scores=True)
    sess.step_medoid()
    exact = check_medoid_step(w, sess, k_c)
    assert exact >= 0.9 * w.cfg.batch * w.cfg.n_q_heads
    # the page step still works on the same session afterwards, and the medoid step again after it
    sess.step()
    torch.cuda.synchronize()
    first = sess.sel_clusters.clone()
    sess.step_medoid()
    torch.cuda.synchronize()
    assert torch.equal(first, sess.sel_clusters)
    check_medoid_step(w, sess, k_c)
    sess.close()


def test_medoid_step_rejects_bad_arguments_and_flags_bad_members():
    w = W.generate(CASES["c3_small"], seed=41, device=DEV)
    sess = Session(w, keep_gathered=True)
    sess.enable_medoid_index(4)
    with pytest.raises(B.SwarmError):                       # gathered outputs are not part of this step
        B.swarm_step_medoid(sess.ctx, sess.inputs, sess.medoid_index, sess.outputs)
    bad = B.make_medoid_index(medoid_ksum=sess.medoid_ksum, cluster_page_ptr=sess.cluster_page_ptr,
                              cluster_pages=sess.cluster_pages, cluster_ctx_len=sess.cluster_ctx_len, top_k_clusters=0,
                              max_clusters_per_req=sess.max_clusters_per_req)
    with pytest.raises(B.SwarmError):
        B.swarm_step_medoid(sess.ctx, sess.inputs, bad, sess.medoid_outputs)
    sess.cluster_pages.fill_(1 << 20)                       # members outside every request: flagged, never followed
    sess.step_medoid()
    torch.cuda.synchronize()
    assert sess.status() & B.DEV_BAD_PAGE
    sess.cluster_page_ptr.fill_(1 << 40)                    # member offsets beyond the member array: skipped
    sess.step_medoid()
    torch.cuda.synchronize()
    assert sess.status() & B.DEV_BAD_CLUSTER
    sess.close()


def test_medoid_step_full_size_c2():
    w = W.generate(W.CONFIGS["c2_128k"], seed=43, device=DEV)
    sess = Session(w)
    sess.enable_medoid_index(32, keep_scores=True)          # 32 clusters of 8 pages: the page step's 256 pages per head
    sess.step_medoid()
    check_medoid_step(w, sess, 32)
    sess.close()


# ---- batched submission order (Sec. 5.1): heads of all buckets per batch -----------------------------------
def check_submit_order(w, sess, flags=0):
    torch.cuda.synchronize()
    tabs = parity.host_tables(w)
    n = int(sess.o.n_uniq.cpu().numpy()[0])
    uniq = sess.o.uniq.cpu().numpy()[:n]
    queue_of = sess.o.queue_of.cpu().numpy()[:n]
    want, rounds = oracle.submit_order(queue_of, tabs["replica_mask"][uniq], w.cfg.n_queues, flags)
    info = sess.submit_info.cpu().numpy()
    assert info[0] == rounds and info[1] == len(want)
    assert np.array_equal(sess.submit_order.cpu().numpy()[: len(want)], want)
    return len(want)


@pytest.mark.parametrize("flags", [0, B.ORDER_BY_ID])
@pytest.mark.parametrize("name", ["c2_small", "c3_small", "c5_small"])
def test_submit_order_matches_oracle(name, flags):
    w = W.generate(CASES[name], seed=47, device=DEV)
    sess = Session(w, flags=flags)
    sess.enable_submit_order()
    sess.step()
    parity.check_step(w, sess, flags=flags)
    assert check_submit_order(w, sess, flags) > 0
    sess.submit_order.fill_(-1)
    sess.select()
    sess.resolve()                                          # the separate call writes it too
    check_submit_order(w, sess, flags)
    sess.enable_medoid_index(5)
    sess.step_medoid()
    check_submit_order(w, sess, flags)
    B.swarm_set_submit_order(sess.ctx, None, None)          # detached: nothing is written any more
    sess.submit_order.fill_(-7)
    sess.step()
    torch.cuda.synchronize()
    assert int(sess.submit_order.max()) == -7
    sess.close()


def test_submit_order_full_size_and_bad_masks():
    w = W.generate(W.CONFIGS["c3_batched"], seed=53, device=DEV)     # 3071 clusters, half of them with two replicas
    sess = Session(w)
    sess.enable_submit_order()
    sess.step()
    assert check_submit_order(w, sess) > 2000
    w.cluster_replica_mask[::7] = 0                         # no replica anywhere: never submitted
    sess.step()
    torch.cuda.synchronize()
    assert sess.status() & B.DEV_BAD_REPLICA
    check_submit_order(w, sess)
    sess.close()


# ---- Algorithm 1 (offline co-activation clustering) ---------------------------------------------------------
def check_clusters(dist, tau, cap=None):
    density, ptr, members, medoid = B.swarm_build_clusters(dist, tau, members_cap=cap)
    torch.cuda.synchronize()
    d_host = dist.cpu().numpy()
    # the rule: every step agrees with Eq. 5's plain average (double, from scratch) outside a band of 1e-5 * tau
    # around the radius; where no decision falls inside the band the clustering is the plain oracle's exactly
    near = oracle.replay_clusters(d_host, tau, ptr.cpu().numpy(), members.cpu().numpy(), medoid.cpu().numpy(), near_rtol=1e-5)
    rho_p, ptr_p, members_p, medoid_p, near_p = oracle.build_clusters_plain(d_host, tau, members_cap=cap, near_rtol=1e-5)
    assert np.array_equal(density.cpu().numpy(), rho_p)
    if near == 0 and near_p == 0:
        assert np.array_equal(ptr.cpu().numpy(), ptr_p) and np.array_equal(members.cpu().numpy(), members_p)
        assert np.array_equal(medoid.cpu().numpy(), medoid_p)
    # and, beyond the rule, the fp32 reading of the oracle (running sum in joining order) bit for bit
    rho, ptr_ref, members_ref, medoid_ref = oracle.build_clusters(d_host, tau, members_cap=cap)
    assert np.array_equal(density.cpu().numpy(), rho)
    assert np.array_equal(medoid.cpu().numpy(), medoid_ref)
    assert np.array_equal(ptr.cpu().numpy(), ptr_ref)
    assert np.array_equal(members.cpu().numpy(), members_ref)
    return len(medoid_ref), len(members_ref)


@pytest.mark.parametrize("n,topics,tau", [(5, 1, 0.5), (37, 3, 0.4), (256, 8, 0.38), (1000, 20, 0.4),
                                          (1027, 12, 0.33), (2048, 64, 0.45), (3000, 30, 0.05), (600, 4, 1.0),
                                          (8192, 64, 0.4)])
def test_algorithm1_matches_oracle(n, topics, tau):
    dist = W.coactivation_distances(n, topics, seed=n, device=DEV)
    n_clusters, n_members = check_clusters(dist, tau, cap=64 * n if tau < 1.0 else None)
    assert n_members >= n and n_clusters >= 1
    if tau == 0.05:
        assert n_clusters == n                              # radius below every distance: singletons
    if tau == 1.0:
        assert n_clusters == 1 and n_members == n           # radius above every distance: one cluster


def test_algorithm1_hand_case_and_capacity():
    d = np.full((5, 5), 0.9, dtype=np.float32)
    np.fill_diagonal(d, 0.0)
    for (i, j), v in {(0, 1): 0.1, (0, 2): 0.2, (1, 2): 0.3, (3, 4): 0.1, (2, 3): 0.4, (2, 4): 0.5}.items():
        d[i, j] = d[j, i] = v
    dist = torch.from_numpy(d).to(DEV)
    density, ptr, members, medoid = B.swarm_build_clusters(dist, 0.5)
    assert density.tolist() == [2, 2, 4, 2, 2] and ptr.tolist() == [0, 3, 6]
    assert members.tolist() == [2, 0, 1, 3, 4, 2] and medoid.tolist() == [2, 3]
    with pytest.raises(B.SwarmError):                       # six memberships do not fit five slots
        B.swarm_build_clusters(dist, 0.5, members_cap=5)
    with pytest.raises(B.SwarmError):
        B.swarm_build_clusters(dist, -1.0)


def test_algorithm1_clusters_drive_the_medoid_step():
    """Clusters with replicas built on the GPU from a distance matrix, then used as the index of the medoid step."""
    cfg = small("c2_128k", ctx_len=16 * 640, top_k=32, n_topics=8)
    w = W.generate(cfg, seed=59, device=DEV)
    P = cfg.max_pages()
    dist = W.coactivation_distances(P, 16, seed=61, device=DEV)
    density, ptr, members, medoid = B.swarm_build_clusters(dist, 0.4, members_cap=64 * P)
    C = len(medoid)
    assert len(members) > P                                 # some pages sit in several clusters
    # cluster tables of the workload replaced by the ones just built (one request)
    sizes = (ptr[1:] - ptr[:-1]).to(torch.int16)
    rng = np.random.default_rng(3)
    mask = torch.from_numpy(np.array([(1 << int(a)) | (1 << int(b)) for a, b in
                                      zip(rng.integers(0, 8, C), rng.integers(0, 8, C))], dtype=np.int32)).to(DEV)
    w.cluster_base = torch.tensor([0, C], dtype=torch.int64, device=DEV)
    w.cluster_replica_mask, w.cluster_size = mask, sizes
    w.page2cluster = torch.zeros(P, dtype=torch.int32, device=DEV)      # not read by the medoid step
    sess = Session(w)
    k_c = 6
    sess.cluster_page_ptr, sess.cluster_pages, sess.medoid_page = ptr.to(torch.int64), members, medoid
    sess.max_clusters_per_req = C
    sess.medoid_ksum = torch.empty((C, cfg.n_kv_heads, 2, cfg.head_dim), dtype=torch.bfloat16, device=DEV)
    sess.cluster_ctx_len = torch.empty(4, dtype=torch.int32, device=DEV)
    B.swarm_build_medoid_index(sess.ctx, sess.inputs, medoid, sess.medoid_ksum, sess.cluster_ctx_len)
    sess.medoid_index = B.make_medoid_index(medoid_ksum=sess.medoid_ksum, cluster_page_ptr=sess.cluster_page_ptr,
                                            cluster_pages=members, cluster_ctx_len=sess.cluster_ctx_len,
                                            top_k_clusters=k_c, max_clusters_per_req=C)
    i32 = dict(dtype=torch.int32, device=DEV)
    sess.sel_clusters = torch.empty((1, cfg.n_q_heads, k_c), **i32)
    sess.n_sel_clusters = torch.empty((1, cfg.n_q_heads), **i32)
    sess.cluster_scores = None
    o = sess.o
    sess.medoid_outputs = B.make_outputs(sel=sess.sel_clusters, n_sel=sess.n_sel_clusters, uniq=o.uniq,
                                         queue_of=o.queue_of, n_uniq=o.n_uniq, queue_load=o.queue_load, out=o.out,
                                         lse=o.lse)
    sess.step_medoid()
    torch.cuda.synchronize()
    assert sess.status() == 0
    # oracle: scores/top-k over the medoids, union of the members, scheduling of the selected clusters
    tabs = parity.host_tables(w)
    ksum = W.bits_u16(sess.ksum)
    rows = oracle.medoid_rows(ksum, tabs["page_base"], tabs["cluster_base"], medoid.cpu().numpy())
    len_c = np.array([C * cfg.page_size], np.int32)
    s64, s32, cond = oracle.scores(W.bits_u16(w.q), rows, tabs["cluster_base"], len_c, cfg.n_kv_heads, cfg.page_size, C)
    sel_c, n_sel_c = sess.sel_clusters.cpu().numpy(), sess.n_sel_clusters.cpu().numpy()
    for h in range(cfg.n_q_heads):
        parity.check_selection(sel_c[0, h], int(n_sel_c[0, h]), s64[0, h], C, k_c)
    sel_p, n_sel_p = oracle.expand_clusters(sel_c, n_sel_c, tabs["cluster_base"], ptr.cpu().numpy(), members.cpu().numpy())
    ident = np.arange(C, dtype=np.int32)                     # scheduling sees the selected clusters themselves
    uniq, queue_of, load = oracle.resolve(sel_c, n_sel_c, tabs["cluster_base"], ident, tabs["cluster_base"],
                                          tabs["replica_mask"], tabs["cluster_size"], cfg.n_queues, 0)
    n = int(o.n_uniq.cpu().numpy()[0])
    assert n == len(uniq) and np.array_equal(o.uniq.cpu().numpy()[:n], uniq)
    assert np.array_equal(o.queue_of.cpu().numpy()[:n], queue_of)
    assert np.array_equal(o.queue_load.cpu().numpy()[: cfg.n_queues], load)
    k_g, v_g, n_tok = oracle.gather(W.bits_u16(w.kv_pool), sel_p, n_sel_p, tabs["page_base"], tabs["ctx_len"],
                                    cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    out, lse = oracle.attention(W.bits_u16(w.q), k_g, v_g, n_tok)
    parity.check_attention(o.out.cpu().numpy(), o.lse.cpu().numpy(), out, lse)
    sess.close()

    # entry-level scheduling (the paper's exact model): every page of the selected clusters is a unit of its own,
    # with the copies Eq. 7 gives it -- one per cluster that stores it
    entry_masks = oracle.entry_replica_masks(ptr.cpu().numpy(), members.cpu().numpy(), P, cfg.n_queues)
    assert (np.array([bin(int(x)).count("1") for x in entry_masks]) > 1).any()
    sess = Session(w, max_clusters_total=P)
    sess.medoid_ksum = torch.empty((C, cfg.n_kv_heads, 2, cfg.head_dim), dtype=torch.bfloat16, device=DEV)
    len_dev = torch.empty(4, dtype=torch.int32, device=DEV)
    B.swarm_build_medoid_index(sess.ctx, sess.inputs, medoid, sess.medoid_ksum, len_dev)
    masks_dev = torch.from_numpy(entry_masks.view(np.int32)).to(DEV)
    ptr64 = ptr.to(torch.int64)                               # kept alive: the index holds its address
    index = B.make_medoid_index(medoid_ksum=sess.medoid_ksum, cluster_page_ptr=ptr64, cluster_pages=members,
                                cluster_ctx_len=len_dev,
                                top_k_clusters=k_c, max_clusters_per_req=C, entry_replica_mask=masks_dev)
    sel_c2 = torch.empty((1, cfg.n_q_heads, k_c), **i32)
    n_sel_c2 = torch.empty((1, cfg.n_q_heads), **i32)
    o = sess.o
    outs = B.make_outputs(sel=sel_c2, n_sel=n_sel_c2, uniq=o.uniq, queue_of=o.queue_of, n_uniq=o.n_uniq,
                          queue_load=o.queue_load, out=o.out, lse=o.lse)
    sess.enable_submit_order()
    B.swarm_step_medoid(sess.ctx, sess.inputs, index, outs)
    torch.cuda.synchronize()
    assert sess.status() == 0
    assert np.array_equal(sel_c2.cpu().numpy(), sel_c)        # same selection as before
    ones = np.ones(P, dtype=np.uint16)
    ident_p = np.arange(P, dtype=np.int32)
    uniq, queue_of, load = oracle.resolve(sel_p, n_sel_p, tabs["page_base"], ident_p, tabs["page_base"], entry_masks, ones,
                                          cfg.n_queues, oracle.UNIT_LOAD)
    n = int(o.n_uniq.cpu().numpy()[0])
    assert n == len(uniq) and np.array_equal(o.uniq.cpu().numpy()[:n], uniq)
    assert np.array_equal(o.queue_of.cpu().numpy()[:n], queue_of)
    assert np.array_equal(o.queue_load.cpu().numpy()[: cfg.n_queues], load) and int(load.sum()) == n
    want_order, rounds = oracle.submit_order(queue_of, entry_masks[uniq], cfg.n_queues)
    assert np.array_equal(sess.submit_order.cpu().numpy()[:n], want_order)
    parity.check_attention(o.out.cpu().numpy(), o.lse.cpu().numpy(), out, lse)
    sess.close()


@pytest.mark.parametrize("name,k_c,window", [("c2_small", 12, 3), ("c5_small", 4, 2), ("k_exceeds_pages", 7, 5),
                                             ("c4_small", 9, 64), ("c3_small", 1, 40)])
def test_medoid_step_with_local_window(name, k_c, window):
    """The paper's whole Tier-1 step: clusters chosen through the medoid index, attended whole, plus the local
    window (requests shorter than the window are attended densely)."""
    cfg = CASES[name]
    window = min(window, cfg.top_k)                         # the shape allows 0 <= W <= top_k
    w = W.generate(cfg, seed=83, device=DEV)
    sess = Session(w, local_window_pages=window)
    sess.enable_medoid_index(k_c, keep_scores=True)
    sess.step_medoid()
    check_medoid_step(w, sess, k_c, window=window)
    sess.step()                                             # the page step with the same window still works
    parity.check_step(w, sess)
    sess.step_medoid()
    check_medoid_step(w, sess, k_c, window=window)
    sess.close()


def test_medoid_step_entry_level_with_local_window():
    """Entry-level scheduling: the window's pages are units of their own, like the members of the selected clusters."""
    cfg = small("c2_128k", ctx_len=16 * 300 + 7, top_k=32, n_topics=6)
    window = 5
    w = W.generate(cfg, seed=89, device=DEV)
    P = cfg.max_pages()
    ptr, members, medoid = W.cluster_members(w)
    entry_masks = oracle.entry_replica_masks(ptr.cpu().numpy(), members.cpu().numpy(), P, cfg.n_queues)
    # give every third page a second copy so that the scheduling has something to decide
    entry_masks = entry_masks.copy()
    entry_masks[::3] |= np.uint32(1) << ((np.arange(P)[::3] // 3) % cfg.n_queues).astype(np.uint32)
    sess = Session(w, local_window_pages=window, max_clusters_total=P)
    sess.enable_medoid_index(4)
    masks_dev = torch.from_numpy(entry_masks.view(np.int32)).to(DEV)
    index = B.make_medoid_index(medoid_ksum=sess.medoid_ksum, cluster_page_ptr=sess.cluster_page_ptr,
                                cluster_pages=sess.cluster_pages, cluster_ctx_len=sess.cluster_ctx_len, top_k_clusters=4,
                                max_clusters_per_req=sess.max_clusters_per_req, entry_replica_mask=masks_dev)
    B.swarm_step_medoid(sess.ctx, sess.inputs, index, sess.medoid_outputs)
    torch.cuda.synchronize()
    assert sess.status() == 0
    tabs = parity.host_tables(w)
    sel_c, n_sel_c = sess.sel_clusters.cpu().numpy(), sess.n_sel_clusters.cpu().numpy()
    sel_p, n_sel_p = oracle.expand_clusters(sel_c, n_sel_c, tabs["cluster_base"], ptr.cpu().numpy(), members.cpu().numpy(),
                                            tabs["ctx_len"], cfg.page_size, window)
    assert all(set(range(P - window, P)) <= set(sel_p[0, h, : n_sel_p[0, h]].tolist()) for h in range(cfg.n_q_heads))
    uniq, queue_of, load = oracle.resolve(sel_p, n_sel_p, tabs["page_base"], np.arange(P, dtype=np.int32), tabs["page_base"],
                                          entry_masks, np.ones(P, dtype=np.uint16), cfg.n_queues, oracle.UNIT_LOAD)
    o = sess.o
    n = int(o.n_uniq.cpu().numpy()[0])
    assert n == len(uniq) and np.array_equal(o.uniq.cpu().numpy()[:n], uniq)
    assert np.array_equal(o.queue_of.cpu().numpy()[:n], queue_of)
    assert np.array_equal(o.queue_load.cpu().numpy()[: cfg.n_queues], load)
    k_g, v_g, n_tok = oracle.gather(W.bits_u16(w.kv_pool), sel_p, n_sel_p, tabs["page_base"], tabs["ctx_len"],
                                    cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    out, lse = oracle.attention(W.bits_u16(w.q), k_g, v_g, n_tok)
    parity.check_attention(o.out.cpu().numpy(), o.lse.cpu().numpy(), out, lse)
    sess.close()


def test_medoid_step_full_size_c3_and_wide_groups():
    w = W.generate(W.CONFIGS["c3_batched"], seed=67, device=DEV)      # 16 requests, 256 clusters each
    sess = Session(w)
    sess.enable_medoid_index(16, keep_scores=True)
    sess.step_medoid()
    check_medoid_step(w, sess, 16)
    sess.close()
    for name in ("g16_s32", "hkv3_g2", "k1_d1"):                      # 16-head groups on 32-token pages, odd KV heads, one queue
        w = W.generate(EDGE_SHAPES[name], seed=71, device=DEV)
        sess = Session(w)
        sess.enable_medoid_index(3, keep_scores=True)
        sess.step_medoid()
        check_medoid_step(w, sess, 3)
        sess.close()


# ---- admission of clusters to the fast tier by their Eq. 6 score -------------------------------------------
@pytest.mark.parametrize("n,cap_frac", [(5, 0.7), (200, 0.3), (1024, 0.5), (3000, 0.25), (5000, 0.0), (5000, 2.0)])
def test_cache_admission_matches_oracle(n, cap_frac):
    g = torch.Generator(device="cpu").manual_seed(n)
    score = torch.randint(0, 40, (n,), generator=g).to(torch.float32) * 0.25      # many ties
    size = torch.randint(1, 17, (n,), generator=g, dtype=torch.int16)
    cap = int(cap_frac * int(size.sum()))
    resident = torch.full((n + 16,), 7, dtype=torch.uint8, device=DEV)
    info = torch.zeros(4, dtype=torch.int32, device=DEV)
    B.swarm_cache_admit(score.to(DEV), size.to(DEV), cap, resident, info)
    torch.cuda.synchronize()
    want, n_in, used = oracle.cache_admit(score.numpy(), size.numpy().view(np.uint16), cap)
    assert np.array_equal(resident.cpu().numpy()[:n], want) and int(resident[n:].min()) == 7
    assert info.cpu().numpy()[:2].tolist() == [n_in, used]


def test_cache_admission_feeds_the_resident_filter():
    """Scores maintained by the step (Eq. 6) -> admission -> the next step fetches only what is not resident."""
    w = W.generate(CASES["c3_small"], seed=73, device=DEV)
    sess = Session(w)
    C = w.n_clusters
    resident = torch.zeros(C + 16, dtype=torch.uint8, device=DEV)
    freq = torch.zeros(C, dtype=torch.int32, device=DEV)
    score = torch.zeros(C, dtype=torch.float32, device=DEV)
    n_hit = torch.zeros(4, dtype=torch.int32, device=DEV)
    B.swarm_set_cache(sess.ctx, resident=resident, freq=freq, score=score, n_hit=n_hit, t_base=80.0, t_transfer=2.5)
    sess.step()                                             # nothing resident yet: every activated cluster scores
    torch.cuda.synchronize()
    n_first = int(sess.o.n_uniq[0])
    assert int(n_hit[0]) == 0 and int((freq > 0).sum()) == n_first
    B.swarm_cache_admit(score, w.cluster_size, 10_000_000, resident)       # room for everything with a score
    want, _, _ = oracle.cache_admit(score.cpu().numpy(), w.cluster_size.cpu().numpy().view(np.uint16), 10_000_000)
    assert np.array_equal(resident.cpu().numpy()[:C], want) and want.all()
    sess.step()                                             # same query: everything activated is resident now
    torch.cuda.synchronize()
    assert int(sess.o.n_uniq[0]) == 0 and int(n_hit[0]) == n_first
    sess.close()


# ---- the selector report: its figures recomputed on the host in fp64 from the selectors' own lists -------------
@pytest.mark.parametrize("name,k_c", [("c2_small", 12), ("c5_small", 4)])
def test_selector_report_figures(name, k_c):
    from helpers import from_bf16_bits
    from paper_2603_17803_b200 import selector_report as R
    w = W.generate(CASES[name], seed=79, device=DEV)
    rep = R.compare(w, k_c, keep_lists=True)
    cfg, tabs = w.cfg, parity.host_tables(w)
    S, d, g = cfg.page_size, cfg.head_dim, cfg.n_q_heads // cfg.n_kv_heads
    q = from_bf16_bits(W.bits_u16(w.q)).astype(np.float64)
    pool = W.bits_u16(w.kv_pool)
    ptr, members, _ = (t.cpu().numpy() for t in W.cluster_members(w))
    for sel_name in ("pages", "medoids"):
        lists, n_lists = rep[sel_name]["lists"]
        if sel_name == "medoids":                           # the pages those clusters hold
            sel_p, n_p = oracle.expand_clusters(lists, n_lists, tabs["cluster_base"], ptr, members)
        else:
            sel_p, n_p = lists, n_lists
        att_n, mass_r, top_r = [], [], []
        for b in range(cfg.batch):
            ctx = int(tabs["ctx_len"][b])
            P = -(-ctx // S)
            pb = int(tabs["page_base"][b])
            for h in range(cfg.n_q_heads):
                keys = from_bf16_bits(pool[pb:pb + P, h // g, 0]).astype(np.float64).reshape(P * S, d)
                logit = keys @ q[b, h] / np.sqrt(d)
                logit[ctx:] = -np.inf
                prob = np.exp(logit - logit.max())
                mass = (prob / prob.sum()).reshape(P, S).sum(1)
                pages = sel_p[b, h, : n_p[b, h]]
                att_n.append(len(pages))
                mass_r.append(mass[pages].sum())
                best = np.argsort(-mass, kind="stable")[: min(cfg.top_k, P)]
                top_r.append(np.isin(best, pages).mean())
        got = rep[sel_name]
        assert got["attended_pages"] == pytest.approx(np.mean(att_n), rel=1e-6)
        assert got["mass_recall"] == pytest.approx(np.mean(mass_r), abs=2e-4)
        assert got["topk_recall"] == pytest.approx(np.mean(top_r), abs=5e-3)     # near-ties of mass order differently in fp32
        uniq, _, load = oracle.resolve(sel_p, n_p, tabs["page_base"], tabs["page2cluster"], tabs["cluster_base"],
                                       tabs["replica_mask"], tabs["cluster_size"], cfg.n_queues)
        assert got["io_clusters"] == len(uniq) and got["io_pages"] == int(tabs["cluster_size"][uniq].sum())
        assert got["io_pages"] == int(load.sum()) and got["max_queue_load"] == int(load.max())
    # whole clusters attended: the medoid selector's I/O is exactly what its heads attend, no partial clusters
    assert rep["medoids"]["io_pages"] >= rep["medoids"]["attended_pages"]


# ---- the step in two halves: query heads spread over several ctxs (one per GPU in production) ------------------
def test_begin_then_end_is_the_step():
    w = W.generate(CASES["c5_small"], seed=97, device=DEV)
    a, b_ = Session(w), Session(w)
    a.step()
    b_.step_begin()
    flags = b_.cluster_flags()
    assert flags.numel() == w.n_clusters and int(flags.sum()) == int(a.o.n_uniq[0])   # every activated cluster, once
    b_.step_end()
    torch.cuda.synchronize()
    assert int(flags.sum()) == 0                            # consumed
    for name in ("sel", "n_sel", "queue_load", "out", "lse"):
        assert torch.equal(getattr(a.o, name), getattr(b_.o, name)), name
    n = int(a.o.n_uniq[0])
    assert torch.equal(a.o.uniq[:n], b_.o.uniq[:n]) and torch.equal(a.o.queue_of[:n], b_.o.queue_of[:n])
    parity.check_step(w, b_)
    a.close()
    b_.close()


@pytest.mark.parametrize("name,world", [("c2_small", 2), ("c2_small", 4), ("c3_small", 8), ("c5_small", 2)])
def test_head_sharded_step_on_one_device(name, world):
    """`world` ctxs, each with the K/V of its own KV heads, run one after the other on this device; the flag
    exchange (an all-reduce by maximum across GPUs in production) is a plain maximum here.  Every shard must
    derive the unsharded schedule, and the shards' heads together the unsharded selection and attention."""
    from paper_2603_17803_b200 import sharding
    w = W.generate(CASES[name], seed=101, device=DEV)
    full = Session(w)
    full.step()
    parity.check_step(w, full)
    shards = [sharding.shard_workload(w, r, world) for r in range(world)]
    sess = [Session(s, ksum=None) for s in shards]
    for s in sess:
        s.step_begin()
    torch.cuda.synchronize()
    own = [int(s.cluster_flags().sum()) for s in sess]
    union = torch.stack([s.cluster_flags() for s in sess]).amax(0)
    n = int(full.o.n_uniq[0])
    assert int(union.sum()) == n and max(own) <= n
    for s in sess:
        s.cluster_flags().copy_(union)
        s.step_end()
    torch.cuda.synchronize()
    hq = w.cfg.n_q_heads // world
    for r, s in enumerate(sess):
        assert s.status() == 0
        assert int(s.o.n_uniq[0]) == n
        assert torch.equal(s.o.uniq[:n], full.o.uniq[:n]) and torch.equal(s.o.queue_of[:n], full.o.queue_of[:n])
        assert torch.equal(s.o.queue_load[: w.cfg.n_queues], full.o.queue_load[: w.cfg.n_queues])
        assert torch.equal(s.o.sel, full.o.sel[:, r * hq:(r + 1) * hq])
        d_out = (s.o.out - full.o.out[:, r * hq:(r + 1) * hq]).abs().max().item()
        d_lse = (s.o.lse - full.o.lse[:, r * hq:(r + 1) * hq]).abs().max().item()
        assert d_out <= parity.ATTN_ATOL and d_lse <= parity.LSE_ATOL   # split counts differ between the layouts
        assert int(s.cluster_flags().sum()) == 0
    # sharding.sharded_step without a process group is the plain step
    sharding.sharded_step(sess[0])
    torch.cuda.synchronize()
    parity.check_step(shards[0], sess[0])
    for s in sess:
        s.close()
    full.close()
