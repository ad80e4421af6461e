"""swarm_sparse_attn_static: the attention entry point for callers that cannot allocate device memory
(for instance a plugin running inside another framework's allocator callback, or a process with a fixed,
fully reserved memory budget).  Its split-K scratch is a fixed array inside the library, so the test checks
(1) that it reproduces swarm_sparse_attn, (2) on two calls in a row, because the array is shared and keeps
the previous call's contents, and (3) that it refuses problems larger than the array.
Collected last on purpose: a failure here must not hide the other tests in a run that stops at the first one."""
import pytest
import torch

from paper_2603_17803_b200 import binding as B
from paper_2603_17803_b200 import workloads as W
from paper_2603_17803_b200.session import Session

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 1e-4     # the tolerance the fused-step test uses between two launch configurations of the same kernel


def gathered_case(cfg, seed):
    w = W.generate(cfg, seed=seed, device=DEV)
    sess = Session(w, keep_gathered=True)
    sess.select()
    sess.gather()
    sess.sparse_attn()                      # existing entry point: the expected values
    torch.cuda.synchronize()
    return w, sess


@pytest.mark.parametrize("base,kw", [
    ("c2_128k", dict(ctx_len=16 * 1200 + 3, top_k=80, n_topics=8)),
    ("c4_long", dict(batch=2, ctx_len=32 * 500 + 11, top_k=48, n_topics=8)),
])
def test_static_variant_matches_workspace_variant_twice_in_a_row(base, kw):
    cfg = W.scaled(W.CONFIGS[base], **kw)
    w, sess = gathered_case(cfg, seed=21)
    shape = dict(batch=cfg.batch, n_q_heads=cfg.n_q_heads, top_k=cfg.top_k, page_size=cfg.page_size)
    out = torch.full_like(sess.o.out, float("nan"))
    lse = torch.full_like(sess.o.lse, float("nan"))
    B.swarm_sparse_attn_static(w.q, sess.o.k_out, sess.o.v_out, sess.o.n_tok, out=out, lse=lse, **shape)
    torch.cuda.synchronize()
    assert (out - sess.o.out).abs().max().item() <= TOL
    assert (lse - sess.o.lse).abs().max().item() <= TOL

    # second call right after the first, other data: stale partials of call one must not leak into call two
    q2 = (w.q.float() * -0.5 + 0.25).to(torch.bfloat16)
    sess.set_query(q2)
    sess.sparse_attn()
    torch.cuda.synchronize()
    out2 = torch.full_like(out, float("nan"))
    lse2 = torch.full_like(lse, float("nan"))
    B.swarm_sparse_attn_static(q2, sess.o.k_out, sess.o.v_out, sess.o.n_tok, out=out2, lse=lse2, **shape)
    torch.cuda.synchronize()
    assert (out2 - sess.o.out).abs().max().item() <= TOL
    assert (lse2 - sess.o.lse).abs().max().item() <= TOL
    assert (out2 - out).abs().max().item() > 1e-3          # the two calls really differ
    sess.close()


def test_static_variant_across_shapes_and_split_counts_allocates_nothing():
    """Calls of different shapes one after the other on the same stream: 8 heads (18 key-range splits on 148 SMs),
    then 32 heads (4 splits), then 128 heads (1 split), then 8 heads again.  The array is shared, so slots and
    arrival counters left by one shape are what the next one finds.  No device memory may be allocated by the
    calls (this entry point exists for callers that cannot allocate), and the status word stays clear."""
    cases = []
    for base, kw in [("c2_128k", dict(n_q_heads=8, n_kv_heads=2, ctx_len=16 * 900 + 5, top_k=72, n_topics=6)),
                     ("c2_128k", dict(ctx_len=16 * 640, top_k=40, n_topics=8)),
                     ("c4_long", dict(batch=2, ctx_len=32 * 300 + 1, top_k=24, n_topics=8)),
                     ("c2_128k", dict(n_q_heads=8, n_kv_heads=2, ctx_len=16 * 300, top_k=16, n_topics=4))]:
        cfg = W.scaled(W.CONFIGS[base], **kw)
        w, sess = gathered_case(cfg, seed=23)
        cases.append((cfg, w, sess, torch.full_like(sess.o.out, float("nan")), torch.full_like(sess.o.lse, float("nan"))))
    B.swarm_sparse_attn_static_status()                     # set-up for this device done, word cleared
    torch.cuda.synchronize()
    free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    for cfg, w, sess, out, lse in cases:
        B.swarm_sparse_attn_static(w.q, sess.o.k_out, sess.o.v_out, sess.o.n_tok, batch=cfg.batch, n_q_heads=cfg.n_q_heads,
                                   top_k=cfg.top_k, page_size=cfg.page_size, out=out, lse=lse)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
    for cfg, w, sess, out, lse in cases:
        assert (out - sess.o.out).abs().max().item() <= TOL
        assert (lse - sess.o.lse).abs().max().item() <= TOL
    assert B.swarm_sparse_attn_static_status() == 0
    for c in cases:
        c[2].close()


def test_static_variant_reports_a_token_count_beyond_the_buffer():
    """n_tok larger than top_k * page_size: the kernel attends the rows the buffer holds, and says so in the
    status word that swarm_sparse_attn_static_status reads and clears (no fault is provoked: every access
    stays inside the buffers)."""
    cfg = W.scaled(W.CONFIGS["c2_128k"], n_q_heads=8, n_kv_heads=2, ctx_len=16 * 200, top_k=16, n_topics=4)
    w, sess = gathered_case(cfg, seed=25)
    shape = dict(batch=cfg.batch, n_q_heads=cfg.n_q_heads, top_k=cfg.top_k, page_size=cfg.page_size)
    B.swarm_sparse_attn_static_status()
    n_bad = sess.o.n_tok.clone()
    n_bad[0, 3] = cfg.top_k * cfg.page_size + 77
    out, lse = torch.full_like(sess.o.out, float("nan")), torch.full_like(sess.o.lse, float("nan"))
    B.swarm_sparse_attn_static(w.q, sess.o.k_out, sess.o.v_out, n_bad, out=out, lse=lse, **shape)
    assert B.swarm_sparse_attn_static_status() == B.DEV_BAD_LENGTH
    assert B.swarm_sparse_attn_static_status() == 0         # cleared by the read
    # every slot of that head is full here, so the clamped length is the true one
    assert int(sess.o.n_tok[0, 3]) == cfg.top_k * cfg.page_size
    assert (out - sess.o.out).abs().max().item() <= TOL and (lse - sess.o.lse).abs().max().item() <= TOL
    # the workspace variant flags it the same way
    sess.o.n_tok[0, 3] = cfg.top_k * cfg.page_size + 1
    sess.sparse_attn()
    assert sess.status() == B.DEV_BAD_LENGTH
    sess.close()


def test_static_variant_rejects_what_does_not_fit():
    t = torch.zeros(64, dtype=torch.int32, device=DEV)
    f = torch.zeros(64, dtype=torch.float32, device=DEV)
    with pytest.raises(B.SwarmError) as e:
        B.swarm_sparse_attn_static(t, t, t, t, batch=B.STATIC_MAX_HEADS // 8 + 1, n_q_heads=8, top_k=4, page_size=16,
                                   out=f, lse=f)
    assert e.value.code == B.ERR_STATIC_SCRATCH_TOO_SMALL
    with pytest.raises(B.SwarmError) as e:
        B.swarm_sparse_attn_static(t, t, t, t, batch=1, n_q_heads=8, top_k=4, page_size=8, out=f, lse=f)
    assert e.value.code == B.ERR_UNSUPPORTED
