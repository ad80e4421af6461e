"""Pins for the CPU oracle: closed forms, invariants, library routines on special cases, hand-worked
fixtures and brute force on tiny inputs.  None of these re-types the oracle's own loops: each check is a
property a dropped term, a wrong sign, a wrong index or a transposed operand would break."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_round, from_bf16_bits, identity_layout, to_bf16_bits

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, vals = line.split(":")
            out[key.strip()] = [float(v) for v in vals.split()]
    return out


def rand_case(rng, B=2, Hq=4, Hkv=2, d=16, S=4, pages=(5, 7), ctx=None):
    """Random pool with summaries from the oracle; returns float views too."""
    page_base, ctx_len = identity_layout(pages, S, ctx)
    n = int(page_base[-1])
    pool = to_bf16_bits(rng.standard_normal((n, Hkv, 2, S, d)))
    q = to_bf16_bits(rng.standard_normal((B, Hq, d)))
    ksum = oracle.build_summaries(pool, page_base, ctx_len, Hkv, d, S)
    return q, pool, ksum, page_base, ctx_len


# ----------------------------------------------------------------------------------------- summaries

def test_summaries_match_numpy_minmax_and_ignore_padding():
    rng = np.random.default_rng(1)
    S, d, Hkv = 4, 8, 2
    page_base, ctx_len = identity_layout([3, 2], S, ctx=[3 * S - 2, 2 * S])  # request 0: last page has 2 valid
    pool = to_bf16_bits(rng.standard_normal((5, Hkv, 2, S, d)))
    poisoned = pool.copy()
    poisoned[2, :, 0, 2:, :] = to_bf16_bits(np.full((Hkv, 2, d), 1000.0))    # padding tokens of request 0
    ksum = oracle.build_summaries(poisoned, page_base, ctx_len, Hkv, d, S)
    K = from_bf16_bits(pool)[:, :, 0]                                        # [page][kv][S][d]
    for page in range(5):
        valid = 2 if page == 2 else S
        lo = K[page, :, :valid].min(axis=1)
        hi = K[page, :, :valid].max(axis=1)
        assert np.array_equal(from_bf16_bits(ksum[page, :, 0]), lo)
        assert np.array_equal(from_bf16_bits(ksum[page, :, 1]), hi)
    # the V half of the pool must not influence the summaries
    poisoned[:, :, 1] = to_bf16_bits(np.full((5, Hkv, S, d), -777.0))
    assert np.array_equal(oracle.build_summaries(poisoned, page_base, ctx_len, Hkv, d, S), ksum)


# -------------------------------------------------------------------------------------------- scores

def test_score_hand_case():
    g = read_golden("score_hand_case.txt")
    q = to_bf16_bits(np.array(g["q"]).reshape(1, 1, 4))
    ksum = to_bf16_bits(np.array([g["kmin"], g["kmax"]]).reshape(1, 1, 2, 4))
    s64, s32, cond = oracle.scores(q, ksum, [0, 1], [1], Hkv=1, S=1, Pmax=1)
    assert s64[0, 0, 0] == g["score"][0] and s32[0, 0, 0] == g["score"][0]
    assert cond[0, 0, 0] == 3 + 2 + 2 + 5


def test_score_is_upper_bound_on_every_token_and_is_attained():
    rng = np.random.default_rng(2)
    q, pool, ksum, page_base, ctx_len = rand_case(rng)
    B, Hq, d = q.shape
    Hkv, S = 2, 4
    s64, _, _ = oracle.scores(q, ksum, page_base, ctx_len, Hkv, S, Pmax=7)
    qf, K = from_bf16_bits(q), from_bf16_bits(pool)[:, :, 0]
    lo, hi = from_bf16_bits(ksum[:, :, 0]), from_bf16_bits(ksum[:, :, 1])
    for b in range(B):
        P = int(page_base[b + 1] - page_base[b])
        for h in range(Hq):
            kv = h // (Hq // Hkv)
            for p in range(P):
                page = int(page_base[b]) + p
                dots = K[page, kv] @ qf[b, h]                          # every token's true logit (numpy matmul)
                assert dots.max() <= s64[b, h, p] + 1e-9
                kstar = np.where(qf[b, h] > 0, hi[page, kv], lo[page, kv])  # the box corner that attains it
                assert s64[b, h, p] == pytest.approx(float(kstar @ qf[b, h]), rel=1e-12, abs=1e-12)
            assert np.all(np.isneginf(s64[b, h, P:]))                  # pages that do not exist stay untouched


def test_score_single_token_page_is_plain_dot_product():
    rng = np.random.default_rng(3)
    S, d, Hkv = 4, 16, 2
    # request with 2 full pages + a last page holding exactly one valid token
    q, pool, ksum, page_base, ctx_len = rand_case(rng, B=1, Hq=4, Hkv=Hkv, d=d, S=S, pages=(3,), ctx=[2 * S + 1])
    s64, _, _ = oracle.scores(q, ksum, page_base, ctx_len, Hkv, S, Pmax=3)
    qf, K = from_bf16_bits(q), from_bf16_bits(pool)[:, :, 0]
    for h in range(4):
        assert s64[0, h, 2] == pytest.approx(float(np.dot(qf[0, h], K[2, h // 2, 0])), rel=1e-12, abs=1e-12)


def test_score_sign_cases_and_split_identity_and_homogeneity():
    rng = np.random.default_rng(4)
    q, pool, ksum, page_base, ctx_len = rand_case(rng, B=1, Hq=2, Hkv=1, d=32, S=4, pages=(6,))
    lo, hi = from_bf16_bits(ksum[:, 0, 0]), from_bf16_bits(ksum[:, 0, 1])
    qf = from_bf16_bits(q)
    qpos, qneg = to_bf16_bits(np.abs(qf)), to_bf16_bits(-np.abs(qf))
    s_pos, _, _ = oracle.scores(qpos, ksum, page_base, ctx_len, 1, 4, 6)
    s_neg, _, _ = oracle.scores(qneg, ksum, page_base, ctx_len, 1, 4, 6)
    s, _, cond = oracle.scores(q, ksum, page_base, ctx_len, 1, 4, 6)
    for h in range(2):
        a = np.abs(qf[0, h])
        assert np.allclose(s_pos[0, h], hi @ a, rtol=1e-12, atol=1e-12)       # q >= 0  ->  q . kmax
        assert np.allclose(s_neg[0, h], -(lo @ a), rtol=1e-12, atol=1e-12)    # q <= 0  ->  q . kmin
        plus, minus = np.maximum(qf[0, h], 0), np.maximum(-qf[0, h], 0)
        assert np.allclose(s[0, h], hi @ plus - lo @ minus, rtol=1e-12, atol=1e-12)
        assert np.all(cond[0, h] >= np.abs(s[0, h]) - 1e-12)
    s2, _, _ = oracle.scores(to_bf16_bits(2 * qf), ksum, page_base, ctx_len, 1, 4, 6)
    assert np.array_equal(s2, 2 * s)                                         # scaling by 2 is exact


def test_score_gqa_mapping_and_request_offsets():
    # kv head j of request b carries the constant key (10*b + j + 1); score = that constant * sum(q)
    B, Hq, Hkv, d, S = 2, 6, 3, 8, 2
    page_base, ctx_len = identity_layout([2, 3], S)
    ksum = np.zeros((5, Hkv, 2, d))
    for b in range(B):
        for j in range(Hkv):
            ksum[page_base[b]:page_base[b + 1], j] = 10 * b + j + 1
    q = np.ones((B, Hq, d))
    q[:, :, 0] = np.arange(1, Hq + 1)                                        # heads differ: sum(q) = d - 1 + (h+1)
    s64, _, _ = oracle.scores(to_bf16_bits(q), to_bf16_bits(ksum), page_base, ctx_len, Hkv, S, Pmax=3)
    for b in range(B):
        for h in range(Hq):
            want = (10 * b + h // 2 + 1) * (d + h)
            P = int(page_base[b + 1] - page_base[b])
            assert np.all(s64[b, h, :P] == want)


# --------------------------------------------------------------------------------------------- top-k

def brute_topk(scores, k):
    ids = sorted(range(len(scores)), key=lambda i: (-float(scores[i]), i))
    return sorted(ids[: min(k, len(scores))])


def test_topk_matches_exhaustive_sort_with_planted_ties():
    rng = np.random.default_rng(5)
    S = 1
    for trial in range(200):
        P = int(rng.integers(1, 24))
        k = int(rng.integers(1, 28))
        vals = rng.integers(-3, 4, size=P).astype(np.float32)               # few distinct values: many ties
        if trial % 3 == 0:
            vals = vals * 0.0 * rng.choice([-1.0, 1.0], size=P).astype(np.float32)  # mix of +0 and -0
        sc = np.full((1, 1, 32), np.nan, dtype=np.float32)
        sc[0, 0, :P] = vals
        sel, n_sel = oracle.topk(sc, [P], S, k)
        want = brute_topk(vals, k)
        assert n_sel[0, 0] == len(want)
        assert list(sel[0, 0, : len(want)]) == want
        assert np.all(sel[0, 0, len(want):] == -1)


def test_topk_special_cases():
    P, S = 16, 1
    sc = np.zeros((1, 1, P), dtype=np.float32)
    sel, n = oracle.topk(sc, [P], S, 5)
    assert list(sel[0, 0]) == [0, 1, 2, 3, 4]                                # all equal -> lowest ids
    sc[0, 0] = np.arange(P)
    sel, n = oracle.topk(sc, [P], S, P)
    assert list(sel[0, 0]) == list(range(P))                                 # k = P -> everything
    sc[0, 0] = [1, 9, 3, 9, 2, 9, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0]
    sel, n = oracle.topk(sc, [P], S, 1)
    assert list(sel[0, 0]) == [1]                                            # argmax, lowest id among ties
    sel, n = oracle.topk(sc, [P], S, 2)
    assert list(sel[0, 0]) == [1, 3]
    rng = np.random.default_rng(6)
    vals = rng.permutation(P).astype(np.float32)                             # distinct
    perm = rng.permutation(P)
    a, _ = oracle.topk(vals.reshape(1, 1, P), [P], S, 6)
    b, _ = oracle.topk(vals[perm].reshape(1, 1, P), [P], S, 6)
    assert sorted(perm[b[0, 0]]) == sorted(a[0, 0])                          # permuting pages permutes the set


def test_topk_uses_each_requests_own_length():
    S, k = 4, 3
    sc = np.zeros((2, 1, 8), dtype=np.float32)
    sc[0, 0] = [0, 1, 2, 3, 99, 99, 99, 99]                                  # request 0 has only 2 pages
    sc[1, 0] = [5, 1, 7, 3, 9, 0, 2, 8]
    sel, n = oracle.topk(sc, [2 * S - 1, 8 * S], S, k)
    assert list(n[:, 0]) == [2, 3]
    assert list(sel[0, 0]) == [0, 1, -1]
    assert list(sel[1, 0]) == [2, 4, 7]


# ------------------------------------------------------------------------------ resolve and balance

def replay_check(uniq, queue_of, load, mask, size, D, flags):
    """Re-walk the schedule in the rule's order and check each decision was least-loaded among replicas."""
    order = list(range(len(uniq)))
    if not flags & oracle.ORDER_BY_ID:
        order.sort(key=lambda i: (bin(int(mask[uniq[i]])).count("1"), int(uniq[i])))
    L = [0] * D
    for i in order:
        c = int(uniq[i])
        reps = [qd for qd in range(D) if (int(mask[c]) >> qd) & 1]
        best = min(reps, key=lambda qd: (L[qd], qd))
        assert int(queue_of[i]) == best
        L[best] += 1 if flags & oracle.UNIT_LOAD else int(size[c])
    assert L == [int(x) for x in load]


def test_resolve_golden_order_case():
    g = read_golden("schedule_order_case.txt")
    D = int(g["D"][0])
    mask = np.array(g["replica_mask"], dtype=np.uint32)
    size = np.array(g["cluster_size"], dtype=np.uint16)
    sel = np.arange(6, dtype=np.int32).reshape(1, 1, 6)                      # page i -> cluster i
    args = (sel, np.array([[6]], np.int32), [0, 6], np.arange(6, dtype=np.int32), [0, 6], mask, size, D)
    uniq, qof, load = oracle.resolve(*args)
    assert list(uniq) == [0, 1, 2, 3, 4, 5]
    assert list(qof) == [int(x) for x in g["default_queue_of"]]
    assert list(load) == [int(x) for x in g["default_load"]]
    uniq, qof, load = oracle.resolve(*args, flags=oracle.ORDER_BY_ID)
    assert list(qof) == [int(x) for x in g["by_id_queue_of"]]
    assert list(load) == [int(x) for x in g["by_id_load"]]


def random_resolve_case(rng, B=3, Hq=4, k=6, D=5, max_rep=3):
    pages = rng.integers(8, 20, size=B)
    page_base = np.concatenate([[0], np.cumsum(pages)]).astype(np.int64)
    n_clusters = rng.integers(2, 7, size=B)
    cluster_base = np.concatenate([[0], np.cumsum(n_clusters)]).astype(np.int64)
    p2c = np.concatenate([rng.integers(0, n_clusters[b], size=pages[b]) for b in range(B)]).astype(np.int32)
    C = int(cluster_base[-1])
    mask = np.zeros(C, dtype=np.uint32)
    for c in range(C):
        for qd in rng.choice(D, size=int(rng.integers(1, max_rep + 1)), replace=False):
            mask[c] |= np.uint32(1 << int(qd))
    size = rng.integers(1, 17, size=C).astype(np.uint16)
    sel = np.full((B, Hq, k), -1, dtype=np.int32)
    n_sel = np.zeros((B, Hq), dtype=np.int32)
    for b in range(B):
        for h in range(Hq):
            n = int(rng.integers(0, min(k, pages[b]) + 1))
            sel[b, h, :n] = np.sort(rng.choice(pages[b], size=n, replace=False))
            n_sel[b, h] = n
    return sel, n_sel, page_base, p2c, cluster_base, mask, size


@pytest.mark.parametrize("flags", [0, oracle.ORDER_BY_ID, oracle.UNIT_LOAD, oracle.ORDER_BY_ID | oracle.UNIT_LOAD])
def test_resolve_is_set_union_and_every_choice_is_least_loaded(flags):
    rng = np.random.default_rng(7)
    D = 5
    for _ in range(50):
        sel, n_sel, page_base, p2c, cluster_base, mask, size = random_resolve_case(rng, D=D)
        uniq, qof, load = oracle.resolve(sel, n_sel, page_base, p2c, cluster_base, mask, size, D, flags)
        want = set()
        B, Hq, _ = sel.shape
        for b in range(B):
            for h in range(Hq):
                for p in sel[b, h, : n_sel[b, h]]:
                    want.add(int(cluster_base[b]) + int(p2c[page_base[b] + p]))
        assert list(uniq) == sorted(want)                                     # each cluster once, ascending
        assert all((int(mask[c]) >> int(qd)) & 1 for c, qd in zip(uniq, qof))   # routed to a replica
        total = len(uniq) if flags & oracle.UNIT_LOAD else int(size[uniq].sum())
        assert int(load.sum()) == total
        replay_check(uniq, qof, load, mask, size, D, flags)


def test_resolve_single_replica_is_a_histogram_and_full_replication_is_round_robin():
    rng = np.random.default_rng(8)
    D, C = 4, 40
    size = rng.integers(1, 9, size=C).astype(np.uint16)
    sel = np.arange(C, dtype=np.int32).reshape(1, 1, C)
    common = (sel, np.array([[C]], np.int32), [0, C], np.arange(C, dtype=np.int32), [0, C])
    home = rng.integers(0, D, size=C)
    uniq, qof, load = oracle.resolve(*common, (1 << home).astype(np.uint32), size, D)
    assert np.array_equal(qof, home)
    assert np.array_equal(load, np.bincount(home, weights=size, minlength=D).astype(np.int32))
    full = np.full(C, (1 << D) - 1, dtype=np.uint32)
    uniq, qof, load = oracle.resolve(*common, full, size, D, flags=oracle.UNIT_LOAD)
    assert list(qof) == [c % D for c in range(C)]
    assert load.max() - load.min() <= 1


def test_resolve_greedy_within_one_item_of_exhaustive_optimum():
    rng = np.random.default_rng(9)
    worst = 0
    for _ in range(300):
        n = int(rng.integers(1, 7))
        D = int(rng.integers(2, 5))
        mask = np.zeros(n, dtype=np.uint32)
        for c in range(n):
            for qd in rng.choice(D, size=int(rng.integers(1, min(3, D) + 1)), replace=False):
                mask[c] |= np.uint32(1 << int(qd))
        size = np.ones(n, dtype=np.uint16)
        sel = np.arange(n, dtype=np.int32).reshape(1, 1, n)
        _, _, load = oracle.resolve(sel, np.array([[n]], np.int32), [0, n], np.arange(n, dtype=np.int32), [0, n],
                                    mask, size, D)
        choices = [[qd for qd in range(D) if (int(m) >> qd) & 1] for m in mask]
        best = min(max(np.bincount(assign, minlength=D)) for assign in itertools.product(*choices))
        assert best <= load.max() <= best + 1
        worst = max(worst, int(load.max()) - int(best))
    assert worst <= 1


def test_resolve_rejects_bad_tables():
    sel = np.zeros((1, 1, 1), dtype=np.int32)
    n = np.ones((1, 1), dtype=np.int32)
    with pytest.raises(ValueError):
        oracle.resolve(sel, n, [0, 1], [0], [0, 1], np.array([0], np.uint32), np.array([1], np.uint16), 2)   # no replica
    with pytest.raises(ValueError):
        oracle.resolve(sel, n, [0, 1], [0], [0, 1], np.array([4], np.uint32), np.array([1], np.uint16), 2)   # queue >= D
    with pytest.raises(ValueError):
        oracle.resolve(sel, n, [0, 1], [3], [0, 1], np.array([1], np.uint32), np.array([1], np.uint16), 2)   # cluster id


# -------------------------------------------------------------------------------------------- gather

def test_gather_copies_the_right_rows_and_zero_fills():
    B, Hq, Hkv, d, S, k = 2, 4, 2, 8, 4, 3
    page_base, ctx_len = identity_layout([5, 4], S, ctx=[5 * S - 3, 4 * S])   # request 0: last page has 1 valid token
    n = 9
    # every element encodes (page, kv, K/V, token, dim) so a wrong index shows
    idx = np.arange(n * Hkv * 2 * S * d, dtype=np.int64).reshape(n, Hkv, 2, S, d)
    pool = (idx % 65521).astype(np.uint16)
    sel = np.array([[[0, 2, 4], [1, 4, -1], [3, -1, -1], [0, 1, 2]],
                    [[0, 1, 3], [2, -1, -1], [1, 2, 3], [0, 3, -1]]], dtype=np.int32)
    n_sel = (sel >= 0).sum(-1).astype(np.int32)
    k_g, v_g, n_tok = oracle.gather(pool, sel, n_sel, page_base, ctx_len, Hkv, d, S)
    for b in range(B):
        for h in range(Hq):
            rows = 0
            for j in range(k):
                p = sel[b, h, j]
                blockK, blockV = k_g[b, h, j * S:(j + 1) * S], v_g[b, h, j * S:(j + 1) * S]
                if p < 0:
                    assert not blockK.any() and not blockV.any()
                    continue
                valid = 1 if (b == 0 and p == 4) else S
                src = pool[page_base[b] + p, h // 2]
                assert np.array_equal(blockK[:valid], src[0, :valid]) and np.array_equal(blockV[:valid], src[1, :valid])
                assert not blockK[valid:].any() and not blockV[valid:].any()
                rows += valid
            assert n_tok[b, h] == rows


# ----------------------------------------------------------------------------------------- attention

def attn_inputs(rng, B=2, Hq=3, d=16, rows=11, scale=1.0):
    q = to_bf16_bits(rng.standard_normal((B, Hq, d)) * scale)
    K = to_bf16_bits(rng.standard_normal((B, Hq, rows, d)))
    V = to_bf16_bits(rng.standard_normal((B, Hq, rows, d)))
    return q, K, V


def test_attention_hand_case():
    g = read_golden("attention_hand_case.txt")
    q = to_bf16_bits(np.array(g["q"]).reshape(1, 1, 4))
    K = to_bf16_bits(np.array([g["K0"], g["K1"]]).reshape(1, 1, 2, 4))
    V = to_bf16_bits(np.array([g["V0"], g["V1"]]).reshape(1, 1, 2, 4))
    out, lse = oracle.attention(q, K, V, [[2]])
    x0 = g["x0"][0]
    w0 = math.exp(x0) / (1 + math.exp(x0))
    want = w0 * np.array(g["V0"]) + (1 - w0) * np.array(g["V1"])
    assert np.allclose(out[0, 0], want, rtol=1e-14, atol=1e-14)
    assert lse[0, 0] == pytest.approx(math.log(1 + math.exp(x0)), rel=1e-14)


def test_attention_matches_library_sdpa_in_fp64():
    rng = np.random.default_rng(10)
    q, K, V = attn_inputs(rng, scale=2.0)
    n_tok = np.array([[11, 7, 1], [3, 11, 5]], dtype=np.int32)
    out, lse = oracle.attention(q, K, V, n_tok)
    qf, Kf, Vf = (torch.from_numpy(from_bf16_bits(x)) for x in (q, K, V))
    for b in range(2):
        for h in range(3):
            T = n_tok[b, h]
            ref = torch.nn.functional.scaled_dot_product_attention(qf[b, h][None, None], Kf[b, h, :T][None],
                                                                   Vf[b, h, :T][None])
            assert np.allclose(out[b, h], ref[0, 0].numpy(), rtol=1e-12, atol=1e-12)
            logits = (Kf[b, h, :T] @ qf[b, h]) / math.sqrt(16)
            assert lse[b, h] == pytest.approx(float(torch.logsumexp(logits, 0)), rel=1e-12)


def test_attention_closed_forms():
    rng = np.random.default_rng(11)
    q, K, V = attn_inputs(rng, B=1, Hq=1, d=16, rows=9)
    n = [[9]]
    Vf = from_bf16_bits(V)
    same_K = np.repeat(K[:, :, :1], 9, axis=2)
    out, lse = oracle.attention(q, same_K, V, n)
    assert np.allclose(out[0, 0], Vf[0, 0].mean(axis=0), rtol=1e-13, atol=1e-13)        # equal keys -> mean of V
    const_V = to_bf16_bits(np.broadcast_to(bf16_round(rng.standard_normal(16)), (1, 1, 9, 16)))
    out, _ = oracle.attention(q, K, const_V, n)
    assert np.allclose(out[0, 0], from_bf16_bits(const_V)[0, 0, 0], rtol=1e-13, atol=1e-13)  # constant V
    qf = from_bf16_bits(q)[0, 0]
    Kd = from_bf16_bits(K).copy()
    Kd[0, 0, 4] = 40.0 * qf / np.linalg.norm(qf)                                         # one dominant key
    out, _ = oracle.attention(q, to_bf16_bits(Kd), V, n)
    assert np.allclose(out[0, 0], Vf[0, 0, 4], atol=1e-6)
    perm = rng.permutation(9)
    a, la = oracle.attention(q, K, V, n)
    b, lb = oracle.attention(q, K[:, :, perm], V[:, :, perm], n)
    assert np.allclose(a, b, rtol=1e-12, atol=1e-13) and la[0, 0] == pytest.approx(lb[0, 0], rel=1e-13)


def test_attention_halves_merge_by_lse_and_lse_grows_with_tokens():
    rng = np.random.default_rng(12)
    q, K, V = attn_inputs(rng, B=1, Hq=1, d=16, rows=10, scale=1.5)
    whole, lw = oracle.attention(q, K, V, [[10]])
    a, la = oracle.attention(q, K[:, :, :4], V[:, :, :4], [[4]])
    b, lb = oracle.attention(q, K[:, :, 4:], V[:, :, 4:], [[6]])
    wa, wb = np.exp(la - lw), np.exp(lb - lw)
    assert np.allclose(wa * a + wb * b, whole, rtol=1e-12, atol=1e-13)
    assert wa + wb == pytest.approx(1.0, rel=1e-12)
    prev = -np.inf
    for T in range(1, 11):
        _, l = oracle.attention(q, K, V, [[T]])
        assert l[0, 0] > prev
        prev = l[0, 0]


# ----------------------------------------------------------------------------------------- whole step

def test_step_invariants_on_a_scaled_topic_workload():
    from paper_2603_17803_b200 import workloads as W
    cfg = W.scaled(W.CONFIGS["c5_skewed"], batch=3, ctx_range=(300, 900), top_k=8, n_topics=6)
    w = W.generate(cfg, seed=3)
    u = W.bits_u16
    pb, cl = w.page_base.numpy(), w.ctx_len.numpy()
    mask = w.cluster_replica_mask.numpy().view(np.uint32)
    size = w.cluster_size.numpy().view(np.uint16)
    ksum = oracle.build_summaries(u(w.kv_pool), pb, cl, cfg.n_kv_heads, cfg.head_dim, cfg.page_size)
    r = oracle.step(u(w.q), ksum, u(w.kv_pool), pb, cl, w.page2cluster.numpy(), w.cluster_base.numpy(), mask, size,
                    Hkv=cfg.n_kv_heads, S=cfg.page_size, k=cfg.top_k, D=cfg.n_queues, Pmax=cfg.max_pages())
    # every selected page's cluster is fetched, exactly once
    need = set()
    for b in range(cfg.batch):
        for h in range(cfg.n_q_heads):
            for p in r.sel[b, h, : r.n_sel[b, h]]:
                need.add(int(w.cluster_base[b]) + int(w.page2cluster[pb[b] + p]))
    assert sorted(need) == list(r.uniq) and len(set(r.uniq.tolist())) == len(r.uniq)
    assert int(r.load.sum()) == int(size[r.uniq].sum())
    replay_check(r.uniq, r.queue_of, r.load, mask, size, cfg.n_queues, 0)
    # padding tokens (poisoned by the generator) must not leak anywhere
    assert np.abs(r.out).max() < 50 and np.abs(r.score64[np.isfinite(r.score64)]).max() < 1e4
    P = (cl + cfg.page_size - 1) // cfg.page_size
    for b in range(cfg.batch):
        full = cfg.page_size * r.n_sel[b]
        last_sel = (r.sel[b] == P[b] - 1).any(axis=-1)
        tail = cl[b] - cfg.page_size * (P[b] - 1)
        assert np.array_equal(r.n_tok[b], full - last_sel * (cfg.page_size - tail))


# ------------------------------------------------------------------ resident filter and cache counters

def test_resolve_cached_is_set_difference_with_counter_updates_and_eq6_scores():
    rng = np.random.default_rng(13)
    D = 5
    for trial in range(40):
        sel, n_sel, page_base, p2c, cluster_base, mask, size = random_resolve_case(rng, D=D)
        C = int(cluster_base[-1])
        resident = (rng.random(C) < 0.3).astype(np.uint8)
        freq = rng.integers(-3, 10, size=C).astype(np.int32)
        t_base, t_tr = 80.0, 2.5
        uniq, qof, load, n_hit, freq_new, score = oracle.resolve_cached(sel, n_sel, page_base, p2c, cluster_base, mask,
                                                                          size, resident, freq, D, t_base, t_tr)
        activated = set()
        B, Hq, _ = sel.shape
        for b in range(B):
            for h in range(Hq):
                for p in sel[b, h, : n_sel[b, h]]:
                    activated.add(int(cluster_base[b]) + int(p2c[page_base[b] + p]))
        res = {c for c in range(C) if resident[c]}
        assert list(uniq) == sorted(activated - res)                       # E_IO = union minus resident (Eq. 8)
        assert n_hit == len(activated & res)
        want = freq.copy()
        for c in range(C):
            if c in activated:
                want[c] += 1
            elif c in res:
                want[c] -= 1
        assert np.array_equal(freq_new, want)
        assert np.allclose(score, want * (t_base + size * t_tr) / size, rtol=1e-14, atol=0)
        replay_check(uniq, qof, load, mask, size, D, 0)                    # the fetched ones are scheduled as before
    # nothing resident: identical to the plain merge; everything resident: nothing to fetch
    none = np.zeros(C, np.uint8)
    a = oracle.resolve(sel, n_sel, page_base, p2c, cluster_base, mask, size, D)
    b = oracle.resolve_cached(sel, n_sel, page_base, p2c, cluster_base, mask, size, none, freq, D, 1.0, 1.0)
    assert all(np.array_equal(x, y) for x, y in zip(a, b[:3])) and b[3] == 0
    allr = np.ones(C, np.uint8)
    c = oracle.resolve_cached(sel, n_sel, page_base, p2c, cluster_base, mask, size, allr, freq, D, 1.0, 1.0)
    assert len(c[0]) == 0 and int(c[2].sum()) == 0 and c[3] == len(a[0])


def test_cache_score_hand_case():
    # Eq. 6 by hand: f = 6 activations, s = 4 entries, T_base = 100, T_transfer = 5 -> 6 * (100 + 20) / 4 = 180
    sel = np.zeros((1, 1, 1), np.int32)
    out = oracle.resolve_cached(sel, np.ones((1, 1), np.int32), [0, 1], [0], [0, 1], np.array([1], np.uint32),
                                np.array([4], np.uint16), np.array([1], np.uint8), np.array([5], np.int32), 2, 100.0, 5.0)
    assert out[3] == 1 and list(out[4]) == [6] and out[5][0] == 180.0 and len(out[0]) == 0


def test_topk_local_window_is_the_last_pages_plus_the_best_of_the_rest():
    rng = np.random.default_rng(14)
    for _ in range(100):
        P = int(rng.integers(1, 30))
        k = int(rng.integers(1, 12))
        w = int(rng.integers(0, k + 1))
        vals = rng.integers(-4, 5, size=P).astype(np.float32)
        sc = np.full((1, 1, 32), np.nan, dtype=np.float32)
        sc[0, 0, :P] = vals
        sel, n = oracle.topk(sc, [P], 1, k, window=w)
        k_eff = min(k, P)
        window_pages = list(range(max(0, P - w), P))
        rest = brute_topk(vals[: max(0, P - w)], k_eff - len(window_pages)) if k_eff > len(window_pages) else []
        want = sorted(set(window_pages[-k_eff:] if len(window_pages) > k_eff else window_pages) | set(rest))
        assert n[0, 0] == k_eff and list(sel[0, 0, :k_eff]) == want
    with pytest.raises(ValueError):
        oracle.topk(sc, [P], 1, 3, window=4)


# ------------------------------------------------------------------------------- medoid index (cluster mode)

def test_medoid_step_with_one_page_clusters_is_the_page_step():
    """Clusters of one page each, each its own medoid: cluster-granular selection must reduce to page selection."""
    rng = np.random.default_rng(21)
    pages = (9, 6)
    q, pool, ksum, page_base, ctx_len = rand_case(rng, pages=pages, ctx=[9 * 4 - 1, 6 * 4])
    n = int(page_base[-1])
    page2cluster = np.concatenate([np.arange(p) for p in pages]).astype(np.int32)
    cluster_base = page_base.copy()
    mask = rng.integers(1, 8, size=n).astype(np.uint32)
    size = np.ones(n, dtype=np.uint16)
    ptr = np.arange(n + 1, dtype=np.int64)
    r_page = oracle.step(q, ksum, pool, page_base, ctx_len, page2cluster, cluster_base, mask, size, Hkv=2, S=4, k=3,
                         D=3, Pmax=9)
    r_med = oracle.medoid_step(q, ksum, pool, page_base, ctx_len, page2cluster, cluster_base, mask, size, ptr,
                               page2cluster, page2cluster, Hkv=2, S=4, k_c=3, D=3)
    assert np.array_equal(r_med.sel_clusters, r_page.sel) and np.array_equal(r_med.n_sel_clusters, r_page.n_sel)
    assert np.array_equal(r_med.sel_pages[..., :3], r_page.sel)
    assert np.array_equal(r_med.uniq, r_page.uniq) and np.array_equal(r_med.queue_of, r_page.queue_of)
    assert np.array_equal(r_med.load, r_page.load)
    assert np.array_equal(r_med.out, r_page.out) and np.array_equal(r_med.lse, r_page.lse)


def test_medoid_step_scores_medoids_and_attends_whole_clusters():
    from paper_2603_17803_b200 import workloads as W
    cfg = W.scaled(W.CONFIGS["c5_skewed"], batch=3, ctx_range=(300, 900), top_k=8, n_topics=6)
    w = W.generate(cfg, seed=5)
    ptr, members, medoid = (t.numpy() for t in W.cluster_members(w))
    u = W.bits_u16
    pb, cl, cb = w.page_base.numpy(), w.ctx_len.numpy(), w.cluster_base.numpy()
    p2c = w.page2cluster.numpy()
    mask = w.cluster_replica_mask.numpy().view(np.uint32)
    size = w.cluster_size.numpy().view(np.uint16)
    S, Hq = cfg.page_size, cfg.n_q_heads
    # the member lists are the inverse of the page -> cluster table, and each medoid is a member
    for b in range(cfg.batch):
        P = -(-int(cl[b]) // S)
        seen = []
        for c in range(int(cb[b]), int(cb[b + 1])):
            mem = members[ptr[c]:ptr[c + 1]]
            assert np.all(np.diff(mem) > 0) and np.all(p2c[pb[b] + mem] == c - cb[b])
            assert len(mem) == 0 or medoid[c] in mem
            seen += mem.tolist()
        assert sorted(seen) == list(range(P))
    ksum = oracle.build_summaries(u(w.kv_pool), pb, cl, cfg.n_kv_heads, cfg.head_dim, S)
    k_c = 3
    r = oracle.medoid_step(u(w.q), ksum, u(w.kv_pool), pb, cl, p2c, cb, mask, size, ptr, members, medoid,
                           Hkv=cfg.n_kv_heads, S=S, k_c=k_c, D=cfg.n_queues)
    page_s64, page_s32, _ = oracle.scores(u(w.q), ksum, pb, cl, cfg.n_kv_heads, S, cfg.max_pages())
    need = set()
    for b in range(cfg.batch):
        n_c = int(cb[b + 1] - cb[b])
        for h in range(Hq):
            # a cluster's score is the page score of its medoid; the selection is the exhaustive top-k of those
            want_scores = page_s32[b, h, medoid[cb[b]:cb[b + 1]]]
            assert np.array_equal(r.score32[b, h, :n_c], want_scores)
            want = brute_topk(want_scores, k_c)
            n = int(r.n_sel_clusters[b, h])
            assert n == min(k_c, n_c) and list(r.sel_clusters[b, h, :n]) == want
            # all pages of the selected clusters, nothing else
            pages = sorted(p for c in want for p in members[ptr[cb[b] + c]:ptr[cb[b] + c + 1]].tolist())
            assert list(r.sel_pages[b, h, :r.n_sel_pages[b, h]]) == pages
            assert r.n_sel_pages[b, h] == int(size[cb[b] + np.array(want)].sum())
            need.update(int(cb[b]) + c for c in want)
    assert sorted(need) == list(r.uniq)
    replay_check(r.uniq, r.queue_of, r.load, mask, size, cfg.n_queues, 0)
    # attention is Eq. 1 over exactly those pages: recompute one head from the pool in numpy
    b, h = 1, 5
    kvh = h // (Hq // cfg.n_kv_heads)
    pool = W.bits_u16(w.kv_pool)
    f = lambda bits: (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    ks, vs = [], []
    P = -(-int(cl[b]) // S)
    for p in r.sel_pages[b, h, :r.n_sel_pages[b, h]]:
        valid = S if p < P - 1 else int(cl[b]) - S * (P - 1)
        ks.append(f(pool[pb[b] + p, kvh, 0, :valid]))
        vs.append(f(pool[pb[b] + p, kvh, 1, :valid]))
    K, V = np.concatenate(ks), np.concatenate(vs)
    logits = K @ f(u(w.q)[b, h]) / np.sqrt(cfg.head_dim)
    pr = np.exp(logits - logits.max())
    assert np.allclose(r.out[b, h], (pr / pr.sum()) @ V, rtol=1e-9, atol=1e-9)


def test_medoid_step_local_window_joins_every_head_and_covers_the_context_at_full_width():
    """Sec. 4.2, Tier 1 (2): the last W pages are attended whatever the index selects.  Pins: each head's set is the
    union of its clusters' members and the window; W = 0 changes nothing; with W >= P every head attends the whole
    context, i.e. plain dense attention (Eq. 1 over all tokens), and every cluster of the request is scheduled."""
    from paper_2603_17803_b200 import workloads as W
    cfg = W.scaled(W.CONFIGS["c5_skewed"], batch=2, ctx_range=(200, 700), top_k=8, n_topics=5)
    w = W.generate(cfg, seed=11)
    ptr, members, medoid = (t.numpy() for t in W.cluster_members(w))
    u = W.bits_u16
    pb, cl, cb = w.page_base.numpy(), w.ctx_len.numpy(), w.cluster_base.numpy()
    p2c = w.page2cluster.numpy()
    mask = w.cluster_replica_mask.numpy().view(np.uint32)
    size = w.cluster_size.numpy().view(np.uint16)
    S, Hq, g = cfg.page_size, cfg.n_q_heads, cfg.n_q_heads // cfg.n_kv_heads
    ksum = oracle.build_summaries(u(w.kv_pool), pb, cl, cfg.n_kv_heads, cfg.head_dim, S)
    run = lambda window: oracle.medoid_step(u(w.q), ksum, u(w.kv_pool), pb, cl, p2c, cb, mask, size, ptr, members, medoid,
                                            Hkv=cfg.n_kv_heads, S=S, k_c=2, D=cfg.n_queues, window=window)
    r0, r3, rall = run(0), run(3), run(10_000)
    assert np.array_equal(r0.sel_clusters, r3.sel_clusters)            # the window does not touch the index
    f = lambda bits: (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    pool = u(w.kv_pool)
    for b in range(cfg.batch):
        P = -(-int(cl[b]) // S)
        for h in range(Hq):
            base = set(r0.sel_pages[b, h, :r0.n_sel_pages[b, h]].tolist())
            assert set(r3.sel_pages[b, h, :r3.n_sel_pages[b, h]].tolist()) == base | set(range(max(0, P - 3), P))
            assert list(rall.sel_pages[b, h, :rall.n_sel_pages[b, h]]) == list(range(P))
            K = f(pool[pb[b]:pb[b] + P, h // g, 0]).reshape(P * S, -1)[: int(cl[b])]
            V = f(pool[pb[b]:pb[b] + P, h // g, 1]).reshape(P * S, -1)[: int(cl[b])]
            logits = K @ f(u(w.q)[b, h]) / np.sqrt(cfg.head_dim)
            pr = np.exp(logits - logits.max())
            assert np.allclose(rall.out[b, h], (pr / pr.sum()) @ V, rtol=1e-9, atol=1e-9)
    assert list(rall.uniq) == list(range(int(cb[-1])))                  # everything is fetched
    window_clusters = {int(cb[b]) + int(p2c[pb[b] + p]) for b in range(cfg.batch)
                       for p in range(max(0, -(-int(cl[b]) // S) - 3), -(-int(cl[b]) // S))}
    assert set(r3.uniq.tolist()) == set(r0.uniq.tolist()) | window_clusters
    replay_check(r3.uniq, r3.queue_of, r3.load, mask, size, cfg.n_queues, 0)


# --------------------------------------------------------------------------------- batched submission order

def test_submit_order_hand_case():
    # uniq index:        0     1     2     3     4     5
    masks = np.array([0b011, 0b100, 0b110, 0b001, 0b111, 0b010], dtype=np.uint32)   # replicas: 2 1 2 1 3 1
    queue = np.array([1, 2, 2, 0, 0, 1], dtype=np.uint8)
    # visit order by (replicas, index): 1 3 5 | 0 2 | 4 -> buckets: q0 [3, 4], q1 [5, 0], q2 [1, 2]
    order, rounds = oracle.submit_order(queue, masks, 3)
    assert rounds == 2 and list(order) == [3, 5, 1, 4, 0, 2]
    # by position alone: buckets q0 [3, 4], q1 [0, 5], q2 [1, 2]
    order, rounds = oracle.submit_order(queue, masks, 3, oracle.ORDER_BY_ID)
    assert rounds == 2 and list(order) == [3, 0, 1, 4, 5, 2]


@pytest.mark.parametrize("flags", [0, oracle.ORDER_BY_ID])
def test_submit_order_is_a_round_robin_over_the_buckets(flags):
    rng = np.random.default_rng(31)
    for _ in range(20):
        D = 5
        sel, n_sel, page_base, p2c, cbase, mask, size = random_resolve_case(rng, D=D)
        uniq, queue_of, load = oracle.resolve(sel, n_sel, page_base, p2c, cbase, mask, size, D, flags)
        order, rounds = oracle.submit_order(queue_of, mask[uniq], D, flags)
        n = len(uniq)
        assert sorted(order.tolist()) == list(range(n))                       # every cluster exactly once
        counts = np.bincount(queue_of, minlength=D)
        assert rounds == counts.max(initial=0)
        # batch r holds one cluster of every queue that still has one, in queue order
        pos = 0
        taken = np.zeros(D, dtype=np.int64)
        for r in range(rounds):
            qs = [q for q in range(D) if counts[q] > r]
            batch = order[pos:pos + len(qs)]
            assert [int(queue_of[i]) for i in batch] == qs
            pos += len(qs)
            taken[qs] += 1
        assert pos == n
        # inside a bucket: assignment order, i.e. the order in which a replay of the scheduling pass meets them
        key = (lambda i: i) if flags & oracle.ORDER_BY_ID else (lambda i: (bin(int(mask[uniq[i]])).count("1"), i))
        for q in range(D):
            mine = [int(i) for i in order if queue_of[i] == q]
            assert mine == sorted(mine, key=key)


# ------------------------------------------------------------------------ Algorithm 1 (offline clustering)

def sym(n, fill, pairs):
    d = np.full((n, n), fill, dtype=np.float32)
    np.fill_diagonal(d, 0.0)
    for (i, j), v in pairs.items():
        d[i, j] = d[j, i] = v
    return d


def test_algorithm1_hand_case():
    g = read_golden("algorithm1_hand_case.txt")
    d = sym(5, 0.9, {(0, 1): 0.1, (0, 2): 0.2, (1, 2): 0.3, (3, 4): 0.1, (2, 3): 0.4, (2, 4): 0.5})
    rho, ptr, members, medoid = oracle.build_clusters(d, 0.5)
    assert list(rho) == g["rho"] and list(ptr) == g["ptr"] and list(members) == g["members"]
    assert list(medoid) == g["medoid"]


def test_algorithm1_extreme_radii_and_blocks():
    rng = np.random.default_rng(41)
    n = 12
    d = rng.uniform(0.2, 0.8, size=(n, n)).astype(np.float32)
    d = np.minimum(d, d.T)
    np.fill_diagonal(d, 0.0)
    # a radius below every distance: every entry is its own cluster, in index order
    rho, ptr, members, medoid = oracle.build_clusters(d, 0.1)
    assert not rho.any() and list(ptr) == list(range(n + 1)) and list(members) == list(range(n))
    assert list(medoid) == list(range(n))
    # a radius above every distance: one cluster, the others in order of their distance to entry 0
    rho, ptr, members, medoid = oracle.build_clusters(d, 0.9)
    assert np.all(rho == n - 1) and list(ptr) == [0, n] and list(medoid) == [0]
    assert list(members) == [0] + sorted(range(1, n), key=lambda e: (d[0, e], e))
    # well separated blocks of different sizes: the clusters are the blocks, the largest first
    blocks = [[0, 5, 7], [1, 2, 3, 4, 6], [8, 9], [10], [11]]
    d = np.full((n, n), 0.9, dtype=np.float32)
    for blk in blocks:
        for i in blk:
            for j in blk:
                d[i, j] = 0.25
    np.fill_diagonal(d, 0.0)
    rho, ptr, members, medoid = oracle.build_clusters(d, 0.5)
    got = [list(members[ptr[c]:ptr[c + 1]]) for c in range(len(medoid))]
    assert got == [[1, 2, 3, 4, 6], [0, 5, 7], [8, 9], [10], [11]]
    assert list(medoid) == [1, 0, 8, 10, 11]


def test_algorithm1_replay_in_exact_arithmetic():
    """Distances on a grid of 1/64: fp32 sums are exact, so an exact-arithmetic replay must agree everywhere."""
    from fractions import Fraction
    rng = np.random.default_rng(43)
    for n, tau64 in [(30, 20), (64, 28), (90, 16)]:
        g = rng.integers(1, 64, size=(n, n))
        g = np.minimum(g, g.T)
        np.fill_diagonal(g, 0)
        d = (g / 64.0).astype(np.float32)
        tau = tau64 / 64.0
        rho, ptr, members, medoid = oracle.build_clusters(d, tau)
        want_rho = [(g[i] <= tau64).sum() - 1 for i in range(n)]
        assert list(rho) == want_rho
        queue = sorted(range(n), key=lambda i: (-want_rho[i], i))
        covered, clusters, meds = set(), [], []
        for m in queue:
            if len(covered) == n:
                break
            if m in covered:
                continue
            cand = sorted((e for e in range(n) if e != m and g[m, e] <= tau64), key=lambda e: (g[m, e], e))
            mem = [m]
            for c in cand:
                if Fraction(int(sum(g[e, c] for e in mem)), len(mem)) <= tau64:
                    mem.append(c)
            clusters.append(mem)
            meds.append(m)
            covered.update(mem)
        got = [list(members[ptr[c]:ptr[c + 1]]) for c in range(len(medoid))]
        assert got == clusters and list(medoid) == meds
        assert set(members.tolist()) == set(range(n))                       # every entry is covered
        assert any(members.tolist().count(e) > 1 for e in range(n))         # and some sit in several clusters


def test_algorithm1_fp32_reading_agrees_with_the_plain_average_outside_the_band():
    """General (non-grid) distances.  The oracle the GPU is compared with bit for bit decides on an fp32 running
    sum; Eq. 5 is a plain average.  The two must take the same decision whenever |average - tau| > 1e-5 * tau:
    the fp32 clustering is replayed against averages recomputed in double, and where no decision falls inside
    that band the two clusterings are identical."""
    rng = np.random.default_rng(47)
    near_total, exact_cases = 0, 0
    for n, topics, tau in [(40, 3, 0.45), (150, 6, 0.4), (400, 10, 0.38), (257, 5, 0.5), (300, 4, 0.62)]:
        topic = rng.integers(0, topics, size=n)
        base = np.where(topic[:, None] == topic[None, :], 0.22, 0.8)
        d = (base + rng.uniform(-0.2, 0.2, size=(n, n))).astype(np.float32)
        d = np.minimum(d, d.T)
        np.fill_diagonal(d, 0.0)
        rho, ptr, members, medoid = oracle.build_clusters(d, tau)
        near = oracle.replay_clusters(d, tau, ptr, members, medoid, near_rtol=1e-5)
        rho_p, ptr_p, members_p, medoid_p, near_p = oracle.build_clusters_plain(d, tau, near_rtol=1e-5)
        assert np.array_equal(rho, rho_p)
        assert oracle.replay_clusters(d, tau, ptr_p, members_p, medoid_p, near_rtol=1e-5) == near_p
        if near == 0 and near_p == 0:
            assert np.array_equal(ptr, ptr_p) and np.array_equal(members, members_p) and np.array_equal(medoid, medoid_p)
            exact_cases += 1
        near_total += near
    assert exact_cases >= 3, "random distances should rarely come within 1e-5 of the radius"
    print(f"decisions within the band: {near_total}")


def test_algorithm1_replay_rejects_wrong_clusterings():
    """The band replay is itself a checker: a dropped member, a wrong medoid, a swapped order must all fail it."""
    d = sym(5, 0.9, {(0, 1): 0.1, (0, 2): 0.2, (1, 2): 0.3, (3, 4): 0.1, (2, 3): 0.4, (2, 4): 0.5})
    rho, ptr, members, medoid = oracle.build_clusters(d, 0.5)
    assert oracle.replay_clusters(d, 0.5, ptr, members, medoid) == 0
    bad = [
        (np.array([0, 2, 5]), np.array([2, 0, 3, 4, 2]), medoid),            # entry 1 dropped from the first cluster
        (ptr, np.array([2, 1, 0, 3, 4, 2]), medoid),                         # joining order swapped
        (ptr, np.array([0, 2, 1, 3, 4, 2]), np.array([0, 3])),               # wrong medoid
        (np.array([0, 3]), np.array([2, 0, 1]), np.array([2])),              # entries 3 and 4 left uncovered
    ]
    for p_, m_, med_ in bad:
        with pytest.raises(AssertionError):
            oracle.replay_clusters(d, 0.5, p_, m_, med_)
    # a decision exactly on the radius may go either way inside the band, and only there
    d2 = sym(3, 0.9, {(0, 1): 0.2, (0, 2): 0.4, (1, 2): 0.6000000238418579})
    r = oracle.build_clusters_plain(d2, 0.5, near_rtol=1e-5)
    assert r[4] >= 1
    # entry 2's average distance to {0, 1} is 0.5 + 1.2e-8: it joins (one cluster) or not (then it founds [2, 0])
    both = [(np.array([0, 3]), np.array([0, 1, 2]), np.array([0])), (np.array([0, 2, 4]), np.array([0, 1, 2, 0]), np.array([0, 2]))]
    for p_, m_, med_ in both:
        assert oracle.replay_clusters(d2, 0.5, p_, m_, med_, near_rtol=1e-5) >= 1
    with pytest.raises(AssertionError):
        oracle.replay_clusters(d2, 0.5, both[0][0], both[0][1], both[0][2], near_rtol=0.0)   # strictly, it does not join


# ------------------------------------------------------------------------------- Eq. 7 placement of entries

def test_entry_placement_hand_case_and_round_robin():
    # clusters [2 0 1] and [3 4 2] on 4 disks: entries land on disks 0 1 2 | 3 0 1; entry 2 has copies on 0 and 1
    masks = oracle.entry_replica_masks([0, 3, 6], [2, 0, 1, 3, 4, 2], 5, 4)
    assert list(masks) == [0b0010, 0b0100, 0b0011, 0b1000, 0b0001]
    # without replicas every entry has one copy and the disks fill evenly
    rng = np.random.default_rng(51)
    sizes = rng.integers(1, 9, size=40)
    ptr = np.concatenate([[0], np.cumsum(sizes)])
    members = rng.permutation(int(ptr[-1]))
    D = 6
    masks = oracle.entry_replica_masks(ptr, members, int(ptr[-1]), D)
    assert all(bin(int(m)).count("1") == 1 for m in masks)
    per_disk = np.bincount([int(m).bit_length() - 1 for m in masks], minlength=D)
    assert per_disk.max() - per_disk.min() <= 1
    # each cluster's entries sit on consecutive disks (wrap-around), starting where the previous cluster stopped
    for c in range(len(sizes)):
        disks = [int(masks[e]).bit_length() - 1 for e in members[ptr[c]:ptr[c + 1]]]
        assert disks == [(int(ptr[c]) + j) % D for j in range(int(sizes[c]))]


# ------------------------------------------------------------------------------------ cache admission (Eq. 6)

def test_cache_admission_hand_case_and_limits():
    score = np.array([3.0, 9.0, 9.0, 1.0, 5.0], dtype=np.float32)
    size = np.array([4, 2, 3, 1, 6], dtype=np.uint16)
    # order by score: 1, 2 (tie, lower id first), 4, 0, 3 with sizes 2, 3, 6, 4, 1
    res, n, used = oracle.cache_admit(score, size, 11)
    assert list(res) == [0, 1, 1, 0, 1] and n == 3 and used == 11
    res, n, used = oracle.cache_admit(score, size, 10)      # cluster 4 (6 pages) does not fit after 5: admission ends
    assert list(res) == [0, 1, 1, 0, 0] and n == 2 and used == 5
    assert oracle.cache_admit(score, size, 0)[1] == 0
    res, n, used = oracle.cache_admit(score, size, 1000)
    assert res.all() and n == 5 and used == 16
    # growing the capacity never evicts
    rng = np.random.default_rng(61)
    score = rng.integers(0, 20, size=200).astype(np.float32)
    size = rng.integers(1, 17, size=200).astype(np.uint16)
    prev = np.zeros(200, dtype=np.uint8)
    for cap in range(0, 1800, 37):
        res, n, used = oracle.cache_admit(score, size, cap)
        assert np.all(res >= prev) and used <= cap and used == int(size[res == 1].sum())
        if n < 200:                                          # the best cluster left out really does not fit
            nxt = min((c for c in range(200) if not res[c]), key=lambda c: (-score[c], c))
            assert used + int(size[nxt]) > cap
        prev = res
