"""CPU oracle of the per-decode-step KVCache retrieval path -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and never imports it.

The arithmetic lives in ``swarm_oracle.cpp`` (plain C++, double accumulation); this
module compiles it with g++ on first use and exposes thin numpy wrappers.  bf16 tensors
travel as ``uint16`` arrays holding the raw bits.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "swarm_oracle.cpp")
_LIB = os.path.join(_HERE, "libswarm_oracle.so")

ORDER_BY_ID = 1
UNIT_LOAD = 2

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (OpenMP) next to its source; returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        for name in ("oracle_build_summaries", "oracle_scores", "oracle_topk", "oracle_resolve", "oracle_resolve_cached",
                     "oracle_gather", "oracle_attention", "oracle_set_threads"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def _p(a):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


def _arr(x, dtype):
    a = np.ascontiguousarray(x, dtype=dtype)
    return a


def _check(rc, what):
    if rc != 0:
        raise ValueError(f"{what}: oracle status {rc} (1 bad argument, 2 bad table entry, 3 non-finite)")


def set_threads(n: int) -> int:
    """Set the OpenMP thread count (n <= 0 only queries); returns the count in effect."""
    return int(_load().oracle_set_threads(ctypes.c_int(n)))


def build_summaries(kv_pool, page_base, ctx_len, Hkv, d, S):
    """kv_pool uint16 [pages][Hkv][2][S][d] -> ksum uint16 [pages][Hkv][2][d] (min, max over valid tokens)."""
    kv_pool = _arr(kv_pool, np.uint16)
    page_base = _arr(page_base, np.int64)
    ctx_len = _arr(ctx_len, np.int32)
    n_pages = kv_pool.size // (Hkv * 2 * S * d)
    ksum = np.zeros((n_pages, Hkv, 2, d), dtype=np.uint16)
    rc = _load().oracle_build_summaries(_p(kv_pool), _p(page_base), _p(ctx_len), ctypes.c_int32(len(ctx_len)),
                                        ctypes.c_int32(Hkv), ctypes.c_int32(d), ctypes.c_int32(S), _p(ksum))
    _check(rc, "build_summaries")
    return ksum


def scores(q, ksum, page_base, ctx_len, Hkv, S, Pmax):
    """q uint16 [B][Hq][d]; returns (score64 [B][Hq][Pmax], score32, cond); entries p >= P_b are -inf / 0."""
    q = _arr(q, np.uint16)
    ksum = _arr(ksum, np.uint16)
    page_base = _arr(page_base, np.int64)
    ctx_len = _arr(ctx_len, np.int32)
    B, Hq, d = q.shape
    s64 = np.full((B, Hq, Pmax), -np.inf, dtype=np.float64)
    s32 = np.full((B, Hq, Pmax), -np.inf, dtype=np.float32)
    cond = np.zeros((B, Hq, Pmax), dtype=np.float64)
    rc = _load().oracle_scores(_p(q), _p(ksum), _p(page_base), _p(ctx_len), ctypes.c_int32(B), ctypes.c_int32(Hq),
                               ctypes.c_int32(Hkv), ctypes.c_int32(d), ctypes.c_int32(S), ctypes.c_int64(Pmax),
                               _p(s64), _p(s32), _p(cond))
    _check(rc, "scores")
    return s64, s32, cond


def topk(score, ctx_len, S, k, window=0):
    """score float32 [B][Hq][Pmax] -> (sel int32 [B][Hq][k] ascending page id, -1 padded; n_sel [B][Hq]).
    The last ``window`` pages of every request are always selected."""
    score = _arr(score, np.float32)
    ctx_len = _arr(ctx_len, np.int32)
    B, Hq, Pmax = score.shape
    sel = np.empty((B, Hq, k), dtype=np.int32)
    n_sel = np.empty((B, Hq), dtype=np.int32)
    rc = _load().oracle_topk(_p(score), _p(ctx_len), ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(S),
                             ctypes.c_int64(Pmax), ctypes.c_int32(k), ctypes.c_int32(window), _p(sel), _p(n_sel))
    _check(rc, "topk")
    return sel, n_sel


def resolve(sel, n_sel, page_base, page2cluster, cluster_base, replica_mask, cluster_size, D, flags=0):
    """Returns (uniq int32 [n_uniq] ascending global cluster id, queue_of uint8 [n_uniq], load int32 [D])."""
    sel = _arr(sel, np.int32)
    n_sel = _arr(n_sel, np.int32)
    page_base = _arr(page_base, np.int64)
    page2cluster = _arr(page2cluster, np.int32)
    cluster_base = _arr(cluster_base, np.int64)
    replica_mask = _arr(replica_mask, np.uint32)
    cluster_size = _arr(cluster_size, np.uint16)
    B, Hq, k = sel.shape
    cap = max(int(cluster_base[-1]), 1)
    uniq = np.empty(cap, dtype=np.int32)
    queue_of = np.empty(cap, dtype=np.uint8)
    n_uniq = np.zeros(1, dtype=np.int32)
    load = np.zeros(D, dtype=np.int32)
    rc = _load().oracle_resolve(_p(sel), _p(n_sel), _p(page_base), _p(page2cluster), _p(cluster_base),
                                _p(replica_mask), _p(cluster_size), ctypes.c_int32(B), ctypes.c_int32(Hq),
                                ctypes.c_int32(k), ctypes.c_int32(D), ctypes.c_uint32(flags), _p(uniq), _p(queue_of),
                                _p(n_uniq), _p(load))
    _check(rc, "resolve")
    n = int(n_uniq[0])
    return uniq[:n].copy(), queue_of[:n].copy(), load


def resolve_cached(sel, n_sel, page_base, page2cluster, cluster_base, replica_mask, cluster_size, resident, freq, D,
                   t_base, t_transfer, flags=0):
    """Eq. 8 with the resident term plus cache bookkeeping.  Returns (uniq, queue_of, load, n_hit, freq_new, score);
    ``freq`` is not modified."""
    sel = _arr(sel, np.int32)
    n_sel = _arr(n_sel, np.int32)
    page_base = _arr(page_base, np.int64)
    page2cluster = _arr(page2cluster, np.int32)
    cluster_base = _arr(cluster_base, np.int64)
    replica_mask = _arr(replica_mask, np.uint32)
    cluster_size = _arr(cluster_size, np.uint16)
    resident = _arr(resident, np.uint8)
    freq_new = np.array(freq, dtype=np.int32, copy=True)
    B, Hq, k = sel.shape
    cap = max(int(cluster_base[-1]), 1)
    uniq = np.empty(cap, dtype=np.int32)
    queue_of = np.empty(cap, dtype=np.uint8)
    n_uniq = np.zeros(1, dtype=np.int32)
    n_hit = np.zeros(1, dtype=np.int32)
    load = np.zeros(D, dtype=np.int32)
    score = np.zeros(cap, dtype=np.float64)
    rc = _load().oracle_resolve_cached(_p(sel), _p(n_sel), _p(page_base), _p(page2cluster), _p(cluster_base),
                                       _p(replica_mask), _p(cluster_size), _p(resident), _p(freq_new),
                                       ctypes.c_double(t_base), ctypes.c_double(t_transfer), ctypes.c_int32(B),
                                       ctypes.c_int32(Hq), ctypes.c_int32(k), ctypes.c_int32(D), ctypes.c_uint32(flags),
                                       _p(uniq), _p(queue_of), _p(n_uniq), _p(load), _p(n_hit), _p(score))
    _check(rc, "resolve_cached")
    n = int(n_uniq[0])
    return uniq[:n].copy(), queue_of[:n].copy(), load, int(n_hit[0]), freq_new, score[: int(cluster_base[-1])]


def gather(kv_pool, sel, n_sel, page_base, ctx_len, Hkv, d, S):
    """Returns (k_g, v_g uint16 [B][Hq][k*S][d] zero padded, n_tok int32 [B][Hq])."""
    kv_pool = _arr(kv_pool, np.uint16)
    sel = _arr(sel, np.int32)
    n_sel = _arr(n_sel, np.int32)
    page_base = _arr(page_base, np.int64)
    ctx_len = _arr(ctx_len, np.int32)
    B, Hq, k = sel.shape
    k_g = np.empty((B, Hq, k * S, d), dtype=np.uint16)
    v_g = np.empty((B, Hq, k * S, d), dtype=np.uint16)
    n_tok = np.empty((B, Hq), dtype=np.int32)
    rc = _load().oracle_gather(_p(kv_pool), _p(sel), _p(n_sel), _p(page_base), _p(ctx_len), ctypes.c_int32(B),
                               ctypes.c_int32(Hq), ctypes.c_int32(Hkv), ctypes.c_int32(d), ctypes.c_int32(S),
                               ctypes.c_int32(k), _p(k_g), _p(v_g), _p(n_tok))
    _check(rc, "gather")
    return k_g, v_g, n_tok


def attention(q, k_g, v_g, n_tok):
    """q uint16 [B][Hq][d], k_g/v_g uint16 [B][Hq][rows][d] -> (out float64 [B][Hq][d], lse float64 [B][Hq])."""
    q = _arr(q, np.uint16)
    k_g = _arr(k_g, np.uint16)
    v_g = _arr(v_g, np.uint16)
    n_tok = _arr(n_tok, np.int32)
    B, Hq, d = q.shape
    rows = k_g.shape[2]
    out = np.empty((B, Hq, d), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    rc = _load().oracle_attention(_p(q), _p(k_g), _p(v_g), _p(n_tok), ctypes.c_int32(B), ctypes.c_int32(Hq),
                                  ctypes.c_int32(d), ctypes.c_int64(rows), _p(out), _p(lse))
    _check(rc, "attention")
    return out, lse


@dataclass
class StepResult:
    score64: np.ndarray
    score32: np.ndarray
    cond: np.ndarray
    sel: np.ndarray
    n_sel: np.ndarray
    uniq: np.ndarray
    queue_of: np.ndarray
    load: np.ndarray
    k_g: np.ndarray
    v_g: np.ndarray
    n_tok: np.ndarray
    out: np.ndarray
    lse: np.ndarray


def step(q, ksum, kv_pool, page_base, ctx_len, page2cluster, cluster_base, replica_mask, cluster_size, *, Hkv, S, k,
         D, Pmax, flags=0, window=0, sel_override=None) -> StepResult:
    """The whole path, stage after stage.  ``sel_override=(sel, n_sel)`` replaces the oracle's own selection
    for the downstream stages (stage-conditional parity)."""
    d = np.asarray(q).shape[-1]
    s64, s32, cond = scores(q, ksum, page_base, ctx_len, Hkv, S, Pmax)
    sel, n_sel = topk(s32, ctx_len, S, k, window)
    use_sel, use_n = (sel, n_sel) if sel_override is None else sel_override
    uniq, queue_of, load = resolve(use_sel, use_n, page_base, page2cluster, cluster_base, replica_mask,
                                   cluster_size, D, flags)
    k_g, v_g, n_tok = gather(kv_pool, use_sel, use_n, page_base, ctx_len, Hkv, d, S)
    out, lse = attention(q, k_g, v_g, n_tok)
    return StepResult(s64, s32, cond, sel, n_sel, uniq, queue_of, load, k_g, v_g, n_tok, out, lse)


# ---- cluster-granular selection through the medoid index (Sec. 4.2, Tier 1 (1); Sec. 4.1) -------------------
def medoid_rows(ksum, page_base, cluster_base, medoid_page):
    """Index build: row c = the key summary of cluster c's medoid page (c a global cluster id)."""
    ksum = np.asarray(ksum)
    page_base, cluster_base = np.asarray(page_base), np.asarray(cluster_base)
    medoid_page = np.asarray(medoid_page)
    rows = np.zeros((int(cluster_base[-1]),) + ksum.shape[1:], dtype=ksum.dtype)
    for b in range(len(cluster_base) - 1):
        for c in range(int(cluster_base[b]), int(cluster_base[b + 1])):
            rows[c] = ksum[int(page_base[b]) + int(medoid_page[c])]
    return rows


def expand_clusters(sel_c, n_sel_c, cluster_base, cluster_page_ptr, cluster_pages, ctx_len=None, S=None, window=0):
    """Pages of the selected clusters of every (request, head): ascending page id, -1 padded, and their number.
    With ``window`` > 0 the last ``window`` pages of the request (Sec. 4.2, Tier 1 (2): the local window) belong
    to every head's set as well; ``ctx_len`` and the page size ``S`` then give each request's page count."""
    sel_c, n_sel_c = np.asarray(sel_c), np.asarray(n_sel_c)
    B, Hq, _ = sel_c.shape
    lists = [[None] * Hq for _ in range(B)]
    width = 1
    for b in range(B):
        P_b = -(-int(ctx_len[b]) // int(S)) if window > 0 else 0
        for h in range(Hq):
            pages = set(range(max(0, P_b - int(window)), P_b))
            for j in range(int(n_sel_c[b, h])):
                c = int(cluster_base[b]) + int(sel_c[b, h, j])
                pages.update(int(p) for p in cluster_pages[int(cluster_page_ptr[c]):int(cluster_page_ptr[c + 1])])
            lists[b][h] = sorted(pages)
            width = max(width, len(pages))
    sel_p = np.full((B, Hq, width), -1, dtype=np.int32)
    n_sel_p = np.zeros((B, Hq), dtype=np.int32)
    for b in range(B):
        for h in range(Hq):
            n_sel_p[b, h] = len(lists[b][h])
            sel_p[b, h, :len(lists[b][h])] = lists[b][h]
    return sel_p, n_sel_p


@dataclass
class MedoidStepResult:
    score64: np.ndarray
    score32: np.ndarray
    cond: np.ndarray
    sel_clusters: np.ndarray
    n_sel_clusters: np.ndarray
    sel_pages: np.ndarray
    n_sel_pages: np.ndarray
    uniq: np.ndarray
    queue_of: np.ndarray
    load: np.ndarray
    out: np.ndarray
    lse: np.ndarray


def medoid_step(q, ksum, kv_pool, page_base, ctx_len, page2cluster, cluster_base, replica_mask, cluster_size,
                cluster_page_ptr, cluster_pages, medoid_page, *, Hkv, S, k_c, D, flags=0,
                sel_override=None, window=0) -> MedoidStepResult:
    """The step with the medoid index: each cluster is scored by the page upper bound of its medoid page, the k_c
    best clusters of every head are retrieved whole, and the head attends to all of their pages.  The index is a
    context of its own whose "pages" are the clusters, so stages 1-2 are the page routines run on it."""
    d = np.asarray(q).shape[-1]
    cluster_base = np.asarray(cluster_base)
    n_c = (cluster_base[1:] - cluster_base[:-1]).astype(np.int64)
    rows = medoid_rows(ksum, page_base, cluster_base, medoid_page)
    len_c = (n_c * S).astype(np.int32)
    s64, s32, cond = scores(q, rows, cluster_base, len_c, Hkv, S, int(max(1, n_c.max())))
    sel_c, n_sel_c = topk(s32, len_c, S, k_c)
    use_c, use_n = (sel_c, n_sel_c) if sel_override is None else sel_override
    sel_p, n_sel_p = expand_clusters(use_c, use_n, cluster_base, cluster_page_ptr, cluster_pages, ctx_len, S, window)
    uniq, queue_of, load = resolve(sel_p, n_sel_p, page_base, page2cluster, cluster_base, replica_mask, cluster_size,
                                   D, flags)
    k_g, v_g, n_tok = gather(kv_pool, sel_p, n_sel_p, page_base, ctx_len, Hkv, d, S)
    out, lse = attention(q, k_g, v_g, n_tok)
    return MedoidStepResult(s64, s32, cond, sel_c, n_sel_c, sel_p, n_sel_p, uniq, queue_of, load, out, lse)


# ---- batched submission order (Sec. 5.1, last paragraph) ------------------------------------------------------
def submit_order(queue_of, replica_mask_of_uniq, D, flags=0):
    """Order in which the fetched clusters are submitted: the head of every bucket (queue) is taken, queue after
    queue, into one batch; then the next heads; and so on until the buckets are empty.  A bucket holds its
    clusters in the order the scheduling pass assigned them: by (number of replicas ascending, position in uniq
    ascending), or by position alone under ORDER_BY_ID.
    queue_of[i] / replica_mask_of_uniq[i] belong to uniq[i].  Returns (order, n_rounds): order[j] is the index
    into uniq of the j-th submitted cluster."""
    queue_of = np.asarray(queue_of)
    masks = np.asarray(replica_mask_of_uniq, dtype=np.uint32)
    n = len(queue_of)
    visit = list(range(n))
    if not (flags & ORDER_BY_ID):
        visit.sort(key=lambda i: (bin(int(masks[i])).count("1"), i))
    buckets = [[] for _ in range(D)]
    for i in visit:
        q = int(queue_of[i])
        if q < D:                                            # clusters with a bad replica mask (0xFF) are never submitted
            buckets[q].append(i)
    order = []
    rounds = max((len(b) for b in buckets), default=0)
    for r in range(rounds):
        for q in range(D):
            if r < len(buckets[q]):
                order.append(buckets[q][r])
    return np.asarray(order, dtype=np.int32), rounds


# ---- Algorithm 1: offline co-activation clustering ------------------------------------------------------------
def build_clusters(dist, tau, members_cap=None):
    """dist float32 [n][n], tau -> (rho int32 [n], ptr int32 [C + 1], members int32, medoid int32 [C]).
    Clusters in creation order; members in joining order, medoid first; an entry may sit in several clusters."""
    dist = np.ascontiguousarray(dist, dtype=np.float32)
    n = dist.shape[0]
    assert dist.shape == (n, n)
    cap = int(members_cap if members_cap is not None else max(1, n) * 64)
    rho = np.zeros(n, dtype=np.int32)
    ptr = np.zeros(n + 1, dtype=np.int32)
    members = np.zeros(cap, dtype=np.int32)
    medoid = np.zeros(n, dtype=np.int32)
    n_c = np.zeros(1, dtype=np.int32)
    _check(_load().oracle_build_clusters(_p(dist), ctypes.c_int32(n), ctypes.c_float(tau), _p(rho), _p(ptr),
                                         _p(members), ctypes.c_int64(cap), _p(medoid), _p(n_c)), "build_clusters")
    C = int(n_c[0])
    return rho, ptr[:C + 1].copy(), members[:int(ptr[C])].copy(), medoid[:C].copy()


def build_clusters_plain(dist, tau, members_cap=None, near_rtol=1e-5):
    """Algorithm 1 with Step 4's test as Eq. 5 prints it: the average distance to the current members, recomputed
    from scratch in double for every candidate.  Returns (rho, ptr, members, medoid, n_near) where n_near counts
    the join decisions within near_rtol * tau of the radius."""
    dist = np.ascontiguousarray(dist, dtype=np.float32)
    n = dist.shape[0]
    assert dist.shape == (n, n)
    cap = int(members_cap if members_cap is not None else max(1, n) * 64)
    rho = np.zeros(n, dtype=np.int32)
    ptr = np.zeros(n + 1, dtype=np.int32)
    members = np.zeros(cap, dtype=np.int32)
    medoid = np.zeros(n, dtype=np.int32)
    n_c = np.zeros(1, dtype=np.int32)
    n_near = np.zeros(1, dtype=np.int64)
    _check(_load().oracle_build_clusters_plain(_p(dist), ctypes.c_int32(n), ctypes.c_float(tau),
                                               ctypes.c_double(near_rtol), _p(rho), _p(ptr), _p(members),
                                               ctypes.c_int64(cap), _p(medoid), _p(n_c), _p(n_near)),
           "build_clusters_plain")
    C = int(n_c[0])
    return rho, ptr[:C + 1].copy(), members[:int(ptr[C])].copy(), medoid[:C].copy(), int(n_near[0])


def replay_clusters(dist, tau, ptr, members, medoid, near_rtol=1e-5):
    """Band rule for a clustering someone else computed (Algorithm 1; Eq. 4, Eq. 5).  Walks the given clusters in
    order and checks every step against the plain statement: the medoid is the first uncovered entry of the queue
    (density descending, index ascending), the candidates are visited by (distance to the medoid, index), and a
    candidate joined exactly when the average of its distances to the members so far -- recomputed in double -- is
    <= tau, EXCEPT that a decision whose margin |average - tau| is at most near_rtol * tau may go either way (the
    replay then follows the given clustering).  Returns the number of such near decisions; raises AssertionError
    on the first step that is wrong outside the band."""
    d32 = np.ascontiguousarray(dist, dtype=np.float32)
    n = d32.shape[0]
    d64 = d32.astype(np.float64)
    tau32, tau64 = np.float32(tau), float(np.float32(tau))
    within = d32 <= tau32
    rho = within.sum(axis=1) - within.diagonal().astype(np.int64)
    queue = sorted(range(n), key=lambda i: (-int(rho[i]), i))
    covered = np.zeros(n, dtype=bool)
    qi, near = 0, 0
    ptr, members, medoid = np.asarray(ptr), np.asarray(members), np.asarray(medoid)
    for c in range(len(medoid)):
        assert not covered.all(), "a cluster was created after every entry was covered"
        while covered[queue[qi]]:
            qi += 1
        m = queue[qi]
        assert int(medoid[c]) == m, f"cluster {c}: medoid {int(medoid[c])}, expected {m}"
        given = members[ptr[c]:ptr[c + 1]].tolist()
        assert given and given[0] == m, f"cluster {c} does not start with its medoid"
        idx = np.flatnonzero(within[m])
        idx = idx[idx != m]
        cand = idx[np.lexsort((idx, d32[m, idx]))].tolist()     # by (distance to the medoid, index)
        mem, gi = [m], 1
        for e in cand:
            avg = float(d64[mem, e].sum() / len(mem))
            joined = gi < len(given) and given[gi] == e
            if abs(avg - tau64) <= near_rtol * tau64:
                near += 1
            else:
                assert joined == (avg <= tau64), \
                    f"cluster {c}, candidate {e}: average {avg!r} vs tau {tau64!r}, joined={joined}"
            if joined:
                mem.append(e)
                gi += 1
        assert gi == len(given), f"cluster {c} holds entries that are not candidates, or out of order"
        covered[mem] = True
    assert covered.all(), "entries left uncovered"
    return near


# ---- placement of the clusters' entries across the SSDs (Eq. 7) and entry-level scheduling --------------------
def entry_replica_masks(cluster_ptr, cluster_members, n_entries, D):
    """Round-robin placement of Eq. 7: clusters are laid out one after another, a global pointer advances by one
    disk per stored entry, so the j-th entry of cluster i lands on disk (|C_0| + ... + |C_{i-1}| + j) mod D.
    An entry stored with several clusters has one copy per cluster; returns, per entry, the set of disks holding
    a copy as a bit mask (uint32 [n_entries])."""
    cluster_ptr, cluster_members = np.asarray(cluster_ptr), np.asarray(cluster_members)
    masks = np.zeros(n_entries, dtype=np.uint32)
    p_global = 0
    for c in range(len(cluster_ptr) - 1):
        disk = p_global % D                                  # id_i of Eq. 7
        for j in range(int(cluster_ptr[c]), int(cluster_ptr[c + 1])):
            masks[int(cluster_members[j])] |= np.uint32(1 << ((disk + (j - int(cluster_ptr[c]))) % D))
        p_global += int(cluster_ptr[c + 1] - cluster_ptr[c])
    return masks


# ---- which clusters the fast tier holds (Sec. 4.2, Tier 1 (3): cached in descending order of the Eq. 6 score) ----
def cache_admit(score, cluster_size, capacity_pages):
    """Clusters are taken in descending score (ties to the lower id) while they still fit into the capacity,
    counted in pages; the first one that does not fit ends the admission.  Returns (resident uint8 [C],
    clusters admitted, pages used)."""
    score = np.asarray(score, dtype=np.float32)
    size = np.asarray(cluster_size).astype(np.int64)
    order = sorted(range(len(score)), key=lambda c: (-float(score[c]), c))
    resident = np.zeros(len(score), dtype=np.uint8)
    used = 0
    n = 0
    for c in order:
        if used + int(size[c]) > capacity_pages:
            break
        resident[c] = 1
        used += int(size[c])
        n += 1
    return resident, n, used
