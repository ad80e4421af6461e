// swarm_oracle.cpp -- CPU oracle for the per-decode-step KVCache retrieval path.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
// statement of what the retrieval path computes.  It is used by the tests, by
// the smoke check and by the benchmark's CPU-baseline leg.  The CUDA library
// never links, includes or calls anything in here, and nothing in here
// includes anything of the CUDA library: the two share no code.
//
// What each function follows:
//   oracle_build_summaries  per-page element-wise min / max of the keys (the
//                           index the scorer reads; the paper keeps a compact
//                           per-cluster index in fast memory, Sec. 4.2 Tier 1)
//   oracle_scores           relevance score of a page against the query
//                           (Sec. 2.3 scores entries by relevance, e.g. by the
//                           query-key inner product): the page upper bound
//                           sum_i max(q_i*kmin_i, q_i*kmax_i)
//   oracle_topk             Sec. 2.3 activates the best-scoring entries alone:
//                           k best pages per query head, ties to the lower id
//   oracle_resolve          global merge (Eq. 8, without the DRAM-resident
//                           term) and entry-bucket scheduling (Sec. 5.1): sort
//                           by replication factor ascending, route each item
//                           to its currently smallest bucket
//   oracle_resolve_cached   the same with Eq. 8's resident term, the activation-frequency update of
//                           Sec. 5.2 (cache replacement) and the cost-effectiveness score of Eq. 6
//   oracle_gather           the transfer of the selected pages (Sec. 6, the
//                           asynchronous reads), here a byte copy
//   oracle_attention        Eq. 1 over the gathered tokens, one query row
//   oracle_build_clusters   Algorithm 1 (offline co-activation clustering): density of Eq. 4, medoid queue,
//                           expansion by the average distance of Eq. 5; decisions in fp32 (see the function)
//
// Parity status: nothing numeric in the paper pins this path (it prints no
// worked example for it), so against the authors' system every function here
// is "parity unpinned".  Each function is pinned instead to closed forms,
// invariants, library routines on special cases and brute force on tiny
// inputs by the CPU test-suite.
//
// Arithmetic: double accumulation in index order; bf16 inputs are widened
// exactly.  Loops are written in the order of the definitions; the only
// concession to speed is an OpenMP "parallel for" over independent
// (request, head) units, which changes no result.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <set>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline double bf16(uint16_t bits) {
  uint32_t u = static_cast<uint32_t>(bits) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return static_cast<double>(f);
}

inline int64_t pages_of(int32_t ctx_len, int32_t S) { return (static_cast<int64_t>(ctx_len) + S - 1) / S; }

inline int popcount32(uint32_t x) {
  int n = 0;
  while (x) { n += static_cast<int>(x & 1u); x >>= 1; }
  return n;
}

}  // namespace

extern "C" {

enum { ORACLE_OK = 0, ORACLE_BAD_ARG = 1, ORACLE_BAD_TABLE = 2, ORACLE_NONFINITE = 3 };
enum { ORACLE_ORDER_BY_ID = 1u, ORACLE_UNIT_LOAD = 2u };

int oracle_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
  return omp_get_max_threads();
#else
  (void)n;
  return 1;
#endif
}

// ksum[page][kvh][0][i] = min over the page's valid tokens of K[token][i], [1] = max.
// Only the last page of a request can be partial; its padding tokens are ignored.
int oracle_build_summaries(const uint16_t* kv_pool, const int64_t* page_base, const int32_t* ctx_len,
                           int32_t B, int32_t Hkv, int32_t d, int32_t S, uint16_t* ksum) {
  if (!kv_pool || !page_base || !ctx_len || !ksum || B < 1 || Hkv < 1 || d < 1 || S < 1) return ORACLE_BAD_ARG;
  for (int32_t b = 0; b < B; ++b) {
    const int64_t P = pages_of(ctx_len[b], S);
    if (ctx_len[b] < 1 || P > page_base[b + 1] - page_base[b]) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p) {
      const int64_t valid = (p == P - 1) ? ctx_len[b] - static_cast<int64_t>(S) * (P - 1) : S;
      const int64_t page = page_base[b] + p;
      for (int32_t kv = 0; kv < Hkv; ++kv) {
        const uint16_t* K = kv_pool + ((page * Hkv + kv) * 2 + 0) * static_cast<int64_t>(S) * d;
        uint16_t* lo = ksum + ((page * Hkv + kv) * 2 + 0) * static_cast<int64_t>(d);
        uint16_t* hi = ksum + ((page * Hkv + kv) * 2 + 1) * static_cast<int64_t>(d);
        for (int32_t i = 0; i < d; ++i) {
          uint16_t bmin = K[i], bmax = K[i];
          for (int64_t t = 1; t < valid; ++t) {
            const uint16_t x = K[t * d + i];
            if (bf16(x) < bf16(bmin)) bmin = x;
            if (bf16(x) > bf16(bmax)) bmax = x;
          }
          lo[i] = bmin;
          hi[i] = bmax;
        }
      }
    }
  }
  return ORACLE_OK;
}

// score64[b][h][p] = sum_{i<d} max(q[b][h][i]*kmin[p][i], q[b][h][i]*kmax[p][i]),  kv(h) = h / (Hq/Hkv).
// cond[b][h][p]    = sum_i max(|q*kmin|, |q*kmax|)  (size of the terms; used for a rounding floor).
// Entries p >= P_b are left untouched.
int oracle_scores(const uint16_t* q, const uint16_t* ksum, const int64_t* page_base, const int32_t* ctx_len,
                  int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t S, int64_t Pmax,
                  double* score64, float* score32, double* cond) {
  if (!q || !ksum || !page_base || !ctx_len || !score64 || B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv || d < 1 || S < 1)
    return ORACLE_BAD_ARG;
  const int32_t g = Hq / Hkv;
  for (int32_t b = 0; b < B; ++b)
    if (ctx_len[b] < 1 || pages_of(ctx_len[b], S) > Pmax) return ORACLE_BAD_ARG;
  int bad = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1) reduction(| : bad)
  for (int32_t b = 0; b < B; ++b) {
    for (int32_t h = 0; h < Hq; ++h) {
      const int64_t P = pages_of(ctx_len[b], S);
      const int32_t kv = h / g;
      const uint16_t* qv = q + (static_cast<int64_t>(b) * Hq + h) * d;
      for (int64_t p = 0; p < P; ++p) {
        const uint16_t* lo = ksum + (((page_base[b] + p) * Hkv + kv) * 2 + 0) * static_cast<int64_t>(d);
        const uint16_t* hi = lo + d;
        double s = 0.0, a = 0.0;
        for (int32_t i = 0; i < d; ++i) {
          const double x = bf16(qv[i]) * bf16(lo[i]);
          const double y = bf16(qv[i]) * bf16(hi[i]);
          s += std::max(x, y);
          a += std::max(std::fabs(x), std::fabs(y));
        }
        if (!std::isfinite(s)) bad = 1;
        const int64_t o = (static_cast<int64_t>(b) * Hq + h) * Pmax + p;
        score64[o] = s;
        if (score32) score32[o] = static_cast<float>(s);
        if (cond) cond[o] = a;
      }
    }
  }
  return bad ? ORACLE_NONFINITE : ORACLE_OK;
}

// Per (b,h): order the P_b pages by (score descending, page id ascending), keep the first
// k_eff = min(k, P_b), and emit them in ascending page id.  Unused slots are -1.
// Scores compare as real numbers (so -0 == +0).
// Local window (Sec. 4.2, Tier 1 (2)): the last `window` pages of a request are always kept -- they rank
// above every score -- and the remaining k - window places go to the best of the other pages.
int oracle_topk(const float* score, const int32_t* ctx_len, int32_t B, int32_t Hq, int32_t S, int64_t Pmax,
                int32_t k, int32_t window, int32_t* sel, int32_t* n_sel) {
  if (!score || !ctx_len || !sel || !n_sel || B < 1 || Hq < 1 || S < 1 || k < 1 || window < 0 || window > k)
    return ORACLE_BAD_ARG;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int32_t b = 0; b < B; ++b) {
    for (int32_t h = 0; h < Hq; ++h) {
      const int64_t P = pages_of(ctx_len[b], S);
      const float* s = score + (static_cast<int64_t>(b) * Hq + h) * Pmax;
      std::vector<int32_t> ids(static_cast<size_t>(P));
      for (int64_t p = 0; p < P; ++p) ids[static_cast<size_t>(p)] = static_cast<int32_t>(p);
      const int64_t first_window = P - window;              // pages >= this are in the local window
      std::stable_sort(ids.begin(), ids.end(), [s, first_window](int32_t a, int32_t c) {
        const bool wa = a >= first_window, wc = c >= first_window;
        if (wa != wc) return wa;                            // window pages first
        if (wa) return false;                               // among themselves: keep id order
        return s[a] > s[c];
      });
      const int64_t k_eff = std::min<int64_t>(k, P);
      std::vector<int32_t> best(ids.begin(), ids.begin() + k_eff);
      std::sort(best.begin(), best.end());
      int32_t* out = sel + (static_cast<int64_t>(b) * Hq + h) * k;
      for (int64_t j = 0; j < k; ++j) out[j] = j < k_eff ? best[static_cast<size_t>(j)] : -1;
      n_sel[static_cast<int64_t>(b) * Hq + h] = static_cast<int32_t>(k_eff);
    }
  }
  return ORACLE_OK;
}

namespace {

// The activated clusters: G = { cluster_base[b] + page2cluster[page_base[b] + p] : p selected by any head of b }.
int collect_activated(const int32_t* sel, const int32_t* n_sel, const int64_t* page_base, const int32_t* page2cluster,
                      const int64_t* cluster_base, int32_t B, int32_t Hq, int32_t k, std::set<int64_t>& G) {
  for (int32_t b = 0; b < B; ++b) {
    const int64_t n_pages = page_base[b + 1] - page_base[b];
    const int64_t n_clusters = cluster_base[b + 1] - cluster_base[b];
    for (int32_t h = 0; h < Hq; ++h) {
      const int64_t bh = static_cast<int64_t>(b) * Hq + h;
      if (n_sel[bh] < 0 || n_sel[bh] > k) return ORACLE_BAD_ARG;
      for (int32_t j = 0; j < n_sel[bh]; ++j) {
        const int32_t p = sel[bh * k + j];
        if (p < 0 || p >= n_pages) return ORACLE_BAD_TABLE;
        const int32_t c = page2cluster[page_base[b] + p];
        if (c < 0 || c >= n_clusters) return ORACLE_BAD_TABLE;
        G.insert(cluster_base[b] + c);
      }
    }
  }
  return ORACLE_OK;
}

// Bucket scheduling of the clusters in `fetch` (ascending id):
//   order by (number of replicas ascending, id ascending)   [id ascending only, under ORDER_BY_ID]
//   for c in that order: q* = the replica queue of c with the smallest (load, queue id);
//                        queue_of[c] = q*;  load[q*] += cluster_size[c]   [+= 1 under UNIT_LOAD]
int schedule(const std::vector<int64_t>& fetch, const uint32_t* replica_mask, const uint16_t* cluster_size, int32_t D,
             uint32_t flags, int32_t* uniq, uint8_t* queue_of, int32_t* n_uniq, int32_t* load) {
  const uint32_t valid_bits = D == 32 ? 0xFFFFFFFFu : ((1u << D) - 1u);
  std::vector<int64_t> order(fetch);
  for (int64_t c : order)
    if (replica_mask[c] == 0 || (replica_mask[c] & ~valid_bits)) return ORACLE_BAD_TABLE;
  if (!(flags & ORACLE_ORDER_BY_ID))
    std::stable_sort(order.begin(), order.end(), [replica_mask](int64_t a, int64_t c) {
      return popcount32(replica_mask[a]) < popcount32(replica_mask[c]);
    });
  std::vector<int64_t> L(static_cast<size_t>(D), 0);
  std::vector<std::pair<int64_t, int>> placed;  // (cluster id, queue)
  for (int64_t c : order) {
    int best = -1;
    for (int qd = 0; qd < D; ++qd)
      if ((replica_mask[c] >> qd) & 1u)
        if (best < 0 || L[static_cast<size_t>(qd)] < L[static_cast<size_t>(best)]) best = qd;
    L[static_cast<size_t>(best)] += (flags & ORACLE_UNIT_LOAD) ? 1 : cluster_size[c];
    placed.emplace_back(c, best);
  }
  std::sort(placed.begin(), placed.end());
  for (size_t i = 0; i < placed.size(); ++i) {
    uniq[i] = static_cast<int32_t>(placed[i].first);
    queue_of[i] = static_cast<uint8_t>(placed[i].second);
  }
  *n_uniq = static_cast<int32_t>(placed.size());
  for (int qd = 0; qd < D; ++qd) load[qd] = static_cast<int32_t>(L[static_cast<size_t>(qd)]);
  return ORACLE_OK;
}

}  // namespace

// Global merge + bucket scheduling: every activated cluster is fetched (Eq. 8 without the resident term).
// Output: uniq ascending by id, queue_of parallel to uniq, load[D], n_uniq.
int oracle_resolve(const int32_t* sel, const int32_t* n_sel, const int64_t* page_base,
                   const int32_t* page2cluster, const int64_t* cluster_base, const uint32_t* replica_mask,
                   const uint16_t* cluster_size, int32_t B, int32_t Hq, int32_t k, int32_t D, uint32_t flags,
                   int32_t* uniq, uint8_t* queue_of, int32_t* n_uniq, int32_t* load) {
  if (!sel || !n_sel || !page_base || !page2cluster || !cluster_base || !replica_mask || !cluster_size || !uniq ||
      !queue_of || !n_uniq || !load || B < 1 || Hq < 1 || k < 1 || D < 1 || D > 32)
    return ORACLE_BAD_ARG;
  std::set<int64_t> G;
  const int rc = collect_activated(sel, n_sel, page_base, page2cluster, cluster_base, B, Hq, k, G);
  if (rc != ORACLE_OK) return rc;
  return schedule(std::vector<int64_t>(G.begin(), G.end()), replica_mask, cluster_size, D, flags, uniq, queue_of,
                  n_uniq, load);
}

// Global merge with the resident term (Eq. 8) and the cache bookkeeping of Sec. 5.2 / Eq. 6:
//   A = activated clusters;  E_IO = A \ resident  is scheduled as above;  n_hit = |A and resident|
//   freq[c] += 1 for c in A;  freq[c] -= 1 for resident c not in A
//   score[c] = freq[c] * (t_base + size[c] * t_transfer) / size[c]   for every cluster, after the update
int oracle_resolve_cached(const int32_t* sel, const int32_t* n_sel, const int64_t* page_base,
                          const int32_t* page2cluster, const int64_t* cluster_base, const uint32_t* replica_mask,
                          const uint16_t* cluster_size, const uint8_t* resident, int32_t* freq, double t_base,
                          double t_transfer, int32_t B, int32_t Hq, int32_t k, int32_t D, uint32_t flags,
                          int32_t* uniq, uint8_t* queue_of, int32_t* n_uniq, int32_t* load, int32_t* n_hit,
                          double* score) {
  if (!sel || !n_sel || !page_base || !page2cluster || !cluster_base || !replica_mask || !cluster_size || !resident ||
      !freq || !uniq || !queue_of || !n_uniq || !load || !n_hit || !score || B < 1 || Hq < 1 || k < 1 || D < 1 || D > 32)
    return ORACLE_BAD_ARG;
  std::set<int64_t> A;
  const int rc = collect_activated(sel, n_sel, page_base, page2cluster, cluster_base, B, Hq, k, A);
  if (rc != ORACLE_OK) return rc;
  const int64_t n_clusters = cluster_base[B];
  std::vector<int64_t> fetch;
  int32_t hits = 0;
  for (int64_t c : A) {
    freq[c] += 1;
    if (resident[c]) ++hits; else fetch.push_back(c);
  }
  for (int64_t c = 0; c < n_clusters; ++c)
    if (resident[c] && A.find(c) == A.end()) freq[c] -= 1;
  for (int64_t c = 0; c < n_clusters; ++c)
    score[c] = static_cast<double>(freq[c]) * (t_base + cluster_size[c] * t_transfer) / cluster_size[c];
  *n_hit = hits;
  return schedule(fetch, replica_mask, cluster_size, D, flags, uniq, queue_of, n_uniq, load);
}

// Kg/Vg[b][h][j*S + t][:] = pool[page_base[b] + sel[b][h][j]][kv(h)][K/V][t][:] for the valid tokens of the
// page; everything else in the [k*S][d] slab is zero.  n_tok[b][h] = number of valid tokens copied.
int oracle_gather(const uint16_t* kv_pool, const int32_t* sel, const int32_t* n_sel, const int64_t* page_base,
                  const int32_t* ctx_len, int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t S, int32_t k,
                  uint16_t* k_out, uint16_t* v_out, int32_t* n_tok) {
  if (!kv_pool || !sel || !n_sel || !page_base || !ctx_len || !k_out || !v_out || !n_tok || Hq % Hkv)
    return ORACLE_BAD_ARG;
  const int32_t g = Hq / Hkv;
  const int64_t blk = static_cast<int64_t>(S) * d;
  for (int32_t b = 0; b < B; ++b) {
    const int64_t P = pages_of(ctx_len[b], S);
    for (int32_t h = 0; h < Hq; ++h) {
      const int64_t bh = static_cast<int64_t>(b) * Hq + h;
      uint16_t* Ko = k_out + bh * k * blk;
      uint16_t* Vo = v_out + bh * k * blk;
      std::fill(Ko, Ko + k * blk, uint16_t{0});
      std::fill(Vo, Vo + k * blk, uint16_t{0});
      int64_t rows = 0;
      for (int32_t j = 0; j < n_sel[bh]; ++j) {
        const int64_t p = sel[bh * k + j];
        if (p < 0 || p >= P) return ORACLE_BAD_TABLE;
        const int64_t valid = (p == P - 1) ? ctx_len[b] - static_cast<int64_t>(S) * (P - 1) : S;
        const uint16_t* Kp = kv_pool + (((page_base[b] + p) * Hkv + h / g) * 2 + 0) * blk;
        const uint16_t* Vp = Kp + blk;
        for (int64_t t = 0; t < valid; ++t)
          for (int32_t i = 0; i < d; ++i) {
            Ko[(static_cast<int64_t>(j) * S + t) * d + i] = Kp[t * d + i];
            Vo[(static_cast<int64_t>(j) * S + t) * d + i] = Vp[t * d + i];
          }
        rows += valid;
      }
      n_tok[bh] = static_cast<int32_t>(rows);
    }
  }
  return ORACLE_OK;
}

// One query row per (b,h) against its own T = n_tok[b][h] gathered tokens (Eq. 1):
//   x_t = (q . K_t) / sqrt(d);  m = max_t x_t;  l = sum_t exp(x_t - m)
//   out = sum_t exp(x_t - m) V_t / l;  lse = m + ln l
// k_g, v_g are [B][Hq][rows][d] bf16 with rows >= n_tok.
int oracle_attention(const uint16_t* q, const uint16_t* k_g, const uint16_t* v_g, const int32_t* n_tok, int32_t B,
                     int32_t Hq, int32_t d, int64_t rows, double* out, double* lse) {
  if (!q || !k_g || !v_g || !n_tok || !out || !lse || B < 1 || Hq < 1 || d < 1) return ORACLE_BAD_ARG;
  for (int64_t bh = 0; bh < static_cast<int64_t>(B) * Hq; ++bh)
    if (n_tok[bh] < 1 || n_tok[bh] > rows) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t bh = 0; bh < static_cast<int64_t>(B) * Hq; ++bh) {
    const int64_t T = n_tok[bh];
    const uint16_t* qv = q + bh * d;
    const uint16_t* K = k_g + bh * rows * d;
    const uint16_t* V = v_g + bh * rows * d;
    std::vector<double> x(static_cast<size_t>(T));
    double m = -INFINITY;
    for (int64_t t = 0; t < T; ++t) {
      double s = 0.0;
      for (int32_t i = 0; i < d; ++i) s += bf16(qv[i]) * bf16(K[t * d + i]);
      x[static_cast<size_t>(t)] = s / std::sqrt(static_cast<double>(d));
      m = std::max(m, x[static_cast<size_t>(t)]);
    }
    double l = 0.0;
    for (int64_t t = 0; t < T; ++t) l += std::exp(x[static_cast<size_t>(t)] - m);
    for (int32_t i = 0; i < d; ++i) {
      double acc = 0.0;
      for (int64_t t = 0; t < T; ++t) acc += std::exp(x[static_cast<size_t>(t)] - m) * bf16(V[t * d + i]);
      out[bh * d + i] = acc / l;
    }
    lse[bh] = m + std::log(l);
  }
  return ORACLE_OK;
}

// Algorithm 1 (co-activation clustering) on a given distance matrix D [n][n] (fp32, row-major) and radius tau.
// Decisions depend on floating-point comparisons, so they are taken in fp32, the precision of the matrix:
//   density   rho[i] = #{ j != i : D[i][j] <= tau }                                   (Step 3; the listing's <=)
//   medoids   entries by (rho descending, index ascending); a covered entry is skipped
//   expansion C = {m}; candidates { e != m : D[m][e] <= tau } by (D[m][e] ascending, index ascending); every
//             candidate is visited once, in that order, and joins when the average of its distances to the
//             current members is <= tau.  The sum runs in fp32 in the order the members joined, reads
//             D[member][candidate], and is compared against tau * |C| (fp32 product).  Covered entries stay
//             candidates: that is how an entry comes to sit in several clusters.
//   stop      when every entry is covered.
// Output: clusters in creation order as CSR (ptr [n + 1] sized by the caller, members in joining order with the
// medoid first), medoid[c], rho[i].  Returns ORACLE_BAD_ARG if members_cap is too small.
int oracle_build_clusters(const float* D, int32_t n, float tau, int32_t* rho, int32_t* ptr, int32_t* members,
                          int64_t members_cap, int32_t* medoid, int32_t* n_clusters) {
  if (!D || !rho || !ptr || !members || !medoid || !n_clusters || n < 1) return ORACLE_BAD_ARG;
  for (int32_t i = 0; i < n; ++i) {
    int32_t c = 0;
    for (int32_t j = 0; j < n; ++j)
      if (j != i && D[static_cast<int64_t>(i) * n + j] <= tau) ++c;
    rho[i] = c;
  }
  std::vector<int32_t> queue(static_cast<size_t>(n));
  for (int32_t i = 0; i < n; ++i) queue[static_cast<size_t>(i)] = i;
  std::stable_sort(queue.begin(), queue.end(), [rho](int32_t a, int32_t b) { return rho[a] > rho[b]; });
  std::vector<char> covered(static_cast<size_t>(n), 0);
  int32_t n_cov = 0, nc = 0;
  int64_t fill = 0;
  ptr[0] = 0;
  for (int32_t qi = 0; qi < n && n_cov < n; ++qi) {
    const int32_t m = queue[static_cast<size_t>(qi)];
    if (covered[static_cast<size_t>(m)]) continue;
    const float* row_m = D + static_cast<int64_t>(m) * n;
    std::vector<int32_t> cand;
    for (int32_t e = 0; e < n; ++e)
      if (e != m && row_m[e] <= tau) cand.push_back(e);
    std::stable_sort(cand.begin(), cand.end(), [row_m](int32_t a, int32_t b) { return row_m[a] < row_m[b]; });
    std::vector<int32_t> mem{m};
    std::vector<float> sum(cand.size());
    for (size_t ci = 0; ci < cand.size(); ++ci) sum[ci] = row_m[cand[ci]];      // distance to the only member so far
    for (size_t ci = 0; ci < cand.size(); ++ci) {
      const float bound = tau * static_cast<float>(mem.size());
      if (sum[ci] <= bound) {
        const int32_t e = cand[ci];
        mem.push_back(e);
        const float* row_e = D + static_cast<int64_t>(e) * n;
        for (size_t cj = ci + 1; cj < cand.size(); ++cj) sum[cj] = sum[cj] + row_e[cand[cj]];
      }
    }
    if (fill + static_cast<int64_t>(mem.size()) > members_cap) return ORACLE_BAD_ARG;
    for (int32_t e : mem) {
      members[fill++] = e;
      if (!covered[static_cast<size_t>(e)]) { covered[static_cast<size_t>(e)] = 1; ++n_cov; }
    }
    medoid[nc] = m;
    ptr[++nc] = static_cast<int32_t>(fill);
  }
  *n_clusters = nc;
  return ORACLE_OK;
}

// Algorithm 1 again, with Step 4's test written as Eq. 5 states it: for every candidate the AVERAGE of its
// distances to the current members, recomputed from scratch in double over the members in joining order and
// compared with tau in double.  No running sums, nothing in fp32 beyond the matrix entries themselves.  Same
// density, medoid queue, candidate order and outputs as oracle_build_clusters.  *n_near counts the join
// decisions whose margin |average - tau| is at most near_rtol * tau: those are the decisions a different
// summation order or precision may legitimately take the other way.
int oracle_build_clusters_plain(const float* D, int32_t n, float tau, double near_rtol, int32_t* rho, int32_t* ptr,
                                int32_t* members, int64_t members_cap, int32_t* medoid, int32_t* n_clusters,
                                int64_t* n_near) {
  if (!D || !rho || !ptr || !members || !medoid || !n_clusters || !n_near || n < 1) return ORACLE_BAD_ARG;
  const double tau_d = static_cast<double>(tau);
  for (int32_t i = 0; i < n; ++i) {
    int32_t c = 0;
    for (int32_t j = 0; j < n; ++j)
      if (j != i && D[static_cast<int64_t>(i) * n + j] <= tau) ++c;
    rho[i] = c;
  }
  std::vector<int32_t> queue(static_cast<size_t>(n));
  for (int32_t i = 0; i < n; ++i) queue[static_cast<size_t>(i)] = i;
  std::stable_sort(queue.begin(), queue.end(), [rho](int32_t a, int32_t b) { return rho[a] > rho[b]; });
  std::vector<char> covered(static_cast<size_t>(n), 0);
  int32_t n_cov = 0, nc = 0;
  int64_t fill = 0, near = 0;
  ptr[0] = 0;
  for (int32_t qi = 0; qi < n && n_cov < n; ++qi) {
    const int32_t m = queue[static_cast<size_t>(qi)];
    if (covered[static_cast<size_t>(m)]) continue;
    const float* row_m = D + static_cast<int64_t>(m) * n;
    std::vector<int32_t> cand;
    for (int32_t e = 0; e < n; ++e)
      if (e != m && row_m[e] <= tau) cand.push_back(e);
    std::stable_sort(cand.begin(), cand.end(), [row_m](int32_t a, int32_t b) { return row_m[a] < row_m[b]; });
    std::vector<int32_t> mem{m};
    for (int32_t e : cand) {
      double total = 0.0;
      for (int32_t c : mem) total += static_cast<double>(D[static_cast<int64_t>(c) * n + e]);
      const double avg = total / static_cast<double>(mem.size());
      if (std::fabs(avg - tau_d) <= near_rtol * tau_d) ++near;
      if (avg <= tau_d) mem.push_back(e);
    }
    if (fill + static_cast<int64_t>(mem.size()) > members_cap) return ORACLE_BAD_ARG;
    for (int32_t e : mem) {
      members[fill++] = e;
      if (!covered[static_cast<size_t>(e)]) { covered[static_cast<size_t>(e)] = 1; ++n_cov; }
    }
    medoid[nc] = m;
    ptr[++nc] = static_cast<int32_t>(fill);
  }
  *n_clusters = nc;
  *n_near = near;
  return ORACLE_OK;
}

}  // extern "C"
