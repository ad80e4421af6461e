// Stage 4b: single-row attention (Eq. 1) over each head's selected tokens, as split-K flash decoding
// on the tensor cores.
//
// Roofline: every selected K/V page has to come out of HBM once; with one query row per head the
// arithmetic is ~1 flop per byte, so the kernel is bound by HBM bandwidth and everything below is
// about moving each byte once and spending as few issue slots on it as possible.
//
//  * Heads of a GQA group share a KV head and, in practice, about half of their pages.  A CTA
//    therefore serves one (request, KV head, split): it forms the union of its query heads'
//    selections from the per-head page bitmaps the selection kernel leaves behind, takes an equal
//    share of the union's pages (by rank, so the splits are balanced), loads every page of it once, and lets each head take part only in the pages it selected (the others are
//    masked to -inf for that head).  The g <= 8 heads are the M rows of the score MMA.
//  * Pages travel by TMA: cp.async.bulk.tensor tiles of 16 tokens x 64 coordinates with the 128-byte
//    swizzle, completion counted on an mbarrier.  Each warp owns a ring of kStages slots (16 tokens of
//    K and of V = 8 KiB per slot) and keeps it full, so kStages * 8 KiB per warp are always in flight.
//    Every mbarrier wait is bounded; on expiry the warp records SWARM_DEV_TIMEOUT and stops.
//  * Arithmetic: mma.sync m16n8k16 bf16 with fp32 accumulation.  S^T[head][token] = Q K^T takes K
//    tiles with ldmatrix; the probabilities go back in as the B operand of O^T[dim][head] = V^T P^T
//    (V^T through ldmatrix.trans), so all 16 M rows of that MMA carry useful coordinates.  P is fed as
//    a bf16 high part plus a bf16 low part (two MMAs), which keeps the result within fp32 rounding of
//    the exact sum.  About 110 warp instructions per 8 KiB, against ~500 per head on the fp32 pipes.
//  * Softmax state (m, l per head; 128 x 8 outputs) stays in registers; logits in the log2 domain.
//    Warps are merged through shared memory, page ranges (splits) through fp32 partials in global
//    memory: the CTA that arrives last at the group's ticket counter merges them, no second launch.
//
// The same kernel serves the contiguous gathered buffers (swarm_sparse_attn: one head per CTA, every
// page slot of the head) and the paged pool (swarm_step, swarm_sparse_attn_paged).
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>

#define SWARM_TRACE_FILE 2
#include "swarm_internal.cuh"
#include "attn_common.cuh"
#include "resolve_body.cuh"

namespace swarm {
namespace {
using namespace attn_detail;

constexpr int kListCap = 1024;                                     // pages per round = 32 bitmap words
constexpr int kScratchBytes = kListCap * 5;                        // the page list: ids (u32) and head masks (u8)
constexpr int kAttnSmemBytes = 1024 /*alignment slack*/ + kRingBytes + kScratchBytes;

// kFused != 0 (fused step only): CTA 0 of the grid does not attend; it runs cluster resolution (stage 3) beside
// the attention CTAs -- 1: plain, 2: with cache state.  As a kernel of its own on a second stream the serial
// pass stalled for about 2 us each time the attention kernel started or retired; as one more CTA of the same
// grid it does not, and the step needs neither the second stream nor its two events.
// kMode = kFused + 4 * kLines.  kLines (inside a step with a one-wave grid and few lists only): the page bitmaps
// arrive as self-validating words (StepTickets::selmap_ll); instances of their own, because the kernel sits at its
// register limit and the other instances must not pay for the polling code.
template <int S, bool kPaged, int kMode>
__global__ void __launch_bounds__(kAttnWarps * 32, 1)
attn_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV, Geometry geo,
            AttnArgs a, uint32_t* __restrict__ status, const __grid_constant__ ResolveArgs rs) {
  constexpr int kFused = kMode & 3;
  constexpr bool kLines = (kMode & 4) != 0;
  static_assert(kMode == 0 || kPaged, "cluster resolution and word-wise bitmaps ride with the paged kernel only");
  static_assert(resolve_detail::kThreads <= kAttnWarps * 32, "the resolution body runs in a CTA of this kernel");
  if (kFused != 0 && blockIdx.x == 0) {
    // (the body is written for kThreads threads; the CTA's other warps leave, and a CTA-wide barrier counts the
    // threads that have not left)
    if (threadIdx.x < resolve_detail::kThreads) resolve_detail::resolve_body<kFused == 2>(rs, 0, 1);
    return;
  }
  const int cta = (int)blockIdx.x - (kFused != 0 ? 1 : 0);
  constexpr int SB = S / kUnitTokens;                   // 16-token units per page
  // With 16-token pages read from the pool, the K rows and the V rows of a (page, KV head) are adjacent, and one
  // box of 32 rows brings both: two copies of 4 KiB per unit instead of four of 2 KiB (the copy engine's rate per
  // box, not the memory, bounds small boxes).  Slot layout then: [K | V] x coordinates 0-63, [K | V] x 64-127.
  constexpr bool kWide = kPaged && S == kUnitTokens;
  constexpr int kHalf = kWide ? 2 * kBoxBytes : kBoxBytes;   // bytes between the two coordinate halves
  constexpr int kVOff = kWide ? kBoxBytes : 2 * kBoxBytes;   // V tile relative to the K tile
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bars[kAttnWarps][kStages];
  __shared__ int s_wcnt[kAttnWarps];
  __shared__ unsigned s_epoch;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int quad = lane >> 2, tq = lane & 3;            // MMA fragment coordinates of this lane

  // ---- which (request, heads, page range) --------------------------------------------------------
  // The groups are cut into a.n_splits page ranges each, the last a.n_more of them into one more: the host picks
  // n_more so that the grid is a whole number of waves (the smaller CTAs come last).
  const int n_groups = kPaged ? geo.B * geo.Hkv * ((geo.g + 7) / 8) : geo.B * geo.Hq;
  const int slot_stride = a.n_splits + (a.n_more > 0 ? 1 : 0);
  const int base_ctas = (n_groups - a.n_more) * a.n_splits;
  int n_splits, split, grp;
  if (cta < base_ctas) {
    n_splits = a.n_splits;
    grp = cta / n_splits;
    split = cta - grp * n_splits;
  } else {
    n_splits = a.n_splits + 1;
    const int c = cta - base_ctas;
    grp = n_groups - a.n_more + c / n_splits;
    split = c % n_splits;
  }
  int b, kvh = 0, bh0, G;
  if (kPaged) {
    const int tiles = (geo.g + 7) / 8;
    const int tile = grp % tiles, bk = grp / tiles;
    b = bk / geo.Hkv;
    kvh = bk % geo.Hkv;
    bh0 = b * geo.Hq + kvh * geo.g + tile * 8;
    G = min(8, geo.g - tile * 8);
  } else {
    bh0 = grp;
    b = grp / geo.Hq;
    G = 1;
  }

  unsigned char* ring = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);   // TMA swizzle wants 1 KiB alignment
  uint32_t* list_page = reinterpret_cast<uint32_t*>(ring + kRingBytes);
  uint8_t* list_mask = reinterpret_cast<uint8_t*>(list_page + kListCap);

  if (lane == 0) {
#pragma unroll
    for (int sidx = 0; sidx < kStages; ++sidx) mbar_init(&bars[warp][sidx], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  SWARM_STAMP(status, 0);
  SWARM_KERNEL_BEGIN(status, 2);
  // Stand-alone, the next kernel in the stream may set itself up meanwhile.  Inside a step the attention
  // CTAs release their dependents by exiting: with this trigger the step was measured 1.5 us slower.
  const bool ticketed = kPaged && a.tk.sel_ready != nullptr;
  if (kFused == 0 && !ticketed) pdl_launch_dependents();
  // What the CTA needs besides the selection: the request's length and first pool page, and Q as the A operand of
  // S^T = Q K^T (row = head (quad), 8 k-steps of 16 coordinates).  Inside a step these are inputs of the whole
  // step, stable since its first kernel started, and are fetched while the CTA waits for the selection;
  // stand-alone they may come from the previous kernel and are fetched after it.
  uint32_t qa[8][2];
  int len = 0;
  long long pool_row0 = 0;
  auto load_inputs = [&]() {
    if (kPaged) {
      len = a.ctx_len[b];
      pool_row0 = a.page_base[b];
      asm volatile("prefetch.tensormap [%0];" ::"l"(&mapK) : "memory");
    }
    const bool row_ok = quad < G;
    const uint16_t* qrow = a.q + (long long)(bh0 + (row_ok ? quad : 0)) * kHeadDim;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa[ks][0] = row_ok ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + tq * 2) : 0u;
      qa[ks][1] = row_ok ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + tq * 2) : 0u;
    }
  };
  const bool lines = kLines;                            // the bitmaps arrive as self-validating words (then `ticketed` holds)
  if (ticketed) {
    load_inputs();
    // The selection kernel may still be running: wait for the heads of this CTA's KV head only.  The CTA then
    // counts itself as past its wait (no result comes back: an atomic with one held the CTA's next barrier).
    // With self-validating bitmaps there is no wait here: the threads look for their own words below, and what
    // the count says is that the CTA has read the step's epoch (which it is made to wait for).
    if (threadIdx.x == 0) {
      unsigned epoch = 0u;
      if (lines) {
        epoch = *reinterpret_cast<const volatile unsigned*>(a.tk.ctl + kCtlEpoch);
        s_epoch = epoch + 1u;
      } else if (!wait_at_least(a.tk.sel_ready + (long long)b * geo.Hkv + kvh, (unsigned)geo.g)) {
        atomicOr(status, SWARM_DEV_TIMEOUT);
      }
      red_relaxed_add(a.tk.ctl + kCtlAttnPast, 1u + zero_after(epoch));
    }
    __syncthreads();
  } else {
    pdl_wait();                                         // the selection comes from the previous kernel
    load_inputs();
  }
  SWARM_STAMP(status, 1);

  int P = 0, tail = S, total_tok = 0, n_items;          // items: pages of the union (paged) or page slots (gathered)
  int n_words = 0;

  // one bitmap word (32 pages) of every head of the group; the row pitch bounds the loads, so they do not
  // have to wait for the request's length
  const int pitch_words = a.selmap_pitch / 4;
  struct HeadWords { uint32_t v[8]; };
  auto load_raw = [&](int w) -> HeadWords {
    HeadWords hw;
    if (lines) {
      // {word, epoch} pairs written by selection CTAs that may still be running: all heads' pairs are asked for
      // together and asked for again until every one carries this step's flag (bounded)
      const unsigned flag = s_epoch;
      const uint2* base = a.tk.selmap_ll + (long long)bh0 * pitch_words + w;
      unsigned bad = 0u, polls = 0u;
      do {
        bad = 0u;
#pragma unroll
        for (int hh = 0; hh < 8; ++hh) {
          hw.v[hh] = 0u;
          if (hh < G && w < pitch_words) {
            const uint2 v = ll_word_load(base + (long long)hh * pitch_words);
            hw.v[hh] = v.x;
            bad |= v.y ^ flag;
          }
        }
      } while (bad != 0u && ++polls < kLlWaitLimit);
      if (bad != 0u) atomicOr(status, SWARM_DEV_TIMEOUT);
      return hw;
    }
#pragma unroll
    for (int hh = 0; hh < 8; ++hh) {
      hw.v[hh] = 0u;
      if (hh < G && w < pitch_words)
        hw.v[hh] = *reinterpret_cast<const uint32_t*>(a.selmap + (long long)(bh0 + hh) * a.selmap_pitch + (long long)w * 4);
    }
    return hw;
  };
  // their union, with the pages >= P cut off
  auto union_of = [&](int w, const HeadWords& hw) -> uint32_t {
    uint32_t uni = 0u;
#pragma unroll
    for (int hh = 0; hh < 8; ++hh) uni |= hw.v[hh];
    const int first = w * 32;
    if (first + 32 > P) uni &= first >= P ? 0u : (0xFFFFFFFFu >> (32 - (P - first)));
    return uni;
  };
  constexpr int kChunkWords = kAttnWarps * 32;          // bitmap words one pass of the CTA covers
  // (page, head mask) entries of the union pages in `bits` (word w, first rank `rank`) that rank in [lo, hi)
  auto emit_entries = [&](int w, const HeadWords& hw, uint32_t bits, int rank, int lo, int hi) {
    while (bits) {
      const int bit = __ffs(bits) - 1;
      bits &= bits - 1;
      if (rank >= lo && rank < hi) {
        uint32_t hm = 0u;
#pragma unroll
        for (int hh = 0; hh < 8; ++hh) hm |= ((hw.v[hh] >> bit) & 1u) << hh;
        list_page[rank - lo] = (uint32_t)(w * 32 + bit);
        list_mask[rank - lo] = (uint8_t)hm;
      }
      ++rank;
    }
  };
  bool first_list_built = false;                        // the first round's list is written already

  if (kPaged) {
    // number of pages in the union of the group's selections: the splits share them evenly by rank
    HeadWords hw = load_raw((int)threadIdx.x);
    P = pages_of(len, S);
    tail = len - S * (P - 1);
    n_words = min((P + 31) / 32, pitch_words);
    if (n_words <= kChunkWords) {
      // The whole bitmap is one word per thread: one CTA-wide scan gives the size of the union and every
      // thread's first rank, and the first round's list is written from the words already in registers.
      const uint32_t bits = union_of((int)threadIdx.x, hw);
      const int cnt = __popc(bits);
      int incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
      }
      if (lane == 31) s_wcnt[warp] = incl;
      __syncthreads();
      int rank = incl - cnt;
      n_items = 0;
#pragma unroll
      for (int w2 = 0; w2 < kAttnWarps; ++w2) {
        if (w2 < warp) rank += s_wcnt[w2];
        n_items += s_wcnt[w2];
      }
      const int lo = (int)((long long)n_items * split / n_splits);
      const int hi = min((int)((long long)n_items * (split + 1) / n_splits), lo + kListCap);
      if (rank + cnt > lo && rank < hi) emit_entries((int)threadIdx.x, hw, bits, rank, lo, hi);
      first_list_built = true;
    } else {
      int total = 0;
      for (int base = 0; base < n_words; base += kChunkWords) {
        const int w = base + (int)threadIdx.x;
        if (base > 0) hw = load_raw(w);
        total += __popc(union_of(w, hw));
      }
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) total += __shfl_xor_sync(0xFFFFFFFFu, total, o);
      if (lane == 0) s_wcnt[warp] = total;
      __syncthreads();
      n_items = 0;
#pragma unroll
      for (int w2 = 0; w2 < kAttnWarps; ++w2) n_items += s_wcnt[w2];
    }
  } else {
    total_tok = a.n_tok[bh0];
    if (total_tok < 0 || total_tok > geo.k * S) {          // more tokens than the head's buffer holds: attend what it holds
      if (threadIdx.x == 0 && split == 0) atomicOr(status, SWARM_DEV_BAD_LENGTH);
      total_tok = max(0, min(total_tok, geo.k * S));
    }
    n_items = (total_tok + S - 1) / S;
  }
  const int it_begin = (int)((long long)n_items * split / n_splits);
  const int it_end = (int)((long long)n_items * (split + 1) / n_splits);

  const float scale = kLog2e * rsqrtf((float)kHeadDim);

  float m_run = -INFINITY, l_run = 0.f;                 // of head `quad`, over this lane's token columns
  float acc[8][4];                                      // O^T: rows = coordinates 16*mt + quad (+8), cols = heads 2*tq (+1)
#pragma unroll
  for (int mt = 0; mt < 8; ++mt)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[mt][e] = 0.f;

  const uint64_t stream_policy = evict_first_policy();
  // token row of page (or page slot) p of this CTA's tensor: row_base + p * row_stride
  const int row_stride = kPaged ? geo.Hkv * 2 * S : S;
  const int row_base = kPaged ? (int)((pool_row0 * geo.Hkv + kvh) * 2 * S) : (int)((long long)bh0 * geo.k * S);
  unsigned char* my_ring = ring + (size_t)warp * kStages * kSlotBytes;
  unsigned fills = 0, drains = 0;                       // units issued / consumed so far (slot = count % kStages)
  bool timed_out = false;
  SWARM_STAMP(status, 2);

  // One round handles up to kListCap pages of this split's share of the union (paged), or all its page slots.
  for (int round0 = it_begin; round0 < it_end; round0 += kPaged ? kListCap : (it_end - it_begin)) {
    int n_list;
    if (kPaged) {
      // pages of the union with rank in [round0, round_end) -> (page, head mask) list, ascending; every
      // thread ranks the pages of its own word with a CTA-wide scan of the per-thread counts
      const int round_end = min(it_end, round0 + kListCap);
      int rank0 = 0;                                    // union pages before the current chunk of words
      const bool have_list = first_list_built && round0 == it_begin;
      for (int base = 0; !have_list && base < n_words && rank0 < round_end; base += kChunkWords) {
        const int w = base + (int)threadIdx.x;
        const HeadWords hw = load_raw(w);
        uint32_t bits = union_of(w, hw);
        const int cnt = __popc(bits);
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
          if (lane >= o) incl += t;
        }
        __syncthreads();                                // the counts of the previous pass, and the previous
        if (lane == 31) s_wcnt[warp] = incl;            // round's list, are no longer read
        __syncthreads();
        int rank = rank0 + incl - cnt;                  // rank of this thread's first union page
#pragma unroll
        for (int w2 = 0; w2 < kAttnWarps; ++w2) {
          if (w2 < warp) rank += s_wcnt[w2];
          rank0 += s_wcnt[w2];
        }
        if (rank + cnt > round0 && rank < round_end) emit_entries(w, hw, bits, rank, round0, round_end);
      }
      __syncthreads();
      n_list = round_end - round0;
    } else {
      n_list = it_end - it_begin;
    }
    SWARM_STAMP(status, 3);

    // this warp's entries: warp, warp + 4, ...; each is SB units of 16 tokens
    const int n_mine = (n_list - warp + kAttnWarps - 1) / kAttnWarps;
    const int units = (n_mine > 0 && !timed_out) ? n_mine * SB : 0;   // after a timeout only the barriers are kept

    auto entry_page = [&](int i) -> int {               // page id (paged) or page slot (gathered) of entry i
      return kPaged ? (int)list_page[warp + kAttnWarps * i] : round0 + warp + kAttnWarps * i;
    };
    auto issue = [&](int u) {
      if (lane == 0) {
        const int pg = entry_page(u / SB), sb = u % SB;
        // token row of the unit's K rows (the row count fits 31 bits: checked at launch)
        const int rowK = row_base + pg * row_stride + sb * kUnitTokens;
        const unsigned slot = fills % kStages;
        const uint32_t dst = smem_addr(my_ring + slot * kSlotBytes);
        uint64_t* bar = &bars[warp][slot];
        mbar_expect_tx(bar, kSlotBytes);
        if (kWide) {                                   // mapK's box is 32 rows here: K then V
          tma_load_rows(dst, &mapK, rowK, bar, stream_policy);
        } else {
          tma_load_rows(dst, &mapK, rowK, bar, stream_policy);
          tma_load_rows(dst + 2 * kBoxBytes, &mapV, kPaged ? rowK + S : rowK, bar, stream_policy);
        }
      }
      ++fills;
    };

    int issued = 0;
    for (; issued < min(units, kStages); ++issued) issue(issued);
    for (int u = 0; u < units; ++u) {
      const unsigned slot = drains % kStages, parity = (drains / kStages) & 1u;
      unsigned polls = 0;
      while (!mbar_try_wait(&bars[warp][slot], parity) && ++polls < kWaitLimit) {}
      if (__any_sync(0xFFFFFFFFu, polls >= kWaitLimit)) { timed_out = true; break; }
      ++drains;

      const int ei = u / SB, sb = u % SB;
      const int pg = entry_page(ei);
      const unsigned hm = kPaged ? list_mask[warp + kAttnWarps * ei] : 1u;
      int valid;
      if (kPaged) valid = (pg == P - 1) ? tail : S;
      else valid = min(S, total_tok - pg * S);
      const int v16 = min(kUnitTokens, valid - sb * kUnitTokens);
      if (v16 > 0)
        attend_unit<kHalf, kVOff>(my_ring + slot * kSlotBytes, v16, quad < G && ((hm >> quad) & 1u), lane, qa, scale, m_run,
                                  l_run, acc);
      __syncwarp();                                     // every lane is done reading the slot
      if (issued < units) { issue(issued); ++issued; }
    }
  }
  if (timed_out) {
    // give the copies still in flight a bounded chance to land before the shared memory is released
    for (; drains < fills; ++drains) {
      const unsigned slot = drains % kStages, parity = (drains / kStages) & 1u;
      unsigned polls = 0;
      while (!mbar_try_wait(&bars[warp][slot], parity) && ++polls < kWaitLimit) {}
    }
    if (lane == 0) atomicOr(status, SWARM_DEV_TIMEOUT);
  }
  SWARM_STAMP(status, 4);
  SWARM_STAMP_ANY_CTA(status, 7);
  // All pages read.  Inside a chain of steps the next kernel's CTAs may now take the SMs that CTAs of this kernel
  // leave: they wait for this kernel's completion before they touch anything that depends on it.
  if (kFused == 0 && ticketed && a.release_early) pdl_launch_dependents();

  // ---- merge the warps of the CTA ---------------------------------------------------------------------
  // Every warp posts its (max, sum) per head and its raw accumulators into its own ring (idle now: all its copies
  // have been consumed), so nobody waits for anybody before posting; after the one barrier warp h sums head h
  // over the warps on their common scale, four coordinates per lane, and is the one that publishes (or
  // finishes) that head.
  // rows of 128 + 4 floats: the four lanes of a quad store to heads 2*tq, whose rows then start 8 banks apart;
  // the row's spare floats hold the head's (max, sum)
  constexpr int kAccRow = kHeadDim + 4;
  constexpr int kPostStride = kStages * kSlotBytes / 4; // floats between two warps' posts
  static_assert(8 * kAccRow * 4 <= kStages * kSlotBytes, "a warp's post fits its ring");
  {
    float* mine = reinterpret_cast<float*>(my_ring);    // [head 8][kAccRow]
    l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 1);
    l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 2);
    if (tq == 0) {
      mine[quad * kAccRow + kHeadDim] = m_run;
      mine[quad * kAccRow + kHeadDim + 1] = l_run;
    }
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      float* base = mine + 2 * tq * kAccRow + 16 * mt + quad;
      base[0] = acc[mt][0];
      base[kAccRow] = acc[mt][1];
      base[8] = acc[mt][2];
      base[kAccRow + 8] = acc[mt][3];
    }
  }
  __syncthreads();
  SWARM_STAMP(status, 5);
  if (warp < G) {
    const int hh = warp;                                // this warp's head; lane: coordinates 4 * lane .. + 3
    const float* posts = reinterpret_cast<const float*>(ring) + hh * kAccRow;
    float mw[kAttnWarps];
    float M = -INFINITY, L = 0.f;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      mw[w] = posts[w * kPostStride + kHeadDim];
      M = fmaxf(M, mw[w]);
    }
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      const float sc = exp2_or_zero(mw[w], M);
      const float4 v = *reinterpret_cast<const float4*>(posts + w * kPostStride + 4 * lane);
      L = fmaf(posts[w * kPostStride + kHeadDim + 1], sc, L);
      o.x = fmaf(v.x, sc, o.x); o.y = fmaf(v.y, sc, o.y); o.z = fmaf(v.z, sc, o.z); o.w = fmaf(v.w, sc, o.w);
    }
    finish_head(a, bh0 + hh, split, n_splits, slot_stride, lane, M, L, o);
  }
  if (ticketed && threadIdx.x == 0 && blockIdx.x == gridDim.x - 1) {
    // The last CTA of the grid (its KV head is selected last, so it tends to finish last) tidies up: once every
    // CTA is past its wait nobody reads the selection's tickets any more, and they go back to zero for the next
    // step -- after the selection kernel has finished its own bookkeeping, so that the next step (which starts
    // after this kernel) finds all of it done.
    const unsigned n_ctas = gridDim.x - (kFused != 0 ? 1u : 0u);
    if (!wait_at_least(a.tk.ctl + kCtlAttnPast, n_ctas) || !wait_zero(a.tk.ctl + kCtlTopkDone)) atomicOr(status, SWARM_DEV_TIMEOUT);
    for (int i = 0; i < geo.B * geo.Hkv; ++i) a.tk.sel_ready[i] = 0u;
    if (lines) a.tk.ctl[kCtlEpoch] = s_epoch;            // one more step finished: its bitmap words no longer validate
    st_release(a.tk.ctl + kCtlAttnPast, 0u);
  }
  SWARM_STAMP_ANY_CTA(status, 6);
  SWARM_KERNEL_END(status, 2);
}

// Per-head page bitmap from an explicit selection list (for callers that bring their own `sel`).
__global__ void __launch_bounds__(256)
selmap_from_sel_kernel(Geometry geo, const int32_t* __restrict__ sel, const int32_t* __restrict__ n_sel,
                       uint8_t* __restrict__ selmap, int pitch) {
  const int bh = blockIdx.x;
  uint32_t* row = reinterpret_cast<uint32_t*>(selmap + (long long)bh * pitch);
  for (int i = threadIdx.x; i < pitch / 4; i += blockDim.x) row[i] = 0u;
  __syncthreads();
  const int n = min(n_sel[bh], geo.k);
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    const int p = sel[(long long)bh * geo.k + j];
    if (p >= 0 && p < geo.Pmax) atomicOr(&row[p >> 5], 1u << (p & 31));
  }
}

// ---- host side: tensor maps -----------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor of `rows` token rows x 128 coordinates at `base`, seen as (64 coordinates, row, half of the
// coordinates); boxes of 64 coordinates x `box_rows` rows x both halves, 128-byte swizzle (see tma_load_rows)
cudaError_t make_row_map(CUtensorMap* map, const void* base, long long rows, int box_rows = kUnitTokens) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return cudaErrorNotSupported;
  const cuuint64_t dims[3] = {64, (cuuint64_t)rows, 2};
  const cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, 128};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 2};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int S, bool kPaged>
cudaError_t launch_variant(const CUtensorMap& mk, const CUtensorMap& mv, const Geometry& geo, const AttnArgs& a,
                           uint32_t* status, unsigned grid, cudaStream_t st, bool overlap, const ResolveArgs* rs) {
  const dim3 block(kAttnWarps * 32);
  if constexpr (kPaged) {
    const bool lines = a.tk.sel_ready != nullptr && a.tk.selmap_ll != nullptr;
    if (rs != nullptr && rs->has_cache)
      return lines ? launch_pdl(attn_kernel<S, true, 6>, dim3(grid + 1), block, kAttnSmemBytes, st, overlap, mk, mv, geo, a, status, *rs)
                   : launch_pdl(attn_kernel<S, true, 2>, dim3(grid + 1), block, kAttnSmemBytes, st, overlap, mk, mv, geo, a, status, *rs);
    if (rs != nullptr)
      return lines ? launch_pdl(attn_kernel<S, true, 5>, dim3(grid + 1), block, kAttnSmemBytes, st, overlap, mk, mv, geo, a, status, *rs)
                   : launch_pdl(attn_kernel<S, true, 1>, dim3(grid + 1), block, kAttnSmemBytes, st, overlap, mk, mv, geo, a, status, *rs);
    if (lines)
      return launch_pdl(attn_kernel<S, true, 4>, dim3(grid), block, kAttnSmemBytes, st, overlap, mk, mv, geo, a, status, ResolveArgs{});
  }
  return launch_pdl(attn_kernel<S, kPaged, 0>, dim3(grid), block, kAttnSmemBytes, st, overlap, mk, mv, geo, a, status,
                    ResolveArgs{});
}

template <class K>
cudaError_t allow_smem(K kernel) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemBytes);
}

}  // namespace

cudaError_t configure_attention() {
  if (encode_tiled_fn() == nullptr) return cudaErrorNotSupported;   // resolved here, not inside a stream capture
  static_assert(kAttnSmemBytes >= (int)resolve_detail::kResolveSmemBytes, "the resolution CTA stages its items here");
  cudaError_t e = allow_smem(attn_kernel<16, true, 0>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<16, true, 1>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<16, true, 2>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<16, true, 4>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<16, true, 5>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<16, true, 6>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<32, true, 4>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<32, true, 5>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<32, true, 6>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<16, false, 0>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<32, true, 0>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<32, true, 1>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<32, true, 2>);
  if (e == cudaSuccess) e = allow_smem(attn_kernel<32, false, 0>);
  return e;
}

int attention_groups(const Geometry& geo, bool paged) {
  return paged ? geo.B * geo.Hkv * ((geo.g + 7) / 8) : geo.B * geo.Hq;
}

cudaError_t launch_selmap_from_sel(const Geometry& geo, const int32_t* sel, const int32_t* n_sel, uint8_t* selmap,
                                   cudaStream_t st) {
  selmap_from_sel_kernel<<<geo.B * geo.Hq, 256, 0, st>>>(geo, sel, n_sel, selmap, selmap_pitch_bytes(geo.Pmax));
  return cudaGetLastError();
}

cudaError_t launch_attention(const Geometry& geo, const AttnArgs& a, uint32_t* status, cudaStream_t st,
                             bool overlap, const ResolveArgs* fused_resolve) {
  const bool paged = a.kv_pool != nullptr;
  CUtensorMap mk, mv;
  cudaError_t e;
  if (paged) {
    const long long rows = geo.n_pool_pages * geo.Hkv * 2 * geo.S;
    if (rows >= (1LL << 31)) return cudaErrorInvalidValue;
    e = make_row_map(&mk, a.kv_pool, rows, geo.S == kUnitTokens ? 2 * kUnitTokens : kUnitTokens);   // 16-token pages: K and V in one box
    mv = mk;
  } else {
    const long long rows = (long long)geo.B * geo.Hq * geo.k * geo.S;
    if (rows >= (1LL << 31)) return cudaErrorInvalidValue;
    e = make_row_map(&mk, a.k_g, rows);
    if (e == cudaSuccess) e = make_row_map(&mv, a.v_g, rows);
  }
  if (e != cudaSuccess) return e;
  const unsigned grid = (unsigned)attention_groups(geo, paged) * a.n_splits + (unsigned)a.n_more;
  if (geo.S == 16)
    return paged ? launch_variant<16, true>(mk, mv, geo, a, status, grid, st, overlap, fused_resolve)
                 : launch_variant<16, false>(mk, mv, geo, a, status, grid, st, overlap, nullptr);
  return paged ? launch_variant<32, true>(mk, mv, geo, a, status, grid, st, overlap, fused_resolve)
               : launch_variant<32, false>(mk, mv, geo, a, status, grid, st, overlap, nullptr);
}

}  // namespace swarm

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of swarm_sparse_attn (see swarm.h).  The split-K partials live in a
// file-scope device array instead of a caller-provided workspace.  Layout of the array:
//   [0, 256)                       device status word (bits SWARM_DEV_*; read and cleared by
//                                  swarm_sparse_attn_static_status) + padding
//   [256, 256 + kSlots*128*4)      partial accumulators, one 128-float row per (head, split) slot
//   [.., .. + kSlots*2*4)          partial (max, sum) pairs
//   [.., .. + kMaxHeads*4)         per-head arrival counters; zero at load (static storage) and set
//                                  back to zero by the CTA that merges a head, so zero between calls
// Host code must not pass `g_static_scratch` itself to a kernel: on the host that name is only a
// handle.  Its device address is fetched once per device with cudaGetSymbolAddress.
namespace {
constexpr int kStaticSlots = 4096;
static_assert(SWARM_STATIC_SCRATCH_BYTES == 256 + kStaticSlots * (swarm::kHeadDim + 2) * 4 + SWARM_STATIC_MAX_HEADS * 4,
              "header and array size differ");
static __device__ __align__(256) unsigned char g_static_scratch[SWARM_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
struct StaticDevice {
  unsigned char* scratch;   // device address of the array on this device; null until the set-up has run
  int sms;
};
StaticDevice g_static_dev[kMaxDevices] = {};

// Set-up for the current device, on the first call there (idempotent if two threads race): the array's
// address, the SM count, the kernels' shared-memory attribute.  Allocates nothing.
cudaError_t static_device(const StaticDevice** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (g_static_dev[dev].scratch == nullptr) {
    void* p = nullptr;
    int sms = 0;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = swarm::configure_attention();
    if (e != cudaSuccess) return e;
    g_static_dev[dev].sms = sms > 0 ? sms : 1;
    g_static_dev[dev].scratch = static_cast<unsigned char*>(p);
  }
  *out = &g_static_dev[dev];
  return cudaSuccess;
}
}  // namespace

extern "C" int32_t swarm_sparse_attn_static(const void* q, const void* k_g, const void* v_g, const int32_t* n_tok,
                                            int32_t batch, int32_t n_q_heads, int32_t top_k, int32_t page_size,
                                            float* out, float* lse, void* stream) {
  using namespace swarm;
  auto bad = [](const void* p) { return p == nullptr || (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  if (bad(q) || bad(k_g) || bad(v_g) || bad(n_tok) || bad(out) || bad(lse) || batch < 1 || n_q_heads < 1 || top_k < 1)
    return SWARM_ERR_INVALID_ARG;
  if (page_size != 16 && page_size != 32) return SWARM_ERR_UNSUPPORTED;
  const long long bh = (long long)batch * n_q_heads;
  if (bh > SWARM_STATIC_MAX_HEADS) return SWARM_ERR_STATIC_SCRATCH_TOO_SMALL;
  if (bh * top_k >= (1LL << 31)) return SWARM_ERR_UNSUPPORTED;
  const StaticDevice* dev = nullptr;
  if (static_device(&dev) != cudaSuccess) return SWARM_ERR_CUDA;
  // same split heuristic as the ctx path (one wave of CTAs, at least 4 pages per split); the array holds
  // kStaticSlots >= 2 * SWARM_STATIC_MAX_HEADS (head, split) slots, and the last bound keeps any SM count inside it
  long long n = std::max<long long>(1, dev->sms / bh);
  n = std::min<long long>(n, std::max(1, top_k / 4));
  n = std::min<long long>(n, kMaxSplits);
  n = std::min<long long>(n, kStaticSlots / bh);

  unsigned char* base = dev->scratch;
  Geometry geo{};
  geo.B = batch; geo.Hq = n_q_heads; geo.Hkv = n_q_heads; geo.g = 1; geo.S = page_size; geo.k = top_k; geo.D = 1;
  geo.Pmax = top_k; geo.Cmax = 1; geo.flags = 0; geo.n_pool_pages = 0; geo.W = 0;
  AttnArgs a{};
  a.q = static_cast<const uint16_t*>(q);
  a.k_g = static_cast<const uint16_t*>(k_g);
  a.v_g = static_cast<const uint16_t*>(v_g);
  a.n_tok = n_tok;
  a.part_acc = reinterpret_cast<float*>(base + 256);
  a.part_ml = reinterpret_cast<float*>(base + 256 + (size_t)kStaticSlots * kHeadDim * 4);
  a.tickets = reinterpret_cast<unsigned*>(base + 256 + (size_t)kStaticSlots * (kHeadDim + 2) * 4);
  a.out = out;
  a.lse = lse;
  a.n_splits = (int)n;
  return launch_attention(geo, a, reinterpret_cast<uint32_t*>(base), static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? SWARM_OK : SWARM_ERR_CUDA;
}

extern "C" int32_t swarm_sparse_attn_static_status(void* stream, uint32_t* bits) {
  if (bits == nullptr) return SWARM_ERR_INVALID_ARG;
  const StaticDevice* dev = nullptr;
  if (static_device(&dev) != cudaSuccess) return SWARM_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(bits, dev->scratch, sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemsetAsync(dev->scratch, 0, sizeof(uint32_t), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
    return SWARM_ERR_CUDA;
  return SWARM_OK;
}
