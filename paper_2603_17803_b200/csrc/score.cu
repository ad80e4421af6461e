// Stage 1: activation scoring (Sec. 2.3: relevance score of every cached entry against the query).
//
//   score[b][h][p] = sum_i max(q[i]*kmin[p][i], q[i]*kmax[p][i])
//                  = sum_i max(q[i],0)*kmax[p][i] + min(q[i],0)*kmin[p][i]        (kmin <= kmax)
//
// One summary row (page, kv head) is 512 contiguous bytes: 128 bf16 minima then 128 bf16 maxima.
// A warp reads a row with one 16-byte load per lane (lanes 0-15 hold minima, 16-31 maxima), so the
// sign-split form needs one multiply-add per element and query head, with the weights (min(q,0) on
// the low lanes, max(q,0) on the high lanes) held in registers for all G heads of the KV group.
// (Packed fma.rn.f32x2 was measured slower than scalar FMAs on sm_100 for the same work and is not used.)
//
// R rows are handled together; their R*G partial sums are summed across the 32 lanes with a
// transposing butterfly: at each level a lane keeps half of its sums and hands the other half to
// its partner, so 32 sums cost 31 shuffles and sum v ends in lane v (coalesced stores).  Which row
// and which head a lane computes into register slot j is permuted by the lane id (slot j holds sum
// j XOR lane): then every lane keeps the low slots and sends the high slots at every level and the
// butterfly needs no selects.  The permutation is free: it only changes load addresses.
//
// Every warp requests all of its NB*R rows (8 KiB) before it starts the arithmetic, and 12 warps fit
// on an SM, so about 96 KiB per SM are in flight.  HBM-bound: 512 B per row against about 40 warp
// instructions.
#include <cuda.h>

#include <algorithm>

#define SWARM_TRACE_FILE 0
#include "swarm_internal.cuh"

namespace swarm {
namespace {

constexpr int kScoreWarps = 4;
int g_sm_count = 148;                                      // set by configure_score()
}  // namespace
int sm_count() { return g_sm_count; }
namespace {

__host__ __device__ constexpr int ilog2(int x) { return x <= 1 ? 0 : 1 + ilog2(x / 2); }

// Slot j of lane L holds the partial of sum (j XOR (L >> (5 - log2 NV))).  Returns, in every lane, the
// total of sum (L >> (5 - log2 NV)).
template <int NV>
__device__ __forceinline__ float butterfly(float (&v)[NV]) {
  int offset = 16;
#pragma unroll
  for (int n = NV; n > 1; n >>= 1) {
#pragma unroll
    for (int j = 0; j < n / 2; ++j) v[j] += __shfl_xor_sync(0xFFFFFFFFu, v[j + n / 2], offset);
    offset >>= 1;
  }
  float r = v[0];
#pragma unroll
  for (int o = 16 >> ilog2(NV); o >= 1; o >>= 1) r += __shfl_xor_sync(0xFFFFFFFFu, r, o);
  return r;
}

// Weights of this lane's 8 coordinates for the G heads starting at bh0 (= request * Hq + head): min(q,0) on
// the lanes that hold minima, max(q,0) on the lanes that hold maxima; w[c] belongs to head (c XOR head_sel).
template <int G>
__device__ __forceinline__ void load_weights(float (&w)[G][8], const uint16_t* __restrict__ q, long long bh0,
                                             int head_sel, int lane) {
#pragma unroll
  for (int cc = 0; cc < G; ++cc) {
    const uint4 qq = *reinterpret_cast<const uint4*>(q + (bh0 + (cc ^ head_sel)) * kHeadDim + (lane & 15) * 8);
    const uint32_t words[4] = {qq.x, qq.y, qq.z, qq.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float lo = bf16_lo(words[e]), hi = bf16_hi(words[e]);
      w[cc][2 * e] = lane < 16 ? fminf(lo, 0.f) : fmaxf(lo, 0.f);
      w[cc][2 * e + 1] = lane < 16 ? fminf(hi, 0.f) : fmaxf(hi, 0.f);
    }
  }
}

template <int G, int R, int NB>
__global__ void __launch_bounds__(kScoreWarps * 32, 3)
page_score_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ ksum,
                  const int64_t* __restrict__ page_base, const int32_t* __restrict__ ctx_len,
                  float* __restrict__ scores, uint32_t* __restrict__ status) {
  constexpr int NV = G * R;
  constexpr int LOG_NV = ilog2(NV), LOG_G = ilog2(G);
  static_assert(NV <= 32 && (1 << LOG_NV) == NV && (1 << LOG_G) == G, "R and G must be powers of two, R*G <= 32");
  pdl_launch_dependents();   // the next kernel may be scheduled as soon as every CTA of this one runs
  pdl_wait();                // launched behind whatever precedes it in the stream (see launch_mma)
  SWARM_STAMP(status, 0);
  SWARM_KERNEL_BEGIN(status, 0);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tiles = geo.g / G;
  const int kvh = blockIdx.y / tiles, tile = blockIdx.y % tiles;
  const int b = blockIdx.z;
  const int len = ctx_len[b];
  const long long base = page_base[b];
  const int P = pages_of(len, geo.S);
  if (len < 1 || P > page_base[b + 1] - base || P > geo.Pmax) {
    if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0) atomicOr(status, SWARM_DEV_BAD_LENGTH);
    return;
  }
  // a warp owns NB*R consecutive pages; all their rows are requested before any arithmetic
  const int p_warp = (blockIdx.x * kScoreWarps + warp) * (R * NB);
  if (p_warp >= P) return;

  // Sum index = row * G + head.  The row bits are the high bits of the lane id, so the lanes that read
  // the same row in one load instruction are neighbours and every 32-byte sector is used whole.
  const int pi = lane >> (5 - LOG_NV);                      // this lane's slot permutation
  const int row_sel = pi >> LOG_G, head_sel = pi & (G - 1);

  const long long row_stride = (long long)geo.Hkv * 2 * kHeadDim;   // elements between consecutive pages
  const uint16_t* rows = ksum + ((base * geo.Hkv + kvh) * 2) * (long long)kHeadDim + lane * 8;
  uint4 data[NB][R];                                        // data[nb][a] = row (a XOR row_sel) of batch nb
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int a = 0; a < R; ++a) {
      const int p = p_warp + nb * R + (a ^ row_sel);
      data[nb][a] = p < P ? ldg_nc_v4(rows + p * row_stride) : make_uint4(0, 0, 0, 0);
    }

  SWARM_STAMP(status, 1);
  // Weights of this lane's 8 coordinates; w[c] belongs to head (c XOR head_sel).
  const int h0 = kvh * geo.g + tile * G;
  float w[G][8];
  load_weights<G>(w, q, (long long)b * geo.Hq + h0, head_sel, lane);

  SWARM_STAMP(status, 2);
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    const int p0 = p_warp + nb * R;
    if (p0 >= P) break;
    float v[NV];
#pragma unroll
    for (int a = 0; a < R; ++a) {
      const uint32_t words[4] = {data[nb][a].x, data[nb][a].y, data[nb][a].z, data[nb][a].w};
      float x[8];
#pragma unroll
      for (int e = 0; e < 4; ++e) { x[2 * e] = bf16_lo(words[e]); x[2 * e + 1] = bf16_hi(words[e]); }
#pragma unroll
      for (int c = 0; c < G; ++c) {
        float acc = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc = fmaf(w[c][e], x[e], acc);
        v[a * G + c] = acc;
      }
    }
    const float total = butterfly<NV>(v);
    const int r = pi >> LOG_G, hh = pi & (G - 1);
    if ((lane & ((1 << (5 - LOG_NV)) - 1)) == 0 && p0 + r < P)
      scores[((long long)(b * geo.Hq + h0 + hh)) * geo.Pmax + p0 + r] = total;
    SWARM_STAMP(status, 3 + nb);
  }
  SWARM_KERNEL_END(status, 0);
}

// ---- streaming tensor-core variant ---------------------------------------------------------------------
// score[page][head] is a dense contraction: [pages x 256] (minima | maxima) times [256 x heads]
// (min(q,0) | max(q,0)), all operands exactly representable in bf16.  On the fp32 pipes it costs ~100 warp
// instructions per 512-byte row, which was measured to hold a 148-SM streaming kernel at about half of
// the memory bandwidth; as m16n8k16 MMAs (16 pages x up to 8 heads per tile, fp32 accumulation) it costs
// ~3, and the kernel runs at the speed of the bulk copies.
//
// Persistent CTAs, one per SM, on all SMs but the ones left to the selection kernel (see launch_mma).  A block
// is 64 consecutive pages of one request for one PAIR of KV heads: 16 TMA boxes of 16 pages x 2 heads x 64
// coordinates (128-byte swizzle) = 64 KiB.  Blocks are numbered request by request, inside a request pair by
// pair, and dealt to the CTAs round-robin, so that at any moment all CTAs work on the same (request, pair) and
// the pairs of a request are finished one after the other: the selection of a pair's heads starts while the
// later pairs are still being scored (StepTickets::ready).  Reading one pair at a time touches 1 KiB of every
// 4 KiB summary row; measured, that streams at the same rate as whole rows.  A producer warp keeps a 3-slot
// ring full; consumer warp w scores (tile w / 2, head w % 2) of the block that has landed with ldmatrix + mma,
// stores the tile of scores and counts it on the pair's ticket.  Waits are bounded.
constexpr int kMmaConsumers = 8;
constexpr int kMmaThreads = (kMmaConsumers + 3) * 32;      // consumers, the producer warp, the ticket warp, the weight warp
constexpr int kMmaStages = 3;
constexpr int kMmaPages = 16;                              // pages per tile = M of the MMA tile
constexpr int kMmaHeadBytes = 4 * kMmaPages * 128;         // one KV head of one tile: 4 boxes' share, 8 KiB
constexpr int kBoxHeads = 2;                               // KV heads per TMA box (rows of a box: page-major, head-minor)
constexpr int kBlkTiles = kMmaConsumers / kBoxHeads;       // 16-page tiles per block
constexpr int kBlkPages = kBlkTiles * kMmaPages;           // 64
constexpr int kTileBytes = kBoxHeads * kMmaHeadBytes;      // one tile of a pair: 4 boxes of 4 KiB
constexpr int kMmaStageBytes = kBlkTiles * kTileBytes;
// Sign-split weights (min(q,0) | max(q,0), bf16) of the query heads of a block's KV pair travel with the block:
// the producer warp writes them into the ring slot's own weight rows after it has issued the slot's copies, and
// the slot's `full` barrier counts them as a second arrival.  In pair-by-pair order nearly every block of a CTA
// belongs to another pair (and, with several requests, to another request); fetching the weights from global
// memory inside the consumers' loop cost more than the block's arithmetic.  Rows are padded by 16 bytes so that
// the 8 heads a warp reads side by side fall into different banks.  Pairs with more query heads than fit
// (groups of more than 8 heads) are fetched by the consumers from global memory.
constexpr int kWeightRowBytes = 512 + 16;
constexpr int kWeightRowsMax = 16;                         // 2 KV heads x up to 8 query heads
__host__ __device__ constexpr int weight_rows(int g) { return 2 * g <= kWeightRowsMax ? 2 * g : 0; }
__host__ __device__ constexpr int mma_smem_bytes(int g) {
  return 1024 + kMmaStages * (kMmaStageBytes + weight_rows(g) * kWeightRowBytes);
}
constexpr int kStreamMaxBatch = 512;                       // requests whose block counts fit the shared prefix table (2 KiB:
                                                           // the kernel's shared memory leaves room for a selection CTA beside it)
constexpr unsigned kStreamWaitLimit = 1u << 22;

__device__ __forceinline__ uint32_t sm_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool sm_try_wait(uint64_t* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(sm_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// What block `blk` of the launch covers; s_cum[b] = blocks before request b.
struct ScoreBlock {
  int b, hp, page0, n_tiles, P;   // request, KV-head pair, first page (request-local), tiles that exist, pages of the request
};
__device__ __forceinline__ ScoreBlock locate_block(int blk, int& cur_b, const int* s_cum, const int32_t* __restrict__ ctx_len, int S,
                                                   int hpairs) {
  while (s_cum[cur_b + 1] <= blk) ++cur_b;
  ScoreBlock k;
  k.b = cur_b;
  // blocks per pair from the table; the request's length is fetched only for the last block of a pair (the only
  // one that can be partial): a fetch per block sat at the top of every warp's loop
  const int per_pair = (s_cum[cur_b + 1] - s_cum[cur_b]) / hpairs;
  const int c = blk - s_cum[cur_b];
  k.hp = c / per_pair;
  const int j = c - k.hp * per_pair;
  k.page0 = j * kBlkPages;
  if (j + 1 < per_pair) {
    k.P = per_pair * kBlkPages;                              // (an upper bound does: every page of this block exists)
    k.n_tiles = kBlkTiles;
  } else {
    k.P = pages_of(ctx_len[cur_b], S);
    k.n_tiles = min(kBlkTiles, (k.P - k.page0 + kMmaPages - 1) / kMmaPages);
  }
  return k;
}

// 128 registers: with 11 warps that leaves room on the SM for a 256-thread selection CTA beside this one.
// kPairs: every score is also stored as a self-validating {score, epoch + 1} pair (few lists in a one-wave step:
// the selection then reads those, waiting for no ticket); an instance of its own, so that the other one keeps the
// register count that lets a selection CTA sit beside it.
template <bool kPairs, bool kEarly>
__global__ void __maxnreg__(128)
page_score_mma_kernel(const __grid_constant__ CUtensorMap map, Geometry geo, const uint16_t* __restrict__ q,
                      const int64_t* __restrict__ page_base, const int32_t* __restrict__ ctx_len,
                      float* __restrict__ scores, uint32_t* __restrict__ status, unsigned* __restrict__ ready,
                      uint2* __restrict__ scores_ll, const unsigned* __restrict__ ctl) {
  extern __shared__ unsigned char mma_smem_raw[];
  __shared__ __align__(8) uint64_t full[kMmaStages], empty[kMmaStages];
  __shared__ int s_cum[kStreamMaxBatch + 1];               // blocks before request b
  __shared__ int s_abort;
  __shared__ unsigned s_scored[kMmaStages];                // consumer warps done with the blocks of a ring slot, ever growing
  SWARM_KERNEL_BEGIN(status, 0);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned char* ring = mma_smem_raw + ((1024u - (sm_addr(mma_smem_raw) & 1023u)) & 1023u);

  const int hpairs = head_pairs(geo.Hkv);
  if (tid == 0) {
    for (int sidx = 0; sidx < kMmaStages; ++sidx) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(sm_addr(&full[sidx])), "r"(2));   // the copies, the weights
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(sm_addr(&empty[sidx])), "r"(kMmaConsumers));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_abort = 0;
    s_cum[0] = 0;
    for (int sidx = 0; sidx < kMmaStages; ++sidx) s_scored[sidx] = 0u;
  }
  // Launched with programmatic serialization behind whatever precedes it in the stream -- inside a chain of
  // steps the previous step's attention kernel -- so that this kernel's launch and set-up overlap that kernel's
  // tail.  Nothing a predecessor may have written is read before the wait.  In the kEarly instances the caller vouches
  // that the predecessor writes neither the lengths, nor the page bases, nor the summaries: the CTA then lays out
  // its blocks and its producer asks for the first ones before the wait -- they do not depend on the queries --
  // and everything that touches q, the scores or the tickets still comes after it.
  SWARM_STAMP(status, 0);
  if (!kEarly) {
    pdl_wait();
    SWARM_STAMP(status, 1);
    // Only now may the selection kernel be scheduled: its CTAs poll the tickets this kernel raises, and tickets
    // of the previous step are guaranteed to be cleared only once everything before this kernel has finished.
    pdl_launch_dependents();
  }
  if (warp == 1) {                                         // blocks per request, prefix by one warp
    int running = 0;
    for (int b0 = 0; b0 < geo.B; b0 += 32) {
      const int b = b0 + lane;
      int nb = 0;
      if (b < geo.B) {
        const int len = ctx_len[b];
        const int P = pages_of(len, geo.S);
        if (len < 1 || P > page_base[b + 1] - page_base[b] || P > geo.Pmax) atomicOr(status, SWARM_DEV_BAD_LENGTH);
        else nb = ((P + kBlkPages - 1) / kBlkPages) * hpairs;
      }
      int incl = nb;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
      }
      if (b < geo.B) s_cum[b + 1] = running + incl;
      running += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
  }
  __syncthreads();
  SWARM_STAMP(status, 2);
  const int total = s_cum[geo.B];
  const int blk_first = (int)blockIdx.x, blk_step = (int)gridDim.x;
  const int n_blk = blk_first < total ? (total - blk_first + blk_step - 1) / blk_step : 0;

  const int w_rows = weight_rows(geo.g);                  // weight rows per ring slot (0: consumers fetch their own)
  unsigned char* wring = ring + kMmaStages * kMmaStageBytes;
  if (warp == kMmaConsumers) {
    // ---- producer ----
    if (lane == 0) {
      // the summaries are read once per step: evict-first keeps them from displacing the small tables, the
      // workspace and the kernels' own instructions in L2
      uint64_t stream_policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(stream_policy));
      int fb = 0;
      for (int k = 0; k < n_blk; ++k) {
        const int stage = k % kMmaStages;
        if (k >= kMmaStages) {
          const unsigned parity = ((k / kMmaStages) - 1) & 1u;
          unsigned polls = 0;
          while (!sm_try_wait(&empty[stage], parity) && ++polls < kStreamWaitLimit && !s_abort) {}
          if (polls >= kStreamWaitLimit || s_abort) { atomicOr(status, SWARM_DEV_TIMEOUT); s_abort = 1; break; }
        }
        const ScoreBlock blk = locate_block(blk_first + k * blk_step, fb, s_cum, ctx_len, geo.S, hpairs);
        const int page0 = (int)(page_base[blk.b] + blk.page0);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(sm_addr(&full[stage])),
                     "r"((unsigned)(blk.n_tiles * kTileBytes))
                     : "memory");
        // a box carries both heads of the pair (the copy engine's rate per box, not the memory, bounds smaller
        // boxes); the second head of an odd last pair lies outside the tensor and arrives as zeros
        for (int pt = 0; pt < blk.n_tiles; ++pt) {
#pragma unroll
          for (int bx = 0; bx < 4; ++bx) {
            const uint32_t dst = sm_addr(ring + (size_t)stage * kMmaStageBytes + pt * kTileBytes + bx * (kTileBytes / 4));
            asm volatile(
                "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(dst),
                "l"(&map), "r"(bx * 64), "r"(blk.hp * kBoxHeads), "r"(page0 + pt * kMmaPages), "r"(sm_addr(&full[stage])), "l"(stream_policy)
                : "memory");
          }
        }
      }
    }
    return;
  }
  if (kEarly) {                                            // (the producer above reads nothing that depends on a predecessor)
    pdl_wait();
    SWARM_STAMP(status, 1);
    pdl_launch_dependents();
  }
  if (warp == kMmaConsumers + 2) {
    // ---- weight warp: the second arrival on every slot's `full` barrier ----
    // weights of the pair's query heads: row r <-> head (first head of the pair) + r; 16 chunks of 8 coordinates.
    // The rows are fetched into registers before the warp waits for the slot, so the fetch of one block runs
    // beside the consumers' work on the earlier ones.
    int fb = 0;
    for (int k = 0; k < n_blk; ++k) {
      const int stage = k % kMmaStages;
      const ScoreBlock blk = locate_block(blk_first + k * blk_step, fb, s_cum, ctx_len, geo.S, hpairs);
      const int n_chunks = w_rows > 0 ? min(kBoxHeads, geo.Hkv - blk.hp * kBoxHeads) * geo.g * 16 : 0;
      const uint16_t* qpair = q + ((long long)blk.b * geo.Hq + (long long)blk.hp * kBoxHeads * geo.g) * kHeadDim;
      uint4 v[kWeightRowsMax * 16 / 32];
#pragma unroll
      for (int j = 0; j < kWeightRowsMax * 16 / 32; ++j) {
        const int i = lane + 32 * j;
        v[j] = i < n_chunks ? *reinterpret_cast<const uint4*>(qpair + (long long)(i >> 4) * kHeadDim + (i & 15) * 8)
                            : make_uint4(0u, 0u, 0u, 0u);
      }
      int go = 1;
      if (lane == 0 && k >= kMmaStages) {
        const unsigned parity = ((k / kMmaStages) - 1) & 1u;
        unsigned polls = 0;
        while (!sm_try_wait(&empty[stage], parity) && ++polls < kStreamWaitLimit && !s_abort) {}
        if (polls >= kStreamWaitLimit || s_abort) go = 0;   // (the producer reports it)
      }
      if (!__shfl_sync(0xFFFFFFFFu, go, 0)) break;
      unsigned char* wst = wring + (size_t)stage * w_rows * kWeightRowBytes;
#pragma unroll
      for (int j = 0; j < kWeightRowsMax * 16 / 32; ++j) {
        const int i = lane + 32 * j;
        if (i < n_chunks) {
          const uint32_t in[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
          uint32_t neg[4], pos[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {                     // clamp each bf16 by its sign bit
            const uint32_t lo = in[e] & 0xFFFFu, hi = in[e] >> 16;
            neg[e] = ((lo >> 15) ? lo : 0u) | (((hi >> 15) ? hi : 0u) << 16);
            pos[e] = ((lo >> 15) ? 0u : lo) | (((hi >> 15) ? 0u : hi) << 16);
          }
          unsigned char* row = wst + (size_t)(i >> 4) * kWeightRowBytes + (i & 15) * 16;
          *reinterpret_cast<uint4*>(row) = make_uint4(neg[0], neg[1], neg[2], neg[3]);
          *reinterpret_cast<uint4*>(row + 256) = make_uint4(pos[0], pos[1], pos[2], pos[3]);
        }
      }
      __syncwarp();                                         // the lanes' rows are ordered before lane 0's arrival
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(sm_addr(&full[stage])) : "memory");
    }
    return;
  }

  if (warp == kMmaConsumers + 1) {
    // ---- ticket warp ----
    // Raising a ticket needs a GPU-wide release behind the consumers' score stores, which waits for those stores
    // to be acknowledged: about a microsecond per block.  In the consumers' loop that wait held back the ring
    // (measured: +4 us per launch); here one otherwise idle thread pays it.  The consumers count themselves on
    // a per-slot counter in shared memory (release at CTA scope); a slot is refilled only after all of them
    // have arrived on its `empty` barrier, so block k is complete exactly when its slot's counter has reached
    // 8 * (k / slots + 1).
    if (lane == 0 && ready != nullptr) {
      int fb = 0;
      for (int k = 0; k < n_blk; ++k) {
        const int stage = k % kMmaStages;
        const unsigned want = (unsigned)kMmaConsumers * (unsigned)(k / kMmaStages + 1);
        unsigned polls = 0, seen = 0;
        do {
          asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(seen) : "r"(sm_addr(&s_scored[stage])) : "memory");
          if (seen >= want) break;
          __nanosleep(64);
        } while (++polls < kStreamWaitLimit && !s_abort);
        if (seen < want) break;                             // the consumers gave up (they have set the status bit)
        const ScoreBlock blk = locate_block(blk_first + k * blk_step, fb, s_cum, ctx_len, geo.S, hpairs);
        const unsigned units = (unsigned)blk.n_tiles * (unsigned)min(kBoxHeads, geo.Hkv - blk.hp * kBoxHeads);
        red_release_add(ready + (long long)blk.b * hpairs + blk.hp, units);
      }
    }
    return;
  }

  // ---- consumers: warp w <-> (tile w / 2, head w % 2) of the block ----
  // the flag of this step's self-validating scores (the epoch is stable: the previous step has finished)
  const unsigned ll_flag = kPairs ? *reinterpret_cast<const volatile unsigned*>(ctl + kCtlEpoch) + 1u : 0u;
  const int quad = lane >> 2, tq = lane & 3;
  const int pt = warp / kBoxHeads, hl = warp % kBoxHeads;
  const int tiles = (geo.g + 7) / 8;                        // head tiles of 8 per KV head (N of the MMA)
  uint32_t wb[16][2];                                       // B operand: weights of head `quad`, 16 k-steps
  long long w_key = -1;
  int cur_b = 0;
  // weights of head h0 + quad of request b: min(q,0) against the minima (k < 128), max(q,0) against the maxima
  auto load_weights_global = [&](int b, int h0, int nh) {
    w_key = (long long)b * geo.Hq + h0;
    const uint16_t* qrow = q + (w_key + (quad < nh ? quad : 0)) * kHeadDim;
#pragma unroll
    for (int ks = 0; ks < 16; ++ks) {
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int col = ks * 16 + half * 8 + tq * 2;                // 0..255
        uint32_t pr = *reinterpret_cast<const uint32_t*>(qrow + (col & 127));
        // clamp each bf16 by its sign bit: keep negatives for the minima part, positives for the maxima part
        const bool want_neg = col < 128;
        uint32_t lo = pr & 0xFFFFu, hi = pr >> 16;
        if (((lo >> 15) != 0u) != want_neg) lo = 0u;
        if (((hi >> 15) != 0u) != want_neg) hi = 0u;
        wb[ks][half] = quad < nh ? (lo | (hi << 16)) : 0u;
      }
    }
  };
  // the same from the ring slot's weight rows (the block's pair; this warp's KV head is row block hl)
  auto load_weights_slot = [&](int stage, int nh) {
    const unsigned char* row = wring + ((size_t)stage * w_rows + hl * geo.g + (quad < nh ? quad : 0)) * kWeightRowBytes + tq * 4;
#pragma unroll
    for (int ks = 0; ks < 16; ++ks) {
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const uint32_t v = *reinterpret_cast<const uint32_t*>(row + (ks * 16 + half * 8) * 2);
        wb[ks][half] = quad < nh ? v : 0u;
      }
    }
  };
  for (int k = 0; k < n_blk; ++k) {
    const int stage = k % kMmaStages;
    const ScoreBlock blk = locate_block(blk_first + k * blk_step, cur_b, s_cum, ctx_len, geo.S, hpairs);
    const int b = blk.b, P = blk.P;
    const int kvh = blk.hp * kBoxHeads + hl;
    const bool active = kvh < geo.Hkv && pt < blk.n_tiles;
    const int p0 = blk.page0 + pt * kMmaPages;
    // without weight rows in the slot: the weights of the block's first head tile are fetched before the block has landed
    if (w_rows == 0 && active && (long long)b * geo.Hq + kvh * geo.g != w_key) load_weights_global(b, kvh * geo.g, min(8, geo.g));
    {
      const unsigned parity = (k / kMmaStages) & 1u;
      unsigned polls = 0;
      while (!sm_try_wait(&full[stage], parity) && ++polls < kStreamWaitLimit) __nanosleep(32);
      if (__any_sync(0xFFFFFFFFu, polls >= kStreamWaitLimit || s_abort != 0)) {
        if (lane == 0) { atomicOr(status, SWARM_DEV_TIMEOUT); s_abort = 1; }
        break;                                              // (the ticket warp stops at the first block left incomplete)
      }
    }
    SWARM_STAMP(status, 3 + 2 * min(k, 4));
    if (active) {
      // rows of a box: (page, head of the box) pairs, page-major; 128-byte swizzle over the row index
      const uint32_t base = sm_addr(ring + (size_t)stage * kMmaStageBytes + pt * kTileBytes);
      for (int ht = 0; ht < tiles; ++ht) {
        const int h0 = kvh * geo.g + ht * 8, nh = min(8, geo.g - ht * 8);
        if (w_rows > 0) load_weights_slot(stage, nh);
        else if ((long long)b * geo.Hq + h0 != w_key) load_weights_global(b, h0, nh);
        // A tiles: 16 pages x 16 coordinates per k-step; matrices (rows 0-7 | 8-15) x (chunk 2ks | 2ks+1).  Eight
        // tiles are fetched before the MMAs that use them, and the MMAs alternate between two accumulators: issued
        // one by one, every MMA waited for its own ldmatrix and for the MMA before it (~0.5 us per block).
        float acc2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        const int m = lane >> 3, r = (m & 1) * 8 + (lane & 7);
        const uint32_t row_base = base + (uint32_t)((r * kBoxHeads + hl) * 128);
        const int row_sw = (r * kBoxHeads + hl) & 7;
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) {
          uint32_t a[8][4];
#pragma unroll
          for (int k8 = 0; k8 < 8; ++k8) {
            const int cc = 2 * (kh * 8 + k8) + (m >> 1);
            asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                         : "=r"(a[k8][0]), "=r"(a[k8][1]), "=r"(a[k8][2]), "=r"(a[k8][3])
                         : "r"(row_base + (uint32_t)((cc >> 3) * (kTileBytes / 4) + (((cc & 7) ^ row_sw) << 4))));
          }
#pragma unroll
          for (int k8 = 0; k8 < 8; ++k8) {
            float* c = acc2[k8 & 1];
            asm volatile(
                "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                : "r"(a[k8][0]), "r"(a[k8][1]), "r"(a[k8][2]), "r"(a[k8][3]), "r"(wb[kh * 8 + k8][0]), "r"(wb[kh * 8 + k8][1]));
          }
        }
        const float acc[4] = {acc2[0][0] + acc2[1][0], acc2[0][1] + acc2[1][1], acc2[0][2] + acc2[1][2], acc2[0][3] + acc2[1][3]};
        // C: (page p0 + quad, heads 2tq, 2tq+1), (page p0 + quad + 8, same heads)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int hh = 2 * tq + (e & 1), p = p0 + quad + (e >> 1) * 8;
          if (hh < nh && p < P) {
            const long long at = ((long long)b * geo.Hq + h0 + hh) * geo.Pmax + p;
            scores[at] = acc[e];
            if (kPairs) ll_word_store(scores_ll + at, __float_as_uint(acc[e]), ll_flag);
          }
        }
      }
    }
    __syncwarp();
    SWARM_STAMP(status, 4 + 2 * min(k, 4));
    if (lane == 0) {
      // the warp's stores are ordered before this release by the barrier above; the ticket warp takes it from there
      asm volatile("red.release.cta.shared::cta.add.u32 [%0], 1;" ::"r"(sm_addr(&s_scored[stage])) : "memory");
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(sm_addr(&empty[stage])) : "memory");
    }
  }
  SWARM_STAMP(status, 13);
  SWARM_KERNEL_END(status, 0);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn summary_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// summaries as a 3-D bf16 tensor [page][kv head][256]; boxes of 16 pages x 2 KV heads x 64 coordinates
cudaError_t make_summary_map(CUtensorMap* map, const void* ksum, int Hkv, long long n_pool_pages) {
  EncodeTiledFn fn = summary_encode_fn();
  if (fn == nullptr) return cudaErrorNotSupported;
  const cuuint64_t dims[3] = {256, (cuuint64_t)Hkv, (cuuint64_t)n_pool_pages};
  const cuuint64_t strides[2] = {512, (cuuint64_t)Hkv * 512};
  const cuuint32_t box[3] = {64, (cuuint32_t)kBoxHeads, (cuuint32_t)kMmaPages};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ksum), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int G, int R, int NB>
cudaError_t launch_one(const Geometry& geo, const uint16_t* q, const uint16_t* ksum, const int64_t* page_base,
                       const int32_t* ctx_len, float* scores, uint32_t* status, cudaStream_t st) {
  const int pages_per_cta = kScoreWarps * R * NB;
  dim3 grid((geo.Pmax + pages_per_cta - 1) / pages_per_cta, geo.Hkv * (geo.g / G), geo.B);
  return launch_pdl(page_score_kernel<G, R, NB>, grid, dim3(kScoreWarps * 32), 0, st, true, geo, q, ksum, page_base,
                    ctx_len, scores, status);
}

cudaError_t launch_mma(const Geometry& geo, const uint16_t* q, const uint16_t* ksum, const int64_t* page_base,
                       const int32_t* ctx_len, float* scores, uint32_t* status, unsigned* ready, int reserve_sms,
                       uint2* scores_ll, const unsigned* ctl, bool early, cudaStream_t st) {
  CUtensorMap map;
  cudaError_t e = make_summary_map(&map, ksum, geo.Hkv, geo.n_pool_pages);
  if (e != cudaSuccess) return e;
  const long long max_blocks = (long long)geo.B * ((geo.Pmax + kBlkPages - 1) / kBlkPages) * head_pairs(geo.Hkv);
  const int sms = std::max(1, g_sm_count - reserve_sms);
  const int grid = (int)std::min<long long>(sms, std::max<long long>(1, max_blocks));
  const dim3 g(grid), b(kMmaThreads);
  const size_t smem = mma_smem_bytes(geo.g);
  uint2* no_pairs = nullptr;
  const unsigned* no_ctl = nullptr;
  if (scores_ll != nullptr && ctl != nullptr)
    return early ? launch_pdl(page_score_mma_kernel<true, true>, g, b, smem, st, true, map, geo, q, page_base, ctx_len, scores, status, ready, scores_ll, ctl)
                 : launch_pdl(page_score_mma_kernel<true, false>, g, b, smem, st, true, map, geo, q, page_base, ctx_len, scores, status, ready, scores_ll, ctl);
  return early ? launch_pdl(page_score_mma_kernel<false, true>, g, b, smem, st, true, map, geo, q, page_base, ctx_len, scores, status, ready, no_pairs, no_ctl)
               : launch_pdl(page_score_mma_kernel<false, false>, g, b, smem, st, true, map, geo, q, page_base, ctx_len, scores, status, ready, no_pairs, no_ctl);
}

}  // namespace

cudaError_t configure_score() {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  g_sm_count = sms > 0 ? sms : 148;
  if (summary_encode_fn() == nullptr) return cudaErrorNotSupported;   // resolved here, not inside a stream capture
  const int smem = mma_smem_bytes(kWeightRowsMax / 2);
  cudaError_t e2 = cudaFuncSetAttribute(page_score_mma_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e2 == cudaSuccess) e2 = cudaFuncSetAttribute(page_score_mma_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e2 == cudaSuccess) e2 = cudaFuncSetAttribute(page_score_mma_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e2 == cudaSuccess) e2 = cudaFuncSetAttribute(page_score_mma_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  return e2;
}

bool score_streams(const Geometry& geo) { return geo.B <= kStreamMaxBatch && geo.n_pool_pages < (1LL << 31); }
bool score_raises_tickets(const Geometry& geo) { return geo.scorer != SWARM_SCORER_FP32 && score_streams(geo); }

cudaError_t launch_page_score(const Geometry& geo, const uint16_t* q, const uint16_t* ksum,
                              const int64_t* page_base, const int32_t* ctx_len, float* scores, uint32_t* status,
                              cudaStream_t st, unsigned* ready, int reserve_sms, uint2* scores_ll, const unsigned* ctl,
                              bool index_early) {
  // Streaming tensor-core variant whenever the batch fits its prefix table and the pool fits 32-bit TMA
  // coordinates; otherwise the register-resident grid kernel on the fp32 pipes.
  if (score_raises_tickets(geo)) return launch_mma(geo, q, ksum, page_base, ctx_len, scores, status, ready, reserve_sms, scores_ll, ctl, index_early, st);
  // Heads of a KV group are processed G at a time, G the largest of 8/4/2/1 dividing the group size.
  if (geo.g % 8 == 0) return launch_one<8, 4, 4>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  if (geo.g % 4 == 0) return launch_one<4, 8, 2>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  if (geo.g % 2 == 0) return launch_one<2, 8, 2>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  return launch_one<1, 8, 2>(geo, q, ksum, page_base, ctx_len, scores, status, st);
}

}  // namespace swarm
