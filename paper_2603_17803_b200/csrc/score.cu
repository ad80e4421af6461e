// Stage 1: activation scoring (Sec. 2.3: relevance score of every cached entry against the query).
//
//   score[b][h][p] = sum_i max(q[i]*kmin[p][i], q[i]*kmax[p][i])
//                  = sum_i max(q[i],0)*kmax[p][i] + min(q[i],0)*kmin[p][i]        (kmin <= kmax)
//
// One summary row (page, kv head) is 512 contiguous bytes: 128 bf16 minima then 128 bf16 maxima.
// A warp reads a row with one 16-byte load per lane (lanes 0-15 hold minima, 16-31 maxima), so the
// sign-split form needs one multiply-add per element and query head, with the weights (min(q,0) on
// the low lanes, max(q,0) on the high lanes) held in registers for all G heads of the KV group.
// The multiply-adds are issued two at a time (fma.rn.f32x2 on even/odd coordinates).
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
#include <algorithm>

#include "swarm_internal.cuh"

namespace swarm {
namespace {

constexpr int kScoreWarps = 4;
int g_sm_count = 148;                                      // set by configure_score()

__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ float sum2(uint64_t v) {
  float lo, hi;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
  return lo + hi;
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}

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

template <int G, int R, int NB>
__global__ void __launch_bounds__(kScoreWarps * 32, 3)
page_score_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ ksum,
                  const int64_t* __restrict__ page_base, const int32_t* __restrict__ ctx_len,
                  float* __restrict__ scores, uint32_t* __restrict__ status) {
  constexpr int NV = G * R;
  constexpr int LOG_NV = ilog2(NV), LOG_G = ilog2(G);
  static_assert(NV <= 32 && (1 << LOG_NV) == NV && (1 << LOG_G) == G, "R and G must be powers of two, R*G <= 32");
  pdl_launch_dependents();   // the next kernel may be scheduled as soon as every CTA of this one runs
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
  // Weights of this lane's 8 coordinates, as 4 (even, odd) pairs; w[c] belongs to head (c XOR head_sel).
  const int h0 = kvh * geo.g + tile * G;
  uint64_t w[G][4];
#pragma unroll
  for (int c = 0; c < G; ++c) {
    const int h = h0 + (c ^ head_sel);
    const uint4 qq = *reinterpret_cast<const uint4*>(q + ((long long)(b * geo.Hq + h) * kHeadDim + (lane & 15) * 8));
    const uint32_t words[4] = {qq.x, qq.y, qq.z, qq.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float lo = bf16_lo(words[e]), hi = bf16_hi(words[e]);
      w[c][e] = lane < 16 ? pack2(fminf(lo, 0.f), fminf(hi, 0.f)) : pack2(fmaxf(lo, 0.f), fmaxf(hi, 0.f));
    }
  }

  SWARM_STAMP(status, 2);
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    const int p0 = p_warp + nb * R;
    if (p0 >= P) break;
    float v[NV];
#pragma unroll
    for (int a = 0; a < R; ++a) {
      const uint32_t words[4] = {data[nb][a].x, data[nb][a].y, data[nb][a].z, data[nb][a].w};
      uint64_t x[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) x[e] = pack2(bf16_lo(words[e]), bf16_hi(words[e]));
#pragma unroll
      for (int c = 0; c < G; ++c) {
        uint64_t acc = 0ull;
#pragma unroll
        for (int e = 0; e < 4; ++e) acc = ffma2(w[c][e], x[e], acc);
        v[a * G + c] = sum2(acc);
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

#if defined(SWARM_TRACE) && SWARM_TRACE == 3     // phases of the streaming scorer only
#define SCORE_STAMP(status, i) SWARM_STAMP_RAW(status, i, false)
#define SCORE_STAMP_ANY(status, i) SWARM_STAMP_RAW(status, i, true)
#else
#define SCORE_STAMP(status, i) do { } while (0)
#define SCORE_STAMP_ANY(status, i) do { } while (0)
#endif

// ---- streaming variant -----------------------------------------------------------------------------
// One persistent CTA per SM.  The summaries of `ppc` consecutive pages of a request (all KV heads) are one
// contiguous block of memory, so a producer warp brings them in with one bulk asynchronous copy per block
// (64 KiB) into a 3-slot shared-memory ring while 16 consumer warps score the block that has landed:
// the bytes in flight (up to 192 KiB per SM) no longer depend on how many registers the arithmetic needs.
// The CTAs split the blocks of all requests evenly; each (KV head, 8-row batch) of a block is one warp's item.
constexpr int kStreamConsumers = 16;
constexpr int kStreamThreads = (kStreamConsumers + 1) * 32;
constexpr int kStreamStages = 3;
constexpr int kStreamBlockBytes = 64 * 1024;
constexpr int kStreamMaxBatch = 1024;                     // requests whose block counts fit the shared prefix table
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

template <int G, int R>
__global__ void __launch_bounds__(kStreamThreads, 1)
page_score_stream_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ ksum,
                         const int64_t* __restrict__ page_base, const int32_t* __restrict__ ctx_len,
                         float* __restrict__ scores, uint32_t* __restrict__ status, int ppc) {
  constexpr int NV = G * R;
  constexpr int LOG_NV = ilog2(NV), LOG_G = ilog2(G);
  extern __shared__ __align__(128) unsigned char stream_ring[];
  __shared__ __align__(8) uint64_t full[kStreamStages], empty[kStreamStages];
  __shared__ int s_cum[kStreamMaxBatch + 1];               // blocks before request b
  __shared__ int s_abort;
  pdl_launch_dependents();
  SWARM_KERNEL_BEGIN(status, 0);
  SCORE_STAMP(status, 0);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int sidx = 0; sidx < kStreamStages; ++sidx) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(sm_addr(&full[sidx])), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(sm_addr(&empty[sidx])), "r"(kStreamConsumers));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_abort = 0;
    s_cum[0] = 0;
  }
  // blocks per request (serial prefix by one warp: B is small next to the streaming work)
  if (warp == 0) {
    int running = 0;
    for (int b0 = 0; b0 < geo.B; b0 += 32) {
      const int b = b0 + lane;
      int nb = 0;
      if (b < geo.B) {
        const int len = ctx_len[b];
        const int P = pages_of(len, geo.S);
        if (len < 1 || P > page_base[b + 1] - page_base[b] || P > geo.Pmax) atomicOr(status, SWARM_DEV_BAD_LENGTH);
        else nb = (P + ppc - 1) / ppc;
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
  SCORE_STAMP(status, 1);
  const int total = s_cum[geo.B];
  const int blk_lo = (int)((long long)total * blockIdx.x / gridDim.x);
  const int blk_hi = (int)((long long)total * (blockIdx.x + 1) / gridDim.x);
  const int row_bytes = geo.Hkv * 512;                     // summaries of one page, all KV heads

  // request of a block index, found by walking forward (blocks are visited in order)
  int cur_b = 0;
  auto locate = [&](int blk) {
    while (s_cum[cur_b + 1] <= blk) ++cur_b;
    return blk - s_cum[cur_b];                            // block index inside request cur_b
  };

  if (warp == kStreamConsumers) {
    // ---- producer ----
    if (lane == 0) {
      for (int blk = blk_lo; blk < blk_hi; ++blk) {
        const int k = blk - blk_lo, stage = k % kStreamStages;
        if (k >= kStreamStages) {
          const unsigned parity = ((k / kStreamStages) - 1) & 1u;
          unsigned polls = 0;
          while (!sm_try_wait(&empty[stage], parity) && ++polls < kStreamWaitLimit && !s_abort) {}
          if (polls >= kStreamWaitLimit || s_abort) { atomicOr(status, SWARM_DEV_TIMEOUT); s_abort = 1; break; }
        }
        const int c = locate(blk);
        const int b = cur_b;
        const int P = pages_of(ctx_len[b], geo.S);
        const int pages = min(ppc, P - c * ppc);
        const unsigned bytes = (unsigned)(pages * row_bytes);
        const uint16_t* src = ksum + (page_base[b] + (long long)c * ppc) * geo.Hkv * 2 * kHeadDim;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(sm_addr(&full[stage])), "r"(bytes)
                     : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         sm_addr(stream_ring + (size_t)stage * kStreamBlockBytes)),
                     "l"(src), "r"(bytes), "r"(sm_addr(&full[stage]))
                     : "memory");
      }
    }
    return;
  }

  // ---- consumers ----
  const int pi = lane >> (5 - LOG_NV);                      // slot permutation, as in page_score_kernel
  const int row_sel = pi >> LOG_G, head_sel = pi & (G - 1);
  const int tiles = geo.g / G;
  const int batches = (ppc + R - 1) / R;
  const int items_full = geo.Hkv * tiles * batches;
  uint64_t w[G][4];
  int w_key = -1;                                           // (request, kv head, tile) the weights belong to

  auto load_weights = [&](int b, int kvh, int tile) {
    const int key = (b * geo.Hkv + kvh) * tiles + tile;
    if (key == w_key) return;
    w_key = key;
    const int h0 = kvh * geo.g + tile * G;
#pragma unroll
    for (int cc = 0; cc < G; ++cc) {
      const int h = h0 + (cc ^ head_sel);
      const uint4 qq = *reinterpret_cast<const uint4*>(q + ((long long)(b * geo.Hq + h) * kHeadDim + (lane & 15) * 8));
      const uint32_t words[4] = {qq.x, qq.y, qq.z, qq.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float lo = bf16_lo(words[e]), hi = bf16_hi(words[e]);
        w[cc][e] = lane < 16 ? pack2(fminf(lo, 0.f), fminf(hi, 0.f)) : pack2(fmaxf(lo, 0.f), fmaxf(hi, 0.f));
      }
    }
  };
  if (blk_lo < blk_hi) {                                    // the first item's weights, fetched while the first block is in flight
    locate(blk_lo);
    const int kt = warp / batches;
    if (warp < items_full) load_weights(cur_b, kt / tiles, kt % tiles);
  }

  for (int blk = blk_lo; blk < blk_hi; ++blk) {
    const int k = blk - blk_lo, stage = k % kStreamStages;
    const int c = locate(blk);
    const int b = cur_b;
    const int P = pages_of(ctx_len[b], geo.S);
    const int pages = min(ppc, P - c * ppc);
    {
      const unsigned parity = (k / kStreamStages) & 1u;
      unsigned polls = 0;
      while (!sm_try_wait(&full[stage], parity) && ++polls < kStreamWaitLimit && !s_abort) {}
      if (__any_sync(0xFFFFFFFFu, polls >= kStreamWaitLimit || s_abort != 0)) {
        if (lane == 0) { atomicOr(status, SWARM_DEV_TIMEOUT); s_abort = 1; }
        break;
      }
    }
    SCORE_STAMP(status, 2 + 2 * k);
    const unsigned char* blkmem = stream_ring + (size_t)stage * kStreamBlockBytes;
    for (int item = warp; item < items_full; item += kStreamConsumers) {
      const int rb = item % batches, kt = item / batches;
      const int tile = kt % tiles, kvh = kt / tiles;
      if (rb * R >= pages) continue;
      const int h0 = kvh * geo.g + tile * G;
      load_weights(b, kvh, tile);
      float v[NV];
#pragma unroll
      for (int a = 0; a < R; ++a) {
        const int pl = rb * R + (a ^ row_sel);              // page inside the block
        uint4 d = make_uint4(0, 0, 0, 0);
        if (pl < pages) d = *reinterpret_cast<const uint4*>(blkmem + ((size_t)pl * geo.Hkv + kvh) * 512 + lane * 16);
        const uint32_t words[4] = {d.x, d.y, d.z, d.w};
        uint64_t x[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) x[e] = pack2(bf16_lo(words[e]), bf16_hi(words[e]));
#pragma unroll
        for (int cc = 0; cc < G; ++cc) {
          uint64_t acc = 0ull;
#pragma unroll
          for (int e = 0; e < 4; ++e) acc = ffma2(w[cc][e], x[e], acc);
          v[a * G + cc] = sum2(acc);
        }
      }
      const float total_v = butterfly<NV>(v);
      const int r = pi >> LOG_G, hh = pi & (G - 1);
      const int p = c * ppc + rb * R + r;
      if ((lane & ((1 << (5 - LOG_NV)) - 1)) == 0 && rb * R + r < pages)
        scores[((long long)(b * geo.Hq + h0 + hh)) * geo.Pmax + p] = total_v;
    }
    __syncwarp();
    SCORE_STAMP(status, 3 + 2 * k);
    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(sm_addr(&empty[stage])) : "memory");
  }
  SCORE_STAMP_ANY(status, 15);
  SWARM_KERNEL_END(status, 0);
}

template <int G, int R, int NB>
cudaError_t launch_one(const Geometry& geo, const uint16_t* q, const uint16_t* ksum, const int64_t* page_base,
                       const int32_t* ctx_len, float* scores, uint32_t* status, cudaStream_t st) {
  const int pages_per_cta = kScoreWarps * R * NB;
  dim3 grid((geo.Pmax + pages_per_cta - 1) / pages_per_cta, geo.Hkv * (geo.g / G), geo.B);
  page_score_kernel<G, R, NB><<<grid, kScoreWarps * 32, 0, st>>>(geo, q, ksum, page_base, ctx_len, scores, status);
  return cudaGetLastError();
}

template <int G, int R>
cudaError_t launch_stream(const Geometry& geo, const uint16_t* q, const uint16_t* ksum, const int64_t* page_base,
                          const int32_t* ctx_len, float* scores, uint32_t* status, cudaStream_t st) {
  const int ppc = kStreamBlockBytes / (geo.Hkv * 512);
  const long long max_blocks = (long long)geo.B * ((geo.Pmax + ppc - 1) / ppc);
  const int grid = (int)std::min<long long>(g_sm_count, std::max<long long>(1, max_blocks));
  page_score_stream_kernel<G, R><<<grid, kStreamThreads, kStreamStages * kStreamBlockBytes, st>>>(
      geo, q, ksum, page_base, ctx_len, scores, status, ppc);
  return cudaGetLastError();
}

}  // namespace

cudaError_t configure_score() {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  g_sm_count = sms > 0 ? sms : 148;
  const int bytes = kStreamStages * kStreamBlockBytes;
  e = cudaFuncSetAttribute(page_score_stream_kernel<8, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(page_score_stream_kernel<4, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(page_score_stream_kernel<2, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(page_score_stream_kernel<1, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  return e;
}

cudaError_t launch_page_score(const Geometry& geo, const uint16_t* q, const uint16_t* ksum,
                              const int64_t* page_base, const int32_t* ctx_len, float* scores, uint32_t* status,
                              cudaStream_t st) {
  // Streaming variant whenever one page's summaries (all KV heads) fit the block size a few times over and
  // the batch fits its prefix table; otherwise the register-resident grid kernel.
  if (geo.Hkv * 512 * 2 <= kStreamBlockBytes && geo.B <= kStreamMaxBatch) {
    if (geo.g % 8 == 0) return launch_stream<8, 4>(geo, q, ksum, page_base, ctx_len, scores, status, st);
    if (geo.g % 4 == 0) return launch_stream<4, 8>(geo, q, ksum, page_base, ctx_len, scores, status, st);
    if (geo.g % 2 == 0) return launch_stream<2, 8>(geo, q, ksum, page_base, ctx_len, scores, status, st);
    return launch_stream<1, 8>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  }
  // Heads of a KV group are processed G at a time, G the largest of 8/4/2/1 dividing the group size.
  if (geo.g % 8 == 0) return launch_one<8, 4, 4>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  if (geo.g % 4 == 0) return launch_one<4, 8, 2>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  if (geo.g % 2 == 0) return launch_one<2, 8, 2>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  return launch_one<1, 8, 2>(geo, q, ksum, page_base, ctx_len, scores, status, st);
}

}  // namespace swarm
