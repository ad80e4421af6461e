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
#include "swarm_internal.cuh"

namespace swarm {
namespace {

constexpr int kScoreWarps = 4;

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
}

template <int G, int R, int NB>
cudaError_t launch_one(const Geometry& geo, const uint16_t* q, const uint16_t* ksum, const int64_t* page_base,
                       const int32_t* ctx_len, float* scores, uint32_t* status, cudaStream_t st) {
  const int pages_per_cta = kScoreWarps * R * NB;
  dim3 grid((geo.Pmax + pages_per_cta - 1) / pages_per_cta, geo.Hkv * (geo.g / G), geo.B);
  page_score_kernel<G, R, NB><<<grid, kScoreWarps * 32, 0, st>>>(geo, q, ksum, page_base, ctx_len, scores, status);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_page_score(const Geometry& geo, const uint16_t* q, const uint16_t* ksum,
                              const int64_t* page_base, const int32_t* ctx_len, float* scores, uint32_t* status,
                              cudaStream_t st) {
  // Heads of a KV group are processed G at a time, G the largest of 8/4/2/1 dividing the group size.
  if (geo.g % 8 == 0) return launch_one<8, 4, 4>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  if (geo.g % 4 == 0) return launch_one<4, 8, 2>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  if (geo.g % 2 == 0) return launch_one<2, 8, 2>(geo, q, ksum, page_base, ctx_len, scores, status, st);
  return launch_one<1, 8, 2>(geo, q, ksum, page_base, ctx_len, scores, status, st);
}

}  // namespace swarm
