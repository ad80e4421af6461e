// Stage 4b: single-row attention (Eq. 1) over each head's selected tokens, as split-K flash decoding.
//
// Every query head has its own page list, so the contraction is a matrix-vector product: 4*d
// flops per 2*d*2 bytes of K and V, about one flop per byte -- bound by HBM bandwidth, so the
// arithmetic stays on the fp32 pipes and the design effort goes into keeping bytes in flight.
//
// Data movement: each warp owns a ring of kStages shared-memory slots.  A slot holds 16 tokens of K
// and the same 16 tokens of V (2 x 4 KiB).  Lane 0 fills slots with bulk asynchronous copies
// (cp.async.bulk, completion counted in bytes on the slot's mbarrier) up to kStages units ahead, so
// the memory system always has kStages * 8 KiB per warp outstanding while the warp computes on the
// slot that has landed.  Rings are private to a warp: no CTA-wide barrier in the main loop.
// Every mbarrier wait is bounded; on expiry the warp records SWARM_DEV_TIMEOUT and stops.
//
// Compute on a slot: lane (half, c) reads 16 bytes (coordinates [8c, 8c+8)) of token 2i+half for
// i = 0..7, conflict-free.  The 8 partial dot products per lane are summed over the 16 lanes of a
// half with a transposing butterfly (8 shuffles).  Logits live in the log2 domain (q is pre-scaled
// by log2(e)/sqrt(d)); softmax state (m, l, 128 accumulators) stays in fp32 registers.
//
// Work split: grid = (request, head, split); a split's pages are dealt round-robin to the CTA's
// warps.  Warps are merged through shared memory, splits through fp32 partials in global memory:
// the CTA that arrives last at the head's ticket counter merges them and writes out / lse, so no
// second launch is needed.
//
// The same kernel serves the contiguous gathered buffers (swarm_sparse_attn) and the paged pool
// (swarm_step); only the address and valid-token computation differ.
#include "swarm_internal.cuh"

namespace swarm {
namespace {

constexpr int kAttnWarps = 4;
constexpr int kStages = 3;
constexpr int kUnitTokens = 16;
constexpr int kHalfSlotBytes = kUnitTokens * kHeadDim * 2;       // 4 KiB of K (or V)
constexpr int kSlotBytes = 2 * kHalfSlotBytes;
constexpr int kAttnSmemBytes = kAttnWarps * kStages * kSlotBytes;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr unsigned kWaitLimit = 1u << 22;                         // polls of a try_wait that itself blocks briefly

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, unsigned bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_addr(dst)),
               "l"(src), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xFFFFFFFFu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
  return x;
}
__device__ __forceinline__ float exp2_or_zero(float x, float ref) {   // 2^(x-ref), 0 when x = -inf
  return x == -INFINITY ? 0.f : exp2f(x - ref);
}

struct WarpState {
  float m, l, acc[8];
};

// 16 tokens in a shared-memory slot (K rows then V rows, 256 bytes each), of which the first `valid` exist.
__device__ __forceinline__ void attend_16(const unsigned char* __restrict__ slot, int valid, const float (&qf)[8],
                                          int lane, WarpState& st) {
  const int half = lane >> 4, c = lane & 15;
  const uint4* Ks = reinterpret_cast<const uint4*>(slot);
  const uint4* Vs = reinterpret_cast<const uint4*>(slot + kHalfSlotBytes);
  float s[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int t = 2 * i + half;
    const uint4 kr = Ks[t * 16 + c];
    const uint32_t w[4] = {kr.x, kr.y, kr.z, kr.w};
    float a = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      a = fmaf(qf[2 * e], bf16_lo(w[e]), a);
      a = fmaf(qf[2 * e + 1], bf16_hi(w[e]), a);
    }
    s[i] = a;
  }
  // sum over the 16 lanes of the half; afterwards the lane holds the logit of token 2*(c>>1)+half
#pragma unroll
  for (int n = 8, off = 8; n > 1; n >>= 1, off >>= 1) {
    const bool upper = (c & off) != 0;
#pragma unroll
    for (int j = 0; j < n / 2; ++j) {
      const float keep = upper ? s[j + n / 2] : s[j];
      const float send = upper ? s[j] : s[j + n / 2];
      s[j] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, off);
    }
  }
  float x = s[0] + __shfl_xor_sync(0xFFFFFFFFu, s[0], 1);
  const int my_t = 2 * (c >> 1) + half;
  if (my_t >= valid) x = -INFINITY;                     // padding tokens: masked (their bytes may be anything)
  const float m_new = fmaxf(st.m, warp_max(x));
  const float corr = exp2_or_zero(st.m, m_new);
  const float p = exp2_or_zero(x, m_new);
  st.l = st.l * corr + ((c & 1) == 0 ? p : 0.f);
  st.m = m_new;
#pragma unroll
  for (int e = 0; e < 8; ++e) st.acc[e] *= corr;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int t = 2 * i + half;
    const float pi = __shfl_sync(0xFFFFFFFFu, p, half * 16 + 2 * i);
    uint4 vr = Vs[t * 16 + c];
    if (t >= valid) vr = make_uint4(0, 0, 0, 0);        // 0 * garbage must stay 0
    const uint32_t w[4] = {vr.x, vr.y, vr.z, vr.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      st.acc[2 * e] = fmaf(pi, bf16_lo(w[e]), st.acc[2 * e]);
      st.acc[2 * e + 1] = fmaf(pi, bf16_hi(w[e]), st.acc[2 * e + 1]);
    }
  }
}

template <int S, bool kPaged>
__global__ void __launch_bounds__(kAttnWarps * 32)
attn_kernel(Geometry geo, AttnArgs a, uint32_t* __restrict__ status) {
  constexpr int SB = S / kUnitTokens;                   // 16-token units per page
  extern __shared__ __align__(128) unsigned char ring[];
  __shared__ __align__(8) uint64_t bars[kAttnWarps][kStages];
  __shared__ float s_m[kAttnWarps], s_l[kAttnWarps];
  __shared__ float s_acc[kAttnWarps][kHeadDim];
  __shared__ bool s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int split = blockIdx.x % a.n_splits, bh = blockIdx.x / a.n_splits;
  const int b = bh / geo.Hq, h = bh % geo.Hq, kvh = h / geo.g;
  const int c = lane & 15;
  const long long blk = (long long)S * kHeadDim;        // elements per K (or V) block of a page

  if (lane == 0) {
#pragma unroll
    for (int sidx = 0; sidx < kStages; ++sidx) mbar_init(&bars[warp][sidx], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  SWARM_STAMP(status, 0);
  pdl_wait();                                           // the selection comes from the previous kernel
  SWARM_STAMP(status, 1);

  int n_pages, P = 0, tail = S, total_tok = 0;
  long long pool_row0 = 0;
  if (kPaged) {
    n_pages = a.n_sel[bh];
    const int len = a.ctx_len[b];
    P = pages_of(len, S);
    tail = len - S * (P - 1);
    pool_row0 = a.page_base[b];
  } else {
    total_tok = a.n_tok[bh];
    n_pages = (total_tok + S - 1) / S;
  }
  const int j_begin = (int)((long long)n_pages * split / a.n_splits);
  const int j_end = (int)((long long)n_pages * (split + 1) / a.n_splits);

  float qf[8];
  {
    const uint4 qq = *reinterpret_cast<const uint4*>(a.q + (long long)bh * kHeadDim + c * 8);
    const uint32_t w[4] = {qq.x, qq.y, qq.z, qq.w};
    const float scale = kLog2e * rsqrtf((float)kHeadDim);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      qf[2 * e] = bf16_lo(w[e]) * scale;
      qf[2 * e + 1] = bf16_hi(w[e]) * scale;
    }
  }

  WarpState st;
  st.m = -INFINITY;
  st.l = 0.f;
#pragma unroll
  for (int e = 0; e < 8; ++e) st.acc[e] = 0.f;

  unsigned char* my_ring = ring + (size_t)warp * kStages * kSlotBytes;
  unsigned err = 0u;
  SWARM_STAMP(status, 2);

  // This warp's pages are j_begin + warp + kAttnWarps*i, i = 0 .. n_mine-1, handled 32 at a time
  // (lane i holds the i-th page id); each page is SB units of 16 tokens.
  const int n_mine = (j_end - j_begin - warp + kAttnWarps - 1) / kAttnWarps;
  unsigned fills = 0;                                   // units issued so far (slot = fills % kStages)
  unsigned drains = 0;                                  // units consumed so far
  for (int i0 = 0; i0 < n_mine && err == 0u; i0 += 32) {
    const int n_here = min(32, n_mine - i0);
    int my_p = -1;
    if (kPaged && lane < n_here) my_p = a.sel[(long long)bh * geo.k + j_begin + warp + kAttnWarps * (i0 + lane)];
    const int units = n_here * SB;

    auto unit_valid = [&](int u, int p) -> int {        // valid tokens of unit u (page i0 + u/SB, sub-block u%SB)
      const int sb = u % SB;
      int valid;
      if (kPaged) valid = (p == P - 1) ? tail : S;
      else valid = min(S, total_tok - (j_begin + warp + kAttnWarps * (i0 + u / SB)) * S);
      return max(0, min(kUnitTokens, valid - sb * kUnitTokens));
    };
    auto issue = [&](int u) {                           // all lanes call; lane 0 issues the copies
      const int p = __shfl_sync(0xFFFFFFFFu, my_p, u / SB);
      const int sb = u % SB;
      const uint16_t *Kp, *Vp;
      if (kPaged) {
        const int pc = (p < 0 || p >= P) ? 0 : p;       // a corrupt id is flagged when consumed; copy something legal
        Kp = a.kv_pool + (((pool_row0 + pc) * geo.Hkv + kvh) * 2) * blk;
        Vp = Kp + blk;
      } else {
        const long long j = j_begin + warp + kAttnWarps * (i0 + u / SB);
        Kp = a.k_g + ((long long)bh * geo.k + j) * blk;
        Vp = a.v_g + ((long long)bh * geo.k + j) * blk;
      }
      if (lane == 0) {
        const unsigned slot = fills % kStages;
        unsigned char* dst = my_ring + slot * kSlotBytes;
        mbar_expect_tx(&bars[warp][slot], kSlotBytes);
        bulk_copy_g2s(dst, Kp + sb * kUnitTokens * kHeadDim, kHalfSlotBytes, &bars[warp][slot]);
        bulk_copy_g2s(dst + kHalfSlotBytes, Vp + sb * kUnitTokens * kHeadDim, kHalfSlotBytes, &bars[warp][slot]);
      }
      ++fills;
    };

    int issued = 0;
    for (; issued < min(units, kStages); ++issued) issue(issued);
    SWARM_STAMP(status, 3);
    for (int u = 0; u < units; ++u) {
      const unsigned slot = drains % kStages, parity = (drains / kStages) & 1u;
      unsigned polls = 0;
      while (!mbar_try_wait(&bars[warp][slot], parity) && ++polls < kWaitLimit) {}
      if (__any_sync(0xFFFFFFFFu, polls >= kWaitLimit)) { err = SWARM_DEV_TIMEOUT; break; }
      ++drains;
      const int p = __shfl_sync(0xFFFFFFFFu, my_p, u / SB);
      if (kPaged && (p < 0 || p >= P)) {
        if (lane == 0) atomicOr(status, SWARM_DEV_BAD_PAGE);   // corrupt selection: skip the page, keep going
      } else {
        const int v16 = unit_valid(u, p);
        if (v16 > 0) attend_16(my_ring + slot * kSlotBytes, v16, qf, lane, st);
      }
      __syncwarp();                                     // every lane is done reading the slot
      if (issued < units) { issue(issued); ++issued; }
    }
  }
  if (err) {
    // a wait expired: give the copies still in flight a bounded chance to land before the CTA's shared
    // memory is released, then report
    for (; drains < fills; ++drains) {
      const unsigned slot = drains % kStages, parity = (drains / kStages) & 1u;
      unsigned polls = 0;
      while (!mbar_try_wait(&bars[warp][slot], parity) && ++polls < kWaitLimit) {}
    }
    if (lane == 0) atomicOr(status, err);
  }

  SWARM_STAMP(status, 4);
  // merge the two halves of the warp, then the warps of the CTA
  const float l_warp = warp_sum(st.l);
#pragma unroll
  for (int e = 0; e < 8; ++e) st.acc[e] += __shfl_xor_sync(0xFFFFFFFFu, st.acc[e], 16);
  if (lane < 16) {
#pragma unroll
    for (int e = 0; e < 8; ++e) s_acc[warp][c * 8 + e] = st.acc[e];
  }
  if (lane == 0) { s_m[warp] = st.m; s_l[warp] = l_warp; }
  __syncthreads();
  const int t = threadIdx.x;                          // one output coordinate per thread
  float M = s_m[0];
#pragma unroll
  for (int w = 1; w < kAttnWarps; ++w) M = fmaxf(M, s_m[w]);
  float L = 0.f, o = 0.f;
#pragma unroll
  for (int w = 0; w < kAttnWarps; ++w) {
    const float sc = exp2_or_zero(s_m[w], M);
    L += s_l[w] * sc;
    o += s_acc[w][t] * sc;
  }
  if (a.n_splits > 1) {
    // publish this split's partial, then let the last split of the head merge all of them
    const long long slot = (long long)bh * a.n_splits + split;
    __stcg(&a.part_acc[slot * kHeadDim + t], o);
    if (t == 0) { __stcg(&a.part_ml[slot * 2], M); __stcg(&a.part_ml[slot * 2 + 1], L); }
    __threadfence();
    __syncthreads();
    if (t == 0) s_last = (atomicAdd(&a.tickets[bh], 1u) == (unsigned)a.n_splits - 1u);
    __syncthreads();
    SWARM_STAMP(status, 5);
    if (!s_last) return;
    __threadfence();
    const float* ml = a.part_ml + (long long)bh * a.n_splits * 2;
    M = -INFINITY;
    for (int sp = 0; sp < a.n_splits; ++sp) M = fmaxf(M, __ldcg(&ml[2 * sp]));
    L = 0.f;
    o = 0.f;
    for (int sp = 0; sp < a.n_splits; ++sp) {
      const float sc = exp2_or_zero(__ldcg(&ml[2 * sp]), M);
      L += __ldcg(&ml[2 * sp + 1]) * sc;
      o += __ldcg(&a.part_acc[((long long)bh * a.n_splits + sp) * kHeadDim + t]) * sc;
    }
    if (t == 0) a.tickets[bh] = 0u;                     // ready for the next launch
  }
  a.out[(long long)bh * kHeadDim + t] = L > 0.f ? o / L : 0.f;
  if (t == 0) a.lse[bh] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
  SWARM_STAMP_ANY_CTA(status, 6);
}

template <int S, bool kPaged>
cudaError_t launch_variant(const Geometry& geo, const AttnArgs& a, uint32_t* status, cudaStream_t st, bool overlap) {
  const unsigned grid = (unsigned)geo.B * geo.Hq * a.n_splits;
  return launch_pdl(attn_kernel<S, kPaged>, dim3(grid), dim3(kAttnWarps * 32), kAttnSmemBytes, st, overlap, geo, a,
                    status);
}

}  // namespace

cudaError_t configure_attention() {
  cudaError_t e = cudaFuncSetAttribute(attn_kernel<16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_kernel<16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_kernel<32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_kernel<32, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemBytes);
  return e;
}

cudaError_t launch_attention(const Geometry& geo, const AttnArgs& a, uint32_t* status, cudaStream_t st,
                             bool overlap) {
  const bool paged = a.kv_pool != nullptr;
  if (geo.S == 16)
    return paged ? launch_variant<16, true>(geo, a, status, st, overlap)
                 : launch_variant<16, false>(geo, a, status, st, overlap);
  return paged ? launch_variant<32, true>(geo, a, status, st, overlap)
               : launch_variant<32, false>(geo, a, status, st, overlap);
}

}  // namespace swarm

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of swarm_sparse_attn (see swarm.h).  The split-K partials live in a
// file-scope device array instead of a caller-provided workspace.  Layout of the array:
//   [0, 256)                       status word (unused by the contiguous-buffer kernel) + padding
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
unsigned char* g_static_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal

cudaError_t static_scratch_address(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (g_static_ptr[dev] == nullptr) {   // set-up for this device (idempotent if two threads race here)
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_static_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_static_ptr[dev];
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
  // same split heuristic as the ctx path (about 2 CTAs per SM, >= 4 pages per split), capped by the array
  long long n = (148 * 2) / bh;
  n = n < (top_k / 4 > 1 ? top_k / 4 : 1) ? n : (top_k / 4 > 1 ? top_k / 4 : 1);
  n = n < kMaxSplits ? n : kMaxSplits;
  n = n < kStaticSlots / bh ? n : kStaticSlots / bh;
  n = n < 1 ? 1 : n;

  unsigned char* base = nullptr;
  if (static_scratch_address(&base) != cudaSuccess) return SWARM_ERR_CUDA;
  if (configure_attention() != cudaSuccess) return SWARM_ERR_CUDA;   // raises a kernel attribute; allocates nothing
  Geometry geo{};
  geo.B = batch; geo.Hq = n_q_heads; geo.Hkv = n_q_heads; geo.g = 1; geo.S = page_size; geo.k = top_k; geo.D = 1;
  geo.Pmax = top_k; geo.Cmax = 1; geo.flags = 0; geo.n_pool_pages = 0;
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
