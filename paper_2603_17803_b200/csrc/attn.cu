// Stage 4b: single-row attention (Eq. 1) over each head's selected tokens, as split-K flash decoding.
//
// Every query head has its own page list, so the contraction is a matrix-vector product: 4*d
// flops per 2*d*2 bytes of K and V, i.e. bound by HBM bandwidth with arithmetic intensity 1.
// The kernel therefore streams pages with 16-byte loads straight into registers and keeps the
// softmax state (running max m, sum l, 128 accumulators) in fp32 registers of the warp that owns
// the page; nothing is staged through shared memory and no operand is reused.
//
// Work split: grid = (request, head, split); the split's pages are dealt round-robin to the 4
// warps of the CTA.  A warp handles 16 tokens at a time: lane (half, c) loads 16 bytes
// (coordinates [8c, 8c+8)) of token 2i+half for i = 0..7, so each load instruction of the warp
// covers two whole 256-byte token rows.  The 8 partial dot products per lane are summed over the
// 16 lanes of a half with a transposing butterfly (8 shuffles).  Logits are kept in the log2
// domain (q is pre-scaled by log2(e)/sqrt(d)).  Warps, then splits, are merged by their (m, l).
//
// The same kernel serves the contiguous gathered buffers (swarm_sparse_attn) and the paged pool
// (swarm_step); only the address and valid-token computation differ.
#include "swarm_internal.cuh"

namespace swarm {
namespace {

constexpr int kAttnWarps = 4;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

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

// 16 tokens (rows of 256 bytes at Kb / Vb), of which the first `valid` exist.
__device__ __forceinline__ void attend_16(const uint16_t* __restrict__ Kb, const uint16_t* __restrict__ Vb,
                                          int valid, const float (&qf)[8], int lane, WarpState& st) {
  const int half = lane >> 4, c = lane & 15;
  uint4 kr[8], vr[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int t = 2 * i + half;
    const bool ok = t < valid;
    kr[i] = ok ? ldg_nc_v4(Kb + t * kHeadDim + c * 8) : make_uint4(0, 0, 0, 0);
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int t = 2 * i + half;
    const bool ok = t < valid;
    vr[i] = ok ? ldg_nc_v4(Vb + t * kHeadDim + c * 8) : make_uint4(0, 0, 0, 0);
  }
  float s[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t w[4] = {kr[i].x, kr[i].y, kr[i].z, kr[i].w};
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
  if (my_t >= valid) x = -INFINITY;
  const float m_new = fmaxf(st.m, warp_max(x));
  const float corr = exp2_or_zero(st.m, m_new);
  const float p = exp2_or_zero(x, m_new);
  st.l = st.l * corr + ((c & 1) == 0 ? p : 0.f);
  st.m = m_new;
#pragma unroll
  for (int e = 0; e < 8; ++e) st.acc[e] *= corr;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float pi = __shfl_sync(0xFFFFFFFFu, p, half * 16 + 2 * i);
    const uint32_t w[4] = {vr[i].x, vr[i].y, vr[i].z, vr[i].w};
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
  __shared__ float s_m[kAttnWarps], s_l[kAttnWarps];
  __shared__ float s_acc[kAttnWarps][kHeadDim];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int split = blockIdx.x % a.n_splits, bh = blockIdx.x / a.n_splits;
  const int b = bh / geo.Hq, h = bh % geo.Hq, kvh = h / geo.g;
  const int c = lane & 15;
  const long long blk = (long long)S * kHeadDim;

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

  // pages j_begin + warp + 4*i; their ids are fetched 32 at a time (lane i holds the i-th)
  for (int j0 = j_begin + warp; j0 < j_end; j0 += kAttnWarps * 32) {
    int my_p = -1;
    if (kPaged) {
      const int j = j0 + kAttnWarps * lane;
      if (j < j_end) my_p = a.sel[(long long)bh * geo.k + j];
    }
    const int n_here = min(32, (j_end - j0 + kAttnWarps - 1) / kAttnWarps);
    for (int i = 0; i < n_here; ++i) {
      const int j = j0 + kAttnWarps * i;
      const uint16_t *Kp, *Vp;
      int valid;
      if (kPaged) {
        const int p = __shfl_sync(0xFFFFFFFFu, my_p, i);
        if (p < 0 || p >= P) {                      // corrupt selection: flag it and skip the page
          if (lane == 0) atomicOr(status, SWARM_DEV_BAD_PAGE);
          continue;
        }
        Kp = a.kv_pool + (((pool_row0 + p) * geo.Hkv + kvh) * 2) * blk;
        Vp = Kp + blk;
        valid = p == P - 1 ? tail : S;
      } else {
        Kp = a.k_g + ((long long)bh * geo.k + j) * blk;
        Vp = a.v_g + ((long long)bh * geo.k + j) * blk;
        valid = min(S, total_tok - j * S);
      }
#pragma unroll
      for (int sb = 0; sb < S / 16; ++sb) {
        const int v16 = min(16, valid - sb * 16);
        if (v16 > 0) attend_16(Kp + sb * 16 * kHeadDim, Vp + sb * 16 * kHeadDim, v16, qf, lane, st);
      }
    }
  }

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
  if (a.n_splits == 1) {
    a.out[(long long)bh * kHeadDim + t] = L > 0.f ? o / L : 0.f;
    if (t == 0) a.lse[bh] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
  } else {
    const long long slot = (long long)bh * a.n_splits + split;
    a.part_acc[slot * kHeadDim + t] = o;
    if (t == 0) { a.part_ml[slot * 2] = M; a.part_ml[slot * 2 + 1] = L; }
  }
}

// Merges the split partials of one (request, head): out = sum_s w_s acc_s / sum_s w_s l_s, w_s = 2^(m_s - M).
__global__ void __launch_bounds__(kHeadDim)
attn_combine_kernel(int n_splits, const float* __restrict__ part_acc, const float* __restrict__ part_ml,
                    float* __restrict__ out, float* __restrict__ lse) {
  const int bh = blockIdx.x, t = threadIdx.x;
  const float* ml = part_ml + (long long)bh * n_splits * 2;
  float M = -INFINITY;
  for (int s = 0; s < n_splits; ++s) M = fmaxf(M, ml[2 * s]);
  float L = 0.f, o = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const float sc = exp2_or_zero(ml[2 * s], M);
    L += ml[2 * s + 1] * sc;
    o += part_acc[((long long)bh * n_splits + s) * kHeadDim + t] * sc;
  }
  out[(long long)bh * kHeadDim + t] = L > 0.f ? o / L : 0.f;
  if (t == 0) lse[bh] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
}

}  // namespace

cudaError_t launch_attention(const Geometry& geo, const AttnArgs& a, uint32_t* status, cudaStream_t st) {
  const bool paged = a.kv_pool != nullptr;
  const unsigned grid = (unsigned)geo.B * geo.Hq * a.n_splits;
  const int threads = kAttnWarps * 32;
  if (geo.S == 16) {
    if (paged) attn_kernel<16, true><<<grid, threads, 0, st>>>(geo, a, status);
    else attn_kernel<16, false><<<grid, threads, 0, st>>>(geo, a, status);
  } else {
    if (paged) attn_kernel<32, true><<<grid, threads, 0, st>>>(geo, a, status);
    else attn_kernel<32, false><<<grid, threads, 0, st>>>(geo, a, status);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || a.n_splits == 1) return e;
  attn_combine_kernel<<<geo.B * geo.Hq, kHeadDim, 0, st>>>(a.n_splits, a.part_acc, a.part_ml, a.out, a.lse);
  return cudaGetLastError();
}

}  // namespace swarm

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of swarm_sparse_attn (see swarm.h).  The split-K partials live in a
// file-scope device array instead of a caller-provided workspace.  Layout of the array:
//   [0, 256)                       status word (unused by the contiguous-buffer kernel) + padding
//   [256, 256 + kSlots*128*4)      partial accumulators, one 128-float row per (head, split) slot
//   [.., .. + kSlots*2*4)          partial (max, sum) pairs
// Host code must not pass `g_static_scratch` itself to a kernel: on the host that name is only a
// handle.  Its device address is fetched once per device with cudaGetSymbolAddress.
namespace {
constexpr int kStaticSlots = 4096;
static_assert(SWARM_STATIC_SCRATCH_BYTES == 256 + kStaticSlots * (swarm::kHeadDim + 2) * 4, "header and array size differ");
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
  // same split heuristic as the ctx path (about 4 CTAs per SM, >= 4 pages per split), capped by the array
  long long n = (148 * 4 + bh - 1) / bh;
  n = n < (top_k / 4 > 1 ? top_k / 4 : 1) ? n : (top_k / 4 > 1 ? top_k / 4 : 1);
  n = n < kMaxSplits ? n : kMaxSplits;
  n = n < kStaticSlots / bh ? n : kStaticSlots / bh;
  n = n < 1 ? 1 : n;

  unsigned char* base = nullptr;
  if (static_scratch_address(&base) != cudaSuccess) return SWARM_ERR_CUDA;
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
  a.out = out;
  a.lse = lse;
  a.n_splits = (int)n;
  return launch_attention(geo, a, reinterpret_cast<uint32_t*>(base), static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? SWARM_OK : SWARM_ERR_CUDA;
}
