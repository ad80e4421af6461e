// What the two attention kernels share (the one-item-per-CTA kernel and the streaming kernel whose CTAs work
// through many items): constants of the per-warp copy ring, the TMA / mbarrier / MMA primitives, the arithmetic
// of one 16-token unit, and the split-K hand-over of a finished head.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>

#include "swarm_internal.cuh"

namespace swarm {
namespace attn_detail {

// The rings fill the SM's shared memory (24 slots of 8 KiB).  What a warp can stream is bounded by the length of
// a unit's dependent chain (~1000 cycles, of which 32 MMAs at one per ~16 cycles and SM sub-partition), not by its
// copies, so more warps with shallower rings do better than fewer with deeper ones: 12 x 2 against 8 x 3 measured
// 57.9 against 59.4 us (16 requests x 32K tokens), 143 against 146 us (4 x 512K), 182 against 187 us (64 ragged).
constexpr int kAttnWarps = 12;
constexpr int kStages = 2;
constexpr int kUnitTokens = 16;
constexpr int kBoxBytes = kUnitTokens * 128;                       // 16 token rows x 64 bf16
constexpr int kSlotBytes = 4 * kBoxBytes;                          // K lo, K hi, V lo, V hi
constexpr int kRingBytes = kAttnWarps * kStages * kSlotBytes;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr unsigned kWaitLimit = 1u << 22;                          // polls of a try_wait that itself blocks briefly

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
// Tiled TMA load of token rows.  The tensor of rows x 128 coordinates is described as (64 coordinates, row, half):
// the two halves of the 128 coordinates are a third dimension 128 bytes apart, so one copy brings a box of both
// -- in shared memory half 0 of all the box's rows, then half 1, each 128-byte line swizzled by its row.  The pages
// are read once per step: `policy` (evict-first) keeps them from pushing the small tables, the workspace and the
// kernels' own instructions out of L2.
__device__ __forceinline__ void tma_load_rows(uint32_t dst, const CUtensorMap* map, int row, uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(dst),
      "l"(map), "r"(0), "r"(row), "r"(0), "r"(smem_addr(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t evict_first_policy() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float exp2_or_zero(float x, float ref) {   // 2^(x-ref), 0 when x = -inf
  return x == -INFINITY ? 0.f : exp2f(x - ref);
}
// p -> (bf16 high part, bf16 low part) of two values, packed for the MMA's B operand
__device__ __forceinline__ void split_pack(float p0, float p1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat16 h0 = __float2bfloat16_rn(p0), h1 = __float2bfloat16_rn(p1);
  const __nv_bfloat16 l0 = __float2bfloat16_rn(p0 - __bfloat162float(h0)), l1 = __float2bfloat16_rn(p1 - __bfloat162float(h1));
  hi = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
}
// byte offset of 16-byte chunk `chunk` (0..15, 8 coordinates each) of token row `t` inside a K or V tile
// (two 2 KiB boxes of 64 coordinates, each with the 128-byte swizzle)
// `half` = bytes between the box of coordinates 0-63 and the box of coordinates 64-127
__device__ __forceinline__ uint32_t tile_offset(int t, int chunk, int half) {
  return (uint32_t)((chunk >> 3) * half + t * 128 + (((chunk & 7) ^ (t & 7)) << 4));
}


// One 16-token unit of K and V, already in the warp's ring slot, folded into the warp's running softmax state.
// `v16` (1..16) tokens of the unit exist; `head_on`: this lane's head (row `quad` of the score MMA) takes part in
// the unit's page.  kHalf: bytes between the two coordinate halves of a tile, kVOff: V tile relative to the K tile.
//   qa     Q as the A operand of S^T = Q K^T (row = head, 8 k-steps of 16 coordinates)
//   m_run, l_run   running (max, sum) of head `quad` over this lane's token columns, logits in the log2 domain
//   acc    O^T: rows = coordinates 16*mt + quad (+8), columns = heads 2*tq (+1)
template <int kHalf, int kVOff>
__device__ __forceinline__ void attend_unit(unsigned char* slot, int v16, bool head_on, int lane, const uint32_t (&qa)[8][2],
                                            float scale, float& m_run, float& l_run, float (&acc)[8][4]) {
  const int tq = lane & 3;
  const uint32_t kt = smem_addr(slot), vt = kt + kVOff;
  if (v16 < kUnitTokens) {
    // padding tokens: their V rows may hold anything, and 0 * NaN must not reach the accumulators
    unsigned char* vrows = slot + kVOff;
    for (int i = lane; i < (kUnitTokens - v16) * 16; i += 32) {
      const int t = v16 + (i >> 4), ch = i & 15;
      *reinterpret_cast<uint4*>(vrows + tile_offset(t, ch, kHalf)) = make_uint4(0, 0, 0, 0);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // ordered before the slot's next TMA fill
    __syncwarp();
  }
  // S^T[head][token] = Q K^T : 2 token tiles x 8 k-steps
  float sacc[2][4];
#pragma unroll
  for (int nt = 0; nt < 2; ++nt)
#pragma unroll
    for (int e = 0; e < 4; ++e) sacc[nt][e] = 0.f;
#pragma unroll
  for (int s4 = 0; s4 < 4; ++s4) {
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      uint32_t r[4];
      ldmatrix_x4(r, kt + tile_offset(8 * nt + (lane & 7), 4 * s4 + (lane >> 3), kHalf));
      mma_bf16(sacc[nt], qa[2 * s4][0], 0u, qa[2 * s4][1], 0u, r[0], r[1]);
      mma_bf16(sacc[nt], qa[2 * s4 + 1][0], 0u, qa[2 * s4 + 1][1], 0u, r[2], r[3]);
    }
  }
  // softmax of head `quad` over this lane's tokens 2*tq, 2*tq+1, 8+2*tq, 8+2*tq+1
  float x[4] = {sacc[0][0] * scale, sacc[0][1] * scale, sacc[1][0] * scale, sacc[1][1] * scale};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int t = (e >> 1) * 8 + 2 * tq + (e & 1);
    if (!head_on || t >= v16) x[e] = -INFINITY;
  }
  float mx = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
  mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
  mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
  const float m_new = fmaxf(m_run, mx);
  const float corr = m_new == -INFINITY ? 1.f : exp2_or_zero(m_run, m_new);
  float p[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) p[e] = exp2_or_zero(x[e], m_new);
  l_run = l_run * corr + (p[0] + p[1]) + (p[2] + p[3]);
  m_run = m_new;
  uint32_t b0h, b0l, b1h, b1l;
  split_pack(p[0], p[1], b0h, b0l);
  split_pack(p[2], p[3], b1h, b1l);
  // rescale the outputs of heads 2*tq and 2*tq+1 (their factors live in quads 2*tq and 2*tq+1)
  const float c0 = __shfl_sync(0xFFFFFFFFu, corr, 8 * tq), c1 = __shfl_sync(0xFFFFFFFFu, corr, 8 * tq + 4);
  if (__any_sync(0xFFFFFFFFu, corr != 1.f)) {
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      acc[mt][0] *= c0; acc[mt][1] *= c1; acc[mt][2] *= c0; acc[mt][3] *= c1;
    }
  }
  // O^T[coordinate][head] += V^T P^T : 8 tiles of 16 coordinates, P as high + low bf16 parts
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    uint32_t r[4];
    ldmatrix_x4_trans(r, vt + tile_offset(((lane >> 4) & 1) * 8 + (lane & 7), 2 * mt + ((lane >> 3) & 1), kHalf));
    mma_bf16(acc[mt], r[0], r[1], r[2], r[3], b0h, b1h);
    mma_bf16(acc[mt], r[0], r[1], r[2], r[3], b0l, b1l);
  }
}

// A warp holds one head's result over its CTA's page range: (M, L) and four coordinates per lane in `o`, all on
// the scale of M.  With one split that is the head's result; otherwise the warp publishes the partial, and the
// warp that arrives last at the head's ticket (whichever CTA it sits in) merges the head's partials -- the heads
// of a group are thus merged side by side, and nothing waits for a CTA-wide barrier or a staging copy.  The
// finishing warp writes out / lse (and their host mirrors, counting the head as arrived there).
// `n_splits`: page ranges of this head's group; `slot_stride`: partial slots per head (the launch's largest count).
__device__ __forceinline__ void finish_head(const AttnArgs& a, long long bh, int split, int n_splits, int slot_stride,
                                            int lane, float M, float L, float4 o) {
  bool finish = true;                                   // this warp writes the head's final result
  if (n_splits > 1) {
    const long long slot = bh * slot_stride + split;
    __stcg(reinterpret_cast<float4*>(a.part_acc + slot * kHeadDim) + lane, o);
    if (lane == 0) __stcg(reinterpret_cast<float2*>(a.part_ml + slot * 2), make_float2(M, L));
    __syncwarp();                                       // the lanes' stores are ordered before lane 0's release
    unsigned prev = 0u;
    if (lane == 0) prev = atom_acq_rel_add(a.tickets + bh, 1u);
    prev = __shfl_sync(0xFFFFFFFFu, prev, 0);
    __syncwarp();                                       // lane 0's acquire is ordered before the other lanes' loads
    finish = prev == (unsigned)n_splits - 1u;
    if (finish) {
      // every lane sums its 4 coordinates over the splits, weighted to their common scale: (max, sum) of split
      // `lane` and `lane + 32` give the weights.  The first sixteen rows are asked for together with them, so that
      // the merge of up to 16 splits is one trip to L2.
      const float4* rows = reinterpret_cast<const float4*>(a.part_acc + bh * slot_stride * kHeadDim) + lane;
      float4 v[16];
#pragma unroll
      for (int u = 0; u < 16; ++u) v[u] = u < n_splits ? __ldcg(rows + u * (kHeadDim / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
      const float2 ml0 = lane < n_splits ? __ldcg(reinterpret_cast<const float2*>(a.part_ml + (bh * slot_stride + lane) * 2))
                                           : make_float2(-INFINITY, 0.f);
      const float2 ml1 = lane + 32 < n_splits
                             ? __ldcg(reinterpret_cast<const float2*>(a.part_ml + (bh * slot_stride + lane + 32) * 2))
                             : make_float2(-INFINITY, 0.f);
      M = fmaxf(ml0.x, ml1.x);
#pragma unroll
      for (int o2 = 16; o2 >= 1; o2 >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, o2));
      const float w0 = exp2_or_zero(ml0.x, M), w1 = exp2_or_zero(ml1.x, M);
      L = ml0.y * w0 + ml1.y * w1;
#pragma unroll
      for (int o2 = 16; o2 >= 1; o2 >>= 1) L += __shfl_xor_sync(0xFFFFFFFFu, L, o2);
      o = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int sp0 = 0; sp0 < n_splits; sp0 += 16) {
        if (sp0 > 0) {
#pragma unroll
          for (int u = 0; u < 16; ++u)                  // sixteen rows in flight together
            v[u] = sp0 + u < n_splits ? __ldcg(rows + (sp0 + u) * (kHeadDim / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          const int sp = sp0 + u;
          const float ws = __shfl_sync(0xFFFFFFFFu, sp < 32 ? w0 : w1, sp & 31);
          o.x = fmaf(v[u].x, ws, o.x); o.y = fmaf(v[u].y, ws, o.y); o.z = fmaf(v[u].z, ws, o.z); o.w = fmaf(v[u].w, ws, o.w);
        }
      }
      if (lane == 0) a.tickets[bh] = 0u;                // ready for the next launch
    }
  }
  if (finish) {
    const float inv = L > 0.f ? 1.f / L : 0.f;
    const float4 res = make_float4(o.x * inv, o.y * inv, o.z * inv, o.w * inv);
    const float lse_h = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
    reinterpret_cast<float4*>(a.out + bh * kHeadDim)[lane] = res;
    if (lane == 0) a.lse[bh] = lse_h;
    if (a.host.out_h != nullptr) reinterpret_cast<float4*>(a.host.out_h + bh * kHeadDim)[lane] = res;
    if (a.host.lse_h != nullptr && lane == 0) a.host.lse_h[bh] = lse_h;
    if (a.host.done_h != nullptr) {                     // host step: this head's results are in host memory
      __syncwarp();
      if (lane == 0) host_arrive(a.host);
    }
  }
}

}  // namespace attn_detail
}  // namespace swarm
