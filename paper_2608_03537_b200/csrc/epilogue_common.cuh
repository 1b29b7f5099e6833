// Pieces of the epilogue shared by the fused kernels: partial-statistic merges, the cross-thread / cross-CTA
// reduce phase of a stage (Sec. 3.1), and the bf16 row-chunk store.
#pragma once

#include "comfuse.h"
#include "sm100_primitives.cuh"

namespace comfuse {

// ------------------------------------------------------------------------------------------------ merges
// Partials are float2.  The functors merge `b` (nb elements) into `a` (na elements).
struct MergeWelford {  // (mean, M2); pairwise update of Chan et al.
  __device__ __forceinline__ float2 operator()(float2 a, float na, float2 b, float nb) const {
    const float n = na + nb;
    const float delta = b.x - a.x;
    return make_float2(fmaf(delta, nb / n, a.x), a.y + b.y + delta * delta * (na * nb / n));
  }
};
struct MergeSum {  // (sum, unused)
  __device__ __forceinline__ float2 operator()(float2 a, float, float2 b, float) const { return make_float2(a.x + b.x, 0.f); }
};
struct MergeMaxSumExp2 {  // (max, sum of 2^(t - max)); a partial with max = -inf carries nothing
  __device__ __forceinline__ float2 operator()(float2 a, float, float2 b, float) const {
    const float m = fmaxf(a.x, b.x);
    const float fa = (a.x == -INFINITY) ? 0.f : ex2_approx(a.x - m);
    const float fb = (b.x == -INFINITY) ? 0.f : ex2_approx(b.x - m);
    return make_float2(m, a.y * fa + b.y * fb);
  }
};
struct MergeByOp {  // (value, unused) under a run-time reduction operator: comfuse_op_t sum / mean / max / min / prod
  int op;
  __device__ __forceinline__ float2 operator()(float2 a, float, float2 b, float) const {
    float r;
    switch (op) {
      case COMFUSE_OP_RED_MAX: r = fmaxf(a.x, b.x); break;
      case COMFUSE_OP_RED_MIN: r = fminf(a.x, b.x); break;
      case COMFUSE_OP_RED_PROD: r = a.x * b.x; break;
      default: r = a.x + b.x; break;        // sum, mean
    }
    return make_float2(r, 0.f);
  }
};
struct MergeArgmax {  // (value, column index bits); ties -> lower index
  __device__ __forceinline__ float2 operator()(float2 a, float, float2 b, float) const {
    const int ia = __float_as_int(a.y), ib = __float_as_int(b.y);
    const bool take_b = (b.x > a.x) || (b.x == a.x && ib < ia);
    return take_b ? b : a;
  }
};

// The reduce phase above thread level.  All epilogue threads of every CTA that shares the rows call this the same
// number of times.  `per_thread_count` = elements behind each thread's partial (1/NH of the CTA's columns).
// `rank` is this CTA's index among the CN column ranges; the cluster rank of column range c is
// c * rank_stride + rank_offset (CTA pairs interleave two row blocks in one cluster).
// Exchanges alternate between two buffers AND two barriers (`stats_bar`, `stats_bar + 8`): a CTA that has passed
// exchange e may start sending exchange e + 1 while a slow peer's exchange-e message to some third CTA is still in
// flight; with one barrier that early message could complete the third CTA's phase e in place of the late one.
// `xpar` = buffer / barrier of the next exchange, `xphase` = one phase bit per barrier.
template <int CN, class Merge, int NH = 2>
__device__ __forceinline__ float2 cluster_row_reduce(float2 mine, float per_thread_count, Merge merge, float2* s_pre,
                                                     float2* s_stats, uint32_t stats_bar, int row, int h,
                                                     uint32_t rank, int& xpar, uint32_t& xphase, const WaitCtx& w,
                                                     uint32_t rank_stride = 1, uint32_t rank_offset = 0, bool leader_mode = false) {
  // level 2: the NH threads that share the row (one per epilogue warp of the lane quarter), through shared memory
  s_pre[(xpar * NH + h) * 128 + row] = mine;
  named_barrier_sync(1, 128 * NH);
  float2 cta_partial = s_pre[(xpar * NH + 0) * 128 + row];
#pragma unroll
  for (int t = 1; t < NH; ++t) cta_partial = merge(cta_partial, per_thread_count * t, s_pre[(xpar * NH + t) * 128 + row], per_thread_count);
  const float cta_count = static_cast<float>(NH) * per_thread_count;
  if constexpr (CN == 1) {
    // one CTA owns the whole row: the level-2 merge is already the result.  The next call uses the other level-2
    // buffer, and the one after that comes behind the next call's named barrier, which every reader of this one passes first.
    xpar ^= 1;
    return cta_partial;
  }
  // level 3: all-to-all over distributed shared memory; thread h serves the destination ranks congruent to h mod NH
  const uint32_t bar = stats_bar + 8u * xpar;
  const uint32_t phase = (xphase >> xpar) & 1u;
  float2* slot = s_stats + (xpar * CN + rank) * 128 + row;
  {
    // each partial travels as an asynchronous 8-byte store that is counted on the destination's barrier; one local
    // thread arms the barrier with the byte count of the whole exchange (CN peers x 128 rows x 8 bytes)
    const uint32_t slot_addr = smem_u32(slot);
    if (!leader_mode) {
      if (h == 0 && row == 0) mbar_arrive_expect_tx(bar, CN * 128 * 8);
#pragma unroll
      for (int dst = 0; dst < CN; ++dst) {
        if ((dst % NH) == h) {
          const uint32_t peer = dst * rank_stride + rank_offset;
          st_async_f32x2(map_to_cta(slot_addr, peer), cta_partial.x, cta_partial.y, map_to_cta(bar, peer));
        }
      }
      mbar_wait<true>(bar, phase, w);
    } else {
      // leader-follower aggregation (Sec. 3.1, the mode for large CN): every CTA sends its partial to column range 0
      // only (CN messages per row instead of CN^2); that CTA merges in the same rank order and sends the result back.
      // The followers' barrier counts the one returning message, the leader's the CN partials.
      const uint32_t lead = rank_offset;
      if (h == 0 && row == 0) mbar_arrive_expect_tx(bar, (rank == 0 ? CN : 1) * 128 * 8);
      if (h == 0) st_async_f32x2(map_to_cta(slot_addr, lead), cta_partial.x, cta_partial.y, map_to_cta(bar, lead));
      mbar_wait<true>(bar, phase, w);
      if (rank == 0) {
        float2 acc = s_stats[(xpar * CN + 0) * 128 + row];
#pragma unroll
        for (int c = 1; c < CN; ++c) acc = merge(acc, cta_count * c, s_stats[(xpar * CN + c) * 128 + row], cta_count);
        // slot 0 of every follower receives the merged value (thread h serves the followers congruent to h mod NH)
        const uint32_t res_addr = smem_u32(s_stats + (xpar * CN + 0) * 128 + row);
#pragma unroll
        for (int dst = 1; dst < CN; ++dst) {
          if ((dst % NH) == h) {
            const uint32_t peer = dst * rank_stride + rank_offset;
            st_async_f32x2(map_to_cta(res_addr, peer), acc.x, acc.y, map_to_cta(bar, peer));
          }
        }
        xphase ^= 1u << xpar;
        xpar ^= 1;
        __syncwarp();
        return acc;
      }
      const float2 acc = s_stats[(xpar * CN + 0) * 128 + row];
      xphase ^= 1u << xpar;
      xpar ^= 1;
      __syncwarp();
      return acc;
    }
  }
  float2 acc = s_stats[(xpar * CN + 0) * 128 + row];
#pragma unroll
  for (int c = 1; c < CN; ++c) acc = merge(acc, cta_count * c, s_stats[(xpar * CN + c) * 128 + row], cta_count);
  xphase ^= 1u << xpar;
  xpar ^= 1;
  __syncwarp();
  return acc;
}

// 32 consecutive values of one row of an additive mask (bf16, the segment starts on a 16-byte boundary), as log2-domain
// addends: m * log2(e); -inf stays -inf.  `valid` = how many of the 32 columns exist (the rest, and every column of a row
// that does not exist, read as 0: those scores are dropped by the caller's own bounds).
__device__ __forceinline__ void load_mask_log2_32(const uint16_t* seg, int valid, float2 (&m2)[16]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint4 q = make_uint4(0u, 0u, 0u, 0u);
    if (8 * i < valid) q = __ldg(reinterpret_cast<const uint4*>(seg) + i);
    const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) m2[4 * i + k] = mul2(bf16x2_to_f2(w4[k]), splat2(1.4426950408889634f));
  }
}

__device__ __forceinline__ void store_chunk_bf16(uint16_t* dst, const uint32_t (&pk)[16]) {
  uint4* d = reinterpret_cast<uint4*>(dst);
#pragma unroll
  for (int i = 0; i < 4; ++i) d[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
}

}  // namespace comfuse
