// GEMM -> row-reduction subgraph, one kernel (Stage-Stream Execution Model, Sec. 3).
//
// Work decomposition (Sec. 3.1, cluster-granular scheduling): a work item is one 128-row block of the
// output; the CN CTAs of a thread-block cluster own CN adjacent column ranges of that row block, so every
// last-dim reduction is confined to one cluster (Sec. 3, Eq. 1).  Each CTA keeps its whole 128 x BN fp32
// accumulator in tensor memory as NSUB sub-tiles of BNS columns; clusters are persistent and walk the row
// blocks with a stride of the cluster count.
//
// Warp roles inside a CTA (10 warps):
//   warp 0      TMA producer: A (K-major) and B (N-contiguous, "MN-major") tiles into an NSTAGES ring.
//   warp 1      MMA issuer: tcgen05.mma from the ring into the sub-tile's TMEM columns; owns TMEM alloc.
//   warps 2-9   epilogue: thread (q, lane) owns output row 32q+lane (TMEM lane), the two warps that share a
//               lane quarter split the 32-column chunks of every sub-tile between them.
// Sub-tile s+1's MainLoop runs while the epilogue works on sub-tile s, and the next row block's MainLoop
// starts as soon as stage 2 has drained a sub-tile (the PingPong schedule of Sec. 3.3 at sub-tile grain).
//
// Epilogue stages (Sec. 3.1 / 3.2):
//   stage 1  compute : x = f(alpha*Acc, bias, residual, ...) per 32-column fragment, thread-local partial
//                      statistic; x is written back over the accumulator in TMEM (the bypass path).
//            reduce  : the two column-halves of a row merge through shared memory, then every CTA writes its
//                      partial into every peer's shared memory (all-to-all over DSMEM) and arrives on the
//                      peer's mbarrier; each CTA finishes the merge locally in rank order (deterministic).
//   stage 2  PostOp  : normalise the still-resident x, round to bf16 once, store.
//   stage 3  (RMSNorm+max only) a second reduction (row max / argmax) through the same exchange buffers.
#pragma once

#include "epilogue_common.cuh"
#include "fused_params.h"
#include "sm100_primitives.cuh"

namespace comfuse {

template <int EPI, int BNS, int NSUB, int CN, int NSTAGES>
struct FusedCfg {
  static constexpr int kThreads = 320;
  static constexpr int kEpiThreads = 256;
  static constexpr int BN = BNS * NSUB;
  static constexpr int A_BYTES = 128 * 64 * 2;
  static constexpr int B_BYTES = BNS * 64 * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = BN <= 32 ? 32 : BN <= 64 ? 64 : BN <= 128 ? 128 : BN <= 256 ? 256 : 512;
  static constexpr int OFF_VEC = NSTAGES * STAGE_BYTES;
  static constexpr int VEC_BYTES = 3 * BN * 4;
  static constexpr int OFF_STATS = OFF_VEC + VEC_BYTES;
  static constexpr int STATS_BYTES = 2 * CN * 128 * 8;
  static constexpr int OFF_PRE = OFF_STATS + STATS_BYTES;
  static constexpr int PRE_BYTES = 2 * 2 * 128 * 8;
  static constexpr int OFF_BAR = OFF_PRE + PRE_BYTES;
  static constexpr int NUM_BARS = 2 * NSTAGES + 2 * NSUB + 2;
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;
  static constexpr int SMEM_BYTES = OFF_MISC + 16 + 1024;  // + slack to align the base to 1024 bytes
  static_assert(BNS % 64 == 0 && BNS <= 256, "sub-tile width: multiple of 64, at most one UMMA N");
  static_assert(BN <= 512, "accumulator must fit the 512 TMEM columns");
  static_assert((BNS / 32) % 2 == 0, "two epilogue warps split the 32-column chunks evenly");
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

// ------------------------------------------------------------------------------------------------ kernel
template <int EPI, int BNS, int NSUB, int CN, int NSTAGES>
__global__ void __launch_bounds__(320, 1)
fused_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const FusedParams p) {
  using Cfg = FusedCfg<EPI, BNS, NSUB, CN, NSTAGES>;
  constexpr int BN = Cfg::BN;
  constexpr int CHUNKS = BNS / 32;  // 32-column fragments per sub-tile

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t smem_base = smem_u32(smem);

  float* s_bias = reinterpret_cast<float*>(smem + Cfg::OFF_VEC);
  float* s_gamma = s_bias + BN;
  float* s_beta = s_gamma + BN;
  float2* s_stats = reinterpret_cast<float2*>(smem + Cfg::OFF_STATS);
  float2* s_pre = reinterpret_cast<float2*>(smem + Cfg::OFF_PRE);
  const uint32_t bar_base = smem_base + Cfg::OFF_BAR;
  auto bar_full = [&](int s) { return bar_base + 8u * s; };
  auto bar_empty = [&](int s) { return bar_base + 8u * (NSTAGES + s); };
  auto bar_tfull = [&](int s) { return bar_base + 8u * (2 * NSTAGES + s); };
  auto bar_tempty = [&](int s) { return bar_base + 8u * (2 * NSTAGES + NSUB + s); };
  const uint32_t bar_stats = bar_base + 8u * (2 * NSTAGES + 2 * NSUB);
  const uint32_t bar_drain = bar_stats + 8u;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(smem + Cfg::OFF_MISC);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + Cfg::OFF_MISC + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = (CN > 1) ? cluster_ctarank() : 0u;
  const int cluster_id = blockIdx.x / CN;
  const int num_clusters = gridDim.x / CN;
  const int KB = (p.K + 63) >> 6;
  const WaitCtx w{s_abort, p.status, p.timeout_ns};

  // -------------------------------------------------------------------------------------------- set-up
  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGES; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), 1);
    }
    for (int s = 0; s < NSUB; ++s) {
      mbar_init(bar_tfull(s), 1);
      mbar_init(bar_tempty(s), Cfg::kEpiThreads);
    }
    mbar_init(bar_stats, CN * 128);
    mbar_init(bar_drain, 1);
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(s_tmem_base), Cfg::TMEM_COLS);
    tmem_relinquish_alloc_permit();
  }
  if constexpr (EPI == EPI_LN || EPI == EPI_RMS_MAX) {
    // row-vector broadcasts (Sec. 5.2: 1-D parameters) of this CTA's columns, widened to fp32 once
    const int c0 = rank * BN;
    for (int i = threadIdx.x; i < BN; i += Cfg::kThreads) {
      const int c = c0 + i;
      const bool in = c < p.N;
      s_bias[i] = (p.bias && in) ? bf16_lo(p.bias[c]) : 0.f;
      s_gamma[i] = (p.gamma && in) ? bf16_lo(p.gamma[c]) : 1.f;
      s_beta[i] = (p.beta && in) ? bf16_lo(p.beta[c]) : 0.f;
    }
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  if constexpr (CN > 1) cluster_sync_all();  // peers' barriers exist before anyone arrives on them
  const uint32_t tmem_base = *s_tmem_base;

  auto decode_tile = [&](int tile, int& b, int& m0, int& ncta0) {
    const int per_batch = p.mblocks * p.nblocks;
    b = tile / per_batch;
    const int rem = tile - b * per_batch;
    const int mb = rem / p.nblocks;
    const int nb = rem - mb * p.nblocks;
    m0 = mb * 128;
    ncta0 = (nb * CN + static_cast<int>(rank)) * BN;
  };
  // A sub-tile that the causal mask removes entirely is never loaded or multiplied.
  auto subtile_masked = [&](int m0, int n0) { return EPI == EPI_SOFTMAX && p.causal && n0 > m0 + 127; };
  // EPI_NONE walks column blocks; a sub-tile completely past N is skipped as well.
  auto subtile_skipped = [&](int m0, int n0) { return subtile_masked(m0, n0) || n0 >= p.N; };

  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < p.total_tiles && ok; tile += num_clusters) {
        int b, m0, ncta0;
        decode_tile(tile, b, m0, ncta0);
        for (int sub = 0; sub < NSUB && ok; ++sub) {
          const int n0 = ncta0 + sub * BNS;
          if (subtile_skipped(m0, n0)) continue;
          for (int kb = 0; kb < KB; ++kb) {
            if (!mbar_wait<false>(bar_empty(stage), phase ^ 1u, w)) { ok = false; break; }
            const uint32_t sa = smem_base + stage * Cfg::STAGE_BYTES;
            const uint32_t sb = sa + Cfg::A_BYTES;
            mbar_arrive_expect_tx(bar_full(stage), Cfg::STAGE_BYTES);
            tma_load_3d(sa, &tmA, bar_full(stage), kb * 64, m0, b);
#pragma unroll
            for (int j = 0; j < BNS / 64; ++j) tma_load_3d(sb + j * 8192, &tmB, bar_full(stage), n0 + j * 64, kb * 64, b);
            if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(128, BNS, /*a_mn_major=*/false, /*b_mn_major=*/true);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t te_phase[NSUB];
#pragma unroll
      for (int s = 0; s < NSUB; ++s) te_phase[s] = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < p.total_tiles && ok; tile += num_clusters) {
        int b, m0, ncta0;
        decode_tile(tile, b, m0, ncta0);
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
          const int n0 = ncta0 + sub * BNS;
          if (!ok || subtile_skipped(m0, n0)) continue;
          if (!mbar_wait<false>(bar_tempty(sub), te_phase[sub] ^ 1u, w)) { ok = false; continue; }
          te_phase[sub] ^= 1u;
          tcgen05_fence_after_sync();
          const uint32_t d_tmem = tmem_base + sub * BNS;
          for (int kb = 0; kb < KB; ++kb) {
            if (!mbar_wait<false>(bar_full(stage), phase, w)) { ok = false; break; }
            tcgen05_fence_after_sync();
            const uint32_t sa = smem_base + stage * Cfg::STAGE_BYTES;
            const uint32_t sb = sa + Cfg::A_BYTES;
            const uint64_t adesc = make_smem_desc_sw128(sa, 16, 1024);
            const uint64_t bdesc = make_smem_desc_sw128(sb, /*lbo: next 64-column block*/ 8192, /*sbo: next 8 K rows*/ 1024);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              // K advances by 16 elements: 32 bytes inside A's swizzled row, 16 K-lines (2048 bytes) in B
              umma_bf16_ss(d_tmem, adesc + static_cast<uint64_t>(k * 2), bdesc + static_cast<uint64_t>(k * 128), idesc,
                           (kb | k) != 0 ? 1u : 0u);
            }
            umma_commit(bar_empty(stage));
            if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
          }
          if (ok) umma_commit(bar_tfull(sub));
        }
      }
      // Everything issued must have retired before TMEM is freed, also on the early-exit path.
      umma_commit(bar_drain);
      mbar_wait<false>(bar_drain, 0, w);
    }
  } else {
    // ------------------------------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;         // TMEM lane quarter this warp may touch
    const int h = (warp - 2) >> 2;  // which half of the 32-column chunks
    const int row = q * 32 + lane;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    uint32_t tf_phase[NSUB];
#pragma unroll
    for (int s = 0; s < NSUB; ++s) tf_phase[s] = 0;
    int xpar = 0;
    uint32_t xphase = 0;
    (void)xpar; (void)xphase; (void)s_pre; (void)s_stats; (void)s_bias; (void)s_gamma; (void)s_beta;
    constexpr float kThreadCount = static_cast<float>(BN / 2);  // columns behind one thread's partial

    for (int tile = cluster_id; tile < p.total_tiles; tile += num_clusters) {
      int b, m0, ncta0;
      decode_tile(tile, b, m0, ncta0);
      const int grow = m0 + row;
      const bool valid = grow < p.M;
      uint16_t* yrow = p.Y + static_cast<long long>(b) * p.batch_stride_y + static_cast<long long>(grow) * p.ldy;
      const uint16_t* rrow =
          p.residual ? p.residual + static_cast<long long>(b) * p.batch_stride_r + static_cast<long long>(grow) * p.ldr
                     : nullptr;

      if constexpr (EPI == EPI_NONE) {
        // plain GEMM: Z = bf16(Acc), used by the unfused path
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
          const int n0 = ncta0 + sub * BNS;
          if (subtile_skipped(m0, n0)) continue;
          mbar_wait<false>(bar_tfull(sub), tf_phase[sub], w);
          tf_phase[sub] ^= 1u;
          __syncwarp();
          tcgen05_fence_after_sync();
#pragma unroll
          for (int c = 0; c < CHUNKS / 2; ++c) {
            const int lc = sub * BNS + (2 * c + h) * 32;
            uint32_t v[32];
            tmem_ld_32cols(lane_base + lc, v);
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
            const int col = ncta0 + lc;
            if (valid) {
              if (col + 32 <= p.N) {
                store_chunk_bf16(yrow + col, pk);
              } else {
#pragma unroll
                for (int g = 0; g < 4; ++g)
                  if (col + 8 * g + 8 <= p.N)
                    *reinterpret_cast<uint4*>(yrow + col + 8 * g) = make_uint4(pk[4 * g], pk[4 * g + 1], pk[4 * g + 2], pk[4 * g + 3]);
              }
            }
          }
          tcgen05_fence_before_sync();
          mbar_arrive(bar_tempty(sub));
        }
      } else if constexpr (EPI == EPI_LN) {
        // ---------------- stage 1: x = alpha*Acc + bias + R ; thread-local (mean, M2)
        float2 part = make_float2(0.f, 0.f);
        float n_run = 0.f;
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
          mbar_wait<false>(bar_tfull(sub), tf_phase[sub], w);
          tf_phase[sub] ^= 1u;
          __syncwarp();
          tcgen05_fence_after_sync();
#pragma unroll
          for (int c = 0; c < CHUNKS / 2; ++c) {
            const int lc = sub * BNS + (2 * c + h) * 32;
            uint32_t v[32];
            tmem_ld_32cols(lane_base + lc, v);
            uint4 rr[4];
#pragma unroll
            for (int g = 0; g < 4; ++g)
              rr[g] = (valid && rrow) ? __ldg(reinterpret_cast<const uint4*>(rrow + ncta0 + lc) + g) : make_uint4(0, 0, 0, 0);
            const uint32_t* r32 = reinterpret_cast<const uint32_t*>(rr);
            float sum = 0.f;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float x0 = fmaf(p.alpha, __uint_as_float(v[2 * j]), s_bias[lc + 2 * j]) + bf16_lo(r32[j]);
              const float x1 = fmaf(p.alpha, __uint_as_float(v[2 * j + 1]), s_bias[lc + 2 * j + 1]) + bf16_hi(r32[j]);
              v[2 * j] = __float_as_uint(x0);
              v[2 * j + 1] = __float_as_uint(x1);
              sum += x0 + x1;
            }
            const float cmean = sum * (1.f / 32.f);
            float cm2 = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float d = __uint_as_float(v[j]) - cmean;
              cm2 = fmaf(d, d, cm2);
            }
            part = (n_run == 0.f) ? make_float2(cmean, cm2) : MergeWelford()(part, n_run, make_float2(cmean, cm2), 32.f);
            n_run += 32.f;
            tmem_st_32cols(lane_base + lc, v);  // bypass path: x stays resident for stage 2
          }
        }
        tmem_st_wait();
        // ---------------- reduce across the thread pair and the cluster
        const float2 tot = cluster_row_reduce<CN>(part, kThreadCount, MergeWelford(), s_pre, s_stats, bar_stats, row, h,
                                                  rank, xpar, xphase, w);
        const float mu = tot.x;
        const float rstd = rsqrtf(tot.y * (1.f / static_cast<float>(CN * BN)) + p.eps);
        // ---------------- stage 2: (x - mean) * rstd * gamma + beta, round once, store
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
#pragma unroll
          for (int c = 0; c < CHUNKS / 2; ++c) {
            const int lc = sub * BNS + (2 * c + h) * 32;
            uint32_t v[32];
            tmem_ld_32cols(lane_base + lc, v);
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float y0 = fmaf((__uint_as_float(v[2 * j]) - mu) * rstd, s_gamma[lc + 2 * j], s_beta[lc + 2 * j]);
              const float y1 = fmaf((__uint_as_float(v[2 * j + 1]) - mu) * rstd, s_gamma[lc + 2 * j + 1], s_beta[lc + 2 * j + 1]);
              pk[j] = pack_bf16x2_rn(y0, y1);
            }
            if (valid) store_chunk_bf16(yrow + ncta0 + lc, pk);
          }
          tcgen05_fence_before_sync();
          mbar_arrive(bar_tempty(sub));
        }
      } else if constexpr (EPI == EPI_RMS_MAX) {
        // ---------------- stage 1: H = GELU(alpha*Acc + bias) + R ; thread-local sum of squares
        float ss = 0.f;
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
          mbar_wait<false>(bar_tfull(sub), tf_phase[sub], w);
          tf_phase[sub] ^= 1u;
          __syncwarp();
          tcgen05_fence_after_sync();
#pragma unroll
          for (int c = 0; c < CHUNKS / 2; ++c) {
            const int lc = sub * BNS + (2 * c + h) * 32;
            uint32_t v[32];
            tmem_ld_32cols(lane_base + lc, v);
            uint4 rr[4];
#pragma unroll
            for (int g = 0; g < 4; ++g)
              rr[g] = (valid && rrow) ? __ldg(reinterpret_cast<const uint4*>(rrow + ncta0 + lc) + g) : make_uint4(0, 0, 0, 0);
            const uint32_t* r32 = reinterpret_cast<const uint32_t*>(rr);
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float z0 = fmaf(p.alpha, __uint_as_float(v[2 * j]), s_bias[lc + 2 * j]);
              const float z1 = fmaf(p.alpha, __uint_as_float(v[2 * j + 1]), s_bias[lc + 2 * j + 1]);
              const float h0 = gelu_tanh_f32(z0) + bf16_lo(r32[j]);
              const float h1 = gelu_tanh_f32(z1) + bf16_hi(r32[j]);
              v[2 * j] = __float_as_uint(h0);
              v[2 * j + 1] = __float_as_uint(h1);
              s0 = fmaf(h0, h0, s0);
              s1 = fmaf(h1, h1, s1);
            }
            ss += s0 + s1;
            tmem_st_32cols(lane_base + lc, v);
          }
        }
        tmem_st_wait();
        const float2 tot = cluster_row_reduce<CN>(make_float2(ss, 0.f), kThreadCount, MergeSum(), s_pre, s_stats, bar_stats,
                                                  row, h, rank, xpar, xphase, w);
        const float rstd = rsqrtf(tot.x * (1.f / static_cast<float>(CN * BN)) + p.eps);
        // ---------------- stage 2: Y = H * rstd * g ; thread-local (max, argmax) of the unrounded Y
        float best = -INFINITY;
        int best_col = 0x7FFFFFFF;
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
#pragma unroll
          for (int c = 0; c < CHUNKS / 2; ++c) {
            const int lc = sub * BNS + (2 * c + h) * 32;
            uint32_t v[32];
            tmem_ld_32cols(lane_base + lc, v);
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float y0 = __uint_as_float(v[2 * j]) * rstd * s_gamma[lc + 2 * j];
              const float y1 = __uint_as_float(v[2 * j + 1]) * rstd * s_gamma[lc + 2 * j + 1];
              if (y0 > best) { best = y0; best_col = ncta0 + lc + 2 * j; }
              if (y1 > best) { best = y1; best_col = ncta0 + lc + 2 * j + 1; }
              pk[j] = pack_bf16x2_rn(y0, y1);
            }
            if (valid) store_chunk_bf16(yrow + ncta0 + lc, pk);
          }
          tcgen05_fence_before_sync();
          mbar_arrive(bar_tempty(sub));
        }
        // ---------------- stage 3: second chained reduction, same exchange buffers (Sec. 3.2)
        const float2 mx = cluster_row_reduce<CN>(make_float2(best, __int_as_float(best_col)), kThreadCount, MergeArgmax(),
                                                 s_pre, s_stats, bar_stats, row, h, rank, xpar, xphase, w);
        if (rank == 0 && h == 0 && valid) {
          const long long o = static_cast<long long>(b) * p.M + grow;
          p.row_max[o] = mx.x;
          p.row_argmax[o] = __float_as_int(mx.y);
        }
      } else {  // EPI_SOFTMAX
        // Scores are handled in the log2 domain: t = Acc * (alpha * log2 e), so exp(x - m) = 2^(t - m_t).
        const float sc = p.alpha * 1.4426950408889634f;
        // chunk classification under the causal mask, uniform over the warp's 32 rows so that the warp-wide
        // TMEM loads stay convergent: 2 = all live, 1 = crosses the diagonal, 0 = all masked
        const int wrow0 = m0 + q * 32;
        auto chunk_state = [&](int col0) { return !p.causal ? 2 : (col0 + 31 <= wrow0 ? 2 : (col0 > wrow0 + 31 ? 0 : 1)); };
        // ---------------- pass A: thread-local row max
        float mloc = -INFINITY;
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
          const int n0 = ncta0 + sub * BNS;
          if (subtile_masked(m0, n0)) continue;
          mbar_wait<false>(bar_tfull(sub), tf_phase[sub], w);
          tf_phase[sub] ^= 1u;
          __syncwarp();
          tcgen05_fence_after_sync();
#pragma unroll
          for (int c = 0; c < CHUNKS / 2; ++c) {
            const int lc = sub * BNS + (2 * c + h) * 32;
            const int st = chunk_state(ncta0 + lc);
            if (st == 0) continue;
            uint32_t v[32];
            tmem_ld_32cols(lane_base + lc, v);
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float t = __uint_as_float(v[j]) * sc;
              if (st == 2 || ncta0 + lc + j <= grow) mloc = fmaxf(mloc, t);
            }
          }
        }
        // ---------------- pass B: e = 2^(t - mloc), thread-local sum, e written back over the scores
        float lloc = 0.f;
        const float msub = (mloc == -INFINITY) ? 0.f : mloc;
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
          const int n0 = ncta0 + sub * BNS;
          if (subtile_masked(m0, n0)) continue;
#pragma unroll
          for (int c = 0; c < CHUNKS / 2; ++c) {
            const int lc = sub * BNS + (2 * c + h) * 32;
            const int st = chunk_state(ncta0 + lc);
            if (st == 0) continue;
            uint32_t v[32];
            tmem_ld_32cols(lane_base + lc, v);
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              float e0 = ex2_approx(fmaf(__uint_as_float(v[j]), sc, -msub));
              float e1 = ex2_approx(fmaf(__uint_as_float(v[j + 1]), sc, -msub));
              if (st != 2) {
                if (ncta0 + lc + j > grow) e0 = 0.f;
                if (ncta0 + lc + j + 1 > grow) e1 = 0.f;
              }
              v[j] = __float_as_uint(e0);
              v[j + 1] = __float_as_uint(e1);
              s0 += e0;
              s1 += e1;
            }
            lloc += s0 + s1;
            tmem_st_32cols(lane_base + lc, v);
          }
        }
        tmem_st_wait();
        const float2 tot = cluster_row_reduce<CN>(make_float2(mloc, lloc), kThreadCount, MergeMaxSumExp2(), s_pre, s_stats,
                                                  bar_stats, row, h, rank, xpar, xphase, w);
        // p = e * 2^(mloc - m) / l ; a row with nothing live is a row of zeros
        const float f = (mloc == -INFINITY || tot.y == 0.f) ? 0.f : ex2_approx(mloc - tot.x) / tot.y;
        // ---------------- pass C: scale, round once, store (zeros where masked)
#pragma unroll
        for (int sub = 0; sub < NSUB; ++sub) {
          const int n0 = ncta0 + sub * BNS;
          const bool masked_sub = subtile_masked(m0, n0);
#pragma unroll
          for (int c = 0; c < CHUNKS / 2; ++c) {
            const int lc = sub * BNS + (2 * c + h) * 32;
            const int st = masked_sub ? 0 : chunk_state(ncta0 + lc);
            uint32_t pk[16];
            if (st == 0) {
#pragma unroll
              for (int j = 0; j < 16; ++j) pk[j] = 0u;
            } else {
              uint32_t v[32];
              tmem_ld_32cols(lane_base + lc, v);
#pragma unroll
              for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2_rn(__uint_as_float(v[2 * j]) * f, __uint_as_float(v[2 * j + 1]) * f);
            }
            if (valid) store_chunk_bf16(yrow + ncta0 + lc, pk);
          }
          if (!masked_sub) {
            tcgen05_fence_before_sync();
            mbar_arrive(bar_tempty(sub));
          }
        }
      }
    }
  }

  // -------------------------------------------------------------------------------------------- teardown
  tcgen05_fence_before_sync();
  __syncthreads();
  if constexpr (CN > 1) cluster_sync_all();  // no peer may still write into or arrive on this CTA's shared memory
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after_sync();
    tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
  }
}

}  // namespace comfuse
