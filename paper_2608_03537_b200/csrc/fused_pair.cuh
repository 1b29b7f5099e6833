// GEMM -> row-reduction subgraph in one kernel, CTA-pair edition (Stage-Stream Execution Model, Sec. 3).
//
// Why pairs: one SM's shared memory delivers 128 B/clk, and a 128 x 256 x 16 bf16 UMMA that reads both operands
// from shared memory already needs 96 B/clk before TMA has written the next tiles.  With cta_group::2 two CTAs
// multiply 256 rows at once: each holds its own 128 rows of A and only HALF of the B tile, so the per-SM operand
// traffic (and the L2 -> shared-memory fill) of the weight operand halves.  No multicast copies are used: each
// CTA fetches its own half with ordinary TMA loads that signal the issuing (even) CTA's barrier.
//
// Work decomposition (Sec. 3.1, cluster-granular scheduling with a secondary mapping by CTA rank): a cluster has
// 2*CN CTAs; cluster rank r works on row block (r & 1) of a pair of adjacent 128-row blocks and on column range
// (r >> 1) of CN.  All CTAs with the same (r & 1) share rows and form one reduction group (Sec. 3, Eq. 1); they
// exchange per-row partial statistics over distributed shared memory.  Clusters are persistent and walk the row
// block pairs with a stride of the cluster count.
//
// Inside a CTA (10 warps): warp 0 = TMA producer, warp 1 = TMEM allocation and (even CTA only) UMMA issue,
// warps 2-9 = epilogue (thread = one accumulator row; the two warps of a lane quarter split the 32-column chunks).
// The CTA's BN = BNS0 + BNS1 accumulator columns advance in lock step (A is fetched once per K block), NACC
// accumulator buffers let the next tile's MainLoop overlap this tile's epilogue when 2*BN <= 512 columns.
#pragma once

#include "epilogue_common.cuh"
#include "fused_params.h"
#include "sm100_primitives.cuh"

namespace comfuse {

template <int EPI, int BNS0, int BNS1, int CN, int NACC, int NSTAGES>
struct PairCfg {
  static constexpr int kThreads = 320;
  static constexpr int kEpiThreads = 256;
  static constexpr int BN = BNS0 + BNS1;
  static constexpr int A_BYTES = 128 * 64 * 2;
  static constexpr int B0_BYTES = (BNS0 / 2) * 64 * 2;  // this CTA's half of sub-tile 0's B tile
  static constexpr int B1_BYTES = (BNS1 / 2) * 64 * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B0_BYTES + B1_BYTES;
  static constexpr int ACC_COLS = NACC * BN;
  static constexpr int TMEM_COLS = ACC_COLS <= 32 ? 32 : ACC_COLS <= 64 ? 64 : ACC_COLS <= 128 ? 128 : ACC_COLS <= 256 ? 256 : 512;
  static constexpr int OFF_VEC = NSTAGES * STAGE_BYTES;
  static constexpr int VEC_BYTES = 3 * BN * 4;
  static constexpr int OFF_STATS = OFF_VEC + VEC_BYTES;
  static constexpr int STATS_BYTES = 2 * CN * 128 * 8;
  static constexpr int OFF_PRE = OFF_STATS + STATS_BYTES;
  static constexpr int PRE_BYTES = 2 * 2 * 128 * 8;
  static constexpr int OFF_BAR = OFF_PRE + PRE_BYTES;
  static constexpr int NUM_BARS = 2 * NSTAGES + 2 * NACC + 2;
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;
  static constexpr int SMEM_BYTES = OFF_MISC + 16 + 1024;
  static_assert(BNS0 % 128 == 0 && BNS0 <= 256 && BNS1 % 128 == 0 && BNS1 <= 256, "each CTA's half must be whole 64-column boxes");
  static_assert(BNS0 > 0 && ACC_COLS <= 512, "accumulators must fit the 512 TMEM columns");
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
  static_assert(SMEM_BYTES > 116 * 1024, "one CTA per SM is assumed (TMEM allocation never waits for a co-resident CTA)");
};

template <int EPI, int BNS0, int BNS1, int CN, int NACC, int NSTAGES>
__global__ void __launch_bounds__(320, 1)
fused_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const FusedParams p) {
  using Cfg = PairCfg<EPI, BNS0, BNS1, CN, NACC, NSTAGES>;
  constexpr int BN = Cfg::BN;
  constexpr int CHUNK_PAIRS = BN / 64;  // each epilogue thread handles one 32-column chunk of every 64 columns

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
  auto bar_tfull = [&](int a) { return bar_base + 8u * (2 * NSTAGES + a); };
  auto bar_tempty = [&](int a) { return bar_base + 8u * (2 * NSTAGES + NACC + a); };
  const uint32_t bar_stats = bar_base + 8u * (2 * NSTAGES + 2 * NACC);
  const uint32_t bar_drain = bar_stats + 8u;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(smem + Cfg::OFF_MISC);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + Cfg::OFF_MISC + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t pm = rank & 1u;           // which row block of the pair
  const uint32_t crank = rank >> 1;        // which column range
  const uint32_t leader = rank & ~1u;      // cluster rank of the CTA that issues the pair's UMMAs
  const uint32_t peer = rank ^ 1u;
  constexpr int CLUSTER = 2 * CN;
  const int cluster_id = blockIdx.x / CLUSTER;
  const int num_clusters = gridDim.x / CLUSTER;
  const int KB = (p.K + 63) >> 6;
  const WaitCtx w{s_abort, p.status, p.timeout_ns};

  // -------------------------------------------------------------------------------------------- set-up
  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGES; ++s) {
      mbar_init(bar_full(s), 2);   // one arrive.expect_tx from each CTA of the pair (used in the even CTA only)
      mbar_init(bar_empty(s), 1);  // one commit from the issuing CTA
    }
    for (int a = 0; a < NACC; ++a) {
      mbar_init(bar_tfull(a), 1);
      mbar_init(bar_tempty(a), 2 * Cfg::kEpiThreads);  // both CTAs' epilogue threads (used in the even CTA only)
    }
    mbar_init(bar_stats, CN * 128);
    mbar_init(bar_drain, 1);
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(s_tmem_base), Cfg::TMEM_COLS);
    tmem_relinquish_alloc_permit_pair();
  }
  if constexpr (EPI == EPI_LN || EPI == EPI_RMS_MAX) {
    const int c0 = crank * BN;
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
  cluster_sync_all();  // every CTA's barriers exist before any peer signals them
  const uint32_t tmem_base = *s_tmem_base;

  // tile -> (batch, first row of the pair, first column of this CTA)
  auto decode_tile = [&](int tile, int& b, int& mpair0, int& ncta0) {
    const int per_batch = p.mpairs * p.nblocks;
    b = tile / per_batch;
    const int rem = tile - b * per_batch;
    const int mp = rem / p.nblocks;
    const int nb = rem - mp * p.nblocks;
    mpair0 = mp * 256;
    ncta0 = (nb * CN + static_cast<int>(crank)) * BN;
  };
  // Number of leading sub-tiles the pair has to compute: a sub-tile is dropped when it lies past N, or when the
  // causal mask removes it for BOTH row blocks of the pair.  Every role evaluates the same predicate.
  auto live_subtiles = [&](int mpair0, int ncta0) {
    auto dead = [&](int n0) { return n0 >= p.N || (EPI == EPI_SOFTMAX && p.causal && n0 > mpair0 + 255); };
    if (dead(ncta0)) return 0;
    if (BNS1 == 0 || dead(ncta0 + BNS0)) return 1;
    return 2;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < p.total_tiles && ok; tile += num_clusters) {
        int b, mpair0, ncta0;
        decode_tile(tile, b, mpair0, ncta0);
        const int nlive = live_subtiles(mpair0, ncta0);
        if (nlive == 0) continue;
        const int m0 = mpair0 + static_cast<int>(pm) * 128;
        const uint32_t bytes = Cfg::A_BYTES + Cfg::B0_BYTES + (nlive > 1 ? Cfg::B1_BYTES : 0);
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait<false>(bar_empty(stage), phase ^ 1u, w)) { ok = false; break; }
          const uint32_t sa = smem_base + stage * Cfg::STAGE_BYTES;
          const uint32_t sb0 = sa + Cfg::A_BYTES;
          const uint32_t sb1 = sb0 + Cfg::B0_BYTES;
          const uint32_t full = map_to_cta(bar_full(stage), leader);
          mbar_arrive_expect_tx_cluster(full, bytes);
          tma_load_3d_pair(sa, &tmA, full, kb * 64, m0, b);
#pragma unroll
          for (int j = 0; j < BNS0 / 128; ++j)
            tma_load_3d_pair(sb0 + j * 8192, &tmB, full, ncta0 + static_cast<int>(pm) * (BNS0 / 2) + j * 64, kb * 64, b);
          if (nlive > 1) {
#pragma unroll
            for (int j = 0; j < BNS1 / 128; ++j)
              tma_load_3d_pair(sb1 + j * 8192, &tmB, full, ncta0 + BNS0 + static_cast<int>(pm) * (BNS1 / 2) + j * 64, kb * 64, b);
          }
          if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ UMMA issuer (even CTA)
    if (lane == 0 && pm == 0) {
      constexpr uint32_t idesc0 = make_idesc_bf16(256, BNS0, false, true);
      constexpr uint32_t idesc1 = make_idesc_bf16(256, BNS1 > 0 ? BNS1 : 16, false, true);
      int stage = 0;
      uint32_t phase = 0;
      int acc_it = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < p.total_tiles && ok; tile += num_clusters) {
        int b, mpair0, ncta0;
        decode_tile(tile, b, mpair0, ncta0);
        const int nlive = live_subtiles(mpair0, ncta0);
        if (nlive == 0) continue;
        const int buf = acc_it % NACC;
        const uint32_t aphase = static_cast<uint32_t>(acc_it / NACC) & 1u;
        ++acc_it;
        if (!mbar_wait<true>(bar_tempty(buf), aphase ^ 1u, w)) { ok = false; break; }
        tcgen05_fence_after_sync();
        const uint32_t d0 = tmem_base + buf * BN;
        const uint32_t d1 = d0 + BNS0;
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait<false>(bar_full(stage), phase, w)) { ok = false; break; }
          tcgen05_fence_after_sync();
          const uint32_t sa = smem_base + stage * Cfg::STAGE_BYTES;
          const uint64_t adesc = make_smem_desc_sw128(sa, 16, 1024);
          const uint64_t bdesc0 = make_smem_desc_sw128(sa + Cfg::A_BYTES, 8192, 1024);
          const uint64_t bdesc1 = make_smem_desc_sw128(sa + Cfg::A_BYTES + Cfg::B0_BYTES, 8192, 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint32_t acc = (kb | k) != 0 ? 1u : 0u;
            umma_bf16_ss_pair(d0, adesc + static_cast<uint64_t>(k * 2), bdesc0 + static_cast<uint64_t>(k * 128), idesc0, acc);
            if (BNS1 > 0 && nlive > 1)
              umma_bf16_ss_pair(d1, adesc + static_cast<uint64_t>(k * 2), bdesc1 + static_cast<uint64_t>(k * 128), idesc1, acc);
          }
          // the stage is free in both CTAs once these UMMAs have read it
          umma_commit_pair(bar_empty(stage));
          umma_commit_pair(map_to_cta(bar_empty(stage), peer));
          if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) {
          umma_commit_pair(bar_tfull(buf));
          umma_commit_pair(map_to_cta(bar_tfull(buf), peer));
        }
      }
      umma_commit_pair(bar_drain);  // nothing may still be writing either CTA's TMEM when it is freed
      mbar_wait<false>(bar_drain, 0, w);
    }
  } else {
    // ------------------------------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;
    const int h = (warp - 2) >> 2;
    const int row = q * 32 + lane;
    int xpar = 0;
    uint32_t xphase = 0;
    int acc_it = 0;
    (void)xpar; (void)xphase; (void)s_pre; (void)s_stats; (void)s_bias; (void)s_gamma; (void)s_beta;
    constexpr float kThreadCount = static_cast<float>(BN / 2);
    const uint32_t tempty_leader_base = map_to_cta(bar_tempty(0), leader);

    for (int tile = cluster_id; tile < p.total_tiles; tile += num_clusters) {
      int b, mpair0, ncta0;
      decode_tile(tile, b, mpair0, ncta0);
      const int nlive = live_subtiles(mpair0, ncta0);
      const int m0 = mpair0 + static_cast<int>(pm) * 128;
      const int grow = m0 + row;
      const bool valid = grow < p.M;
      uint16_t* yrow = p.Y + static_cast<long long>(b) * p.batch_stride_y + static_cast<long long>(grow) * p.ldy;
      const uint16_t* rrow =
          p.residual ? p.residual + static_cast<long long>(b) * p.batch_stride_r + static_cast<long long>(grow) * p.ldr
                     : nullptr;
      const int buf = acc_it % NACC;
      const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * BN;
      if (nlive > 0) {
        mbar_wait<false>(bar_tfull(buf), static_cast<uint32_t>(acc_it / NACC) & 1u, w);
        ++acc_it;
        __syncwarp();
        tcgen05_fence_after_sync();
      }
      auto release_accumulator = [&]() {
        if (nlive > 0) {
          tcgen05_fence_before_sync();
          mbar_arrive_cluster(tempty_leader_base + 8u * buf);
        }
      };

      if constexpr (EPI == EPI_NONE) {
#pragma unroll
        for (int c = 0; c < CHUNK_PAIRS; ++c) {
          const int lc = (2 * c + h) * 32;
          const int col = ncta0 + lc;
          if (col >= p.N) continue;
          uint32_t v[32];
          tmem_ld_32cols(lane_base + lc, v);
          uint32_t pk[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
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
        release_accumulator();
      } else if constexpr (EPI == EPI_LN) {
        // ---------------- stage 1: x = alpha*Acc + bias + R ; thread-local (mean, M2); x written back (bypass path)
        float2 part = make_float2(0.f, 0.f);
        float n_run = 0.f;
#pragma unroll
        for (int c = 0; c < CHUNK_PAIRS; ++c) {
          const int lc = (2 * c + h) * 32;
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
          tmem_st_32cols(lane_base + lc, v);
        }
        tmem_st_wait();
        const float2 tot = cluster_row_reduce<CN>(part, kThreadCount, MergeWelford(), s_pre, s_stats, bar_stats, row, h, crank,
                                                  xpar, xphase, w, 2u, pm);
        const float mu = tot.x;
        const float rstd = rsqrtf(tot.y * (1.f / static_cast<float>(CN * BN)) + p.eps);
        // ---------------- stage 2: normalise the resident x, round once, store
#pragma unroll
        for (int c = 0; c < CHUNK_PAIRS; ++c) {
          const int lc = (2 * c + h) * 32;
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
        release_accumulator();
      } else if constexpr (EPI == EPI_RMS_MAX) {
        // ---------------- stage 1: H = GELU(alpha*Acc + bias) + R ; thread-local sum of squares; H written back
        float ss = 0.f;
#pragma unroll
        for (int c = 0; c < CHUNK_PAIRS; ++c) {
          const int lc = (2 * c + h) * 32;
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
        tmem_st_wait();
        const float2 tot = cluster_row_reduce<CN>(make_float2(ss, 0.f), kThreadCount, MergeSum(), s_pre, s_stats, bar_stats, row,
                                                  h, crank, xpar, xphase, w, 2u, pm);
        const float rstd = rsqrtf(tot.x * (1.f / static_cast<float>(CN * BN)) + p.eps);
        // ---------------- stage 2: Y = H * rstd * g ; thread-local (max, argmax) of the unrounded Y
        float best = -INFINITY;
        int best_col = 0x7FFFFFFF;
#pragma unroll
        for (int c = 0; c < CHUNK_PAIRS; ++c) {
          const int lc = (2 * c + h) * 32;
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
        release_accumulator();
        // ---------------- stage 3: the second, chained reduction reuses the exchange buffers (Sec. 3.2)
        const float2 mx = cluster_row_reduce<CN>(make_float2(best, __int_as_float(best_col)), kThreadCount, MergeArgmax(), s_pre,
                                                 s_stats, bar_stats, row, h, crank, xpar, xphase, w, 2u, pm);
        if (crank == 0 && h == 0 && valid) {
          const long long o = static_cast<long long>(b) * p.M + grow;
          p.row_max[o] = mx.x;
          p.row_argmax[o] = __float_as_int(mx.y);
        }
      } else {  // EPI_SOFTMAX
        // log2 domain: t = Acc * (alpha * log2 e), so exp(x - m) = 2^(t - m_t)
        const float sc = p.alpha * 1.4426950408889634f;
        // chunk classification under the causal mask, uniform over the warp's 32 rows so that the warp-wide TMEM
        // loads stay convergent: 2 = all live, 1 = crosses the diagonal, 0 = all masked
        const int wrow0 = m0 + q * 32;
        auto chunk_state = [&](int col0) { return !p.causal ? 2 : (col0 + 31 <= wrow0 ? 2 : (col0 > wrow0 + 31 ? 0 : 1)); };
        // ---------------- pass A: thread-local row max
        float mloc = -INFINITY;
#pragma unroll
        for (int c = 0; c < CHUNK_PAIRS; ++c) {
          const int lc = (2 * c + h) * 32;
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
        // ---------------- pass B: e = 2^(t - mloc), thread-local sum, e written back over the scores
        float lloc = 0.f;
        const float msub = (mloc == -INFINITY) ? 0.f : mloc;
#pragma unroll
        for (int c = 0; c < CHUNK_PAIRS; ++c) {
          const int lc = (2 * c + h) * 32;
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
        tmem_st_wait();
        const float2 tot = cluster_row_reduce<CN>(make_float2(mloc, lloc), kThreadCount, MergeMaxSumExp2(), s_pre, s_stats,
                                                  bar_stats, row, h, crank, xpar, xphase, w, 2u, pm);
        const float f = (mloc == -INFINITY || tot.y == 0.f) ? 0.f : ex2_approx(mloc - tot.x) / tot.y;
        // ---------------- pass C: scale, round once, store (zeros where masked)
#pragma unroll
        for (int c = 0; c < CHUNK_PAIRS; ++c) {
          const int lc = (2 * c + h) * 32;
          const int st = chunk_state(ncta0 + lc);
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
        release_accumulator();
      }
    }
  }

  // -------------------------------------------------------------------------------------------- teardown
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // no peer may still signal this CTA's barriers, write its shared memory or its TMEM
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after_sync();
    tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
  }
}

}  // namespace comfuse
