// Row softmax behind a SHORT-K GEMM:  P = softmax(alpha * A.B + mask)  over the last dimension, for K so small that
// computing a score tile twice is cheaper than moving it (the attention-score pattern of Sec. 6.1: K = head size).
//
// Stage-Stream view (Sec. 3): the row reduction (max, sum of exponentials) is the stage boundary.  The general kernel
// keeps a whole row block on-chip by spreading its columns over a cluster and aggregating the partial statistics
// through distributed shared memory (Sec. 3.2).  With K <= 256 the producer stage is so cheap that this kernel takes
// the other side of the same trade: one CTA pair owns 256 complete rows, streams the row through tensor memory in
// 256-column chunks TWICE (MainLoop re-run instead of on-chip residency), and needs no cross-CTA exchange at all:
//
//   pass 0   for every live chunk:  S = A.B_chunk (UMMA, cta_group::2)  ->  online (max, sum) per thread
//   merge    the four threads that share a row combine their partials through shared memory
//   pass 1   for every live chunk:  S again  ->  P = 2^(S*alpha*log2e - (max + log2 sum))  ->  bf16 box -> TMA store
//
// Clusters are pairs, so all SMs are used (wider clusters leave SMs idle), any N fits, and the accumulator slots
// alternate so that the UMMAs of chunk u+1 run under the epilogue of chunk u.  Under a causal mask, chunks above the
// diagonal are neither computed nor staged: the epilogue warps write their zeros with plain stores, a few rows after
// every chunk pass, from a cursor that runs through the cluster's tiles on its own.
//
// Warp roles as in the general kernel: warp 0 TMA producer, warp 1 TMEM allocation + UMMA issue (even CTA),
// 16 epilogue warps (thread = row; warp e takes lane quarter e % 4 and 64-column group e / 4 of each chunk), last warp
// issues the TMA stores of the staged boxes.  Every wait is bounded.
#pragma once

#include "epilogue_common.cuh"
#include "fused_params.h"
#include "sm100_primitives.cuh"

namespace comfuse {

template <int NSTAGES, int YBOXES>
struct RowSoftmaxCfg {
  static constexpr int kEpiWarps = 16;
  static constexpr int kStoreWarp = 2 + kEpiWarps;
  static constexpr int kZeroWarp = kStoreWarp + 1;
  static constexpr int kThreads = 32 * (kZeroWarp + 1);
  static constexpr int ZERO_TMA_LANES = 4;                   // zero boxes in flight per SM
  static constexpr int CHUNK = 256;                          // columns per UMMA and per accumulator slot
  // Which of a 32-column fragment's 16 column pairs take 2^x from the FMA-pipe polynomial instead of the MUFU unit
  // (bit j = pair j).  The MUFU unit delivers 16 results per clock per SM and is this kernel's busiest pipe; the
  // polynomial costs about six issue slots per value.  Measured on the attention-score workload: none 126.2 us,
  // 2 of 16 pairs 123.7, 3: 123.1, 4: 122.7, 5: 123.9, 6: 124.8, 8: 128.8.
  static constexpr uint32_t POLY_PAIRS = 0x1248u;            // pairs 3, 6, 9, 12
  static constexpr int A_BYTES = 128 * 64 * 2;
  static constexpr int STAGE_BYTES = A_BYTES + (CHUNK / 2) * 64 * 2;  // A block + this CTA's half of the B chunk
  static constexpr int WARP_BOX_BYTES = 32 * 64 * 2;
  static constexpr int OFF_YBUF = NSTAGES * STAGE_BYTES;
  static constexpr int YBUF_BYTES = kEpiWarps * YBOXES * WARP_BOX_BYTES;
  static constexpr int OFF_ZERO = OFF_YBUF + YBUF_BYTES;     // constant zero box
  static constexpr int OFF_PRE = OFF_ZERO + WARP_BOX_BYTES;  // per-row partials of the 4 column groups, two tile parities
  static constexpr int PRE_BYTES = 2 * 4 * 128 * 8;
  static constexpr int OFF_BAR = OFF_PRE + PRE_BYTES;
  static constexpr int NUM_BARS = 2 * NSTAGES + 4 + 1 + 2 * kEpiWarps * YBOXES;
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;
  static constexpr int SMEM_BYTES = OFF_MISC + 16 + 1024;
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
  static_assert(SMEM_BYTES > 116 * 1024, "one CTA per SM is assumed (TMEM allocation never waits for a co-resident CTA)");
  static_assert(NSTAGES >= 2 && NSTAGES <= 8 && YBOXES >= 1 && YBOXES <= 4, "ring and staging depths");
};

// BKM: the B operand is stored [N, K] (one box of this CTA's 128 columns x 64 contraction elements per stage, K-major for the
// UMMA, like A) instead of [K, N] (two boxes of 64 contraction rows x 64 columns, MN-major).
template <int NSTAGES, int YBOXES, bool BKM>
__global__ void __launch_bounds__(32 * 20, 1)
softmax_rows_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmY, const FusedParams p) {
  using Cfg = RowSoftmaxCfg<NSTAGES, YBOXES>;
  constexpr int CHUNK = Cfg::CHUNK;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t smem_base = smem_u32(smem);

  float2* s_pre = reinterpret_cast<float2*>(smem + Cfg::OFF_PRE);
  const uint32_t bar_base = smem_base + Cfg::OFF_BAR;
  auto bar_full = [&](int s) { return bar_base + 8u * s; };                     // K-block stage landed (even CTA)
  auto bar_empty = [&](int s) { return bar_base + 8u * (NSTAGES + s); };        // stage may be overwritten
  auto bar_tfull = [&](int a) { return bar_base + 8u * (2 * NSTAGES + a); };    // accumulator slot complete
  auto bar_tempty = [&](int a) { return bar_base + 8u * (2 * NSTAGES + 2 + a); };  // slot drained by both CTAs (even CTA)
  const uint32_t bar_drain = bar_base + 8u * (2 * NSTAGES + 4);
  auto bar_yfull = [&](int e, int k) { return bar_drain + 8u + 8u * (e * YBOXES + k); };
  auto bar_yfree = [&](int e, int k) { return bar_drain + 8u + 8u * (Cfg::kEpiWarps * YBOXES + e * YBOXES + k); };
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(smem + Cfg::OFF_MISC);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + Cfg::OFF_MISC + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t pm = cluster_ctarank();  // which 128-row block of the pair; rank 0 issues the UMMAs
  const int cluster_id = blockIdx.x >> 1;
  const int num_clusters = gridDim.x >> 1;
  const int KB = (p.K + 63) >> 6;
  const int nch = (p.N + CHUNK - 1) / CHUNK;
  const int rounds = (p.total_tiles + num_clusters - 1) / num_clusters;
  const WaitCtx w{s_abort, p.status, p.timeout_ns};
  griddep_launch_dependents();  // the next kernel's set-up may overlap this kernel (it waits before touching memory)

  // -------------------------------------------------------------------------------------------- set-up
  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGES; ++s) {
      mbar_init(bar_full(s), 2);   // one arrive.expect_tx from each CTA of the pair
      mbar_init(bar_empty(s), 1);  // one commit from the issuing CTA
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull(a), 1);
      mbar_init(bar_tempty(a), 2 * Cfg::kEpiWarps);  // one arrival per epilogue warp of both CTAs
    }
    mbar_init(bar_drain, 1);
    for (int e = 0; e < Cfg::kEpiWarps; ++e)
      for (int k = 0; k < YBOXES; ++k) {
        mbar_init(bar_yfull(e, k), 1);
        mbar_init(bar_yfree(e, k), 1);
      }
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    prefetch_tensormap(&tmY);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(s_tmem_base), 2 * CHUNK);
    tmem_relinquish_alloc_permit_pair();
  }
  for (int i = threadIdx.x; i < Cfg::WARP_BOX_BYTES / 4; i += Cfg::kThreads) reinterpret_cast<uint32_t*>(smem + Cfg::OFF_ZERO)[i] = 0u;
  fence_proxy_async_smem();  // the zero box is read by TMA stores
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  cluster_sync_after_init();  // both CTAs' barriers exist before the peer signals them
  const uint32_t tmem_base = *s_tmem_base;
  griddep_wait();  // the set-up above may overlap the previous kernel's tail; global memory is touched only below

  // Tile of this cluster in round r.  Tiles are ordered by falling cost (under a causal mask a lower row block has
  // more live chunks) and dealt to the clusters in alternating direction, so the clusters' sums stay close.
  auto tile_at = [&](int r, int& b, int& mpair0, int& live_chunks) {
    const int pos = r * num_clusters + ((r & 1) ? num_clusters - 1 - cluster_id : cluster_id);
    if (pos >= p.total_tiles) return false;
    const int mp = p.mpairs - 1 - pos / p.batch;
    b = pos - (pos / p.batch) * p.batch;
    mpair0 = mp * 256;
    live_chunks = p.causal ? (mp + 1 < nch ? mp + 1 : nch) : nch;  // chunk c is live iff c*256 <= mpair0 + 255
    return true;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      // every operand chunk is read twice per tile and the K matrix by every tile of its batch, while 16 times as many
      // output bytes stream through the L2: ask it to keep the operands
      const uint64_t keep = l2_policy_evict_last();
      for (int r = 0; r < rounds && ok; ++r) {
        int b, mpair0, L;
        if (!tile_at(r, b, mpair0, L)) continue;
        const int m0 = mpair0 + static_cast<int>(pm) * 128;
        for (int u = 0; u < 2 * L && ok; ++u) {
        const int c = u < L ? u : u - L;  // pass 0 over the live chunks, then pass 1
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait<false>(bar_empty(stage), phase ^ 1u, w)) { ok = false; break; }  // passes on a fresh barrier
          const uint32_t sa = smem_base + stage * Cfg::STAGE_BYTES;
          const uint32_t full = map_to_cta(bar_full(stage), 0);
          mbar_arrive_expect_tx_cluster(full, Cfg::STAGE_BYTES);
          tma_load_3d_pair_hint(sa, &tmA, full, kb * 64, m0, b, keep);
          // this CTA's half of the UMMA's B tile: two boxes of 64 columns, 8 KB apart
          const int col = c * CHUNK + static_cast<int>(pm) * (CHUNK / 2);
          if constexpr (BKM) {  // two boxes of 64 rows of B (columns of the product) x 64 contraction elements
            tma_load_3d_pair_hint(sa + Cfg::A_BYTES, &tmB, full, kb * 64, col, b, keep);
            tma_load_3d_pair_hint(sa + Cfg::A_BYTES + 8192, &tmB, full, kb * 64, col + 64, b, keep);
          } else {
            tma_load_3d_pair_hint(sa + Cfg::A_BYTES, &tmB, full, col, kb * 64, b, keep);
            tma_load_3d_pair_hint(sa + Cfg::A_BYTES + 8192, &tmB, full, col + 64, kb * 64, b, keep);
          }
          if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
        }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ UMMA issuer (even CTA)
    if (lane == 0 && pm == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t slot_uses[2] = {0, 0};
      uint32_t unit = 0;
      constexpr uint32_t idesc = make_idesc_bf16(256, CHUNK, false, !BKM);
      bool ok = true;
      uint32_t total_units = 0;
      for (int r = 0; r < rounds; ++r) {
        int b, mpair0, L;
        if (tile_at(r, b, mpair0, L)) total_units += 2u * L;
      }
      while (ok && unit < total_units) {
        const int slot = static_cast<int>(unit & 1u);
        ++unit;
        if (!mbar_wait<false>(bar_tempty(slot), (slot_uses[slot] & 1u) ^ 1u, w)) break;
        ++slot_uses[slot];
        tcgen05_fence_after_sync();
        const uint32_t d_tmem = tmem_base + slot * CHUNK;
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait<false>(bar_full(stage), phase, w)) { ok = false; break; }
          tcgen05_fence_after_sync();
          const uint32_t sa = smem_base + stage * Cfg::STAGE_BYTES;
          const uint64_t adesc = make_smem_desc_sw128(sa, 16, 1024);
          const uint64_t bdesc = BKM ? make_smem_desc_sw128(sa + Cfg::A_BYTES, 16, 1024)
                                     : make_smem_desc_sw128(sa + Cfg::A_BYTES, /*next 64-column block*/ 8192, /*next 8 K rows*/ 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k)  // K advances by 16 elements: 32 bytes inside a K-major operand's swizzled row, 2048 bytes in an MN-major B
            umma_bf16_ss_pair(d_tmem, adesc + static_cast<uint64_t>(k * 2), bdesc + static_cast<uint64_t>(BKM ? k * 2 : k * 128), idesc,
                              (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair_both(bar_empty(stage));
          if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair_both(bar_tfull(slot));
      }
      umma_commit_pair(bar_drain);  // nothing may still be writing either CTA's TMEM when it is freed
      mbar_wait<false>(bar_drain, 0, w);
    }
  } else if (warp == Cfg::kStoreWarp) {
    // ------------------------------------------------------------------------------------------ store warp
    // Lane e mirrors epilogue warp e: per live chunk, wait until the box is staged, store it, hand the staging box back.
    if (lane < Cfg::kEpiWarps) {
      const int e = lane;
      const int q = (e + 2) & 3;
      const int h = e >> 2;
      constexpr int D = YBOXES - 1;
      const uint32_t ybox0 = smem_base + Cfg::OFF_YBUF + e * YBOXES * Cfg::WARP_BOX_BYTES;
      const uint64_t stream_out = l2_policy_evict_first();  // the output is never read again
      uint32_t n = 0;
      bool ok = true;
      for (int r = 0; r < rounds && ok; ++r) {
        int b, mpair0, L;
        if (!tile_at(r, b, mpair0, L)) continue;
        for (int c = 0; c < L; ++c) {
        const int col = c * CHUNK + h * 64;
        if (col >= p.N) break;
        const uint32_t sel = n % YBOXES;
        if (!mbar_wait<false>(bar_yfull(e, sel), (n / YBOXES) & 1u, w)) { ok = false; break; }
#ifdef COMFUSE_TRACE
        if (!(p.trace_flags & 1))
#endif
        if (COMFUSE_IN_BOUNDS(col >= 0 && col < p.N && (col & 7) == 0 && mpair0 >= 0 && b >= 0 && b < p.batch, p.status))
        tma_store_3d_hint(&tmY, ybox0 + sel * Cfg::WARP_BOX_BYTES, col, mpair0 + static_cast<int>(pm) * 128 + q * 32, b, stream_out);
        tma_store_commit();
        if (n >= static_cast<uint32_t>(D)) {
          tma_store_wait_read<D>();
          mbar_arrive(bar_yfree(e, (n - D) % YBOXES));
        }
        ++n;
        }
      }
      tma_store_wait_read<0>();  // shared memory must outlive the last stores' reads (the stores complete at kernel end)
    }
  } else if (warp == Cfg::kZeroWarp) {
    // ------------------------------------------------------------------------------------------ zero-box warp
    // The chunks above the causal diagonal hold zeros and depend on nothing.  A few lanes, each with one TMA store of a
    // constant zero box in flight, walk them with a cursor of their own, independent of the epilogue (asynchronous
    // stores: plain stores would share the SM's memory-instruction queue with the epilogue's exponentials and
    // shared-memory traffic).  Few boxes in flight, so that a staged box never queues far behind zeros.
    if (lane < Cfg::ZERO_TMA_LANES && p.causal) {
      const uint64_t stream_out = l2_policy_evict_first();
      uint32_t k = 0;
      for (int r = 0; r < rounds; ++r) {
        int b, mpair0, L;
        if (!tile_at(r, b, mpair0, L)) continue;
        const int y0 = mpair0 + static_cast<int>(pm) * 128;
        for (int c = L; c < nch; ++c)
          for (int i = 0; i < 16; ++i, ++k) {
            if (k % Cfg::ZERO_TMA_LANES != static_cast<uint32_t>(lane)) continue;
            const int col = c * CHUNK + (i >> 2) * 64;
            if (col >= p.N) continue;
            tma_store_wait_all();
#ifdef COMFUSE_TRACE
            if (!(p.trace_flags & 4))
#endif
            if (COMFUSE_IN_BOUNDS(col >= 0 && (col & 7) == 0 && y0 >= 0 && b >= 0 && b < p.batch, p.status))
            tma_store_3d_hint(&tmY, smem_base + Cfg::OFF_ZERO, col, y0 + (i & 3) * 32, b, stream_out);
            tma_store_commit();
          }
      }
      tma_store_wait_read<0>();
    }
  } else {
    // ------------------------------------------------------------------------------------------ epilogue warps
    const int e = warp - 2;
    const int q = warp & 3;  // TMEM lane quarter this warp may touch: rows 32q .. 32q+31 of the CTA's row block
    const int h = e >> 2;    // the 64-column group of every chunk this warp takes
    const int row = q * 32 + lane;
    const uint32_t lane_sel = static_cast<uint32_t>(q * 32) << 16;
    const uint32_t tempty_leader = map_to_cta(bar_tempty(0), 0);
    const uint32_t ybox0 = smem_base + Cfg::OFF_YBUF + e * YBOXES * Cfg::WARP_BOX_BYTES;
    uint32_t slot_uses[2] = {0, 0};
    uint32_t unit = 0, nbox = 0, tile_par = 0;
    // log2 domain: t = Acc * (alpha * log2 e), so exp(x - m) = 2^(t - m_t)
    // with a soft-cap the accumulators are mapped to capped log2-domain scores right after they are loaded, and sc = 1
    const bool capped = p.softcap > 0.f;
    const SoftcapLog2 cap_fn(p.alpha, capped ? p.softcap : 1.f);
    const float sc = capped ? 1.f : p.alpha * 1.4426950408889634f;
    const bool additive = p.mask != nullptr;  // additive mask tensor, applied behind the scale / soft-cap
    constexpr uint32_t poly_pairs = Cfg::POLY_PAIRS;

#ifdef COMFUSE_TRACE
    int trace_ix = 0;
#define ROWS_TRACE_POINT()                                                                             \
  do {                                                                                                 \
    if (p.trace && blockIdx.x == 0 && warp == 2 && lane == 0 && trace_ix < 60) p.trace[trace_ix++] = globaltimer_ns(); \
  } while (0)
#else
#define ROWS_TRACE_POINT() do { } while (0)
#endif
    auto wait_slot = [&](int slot) {
      ROWS_TRACE_POINT();
      mbar_wait<false>(bar_tfull(slot), slot_uses[slot] & 1u, w);
      ++slot_uses[slot];
      __syncwarp();
      tcgen05_fence_after_sync();
      ROWS_TRACE_POINT();
    };
    auto release_slot = [&](int slot) {
      tcgen05_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_noflush(tempty_leader + 8u * slot);
    };

    for (int r = 0; r < rounds; ++r) {
      int b, mpair0, L;
      if (!tile_at(r, b, mpair0, L)) continue;
      float m_run = -INFINITY, s_run = 0.f;  // pass 0: this thread's running maximum and sum of 2^(t - max)
      float off = INFINITY;                  // pass 1: P = 2^(t - off)
      for (int u = 0; u < 2 * L; ++u) {
        {
          const int pass = u < L ? 0 : 1, c = u < L ? u : u - L;
          const int m0 = mpair0 + static_cast<int>(pm) * 128;
          const int grow = m0 + row;
          // last live column of this thread's row, and of the warp's first / last row (fragment classification must be
          // uniform over the warp so that the warp-wide TMEM loads stay convergent)
          const int lim = p.causal ? (grow < p.N - 1 ? grow : p.N - 1) : p.N - 1;
          const int wrow0 = m0 + q * 32;
          const int lim_lo = p.causal ? (wrow0 < p.N - 1 ? wrow0 : p.N - 1) : p.N - 1;
          const int lim_hi = p.causal ? (wrow0 + 31 < p.N - 1 ? wrow0 + 31 : p.N - 1) : p.N - 1;
          // 2 = all 32 columns live for all 32 rows, 0 = none live for any row, 1 = mixed
          auto frag_state = [&](int col0) { return col0 + 31 <= lim_lo ? 2 : (col0 > lim_hi ? 0 : 1); };

          const int slot = static_cast<int>(unit & 1u);
          ++unit;
          wait_slot(slot);
          const uint32_t taddr = tmem_base + lane_sel + slot * CHUNK + h * 64;
          const int colg = c * CHUNK + h * 64;
          if (pass == 0) {
            // ---------------- pass 0: online (max, sum of 2^(t - max)) over this thread's columns of the chunk
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int col0 = colg + half * 32;
              const int st = frag_state(col0);
              if (st == 0) continue;
              uint32_t v[32];
              tmem_ld_32cols(taddr + half * 32, v);
              if (capped) {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(cap_fn(__uint_as_float(v[j])));
              }
              float2 tv[16];
              if (additive) {  // a full-tensor operand of the epilogue (Sec. 5.2): this thread's 32 mask values from global memory
                float2 m2[16];
                load_mask_log2_32(p.mask + static_cast<long long>(grow) * p.N + col0, grow < p.M ? p.N - col0 : 0, m2);
#pragma unroll
                for (int j = 0; j < 16; ++j) tv[j] = fma2(f2_from_bits(v[2 * j], v[2 * j + 1]), splat2(sc), m2[j]);
              } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) tv[j] = mul2(f2_from_bits(v[2 * j], v[2 * j + 1]), splat2(sc));
              }
              if (st != 2) {  // the fragment crosses the diagonal (or the end of the row): rare, kept out of the main path
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  if (col0 + 2 * j > lim) tv[j].x = -INFINITY;
                  if (col0 + 2 * j + 1 > lim) tv[j].y = -INFINITY;
                }
              }
              float mx0 = m_run, mx1 = -INFINITY;
#pragma unroll
              for (int j = 0; j < 16; j += 2) {
                mx0 = max3(mx0, tv[j].x, tv[j].y);
                mx1 = max3(mx1, tv[j + 1].x, tv[j + 1].y);
              }
              const float m_new = fmaxf(mx0, mx1);
              if ((st == 2 && !additive) || m_new != -INFINITY) {  // else every column seen so far is masked for this row
                float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
                const float2 neg_m = splat2(-m_new);
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                  const float2 d0 = add2(tv[j], neg_m), d1 = add2(tv[j + 1], neg_m);
                  acc0 = add2(acc0, ((poly_pairs >> j) & 1u) ? ex2_poly2(d0) : make_float2(ex2_approx(d0.x), ex2_approx(d0.y)));
                  acc1 = add2(acc1, ((poly_pairs >> (j + 1)) & 1u) ? ex2_poly2(d1) : make_float2(ex2_approx(d1.x), ex2_approx(d1.y)));
                }
                const float2 acc = add2(acc0, acc1);
                s_run = fmaf(s_run, ex2_approx(m_run - m_new), acc.x + acc.y);
                m_run = m_new;
              }
            }
            release_slot(slot);
          } else {
            // ---------------- pass 1: the scores again, normalised, rounded once, staged and stored
            uint32_t pk[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int col0 = colg + half * 32;
              const int st = frag_state(col0);
              if (st == 0) {
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[half * 16 + j] = 0u;
              } else {
                uint32_t v[32];
                tmem_ld_32cols(taddr + half * 32, v);
                if (capped) {
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(cap_fn(__uint_as_float(v[j])));
                }
                float2 ev[16];
                if (additive) {
                  float2 m2[16];
                  load_mask_log2_32(p.mask + static_cast<long long>(grow) * p.N + col0, grow < p.M ? p.N - col0 : 0, m2);
#pragma unroll
                  for (int j = 0; j < 16; ++j) {  // (a masked score is -inf, and so is -inf - off: its probability is an exact zero)
                    const float2 t01 = fma2(f2_from_bits(v[2 * j], v[2 * j + 1]), splat2(sc), add2(m2[j], splat2(-off)));
                    ev[j] = make_float2(ex2_approx(t01.x), ex2_approx(t01.y));
                  }
                } else {
#pragma unroll
                  for (int j = 0; j < 16; ++j) {
                    const float2 t01 = fma2(f2_from_bits(v[2 * j], v[2 * j + 1]), splat2(sc), splat2(-off));
                    ev[j] = ((poly_pairs >> j) & 1u) ? ex2_poly2(t01) : make_float2(ex2_approx(t01.x), ex2_approx(t01.y));
                  }
                }
                if (st != 2) {  // crosses the diagonal (or the end of the row)
#pragma unroll
                  for (int j = 0; j < 16; ++j) {
                    if (col0 + 2 * j > lim) ev[j].x = 0.f;
                    if (col0 + 2 * j + 1 > lim) ev[j].y = 0.f;
                  }
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[half * 16 + j] = pack_bf16x2_rn(ev[j]);
              }
            }
            release_slot(slot);
            if (colg < p.N) {
              const uint32_t sel = nbox % YBOXES;
              const uint32_t ybox = ybox0 + sel * Cfg::WARP_BOX_BYTES;
              // the store of the box's previous contents has read it out
              mbar_wait<false>(bar_yfree(e, sel), ((nbox / YBOXES) & 1u) ^ 1u, w);
              ++nbox;
              __syncwarp();
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const uint32_t a = ybox + static_cast<uint32_t>(lane * 128 + ((i ^ (lane & 7)) << 4));  // 128-byte swizzle
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[4 * i]), "r"(pk[4 * i + 1]),
                             "r"(pk[4 * i + 2]), "r"(pk[4 * i + 3])
                             : "memory");
              }
              fence_proxy_async_smem();
              __syncwarp();
              if (lane == 0) mbar_arrive(bar_yfull(e, sel));
            }
          }
        }
        if (u == L - 1) {
          // ---------------- pass 0 of the tile is complete: merge the four column groups of the row (they live in the
          // four warps of this lane quarter); the result serves the tile's pass 1, which starts with the next unit
          float2* pre = s_pre + tile_par * 512;
          tile_par ^= 1u;
          pre[h * 128 + row] = make_float2(m_run, s_run);
          named_barrier_sync(1 + q, 128);
          float m_row = -INFINITY, s_row = 0.f;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 o = pre[i * 128 + row];
            const float m_new = fmaxf(m_row, o.x);
            if (m_new != -INFINITY) {
              s_row = s_row * ex2_approx(m_row - m_new) + o.y * ex2_approx(o.x - m_new);
              m_row = m_new;
            }
          }
          // a row without a live column (cannot happen under the causal mask) is all zero: 2^(-inf)
          off = s_row > 0.f ? m_row + __log2f(s_row) : INFINITY;
        }
      }
    }
  }

  // -------------------------------------------------------------------------------------------- teardown
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // the peer may no longer signal this CTA's barriers or write its TMEM
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after_sync();
    tmem_dealloc_pair(tmem_base, 2 * CHUNK);
  }
}

}  // namespace comfuse
