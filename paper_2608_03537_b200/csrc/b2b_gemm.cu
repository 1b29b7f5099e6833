// Fused back-to-back GEMM, attention form (Sec. 4 with a row softmax as F; the Target- and Self-Attention shapes of
// Sec. 6.2):  P = alpha X W1,  S = exp(P - rowmax),  O = (S W2) / rowsum, per batch.  Neither P nor S is written to
// global memory.  (The MLP form lives in b2b_mlp.cu, the ReLU MLP form with K streamed in b2b_stream.cu.)
//
// One CTA pair owns 256 rows; the two P slots hold a whole score row of 256 source positions (512 run as two sub-tiles
// with their own maxima, combined when O is normalised); O accumulates in tensor memory.  X, the two W1 chunks and the
// two W2 chunks flow through ONE ring of 16 KB slots (Sec. 4.2, unified circular buffer), in the order the consumers need
// them; the roles are software-pipelined over the cluster's tiles (see the UMMA lane).
//
// CTA pairs (cta_group::2): each CTA holds its own 128 rows of X / S and half (64 columns) of every weight chunk.
#include <cuda_runtime.h>

#include <atomic>

#include "b2b_params.h"
#include "epilogue_common.cuh"
#include "fused_pair.cuh"
#include "host_common.h"
#include "sm100_primitives.cuh"

namespace comfuse {

namespace {

constexpr int kB2bEpiWarps = 16;                       // four per TMEM lane quarter, 32 columns of a 128-column chunk each
constexpr int kB2bEpiThreads = 32 * kB2bEpiWarps;
constexpr int kB2bThreads = 32 * (2 + kB2bEpiWarps);  // producer, UMMA, epilogue warps
constexpr int kSlotBytes = 128 * 64 * 2;  // one 128 x 64 bf16 box
constexpr int kRingSlots = 8;

struct B2bSmem {
  static constexpr int OFF_RING = 0;
  static constexpr int OFF_S = kRingSlots * kSlotBytes;            // 2 buffers x 2 K blocks
  static constexpr int OFF_YBUF = OFF_S + 4 * kSlotBytes;          // output staging box (the second one is the idle eighth ring slot)
  static constexpr int OFF_PRE = OFF_YBUF + kSlotBytes;            // float2 [2][4][128]
  static constexpr int OFF_STATS = OFF_PRE + 2 * 4 * 128 * 8;      // float2 [2][1][128]
  static constexpr int OFF_BAR = OFF_STATS + 2 * 128 * 8;
  // barriers: full[8] empty[8] (8 unused) pfull[2] sfull[2] sempty[2] ofull[2] oempty[2] stats[2] drain pfree
  static constexpr int NUM_BARS = 3 * kRingSlots + 10 + 4;
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;
  static constexpr int BYTES = OFF_MISC + 16 + 1024;
};
static_assert(B2bSmem::BYTES <= 232448, "shared memory budget");

// NHALF: sub-tiles of 256 source positions per score row, 1 or 2.
template <int NHALF>
__global__ void __launch_bounds__(kB2bThreads, 1)
b2b_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW1,
                const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmO, const B2bParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t smem_base = smem_u32(smem);

  float2* s_pre = reinterpret_cast<float2*>(smem + B2bSmem::OFF_PRE);
  float2* s_stats = reinterpret_cast<float2*>(smem + B2bSmem::OFF_STATS);
  const uint32_t bar_base = smem_base + B2bSmem::OFF_BAR;
  auto bar_full = [&](int s) { return bar_base + 8u * s; };                        // weight / X slot landed (even CTA)
  auto bar_empty = [&](int s) { return bar_base + 8u * (kRingSlots + s); };        // slot may be overwritten
  auto bar_pfull = [&](int a) { return bar_base + 8u * (3 * kRingSlots + a); };    // P slot complete
  auto bar_sfull = [&](int a) { return bar_base + 8u * (3 * kRingSlots + 2 + a); };   // S buffer written by both CTAs (even CTA)
  auto bar_sempty = [&](int a) { return bar_base + 8u * (3 * kRingSlots + 4 + a); };  // S buffer read by ML2
  auto bar_ofull = [&](int a) { return bar_base + 8u * (3 * kRingSlots + 6 + a); };   // O slot complete
  auto bar_oempty = [&](int a) { return bar_base + 8u * (3 * kRingSlots + 8 + a); };  // O slot drained by both CTAs (even CTA)
  const uint32_t bar_stats = bar_base + 8u * (3 * kRingSlots + 10);
  const uint32_t bar_drain = bar_stats + 16u;
  const uint32_t bar_pfree = bar_drain + 8u;  // attention form: both P slots read by every epilogue warp (even CTA)
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(smem + B2bSmem::OFF_MISC);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + B2bSmem::OFF_MISC + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // cluster of exactly two CTAs
  const uint32_t pm = rank & 1u;
  const uint32_t leader = 0u;
  const int cluster_id = blockIdx.x >> 1;
  const int num_clusters = gridDim.x >> 1;
  const int total_tiles = p.batch * p.mpairs;
  // attention form: a score row of 512 source positions is processed as two sub-tiles of 256 (each with its own maximum
  // and its own O slot) that the normalisation step combines; nsub = sub-tiles this cluster walks
  constexpr int nhalf = NHALF;
  const int my_tiles = cluster_id < total_tiles ? (total_tiles - cluster_id + num_clusters - 1) / num_clusters : 0;
  const int nsub = my_tiles * nhalf;
  // The epilogue, not the loads, sets the pace: the ring walks seven of the eight slots and the eighth is a second output
  // staging box, so that both 64-column halves of a tile are staged and stored together.
  constexpr int RING = kRingSlots - 1;
  const WaitCtx w{s_abort, p.status, p.timeout_ns};
  griddep_launch_dependents();  // the next kernel's set-up may overlap this kernel (it waits before touching memory)
#ifdef COMFUSE_TRACE
  if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) p.trace[62] = globaltimer_ns();  // kernel entry
#endif

  if (threadIdx.x == 0) {
    for (int s = 0; s < kRingSlots; ++s) {
      mbar_init(bar_full(s), 2);
      mbar_init(bar_empty(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_pfull(a), 1);
      mbar_init(bar_sfull(a), 2 * kB2bEpiWarps);   // one arrival per epilogue warp of both CTAs
      mbar_init(bar_sempty(a), 1);
      mbar_init(bar_ofull(a), 1);
      mbar_init(bar_oempty(a), 2 * kB2bEpiWarps);
    }
    mbar_init(bar_stats, 4);
    mbar_init(bar_stats + 8u, 4);
    mbar_init(bar_drain, 1);
    mbar_init(bar_pfree, 2 * kB2bEpiWarps);
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tensormap(&tmX);
    prefetch_tensormap(&tmW1);
    prefetch_tensormap(&tmW2);
    prefetch_tensormap(&tmO);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(s_tmem_base), 512);
    tmem_relinquish_alloc_permit_pair();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  cluster_sync_after_init();  // every CTA's barriers exist before any peer signals them
  const uint32_t tmem_base = *s_tmem_base;
  griddep_wait();  // the set-up above may overlap the previous kernel's tail; global memory is touched only below
  // TMEM columns: P slots at 0 and 128, O slots at 256 and 384
  auto ring_addr = [&](int s) { return smem_base + B2bSmem::OFF_RING + s * kSlotBytes; };
  auto s_addr = [&](int buf, int kb) { return smem_base + B2bSmem::OFF_S + (buf * 2 + kb) * kSlotBytes; };

  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      RingPos<RING> ring;
      bool ok = true;
      // one box into the current slot (a pair operand: signals the even CTA's full barrier)
      int bz = 0;  // batch coordinate of the current tile
      auto push = [&](const CUtensorMap* tm, int x, int y, int) {
        if (!ok) return;
        if (!mbar_wait<false>(bar_empty(ring.stage), ring.phase ^ 1u, w)) { ok = false; return; }
        const uint32_t full = map_to_cta(bar_full(ring.stage), leader);
        mbar_arrive_expect_tx_cluster(full, kSlotBytes);
        tma_load_3d_pair(ring_addr(ring.stage), tm, full, x, y, bz);
        ring.advance();
      };
      const int wcol = static_cast<int>(pm) * 64;  // this CTA's half of every 128-column weight chunk
      {
        // software-pipelined over tiles (see the UMMA lane): Q and K of tile t+1 go in before V of tile t
        // sub-tile k of this cluster = 256 source positions (`half`) of its (k / nhalf)-th row tile
        auto push_qk = [&](int k) {
          const int tile = cluster_id + (k / nhalf) * num_clusters, half = k % nhalf;
          bz = tile / p.mpairs;
          const int m0 = (tile - bz * p.mpairs) * 256 + static_cast<int>(pm) * 128;
          push(&tmX, 0, m0, 0);
          push(&tmX, 64, m0, 0);
          push(&tmW1, half * 256 + 0 * 128 + wcol, 0, 0);
          push(&tmW1, half * 256 + 1 * 128 + wcol, 0, 0);
        };
        if (nsub > 0) push_qk(0);
        for (int k = 0; k < nsub && ok; ++k) {
          if (k + 1 < nsub) push_qk(k + 1);
          const int tile = cluster_id + (k / nhalf) * num_clusters, half = k % nhalf;
          bz = tile / p.mpairs;
          push(&tmW2, wcol, half * 256 + 0 * 128, 0);
          push(&tmW2, wcol, half * 256 + 1 * 128, 0);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ UMMA issuer (even CTA)
    if (lane == 0 && pm == 0) {
      constexpr uint32_t idesc_ml1 = make_idesc_bf16(256, 128, false, true);
      constexpr uint32_t idesc_ml2 = make_idesc_bf16(256, 128, false, true);
      RingPos<RING> ring;
      uint32_t full_bits = 0;
      uint32_t sfull_uses[2] = {0, 0};
      uint32_t tile_it = 0;
      bool ok = true;
      auto wait_slot = [&]() {  // the next ring item is a pair operand: wait until both halves have landed
        if (!ok) return 0u;
        if (!mbar_wait<false>(bar_full(ring.stage), (full_bits >> ring.stage) & 1u, w)) { ok = false; return 0u; }
        full_bits ^= 1u << ring.stage;
        tcgen05_fence_after_sync();
        return ring_addr(ring.stage);
      };
      auto release_slot = [&](int stage) {
        umma_commit_pair_both(bar_empty(stage));
      };
      {
        // Software-pipelined over the cluster's tiles: the scores of tile t+1 (ML1) are issued as soon
        // as the epilogue has read the scores of tile t out of the P slots, BEFORE S.V of tile t (ML2), so that the
        // epilogue can go from the softmax of tile t straight to the softmax of tile t+1 while ML2(t) runs, and finds
        // O(t) complete when it comes back for the normalisation.
        auto ml1 = [&]() {  // P[0], P[1] = Q . Kt chunks 0, 1 of the next tile in the ring
          const int xs0 = ring.stage;
          const uint32_t x0 = wait_slot();
          ring.advance();
          const int xs1 = ring.stage;
          const uint32_t x1 = wait_slot();
          ring.advance();
          const uint64_t xdesc0 = make_smem_desc_sw128(x0, 16, 1024);
          const uint64_t xdesc1 = make_smem_desc_sw128(x1, 16, 1024);
          for (int j = 0; j < 2 && ok; ++j) {
            const int wstage = ring.stage;
            const uint32_t wa = wait_slot();
            ring.advance();
            if (!ok) return;
            const uint64_t wdesc = make_smem_desc_sw128(wa, 8192, 1024);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              umma_bf16_ss_pair(tmem_base + j * 128, (kk < 4 ? xdesc0 : xdesc1) + static_cast<uint64_t>((kk & 3) * 2),
                                wdesc + static_cast<uint64_t>(kk * 128), idesc_ml1, kk != 0 ? 1u : 0u);
            release_slot(wstage);
            umma_commit_pair_both(bar_pfull(j));
          }
          release_slot(xs0);
          release_slot(xs1);
        };
        if (nsub > 0) ml1();
        for (int k = 0; k < nsub && ok; ++k, ++tile_it) {
          const int obuf = tile_it & 1u;
          const uint32_t d_o = tmem_base + 256 + obuf * 128;
          if (k + 1 < nsub) {
            if (!mbar_wait<false>(bar_pfree, tile_it & 1u, w)) { ok = false; break; }  // the epilogue holds tile t's scores in registers
            tcgen05_fence_after_sync();
            ml1();
            if (!ok) break;
          }
          if (!mbar_wait<false>(bar_oempty(obuf), ((tile_it >> 1) & 1u) ^ 1u, w)) { ok = false; break; }
          tcgen05_fence_after_sync();
          for (int j = 0; j < 2 && ok; ++j) {  // O = S . V, two K halves of 128 source positions
            const int wstage = ring.stage;
            const uint32_t wa = wait_slot();
            ring.advance();
            if (!ok) break;
            if (!mbar_wait<false>(bar_sfull(j), sfull_uses[j] & 1u, w)) { ok = false; break; }
            ++sfull_uses[j];
            tcgen05_fence_after_sync();
            const uint64_t wdesc = make_smem_desc_sw128(wa, 8192, 1024);
            const uint64_t sdesc0 = make_smem_desc_sw128(s_addr(j, 0), 16, 1024);
            const uint64_t sdesc1 = make_smem_desc_sw128(s_addr(j, 1), 16, 1024);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              umma_bf16_ss_pair(d_o, (kk < 4 ? sdesc0 : sdesc1) + static_cast<uint64_t>((kk & 3) * 2), wdesc + static_cast<uint64_t>(kk * 128),
                                idesc_ml2, (j | kk) != 0 ? 1u : 0u);
            release_slot(wstage);
            umma_commit_pair_both(bar_sempty(j));
          }
          if (ok) {
            umma_commit_pair_both(bar_ofull(obuf));
          }
        }
      }
      umma_commit_pair(bar_drain);
      mbar_wait<false>(bar_drain, 0, w);
    }
  } else {
    // ------------------------------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;          // TMEM lane quarter: rows 32q .. 32q+31
    const int hh = (warp - 2) >> 2;  // which 32 columns of every 128-column chunk / of the 128 output columns
    const int row = q * 32 + lane;
    const int epi_tid = threadIdx.x - 64;
    const bool store_thread = epi_tid == 0;
    const uint32_t lane_sel = static_cast<uint32_t>(q * 32) << 16;
    const uint32_t ybuf = smem_base + B2bSmem::OFF_YBUF;
    const uint32_t sfull_leader = map_to_cta(bar_sfull(0), leader);
    const uint32_t oempty_leader = map_to_cta(bar_oempty(0), leader);
    const int kblk = hh >> 1;            // K block of S (and residual box) this thread's columns fall into
    const int chunk0 = (hh & 1) * 4;     // first of its four 16-byte chunks inside that 128-byte row
    RingPos<RING> ring;
    uint32_t puses[2] = {0, 0}, suses[2] = {0, 0};
    int xpar = 0;
    uint32_t xphase = 0;
#ifdef COMFUSE_TRACE
    int trace_ix = 0;
#define B2B_TRACE_POINT()                                                                                \
  do {                                                                                                   \
    if (p.trace && blockIdx.x == 0 && warp == 2 && lane == 0 && trace_ix < 60) p.trace[trace_ix++] = globaltimer_ns(); \
  } while (0)
#else
#define B2B_TRACE_POINT() do { } while (0)
#endif

    {
      // ================= software-pipelined over the cluster's tiles:
      //   softmax(t0) | softmax(t1) finish(t0) | softmax(t2) finish(t1) | ... | finish(last)
      // so that S.V of tile t (ML2) runs under the softmax of tile t+1 and the UMMA lane never waits for this epilogue
      // longer than one softmax.
      // ---------------- Epi1 (N1 = 256: the two P slots hold one whole score row): row max and sum of exponentials
      // across the two chunks and the four threads of the row, then S = bf16(2^(t - max)) as the next UMMAs' A operand;
      // returns 1 / (row sum), applied in the tile's finish step (O = (S.V) / sum)
      auto softmax_tile = [&]() -> float2 {
        for (int pb = 0; pb < 2; ++pb) {
          mbar_wait<false>(bar_pfull(pb), puses[pb] & 1u, w);
          ++puses[pb];
        }
        __syncwarp();
        tcgen05_fence_after_sync();
        B2B_TRACE_POINT();  // scores of the sub-tile complete
        const float sc = p.alpha * 1.4426950408889634f;  // log2 domain
        uint32_t v0[32], v1[32];
        tmem_ld_32cols(tmem_base + lane_sel + 0 * 128 + hh * 32, v0);
        tmem_ld_32cols(tmem_base + lane_sel + 1 * 128 + hh * 32, v1);
        // the scores are in registers: the P slots may take the next tile's scores
        tcgen05_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_noflush(map_to_cta(bar_pfree, leader));
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          mx0 = max3(mx0, __uint_as_float(v0[i]), __uint_as_float(v0[i + 1]));
          mx1 = max3(mx1, __uint_as_float(v1[i]), __uint_as_float(v1[i + 1]));
        }
        // sc > 0 is required (checked by the host): the maximum of the scaled scores is the scaled maximum
        const float mloc = fmaxf(mx0, mx1) * sc;
        float2 a0 = splat2(0.f), a1 = splat2(0.f);
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float2 d0 = fma2(f2_from_bits(v0[i], v0[i + 1]), splat2(sc), splat2(-mloc));
          const float2 d1 = fma2(f2_from_bits(v1[i], v1[i + 1]), splat2(sc), splat2(-mloc));
          // every other pair of the second chunk (a quarter of the scores) takes 2^x from the FMA-pipe polynomial (relative
          // error 4e-6): the MUFU unit is the busiest pipe of this loop (measured: a quarter 29.4 us on a1, none 30.1, half 30.3)
          const float2 e0 = make_float2(ex2_approx(d0.x), ex2_approx(d0.y));
          const float2 e1 = (i & 2) ? ex2_poly2(d1) : make_float2(ex2_approx(d1.x), ex2_approx(d1.y));
          v0[i] = __float_as_uint(e0.x); v0[i + 1] = __float_as_uint(e0.y);
          v1[i] = __float_as_uint(e1.x); v1[i + 1] = __float_as_uint(e1.y);
          a0 = add2(a0, e0);
          a1 = add2(a1, e1);
        }
        const float lloc = (a0.x + a0.y) + (a1.x + a1.y);
        const float2 tot = cluster_row_reduce<1, MergeMaxSumExp2, 4>(make_float2(mloc, lloc), 64.f, MergeMaxSumExp2(), s_pre, s_stats,
                                                                     bar_stats, row, hh, 0u, xpar, xphase, w);
        B2B_TRACE_POINT();  // exponentials done, row statistics merged
        const float f = ex2_approx(mloc - tot.x);  // this thread's exponentials are relative to its own maximum
        // the S buffers are free once ML2 of the previous tile has read them
        for (int pb = 0; pb < 2; ++pb) {
          mbar_wait<false>(bar_sempty(pb), (suses[pb] & 1u) ^ 1u, w);
          ++suses[pb];
        }
        __syncwarp();
        B2B_TRACE_POINT();  // S buffers free
#pragma unroll
        for (int pb = 0; pb < 2; ++pb) {
          const uint32_t(&vv)[32] = pb ? v1 : v0;
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2_rn(mul2(f2_from_bits(vv[2 * i], vv[2 * i + 1]), splat2(f)));
          const uint32_t sb = s_addr(pb, kblk);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t a = sb + swz128(row, chunk0 + i);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]),
                         "r"(pk[4 * i + 3])
                         : "memory");
          }
        }
        fence_proxy_async_smem();  // S writes are visible to the tensor core's shared-memory reads
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_cluster_noflush(sfull_leader);
          mbar_arrive_cluster_noflush(sfull_leader + 8u);
        }
        B2B_TRACE_POINT();  // S handed to the tensor pipe
        return tot;  // (row maximum in the log2 domain, sum of 2^(t - maximum)) of this sub-tile
      };
      // ---------------- Epi2: O = (S.V) / (row sum), rounded once, two 128 x 64 boxes staged and stored together
      // `it` = number of the row tile's first sub-tile; ml0 / ml1 = (maximum, sum) of its one or two sub-tiles
      auto finish_tile = [&](int tile, uint32_t it, float2 ml0, float2 ml1) {
        const int bz = tile / p.mpairs;
        const int m0 = (tile - bz * p.mpairs) * 256 + static_cast<int>(pm) * 128;
        uint32_t pk[16];
        if constexpr (NHALF == 1) {
          const int obuf = it & 1u;
          const float inv_l = ml0.y > 0.f ? 1.f / ml0.y : 0.f;
          mbar_wait<false>(bar_ofull(obuf), (it >> 1) & 1u, w);
          __syncwarp();
          tcgen05_fence_after_sync();
          B2B_TRACE_POINT();  // S.V of the tile complete
          uint32_t v[32];
          tmem_ld_32cols(tmem_base + lane_sel + 256 + obuf * 128 + hh * 32, v);
#pragma unroll
          for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2_rn(mul2(f2_from_bits(v[2 * i], v[2 * i + 1]), splat2(inv_l)));
          tcgen05_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster_noflush(oempty_leader + 8u * obuf);
        } else {
          // two sub-tiles, each exponentiated against its own maximum: O = (O0 2^(m0-m) + O1 2^(m1-m)) / (l0 2^(m0-m) + l1 2^(m1-m))
          const float mm = fmaxf(ml0.x, ml1.x);
          const float f0 = ml0.x == -INFINITY ? 0.f : ex2_approx(ml0.x - mm), f1 = ml1.x == -INFINITY ? 0.f : ex2_approx(ml1.x - mm);
          const float l = ml0.y * f0 + ml1.y * f1;
          const float inv_l = l > 0.f ? 1.f / l : 0.f;
          const float2 w0 = splat2(f0 * inv_l), w1 = splat2(f1 * inv_l);
          mbar_wait<false>(bar_ofull(0), (it >> 1) & 1u, w);  // `it` is even: slot 0 holds the first sub-tile's S.V, slot 1 the second's
          mbar_wait<false>(bar_ofull(1), (it >> 1) & 1u, w);
          __syncwarp();
          tcgen05_fence_after_sync();
          uint32_t v0[32], v1[32];
          tmem_ld_32cols(tmem_base + lane_sel + 256 + 0 * 128 + hh * 32, v0);
          tmem_ld_32cols(tmem_base + lane_sel + 256 + 1 * 128 + hh * 32, v1);
#pragma unroll
          for (int i = 0; i < 16; ++i)
            pk[i] = pack_bf16x2_rn(fma2(f2_from_bits(v1[2 * i], v1[2 * i + 1]), w1, mul2(f2_from_bits(v0[2 * i], v0[2 * i + 1]), w0)));
          tcgen05_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive_cluster_noflush(oempty_leader);
            mbar_arrive_cluster_noflush(oempty_leader + 8u);
          }
        }
        // both halves at once: columns 0..63 go to the staging box, columns 64..127 to the idle eighth ring slot
        if (store_thread) tma_store_wait_read<0>();  // the previous tile's stores have read both boxes
        named_barrier_sync(3, kB2bEpiThreads);
        {
          const uint32_t box = kblk == 0 ? ybuf : ring_addr(kRingSlots - 1);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t a = box + swz128(row, chunk0 + i);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]),
                         "r"(pk[4 * i + 3])
                         : "memory");
          }
        }
        fence_proxy_async_smem();
        named_barrier_sync(3, kB2bEpiThreads);
        if (store_thread) {
          tma_store_3d(&tmO, ybuf, 0, m0, bz);
          tma_store_3d(&tmO, ring_addr(kRingSlots - 1), 64, m0, bz);
          tma_store_commit();
        }
        B2B_TRACE_POINT();  // tile stored
      };
      // Order (the S buffers and the O slots are handed back by the steps named behind the arrows):
      //   one sub-tile per row tile:   softmax(0) | softmax(t+1), finish(t) ...
      //   two sub-tiles per row tile:  softmax(0), softmax(1) | softmax(2t+2), finish(t), softmax(2t+3) ...
      // (S.V of sub-tile 2t+2 needs O slot 0, which finish(t) releases; the softmax of 2t+3 needs the S buffers that
      // S.V of 2t+2 releases, so it must come behind finish(t).)
      float2 ml_a = make_float2(-INFINITY, 0.f), ml_b = ml_a;
      if (nsub > 0) ml_a = softmax_tile();
      if (nhalf == 2 && nsub > 1) ml_b = softmax_tile();
      for (int i = 0; i < my_tiles; ++i) {
        const int tile = cluster_id + i * num_clusters;
        const int first = i * nhalf;
        const float2 c0 = ml_a, c1 = ml_b;
        if constexpr (NHALF == 1) {
          if (first + 1 < nsub) ml_a = softmax_tile();
          finish_tile(tile, static_cast<uint32_t>(first), c0, c0);
        } else {
          if (first + 2 < nsub) ml_a = softmax_tile();
          finish_tile(tile, static_cast<uint32_t>(first), c0, c1);
          if (first + 3 < nsub) ml_b = softmax_tile();
        }
      }
    }
    if (store_thread) tma_store_wait_read<0>();  // the staging buffer must outlive the last store's read
  }

#ifdef COMFUSE_TRACE
  if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) p.trace[61] = globaltimer_ns();  // epilogue warps done
#endif
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after_sync();
    tmem_dealloc_pair(tmem_base, 512);
  }
#ifdef COMFUSE_TRACE
  if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) p.trace[63] = globaltimer_ns();  // kernel exit
#endif
}

}  // namespace

bool b2b_fused_supported(int K, int N1, int N2, int mode) {
  // attention form: 256 source positions fill the two P slots; 512 run as two sub-tiles combined at the normalisation
  if (mode == 1) return K == 128 && N2 == 128 && (N1 == 256 || N1 == 512);
  return b2b_mlp_supported(K, N1, N2);
}

cudaError_t launch_b2b_fused(const void* X, const void* W1, const void* W2, B2bParams p, cudaStream_t st) {
  const DeviceInfo* dev = current_device_info();
  if (!dev) return cudaErrorInvalidDevice;
  CUtensorMap tmX, tmW1, tmW2, tmO;
  const uint64_t M = p.M, K = p.K, N1 = p.N1, N2 = p.N2;
  if (p.batch < 1) p.batch = 1;
  const uint64_t nb = static_cast<uint64_t>(p.batch);  // dense [batch, rows, cols] tensors
  // all boxes are 64 elements x 128 rows
  if (!encode_tmap_bf16_3d(&tmX, X, K, M, nb, K * 2, M * K * 2, 128) ||
      !encode_tmap_bf16_3d(&tmW1, W1, N1, K, nb, N1 * 2, K * N1 * 2, 128) ||
      !encode_tmap_bf16_3d(&tmW2, W2, N2, N1, nb, N2 * 2, N1 * N2 * 2, 128) ||
      !encode_tmap_bf16_3d(&tmO, p.O, N2, M, nb, N2 * 2, M * N2 * 2, 128))
    return cudaErrorInvalidValue;
  p.mblocks = (p.M + 127) / 128;
  p.mpairs = (p.mblocks + 1) / 2;

  constexpr int kMaxDev = 64;
  static std::atomic<int> max_clusters[kMaxDev];  // 0 = kernel not configured yet on that device (set last, released)
  const int di = dev->device < kMaxDev ? dev->device : kMaxDev - 1;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.blockDim = dim3(kB2bThreads, 1, 1);
  cfg.dynamicSmemBytes = B2bSmem::BYTES;
  cfg.stream = st;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // set-up may overlap the previous kernel's tail
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic_launch_enabled() ? 2 : 1;
  int ncl = max_clusters[di].load(std::memory_order_acquire);
  if (ncl == 0) {
    cudaError_t e = cudaFuncSetAttribute(b2b_pair_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, B2bSmem::BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(b2b_pair_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, B2bSmem::BYTES);
    if (e != cudaSuccess) return e;
    int n = 0;
    cfg.gridDim = dim3(2 * dev->sm_count, 1, 1);
    e = cudaOccupancyMaxActiveClusters(&n, b2b_pair_kernel<1>, &cfg);
    if (e != cudaSuccess) return e;
    if (n <= 0) return cudaErrorLaunchOutOfResources;
    max_clusters[di].store(n, std::memory_order_release);
    ncl = n;
  }
  const int tiles = p.batch * p.mpairs;
  const int clusters = tiles < ncl ? tiles : ncl;
  cfg.gridDim = dim3(clusters * 2, 1, 1);
  count_launch();
  if (p.mode != 1) return cudaErrorInvalidValue;  // the MLP forms have kernels of their own
  return p.N1 == 512 ? cudaLaunchKernelEx(&cfg, b2b_pair_kernel<2>, tmX, tmW1, tmW2, tmO, p)
                     : cudaLaunchKernelEx(&cfg, b2b_pair_kernel<1>, tmX, tmW1, tmW2, tmO, p);
}

}  // namespace comfuse
