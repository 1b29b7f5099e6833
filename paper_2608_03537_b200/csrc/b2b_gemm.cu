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
constexpr int kB2bFinWarps = 4;                        // one per TMEM lane quarter: a thread per row normalises and stores O
constexpr int kMl2Warp = 2 + kB2bEpiWarps + kB2bFinWarps;  // its first lane issues S.V; the scores have a lane of their own (warp 1)
constexpr int kB2bThreads = 32 * (kMl2Warp + 1);       // producer, score UMMAs, softmax warps, finish warps, S.V UMMAs
constexpr int kSlotBytes = 128 * 64 * 2;  // one 128 x 64 bf16 box
constexpr int kRingSlots = 8;

struct B2bSmem {
  static constexpr int OFF_RING = 0;
  static constexpr int OFF_S = kRingSlots * kSlotBytes;            // 2 buffers x 2 K blocks
  static constexpr int OFF_YBUF = OFF_S + 4 * kSlotBytes;          // output staging box (the second one is the idle eighth ring slot)
  static constexpr int OFF_PRE = OFF_YBUF + kSlotBytes;            // float [2][4][128]: the row maxima of the four threads of a row
  static constexpr int OFF_ML = OFF_PRE + 2 * 4 * 128 * 4;         // float [4][5][128]: row maximum and four partial row sums of the last four sub-tiles
  static constexpr int OFF_BAR = OFF_ML + 4 * 5 * 128 * 4;
  // barriers: full[8] empty[8] (8 unused) pfull[2] sfull[2] sempty[2] ofull[2] oempty[2] stats[2] drain pfree drain2 lfull[4]
  static constexpr int NUM_BARS = 3 * kRingSlots + 10 + 4 + 5;
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;
  static constexpr int BYTES = OFF_MISC + 16 + 1024;
};
static_assert(B2bSmem::BYTES <= 232448, "shared memory budget");

// NHALF: sub-tiles of 256 source positions per score row, 1 or 2.  KM: the keys (W1) are stored [batch, N1, K], one key per
// row, and feed the score UMMAs as a K-major operand (two 64 x 64 boxes per slot: contraction elements 0..63 and 64..127 of
// this CTA's 64 keys); else [batch, K, N1], an MN-major operand (one 128 x 64 box per slot).  RAGGED: N1 is not NHALF * 256;
// scores of the source positions from N1 on (zeros: their keys were loaded out of bounds) are set to -inf before the softmax.
template <int NHALF, bool KM, bool RAGGED>
__global__ void __launch_bounds__(kB2bThreads, 1)
b2b_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW1,
                const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmO, const B2bParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t smem_base = smem_u32(smem);

  float* s_mx = reinterpret_cast<float*>(smem + B2bSmem::OFF_PRE);
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
  const uint32_t bar_pfree = bar_drain + 8u;  // both P slots read by every softmax warp (even CTA)
  const uint32_t bar_drain2 = bar_pfree + 8u;
  auto bar_lfull = [&](int a) { return bar_pfree + 16u + 8u * a; };  // row statistics of sub-tile k in slot k & 3 (this CTA)
  float* s_ml = reinterpret_cast<float*>(smem + B2bSmem::OFF_ML);
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
#ifdef COMFUSE_TRACE
#define B2B_TRACE_AT(ix) do { if (p.trace && blockIdx.x == 0) p.trace[ix] = globaltimer_ns(); } while (0)
#else
#define B2B_TRACE_AT(ix) do { } while (0)
#endif
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
      mbar_init(bar_oempty(a), 2 * kB2bFinWarps);
    }
    for (int a = 0; a < 4; ++a) mbar_init(bar_lfull(a), kB2bEpiWarps);
    mbar_init(bar_drain2, 1);
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
      // row-major keys: this CTA's 64 keys from `key0` on, as two boxes of 64 contraction elements each in one slot
      auto push_keys = [&](int key0) {
        if (!ok) return;
        if (!mbar_wait<false>(bar_empty(ring.stage), ring.phase ^ 1u, w)) { ok = false; return; }
        const uint32_t full = map_to_cta(bar_full(ring.stage), leader);
        mbar_arrive_expect_tx_cluster(full, kSlotBytes);
        tma_load_3d_pair(ring_addr(ring.stage), &tmW1, full, 0, key0, bz);
        tma_load_3d_pair(ring_addr(ring.stage) + kSlotBytes / 2, &tmW1, full, 64, key0, bz);
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
          if constexpr (KM) {
            push_keys(half * 256 + 0 * 128 + wcol);
            push_keys(half * 256 + 1 * 128 + wcol);
          } else {
            push(&tmW1, half * 256 + 0 * 128 + wcol, 0, 0);
            push(&tmW1, half * 256 + 1 * 128 + wcol, 0, 0);
          }
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
    // ------------------------------------------------------------------------------------------ score UMMAs (even CTA)
    // The scores and S.V have an issuing lane each, so that a wait of one (the S buffers, an O slot) never holds back the
    // other.  Both walk the same ring sequence, QK(0) | QK(k+1), V(k) ..., each taking its own items and stepping
    // over the other's; the barrier parity of a slot is the ring's wrap count, whoever used the slot last.  A lane that
    // steps over slots never saw their barriers complete, so each of its own waits must come behind an event that
    // implies the slot's PREVIOUS fill has landed and been consumed (else the parity test passes on the older phase):
    // here the scores of sub-tile k+1 wait for pfree(k) first, which lies behind S.V of sub-tile k-2 (the previous tenant
    // of their first slot); the other three slots' previous tenants are this lane's own.
    if (lane == 0 && pm == 0) {
      constexpr uint32_t idesc_ml1 = make_idesc_bf16(256, 128, false, !KM);
      RingPos<RING> ring;
      bool ok = true;
      auto wait_slot = [&]() {  // the next ring item is a pair operand: wait until both halves have landed
        if (!ok) return 0u;
        if (!mbar_wait<false>(bar_full(ring.stage), ring.phase, w)) { ok = false; return 0u; }
        tcgen05_fence_after_sync();
        return ring_addr(ring.stage);
      };
      auto release_slot = [&](int stage) { umma_commit_pair_both(bar_empty(stage)); };
      auto ml1 = [&]() {  // P[0], P[1] = Q . Kt chunks 0, 1 of the next sub-tile in the ring
        const int xs0 = ring.stage;
        const uint32_t x0 = wait_slot();
        ring.advance();
        const int xs1 = ring.stage;
        const uint32_t x1 = wait_slot();
        ring.advance();
        const uint64_t xdesc0 = make_smem_desc_sw128(x0, 16, 1024);
        const uint64_t xdesc1 = make_smem_desc_sw128(x1, 16, 1024);
        int wst[2] = {0, 0};
        for (int j = 0; j < 2 && ok; ++j) {
          const int wstage = ring.stage;
          const uint32_t wa = wait_slot();
          ring.advance();
          if (!ok) return;
          if constexpr (KM) {
            const uint64_t wdesc0 = make_smem_desc_sw128(wa, 16, 1024);
            const uint64_t wdesc1 = make_smem_desc_sw128(wa + kSlotBytes / 2, 16, 1024);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              umma_bf16_ss_pair(tmem_base + j * 128, (kk < 4 ? xdesc0 : xdesc1) + static_cast<uint64_t>((kk & 3) * 2),
                                (kk < 4 ? wdesc0 : wdesc1) + static_cast<uint64_t>((kk & 3) * 2), idesc_ml1, kk != 0 ? 1u : 0u);
          } else {
            const uint64_t wdesc = make_smem_desc_sw128(wa, 8192, 1024);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              umma_bf16_ss_pair(tmem_base + j * 128, (kk < 4 ? xdesc0 : xdesc1) + static_cast<uint64_t>((kk & 3) * 2),
                                wdesc + static_cast<uint64_t>(kk * 128), idesc_ml1, kk != 0 ? 1u : 0u);
          }
          wst[j] = wstage;
        }
        // one commit tells the softmax warps that both chunks are complete (it is the one on the critical path: the slots
        // are handed back behind it)
        if (ok) umma_commit_pair_both(bar_pfull(0));
        release_slot(wst[0]);
        release_slot(wst[1]);
        release_slot(xs0);
        release_slot(xs1);
      };
      if (nsub > 0) ml1();
      for (int k = 0; k < nsub && ok; ++k) {
        if (k + 1 < nsub) {
          // the softmax warps hold sub-tile k's scores in registers: the P slots take the scores of sub-tile k+1
          if (!mbar_wait<false>(bar_pfree, static_cast<uint32_t>(k) & 1u, w)) { ok = false; break; }
          tcgen05_fence_after_sync();
          if (k < 30) B2B_TRACE_AT(200 + 2 * k);
          ml1();
          if (k < 30) B2B_TRACE_AT(201 + 2 * k);
        }
        ring.skip(2);  // V(k) belongs to the other lane
      }
      umma_commit_pair(bar_drain);
      mbar_wait<false>(bar_drain, 0, w);
    }
  } else if (warp == kMl2Warp) {
    // ------------------------------------------------------------------------------------------ S.V UMMAs (even CTA)
    if (lane == 0 && pm == 0) {
      constexpr uint32_t idesc_ml2 = make_idesc_bf16(256, 128, false, true);
      RingPos<RING> ring;
      bool ok = true;
      auto wait_slot = [&]() {
        if (!ok) return 0u;
        if (!mbar_wait<false>(bar_full(ring.stage), ring.phase, w)) { ok = false; return 0u; }
        tcgen05_fence_after_sync();
        return ring_addr(ring.stage);
      };
      if (nsub > 0) ring.skip(4);  // QK(0)
      for (int k = 0; k < nsub && ok; ++k) {
        const uint32_t uk = static_cast<uint32_t>(k);
        const int obuf = k & 1;
        const uint32_t d_o = tmem_base + 256 + obuf * 128;
        if (k + 1 < nsub) ring.skip(4);  // QK(k+1)
        if (!mbar_wait<false>(bar_oempty(obuf), ((uk >> 1) & 1u) ^ 1u, w)) { ok = false; break; }
        tcgen05_fence_after_sync();
        if (k < 30) B2B_TRACE_AT(300 + 2 * k);
        for (int j = 0; j < 2 && ok; ++j) {  // O = S . V, two K halves of 128 source positions
          // S first, the V slot second.  A parity wait tells "the fill I expect has landed" from "the fill before it has not
          // even landed yet" only if this lane looks at the slot AFTER that earlier fill has completed; the earlier fill
          // of a V slot is a Q / K box of the same sub-tile (or this lane's own previous V box), which the score UMMAs
          // consumed before the softmax that has just handed S over could start.  Looked at earlier (at kernel start, say),
          // the wait would pass on an empty slot.
          if (!mbar_wait<false>(bar_sfull(j), uk & 1u, w)) { ok = false; break; }
          const int wstage = ring.stage;
          const uint32_t wa = wait_slot();
          ring.advance();
          if (!ok) break;
          tcgen05_fence_after_sync();
          const uint64_t wdesc = make_smem_desc_sw128(wa, 8192, 1024);
          const uint64_t sdesc0 = make_smem_desc_sw128(s_addr(j, 0), 16, 1024);
          const uint64_t sdesc1 = make_smem_desc_sw128(s_addr(j, 1), 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            umma_bf16_ss_pair(d_o, (kk < 4 ? sdesc0 : sdesc1) + static_cast<uint64_t>((kk & 3) * 2), wdesc + static_cast<uint64_t>(kk * 128),
                              idesc_ml2, (j | kk) != 0 ? 1u : 0u);
          umma_commit_pair_both(bar_empty(wstage));
          umma_commit_pair_both(bar_sempty(j));
        }
        if (ok) umma_commit_pair_both(bar_ofull(obuf));
        if (k < 30) B2B_TRACE_AT(301 + 2 * k);
      }
      umma_commit_pair(bar_drain2);
      mbar_wait<false>(bar_drain2, 0, w);
    }
  } else if (warp < 2 + kB2bEpiWarps) {
    // ------------------------------------------------------------------------------------------ softmax warps
    const int q = warp & 3;          // TMEM lane quarter: rows 32q .. 32q+31
    const int hh = (warp - 2) >> 2;  // which 32 columns of every 128-column chunk
    const int row = q * 32 + lane;
    const uint32_t lane_sel = static_cast<uint32_t>(q * 32) << 16;
    const uint32_t sfull_leader = map_to_cta(bar_sfull(0), leader);
    const int kblk = hh >> 1;            // K block of S this thread's columns fall into
    const int chunk0 = (hh & 1) * 4;     // first of its four 16-byte chunks inside that 128-byte row
    uint32_t puses[2] = {0, 0}, suses[2] = {0, 0};
    int xpar = 0;
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
      // One sub-tile after the other: the two P slots hold one whole score row of 256 source positions.  Row max and sum
      // of exponentials across the two chunks and the four threads of the row, then S = bf16(2^(t - max)) as the next
      // UMMAs' A operand.  S.V of sub-tile k runs under the softmax of sub-tile k+1; the division by the row sum is the
      // finish warps' work.
      auto softmax_tile = [&](int k) {
        mbar_wait<false>(bar_pfull(0), puses[0] & 1u, w);  // both chunks: the score lane commits once per sub-tile
        ++puses[0];
        __syncwarp();
        tcgen05_fence_after_sync();
        B2B_TRACE_POINT();  // scores of the sub-tile complete
        const float sc = p.alpha * 1.4426950408889634f;  // log2 domain
        uint32_t v0[32], v1[32];
        tmem_ld_32cols(tmem_base + lane_sel + 0 * 128 + hh * 32, v0);
        tmem_ld_32cols(tmem_base + lane_sel + 1 * 128 + hh * 32, v1);
        // the scores are in registers: the P slots may take the next sub-tile's scores
        tcgen05_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_noflush(map_to_cta(bar_pfree, leader));
        {
          // A source length that is not a multiple of 256: the keys from N1 on read as zeros (the loads fill outside the
          // tensor), their scores count as -inf -- 2^(-inf - m) = 0 goes into S for them, and nothing into the row sum.
          // The thread's two blocks of 32 columns are the same for every row: the test is uniform over the warp.
          const int key0 = (k % nhalf) * 256 + hh * 32;
          const int nv0 = p.N1 - key0, nv1 = p.N1 - (key0 + 128);
          if (RAGGED && nv0 < 32) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i >= nv0) v0[i] = 0xFF800000u;
          }
          if (RAGGED && nv1 < 32) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i >= nv1) v1[i] = 0xFF800000u;
          }
        }
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          mx0 = max3(mx0, __uint_as_float(v0[i]), __uint_as_float(v0[i + 1]));
          mx1 = max3(mx1, __uint_as_float(v1[i]), __uint_as_float(v1[i + 1]));
        }
        // The row maximum first (the four threads of a row sit in the four warps of one lane quarter: shared memory and a
        // barrier of those 128 threads), so that the exponentials come out against the final maximum and go straight
        // into S; the row SUM is not needed here at all, the finish warps add the four partial sums.
        // sc > 0 is required (checked by the host): the maximum of the scaled scores is the scaled maximum.
        s_mx[(xpar * 4 + hh) * 128 + row] = fmaxf(mx0, mx1) * sc;
        named_barrier_sync(1 + q, 128);
        const float m = fmaxf(fmaxf(s_mx[(xpar * 4 + 0) * 128 + row], s_mx[(xpar * 4 + 1) * 128 + row]),
                              fmaxf(s_mx[(xpar * 4 + 2) * 128 + row], s_mx[(xpar * 4 + 3) * 128 + row]));
        xpar ^= 1;  // the write after next comes behind the next barrier, which every reader of this buffer passes first
        B2B_TRACE_POINT();  // row maximum known
        float2 acc = splat2(0.f);
#pragma unroll
        for (int pb = 0; pb < 2; ++pb) {
          uint32_t(&vv)[32] = pb ? v1 : v0;
          // S buffer pb is free once S.V of the previous sub-tile has read it
          mbar_wait<false>(bar_sempty(pb), (suses[pb] & 1u) ^ 1u, w);
          ++suses[pb];
          __syncwarp();
          if (pb == 0) B2B_TRACE_POINT();  // first S buffer free
          const uint32_t sb = s_addr(pb, kblk);
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint32_t pk[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int i = 8 * g + 2 * j;
              const float2 d = fma2(f2_from_bits(vv[i], vv[i + 1]), splat2(sc), splat2(-m));
              // all exponentials on the MUFU unit: with the row maximum known beforehand the loop has no rescaling left,
              // and moving a share of them to an FMA-pipe polynomial no longer pays (measured on the target-attention
              // shape: none 23.7 us, an eighth 23.9, a quarter 24.5, a half 26.6)
              const float2 e = make_float2(ex2_approx(d.x), ex2_approx(d.y));
              acc = add2(acc, e);
              pk[j] = pack_bf16x2_rn(e);
            }
            const uint32_t a = sb + swz128(row, chunk0 + g);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
          }
          fence_proxy_async_smem();  // S writes are visible to the tensor core's shared-memory reads
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster_noflush(sfull_leader + 8u * pb);  // S.V may start on this half
        }
        // (maximum in the log2 domain, partial sum of 2^(t - maximum)) of this sub-tile for the finish warps; the slot's
        // previous tenant, sub-tile k-4, was read before the O slot that S.V of sub-tile k-1 needed was handed back
        float* ml = s_ml + (k & 3) * 5 * 128;
        if (hh == 0) ml[row] = m;
        ml[(1 + hh) * 128 + row] = acc.x + acc.y;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_lfull(k & 3));
        B2B_TRACE_POINT();  // S handed to the tensor pipe
      };
      for (int k = 0; k < nsub; ++k) softmax_tile(k);
    }
  } else if (warp < kMl2Warp) {
    // ------------------------------------------------------------------------------------------ finish warps
    // O = (S.V) / (row sum), rounded once: a thread per row walks the 128 output columns in four blocks, stages its warp's
    // 32 rows in the two output boxes (columns 0..63 in the staging box, 64..127 in the idle eighth ring slot) and stores
    // them, while the softmax warps are already on the next sub-tile.
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const uint32_t lane_sel = static_cast<uint32_t>(q * 32) << 16;
    const uint32_t oempty_leader = map_to_cta(bar_oempty(0), leader);
    const uint32_t box0 = smem_base + B2bSmem::OFF_YBUF, box1 = ring_addr(kRingSlots - 1);
    auto stage_block = [&](int cb, const uint32_t (&pk)[16]) {
      const uint32_t box = cb < 2 ? box0 : box1;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t a = box + swz128(row, (cb & 1) * 4 + i);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]),
                     "r"(pk[4 * i + 3])
                     : "memory");
      }
    };
    for (int i = 0; i < my_tiles; ++i) {
      const int tile = cluster_id + i * num_clusters;
      const uint32_t k0 = static_cast<uint32_t>(i * nhalf);  // the row tile's first sub-tile
      const int bz = tile / p.mpairs;
      const int m0 = (tile - bz * p.mpairs) * 256 + static_cast<int>(pm) * 128;
      if (lane == 0) tma_store_wait_read<0>();  // the previous tile's stores have read this warp's rows of both boxes
      __syncwarp();
      if constexpr (NHALF == 1) {
        const int obuf = k0 & 1u;
        mbar_wait<false>(bar_lfull(k0 & 3u), (k0 >> 2) & 1u, w);
        const float* ml = s_ml + (k0 & 3u) * 5 * 128 + row;
        const float l = (ml[128] + ml[256]) + (ml[384] + ml[512]);
        const float inv_l = l > 0.f ? 1.f / l : 0.f;
        if (warp == 2 + kB2bEpiWarps && lane == 0 && i < 20) B2B_TRACE_AT(100 + 3 * i);
        mbar_wait<false>(bar_ofull(obuf), (k0 >> 1) & 1u, w);
        __syncwarp();
        tcgen05_fence_after_sync();
        if (warp == 2 + kB2bEpiWarps && lane == 0 && i < 20) B2B_TRACE_AT(101 + 3 * i);
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t v[32], pk[16];
          tmem_ld_32cols(tmem_base + lane_sel + 256 + obuf * 128 + cb * 32, v);
#pragma unroll
          for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2_rn(mul2(f2_from_bits(v[2 * j], v[2 * j + 1]), splat2(inv_l)));
          stage_block(cb, pk);
        }
        tcgen05_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_noflush(oempty_leader + 8u * obuf);
      } else {
        // two sub-tiles, each exponentiated against its own maximum: O = (O0 2^(m0-m) + O1 2^(m1-m)) / (l0 2^(m0-m) + l1 2^(m1-m));
        // k0 is even: slot 0 holds the first sub-tile's S.V, slot 1 the second's
        mbar_wait<false>(bar_lfull(k0 & 3u), (k0 >> 2) & 1u, w);
        mbar_wait<false>(bar_lfull((k0 + 1u) & 3u), (k0 >> 2) & 1u, w);
        const float* pa = s_ml + (k0 & 3u) * 5 * 128 + row;
        const float* pb = s_ml + ((k0 + 1u) & 3u) * 5 * 128 + row;
        const float2 ml0 = make_float2(pa[0], (pa[128] + pa[256]) + (pa[384] + pa[512]));
        const float2 ml1 = make_float2(pb[0], (pb[128] + pb[256]) + (pb[384] + pb[512]));
        const float mm = fmaxf(ml0.x, ml1.x);
        const float f0 = ml0.x == -INFINITY ? 0.f : ex2_approx(ml0.x - mm), f1 = ml1.x == -INFINITY ? 0.f : ex2_approx(ml1.x - mm);
        const float l = ml0.y * f0 + ml1.y * f1;
        const float inv_l = l > 0.f ? 1.f / l : 0.f;
        const float2 w0 = splat2(f0 * inv_l), w1 = splat2(f1 * inv_l);
        mbar_wait<false>(bar_ofull(0), (k0 >> 1) & 1u, w);
        mbar_wait<false>(bar_ofull(1), (k0 >> 1) & 1u, w);
        __syncwarp();
        tcgen05_fence_after_sync();
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t v0[32], v1[32], pk[16];
          tmem_ld_32cols(tmem_base + lane_sel + 256 + 0 * 128 + cb * 32, v0);
          tmem_ld_32cols(tmem_base + lane_sel + 256 + 1 * 128 + cb * 32, v1);
#pragma unroll
          for (int j = 0; j < 16; ++j)
            pk[j] = pack_bf16x2_rn(fma2(f2_from_bits(v1[2 * j], v1[2 * j + 1]), w1, mul2(f2_from_bits(v0[2 * j], v0[2 * j + 1]), w0)));
          stage_block(cb, pk);
        }
        tcgen05_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_cluster_noflush(oempty_leader);
          mbar_arrive_cluster_noflush(oempty_leader + 8u);
        }
      }
      fence_proxy_async_smem();  // the staged rows are visible to the TMA store
      __syncwarp();
      if (warp == 2 + kB2bEpiWarps && lane == 0 && i < 20) B2B_TRACE_AT(102 + 3 * i);
      if (lane == 0 && COMFUSE_IN_BOUNDS(m0 >= 0 && m0 + q * 32 < p.mpairs * 256 && bz >= 0 && bz < p.batch, p.status)) {
        tma_store_3d(&tmO, box0 + q * 4096, 0, m0 + q * 32, bz);
        tma_store_3d(&tmO, box1 + q * 4096, 64, m0 + q * 32, bz);
        tma_store_commit();
      }
    }
    if (warp == 2 + kB2bEpiWarps && lane == 0) B2B_TRACE_AT(192);
    if (lane == 0) tma_store_wait_read<0>();  // the staging boxes must outlive the last store's read
    if (warp == 2 + kB2bEpiWarps && lane == 0) B2B_TRACE_AT(193);
  }

#ifdef COMFUSE_TRACE
  if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) p.trace[61] = globaltimer_ns();  // epilogue warps done
#endif
  tcgen05_fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 64) B2B_TRACE_AT(190);
  cluster_sync_all();
  if (threadIdx.x == 64) B2B_TRACE_AT(191);
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
  // (any source length up to 512 that is a multiple of 8: the positions from N1 on are masked)
  if (mode == 1) return K == 128 && N2 == 128 && N1 >= 8 && N1 <= 512 && N1 % 8 == 0;
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
      !(p.keys_row_major ? encode_tmap_bf16_3d(&tmW1, W1, K, N1, nb, K * 2, N1 * K * 2, 64)   // [batch, N1, K]: 64 keys x 64 elements
                         : encode_tmap_bf16_3d(&tmW1, W1, N1, K, nb, N1 * 2, K * N1 * 2, 128)) ||
      !encode_tmap_bf16_3d(&tmW2, W2, N2, N1, nb, N2 * 2, N1 * N2 * 2, 128) ||
      !encode_tmap_bf16_3d(&tmO, p.O, N2, M, nb, N2 * 2, M * N2 * 2, 32))  // a finish warp stores its 32 rows
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
    cudaError_t e = cudaSuccess;
    for (void (*k)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, B2bParams) :
         {b2b_pair_kernel<1, false, false>, b2b_pair_kernel<2, false, false>, b2b_pair_kernel<1, true, false>,
          b2b_pair_kernel<2, true, false>, b2b_pair_kernel<1, false, true>, b2b_pair_kernel<2, false, true>,
          b2b_pair_kernel<1, true, true>, b2b_pair_kernel<2, true, true>}) {
      e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, B2bSmem::BYTES);
      if (e != cudaSuccess) return e;
    }
    int n = 0;
    cfg.gridDim = dim3(2 * dev->sm_count, 1, 1);
    e = cudaOccupancyMaxActiveClusters(&n, b2b_pair_kernel<1, false, false>, &cfg);
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
  const bool two = p.N1 > 256, ragged = p.N1 % 256 != 0;
  auto go = [&](auto kern) { return cudaLaunchKernelEx(&cfg, kern, tmX, tmW1, tmW2, tmO, p); };
  if (p.keys_row_major) {
    if (ragged) return two ? go(b2b_pair_kernel<2, true, true>) : go(b2b_pair_kernel<1, true, true>);
    return two ? go(b2b_pair_kernel<2, true, false>) : go(b2b_pair_kernel<1, true, false>);
  }
  if (ragged) return two ? go(b2b_pair_kernel<2, false, true>) : go(b2b_pair_kernel<1, false, true>);
  return two ? go(b2b_pair_kernel<2, false, false>) : go(b2b_pair_kernel<1, false, false>);
}

}  // namespace comfuse
