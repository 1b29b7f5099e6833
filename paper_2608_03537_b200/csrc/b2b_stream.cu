// Fused back-to-back GEMM whose FIRST contraction streams K (Sec. 4, Eq. 2):
//   P = X W1,  S = ReLU(P + b1),  O = ReLU(S W2 + b2)          X [M, K], W1 [K, N1], W2 [N1, 128]
// the two-layer MLP form of the paper's DLRM workload (Sec. 6.2: 1024 -> 512 -> 128).  Neither P nor S is written to
// global memory.
//
// Where it differs from the K = 128 kernel (b2b_gemm.cu): there a P chunk costs eight UMMAs, here it costs K / 16 of them,
// so N1 is cut into HALVES of 256 columns (one UMMA N) and tensor memory into two slots of 256 columns.  One CTA pair
// (cta_group::2) owns 256 rows.  The output is staged in the S buffer, idle between the tile's last ML2 and the next Epi1.
//
// N1 = 512, both halves in LOCK-STEP (default): a ring stage (48 KB, three stages) holds one K block of X and this CTA's
// 128 columns of W1 for BOTH halves; the X block in shared memory feeds the UMMAs of half 0 (slot 0) and half 1 (slot 1), so X
// is streamed once and the MainLoop needs 109 B/clk of shared-memory traffic instead of 128.  Then Epi1(0) -> ML2(0),
// Epi1(1) -> ML2(1) with O in the first 128 columns of slot 0 (read out by Epi1(0) before S of half 0 exists), Epi2; the next
// tile's MainLoop waits for both slots, i.e. the epilogue of a tile is exposed, which the faster MainLoop more than pays for.
//
// N1 = 256 (and N1 = 512 with COMFUSE_B2B_STREAM_LOCK=0), ALTERNATING slots: the slots change roles -- half 0 of tile t ->
// slot s0 = t & 1, half 1 -> the other slot; once Epi1 has read half 0 out of s0, O(t) accumulates in the first 128 columns of
// s0; tile t+1 starts in the slot that held half 1 of tile t.  Per unit u = (tile, half) the UMMA lane issues
//   ML1(u) first K blocks | ML2(u - 1) | ML1(u) remaining K blocks
// so that Epi1(u - 1) (bias, ReLU, bf16, swizzled A operand in shared memory) has half a MainLoop to finish before the
// tensor pipe asks for S, and S needs one shared-memory buffer only (Sec. 4.3's staggered pipeline with the second
// MainLoop folded into the first one's stream).  The epilogue warps run Epi2(t - 1), Epi1(t, 0), Epi1(t, 1), ...
// Ring (Sec. 4.2, unified circular buffer): five stages of 32 KB in consumption order; an ML1 stage holds one K block of X
// (128 rows x 64) and of this CTA's 128 columns of W1 (two 64 x 64 boxes), an ML2 stage this CTA's 64 columns of the
// 256 W2 rows of a half (in both schedules).
#include <cuda_runtime.h>

#include <atomic>

#include <cstdlib>

#include "b2b_params.h"
#include "fused_pair.cuh"
#include "host_common.h"
#include "sm100_primitives.cuh"

namespace comfuse {

namespace {

constexpr int kEpiWarps = 16;  // four per TMEM lane quarter
constexpr int kEpiThreads = 32 * kEpiWarps;
constexpr int kThreads = 32 * (2 + kEpiWarps);  // producer, UMMA, epilogue warps
constexpr int kBoxBytes = 128 * 64 * 2;         // one 128 x 64 bf16 box
// LOCK (N1 = 512): both halves of P are computed in lock-step from ONE copy of the X block (a stage = X block + the W1
// blocks of both halves, 48 KB; three stages); otherwise a stage is 32 KB and there are five.
template <bool LOCK>
struct StreamSmem {
  static constexpr int kStages = LOCK ? 3 : 5;
  static constexpr int kStageBytes = LOCK ? 3 * kBoxBytes : 2 * kBoxBytes;
  static constexpr int OFF_RING = 0;
  static constexpr int OFF_S = kStages * kStageBytes;  // four K blocks of S; the output staging boxes live in the first two
  static constexpr int OFF_B1 = OFF_S + 4 * kBoxBytes;  // bf16 [512]
  static constexpr int OFF_B2 = OFF_B1 + 512 * 2;       // bf16 [128]
  static constexpr int OFF_BAR = OFF_B2 + 128 * 2;
  // barriers: full[kStages] empty[kStages] pfull[2] pfree[2] sfull sempty ofull drain
  static constexpr int NUM_BARS = 2 * kStages + 8;
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;
  static constexpr int BYTES = OFF_MISC + 16 + 1024;
};
static_assert(StreamSmem<false>::BYTES <= 232448 && StreamSmem<true>::BYTES <= 232448, "shared memory budget");

template <bool LOCK>
__global__ void __launch_bounds__(kThreads, 1)
b2b_stream_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW1,
                  const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmO, const B2bParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t smem_base = smem_u32(smem);
  using Smem = StreamSmem<LOCK>;
  constexpr int kStages = Smem::kStages;
  constexpr int kStageBytes = Smem::kStageBytes;

  uint16_t* s_b1 = reinterpret_cast<uint16_t*>(smem + Smem::OFF_B1);
  uint16_t* s_b2 = reinterpret_cast<uint16_t*>(smem + Smem::OFF_B2);
  const uint32_t bar_base = smem_base + Smem::OFF_BAR;
  auto bar_full = [&](int s) { return bar_base + 8u * s; };               // stage landed in both CTAs (even CTA)
  auto bar_empty = [&](int s) { return bar_base + 8u * (kStages + s); };  // stage read by the tensor pipe
  auto bar_pfull = [&](int a) { return bar_base + 8u * (2 * kStages + a); };      // P half complete in slot a
  auto bar_pfree = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };  // slot a read by both CTAs (even CTA)
  const uint32_t bar_sfull = bar_base + 8u * (2 * kStages + 4);   // S written by both CTAs (even CTA)
  const uint32_t bar_sempty = bar_sfull + 8u;                     // S read by ML2
  const uint32_t bar_ofull = bar_sfull + 16u;                     // O of a tile complete
  const uint32_t bar_drain = bar_sfull + 24u;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(smem + Smem::OFF_MISC);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + Smem::OFF_MISC + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // cluster of exactly two CTAs
  const uint32_t pm = rank & 1u;
  const uint32_t leader = 0u;
  const int cluster_id = blockIdx.x >> 1;
  const int num_clusters = gridDim.x >> 1;
  const int KB = (p.K + 63) / 64;   // K blocks of ML1 (the last one zero-filled past K)
  const int KBa = (KB + 1) / 2;     // ML2 of the previous unit is issued behind this many of them
  const int NH = (p.N1 + 255) / 256;  // halves of N1: 1 or 2; hidden columns past N1 load as zeros and stay zero (ReLU(0 + 0))
  const int total_tiles = p.mpairs;
  const int my_tiles = cluster_id < total_tiles ? (total_tiles - cluster_id + num_clusters - 1) / num_clusters : 0;
  const int nunits = my_tiles * NH;
  const WaitCtx w{s_abort, p.status, p.timeout_ns};
  griddep_launch_dependents();

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full(s), 2);
      mbar_init(bar_empty(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_pfull(a), 1);
      mbar_init(bar_pfree(a), 2 * kEpiWarps);  // one arrival per epilogue warp of both CTAs
    }
    mbar_init(bar_sfull, 2 * kEpiWarps);
    mbar_init(bar_sempty, 1);
    mbar_init(bar_ofull, 1);
    mbar_init(bar_drain, 1);
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
  griddep_wait();  // global memory is touched only below
  auto ring_addr = [&](int s) { return smem_base + Smem::OFF_RING + s * kStageBytes; };
  const uint32_t s_base = smem_base + Smem::OFF_S;
  // unit u of this cluster = half (u % NH) of its (u / NH)-th tile; P of that half goes to slot ((u / NH) & 1) ^ half,
  // O of the tile to the first 128 columns of slot (u / NH) & 1
  auto tile_m0 = [&](int it) { return (cluster_id + it * num_clusters) * 256 + static_cast<int>(pm) * 128; };

  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      RingPos<kStages> ring;
      bool ok = true;
      auto next_stage = [&](uint32_t& sa, uint32_t& full, uint32_t bytes) {
        if (!ok) return false;
        if (!mbar_wait<false>(bar_empty(ring.stage), ring.phase ^ 1u, w)) { ok = false; return false; }
        sa = ring_addr(ring.stage);
        full = map_to_cta(bar_full(ring.stage), leader);
        mbar_arrive_expect_tx_cluster(full, bytes);
        ring.advance();
        return true;
      };
      auto push_ml1 = [&](int m0, int h, int kb) {
        uint32_t sa, full;
        if (!next_stage(sa, full, kStageBytes)) return;
        const int n0 = h * 256 + static_cast<int>(pm) * 128;  // this CTA's half of the UMMA's 256 columns
        tma_load_3d_pair(sa, &tmX, full, kb * 64, m0, 0);
        tma_load_3d_pair(sa + kBoxBytes, &tmW1, full, n0, kb * 64, 0);
        tma_load_3d_pair(sa + kBoxBytes + 8192, &tmW1, full, n0 + 64, kb * 64, 0);
        if (LOCK) {  // the same columns of the second half behind them
          tma_load_3d_pair(sa + 2 * kBoxBytes, &tmW1, full, n0 + 256, kb * 64, 0);
          tma_load_3d_pair(sa + 2 * kBoxBytes + 8192, &tmW1, full, n0 + 256 + 64, kb * 64, 0);
        }
      };
      auto push_w2 = [&](int h) {
        uint32_t sa, full;
        if (!next_stage(sa, full, 2 * kBoxBytes)) return;
        const int c0 = static_cast<int>(pm) * 64;  // this CTA's half of the 128 output columns
        tma_load_3d_pair(sa, &tmW2, full, c0, h * 256, 0);
        tma_load_3d_pair(sa + kBoxBytes, &tmW2, full, c0, h * 256 + 128, 0);
      };
      if constexpr (LOCK) {
        for (int it = 0; it < my_tiles && ok; ++it) {
          const int m0 = tile_m0(it);
          for (int kb = 0; kb < KB; ++kb) push_ml1(m0, 0, kb);
          push_w2(0);
          push_w2(1);
        }
      } else {
        for (int u = 0; u < nunits && ok; ++u) {
          const int m0 = tile_m0(u / NH), h = u % NH;
          for (int kb = 0; kb < KBa; ++kb) push_ml1(m0, h, kb);
          if (u > 0) push_w2((u - 1) % NH);
          for (int kb = KBa; kb < KB; ++kb) push_ml1(m0, h, kb);
        }
        if (nunits > 0) push_w2((nunits - 1) % NH);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ UMMA issuer (even CTA)
    if (lane == 0 && pm == 0) {
      constexpr uint32_t idesc_ml1 = make_idesc_bf16(256, 256, false, true);
      constexpr uint32_t idesc_ml2 = make_idesc_bf16(256, 128, false, true);
      RingPos<kStages> ring;
      uint32_t full_bits = 0, slot_uses[2] = {0, 0}, sfull_uses = 0;
      bool ok = true;
      auto wait_stage = [&]() {
        if (!ok) return 0u;
        if (!mbar_wait<false>(bar_full(ring.stage), (full_bits >> ring.stage) & 1u, w)) { ok = false; return 0u; }
        full_bits ^= 1u << ring.stage;
        tcgen05_fence_after_sync();
        return ring_addr(ring.stage);
      };
      auto release_stage = [&]() {
        umma_commit_pair_both(bar_empty(ring.stage));
        ring.advance();
      };
      auto ml1_blocks = [&](uint32_t d_p, int kb0, int kb1) {
        for (int kb = kb0; kb < kb1 && ok; ++kb) {
          const uint32_t sa = wait_stage();
          if (!ok) return;
          const uint64_t adesc = make_smem_desc_sw128(sa, 16, 1024);
          const uint64_t bdesc = make_smem_desc_sw128(sa + kBoxBytes, /*next 64-column block*/ 8192, /*next 8 K rows*/ 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_bf16_ss_pair(d_p, adesc + static_cast<uint64_t>(k * 2), bdesc + static_cast<uint64_t>(k * 128), idesc_ml1,
                              (kb | k) != 0 ? 1u : 0u);
          release_stage();
        }
      };
      auto ml2 = [&](int u) {  // O(tile of u) (+)= S(u) . W2[half of u]
        const uint32_t sa = wait_stage();
        if (!ok) return;
        if (!mbar_wait<false>(bar_sfull, sfull_uses & 1u, w)) { ok = false; return; }
        ++sfull_uses;
        tcgen05_fence_after_sync();
        const int it = u / NH, h = u % NH;
        const uint32_t d_o = tmem_base + static_cast<uint32_t>(LOCK ? 0 : (it & 1) * 256);
        const uint64_t wdesc = make_smem_desc_sw128(sa, 8192, 1024);
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const uint64_t sdesc = make_smem_desc_sw128(s_base + (k >> 2) * kBoxBytes, 16, 1024) + static_cast<uint64_t>((k & 3) * 2);
          umma_bf16_ss_pair(d_o, sdesc, wdesc + static_cast<uint64_t>(k * 128), idesc_ml2, (h | k) != 0 ? 1u : 0u);
        }
        release_stage();
        umma_commit_pair_both(bar_sempty);
        if (h == NH - 1) {
          umma_commit_pair_both(bar_ofull);
        }
      };
      if constexpr (LOCK) {
        // both halves in lock-step: the X block of a stage feeds the UMMAs of half 0 (slot 0) and of half 1 (slot 1); the tile's
        // two ML2s follow its MainLoop, O in the first 128 columns of slot 0 (read out by Epi1 before S of half 0 exists)
        for (int it = 0; it < my_tiles && ok; ++it) {
          for (int slot = 0; slot < 2 && ok; ++slot) {
            if (slot_uses[slot] > 0 && !mbar_wait<false>(bar_pfree(slot), (slot_uses[slot] - 1u) & 1u, w)) ok = false;
            ++slot_uses[slot];
          }
          if (!ok) break;
          tcgen05_fence_after_sync();
          for (int kb = 0; kb < KB && ok; ++kb) {
            const uint32_t sa = wait_stage();
            if (!ok) break;
            const uint64_t adesc = make_smem_desc_sw128(sa, 16, 1024);
            const uint64_t bdesc0 = make_smem_desc_sw128(sa + kBoxBytes, 8192, 1024);
            const uint64_t bdesc1 = make_smem_desc_sw128(sa + 2 * kBoxBytes, 8192, 1024);
            if (kb + 1 < KB) {
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const uint32_t acc = (kb | k) != 0 ? 1u : 0u;
                umma_bf16_ss_pair(tmem_base, adesc + static_cast<uint64_t>(k * 2), bdesc0 + static_cast<uint64_t>(k * 128), idesc_ml1, acc);
                umma_bf16_ss_pair(tmem_base + 256, adesc + static_cast<uint64_t>(k * 2), bdesc1 + static_cast<uint64_t>(k * 128), idesc_ml1, acc);
              }
            } else {
              // last K block: half 0 first, so that its epilogue starts while the tensor pipe finishes half 1
#pragma unroll
              for (int half = 0; half < 2; ++half) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                  umma_bf16_ss_pair(tmem_base + half * 256, adesc + static_cast<uint64_t>(k * 2),
                                    (half ? bdesc1 : bdesc0) + static_cast<uint64_t>(k * 128), idesc_ml1, (kb | k) != 0 ? 1u : 0u);
                umma_commit_pair_both(bar_pfull(half));
              }
            }
            release_stage();
          }
          if (!ok) break;
          ml2(2 * it);
          ml2(2 * it + 1);
        }
      }
      for (int u = 0; !LOCK && u < nunits && ok; ++u) {
        const int it = u / NH, h = u % NH;
        const int slot = (it & 1) ^ h;
        // the slot's previous content (a P half read by Epi1, or an O read by Epi2) has been read by both CTAs
        if (slot_uses[slot] > 0) {
          if (!mbar_wait<false>(bar_pfree(slot), (slot_uses[slot] - 1u) & 1u, w)) { ok = false; break; }
          tcgen05_fence_after_sync();
        }
        ++slot_uses[slot];
        const uint32_t d_p = tmem_base + static_cast<uint32_t>(slot * 256);
        ml1_blocks(d_p, 0, KBa);
        if (u > 0) ml2(u - 1);
        ml1_blocks(d_p, KBa, KB);
        if (ok) {
          umma_commit_pair_both(bar_pfull(slot));
        }
      }
      if (!LOCK && nunits > 0 && ok) ml2(nunits - 1);
      umma_commit_pair(bar_drain);  // nothing may still be writing either CTA's TMEM when it is freed
      mbar_wait<false>(bar_drain, 0, w);
    }
  } else {
    // ------------------------------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;          // TMEM lane quarter: rows 32q .. 32q+31
    const int hh = (warp - 2) >> 2;  // Epi1: K block of S (64 columns of the half); Epi2: 32 of the 128 output columns
    const int row = q * 32 + lane;
    const int epi_tid = threadIdx.x - 64;
    const bool store_thread = epi_tid == 0;
    for (int i = epi_tid; i < 512; i += kEpiThreads) s_b1[i] = (p.b1 && i < p.N1) ? p.b1[i] : static_cast<uint16_t>(0);
    for (int i = epi_tid; i < 128; i += kEpiThreads) s_b2[i] = p.b2 ? p.b2[i] : static_cast<uint16_t>(0);
    named_barrier_sync(2, kEpiThreads);
    const uint32_t lane_sel = static_cast<uint32_t>(q * 32) << 16;
    const uint32_t sfull_leader = map_to_cta(bar_sfull, leader);
    const uint32_t pfree_leader = map_to_cta(bar_pfree(0), leader);
    uint32_t puses[2] = {0, 0}, suses = 0;

    // ---------------- Epi1(u): S = bf16(ReLU(P + b1)) of one half, as the A operand of ML2(u)
    auto epi1 = [&](int u) {
      const int it = u / NH, h = u % NH;
      const int slot = LOCK ? h : ((it & 1) ^ h);
      mbar_wait<false>(bar_pfull(slot), puses[slot] & 1u, w);
      ++puses[slot];
      __syncwarp();
      tcgen05_fence_after_sync();
      uint32_t pk[32];
#pragma unroll
      for (int part = 0; part < 2; ++part) {
        uint32_t v[32];
        tmem_ld_32cols(tmem_base + lane_sel + static_cast<uint32_t>(slot * 256 + hh * 64 + part * 32), v);
        if (part == 1) {
          // the slot has been read (the loads wait for their data).  Half 1 does not host O: its slot is free for the next
          // tile's first half from here on -- the UMMA lane is waiting for exactly this
          tcgen05_fence_before_sync();
          __syncwarp();
          if (h == 1 && lane == 0) mbar_arrive_cluster_noflush(pfree_leader + 8u * slot);
        }
        const uint4* b4 = reinterpret_cast<const uint4*>(s_b1 + h * 256 + hh * 64 + part * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint4 bb = b4[i];
          const uint32_t bw[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float2 x = add2(f2_from_bits(v[8 * i + 2 * j], v[8 * i + 2 * j + 1]), bf16x2_to_f2(bw[j]));
            pk[part * 16 + 4 * i + j] = pack_bf16x2_rn(fmaxf(x.x, 0.f), fmaxf(x.y, 0.f));
          }
        }
      }
      // the S buffer: the output boxes that Epi2 staged there have been read by their stores ...
      if (h == 0 && it > 0) {
        if (store_thread) tma_store_wait_read<0>();
        named_barrier_sync(3, kEpiThreads);
      }
      // ... and ML2 of the previous unit has read S
      mbar_wait<false>(bar_sempty, (suses & 1u) ^ 1u, w);
      ++suses;
      __syncwarp();
      const uint32_t sb = s_base + hh * kBoxBytes;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t a = sb + swz128(row, i);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]),
                     "r"(pk[4 * i + 3])
                     : "memory");
      }
      fence_proxy_async_smem();  // S writes are visible to the tensor core's shared-memory reads
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_noflush(sfull_leader);
    };
    // ---------------- Epi2(it): O = bf16(ReLU(acc + b2)), two 128 x 64 boxes staged in the S buffer and stored together
    auto epi2 = [&](int it) {
      const int oslot = LOCK ? 0 : (it & 1);
      mbar_wait<false>(bar_ofull, static_cast<uint32_t>(it) & 1u, w);  // also: the tile's last ML2 has read S
      __syncwarp();
      tcgen05_fence_after_sync();
      uint32_t v[32];
      tmem_ld_32cols(tmem_base + lane_sel + static_cast<uint32_t>(oslot * 256 + hh * 32), v);
      tcgen05_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_noflush(pfree_leader + 8u * oslot);
      uint32_t pk[16];
      const uint4* b4 = reinterpret_cast<const uint4*>(s_b2 + hh * 32);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 bb = b4[i];
        const uint32_t bw[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 x = add2(f2_from_bits(v[8 * i + 2 * j], v[8 * i + 2 * j + 1]), bf16x2_to_f2(bw[j]));
          pk[4 * i + j] = pack_bf16x2_rn(fmaxf(x.x, 0.f), fmaxf(x.y, 0.f));
        }
      }
      const uint32_t box = s_base + (hh >> 1) * kBoxBytes;  // columns 0..63 | 64..127
      const int chunk0 = (hh & 1) * 4;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t a = box + swz128(row, chunk0 + i);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]),
                     "r"(pk[4 * i + 3])
                     : "memory");
      }
      fence_proxy_async_smem();
      named_barrier_sync(3, kEpiThreads);
      if (store_thread) {
        const int m0 = tile_m0(it);
        if (COMFUSE_IN_BOUNDS(m0 >= 0 && m0 < p.mpairs * 256, p.status)) {
          tma_store_3d(&tmO, s_base, 0, m0, 0);
          tma_store_3d(&tmO, s_base + kBoxBytes, 64, m0, 0);
        }
        tma_store_commit();
      }
    };
    for (int u = 0; u < nunits; ++u) {
      if (u > 0 && u % NH == 0) epi2(u / NH - 1);
      epi1(u);
    }
    if (nunits > 0) epi2(my_tiles - 1);
    if (store_thread) tma_store_wait_read<0>();  // the staging boxes must outlive the last store's read
  }

  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after_sync();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

}  // namespace

// COMFUSE_B2B_STREAM_LOCK=0 runs N1 = 512 on the alternating-slot schedule as well (for comparison)
static bool stream_lock_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("COMFUSE_B2B_STREAM_LOCK");
    return !(e && e[0] == '0');
  }();
  return on;
}

bool b2b_stream_supported(int K, int N1, int N2) { return N2 == 128 && N1 >= 8 && N1 <= 512 && N1 % 8 == 0 && K >= 8 && K % 8 == 0; }

cudaError_t launch_b2b_stream(const void* X, const void* W1, const void* W2, B2bParams p, cudaStream_t st) {
  const DeviceInfo* dev = current_device_info();
  if (!dev) return cudaErrorInvalidDevice;
  CUtensorMap tmX, tmW1, tmW2, tmO;
  const uint64_t M = p.M, K = p.K, N1 = p.N1, N2 = p.N2;
  // boxes of 64 elements: X, W2 and O 128 rows, W1 64 rows (one K block)
  if (!encode_tmap_bf16_3d(&tmX, X, K, M, 1, K * 2, M * K * 2, 128) ||
      !encode_tmap_bf16_3d(&tmW1, W1, N1, K, 1, N1 * 2, K * N1 * 2, 64) ||
      !encode_tmap_bf16_3d(&tmW2, W2, N2, N1, 1, N2 * 2, N1 * N2 * 2, 128) ||
      !encode_tmap_bf16_3d(&tmO, p.O, N2, M, 1, N2 * 2, M * N2 * 2, 128))
    return cudaErrorInvalidValue;
  p.batch = 1;
  p.mblocks = (p.M + 127) / 128;
  p.mpairs = (p.mblocks + 1) / 2;

  constexpr int kMaxDev = 64;
  static std::atomic<int> max_clusters[kMaxDev];  // 0 = kernel not configured yet on that device (set last, released)
  const int di = dev->device < kMaxDev ? dev->device : kMaxDev - 1;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.blockDim = dim3(kThreads, 1, 1);
  const bool lock = p.N1 > 256 && stream_lock_enabled();
  cfg.dynamicSmemBytes = lock ? StreamSmem<true>::BYTES : StreamSmem<false>::BYTES;
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
    cudaError_t e = cudaFuncSetAttribute(b2b_stream_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, StreamSmem<false>::BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(b2b_stream_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, StreamSmem<true>::BYTES);
    if (e != cudaSuccess) return e;
    int n = 0;
    cfg.gridDim = dim3(2 * dev->sm_count, 1, 1);
    cfg.dynamicSmemBytes = StreamSmem<false>::BYTES;  // both instantiations: one CTA per SM
    e = cudaOccupancyMaxActiveClusters(&n, b2b_stream_kernel<false>, &cfg);
    cfg.dynamicSmemBytes = lock ? StreamSmem<true>::BYTES : StreamSmem<false>::BYTES;
    if (e != cudaSuccess) return e;
    if (n <= 0) return cudaErrorLaunchOutOfResources;
    max_clusters[di].store(n, std::memory_order_release);
    ncl = n;
  }
  const int tiles = p.mpairs;
  const int clusters = tiles < ncl ? tiles : ncl;
  cfg.gridDim = dim3(clusters * 2, 1, 1);
  count_launch();
  return lock ? cudaLaunchKernelEx(&cfg, b2b_stream_kernel<true>, tmX, tmW1, tmW2, tmO, p)
              : cudaLaunchKernelEx(&cfg, b2b_stream_kernel<false>, tmX, tmW1, tmW2, tmO, p);
}

}  // namespace comfuse
