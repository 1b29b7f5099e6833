// GEMM -> row-reduction subgraph in one kernel (Stage-Stream Execution Model, Sec. 3), built on CTA pairs.
//
// Why pairs: one SM's shared memory delivers 128 B/clk, and a 128 x 256 x 16 bf16 UMMA that reads both operands
// from shared memory already needs 96 B/clk before TMA has written the next tiles.  With cta_group::2 two CTAs
// multiply 256 rows at once: each holds its own 128 rows of A and only HALF of the B tile, so the per-SM operand
// traffic (and the L2 -> shared-memory fill) of the weight operand halves.  Every CTA fetches its
// own half with ordinary (single-destination) TMA loads that signal the issuing (even) CTA's barrier.
//
// Work decomposition (Sec. 3.1, cluster-granular scheduling with a secondary mapping by CTA rank): a cluster has
// 2*CN CTAs; cluster rank r works on row block (r & 1) of a pair of adjacent 128-row blocks and on column range
// (r >> 1) of CN.  All CTAs with the same (r & 1) share rows and form one reduction group (Sec. 3, Eq. 1); they
// exchange per-row partial statistics over distributed shared memory.  Clusters are persistent and walk the row
// block pairs with a stride of the cluster count.
//
// Inside a CTA (10 warps): warp 0 = TMA producer, warp 1 = TMEM allocation and (even CTA only) UMMA issue,
// warps 2-9 = epilogue (thread = one accumulator row; the two warps of a lane quarter take alternate 64-column
// groups).  Each epilogue warp is its own pipeline: it reads its 32 rows of the residual box, stages its 32 x 64
// output box in a private shared-memory buffer and issues its own TMA store, so no CTA-wide barrier sits on the
// per-group path.  warp 10 = store warp: lane e waits for epilogue warp e's staged boxes and issues their TMA stores, so
// the epilogue warps never stall on the store engine (about 40 GB/s per SM) and run ahead by the staging depth.
//
// Pipelining (Sec. 3.3, PingPong at sub-tile grain).  The CTA's BN columns are one or two sub-tiles, each with its
// own TMEM slot and full/empty barriers.  The MainLoop of sub-tile 1 runs while the epilogue's stage 1 works on
// sub-tile 0, and the next tile's sub-tile 0 starts as soon as stage 2 has drained that slot.  A CTA with a single
// sub-tile of at most 256 columns alternates between the two slots from tile to tile.
//
// One circular shared-memory buffer feeds both consumers (the unified multi-stage buffer of Sec. 4.2, applied to
// the epilogue operand): after the K blocks of a sub-tile the producer pushes that sub-tile's residual tile through
// the same ring, 128 rows x 64 columns per TMA box, so the epilogue reads the residual from swizzled shared memory
// instead of issuing one scattered global load per row.  Results leave the same way: 32 x 64 bf16 boxes are
// written to swizzled per-warp staging buffers and stored with TMA.
#pragma once

#include "comfuse.h"
#include "epilogue_common.cuh"
#include "fused_params.h"
#include "sm100_primitives.cuh"

namespace comfuse {

template <int EPI, int BNS0, int BNS1, int CN, int NSTAGES, int LOCK = 0, int EPW = 2>
struct PairCfg {
  // EPW epilogue warps per TMEM lane quarter (2 or 4): they take the 64-column groups g with g % EPW == their index
  static constexpr int kEpiWarps = 4 * EPW;
  static constexpr int kEpiThreads = 32 * kEpiWarps;
  static constexpr int kStoreWarp = 2 + kEpiWarps;
  static constexpr int kThreads = 32 * (kStoreWarp + 1);  // producer, UMMA, epilogue warps, store warp
  static constexpr int NSUB = BNS1 > 0 ? 2 : 1;
  static constexpr int BN = BNS0 + BNS1;
  static constexpr int BNSMAX = BNS0 > BNS1 ? BNS0 : BNS1;
  static constexpr int A_BYTES = 128 * 64 * 2;
  static constexpr int GROUP_BYTES = 128 * 64 * 2;                        // one 128 x 64 bf16 box
  // LOCK = 1: both sub-tiles advance in lock step, one ring stage carries A and BOTH sub-tiles' B halves (A is fetched
  // and read once per K block: less L2 -> shared-memory traffic, no overlap between the sub-tiles' epilogue and MainLoop).
  static constexpr int STAGE_BYTES = A_BYTES + ((LOCK ? BN : BNSMAX) / 2) * 64 * 2;  // A tile + this CTA's half of the B tile(s)
  static constexpr int GROUPS_PER_STAGE = STAGE_BYTES / GROUP_BYTES;      // residual boxes one ring stage can carry
  static constexpr int ACC_COLS = NSUB == 2 ? BN : 2 * BNS0;              // two TMEM slots
  static constexpr int ESUB = LOCK ? 1 : NSUB;                            // units the epilogue sees per tile
  static constexpr int TMEM_COLS = ACC_COLS <= 32 ? 32 : ACC_COLS <= 64 ? 64 : ACC_COLS <= 128 ? 128 : ACC_COLS <= 256 ? 256 : 512;
  static constexpr int OFF_YBUF = NSTAGES * STAGE_BYTES;
  static constexpr int WARP_BOX_BYTES = 32 * 64 * 2;                      // one warp's 32 x 64 bf16 output box
  static constexpr int FIXED_BYTES = 3 * BN * 4 + 2 * CN * 128 * 8 + 2 * EPW * 128 * 8 + (4 * NSTAGES + 7 + 192) * 8 + 16 + 1024;
  static constexpr int YBOX_ROOM = (232448 - NSTAGES * STAGE_BYTES - FIXED_BYTES) / (kEpiWarps * WARP_BOX_BYTES);
  static constexpr int YBOXES = YBOX_ROOM >= 4 ? 4 : YBOX_ROOM;           // staging boxes per epilogue warp
  static constexpr int YBUF_BYTES = YBOXES * kEpiWarps * WARP_BOX_BYTES;
  // Softmax only: the CTA's 64-column groups are interleaved with its peers' (group g of column range c is global
  // group g*CN + c), so that a causal mask leaves every CTA of the reduction group the same share of live columns.
  static constexpr bool INTERLEAVE = EPI == EPI_SOFTMAX;
  static constexpr int OFF_VEC = OFF_YBUF + YBUF_BYTES;
  static constexpr int VEC_BYTES = 3 * BN * 4;
  static constexpr int OFF_STATS = OFF_VEC + VEC_BYTES;
  static constexpr int STATS_BYTES = 2 * CN * 128 * 8;
  static constexpr int OFF_PRE = OFF_STATS + STATS_BYTES;
  static constexpr int PRE_BYTES = 2 * EPW * 128 * 8;
  static constexpr int OFF_BAR = OFF_PRE + PRE_BYTES;
  static constexpr int NUM_BARS = 4 * NSTAGES + 4 + 3 + 192;  // + staging-box full/free/last-tile, up to 16 warps x 4 boxes each
  // A CTA's LAST tile has the whole circular buffer to itself once its accumulator is complete (nothing is loaded after
  // it), so every output box of that tile gets a staging box of its own there and no epilogue warp waits for a store.
  static constexpr int BOXES_PER_WARP = BN / 64 / EPW;
  static constexpr bool RING_STAGING = EPI != EPI_SOFTMAX && ESUB == 1 && BOXES_PER_WARP <= 4 &&
                                       kEpiWarps * BOXES_PER_WARP * WARP_BOX_BYTES <= NSTAGES * STAGE_BYTES;
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;
  static constexpr int SMEM_BYTES = OFF_MISC + 16 + 1024;
  static_assert(BNS0 % 128 == 0 && BNS0 <= 256 && BNS1 % 128 == 0 && BNS1 <= 256, "each CTA's half must be whole 64-column boxes");
  static_assert(BNS0 > 0 && ACC_COLS <= 512, "accumulators must fit the 512 TMEM columns");
  static_assert(NSTAGES <= 8, "per-stage phase bits are kept in one byte");
  static_assert(GROUPS_PER_STAGE >= 2, "a residual stage carries one even and one odd 64-column group");
  static_assert(!LOCK || NSUB == 2, "lock step needs two sub-tiles");
  static_assert(EPW == 2 || EPW == 4, "two or four epilogue warps per lane quarter");
  static_assert((BNS0 / 64) % EPW == 0 && (BNS1 / 64) % EPW == 0, "every epilogue warp gets the same number of groups");
  static_assert(EPW == 2 || EPI == EPI_SOFTMAX || EPI == EPI_NONE || EPI == EPI_ELEMENTWISE, "residual stages carry one group per warp pair");
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
  static_assert(YBOXES >= 1, "at least one staging box per epilogue warp");
  static_assert(SMEM_BYTES > 116 * 1024, "one CTA per SM is assumed (TMEM allocation never waits for a co-resident CTA)");
};

// Position in the circular buffer; every role walks the same sequence of stage uses.
template <int NSTAGES>
struct RingPos {
  int stage = 0;
  uint32_t phase = 0;
  __device__ __forceinline__ void advance() {
    if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
  }
  __device__ __forceinline__ void skip(int n) {
    stage += n;
    while (stage >= NSTAGES) { stage -= NSTAGES; phase ^= 1u; }
  }
};

// 16-byte chunk `c` (0..7) of row `r` inside a 128-byte-swizzled 128 x 64 bf16 box.
__device__ __forceinline__ uint32_t swz128(int r, int c) { return static_cast<uint32_t>(r * 128 + ((c ^ (r & 7)) << 4)); }

template <int EPI, int BNS0, int BNS1, int CN, int NSTAGES, int LOCK, int EPW>
__global__ void __launch_bounds__(32 * (3 + 4 * EPW), 1)
fused_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmR, const __grid_constant__ CUtensorMap tmY, const FusedParams p) {
  using Cfg = PairCfg<EPI, BNS0, BNS1, CN, NSTAGES, LOCK, EPW>;
  constexpr bool kIsRms = EPI == EPI_RMS_MAX || EPI == EPI_RMS_MAX_LINEAR;  // the latter: no GELU in stage 1
  constexpr bool kIsPlain = EPI == EPI_NONE || EPI == EPI_ELEMENTWISE;      // no reduction: column blocks are independent
  constexpr int BN = Cfg::BN;
  constexpr int NSUB = Cfg::NSUB;
  constexpr int ESUB = Cfg::ESUB;
  constexpr int GPS = 2;  // residual boxes per ring stage: one even and one odd group
  // what the epilogue (and the store warp) see as unit `sub` of a tile: its width and its first local 64-column group
  auto unit_width = [](int sub) { return LOCK ? BN : (sub ? BNS1 : BNS0); };
  auto unit_lg0 = [](int sub) { return LOCK ? 0 : (sub ? BNS0 / 64 : 0); };

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
  auto bar_full = [&](int s) { return bar_base + 8u * s; };                     // K-block stage landed (even CTA)
  auto bar_empty = [&](int s) { return bar_base + 8u * (NSTAGES + s); };        // stage may be overwritten
  auto bar_rfull = [&](int s) { return bar_base + 8u * (2 * NSTAGES + s); };    // residual stage landed (own CTA)
  auto bar_rdone = [&](int s) { return bar_base + 8u * (3 * NSTAGES + s); };    // residual stage read by all 8 warps
  auto bar_tfull = [&](int a) { return bar_base + 8u * (4 * NSTAGES + a); };    // accumulator slot complete
  auto bar_tempty = [&](int a) { return bar_base + 8u * (4 * NSTAGES + 2 + a); };  // slot drained by both CTAs (even CTA)
  const uint32_t bar_stats = bar_base + 8u * (4 * NSTAGES + 4);
  const uint32_t bar_drain = bar_stats + 16u;  // two statistics barriers (one per exchange parity)
  auto bar_yfull = [&](int e, int k) { return bar_drain + 8u + 8u * (e * 4 + k); };        // staging box written (epilogue warp e)
  auto bar_yfree = [&](int e, int k) { return bar_drain + 8u + 8u * (64 + e * 4 + k); };   // staging box read out by its TMA store
  auto bar_ylast = [&](int e, int k) { return bar_drain + 8u + 8u * (128 + e * 4 + k); };  // last tile: box k of warp e staged in the ring
  auto ring_box = [&](int e, int k) { return smem_base + static_cast<uint32_t>((e * Cfg::BOXES_PER_WARP + k) * Cfg::WARP_BOX_BYTES); };
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(smem + Cfg::OFF_MISC);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + Cfg::OFF_MISC + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t pm = rank & 1u;       // which row block of the pair
  const uint32_t crank = rank >> 1;    // which column range
  const uint32_t leader = rank & ~1u;  // cluster rank of the CTA that issues the pair's UMMAs
  const uint16_t pair_mask = static_cast<uint16_t>(3u << leader);  // the pair's two CTAs, for commits that signal both
  constexpr int CLUSTER = 2 * CN;
  const int cluster_id = blockIdx.x / CLUSTER;
  const int num_clusters = gridDim.x / CLUSTER;
  const int KB = (p.K + 63) >> 6;
  const bool has_res = (EPI == EPI_LN || kIsRms || EPI == EPI_PROGRAM) && p.residual != nullptr;
  // The last tile's output boxes may be staged in the circular buffer only if nothing is still arriving there when they
  // are written: a stage program that stores in its first pass, and the two-kernel form, which stores in stage 1, do so
  // while the residual boxes are still coming in.
  const bool ring_idle_at_store = !(EPI == EPI_PROGRAM && has_res && p.program.terminal_pass == 0) && !(p.wide && has_res);
  const WaitCtx w{s_abort, p.status, p.timeout_ns};
  griddep_launch_dependents();  // the next kernel's set-up may overlap this kernel (it waits before touching memory)

#ifdef COMFUSE_TRACE
  if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) p.trace[62] = globaltimer_ns();  // kernel entry
#endif
  // -------------------------------------------------------------------------------------------- set-up
  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGES; ++s) {
      mbar_init(bar_full(s), 2);   // one arrive.expect_tx from each CTA of the pair
      mbar_init(bar_empty(s), 1);  // one commit from the issuing CTA
      mbar_init(bar_rfull(s), 1);
      mbar_init(bar_rdone(s), 8);  // one arrive per epilogue warp
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull(a), 1);
      mbar_init(bar_tempty(a), 2 * Cfg::kEpiWarps);  // one arrival per epilogue warp of both CTAs
    }
    mbar_init(bar_stats, CN == 1 ? 4 : 1);       // one CTA: an arrival per lane quarter; else one arming arrive + bytes
    mbar_init(bar_stats + 8u, CN == 1 ? 4 : 1);
    mbar_init(bar_drain, 1);
    for (int e = 0; e < Cfg::kEpiWarps; ++e)
      for (int k = 0; k < 4; ++k) {
        mbar_init(bar_yfull(e, k), 1);
        mbar_init(bar_yfree(e, k), 1);
        mbar_init(bar_ylast(e, k), 1);
      }
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    prefetch_tensormap(&tmY);
    if (has_res) prefetch_tensormap(&tmR);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(s_tmem_base), Cfg::TMEM_COLS);
    tmem_relinquish_alloc_permit_pair();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  cluster_sync_after_init();  // every CTA's barriers exist before any peer signals them
  const uint32_t tmem_base = *s_tmem_base;
  // Everything above touched no global memory and may overlap the previous kernel's tail; everything below may read what
  // that kernel wrote (or overwrite what it still reads).
  griddep_wait();

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
  // First global column of this CTA's local 64-column group `lg` (0 .. BN/64-1).
  auto group_col = [&](int ncta0, int lg) { return Cfg::INTERLEAVE ? (lg * CN + static_cast<int>(crank)) * 64 : ncta0 + lg * 64; };
  // A sub-tile is not computed when it lies past N, or when the causal mask removes it for BOTH row blocks of the
  // pair (its first group has the smallest columns).  Every role evaluates the same predicate.
  // (the normalising kinds read every accumulator column of the instantiation: where it is wider than the row, the columns
  // from N on must BE zeros -- computed from operands that read as zeros -- not whatever the slot held before)
  constexpr bool kAllUnitsLive = EPI == EPI_LN || kIsRms || EPI == EPI_PROGRAM;
  auto unit_live = [&](int mpair0, int n0) { return (kAllUnitsLive || n0 < p.N) && !(EPI == EPI_SOFTMAX && p.causal && n0 > mpair0 + 255); };

  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      RingPos<NSTAGES> ring;
      bool ok = true;
      // A stage is handed back by the UMMA commit (K-block use) or by the eight epilogue warps (residual use); the two
      // kinds have their own barriers, so the producer remembers each stage's last use and each barrier's phase.
      uint32_t used = 0, last_res = 0, empty_bits = 0, rdone_bits = 0;
      // L2 priorities: the B operand (weights) is re-read by every row block, the residual is read exactly once
      const uint64_t once = l2_policy_evict_first();
      auto wait_stage_free = [&](int st) {
        const uint32_t bit = 1u << st;
        if (!(used & bit)) return true;
        if (last_res & bit) {
          if (!mbar_wait<false>(bar_rdone(st), (rdone_bits >> st) & 1u, w)) return false;
          rdone_bits ^= bit;
        } else {
          if (!mbar_wait<false>(bar_empty(st), (empty_bits >> st) & 1u, w)) return false;
          empty_bits ^= bit;
        }
        return true;
      };
      for (int tile = cluster_id; tile < p.total_tiles && ok; tile += num_clusters) {
        int b, mpair0, ncta0;
        decode_tile(tile, b, mpair0, ncta0);
        const int m0 = mpair0 + static_cast<int>(pm) * 128;
#pragma unroll
        for (int sub = 0; sub < ESUB; ++sub) {
          const int W = unit_width(sub);
          const int lg0 = unit_lg0(sub);  // first local 64-column group of the unit
          const int n0 = group_col(ncta0, lg0);
          if (!ok || !unit_live(mpair0, n0)) continue;
          const uint32_t bytes = Cfg::A_BYTES + (W / 2) * 128;
          for (int kb = 0; kb < KB; ++kb) {
            if (!wait_stage_free(ring.stage)) { ok = false; break; }
            used |= 1u << ring.stage;
            last_res &= ~(1u << ring.stage);
            const uint32_t sa = smem_base + ring.stage * Cfg::STAGE_BYTES;
            const uint32_t full = map_to_cta(bar_full(ring.stage), leader);
            mbar_arrive_expect_tx_cluster(full, bytes);
            tma_load_3d_pair(sa, &tmA, full, kb * 64, m0, b);
            // this CTA's half of each UMMA's B tile: boxes of 64 columns, 8 KB apart (B stored [K, N]: 64 contraction rows x
            // 64 columns, MN-major for the UMMA; B stored [N, K]: 64 rows of B = columns of the product x 64 contraction
            // elements, K-major like A -- same bytes, same places, the two coordinates change roles)
            auto load_b_half = [&](uint32_t dst, int first_group, int width) {
              for (int j = 0; j < width / 128; ++j) {
                const int col = group_col(ncta0, first_group + static_cast<int>(pm) * (width / 128) + j);
                if (p.b_nk) tma_load_3d_pair(dst + j * 8192, &tmB, full, kb * 64, col, b);
                else tma_load_3d_pair(dst + j * 8192, &tmB, full, col, kb * 64, b);
              }
            };
            if (LOCK) {
              load_b_half(sa + Cfg::A_BYTES, 0, BNS0);
              load_b_half(sa + Cfg::A_BYTES + (BNS0 / 2) * 128, BNS0 / 64, BNS1);
            } else {
              load_b_half(sa + Cfg::A_BYTES, lg0, W);
            }
            ring.advance();
          }
          if (ok && has_res) {
            // the sub-tile's residual tile rides the same ring, right behind its last K block
            const int groups = W / 64;
            for (int g0 = 0; g0 < groups; g0 += GPS) {
              if (!wait_stage_free(ring.stage)) { ok = false; break; }
              used |= 1u << ring.stage;
              last_res |= 1u << ring.stage;
              const int ng = groups - g0 < GPS ? groups - g0 : GPS;
              const uint32_t sr = smem_base + ring.stage * Cfg::STAGE_BYTES;
              mbar_arrive_expect_tx(bar_rfull(ring.stage), ng * Cfg::GROUP_BYTES);
              for (int g = 0; g < ng; ++g)
                tma_load_3d_hint(sr + g * Cfg::GROUP_BYTES, &tmR, bar_rfull(ring.stage), group_col(ncta0, lg0 + g0 + g), m0, b, once);
              ring.advance();
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ UMMA issuer (even CTA)
    if (lane == 0 && pm == 0) {
      RingPos<NSTAGES> ring;
      uint32_t full_bits = 0;     // per-stage phase of bar_full (a stage is not a K-block stage on every lap)
      uint32_t slot_uses[2] = {0, 0};
      uint32_t unit_count = 0;
      bool ok = true;
      // B stored [K, N] is an MN-major operand (64-column blocks 8 KB apart, 8 contraction rows 1 KB apart), B stored [N, K]
      // a K-major one like A; everything that depends on it is computed once, outside the K loop
      const bool bkm = p.b_nk != 0;
      const uint64_t bdesc_layout = bkm ? make_smem_desc_sw128(0, 16, 1024) : make_smem_desc_sw128(0, 8192, 1024);
      const uint64_t bstep[4] = {0, bkm ? 2u : 128u, bkm ? 4u : 256u, bkm ? 6u : 384u};
      for (int tile = cluster_id; tile < p.total_tiles && ok; tile += num_clusters) {
        int b, mpair0, ncta0;
        decode_tile(tile, b, mpair0, ncta0);
#pragma unroll
        for (int sub = 0; sub < ESUB; ++sub) {
          const int W = unit_width(sub);
          const int lg0 = unit_lg0(sub);  // first local 64-column group of the unit
          const int n0 = group_col(ncta0, lg0);
          if (!ok || !unit_live(mpair0, n0)) continue;
          const int slot = LOCK ? 0 : (NSUB == 2 ? sub : static_cast<int>(unit_count & 1u));
          ++unit_count;
          if (!mbar_wait<false>(bar_tempty(slot), (slot_uses[slot] & 1u) ^ 1u, w)) { ok = false; continue; }
          ++slot_uses[slot];
          tcgen05_fence_after_sync();
          const uint32_t d_tmem = tmem_base + (slot ? BNS0 : 0);
          const uint32_t idesc0 = bkm ? make_idesc_bf16(256, BNS0, false, false) : make_idesc_bf16(256, BNS0, false, true);
          const uint32_t idesc1 = bkm ? make_idesc_bf16(256, BNS1 > 0 ? BNS1 : 16, false, false) : make_idesc_bf16(256, BNS1 > 0 ? BNS1 : 16, false, true);
          const uint32_t idesc = (!LOCK && sub) ? idesc1 : idesc0;
          for (int kb = 0; kb < KB; ++kb) {
            if (!mbar_wait<false>(bar_full(ring.stage), (full_bits >> ring.stage) & 1u, w)) { ok = false; break; }
            full_bits ^= 1u << ring.stage;
            tcgen05_fence_after_sync();
            const uint32_t sa = smem_base + ring.stage * Cfg::STAGE_BYTES;
            const uint64_t adesc = make_smem_desc_sw128(sa, 16, 1024);
            // B: the descriptor's layout half was fixed before the loops; only the address field changes per stage
            // (the address field takes the offset inside the CTA's shared-memory window: a shared address also carries the CTA's
            // rank in the cluster above bit 18)
            const uint64_t bdesc = bdesc_layout + (((sa + Cfg::A_BYTES) & 0x3FFFFu) >> 4);
            const uint64_t bdesc1 = bdesc + (((BNS0 / 2) * 128) >> 4);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              // K advances by 16 elements: 32 bytes inside A's (or a K-major B's) swizzled row, 16 K-lines (2048 bytes) in an MN-major B
              const uint32_t acc = (kb | k) != 0 ? 1u : 0u;
              umma_bf16_ss_pair(d_tmem, adesc + static_cast<uint64_t>(k * 2), bdesc + bstep[k], idesc, acc);
              if (LOCK)  // the second sub-tile reuses the A tile that is already in shared memory
                umma_bf16_ss_pair(d_tmem + BNS0, adesc + static_cast<uint64_t>(k * 2), bdesc1 + bstep[k], idesc1, acc);
            }
            // the stage is free in both CTAs once these UMMAs have read it
            umma_commit_pair_both(bar_empty(ring.stage), pair_mask);
            ring.advance();
          }
          if (ok) {
            umma_commit_pair_both(bar_tfull(slot), pair_mask);
            if (has_res) ring.skip((W / 64 + GPS - 1) / GPS);  // the residual stages belong to the epilogue
          }
        }
      }
      umma_commit_pair(bar_drain);  // nothing may still be writing either CTA's TMEM when it is freed
      mbar_wait<false>(bar_drain, 0, w);
    }
  } else if (warp == Cfg::kStoreWarp) {
    // ------------------------------------------------------------------------------------------ store warp
    // Lane e mirrors epilogue warp e's sequence of output boxes: wait until the box is staged, store it with TMA, and
    // hand the staging box back once the store has read it.  D stores stay in flight per lane.
    if (lane < Cfg::kEpiWarps) {
      const int e = lane;
      const int q = (e + 2) & 3;
      const int h = e >> 2;
      constexpr int D = Cfg::YBOXES - 1;
      const uint32_t ybox0 = smem_base + Cfg::OFF_YBUF + e * Cfg::YBOXES * Cfg::WARP_BOX_BYTES;
      const uint64_t once = l2_policy_evict_first();  // the output is not read again by this kernel
      uint32_t n = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < p.total_tiles && ok; tile += num_clusters) {
        int b, mpair0, ncta0;
        decode_tile(tile, b, mpair0, ncta0);
        const int m0 = mpair0 + static_cast<int>(pm) * 128;
        const bool in_ring = Cfg::RING_STAGING && tile + num_clusters >= p.total_tiles && ring_idle_at_store;
        int kk = 0;  // box of this tile
        for (int sub = 0; sub < ESUB && ok; ++sub) {
          const int W = unit_width(sub);
          const int lg0 = unit_lg0(sub);
          if (kIsPlain && !unit_live(mpair0, group_col(ncta0, lg0))) continue;
          for (int g = h; g < W / 64; g += EPW) {
            const int col = group_col(ncta0, lg0 + g);
            if (kIsPlain && col >= p.N) break;
            if (in_ring) {
              if (!mbar_wait<false>(bar_ylast(e, kk), 0, w)) { ok = false; break; }
#ifdef COMFUSE_TRACE
              if (!(p.trace_flags & 1))
#endif
              if (col < p.N)  // (a group of a partial last tile may lie outside the matrix altogether: nothing to store)
              if (COMFUSE_IN_BOUNDS(col >= 0 && col < p.N && (col & 7) == 0 && m0 + q * 32 >= 0 && b >= 0 && b < p.batch, p.status))
              tma_store_3d_hint(&tmY, ring_box(e, kk), col, m0 + q * 32, b, once);
              tma_store_commit();
              ++kk;
              continue;
            }
            const uint32_t sel = n % Cfg::YBOXES;
            if (!mbar_wait<false>(bar_yfull(e, sel), (n / Cfg::YBOXES) & 1u, w)) { ok = false; break; }
#ifdef COMFUSE_TRACE
            if (!(p.trace_flags & 1))
#endif
            if (col < p.N)
            if (COMFUSE_IN_BOUNDS(col >= 0 && col < p.N && (col & 7) == 0 && m0 + q * 32 >= 0 && b >= 0 && b < p.batch, p.status))
            tma_store_3d_hint(&tmY, ybox0 + sel * Cfg::WARP_BOX_BYTES, col, m0 + q * 32, b, once);
            tma_store_commit();
            if (n >= static_cast<uint32_t>(D)) {
              tma_store_wait_read<D>();
              mbar_arrive(bar_yfree(e, (n - D) % Cfg::YBOXES));
            }
            ++n;
          }
        }
      }
      tma_store_wait_read<0>();  // the staging boxes must outlive the last stores' reads (the stores themselves complete at kernel end)
    }
  } else {
    // ------------------------------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;         // TMEM lane quarter this warp may touch: rows 32q .. 32q+31 of the tile
    const int h = (warp - 2) >> 2;  // this warp takes the 64-column groups g with g % EPW == h
    const int row = q * 32 + lane;
    const uint32_t lane_sel = static_cast<uint32_t>(q * 32) << 16;
    int xpar = 0;
    uint32_t xphase = 0;
    (void)xpar; (void)xphase; (void)s_pre; (void)s_stats; (void)s_bias; (void)s_gamma; (void)s_beta;
    if constexpr (EPI == EPI_LN || kIsRms || EPI == EPI_PROGRAM) {
      // row-vector broadcasts (Sec. 5.2: 1-D parameters) of this CTA's columns, widened to fp32 once, by the epilogue warps
      // (they have nothing else to do until the first accumulator is complete); wide rows: the bias of the tile's column
      // block is loaded per tile instead, gamma/beta are identity
      const int c0 = crank * BN;
      for (int i = threadIdx.x - 64; i < BN; i += Cfg::kEpiThreads) {
        const int c = c0 + i;
        const bool in = c < p.N;
        s_bias[i] = (p.bias && in && !p.wide) ? bf16_lo(p.bias[c]) : 0.f;
        s_gamma[i] = (p.gamma && in) ? bf16_lo(p.gamma[c]) : 1.f;
        s_beta[i] = (p.beta && in) ? bf16_lo(p.beta[c]) : 0.f;
      }
      named_barrier_sync(3, Cfg::kEpiThreads);
    }
    RingPos<NSTAGES> ring;
    uint32_t rfull_bits = 0;
    uint32_t slot_uses[2] = {0, 0};
    uint32_t unit_count = 0;
    constexpr float kThreadCount = static_cast<float>(BN / EPW);  // columns behind one thread's partial
    const uint32_t tempty_leader = map_to_cta(bar_tempty(0), leader);
    const uint32_t ybox0 = smem_base + Cfg::OFF_YBUF + (warp - 2) * Cfg::YBOXES * Cfg::WARP_BOX_BYTES;  // this warp's staging boxes
    uint32_t ybox_sel = 0;

    // Stage this thread's 64 packed columns (its row of the warp's 32 x 64 box) and store the box with TMA.
    // pk[0..15] are columns 0..31 of the group, pk[16..31] columns 32..63.
    uint32_t ybox_count = 0;
#ifdef COMFUSE_TRACE
    int trace_ix = 0;
#define COMFUSE_TRACE_POINT()                                                                          \
  do {                                                                                                 \
    if (p.trace && blockIdx.x == 0 && warp == 2 && lane == 0 && trace_ix < 60) p.trace[trace_ix++] = globaltimer_ns(); \
  } while (0)
#else
#define COMFUSE_TRACE_POINT() do { } while (0)
#endif
    bool in_ring = false;  // this tile's boxes are staged in the (idle) circular buffer
    int ring_k = 0;
    auto store_box = [&](const uint32_t (&pk)[32]) {
      uint32_t ybox, ybar;
      if (Cfg::RING_STAGING && in_ring) {
        ybox = ring_box(warp - 2, ring_k);
        ybar = bar_ylast(warp - 2, ring_k);
        ++ring_k;
      } else {
        const uint32_t sel = ybox_sel;
        ybox = ybox0 + sel * Cfg::WARP_BOX_BYTES;
        ybar = bar_yfull(warp - 2, sel);
        if (++ybox_sel == Cfg::YBOXES) ybox_sel = 0;
        // the store of the box's previous contents has read it out
        mbar_wait<false>(bar_yfree(warp - 2, sel), ((ybox_count / Cfg::YBOXES) & 1u) ^ 1u, w);
        ++ybox_count;
      }
      __syncwarp();
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t a = ybox + swz128(lane, i);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]),
                     "r"(pk[4 * i + 3])
                     : "memory");
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(ybar);
    };
    // This thread's 64 residual values of box `gg` of a residual stage, as 32 packed bf16 pairs.
    auto load_residual = [&](uint32_t stage_addr, int gg, uint32_t (&r32)[32]) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t a = stage_addr + gg * Cfg::GROUP_BYTES + swz128(row, i);
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(r32[4 * i]), "=r"(r32[4 * i + 1]), "=r"(r32[4 * i + 2]), "=r"(r32[4 * i + 3])
                     : "r"(a));
      }
    };

    for (int tile = cluster_id; tile < p.total_tiles; tile += num_clusters) {
      COMFUSE_TRACE_POINT();
      int b, mpair0, ncta0;
      decode_tile(tile, b, mpair0, ncta0);
      const int m0 = mpair0 + static_cast<int>(pm) * 128;
      const int grow = m0 + row;
      in_ring = Cfg::RING_STAGING && tile + num_clusters >= p.total_tiles && ring_idle_at_store;
      const bool valid = grow < p.M;

      // the slot of each sub-tile of this tile, and whether it is computed at all
      bool live[ESUB];
      int slot[ESUB];
#pragma unroll
      for (int sub = 0; sub < ESUB; ++sub) {
        live[sub] = unit_live(mpair0, group_col(ncta0, unit_lg0(sub)));
        slot[sub] = LOCK ? 0 : (NSUB == 2 ? sub : static_cast<int>(unit_count & 1u));
        if (live[sub]) ++unit_count;
      }
      auto wait_accumulator = [&](int sub) {
        if (live[sub]) {
          mbar_wait<false>(bar_tfull(slot[sub]), slot_uses[slot[sub]] & 1u, w);
          ++slot_uses[slot[sub]];
          __syncwarp();
          tcgen05_fence_after_sync();
          ring.skip(KB);  // the K-block stages of this sub-tile were the UMMA's
        }
      };
      auto release_accumulator = [&](int sub) {
        if (live[sub]) {
          tcgen05_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster_noflush(tempty_leader + 8u * slot[sub]);
        }
      };
      auto tmem_of = [&](int sub) { return tmem_base + lane_sel + (slot[sub] ? BNS0 : 0); };

      if constexpr (kIsPlain) {
#pragma unroll
        for (int sub = 0; sub < ESUB; ++sub) {
          if (!live[sub]) continue;
          wait_accumulator(sub);
          const int W = unit_width(sub);
          const int lg0 = unit_lg0(sub);
          for (int g = h; g < W / 64; g += EPW) {
            const int gcol = group_col(ncta0, lg0 + g);
            if (gcol >= p.N) break;
            uint32_t pk[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              uint32_t v[32];
              tmem_ld_32cols(tmem_of(sub) + g * 64 + half * 32, v);
              if constexpr (EPI == EPI_ELEMENTWISE) {
                // y = act(alpha * acc + bias): the bias of these 32 columns straight from global memory (bf16 pairs; the
                // column block differs from tile to tile, N is a multiple of 8 and the group starts on a multiple of 64)
                const int c0 = gcol + half * 32;
                const float2 al = splat2(p.alpha);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  float2 bb = splat2(0.f);
                  if (p.bias && c0 + 2 * j < p.N) bb = bf16x2_to_f2(__ldg(reinterpret_cast<const uint32_t*>(p.bias + c0) + j));
                  float2 z = fma2(al, f2_from_bits(v[2 * j], v[2 * j + 1]), bb);
                  switch (p.activation) {
                    case COMFUSE_OP_RELU: z = make_float2(fmaxf(z.x, 0.f), fmaxf(z.y, 0.f)); break;
                    case COMFUSE_OP_GELU_TANH: z = gelu_tanh_f32x2(z); break;
                    case COMFUSE_OP_TANH:
                      z = make_float2(1.f - 2.f * __fdividef(1.f, 1.f + ex2_approx(2.8853900817779268f * z.x)),
                                      1.f - 2.f * __fdividef(1.f, 1.f + ex2_approx(2.8853900817779268f * z.y)));
                      break;
                    case COMFUSE_OP_SIGMOID:
                      z = make_float2(__fdividef(1.f, 1.f + ex2_approx(-1.4426950408889634f * z.x)),
                                      __fdividef(1.f, 1.f + ex2_approx(-1.4426950408889634f * z.y)));
                      break;
                    default: break;
                  }
                  pk[half * 16 + j] = pack_bf16x2_rn(z.x, z.y);
                }
              } else {
#pragma unroll
                for (int j = 0; j < 16; ++j)
                  pk[half * 16 + j] = pack_bf16x2_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
              }
            }
            store_box(pk);
          }
          release_accumulator(sub);
        }
      } else if constexpr (EPI == EPI_LN || kIsRms) {
        // ---------------- stage 1 (compute): x = f(alpha*Acc + bias, R); thread-local partial statistic; x is written
        // back over the accumulator in TMEM (the bypass path of Sec. 3.2)
        float2 part = make_float2(0.f, 0.f);
        float n_run = 0.f;
        if (p.wide) {
          // this tile's column block differs from the previous tile's: fetch its bias (every epilogue thread of the CTA
          // has left stage 1 of the previous tile, the cluster-wide reduce there waits for all rows)
          if (p.bias)
            for (int i = threadIdx.x - 64; i < BN; i += Cfg::kEpiThreads) s_bias[i] = ncta0 + i < p.N ? bf16_lo(p.bias[ncta0 + i]) : 0.f;
          named_barrier_sync(3, Cfg::kEpiThreads);
        }
        COMFUSE_TRACE_POINT();
#pragma unroll
        for (int sub = 0; sub < ESUB; ++sub) {
          wait_accumulator(sub);
          COMFUSE_TRACE_POINT();
          const int W = unit_width(sub);
          const int lsub = unit_lg0(sub) * 64;  // first column of the unit inside the CTA's column range
          const uint32_t taddr = tmem_of(sub);
          for (int g = h; g < W / 64; g += EPW) {
            // groups (g - h, g - h + 1) share one residual stage; this warp reads box h of it
            uint32_t r32[32];
            if (has_res) {
              mbar_wait<false>(bar_rfull(ring.stage), (rfull_bits >> ring.stage) & 1u, w);
              rfull_bits ^= 1u << ring.stage;
              __syncwarp();
              load_residual(smem_base + ring.stage * Cfg::STAGE_BYTES, h, r32);
              __syncwarp();
              if (lane == 0) mbar_arrive(bar_rdone(ring.stage));  // this warp is done with the stage
              ring.advance();
              COMFUSE_TRACE_POINT();
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) r32[j] = 0u;
            }
            uint32_t pkw[32];  // two-kernel form: the group's un-normalised values as fp16 pairs
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int lc = lsub + g * 64 + half * 32;
              uint32_t v[32];
              tmem_ld_32cols(taddr + g * 64 + half * 32, v);
              const float4* bias4 = reinterpret_cast<const float4*>(s_bias + lc);
              if constexpr (EPI == EPI_LN) {
                float2 s01 = splat2(0.f), s23 = splat2(0.f);
                const float2 al = splat2(p.alpha);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  const float4 bb = bias4[j];
                  const float2 x01 = add2(fma2(al, f2_from_bits(v[4 * j], v[4 * j + 1]), make_float2(bb.x, bb.y)),
                                          bf16x2_to_f2(r32[half * 16 + 2 * j]));
                  const float2 x23 = add2(fma2(al, f2_from_bits(v[4 * j + 2], v[4 * j + 3]), make_float2(bb.z, bb.w)),
                                          bf16x2_to_f2(r32[half * 16 + 2 * j + 1]));
                  v[4 * j] = __float_as_uint(x01.x); v[4 * j + 1] = __float_as_uint(x01.y);
                  v[4 * j + 2] = __float_as_uint(x23.x); v[4 * j + 3] = __float_as_uint(x23.y);
                  s01 = add2(s01, x01);
                  s23 = add2(s23, x23);
                }
                const float cmean = ((s01.x + s01.y) + (s23.x + s23.y)) * (1.f / 32.f);
                const float2 nm = splat2(-cmean);
                float2 q01 = splat2(0.f), q23 = splat2(0.f);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  const float2 d01 = add2(f2_from_bits(v[4 * j], v[4 * j + 1]), nm);
                  const float2 d23 = add2(f2_from_bits(v[4 * j + 2], v[4 * j + 3]), nm);
                  q01 = fma2(d01, d01, q01);
                  q23 = fma2(d23, d23, q23);
                }
                const float q0 = q01.x, q1 = q01.y, q2 = q23.x, q3 = q23.y;
                const float2 cpart = make_float2(cmean, (q0 + q1) + (q2 + q3));
                part = (n_run == 0.f) ? cpart : MergeWelford()(part, n_run, cpart, 32.f);
                n_run += 32.f;
              } else {
                float2 q01 = splat2(0.f), q23 = splat2(0.f);
                const float2 al = splat2(p.alpha);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  const float4 bb = bias4[j];
                  float2 z01 = fma2(al, f2_from_bits(v[4 * j], v[4 * j + 1]), make_float2(bb.x, bb.y));
                  float2 z23 = fma2(al, f2_from_bits(v[4 * j + 2], v[4 * j + 3]), make_float2(bb.z, bb.w));
                  if constexpr (EPI == EPI_RMS_MAX) {
                    z01 = gelu_tanh_f32x2(z01);
                    z23 = gelu_tanh_f32x2(z23);
                  }
                  const float2 h01 = add2(z01, bf16x2_to_f2(r32[half * 16 + 2 * j]));
                  const float2 h23 = add2(z23, bf16x2_to_f2(r32[half * 16 + 2 * j + 1]));
                  v[4 * j] = __float_as_uint(h01.x); v[4 * j + 1] = __float_as_uint(h01.y);
                  v[4 * j + 2] = __float_as_uint(h23.x); v[4 * j + 3] = __float_as_uint(h23.y);
                  q01 = fma2(h01, h01, q01);
                  q23 = fma2(h23, h23, q23);
                }
                const float q0 = q01.x, q1 = q01.y, q2 = q23.x, q3 = q23.y;
                part.x += (q0 + q1) + (q2 + q3);
              }
              if (p.wide) {
                // two-kernel form: x leaves the chip here, once, as fp16 (11 significant bits: the detour costs the result
                // a quarter of a bf16 half-ulp); the second kernel normalises it.  No write-back, no stage 2.
#pragma unroll
                for (int j = 0; j < 16; ++j) pkw[half * 16 + j] = pack_f16x2_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
              } else {
                tmem_st_32cols(taddr + g * 64 + half * 32, v);
              }
            }
            if (p.wide) store_box(pkw);
            COMFUSE_TRACE_POINT();
          }
          if (p.wide) release_accumulator(sub);
        }
        tmem_st_wait();
        COMFUSE_TRACE_POINT();
        // ---------------- stage 1 (reduce): thread pair, then the CTAs that share these rows
        float2 tot;
        if constexpr (EPI == EPI_LN) {
          tot = cluster_row_reduce<CN, MergeWelford, EPW>(part, kThreadCount, MergeWelford(), s_pre, s_stats, bar_stats, row, h, crank, xpar, xphase, w,
                                       2u, pm, p.leader_reduce != 0);
        } else {
          tot = cluster_row_reduce<CN, MergeSum, EPW>(part, kThreadCount, MergeSum(), s_pre, s_stats, bar_stats, row, h, crank, xpar, xphase, w, 2u,
                                       pm, p.leader_reduce != 0);
        }
        COMFUSE_TRACE_POINT();
        // wide rows: the statistic covers this column block only; store x as it is (gamma = 1, beta = 0 were loaded) and
        // leave the normalisation to the second kernel
        float mu = (EPI == EPI_LN && !p.wide) ? tot.x : 0.f;
        float sq = EPI == EPI_LN ? tot.y : tot.x;
        // The instantiation may be wider than the row (N = 1000 on the 1024-column form): the columns from N on hold exact
        // zeros (operands outside the matrix read as zeros, the row vectors are masked), which add nothing to a sum or to a
        // sum of squares.  The statistic of the N valid columns follows from the one over all W: S = W mean', Sxx = M2' +
        // W mean'^2, mean = S / N, M2 = Sxx - N mean^2.
        constexpr float kW = static_cast<float>(CN * BN);
        const bool ragged = !p.wide && p.N != CN * BN;
        const float nf = ragged ? static_cast<float>(p.N) : kW;
        if (EPI == EPI_LN && ragged) {
          const float s_all = kW * mu, sxx = sq + kW * mu * mu;
          mu = s_all / nf;
          sq = fmaxf(sxx - nf * mu * mu, 0.f);
        }
        const float rstd = p.wide ? 1.f : rsqrtf(sq / nf + p.eps);
        if (p.wide) {
          if (crank == 0 && h == 0 && valid) {
            const int nb = (ncta0 / (CN * BN));
            if (COMFUSE_IN_BOUNDS(nb >= 0 && nb < p.nblocks && grow >= 0 && grow < p.M && b >= 0 && b < p.batch, p.status))
            p.wide_partials[(static_cast<long long>(b) * p.M + grow) * p.nblocks + nb] = tot;
          }
          continue;  // the row is finished by the second kernel
        }
        // ---------------- stage 2 (PostOp): normalise the resident x, round once, store
        float best = -INFINITY;
        int best_col = 0x7FFFFFFF;
#pragma unroll
        for (int sub = 0; sub < ESUB; ++sub) {
          const int W = unit_width(sub);
          const int lsub = unit_lg0(sub) * 64;
          const uint32_t taddr = tmem_of(sub);
          for (int g = h; g < W / 64; g += EPW) {
            uint32_t pk[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int lc = lsub + g * 64 + half * 32;
              uint32_t v[32];
              tmem_ld_32cols(taddr + g * 64 + half * 32, v);
              const float4* g4 = reinterpret_cast<const float4*>(s_gamma + lc);
              const float4* b4 = reinterpret_cast<const float4*>(s_beta + lc);
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const float4 gg = g4[j];
                float y0, y1, y2, y3;
                if constexpr (EPI == EPI_LN) {
                  // y = (x - mu) * rstd * gamma + beta as two packed FMAs: n = x * rstd + (-mu * rstd), y = n * gamma + beta
                  const float4 be = b4[j];
                  const float2 n01 = fma2(f2_from_bits(v[4 * j], v[4 * j + 1]), splat2(rstd), splat2(-mu * rstd));
                  const float2 n23 = fma2(f2_from_bits(v[4 * j + 2], v[4 * j + 3]), splat2(rstd), splat2(-mu * rstd));
                  const float2 y01 = fma2(n01, make_float2(gg.x, gg.y), make_float2(be.x, be.y));
                  const float2 y23 = fma2(n23, make_float2(gg.z, gg.w), make_float2(be.z, be.w));
                  y0 = y01.x; y1 = y01.y; y2 = y23.x; y3 = y23.y;
                } else {
                  const float2 y01 = mul2(mul2(f2_from_bits(v[4 * j], v[4 * j + 1]), splat2(rstd)), make_float2(gg.x, gg.y));
                  const float2 y23 = mul2(mul2(f2_from_bits(v[4 * j + 2], v[4 * j + 3]), splat2(rstd)), make_float2(gg.z, gg.w));
                  y0 = y01.x; y1 = y01.y; y2 = y23.x; y3 = y23.y;
                  const int c = ncta0 + lc + 4 * j;
                  if (c + 3 < p.N) {  // (four columns at a time: N is a multiple of 8, so a group of four is inside or outside)
                    if (y0 > best) { best = y0; best_col = c; }
                    if (y1 > best) { best = y1; best_col = c + 1; }
                    if (y2 > best) { best = y2; best_col = c + 2; }
                    if (y3 > best) { best = y3; best_col = c + 3; }
                  }
                }
                v[4 * j] = __float_as_uint(y0); v[4 * j + 1] = __float_as_uint(y1);
                v[4 * j + 2] = __float_as_uint(y2); v[4 * j + 3] = __float_as_uint(y3);
              }
              // round once.  Wide rows: this is the un-normalised row on its way to the second kernel, which keeps 11
              // significant bits (fp16) instead of 8, so that the detour costs the result a quarter of a bf16 half-ulp
              if (p.wide) {
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[half * 16 + j] = pack_f16x2_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
              } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[half * 16 + j] = pack_bf16x2_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
              }
            }
            if (EPI == EPI_LN && p.post_relu && !p.wide) {
              // LayerNorm-ReLU pattern: on the rounded pairs (rounding is monotone and 0 is exact, so the order does not
              // matter); wide rows: the second kernel applies it
#pragma unroll
              for (int j = 0; j < 32; ++j) asm("max.bf16x2 %0, %0, %1;" : "+r"(pk[j]) : "r"(0u));
            }
            store_box(pk);
            COMFUSE_TRACE_POINT();
          }
          release_accumulator(sub);
        }
        if (kIsRms && !p.wide) {
          // ---------------- stage 3: the second, chained reduction reuses the exchange buffers (Sec. 3.2)
          const float2 mx = cluster_row_reduce<CN, MergeArgmax, EPW>(make_float2(best, __int_as_float(best_col)), kThreadCount, MergeArgmax(), s_pre,
                                                   s_stats, bar_stats, row, h, crank, xpar, xphase, w, 2u, pm, p.leader_reduce != 0);
          if (crank == 0 && h == 0 && valid) {
            const long long o = static_cast<long long>(b) * p.M + grow;
            if (COMFUSE_IN_BOUNDS(o >= 0 && o < static_cast<long long>(p.batch) * p.M, p.status)) {
              p.row_max[o] = mx.x;
              p.row_argmax[o] = __float_as_int(mx.y);
            }
          }
        }
      } else if constexpr (EPI == EPI_PROGRAM) {
        // ---------------- epilogue given as data: the stage program's passes over the TMEM-resident x (Sec. 3, Sec. 5.3).
        // ONE interpreter loop (one copy of every operation's code: the kernel is instruction-fetch bound otherwise)
        // runs the pass's micro-instruction stream on each 32-column fragment: v is the working fragment, x the resident one.
        static_assert(ESUB == 1, "stage programs run on single-unit tiles");
        // `sp` is the program's structure, `rp` its run-time part (immediates, row-output pointers).  In the ordinary build
        // both are the kernel parameter and the loops below are an interpreter; when the program is compiled into the
        // kernel (COMFUSE_COMPILED_PROGRAM: a constant table in front of this header, Sec. 5's code generation), the sweep and
        // instruction loops unroll and every dispatch below folds to the one operation it selects.
        const StageProgram& rp = p.program;
#ifdef COMFUSE_COMPILED_PROGRAM
        const StageProgram& sp = kCompiledProgram;
#define COMFUSE_PROGRAM_LOOP _Pragma("unroll")
#else
        const StageProgram& sp = p.program;
#define COMFUSE_PROGRAM_LOOP _Pragma("unroll 1")
#endif
        float sc[kStageMaxScalars];  // this row's scalars (reduction results and arithmetic on them)
#pragma unroll
        for (int i = 0; i < kStageMaxScalars; ++i) sc[i] = 0.f;
        const float* vecs[3] = {s_bias, s_gamma, s_beta};
        float racc[kStageMaxRed];  // thread-local partials (value; column for an arg max); indexed at run time
        int ridx[kStageMaxRed];
        float2 sc_topk[kStageMaxRed];  // Top-K: the row's pick of round 0 (value, column bits), kept until its later rounds run
COMFUSE_PROGRAM_LOOP
        for (int r = 0; r < kStageMaxRed; ++r) {
          const int op = r < sp.n_red ? sp.red[r].op : COMFUSE_OP_RED_SUM;
          racc[r] = op == COMFUSE_OP_RED_PROD ? 1.f : (op == COMFUSE_OP_RED_MAX || op == COMFUSE_OP_RED_ARGMAX) ? -INFINITY
                    : op == COMFUSE_OP_RED_MIN ? INFINITY : 0.f;
          ridx[r] = 0x7FFFFFFF;
        }
        // indexed at run time (a small local-memory array: one load instead of a chain of selects)
        auto scalar_get = [&](int kind, int ix, float imm) { return kind == CHO_SCALAR ? sc[ix & (kStageMaxScalars - 1)] : imm; };
        auto scalar_set = [&](int ix, float val) { sc[ix & (kStageMaxScalars - 1)] = val; };
        wait_accumulator(0);
        const uint32_t taddr = tmem_of(0);
        constexpr int kFrags = 2 * (BN / 64) / EPW;  // this thread's 32-column fragments of the tile
        uint32_t r32[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) r32[j] = 0u;
        uint32_t ybox = 0, ybar = 0;

        // A sweep runs a micro-instruction range over this thread's fragments.  Ordinary sweeps are the passes; behind a
        // pass's merges every Top-K reduction of that pass adds K - 1 sweeps of its own code range (`topk_r` >= 0), each
        // looking for the best element behind the previous pick (pv, pc).  The host laid the order down in sp.sweep[].
        float pv = 0.f;
        int pc = 0;
COMFUSE_PROGRAM_LOOP
        for (int s = 0; s < sp.n_sweeps; ++s) {
          const int pass = sp.sweep[s].pass, topk_r = sp.sweep[s].topk_r, topk_round = sp.sweep[s].topk_round;
          const int i0 = sp.sweep[s].i0, i1 = sp.sweep[s].i1;
          if (topk_r >= 0) {
            if (topk_round == 1) { pv = sc_topk[topk_r].x; pc = __float_as_int(sc_topk[topk_r].y); }
            racc[topk_r] = -INFINITY;
            ridx[topk_r] = 0x7FFFFFFF;
          }
#pragma unroll 1
          for (int f = 0; f < kFrags; ++f) {
            const int g = h + EPW * (f >> 1), half = f & 1;
            const int lc = g * 64 + half * 32;  // first CTA-local column of the fragment
            const int col0 = ncta0 + lc;
            if (pass == 0 && topk_r < 0 && half == 0 && has_res) {
              // the residual box of this group rides the operand ring (one stage per warp pair and group)
              mbar_wait<false>(bar_rfull(ring.stage), (rfull_bits >> ring.stage) & 1u, w);
              rfull_bits ^= 1u << ring.stage;
              __syncwarp();
              load_residual(smem_base + ring.stage * Cfg::STAGE_BYTES, h, r32);
              __syncwarp();
              if (lane == 0) mbar_arrive(bar_rdone(ring.stage));
              ring.advance();
            }
            float v[32], x[32];
#ifdef COMFUSE_COMPILED_PROGRAM
            float tq[kStageMaxTemps][32];  // temporaries: constant indices after unrolling, so registers (unused ones vanish)
#endif
            {
              uint32_t vb[32];
              tmem_ld_32cols(taddr + lc, vb);
#pragma unroll
              for (int j = 0; j < 32; ++j) { v[j] = __uint_as_float(vb[j]); x[j] = v[j]; }
            }
COMFUSE_PROGRAM_LOOP
            for (int i = i0; i < i1; ++i) {
              const ChainInstr ci = sp.code[i];
              const int op = ci.op;
              if (op >= COMFUSE_OP_ADD && op <= kChainMov) {
                // ---- binary with a row-uniform operand (constant or per-row scalar): applied directly
                if (ci.operand == CHO_SCALAR || ci.operand == CHO_CONST) {
                  const float sv = scalar_get(ci.operand, ci.index, rp.code[i].imm);
                  const float2 s2 = make_float2(sv, sv);
                  switch (op) {
                    case COMFUSE_OP_ADD:
#pragma unroll
                      for (int j = 0; j < 32; j += 2) { const float2 t = add2(make_float2(v[j], v[j + 1]), s2); v[j] = t.x; v[j + 1] = t.y; }
                      break;
                    case COMFUSE_OP_SUB: {
                      const float2 n2 = make_float2(-sv, -sv);
#pragma unroll
                      for (int j = 0; j < 32; j += 2) { const float2 t = add2(make_float2(v[j], v[j + 1]), n2); v[j] = t.x; v[j + 1] = t.y; }
                      break;
                    }
                    case COMFUSE_OP_MUL:
#pragma unroll
                      for (int j = 0; j < 32; j += 2) { const float2 t = mul2(make_float2(v[j], v[j + 1]), s2); v[j] = t.x; v[j + 1] = t.y; }
                      break;
                    case COMFUSE_OP_DIV:
#pragma unroll
                      for (int j = 0; j < 32; ++j) v[j] = __fdividef(v[j], sv);
                      break;
                    case COMFUSE_OP_MAX:
#pragma unroll
                      for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], sv);
                      break;
                    case COMFUSE_OP_MIN:
#pragma unroll
                      for (int j = 0; j < 32; ++j) v[j] = fminf(v[j], sv);
                      break;
                    case kChainRsub:
#pragma unroll
                      for (int j = 0; j < 32; ++j) v[j] = sv - v[j];
                      break;
                    case kChainMov:
#pragma unroll
                      for (int j = 0; j < 32; ++j) v[j] = sv;
                      break;
                    default:  // kChainRdiv
#pragma unroll
                      for (int j = 0; j < 32; ++j) v[j] = __fdividef(sv, v[j]);
                      break;
                  }
                  continue;
                }
                // ---- binary with a per-column operand: materialise the operand of the fragment, then apply
                float o[32];
                switch (ci.operand) {
                  case CHO_ROWVEC: {
                    const float4* v4 = reinterpret_cast<const float4*>(vecs[ci.index] + lc);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                      const float4 t4 = v4[j];
                      o[4 * j] = t4.x; o[4 * j + 1] = t4.y; o[4 * j + 2] = t4.z; o[4 * j + 3] = t4.w;
                    }
                    break;
                  }
                  case CHO_RESIDUAL:
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                      const float2 t2 = bf16x2_to_f2(half ? r32[16 + j] : r32[j]);
                      o[2 * j] = t2.x; o[2 * j + 1] = t2.y;
                    }
                    break;
                  case CHO_X:  // the resident tensor (before XSAVE: the accumulator as loaded)
#pragma unroll
                    for (int j = 0; j < 32; ++j) o[j] = x[j];
                    break;
#ifdef COMFUSE_COMPILED_PROGRAM
                  case CHO_T:
#pragma unroll
                    for (int j = 0; j < 32; ++j) o[j] = tq[ci.index][j];
                    break;
#endif
                  default:  // CHO_MASK
#pragma unroll
                    for (int j = 0; j < 32; ++j) o[j] = (col0 + j <= grow) ? 0.f : -INFINITY;
                    break;
                }
                switch (op) {
                  case COMFUSE_OP_ADD:
#pragma unroll
                    for (int j = 0; j < 32; j += 2) { const float2 t = add2(make_float2(v[j], v[j + 1]), make_float2(o[j], o[j + 1])); v[j] = t.x; v[j + 1] = t.y; }
                    break;
                  case COMFUSE_OP_SUB:
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = v[j] - o[j];
                    break;
                  case COMFUSE_OP_MUL:
#pragma unroll
                    for (int j = 0; j < 32; j += 2) { const float2 t = mul2(make_float2(v[j], v[j + 1]), make_float2(o[j], o[j + 1])); v[j] = t.x; v[j + 1] = t.y; }
                    break;
                  case COMFUSE_OP_DIV:
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __fdividef(v[j], o[j]);
                    break;
                  case COMFUSE_OP_MAX:
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], o[j]);
                    break;
                  case COMFUSE_OP_MIN:
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = fminf(v[j], o[j]);
                    break;
                  case kChainRsub:
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = o[j] - v[j];
                    break;
                  case kChainMov:
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = o[j];
                    break;
                  default:  // kChainRdiv
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __fdividef(o[j], v[j]);
                    break;
                }
                continue;
              }
              switch (op) {
                case COMFUSE_OP_NEG:
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = -v[j];
                  break;
                case COMFUSE_OP_ABS:
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = fabsf(v[j]);
                  break;
                case COMFUSE_OP_SQUARE:
#pragma unroll
                  for (int j = 0; j < 32; j += 2) { const float2 t = mul2(make_float2(v[j], v[j + 1]), make_float2(v[j], v[j + 1])); v[j] = t.x; v[j + 1] = t.y; }
                  break;
                case COMFUSE_OP_SQRT:
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = __fsqrt_rn(v[j]);
                  break;
                case COMFUSE_OP_RSQRT:
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = rsqrtf(v[j]);
                  break;
                case COMFUSE_OP_RECIP:
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = __fdividef(1.f, v[j]);
                  break;
                case COMFUSE_OP_EXP:
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = ex2_approx(v[j] * 1.4426950408889634f);
                  break;
                case COMFUSE_OP_LOG:
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = __logf(v[j]);
                  break;
                case COMFUSE_OP_TANH:  // 1 - 2 / (1 + e^(2x)): absolute error about 1e-7 (tanh.approx has 2^-11 relative)
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = 1.f - 2.f * __fdividef(1.f, 1.f + ex2_approx(2.8853900817779268f * v[j]));
                  break;
                case COMFUSE_OP_RELU:
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.f);
                  break;
                case COMFUSE_OP_GELU_TANH:
#pragma unroll
                  for (int j = 0; j < 32; j += 2) {
                    const float2 gz = gelu_tanh_f32x2(make_float2(v[j], v[j + 1]));
                    v[j] = gz.x; v[j + 1] = gz.y;
                  }
                  break;
                case COMFUSE_OP_SIGMOID:
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = __fdividef(1.f, 1.f + ex2_approx(-1.4426950408889634f * v[j]));
                  break;
                case kChainXsave: {  // x = v; written back over the accumulator when a later pass (or sweep) reads it
#pragma unroll
                  for (int j = 0; j < 32; ++j) x[j] = v[j];
                  if (sp.n_passes > 1 || sp.x_writeback) {
                    uint32_t vb[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) vb[j] = __float_as_uint(v[j]);
                    tmem_st_32cols(taddr + lc, vb);
                  }
                  break;
                }
#ifdef COMFUSE_COMPILED_PROGRAM
                case kChainTsave:
#pragma unroll
                  for (int j = 0; j < 32; ++j) tq[ci.index][j] = v[j];
                  break;
#endif
                case kChainXload:
#pragma unroll
                  for (int j = 0; j < 32; ++j) v[j] = x[j];
                  break;
                case kChainAcc: {  // thread-local partial of reduction ci.index over v
                  const int r = ci.index;
                  if (topk_r >= 0) {
                    if (r != topk_r) break;  // another reduction's accumulate inside this one's code range
                    // best element behind the previous pick: smaller value, or the same value in a later column
                    float a = racc[r];
                    int ai = ridx[r];
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                      const bool behind = v[j] < pv || (v[j] == pv && col0 + j > pc);
                      if (behind && v[j] > a) { a = v[j]; ai = col0 + j; }  // columns rise: a strict compare keeps the lowest
                    }
                    racc[r] = a;
                    ridx[r] = ai;
                    break;
                  }
                  float a = racc[r];
                  switch (sp.red[r].op) {
                    case COMFUSE_OP_RED_SUM:
                    case COMFUSE_OP_RED_MEAN: {
                      float t0 = 0.f, t1 = 0.f, t2 = 0.f, t3 = 0.f;
#pragma unroll
                      for (int j = 0; j < 32; j += 4) { t0 += v[j]; t1 += v[j + 1]; t2 += v[j + 2]; t3 += v[j + 3]; }
                      a += (t0 + t1) + (t2 + t3);
                      break;
                    }
                    case COMFUSE_OP_RED_MIN: {
                      float t0 = v[0], t1 = v[1], t2 = v[2], t3 = v[3];
#pragma unroll
                      for (int j = 4; j < 32; j += 4) { t0 = fminf(t0, v[j]); t1 = fminf(t1, v[j + 1]); t2 = fminf(t2, v[j + 2]); t3 = fminf(t3, v[j + 3]); }
                      a = fminf(a, fminf(fminf(t0, t1), fminf(t2, t3)));
                      break;
                    }
                    case COMFUSE_OP_RED_PROD: {
                      float t0 = 1.f, t1 = 1.f, t2 = 1.f, t3 = 1.f;
#pragma unroll
                      for (int j = 0; j < 32; j += 4) { t0 *= v[j]; t1 *= v[j + 1]; t2 *= v[j + 2]; t3 *= v[j + 3]; }
                      a *= (t0 * t1) * (t2 * t3);
                      break;
                    }
                    default: {  // max and arg max: the fragment's maximum by a tree; for the arg max its first column
                      // (columns rise from fragment to fragment, a strict compare against the running best keeps the lowest)
                      float t0 = v[0], t1 = v[1];
#pragma unroll
                      for (int j = 2; j < 30; j += 4) { t0 = max3(t0, v[j], v[j + 1]); t1 = max3(t1, v[j + 2], v[j + 3]); }
                      const float fm = max3(t0, t1, fmaxf(v[30], v[31]));
                      if (sp.red[r].op == COMFUSE_OP_RED_ARGMAX) {
                        if (fm > a) {
                          int ix = 31;
#pragma unroll
                          for (int j = 30; j >= 0; --j) ix = (v[j] == fm) ? j : ix;
                          ridx[r] = col0 + ix;
                          a = fm;
                        }
                      } else {
                        a = fmaxf(a, fm);
                      }
                      break;
                    }
                  }
                  racc[r] = a;
                  break;
                }
                default: {  // kChainEmit: round v once and put this half of the row into the warp's staging box
                  if (topk_r >= 0) break;
                  if (half == 0) {
                    if (Cfg::RING_STAGING && in_ring) {
                      ybox = ring_box(warp - 2, ring_k);
                      ybar = bar_ylast(warp - 2, ring_k);
                      ++ring_k;
                    } else {
                      const uint32_t sel = ybox_sel;
                      ybox = ybox0 + sel * Cfg::WARP_BOX_BYTES;
                      ybar = bar_yfull(warp - 2, sel);
                      if (++ybox_sel == Cfg::YBOXES) ybox_sel = 0;
                      mbar_wait<false>(bar_yfree(warp - 2, sel), ((ybox_count / Cfg::YBOXES) & 1u) ^ 1u, w);
                      ++ybox_count;
                    }
                    __syncwarp();
                  }
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    const uint32_t a = ybox + swz128(lane, half * 4 + q);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pack_bf16x2_rn(v[8 * q], v[8 * q + 1])),
                                 "r"(pack_bf16x2_rn(v[8 * q + 2], v[8 * q + 3])), "r"(pack_bf16x2_rn(v[8 * q + 4], v[8 * q + 5])),
                                 "r"(pack_bf16x2_rn(v[8 * q + 6], v[8 * q + 7]))
                                 : "memory");
                  }
                  if (half == 1) {
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(ybar);
                  }
                  break;
                }
              }
            }
          }
          if (topk_r >= 0) {
            // ---- a Top-K sweep is complete: merge the candidates, deliver the pick, go on to the next round / reduction / pass
            const float2 tot = cluster_row_reduce<CN, MergeArgmax, EPW>(make_float2(racc[topk_r], __int_as_float(ridx[topk_r])), kThreadCount,
                                                                       MergeArgmax(), s_pre, s_stats, bar_stats, row, h, crank, xpar, xphase, w,
                                                                       2u, pm, p.leader_reduce != 0);
            pv = tot.x;
            pc = __float_as_int(tot.y);
            if (crank == 0 && h == 0 && valid) {
              const long long o = (static_cast<long long>(b) * p.M + grow) * sp.red[topk_r].k + topk_round;
COMFUSE_PROGRAM_LOOP
              for (int q2 = 0; q2 < sp.n_row_out; ++q2)
                if (sp.out[q2].topk_red == topk_r + 1) {
                  if (sp.out[q2].is_int) static_cast<int*>(rp.out[q2].ptr)[o] = pc;
                  else static_cast<float*>(rp.out[q2].ptr)[o] = pv;
                }
            }
            if (sp.sweep[s].release) release_accumulator(0);
            continue;
          }
          if (pass == 0) tmem_st_wait();
          // ---- stage boundary: merges of the pass's reductions in program order (every CTA of the group makes the same
          // calls), then the per-row arithmetic that depends on them
COMFUSE_PROGRAM_LOOP
          for (int r = 0; r < sp.n_red; ++r) {
            if (sp.red[r].pass != pass) continue;
            const int op = sp.red[r].op;
            float2 tot;
            const float2 mine = make_float2(racc[r], __int_as_float(ridx[r]));
            if (op == COMFUSE_OP_RED_ARGMAX)
              tot = cluster_row_reduce<CN, MergeArgmax, EPW>(mine, kThreadCount, MergeArgmax(), s_pre, s_stats, bar_stats, row, h, crank, xpar, xphase,
                                                            w, 2u, pm, p.leader_reduce != 0);
            else
              tot = cluster_row_reduce<CN, MergeByOp, EPW>(mine, kThreadCount, MergeByOp{op}, s_pre, s_stats, bar_stats, row, h, crank, xpar, xphase,
                                                          w, 2u, pm, p.leader_reduce != 0);
            if (sp.red[r].k > 0) {
              // Top-K, round 0: the pass's own arg max; the later rounds follow behind the pass's merges
              sc_topk[r] = tot;
              if (crank == 0 && h == 0 && valid) {
                const long long o = (static_cast<long long>(b) * p.M + grow) * sp.red[r].k;
COMFUSE_PROGRAM_LOOP
                for (int q2 = 0; q2 < sp.n_row_out; ++q2)
                  if (sp.out[q2].topk_red == r + 1) {
                    if (sp.out[q2].is_int) static_cast<int*>(rp.out[q2].ptr)[o] = __float_as_int(tot.y);
                    else static_cast<float*>(rp.out[q2].ptr)[o] = tot.x;
                  }
              }
              continue;
            }
            float val = op == COMFUSE_OP_RED_ARGMAX ? static_cast<float>(__float_as_int(tot.y)) : tot.x;
            if (op == COMFUSE_OP_RED_MEAN) val *= 1.f / static_cast<float>(CN * BN);
            scalar_set(sp.red[r].dst, val);
          }
COMFUSE_PROGRAM_LOOP
          for (int i = 0; i < sp.n_scalar_instr; ++i) {
            const ScalarInstr si = sp.sc[i];
            if (si.after_pass != pass) continue;
            const float a = scalar_get(si.a_kind, si.a, rp.sc[i].a_imm);
            const float bq = scalar_get(si.b_kind, si.b, rp.sc[i].b_imm);
            float rv;
            switch (si.op) {
              case COMFUSE_OP_NEG: rv = -a; break;
              case COMFUSE_OP_ABS: rv = fabsf(a); break;
              case COMFUSE_OP_SQUARE: rv = a * a; break;
              case COMFUSE_OP_SQRT: rv = sqrtf(a); break;
              case COMFUSE_OP_RSQRT: rv = rsqrtf(a); break;
              case COMFUSE_OP_RECIP: rv = 1.f / a; break;
              case COMFUSE_OP_EXP: rv = expf(a); break;
              case COMFUSE_OP_LOG: rv = logf(a); break;
              case COMFUSE_OP_TANH: rv = tanhf(a); break;
              case COMFUSE_OP_RELU: rv = fmaxf(a, 0.f); break;
              case COMFUSE_OP_GELU_TANH: rv = 0.5f * a * (1.f + tanhf(0.7978845608028654f * (a + 0.044715f * a * a * a))); break;
              case COMFUSE_OP_SIGMOID: rv = 1.f / (1.f + expf(-a)); break;
              case COMFUSE_OP_ADD: rv = a + bq; break;
              case COMFUSE_OP_SUB: rv = a - bq; break;
              case COMFUSE_OP_MUL: rv = a * bq; break;
              case COMFUSE_OP_DIV: rv = a / bq; break;
              case COMFUSE_OP_MAX: rv = fmaxf(a, bq); break;
              default: rv = fminf(a, bq); break;
            }
            scalar_set(si.dst, rv);
          }
          if (sp.sweep[s].release) release_accumulator(0);
        }
        if (crank == 0 && h == 0 && valid) {
          const long long o = static_cast<long long>(b) * p.M + grow;
COMFUSE_PROGRAM_LOOP
          for (int r = 0; r < sp.n_row_out; ++r) {
            if (sp.out[r].topk_red) continue;  // delivered round by round
            const float val = scalar_get(CHO_SCALAR, sp.out[r].scalar, 0.f);
            if (sp.out[r].is_int) static_cast<int*>(rp.out[r].ptr)[o] = static_cast<int>(val);
            else static_cast<float*>(rp.out[r].ptr)[o] = val;
          }
        }
#undef COMFUSE_PROGRAM_LOOP
      } else {  // EPI_SOFTMAX
        // log2 domain: t = Acc * (alpha * log2 e), so exp(x - m) = 2^(t - m_t)
        // with a soft-cap the accumulators are mapped to capped log2-domain scores right after they are loaded, and sc = 1
        const bool capped = p.softcap > 0.f;
        const SoftcapLog2 cap_fn(p.alpha, capped ? p.softcap : 1.f);
        const float sc = capped ? 1.f : p.alpha * 1.4426950408889634f;
        const bool additive = p.mask != nullptr;  // additive mask tensor, applied behind the scale / soft-cap
        // The last live column of a row: the diagonal under the causal mask, and never beyond the row's end -- the
        // instantiation may be wider than the row (N = 1000 on the 1024-column form), columns from N on are masked.
        // Fragment classification, uniform over the warp's 32 rows so that the warp-wide TMEM loads stay convergent:
        // 2 = all live, 1 = crosses the limit of some row, 0 = all masked
        const int wrow0 = m0 + q * 32;
        const int nlast = p.N - 1;
        const int rlim = p.causal ? (grow < nlast ? grow : nlast) : nlast;
        const int wlim_lo = p.causal ? (wrow0 < nlast ? wrow0 : nlast) : nlast;
        const int wlim_hi = p.causal ? (wrow0 + 31 < nlast ? wrow0 + 31 : nlast) : nlast;
        auto frag_state = [&](int col0) { return col0 + 31 <= wlim_lo ? 2 : (col0 > wlim_hi ? 0 : 1); };
        COMFUSE_TRACE_POINT();
        // ---------------- pass A: thread-local row max
        float mloc = -INFINITY;
#pragma unroll
        for (int sub = 0; sub < ESUB; ++sub) {
          wait_accumulator(sub);
          if (!live[sub]) continue;
          const int W = unit_width(sub);
          const int lg0 = unit_lg0(sub);
          for (int g = h; g < W / 64; g += EPW) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int col0 = group_col(ncta0, lg0 + g) + half * 32;
              const int st = frag_state(col0);
              if (st == 0) continue;
              uint32_t v[32];
              tmem_ld_32cols(tmem_of(sub) + g * 64 + half * 32, v);
              if (capped) {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(cap_fn(__uint_as_float(v[j])));
              }
              float m0v = -INFINITY, m1v = -INFINITY;
              if (additive) {
                // a full-tensor operand of the epilogue (Sec. 5.2): t = score + mask, written back over the accumulator so
                // that pass B finds it there
                float2 m2[16];
                load_mask_log2_32(p.mask + static_cast<long long>(grow) * p.N + col0, valid ? (p.N - col0 < 32 ? p.N - col0 : 32) : 0, m2);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  const float2 t01 = fma2(f2_from_bits(v[2 * j], v[2 * j + 1]), splat2(sc), m2[j]);
                  v[2 * j] = __float_as_uint(t01.x);
                  v[2 * j + 1] = __float_as_uint(t01.y);
                  if (st == 2 || col0 + 2 * j <= rlim) m0v = fmaxf(m0v, t01.x);
                  if (st == 2 || col0 + 2 * j + 1 <= rlim) m1v = fmaxf(m1v, t01.y);
                }
                tmem_st_32cols(tmem_of(sub) + g * 64 + half * 32, v);
              } else {
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                  const float t0 = __uint_as_float(v[j]) * sc, t1 = __uint_as_float(v[j + 1]) * sc;
                  if (st == 2 || col0 + j <= rlim) m0v = fmaxf(m0v, t0);
                  if (st == 2 || col0 + j + 1 <= rlim) m1v = fmaxf(m1v, t1);
                }
              }
              mloc = fmaxf(mloc, fmaxf(m0v, m1v));
            }
          }
        }
        if (additive) tmem_st_wait();
        COMFUSE_TRACE_POINT();
        // ---------------- pass B: e = 2^(t - mloc), thread-local sum, e written back over the scores
        float lloc = 0.f;
        const float msub = (mloc == -INFINITY) ? 0.f : mloc;
#pragma unroll
        for (int sub = 0; sub < ESUB; ++sub) {
          if (!live[sub]) continue;
          const int W = unit_width(sub);
          const int lg0 = unit_lg0(sub);
          for (int g = h; g < W / 64; g += EPW) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int col0 = group_col(ncta0, lg0 + g) + half * 32;
              const int st = frag_state(col0);
              if (st == 0) continue;
              uint32_t v[32];
              tmem_ld_32cols(tmem_of(sub) + g * 64 + half * 32, v);
              if (capped && !additive) {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(cap_fn(__uint_as_float(v[j])));
              }
              float s0 = 0.f, s1 = 0.f;
              const float scb = additive ? 1.f : sc;  // with a mask tensor pass A has left t itself in the accumulator
#pragma unroll
              for (int j = 0; j < 32; j += 2) {
                const float2 t01 = fma2(f2_from_bits(v[j], v[j + 1]), splat2(scb), splat2(-msub));
                float e0 = ex2_approx(t01.x);
                float e1 = ex2_approx(t01.y);
                if (st != 2) {
                  if (col0 + j > rlim) e0 = 0.f;
                  if (col0 + j + 1 > rlim) e1 = 0.f;
                }
                v[j] = __float_as_uint(e0);
                v[j + 1] = __float_as_uint(e1);
                s0 += e0;
                s1 += e1;
              }
              lloc += s0 + s1;
              tmem_st_32cols(tmem_of(sub) + g * 64 + half * 32, v);
            }
          }
        }
        tmem_st_wait();
        COMFUSE_TRACE_POINT();
        const float2 tot = cluster_row_reduce<CN, MergeMaxSumExp2, EPW>(make_float2(mloc, lloc), kThreadCount, MergeMaxSumExp2(), s_pre, s_stats,
                                                  bar_stats, row, h, crank, xpar, xphase, w, 2u, pm, p.leader_reduce != 0);
        const float f = (mloc == -INFINITY || tot.y == 0.f) ? 0.f : ex2_approx(mloc - tot.x) / tot.y;
        COMFUSE_TRACE_POINT();
        // ---------------- pass C: scale, round once, store (zeros where masked)
#pragma unroll
        for (int sub = 0; sub < ESUB; ++sub) {
          const int W = unit_width(sub);
          const int lg0 = unit_lg0(sub);
          for (int g = h; g < W / 64; g += EPW) {
            uint32_t pk[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int col0 = group_col(ncta0, lg0 + g) + half * 32;
              const int st = live[sub] ? frag_state(col0) : 0;
              if (st == 0) {
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[half * 16 + j] = 0u;
              } else {
                uint32_t v[32];
                tmem_ld_32cols(tmem_of(sub) + g * 64 + half * 32, v);
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[half * 16 + j] = pack_bf16x2_rn(mul2(f2_from_bits(v[2 * j], v[2 * j + 1]), splat2(f)));
              }
            }
            store_box(pk);
          }
          release_accumulator(sub);
        }
      }
    }
  }

  // -------------------------------------------------------------------------------------------- teardown
#ifdef COMFUSE_TRACE
  if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) p.trace[61] = globaltimer_ns();  // epilogue warps done
#endif
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // no peer may still signal this CTA's barriers, write its shared memory or its TMEM
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after_sync();
    tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
  }
#ifdef COMFUSE_TRACE
  if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) p.trace[63] = globaltimer_ns();  // kernel exit
#endif
}

}  // namespace comfuse
