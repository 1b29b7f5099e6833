// Fused back-to-back GEMM, MLP form (Sec. 4):  P = X W1,  S = GELU_tanh(P + b1),  O' = S W2 + b2 + X,  O = LayerNorm(O'),
// K = N2 = 128, N1 = 8 .. 4096, a multiple of 8 (the chunks of N1 stream through; only the bias b1 is held whole).  Neither P nor S is
// written to global memory.
//
// Dataflow (Sec. 4.1, adapted): N1 is cut into 128-column chunks; one CTA pair walks all chunks of its 256 rows and
// accumulates O in tensor memory (deterministic, no cross-CTA partial sums).  The chunks of all the pair's tiles form ONE
// flat stream c = 0, 1, 2, ...: the roles below never drain at a tile boundary.
//
// Roles (Sec. 4.2 / 4.3: the stages ML1 -> Epi1 -> ML2 -> Epi2 each on warps of their own, staggered):
//   warp 0        producer: X tiles into two resident buffers, W1 / W2 chunk halves into two slots each (chunk parity)
//   warp 1        ML1 lane (even CTA): P(c + 2) as soon as the Epi1 warps hold chunk c in registers
//   warp 22       ML2 lane (even CTA): O = X (2 I), then O += S_c W2_c as soon as S_c is written.  Two issuing lanes because
//                 a UMMA of this size occupies its issuing thread about as long as the tensor pipe, and so does every wait
//   warps 2..17   Epi1: a thread owns one row and 32 columns of every chunk, reads them, frees the P slot at once,
//                 then bias + 2 GELU + bf16 into the S buffer of the chunk's parity
//   warps 18..21  Epi2: a thread owns one whole output row (no cross-thread reduce): + b2, LayerNorm, bf16, store; it
//                 runs under the Epi1 / ML work of the next tile
// The residual is added by the tensor pipe (the tile's A operand times twice the identity, exact in fp32), and the whole
// accumulator is kept at twice its value: S = 2 GELU saves Epi1 a multiplication, and LayerNorm(2 x) with 4 eps is
// LayerNorm(x) with eps.  The normalised row is staged over the tile's X buffer, idle by then, and stored from there by TMA.
#include <cuda_runtime.h>

#include <atomic>

#include "b2b_params.h"
#include "fused_pair.cuh"
#include "host_common.h"
#include "sm100_primitives.cuh"

namespace comfuse {

namespace {

constexpr int kEpi1Warps = 16;
constexpr int kEpi2Warps = 4;
constexpr int kEpiThreads = 32 * (kEpi1Warps + kEpi2Warps);
constexpr int kMlpThreads = 32 * (3 + kEpi1Warps + kEpi2Warps);
constexpr int kMl2Warp = 2 + kEpi1Warps + kEpi2Warps;
constexpr int kBoxBytes = 128 * 64 * 2;  // one 128 x 64 bf16 box
constexpr int kWSlots = 4;

struct MlpSmem {
  static constexpr int OFF_X = 0;                               // [2 tiles][2 K blocks]
  static constexpr int OFF_W = OFF_X + 4 * kBoxBytes;           // ring
  static constexpr int OFF_S = OFF_W + kWSlots * kBoxBytes;     // [2 buffers][2 K blocks]
  static constexpr int OFF_I = OFF_S + 4 * kBoxBytes;           // this CTA's 64 columns of 2 I (128 x 128), laid out like a W2 chunk
  static constexpr int kMaxN1 = 4096;
  static constexpr int OFF_B1 = OFF_I + kBoxBytes;              // fp32 [kMaxN1]
  static constexpr int OFF_VEC = OFF_B1 + kMaxN1 * 4;           // 2 b2, gamma, beta fp32 [128] each
  static constexpr int OFF_BAR = OFF_VEC + 3 * 128 * 4;
  // xfull[2] xempty[2] wfull[4] (4 unused) pfull[2] pfree[2] sfull[2] sempty[2] ofull[2] oempty[2] drain[2] eye
  static constexpr int NUM_BARS = 4 + 2 * kWSlots + 12 + 3;
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;
  static constexpr int BYTES = OFF_MISC + 16 + 1024;
};
static_assert(MlpSmem::BYTES <= 232448, "shared memory budget");

// y Phi(x) (y = x: GELU) with Phi(x) = 0.5 (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))) from the FMA pipe alone: Phi - 0.5 is odd, so
// Phi(x) = sat(0.5 + x R(min(x^2, 12.96))), R a degree-5 minimax polynomial (|error of x Phi| <= 4.1e-4 for every x; the
// saturating multiply-add pins Phi to [0, 1] where the polynomial's range ends).  No MUFU instruction.
__device__ __forceinline__ float2 gelu_poly_f32x2(float2 y, float2 z) {  // y Phi(z)
  float2 t = mul2(z, z);
  t.x = fminf(t.x, 12.96f);
  t.y = fminf(t.y, 12.96f);
  float2 r = fma2(splat2(-6.2840461246e-07f), t, splat2(3.1895157566e-05f));
  r = fma2(r, t, splat2(-6.8363819012e-04f));
  r = fma2(r, t, splat2(8.2311123259e-03f));
  r = fma2(r, t, splat2(-6.3471492633e-02f));
  r = fma2(r, t, splat2(3.9699813149e-01f));
  float2 phi;
  asm("fma.rn.sat.f32 %0, %1, %2, 0f3F000000;" : "=f"(phi.x) : "f"(z.x), "f"(r.x));
  asm("fma.rn.sat.f32 %0, %1, %2, 0f3F000000;" : "=f"(phi.y) : "f"(z.y), "f"(r.y));
  return mul2(y, phi);
}

// 32 accumulator columns -> bias, 2 GELU, bf16.  The factor 0.5 of the GELU is left to Epi2 (O = 0.5 (2S) W2: a power of
// two commutes with the bf16 rounding of S), which saves one instruction per pair here.  One pair in every POLY_EVERY
// takes the FMA-pipe form, the others tanh.approx: the MUFU unit (16 results per clock and SM) bounds this loop.
template <int POLY_EVERY>
__device__ __forceinline__ void gelu2_pack_32(const uint32_t (&v)[32], const float* bias, uint32_t (&pk)[16], int tf = 0) {
  const float4* b4 = reinterpret_cast<const float4*>(bias);
#ifdef COMFUSE_TRACE
  if (tf & 1) {  // experiment: no transcendental, no bias
#pragma unroll
    for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2_rn(f2_from_bits(v[2 * i], v[2 * i + 1]));
    return;
  }
#endif
  const float2 c0 = splat2(0.7978845608028654f);
  const float2 c1 = splat2(0.7978845608028654f * 0.044715f);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
#ifdef COMFUSE_TRACE
    const float4 bb = (tf & 4) ? make_float4(0.f, 0.f, 0.f, 0.f) : b4[i];
#else
    const float4 bb = b4[i];
#endif
    float2 g[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float2 z = add2(f2_from_bits(v[4 * i + 2 * h], v[4 * i + 2 * h + 1]), h ? make_float2(bb.z, bb.w) : make_float2(bb.x, bb.y));
      const int pair = 2 * i + h;
      if (POLY_EVERY > 0 && pair % POLY_EVERY == POLY_EVERY - 1) {
        g[h] = gelu_poly_f32x2(add2(z, z), z);
      } else {
        const float2 u = mul2(z, fma2(c1, mul2(z, z), c0));
        g[h] = fma2(z, make_float2(tanh_approx(u.x), tanh_approx(u.y)), z);  // z (1 + tanh u) = 2 GELU(z)
      }
    }
    pk[2 * i] = pack_bf16x2_rn(g[0]);
    pk[2 * i + 1] = pack_bf16x2_rn(g[1]);
  }
}
// four 16-byte chunks (chunk0 ..) of this thread's row of a 128-byte-swizzled box
__device__ __forceinline__ void store_row_chunks(const uint32_t (&pk)[16], uint32_t box, int row, int chunk0) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t a = box + swz128(row, chunk0 + i);
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]), "r"(pk[4 * i + 3])
                 : "memory");
  }
}

#ifndef COMFUSE_B2B_POLY_EVERY
#define COMFUSE_B2B_POLY_EVERY 4
#endif

__global__ void __launch_bounds__(kMlpThreads, 1)
b2b_mlp_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW1,
               const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmO, const B2bParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t smem_base = smem_u32(smem);

  float* s_b1 = reinterpret_cast<float*>(smem + MlpSmem::OFF_B1);
  float* s_b2 = reinterpret_cast<float*>(smem + MlpSmem::OFF_VEC);
  float* s_gamma = s_b2 + 128;
  float* s_beta = s_gamma + 128;
  const uint32_t bar_base = smem_base + MlpSmem::OFF_BAR;
  auto bar_xfull = [&](int b) { return bar_base + 8u * b; };                      // X tile landed in both CTAs (even CTA)
  auto bar_xempty = [&](int b) { return bar_base + 8u * (2 + b); };               // ML1 and Epi2 are done with the X buffer
  auto bar_wfull = [&](int s) { return bar_base + 8u * (4 + s); };                // weight slot landed (even CTA)
  constexpr int B0 = 4 + 2 * kWSlots;
  auto bar_pfull = [&](int a) { return bar_base + 8u * (B0 + a); };       // P slot complete
  auto bar_pfree = [&](int a) { return bar_base + 8u * (B0 + 2 + a); };   // P slot read by its Epi1 set in both CTAs (even CTA)
  auto bar_sfull = [&](int a) { return bar_base + 8u * (B0 + 4 + a); };   // S buffer written by both CTAs (even CTA)
  auto bar_sempty = [&](int a) { return bar_base + 8u * (B0 + 6 + a); };  // S buffer read by ML2
  auto bar_ofull = [&](int a) { return bar_base + 8u * (B0 + 8 + a); };   // O slot complete
  auto bar_oempty = [&](int a) { return bar_base + 8u * (B0 + 10 + a); }; // O slot drained by both CTAs (even CTA)
  const uint32_t bar_drain = bar_base + 8u * (B0 + 12);
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(smem + MlpSmem::OFF_MISC);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + MlpSmem::OFF_MISC + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // cluster of exactly two CTAs
  const uint32_t pm = rank & 1u;
  const uint32_t leader = 0u;
  const int cluster_id = blockIdx.x >> 1;
  const int num_clusters = gridDim.x >> 1;
  const int NC = (p.N1 + 127) / 128;  // a partial last chunk: W1 columns and W2 rows past N1 load as zeros, GELU(0 + 0) = 0
  const int total_tiles = p.batch * p.mpairs;
  const int my_tiles = cluster_id < total_tiles ? (total_tiles - cluster_id + num_clusters - 1) / num_clusters : 0;
  const int total = my_tiles * NC;  // chunks of this cluster's flat stream
  const WaitCtx w{s_abort, p.status, p.timeout_ns};
  griddep_launch_dependents();  // the next kernel's set-up may overlap this kernel (it waits before touching memory)
#ifdef COMFUSE_TRACE
  // phase timestamps of CTA 0 into a uint64[256] buffer: Epi1 set 0 at 0, set 1 at 40, Epi2 at 80, UMMA lane at 120, producer at 200
  int trace_ix = 0;
#define MLP_TRACE(cond, base, limit)                                                                             \
  do {                                                                                                           \
    if (p.trace && blockIdx.x == 0 && (cond) && trace_ix < (limit)) p.trace[(base) + trace_ix++] = globaltimer_ns(); \
  } while (0)
  if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) { p.trace[250] = globaltimer_ns(); p.trace[248] = clock64(); }  // kernel entry (time, cycles)
#else
#define MLP_TRACE(cond, base, limit) do { } while (0)
#endif

  if (threadIdx.x == 0) {
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_xfull(b), 2);
      mbar_init(bar_xempty(b), kEpi2Warps);  // every Epi2 warp, once its output stores have read the buffer
      mbar_init(bar_pfull(b), 1);
      mbar_init(bar_pfree(b), 2 * kEpi1Warps);  // every Epi1 warp of both CTAs
      mbar_init(bar_sfull(b), 2 * kEpi1Warps);
      mbar_init(bar_sempty(b), 1);
      mbar_init(bar_ofull(b), 1);
      mbar_init(bar_oempty(b), 2 * kEpi2Warps);
    }
    for (int s = 0; s < kWSlots; ++s) mbar_init(bar_wfull(s), 2);
    mbar_init(bar_drain, 1);
    mbar_init(bar_drain + 8u, 1);
    mbar_init(bar_drain + 16u, 1);  // the identity operand is written
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
  auto x_addr = [&](int buf, int kb) { return smem_base + MlpSmem::OFF_X + (buf * 2 + kb) * kBoxBytes; };
  auto w_addr = [&](int s) { return smem_base + MlpSmem::OFF_W + s * kBoxBytes; };
  auto s_addr = [&](int buf, int kb) { return smem_base + MlpSmem::OFF_S + (buf * 2 + kb) * kBoxBytes; };
  auto tile_of = [&](int i) { return cluster_id + i * num_clusters; };

  // Weight slots: W1 of chunk c lives in slot (c & 1), W2 of chunk c in slot 2 + (c & 1); each CTA holds its 64-column half.
  // A slot is handed back by the ONE commit its consumer issues anyway: ML1(c)'s completion (pfull) frees W1 slot c & 1
  // for chunk c + 2, ML2(c)'s completion (sempty) frees W2 slot c & 1 for chunk c + 2.  (The phase waited for is always
  // the barrier's latest one: the next phase belongs to the UMMAs that need the very load being issued.)
  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      int xi = 0;  // next X tile of this cluster to fetch
      // X of the cluster's xi-th tile into buffer xi & 1 (this CTA's 128 rows, two K blocks); false = buffer still in use
      auto push_x = [&](bool blocking) {
        if (!ok || xi >= my_tiles) return true;
        const int b = xi & 1;
        const uint32_t parity = ((xi >> 1) & 1u) ^ 1u;
        if (blocking) {
          if (!mbar_wait<false>(bar_xempty(b), parity, w)) { ok = false; return true; }
        } else if (!mbar_try_wait(bar_xempty(b), parity)) {
          return false;
        }
        const int tile = tile_of(xi);
        const int bz = tile / p.mpairs;
        const int m0 = (tile - bz * p.mpairs) * 256 + static_cast<int>(pm) * 128;
        const uint32_t full = map_to_cta(bar_xfull(b), leader);
        mbar_arrive_expect_tx_cluster(full, 2 * kBoxBytes);
        tma_load_3d_pair(x_addr(b, 0), &tmX, full, 0, m0, bz);
        tma_load_3d_pair(x_addr(b, 1), &tmX, full, 64, m0, bz);
        ++xi;
        return true;
      };
      auto push_w = [&](int slot, const CUtensorMap* tm, int x, int y) {
        const uint32_t full = map_to_cta(bar_wfull(slot), leader);
        MLP_TRACE(true, 200, 48);  // weight push
        mbar_arrive_expect_tx_cluster(full, kBoxBytes);
        tma_load_3d_pair(w_addr(slot), tm, full, x, y, 0);
      };
      const int wcol = static_cast<int>(pm) * 64;
      int j1 = 0, t1 = 0;  // chunk-in-tile / tile of the next W1 chunk
      // W1 of chunk c1 into slot c1 & 1 once ML1(c1 - 2) has completed
      auto push_w1 = [&](int c1) {
        if (j1 == 0)
          while (ok && xi <= t1) push_x(true);  // the chunk's X tile must be on its way before its first W1
        if (c1 >= 2 && ok && !mbar_wait<false>(bar_pfull(c1 & 1), ((c1 - 2) >> 1) & 1u, w)) ok = false;
        if (ok) push_w(c1 & 1, &tmW1, j1 * 128 + wcol, 0);
        if (++j1 == NC) { j1 = 0; ++t1; }
      };
      push_x(true);
      push_x(true);
      if (total > 0) push_w1(0);
      if (total > 1) push_w1(1);
      int j2 = 0;
      for (int c = 0; c < total && ok; ++c) {
        // in the order in which the slots come free: ML1(c) completes about one chunk before ML2(c - 2)
        if (c + 2 < total) push_w1(c + 2);
        // W2 of chunk c into slot 2 + (c & 1) once ML2(c - 2) has completed
        if (c >= 2 && ok && !mbar_wait<false>(bar_sempty(c & 1), ((c - 2) >> 1) & 1u, w)) { ok = false; break; }
        if (ok) push_w(2 + (c & 1), &tmW2, wcol, j2 * 128);
        if (++j2 == NC) j2 = 0;
        push_x(false);  // fetch the next X tile as soon as its buffer is free
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------ ML1 lane (even CTA)
    if (lane == 0 && pm == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(256, 128, false, true);
      int j1 = 0, t1 = 0;  // chunk-in-tile, tile
      for (int c = 0; c < total; ++c) {
        // P[c & 1] = X(t1) . W1[:, chunk j1]; the slot is free once the Epi1 warps hold chunk c - 2 in registers
        const int sb = c & 1;
        if (c >= 2 && !mbar_wait<false>(bar_pfree(sb), ((c - 2) >> 1) & 1u, w)) break;
        if (j1 == 0 && !mbar_wait<false>(bar_xfull(t1 & 1), (t1 >> 1) & 1u, w)) break;
        if (!mbar_wait<false>(bar_wfull(sb), (c >> 1) & 1u, w)) break;
        tcgen05_fence_after_sync();
        const uint64_t xdesc0 = make_smem_desc_sw128(x_addr(t1 & 1, 0), 16, 1024);
        const uint64_t xdesc1 = make_smem_desc_sw128(x_addr(t1 & 1, 1), 16, 1024);
        const uint64_t wdesc = make_smem_desc_sw128(w_addr(sb), 8192, 1024);
        const uint32_t d_p = tmem_base + sb * 128;
        MLP_TRACE(true, 120, 40);  // ML1 issue
#ifdef COMFUSE_TRACE
        if (!(p.trace_flags & 128))
#endif
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_bf16_ss_pair(d_p, (k < 4 ? xdesc0 : xdesc1) + static_cast<uint64_t>((k & 3) * 2), wdesc + static_cast<uint64_t>(k * 128),
                            idesc, k != 0 ? 1u : 0u);
        umma_commit_pair_both(bar_pfull(sb));  // P chunk complete; W1 slot free
        if (++j1 == NC) { j1 = 0; ++t1; }
      }
      umma_commit_pair(bar_drain);
      mbar_wait<false>(bar_drain, 0, w);
    }
  } else if (warp == kMl2Warp) {
    // ------------------------------------------------------------------------------------------ ML2 lane (even CTA)
    if (lane == 0 && pm == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(256, 128, false, true);
      int j2 = 0, t2 = 0;
      for (int c = 0; c < total; ++c) {
        // O(t2) += S_c . W2[chunk j2, :]
        const int sb = c & 1;
        const uint32_t d_o = tmem_base + 256 + (t2 & 1) * 128;
        if (j2 == 0) {
          // a new tile: O = X (2 I) -- the residual, at the scale of the rest -- while the first S chunk is being written.
          // The O slot must have been drained by Epi2 of the tile before the previous one.
          if (!mbar_wait<false>(bar_oempty(t2 & 1), ((t2 >> 1) & 1u) ^ 1u, w)) break;
          if (!mbar_wait<false>(bar_xfull(t2 & 1), (t2 >> 1) & 1u, w)) break;
          if (t2 == 0 && !mbar_wait<false>(bar_drain + 16u, 0, w)) break;
          tcgen05_fence_after_sync();
          const uint64_t xdesc0 = make_smem_desc_sw128(x_addr(t2 & 1, 0), 16, 1024);
          const uint64_t xdesc1 = make_smem_desc_sw128(x_addr(t2 & 1, 1), 16, 1024);
          const uint64_t eye_desc = make_smem_desc_sw128(smem_base + MlpSmem::OFF_I, 8192, 1024);
#pragma unroll
          for (int k = 0; k < 8; ++k)
            umma_bf16_ss_pair(d_o, (k < 4 ? xdesc0 : xdesc1) + static_cast<uint64_t>((k & 3) * 2), eye_desc + static_cast<uint64_t>(k * 128), idesc,
                              k != 0 ? 1u : 0u);
        }
        if (!mbar_wait<false>(bar_wfull(2 + sb), (c >> 1) & 1u, w)) break;
        if (!mbar_wait<false>(bar_sfull(sb), (c >> 1) & 1u, w)) break;
        tcgen05_fence_after_sync();
        const uint64_t wdesc = make_smem_desc_sw128(w_addr(2 + sb), 8192, 1024);
        const uint64_t sdesc0 = make_smem_desc_sw128(s_addr(sb, 0), 16, 1024);
        const uint64_t sdesc1 = make_smem_desc_sw128(s_addr(sb, 1), 16, 1024);
        MLP_TRACE(true, 160, 40);  // ML2 issue
#ifdef COMFUSE_TRACE
        if (!(p.trace_flags & 128))
#endif
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_bf16_ss_pair(d_o, (k < 4 ? sdesc0 : sdesc1) + static_cast<uint64_t>((k & 3) * 2), wdesc + static_cast<uint64_t>(k * 128), idesc,
                            1u);
        umma_commit_pair_both(bar_sempty(sb));  // S buffer and W2 slot free
        if (j2 == NC - 1) umma_commit_pair_both(bar_ofull(t2 & 1));
        if (++j2 == NC) { j2 = 0; ++t2; }
      }
      umma_commit_pair(bar_drain + 8u);
      mbar_wait<false>(bar_drain + 8u, 0, w);
    }
  } else {
    // the row vectors, widened to fp32 once, by the epilogue warps (idle until the first P chunk is complete)
    const int epi_tid = threadIdx.x - 64;
    for (int i = epi_tid; i < NC * 128; i += kEpiThreads) s_b1[i] = (p.b1 && i < p.N1) ? bf16_lo(p.b1[i]) : 0.f;
    {
      // this CTA's 64 columns of 2 I as a B operand: row k is one 128-byte line, 16-byte chunks swizzled by k & 7 (the
      // layout a TMA load of a W2 chunk half produces); column n of the half is column 64 pm + n of the identity
      uint4* id4 = reinterpret_cast<uint4*>(smem + MlpSmem::OFF_I);
      for (int i = epi_tid; i < kBoxBytes / 16; i += kEpiThreads) id4[i] = make_uint4(0u, 0u, 0u, 0u);
      named_barrier_sync(2, kEpiThreads);
      if (epi_tid < 64) {
        const int n = epi_tid, k = 64 * static_cast<int>(pm) + n;
        uint16_t* line = reinterpret_cast<uint16_t*>(smem + MlpSmem::OFF_I + k * 128);
        line[(((n >> 3) ^ (k & 7)) << 3) + (n & 7)] = 0x4000;  // bf16 2.0
      }
      fence_proxy_async_smem();
    }
    for (int i = epi_tid; i < 128; i += kEpiThreads) {
      s_b2[i] = p.b2 ? 2.f * bf16_lo(p.b2[i]) : 0.f;  // the accumulator is kept at twice its value
      s_gamma[i] = p.gamma ? bf16_lo(p.gamma[i]) : 1.f;
      s_beta[i] = p.beta ? bf16_lo(p.beta[i]) : 0.f;
    }
    named_barrier_sync(2, kEpiThreads);
    if (epi_tid == 0) mbar_arrive(bar_drain + 16u);
    const int q = warp & 3;  // TMEM lane quarter: rows 32q .. 32q+31
    const int row = q * 32 + lane;
    const uint32_t lane_sel = static_cast<uint32_t>(q * 32) << 16;
#define MLP_TRACE_EPI1() MLP_TRACE((warp == 2 || warp == 6 || warp == 10 || warp == 14) && lane == 0, 256 + (warp >> 2) * 40, 40)
#define MLP_TRACE_EPI2() MLP_TRACE(warp == 2 + kEpi1Warps && lane == 0, 80, 40)
#ifdef COMFUSE_TRACE
    const int tf = p.trace_flags;
#else
    constexpr int tf = 0;
#endif
    if (warp < 2 + kEpi1Warps) {
      // ---------------------------------------------------------------------------------------- Epi1
      // S_c = bf16(2 GELU(P_c + b1)) as the A operand of ML2(c): K-major, 128-byte swizzle; this thread's 32 columns are
      // four 16-byte chunks of its row in K block hh >> 1 of S buffer c & 1
      const int hh = (warp - 2) >> 2;
      const int kblk = hh >> 1, chunk0 = (hh & 1) * 4;
      const uint32_t pfree_leader = map_to_cta(bar_pfree(0), leader);
      const uint32_t sfull_leader = map_to_cta(bar_sfull(0), leader);
      int j = 0;
      for (int c = 0; c < total; ++c) {
        const int sb = c & 1;
        const uint32_t use = static_cast<uint32_t>(c) >> 1;
        mbar_wait<false>(bar_pfull(sb), use & 1u, w);
        __syncwarp();
        tcgen05_fence_after_sync();
        MLP_TRACE_EPI1();
        uint32_t v[32];
        tmem_ld_32cols(tmem_base + lane_sel + sb * 128 + hh * 32, v);
        // the chunk is in registers: its P slot may take chunk c + 2
        tcgen05_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_noflush(pfree_leader + 8u * sb);
        uint32_t pk[16];
        gelu2_pack_32<COMFUSE_B2B_POLY_EVERY>(v, s_b1 + j * 128 + hh * 32, pk, tf);
        // the S buffer is free once ML2 of chunk c - 2 has read it
        mbar_wait<false>(bar_sempty(sb), (use & 1u) ^ 1u, w);
        __syncwarp();
        store_row_chunks(pk, s_addr(sb, kblk), row, chunk0);
        fence_proxy_async_smem();  // S writes are visible to the tensor core's shared-memory reads
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_noflush(sfull_leader + 8u * sb);
        MLP_TRACE_EPI1();
        if (++j == NC) j = 0;
      }
      // ---------------------------------------------------------------------------------------- Epi2 of the LAST tile
      // Nothing is left to overlap it with, so the sixteen Epi1 warps take it instead of the four Epi2 warps: a thread owns
      // 32 of its row's 128 columns, the row statistics are merged across the four threads of the row through shared
      // memory (an S buffer: every UMMA that read it is complete once the O slot is full).
      if (my_tiles > 0) {
        const int i = my_tiles - 1;
        const int tile = tile_of(i);
        const int bz = tile / p.mpairs;
        const int m0 = (tile - bz * p.mpairs) * 256 + static_cast<int>(pm) * 128 + q * 32;
        const int ob = i & 1;
        const bool affine = p.gamma != nullptr || p.beta != nullptr;
        float2* s_part = reinterpret_cast<float2*>(smem + MlpSmem::OFF_S);  // [4][128] (mean, M2) of a thread's 32 columns
        mbar_wait<false>(bar_ofull(ob), (static_cast<uint32_t>(i) >> 1) & 1u, w);
        __syncwarp();
        tcgen05_fence_after_sync();
        uint32_t v[32];
        tmem_ld_32cols(tmem_base + lane_sel + 256 + ob * 128 + hh * 32, v);
        const float4* b4 = reinterpret_cast<const float4*>(s_b2 + hh * 32);
        const float shift = __uint_as_float(v[0]) + s_b2[hh * 32];
        const float2 ns = splat2(-shift);
        float2 s1 = splat2(0.f), s2 = splat2(0.f);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const float4 bb = b4[k];
          const float2 x01 = add2(f2_from_bits(v[4 * k], v[4 * k + 1]), make_float2(bb.x, bb.y));
          const float2 x23 = add2(f2_from_bits(v[4 * k + 2], v[4 * k + 3]), make_float2(bb.z, bb.w));
          v[4 * k] = __float_as_uint(x01.x); v[4 * k + 1] = __float_as_uint(x01.y);
          v[4 * k + 2] = __float_as_uint(x23.x); v[4 * k + 3] = __float_as_uint(x23.y);
          const float2 d01 = add2(x01, ns), d23 = add2(x23, ns);
          s1 = add2(s1, add2(d01, d23));
          s2 = fma2(d01, d01, s2);
          s2 = fma2(d23, d23, s2);
        }
        const float dsum = s1.x + s1.y;
        const float2 mine = make_float2(shift + dsum * (1.f / 32.f), fmaxf((s2.x + s2.y) - dsum * dsum * (1.f / 32.f), 0.f));
        s_part[hh * 128 + row] = mine;
        named_barrier_sync(3 + q, 128);  // the four warps of this lane quarter
        const float2 p0 = s_part[row], p1 = s_part[128 + row], p2 = s_part[256 + row], p3 = s_part[384 + row];
        const float mu = ((p0.x + p1.x) + (p2.x + p3.x)) * 0.25f;
        const float d0 = p0.x - mu, d1 = p1.x - mu, d2 = p2.x - mu, d3 = p3.x - mu;
        const float m2 = ((p0.y + p1.y) + (p2.y + p3.y)) + 32.f * ((d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3));  // equal-count Chan merge
        const float rstd = rsqrtf(m2 * (1.f / 128.f) + 4.f * p.eps);
        const float2 a2 = splat2(rstd), c2 = splat2(-mu * rstd);
        uint32_t pk[16];
        if (affine) {
          const float4* g4 = reinterpret_cast<const float4*>(s_gamma + hh * 32);
          const float4* be4 = reinterpret_cast<const float4*>(s_beta + hh * 32);
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const float4 gg = g4[k], be = be4[k];
            const float2 n01 = fma2(f2_from_bits(v[4 * k], v[4 * k + 1]), a2, c2);
            const float2 n23 = fma2(f2_from_bits(v[4 * k + 2], v[4 * k + 3]), a2, c2);
            pk[2 * k] = pack_bf16x2_rn(fma2(n01, make_float2(gg.x, gg.y), make_float2(be.x, be.y)));
            pk[2 * k + 1] = pack_bf16x2_rn(fma2(n23, make_float2(gg.z, gg.w), make_float2(be.z, be.w)));
          }
        } else {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            pk[2 * k] = pack_bf16x2_rn(fma2(f2_from_bits(v[4 * k], v[4 * k + 1]), a2, c2));
            pk[2 * k + 1] = pack_bf16x2_rn(fma2(f2_from_bits(v[4 * k + 2], v[4 * k + 3]), a2, c2));
          }
        }
        // staged over the tile's X operand like the other tiles' rows (its UMMAs are complete), one pair of stores per quarter
        store_row_chunks(pk, x_addr(i & 1, hh >> 1), row, (hh & 1) * 4);
        fence_proxy_async_smem();
        named_barrier_sync(3 + q, 128);
        if (hh == 0 && lane == 0 && COMFUSE_IN_BOUNDS(m0 >= 0 && m0 < p.mpairs * 256 && bz >= 0 && bz < p.batch, p.status)) {
          tma_store_3d(&tmO, x_addr(i & 1, 0) + q * 32 * 128, 0, m0, bz);
          tma_store_3d(&tmO, x_addr(i & 1, 1) + q * 32 * 128, 64, m0, bz);
          tma_store_commit();
          tma_store_wait_read<0>();  // the staging boxes must outlive the stores' reads
        }
      }
    } else {
      // ---------------------------------------------------------------------------------------- Epi2
      // The accumulator holds 2 (S W2 + X); x' = O + 2 b2 = 2 x; LayerNorm_eps(x) = (x' - mean') rsqrt(var' + 4 eps).
      // Two passes over the thread's 128 accumulator columns: sums of (x' - shift) and its square (shift = the row's
      // first value, so the subtraction cancels nothing that matters), then normalise, round once, stage, store.
      // The row is staged over the tile's X operand (its UMMAs are complete: the O slot was full), which goes back to the
      // producer when the stores have read it.  (Measured and dropped: storing the rows straight from registers, 64
      // contiguous bytes per thread and fragment -- the second pass took 2 us instead of 0.9 and slowed Epi1 beside it.)
      const uint32_t oempty_leader = map_to_cta(bar_oempty(0), leader);
      const bool affine = p.gamma != nullptr || p.beta != nullptr;
      const float eps4 = 4.f * p.eps;
      int pending_x = -1;  // lane 0: X buffer whose output stores have not yet been seen to have read it
      for (int i = 0; i + 1 < my_tiles; ++i) {  // the last tile is the Epi1 warps' (above)
        const int tile = tile_of(i);
        const int bz = tile / p.mpairs;
        const int m0 = (tile - bz * p.mpairs) * 256 + static_cast<int>(pm) * 128 + q * 32;
        const int ob = i & 1;
        if (lane == 0 && pending_x >= 0) {  // the X buffer goes back to the producer when the stores have read their boxes
          tma_store_wait_read<0>();
          mbar_arrive(bar_xempty(pending_x));
          pending_x = -1;
        }
        mbar_wait<false>(bar_ofull(ob), (i >> 1) & 1u, w);
        __syncwarp();
        tcgen05_fence_after_sync();
        MLP_TRACE_EPI2();
        const uint32_t o_addr = tmem_base + lane_sel + 256 + ob * 128;
        float shift = 0.f;
        float2 s1 = splat2(0.f), s2 = splat2(0.f);
#pragma unroll 1
        for (int f = 0; f < 4; ++f) {
          uint32_t v[32];
          tmem_ld_32cols(o_addr + f * 32, v);
          const float4* b4 = reinterpret_cast<const float4*>(s_b2 + f * 32);
          if (f == 0) shift = __uint_as_float(v[0]) + s_b2[0];
          const float2 ns = splat2(-shift);
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const float4 bb = b4[k];
            const float2 d01 = add2(f2_from_bits(v[4 * k], v[4 * k + 1]), add2(make_float2(bb.x, bb.y), ns));
            const float2 d23 = add2(f2_from_bits(v[4 * k + 2], v[4 * k + 3]), add2(make_float2(bb.z, bb.w), ns));
            s1 = add2(s1, add2(d01, d23));
            s2 = fma2(d01, d01, s2);
            s2 = fma2(d23, d23, s2);
          }
        }
        const float dm = (s1.x + s1.y) * (1.f / 128.f);
        const float mu = shift + dm;
        const float var = fmaxf((s2.x + s2.y) * (1.f / 128.f) - dm * dm, 0.f);
        const float rstd = rsqrtf(var + eps4);
        const float2 a2 = splat2(rstd), c2 = splat2(-mu * rstd);
        MLP_TRACE_EPI2();
#pragma unroll 1
        for (int f = 0; f < 4; ++f) {
          uint32_t v[32];
          tmem_ld_32cols(o_addr + f * 32, v);
          if (f == 3) {
            // the accumulator has been read for the last time: the O slot can be reused by the tile after the next one
            tcgen05_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster_noflush(oempty_leader + 8u * ob);
          }
          const float4* b4 = reinterpret_cast<const float4*>(s_b2 + f * 32);
          uint32_t pk[16];
          if (affine) {
            const float4* g4 = reinterpret_cast<const float4*>(s_gamma + f * 32);
            const float4* be4 = reinterpret_cast<const float4*>(s_beta + f * 32);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const float4 bb = b4[k], gg = g4[k], be = be4[k];
              const float2 n01 = fma2(add2(f2_from_bits(v[4 * k], v[4 * k + 1]), make_float2(bb.x, bb.y)), a2, c2);
              const float2 n23 = fma2(add2(f2_from_bits(v[4 * k + 2], v[4 * k + 3]), make_float2(bb.z, bb.w)), a2, c2);
              pk[2 * k] = pack_bf16x2_rn(fma2(n01, make_float2(gg.x, gg.y), make_float2(be.x, be.y)));
              pk[2 * k + 1] = pack_bf16x2_rn(fma2(n23, make_float2(gg.z, gg.w), make_float2(be.z, be.w)));
            }
          } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const float4 bb = b4[k];
              pk[2 * k] = pack_bf16x2_rn(fma2(add2(f2_from_bits(v[4 * k], v[4 * k + 1]), make_float2(bb.x, bb.y)), a2, c2));
              pk[2 * k + 1] = pack_bf16x2_rn(fma2(add2(f2_from_bits(v[4 * k + 2], v[4 * k + 3]), make_float2(bb.z, bb.w)), a2, c2));
            }
          }
          store_row_chunks(pk, x_addr(i & 1, f >> 1), row, (f & 1) * 4);  // 32 rows of K block f >> 1
          if (f & 1) {
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0 && COMFUSE_IN_BOUNDS(m0 >= 0 && m0 < p.mpairs * 256 && bz >= 0 && bz < p.batch, p.status))
              tma_store_3d(&tmO, x_addr(i & 1, f >> 1) + q * 32 * 128, (f >> 1) * 64, m0, bz);
          }
        }
        if (lane == 0) {
          tma_store_commit();
          pending_x = i & 1;
        }
        MLP_TRACE_EPI2();
      }
      if (lane == 0) tma_store_wait_read<0>();  // the staging boxes must outlive the last stores' reads
    }
  }

#ifdef COMFUSE_TRACE
  if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) p.trace[251] = globaltimer_ns();  // first epilogue warp done
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
  if (p.trace && blockIdx.x == 0 && threadIdx.x == 64) { p.trace[252] = globaltimer_ns(); p.trace[249] = clock64(); }  // kernel exit
#endif
}

}  // namespace

bool b2b_mlp_supported(int K, int N1, int N2) { return K == 128 && N2 == 128 && N1 >= 8 && N1 <= MlpSmem::kMaxN1 && N1 % 8 == 0; }

cudaError_t launch_b2b_mlp(const void* X, const void* W1, const void* W2, B2bParams p, cudaStream_t st) {
  const DeviceInfo* dev = current_device_info();
  if (!dev) return cudaErrorInvalidDevice;
  CUtensorMap tmX, tmW1, tmW2, tmO;
  const uint64_t M = p.M, K = p.K, N1 = p.N1, N2 = p.N2;
  if (p.batch < 1) p.batch = 1;
  const uint64_t nb = static_cast<uint64_t>(p.batch);
  // operand boxes are 64 elements x 128 rows, the output box is one Epi2 warp's 64 x 32
  if (!encode_tmap_bf16_3d(&tmX, X, K, M, nb, K * 2, M * K * 2, 128) ||
      !encode_tmap_bf16_3d(&tmW1, W1, N1, K, 1, N1 * 2, K * N1 * 2, 128) ||
      !encode_tmap_bf16_3d(&tmW2, W2, N2, N1, 1, N2 * 2, N1 * N2 * 2, 128) ||
      !encode_tmap_bf16_3d(&tmO, p.O, N2, M, nb, N2 * 2, M * N2 * 2, 32))
    return cudaErrorInvalidValue;
  p.mblocks = (p.M + 127) / 128;
  p.mpairs = (p.mblocks + 1) / 2;

  constexpr int kMaxDev = 64;
  static std::atomic<int> max_clusters[kMaxDev];  // 0 = kernel not configured yet on that device (set last, released)
  const int di = dev->device < kMaxDev ? dev->device : kMaxDev - 1;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.blockDim = dim3(kMlpThreads, 1, 1);
  cfg.dynamicSmemBytes = MlpSmem::BYTES;
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
    cudaError_t e = cudaFuncSetAttribute(b2b_mlp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MlpSmem::BYTES);
    if (e != cudaSuccess) return e;
    int n = 0;
    cfg.gridDim = dim3(2 * dev->sm_count, 1, 1);
    e = cudaOccupancyMaxActiveClusters(&n, b2b_mlp_kernel, &cfg);
    if (e != cudaSuccess) return e;
    if (n <= 0) return cudaErrorLaunchOutOfResources;
    max_clusters[di].store(n, std::memory_order_release);
    ncl = n;
  }
  const int tiles = p.batch * p.mpairs;
  const int clusters = tiles < ncl ? tiles : ncl;
  cfg.gridDim = dim3(clusters * 2, 1, 1);
  count_launch();
  return cudaLaunchKernelEx(&cfg, b2b_mlp_kernel, tmX, tmW1, tmW2, tmO, p);
}

}  // namespace comfuse
