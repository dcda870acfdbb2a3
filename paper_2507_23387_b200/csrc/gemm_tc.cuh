// The tensor-core kernels of the library, one template:
//
//   <NTERMS = 1, FUSED = false> : D (+)= A16 * B16       one pass of the unfused path (Sec. 5.4
//                                                        runs each product through its own pipeline)
//   <NTERMS = 3, FUSED = false> : C = hi_A hi_B + 2^-s (lo_A hi_B + hi_A lo_B) from FP16 words that
//                                 were split beforehand: all three products of Eq. recover_eqn
//   <NTERMS = 3, FUSED = true>  : the same from the FP32 operands: converter warps split them on
//                                 the fly (Eq. recover_eqn, first two lines), so no FP16 copy of
//                                 A or B ever goes through device memory
//   termwise (Eq. termwise) or elementwise (Eq. elementwise) accumulation for NTERMS == 3.
//
// Structure (one persistent CTA per SM):
//   warps 0-7    accumulate/epilogue warps: tcgen05.ld the TMEM partial sums, add them with FP32
//                round-to-nearest into running sums held in registers, form C, store it
//   not FUSED (384 threads): warp 8 = TMA producer (FP16 tiles global -> shared, swizzled UMMA
//                layout), warp 9 = MMA issuer
//   FUSED (512 threads): warp 13 = TMA producer: FP32 tiles of A and B global -> shared (128-byte
//                swizzle) into a ring of stages; warps 8-11 = converter warps: each FP32 stage is
//                split IN PLACE into (hi, lo) FP16 words laid out as swizzled UMMA atoms (every
//                converter thread works on the same positions of every stage, so its offsets are
//                constants); warps 14-15 = relay threads: the generic -> async proxy fence and, in
//                a CTA pair, the arrival on the leader's barrier, kept off the converter warps;
//                warp 12 = MMA issuer.
//   The MMA issuer is one thread issuing tcgen05.mma kind::f16 (M = 128, N = 256, K = 16).
//
// Why the running sums live in registers.  The tensor core adds products into its FP32
// accumulator without round-to-nearest, so a long chain accumulated only inside TMEM drifts
// (the reason earlier GPU work accumulates outside the matrix unit, Sec. 4.3 last paragraph).
// The k dimension is therefore cut into blocks g of `kchunk` elements (the k-blocks of Sec. 4.5);
// each block's product is accumulated in TMEM from zero and then added, with an IEEE RN FP32
// addition, to the register-resident sum.  For the termwise order only the dominant hi*hi stream
// needs this; the correction stream (scaled by 2^-s at the end) is carried in TMEM for the whole k.
//
// TMEM: 512 columns = two regions of 256 columns (one 128 x 256 FP32 tile each).
//   NTERMS == 1             : the regions alternate between consecutive k-blocks (double buffer)
//   NTERMS == 3 termwise    : R0 = hi*hi partial of the current k-block, R1 = correction stream
//   NTERMS == 3 elementwise : R0 = hi*hi partial, R1 = correction partial of the current k-block
//   NTERMS == 3 reordered elementwise, s <= 15: each k-block's value P_x / s_f + P_hh is formed in
//                             one region (scale-d MMA, see reord_fast); the regions alternate
#pragma once

#include <cuda_fp16.h>

#include <type_traits>

#include "ptx_sm100.cuh"

namespace sgc {

constexpr int kBM = 128;            // CTA tile rows  (UMMA M)
constexpr int kBN = 256;            // CTA tile cols  (UMMA N)
constexpr int kNumEpiWarps = 8;     // warps 0-7
constexpr int kTcThreads = 384;     // not FUSED: + TMA warp + MMA warp (+ 2 idle warps: whole warpgroup)
// FUSED register split between the accumulate warps and the rest (512 threads x 128 registers),
// columns per TMEM load in the accumulate warps, regions a converter warp loads before converting
#ifndef SGC_FUSED_EPI_REGS
#define SGC_FUSED_EPI_REGS 208
#endif
#ifndef SGC_FUSED_OTHER_REGS
#define SGC_FUSED_OTHER_REGS 48
#endif
#ifndef SGC_FUSED_GW
#define SGC_FUSED_GW 64
#endif
#ifndef SGC_CONV_BATCH
#define SGC_CONV_BATCH 2
#endif
#ifndef SGC_CONV_WARPS
#define SGC_CONV_WARPS 4
#endif
constexpr int kNumConvWarps = SGC_CONV_WARPS;      // a multiple of 4 (see the converter role)
// FUSED: + converter warps + MMA warp + TMA warp + 2 relay warps, rounded up to whole warpgroups
constexpr int kFusedThreads = ((kNumEpiWarps + kNumConvWarps + 4 + 3) / 4) * 128;
constexpr uint32_t kTmemCols = 512;

// error codes written to the device error word (which wait gave up)
enum : unsigned int {
  kErrProducerEmptyWait = 0x101,
  kErrMmaFullWait = 0x102,
  kErrMmaTmemEmptyWait = 0x103,
  kErrEpiTmemFullWait = 0x104,
  kErrDrainWait = 0x105,
  kErrConvEmptyWait = 0x106,
  kErrConvFullWait = 0x107,
  kErrRelayWait = 0x108,
  kErrProbeWait = 0x1F0,
};

// Optional role timing (compile with -DSGC_ROLE_TIMING): CTA 0 adds the clocks each role spends in
// its phases to a global table; used only for performance investigations.
#ifdef SGC_ROLE_TIMING
__device__ unsigned long long g_role_timing[16];
#define SGC_T0() const long long sgc_t0_ = clock64()
#define SGC_TADD(slot, cond) do { if (cond) atomicAdd(&g_role_timing[slot], (unsigned long long)(clock64() - sgc_t0_)); } while (0)
#else
#define SGC_T0() do {} while (0)
#define SGC_TADD(slot, cond) do {} while (0)
#endif

struct TcGemmParams {
  int M, N, K;
  float* D;             // output (C for NTERMS == 3)
  long long ldd;
  int accumulate;       // NTERMS == 1 only: D += result
  int order;            // NTERMS == 3: 0 termwise, 1 elementwise
  int kchunk_blocks;    // k-block length in units of the stage depth BK
  float inv_scale;      // 2^-s
  unsigned int* err;    // device error word
  float scale;          // FUSED only: 2^s (the FP32 operands themselves come through the tensor maps)
  // Split-K (not FUSED, NTERMS == 3): the k range is cut into `ksplit` slices of `kslice_blocks`
  // stages (a multiple of kchunk_blocks); unit u = slice * tiles + tile writes its hi*hi sums to
  // Phh + slice * pstride and, termwise, its raw correction sums to Px + slice * pstride (both
  // M x ldp); a reduction kernel forms C.  Phh == nullptr (then ksplit == 1): the kernel writes
  // C itself.  Phh != nullptr with ksplit == 1 is the four-term path, whose reduction kernel
  // adds the low-low product.
  int ksplit;
  int kslice_blocks;
  float* Phh;
  float* Px;
  long long pstride;
  long long ldp;
  // Optional (may be null): thread 0 of CTA 0 stores how long it ran, {SM clocks, nanoseconds of
  // the global timer}, from which the host gets the SM clock the kernel actually ran at.
  unsigned long long* kclock;
};

#ifndef SGC_PAIR_GROUP
#define SGC_PAIR_GROUP 8
#endif
#ifndef SGC_BK3
#define SGC_BK3 64
#endif
template <int NTERMS, bool PAIR = false, bool FUSED = false>
struct TcCfg {
  // k per pipeline stage: 64 for one product; for three products 32 in the fused kernel (FP32
  // stages: six of 32 KB for CTA pairs, four of 48 KB for single CTAs), SGC_BK3 (64, 32 or 16) when
  // TMA loads FP16 words: 64 gives two 96 KB stages (three 64 KB ones for CTA pairs) and measured
  // 1-3 % faster than four stages of 32 across sizes; 16 much slower
  static constexpr int BK = (NTERMS == 1) ? 64 : (FUSED ? 32 : SGC_BK3);
  static constexpr int BN_CTA = PAIR ? kBN / 2 : kBN;     // B columns held by one CTA
  static constexpr int A_ROW_BYTES = BK * 2;              // 128 or 64: also the swizzle span of A
  static constexpr uint32_t A_TILE = kBM * BK * 2;        // one FP16 A tile
  static constexpr uint32_t B_TILE = BK * BN_CTA * 2;     // one FP16 B tile (this CTA's columns)
  // FUSED: a stage is filled by TMA with the FP32 tiles (A: 128 rows x BK; B: BN_CTA / 32 boxes of
  // BK k-rows x 32 columns; rows of 128 bytes, 128-byte swizzle) and converted IN PLACE: every
  // 1 KB region (8 rows x 32 FP32 elements) becomes the 512-byte hi atom and the 512-byte lo atom
  // of the same 8 x 32 elements (rows of 64 bytes, 64-byte swizzle).  One ring, each slot going
  // TMA -> converters -> MMA -> TMA, so the same bytes hold a tile in flight, a tile being split
  // and a tile being multiplied, whichever the pipeline needs more of.
  static constexpr uint32_t A32_TILE = FUSED ? kBM * BK * 4 : 0;
  static constexpr uint32_t B32_TILE = FUSED ? BK * BN_CTA * 4 : 0;
  static constexpr uint32_t STAGE_BYTES =
      FUSED ? (A32_TILE + B32_TILE) : ((NTERMS == 1) ? (A_TILE + B_TILE) : 2 * (A_TILE + B_TILE));
  static constexpr int STAGES = (196608 / STAGE_BYTES) > 8 ? 8 : (int)(196608 / STAGE_BYTES);
  static constexpr uint32_t RING_BYTES = STAGES * STAGE_BYTES;
  // Where the MMA thread finds the operands of a stage, and their descriptor strides.
  static constexpr uint32_t A_LO_OFF = FUSED ? 512 : A_TILE;                 // lo_A relative to hi_A
  static constexpr uint32_t B_OFF = FUSED ? A32_TILE : ((NTERMS == 3) ? 2 * A_TILE : A_TILE);
  static constexpr uint32_t B_LO_OFF = FUSED ? 512 : B_TILE;                 // lo_B relative to hi_B
  static constexpr uint32_t A_SBO = FUSED ? 1024 : 8 * A_ROW_BYTES;          // next 8 rows of A
  static constexpr uint32_t B_LBO = BK * 128;    // next column atom of B (64 columns; FUSED: 32)
  static constexpr uint32_t B_SBO = 1024;        // next 8 k-rows of the same columns
  static constexpr uint32_t STORE_STAGING = kNumEpiWarps * 4096;   // 32 rows x 128 bytes per warp
  static constexpr uint32_t SMEM_BYTES =
      RING_BYTES + 1024 /*align*/ + 256 /*barriers*/ + STORE_STAGING;
};

// Tile rasterisation: groups of `group_m` tile-rows are walked column by column so that the CTAs
// running at the same time share A and B tiles in L2.  A wave of 148 tiles then covers about
// group_m x 148 / group_m tiles; its DRAM traffic is the A rows plus the B columns it spans, least
// when 128 rows x group_m is close to 256 columns x 148 / group_m (16 for 128-row tiles, 8 for
// the 256-row tiles of CTA pairs).
__device__ __forceinline__ void tile_coords(int tile, int num_m, int num_n, int& tm, int& tn,
                                            int group_m = 16) {
  const int kGroupM = group_m;
  const int per_group = kGroupM * num_n;
  const int group = tile / per_group;
  const int first_m = group * kGroupM;
  const int gsz = min(num_m - first_m, kGroupM);
  const int in_group = tile - group * per_group;
  tm = first_m + in_group % gsz;
  tn = in_group / gsz;
}

// Epilogue helper: thread-owned row `row`, columns [col0, col0 + 16) of the output.
__device__ __forceinline__ void store16(float* D, long long ldd, int M, int N, int row, int col0,
                                        const float* v, bool vec_ok, int accumulate) {
  if (row >= M || col0 >= N) return;
  float* p = D + (long long)row * ldd + col0;
  if (vec_ok && col0 + 16 <= N) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float4 o = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
      if (accumulate) {
        const float4 old = *reinterpret_cast<const float4*>(p + 4 * q);
        o.x = __fadd_rn(old.x, o.x); o.y = __fadd_rn(old.y, o.y);
        o.z = __fadd_rn(old.z, o.z); o.w = __fadd_rn(old.w, o.w);
      }
      *reinterpret_cast<float4*>(p + 4 * q) = o;
    }
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (col0 + j < N) p[j] = accumulate ? __fadd_rn(p[j], v[j]) : v[j];
  }
}

// ------------------------------------------------------------------------------------------
// Converter-warp helpers (FUSED).  One "item" is 8 consecutive FP32 elements of a tile row: two
// 16-byte chunks of the FP32 ring in, one 16-byte chunk of the hi tile and one of the lo tile out.
struct ConvScale {
  float scale;            // 2^s
  uint64_t scale2;        // {2^s, 2^s} packed
  uint16_t neg_scale_h;   // -2^s as FP16 (valid when fast)
  bool fast;              // s <= 15
};

// Two elements, plain form:  hi = fl16(x); lo = fl16((x - hi) * 2^s); the subtraction and the
// scaling are exact (Sec. 3.3).
__device__ __forceinline__ void split_pair(uint64_t xp, float scale, uint32_t& hi2, uint32_t& lo2) {
  float x0, x1;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(x0), "=f"(x1) : "l"(xp));
  const __half2 h = __floats2half2_rn(x0, x1);
  const float2 hf = __half22float2(h);
  const __half2 l = __floats2half2_rn(__fmul_rn(__fsub_rn(x0, hf.x), scale),
                                      __fmul_rn(__fsub_rn(x1, hf.y), scale));
  hi2 = *reinterpret_cast<const uint32_t*>(&h);
  lo2 = *reinterpret_cast<const uint32_t*>(&l);
}

// The same words in five instructions per pair, for s <= 15 (2^s representable in FP16):
//   hi = cvt.f16x2(x)       packed conversion
//   xs = x * 2^s            one packed FP32x2 multiply (exact)
//   t  = hi * (-2^s) + xs   one mixed-precision FMA per element (FP16 x FP16 + FP32): the exact value
//                           (x - hi) * 2^s is representable, so the single rounding changes nothing
//   lo = cvt.f16x2(t)
// (For |x| >= 2^(128-s), outside the method's range, xs overflows and lo becomes NaN where the
// plain form gives inf.)
__device__ __forceinline__ void split_pair_fast(uint64_t xp, uint64_t scale2, uint16_t neg_scale_h,
                                                uint32_t& hi2, uint32_t& lo2) {
  float x0, x1;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(x0), "=f"(x1) : "l"(xp));
  uint32_t h;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(h) : "f"(x1), "f"(x0));
  uint64_t xs;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(xs) : "l"(xp), "l"(scale2));
  float xs0, xs1, t0, t1;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(xs0), "=f"(xs1) : "l"(xs));
  uint16_t h0, h1;
  asm("mov.b32 {%0, %1}, %2;" : "=h"(h0), "=h"(h1) : "r"(h));
  asm("fma.rn.f32.f16 %0, %1, %2, %3;" : "=f"(t0) : "h"(h0), "h"(neg_scale_h), "f"(xs0));
  asm("fma.rn.f32.f16 %0, %1, %2, %3;" : "=f"(t1) : "h"(h1), "h"(neg_scale_h), "f"(xs1));
  uint32_t l;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(l) : "f"(t1), "f"(t0));
  hi2 = h;
  lo2 = l;
}

// One item: FP32 chunks at shared addresses src0 / src1 (elements 0-3 / 4-7) -> hi chunk at dst,
// lo chunk at dst + lo_off.  Loading and converting are separate so that a warp can have the
// loads of several items in flight before it starts on the arithmetic of the first.
struct ConvItem { uint64_t x01, x23, x45, x67; };

__device__ __forceinline__ void load_item(ConvItem& it, uint32_t src0, uint32_t src1) {
  asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(it.x01), "=l"(it.x23) : "r"(src0));
  asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(it.x45), "=l"(it.x67) : "r"(src1));
}

template <bool FAST>
__device__ __forceinline__ void convert_store(const ConvItem& it, uint32_t dst, uint32_t lo_off,
                                              const ConvScale& cs) {
  uint4 h, l;
  if (FAST) {
    split_pair_fast(it.x01, cs.scale2, cs.neg_scale_h, h.x, l.x);
    split_pair_fast(it.x23, cs.scale2, cs.neg_scale_h, h.y, l.y);
    split_pair_fast(it.x45, cs.scale2, cs.neg_scale_h, h.z, l.z);
    split_pair_fast(it.x67, cs.scale2, cs.neg_scale_h, h.w, l.w);
  } else {
    split_pair(it.x01, cs.scale, h.x, l.x);
    split_pair(it.x23, cs.scale, h.y, l.y);
    split_pair(it.x45, cs.scale, h.z, l.z);
    split_pair(it.x67, cs.scale, h.w, l.w);
  }
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(h.x), "r"(h.y),
               "r"(h.z), "r"(h.w));
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + lo_off), "r"(l.x), "r"(l.y),
               "r"(l.z), "r"(l.w));
}

__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[16]) { tmem_ld_32x32b_x16(taddr, r); }
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[32]) { tmem_ld_32x32b_x32(taddr, r); }
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[64]) { tmem_ld_32x32b_x64(taddr, r); }

// REORD: the reordered elementwise order (p.order == 2) has its own instantiations, so that its
// accumulate path (two chunk buffers live at once) does not weigh on the register allocation of
// the termwise / elementwise kernels.
template <int NTERMS, bool FUSED, bool PAIR, bool REORD = false>
__global__ void __launch_bounds__(FUSED ? kFusedThreads : kTcThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
               const __grid_constant__ CUtensorMap tmB0, const __grid_constant__ CUtensorMap tmB1,
               const TcGemmParams p) {
  using Cfg = TcCfg<NTERMS, PAIR, FUSED>;
  constexpr int BK = Cfg::BK;
  constexpr int STAGES = Cfg::STAGES;
  // PAIR: the kernel runs as clusters of two CTAs driving tcgen05.mma.cta_group::2.  The pair owns
  // a 256 x 256 tile: CTA rank r holds rows [128 r, 128 r + 128) of A and of the result (its own
  // TMEM lanes) and columns [128 r, 128 r + 128) of the B tile; rank 0 (the leader) issues the MMAs
  // for both, so the "full" and "TMEM drained" barriers that its MMA thread waits on live in the
  // leader and are signalled by both CTAs, while its commits arrive on the barriers of both.
  const uint32_t cta_rank = PAIR ? cluster_ctarank() : 0u;
  const bool leader = (cta_rank == 0);
  // not FUSED: warp 8 loads FP16 tiles; FUSED: the warp after the MMA warp loads FP32 tiles
  constexpr int kMmaWarp = FUSED ? kNumEpiWarps + kNumConvWarps : 9;
  constexpr int kProducerWarp = FUSED ? kMmaWarp + 1 : 8;
  static_assert(!FUSED || NTERMS == 3, "the fused kernel computes all three products");

  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment: the swizzle pattern of TMA and of the UMMA descriptors is a function
  // of the shared-memory address bits, so every tile must start on a 1024-byte boundary.
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::RING_BYTES);
  uint64_t* full_bar = bars;                 // [STAGES]  producer (FUSED: relay threads) -> MMA
  uint64_t* empty_bar = bars + STAGES;       // [STAGES]  MMA -> producer
  uint64_t* tfull_bar = bars + 2 * STAGES;   // [2]       MMA -> epilogue (TMEM region filled)
  uint64_t* tempty_bar = bars + 2 * STAGES + 2;  // [2]   epilogue -> MMA (TMEM region drained)
  uint64_t* drain_bar = bars + 2 * STAGES + 4;   // [1]
  constexpr int kFusedBars = FUSED ? STAGES : 0;
  uint64_t* full32_bar = bars + 2 * STAGES + 5;              // [STAGES]  FUSED: TMA -> converters
  uint64_t* conv_bar = bars + 2 * STAGES + 5 + kFusedBars;   // [STAGES]  FUSED: converters -> relay
  uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 5 + 2 * kFusedBars);
  volatile uint32_t* abort_flag = tmem_base_slot + 1;
  // PAIR: a wait that gives up also raises the peer's flag (shared::cluster address of the same slot)
  const uint32_t peer_abort =
      PAIR ? mapa_u32(smem_u32(tmem_base_slot + 1), cta_rank ^ 1u) : 0u;
  static_assert((2 * STAGES + 5 + 2 * kFusedBars) * 8 + 8 <= 256, "barrier block");
  uint8_t* store_staging = smem + Cfg::RING_BYTES + 256;   // epilogue transposition buffers

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  long long kclock_clk0 = 0;
  unsigned long long kclock_ns0 = 0;
  const bool kclock_on = (p.kclock != nullptr) && blockIdx.x == 0 && threadIdx.x == 0;
  if (kclock_on) {
    kclock_clk0 = clock64();
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(kclock_ns0));
  }
#ifdef SGC_ROLE_TIMING
  long long sgc_k_clk0 = 0;
  unsigned long long sgc_k_ns0 = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    sgc_k_clk0 = clock64();
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(sgc_k_ns0));
  }
#endif

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], (FUSED && PAIR) ? 2 : 1);   // FUSED: one relay thread per CTA
      mbar_init(&empty_bar[s], 1);
    }
    for (int r = 0; r < 2; ++r) {
      mbar_init(&tfull_bar[r], 1);
      mbar_init(&tempty_bar[r], kNumEpiWarps * (PAIR ? 2 : 1));
    }
    for (int s = 0; s < kFusedBars; ++s) {
      mbar_init(&full32_bar[s], 1);
      mbar_init(&conv_bar[s], kNumConvWarps);
    }
    mbar_init(drain_bar, 1);
    *abort_flag = 0u;
    fence_mbar_init();
  }
  if (warp == kProducerWarp && lane == 0) {
    tma_prefetch_desc(&tmA0); tma_prefetch_desc(&tmB0);
    if (NTERMS == 3 && !FUSED) { tma_prefetch_desc(&tmA1); tma_prefetch_desc(&tmB1); }
  }
  if (warp == kMmaWarp) {    // whole warp (the same warp in both CTAs of a pair): all 512 TMEM columns
    if (PAIR) { tmem_alloc_pair(tmem_base_slot, kTmemCols); tmem_relinquish_pair(); }
    else { tmem_alloc(tmem_base_slot, kTmemCols); tmem_relinquish(); }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (PAIR) cluster_sync_all();      // the peer's barriers are initialised before anyone signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_base_slot;

  // Work units: 128-row tiles, or 256-row pair tiles of which this CTA takes row block `cta_rank`.
  const int num_m = PAIR ? (p.M + 2 * kBM - 1) / (2 * kBM) : (p.M + kBM - 1) / kBM;
  const int num_n = (p.N + kBN - 1) / kBN;
  const int num_tiles = num_m * num_n;
  const int first_tile = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int tile_stride = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  auto tile_rc = [&](int tile, int& tm, int& tn) {     // tm in units of 128 rows, tn of 256 columns
    tile_coords(tile, num_m, num_n, tm, tn, PAIR ? SGC_PAIR_GROUP : 16);
    if (PAIR) tm = tm * 2 + (int)cta_rank;
  };
  const int num_kb = (p.K + BK - 1) / BK;                      // pipeline stages per tile
  const int ksplit = FUSED ? 1 : p.ksplit;
  const int num_units = num_tiles * ksplit;
  // Work unit -> tile coordinates and its range of stages [kb0, kb1).
  auto unit_rc = [&](int unit, int& tm, int& tn, int& kb0, int& kb1, int& slice) {
    slice = unit / num_tiles;
    tile_rc(unit - slice * num_tiles, tm, tn);
    kb0 = (ksplit > 1) ? slice * p.kslice_blocks : 0;
    kb1 = (ksplit > 1) ? min(num_kb, kb0 + p.kslice_blocks) : num_kb;
  };
  const int chunk = p.kchunk_blocks;                           // stages per k-block g
  // Reordered elementwise order, fast form: a k-block's value P_x / s_f + P_hh is formed inside one
  // TMEM region (the correction products first, then the first hi*hi MMA scales the accumulator
  // by 2^-s as it adds: tcgen05.mma's scale-d operand), so the accumulate warps read one region per
  // block and the two regions alternate between blocks: block g + 1 accumulates while block g is
  // read.  Needs s <= 15 (the instruction's range) and all stages of a block resident at once.
  const int scale_exp = 127 - (int)((__float_as_uint(p.inv_scale) >> 23) & 0xFFu);
  const bool reord_fast = REORD && (NTERMS == 3) && scale_exp >= 0 && scale_exp <= 15 && 2 * chunk <= STAGES;

  // Register budget when FUSED (512 threads x 128 registers): the accumulate warps hold a
  // 128 x 256 FP32 tile in registers, so warpgroups 2-3 hand registers over to warpgroups 0-1
  // (256 x 168 + 256 x 88 = 65536).  Each setmaxnreg sits at the top of its role's branch so
  // that the code below it is compiled against the new limit.
  if (warp < kNumEpiWarps) {
    if (FUSED) setmaxnreg_inc<SGC_FUSED_EPI_REGS>();
    else setmaxnreg_inc<208>();       // 384 threads x 168: 256 x 208 + 128 x 56 fits the pool
    // ------------------------------------------------------------------ accumulate / epilogue
    const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31 (warp id mod 4)
    const int half = warp >> 2;                   // columns [128*half, 128*half + 128)
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(p.D) & 15) == 0) && ((p.ldd & 3) == 0);
    uint32_t drains[2] = {0, 0};
    uint32_t gchunk = 0;
    bool ok = true;
    float S[128];
    // TMEM is read 64 columns at a time (fewer, longer loads: the tensor pipe is held up for as
    // long as a drain lasts, and the load latency is most of that), 16 where registers are tight.
    constexpr int GW = FUSED ? SGC_FUSED_GW : 64;
    // The k-block additions as packed FP32x2 instructions (IEEE per lane: same results, half the
    // issue slots): elementwise 4096^3 338 -> 365 TFLOP/s.  Not in the fused kernel, whose
    // converter warps keep the packed pipe busy (there it measured 279 -> 246).
    constexpr bool kPackedDrain = !FUSED;
    uint64_t inv_scale2;
    asm("mov.b64 %0, {%1, %1};" : "=l"(inv_scale2) : "f"(p.inv_scale));
    auto add2 = [](float& s0, float& s1, uint32_t v0, uint32_t v1) {
      uint64_t a, b, c;
      asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "f"(s0), "f"(s1));
      asm("mov.b64 %0, {%1, %2};" : "=l"(b) : "r"(v0), "r"(v1));
      asm("add.rn.f32x2 %0, %1, %2;" : "=l"(c) : "l"(a), "l"(b));
      asm("mov.b64 {%0, %1}, %2;" : "=f"(s0), "=f"(s1) : "l"(c));
    };
    auto fma2 = [](float& s0, float& s1, uint32_t v0, uint32_t v1, uint64_t scale2) {
      uint64_t a, b, c;
      asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "f"(s0), "f"(s1));
      asm("mov.b64 %0, {%1, %2};" : "=l"(b) : "r"(v0), "r"(v1));
      asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(c) : "l"(b), "l"(scale2), "l"(a));
      asm("mov.b64 {%0, %1}, %2;" : "=f"(s0), "=f"(s1) : "l"(c));
    };
    auto wait_tfull = [&](int r) -> bool {
      return mbar_wait_bounded(&tfull_bar[r], drains[r] & 1, abort_flag, p.err, kErrEpiTmemFullWait, peer_abort);
    };
    // "TMEM region drained": arrive on the leader's barrier (the peer does so remotely).
    auto arrive_tempty = [&](int r) {
      if (!PAIR || leader) mbar_arrive(&tempty_bar[r]);
      else mbar_arrive_cluster_relaxed(mapa_u32(smem_u32(&tempty_bar[r]), 0));
    };
    for (int unit = first_tile; unit < num_units && ok; unit += tile_stride) {
      int tm, tn, kb0, kb1, slice;
      unit_rc(unit, tm, tn, kb0, kb1, slice);
      const int unit_chunks = (kb1 - kb0 + chunk - 1) / chunk;
      for (int c = 0; c < unit_chunks && ok; ++c, ++gchunk) {
        const int r_main = (NTERMS == 1 || reord_fast) ? (int)(gchunk & 1) : 0;
        const bool with_x = (NTERMS == 3) && (p.order == 1);
        constexpr bool reordered = (NTERMS == 3) && REORD;
        {
          SGC_T0();
          if (!wait_tfull(r_main)) { ok = false; break; }
          SGC_TADD(6, blockIdx.x == 0 && threadIdx.x == 0);
        }
        SGC_T0();
        tc_fence_after_sync();
        const uint32_t t_main = tmem_base + lane_addr + r_main * kBN + half * 128;
        const uint32_t t_x = tmem_base + lane_addr + kBN + half * 128;
        if (reordered && !reord_fast) {
          // Reordered elementwise (Sec. 4.5, last paragraph): the block's corrections, already
          // summed at their own scale, are scaled and added to the block's hi*hi product, and the
          // accumulator takes the block once:  acc = acc + (P_x / s_f + P_hh).  (The fast form
          // gets the block's value ready-made from one region and takes the plain path below.)
          if (!wait_tfull(1)) { ok = false; break; }
          tc_fence_after_sync();
          constexpr int GR = 16;
#pragma unroll
          for (int g = 0; g < 128 / GR; ++g) {
            uint32_t vh[GR], vx[GR];
            tmem_ld_cols(t_main + g * GR, vh);
            tmem_ld_cols(t_x + g * GR, vx);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < GR; ++j) {
              const float block =
                  __fmaf_rn(__uint_as_float(vx[j]), p.inv_scale, __uint_as_float(vh[j]));
              S[g * GR + j] = (c == 0) ? block : __fadd_rn(S[g * GR + j], block);
            }
          }
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            arrive_tempty(r_main);
            arrive_tempty(1);
          }
          drains[r_main]++;
          drains[1]++;
        } else {
#pragma unroll
        for (int g = 0; g < 128 / GW; ++g) {
          uint32_t v[GW];
          tmem_ld_cols(t_main + g * GW, v);
          tmem_ld_wait();
          if (c == 0) {
#pragma unroll
            for (int j = 0; j < GW; ++j) S[g * GW + j] = __uint_as_float(v[j]);
          } else {
            if constexpr (kPackedDrain) {
#pragma unroll
              for (int j = 0; j < GW; j += 2) add2(S[g * GW + j], S[g * GW + j + 1], v[j], v[j + 1]);
            } else {
#pragma unroll
              for (int j = 0; j < GW; ++j) S[g * GW + j] = __fadd_rn(S[g * GW + j], __uint_as_float(v[j]));
            }
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) arrive_tempty(r_main);
        drains[r_main]++;
        if (with_x) {
          // Elementwise: fold this k-block's corrections into the same accumulator, after its
          // hi*hi sum (the bracketing of Eq. elementwise).  The hi*hi region has already gone back
          // to the MMA thread, whose next hi*hi products run while this region is read.
          if (!wait_tfull(1)) { ok = false; break; }
          tc_fence_after_sync();
#pragma unroll
          for (int g = 0; g < 128 / GW; ++g) {
            uint32_t v[GW];
            tmem_ld_cols(t_x + g * GW, v);
            tmem_ld_wait();
            // acc + 2^-s P_x as one FMA: the product with a power of two is exact, so the result is
            // that of the separate multiplication and addition (one rounding either way)
            if constexpr (kPackedDrain) {
#pragma unroll
              for (int j = 0; j < GW; j += 2) fma2(S[g * GW + j], S[g * GW + j + 1], v[j], v[j + 1], inv_scale2);
            } else {
#pragma unroll
              for (int j = 0; j < GW; ++j)
                S[g * GW + j] = __fmaf_rn(__uint_as_float(v[j]), p.inv_scale, S[g * GW + j]);
            }
          }
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) arrive_tempty(1);
          drains[1]++;
        }
        }  // not reordered
        SGC_TADD(7, blockIdx.x == 0 && threadIdx.x == 0);
      }
      if (!ok) break;
      SGC_T0();
      const int row = tm * kBM + quarter * 32 + lane;
      const int col_base = tn * kBN + half * 128;
      // Store the 128 values of this thread's row segment to a row-major matrix.  Vector path:
      // storing straight from registers would write 16 bytes per row per instruction; instead
      // 32 x 32 blocks go through a per-warp staging buffer (16-byte chunks XOR-swizzled by row:
      // conflict-free both ways) and leave as 128-byte row segments, four rows per store.
      auto store_tile = [&](float* base, long long ld, bool vec, int accumulate) {
        if (vec) {
          const uint32_t stg = smem_u32(store_staging + warp * 4096);
          const int row0 = tm * kBM + quarter * 32;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(
                               stg + lane * 128 + ((q ^ (lane & 7)) << 4)),
                           "f"(S[g * 32 + 4 * q]), "f"(S[g * 32 + 4 * q + 1]), "f"(S[g * 32 + 4 * q + 2]),
                           "f"(S[g * 32 + 4 * q + 3])
                           : "memory");
            __syncwarp();
            const int q = lane & 7;
            const int col = col_base + g * 32 + q * 4;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int r = i * 4 + (lane >> 3);
              float4 v;
              asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                           : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                           : "r"(stg + r * 128 + ((q ^ (r & 7)) << 4))
                           : "memory");
              const int grow = row0 + r;
              if (grow < p.M && col < p.N) {
                float* dst = base + (long long)grow * ld + col;
                if (col + 4 <= p.N) {
                  if (accumulate) {
                    const float4 old = *reinterpret_cast<const float4*>(dst);
                    v.x = __fadd_rn(old.x, v.x); v.y = __fadd_rn(old.y, v.y);
                    v.z = __fadd_rn(old.z, v.z); v.w = __fadd_rn(old.w, v.w);
                  }
                  *reinterpret_cast<float4*>(dst) = v;
                } else {
                  const float e[4] = {v.x, v.y, v.z, v.w};
                  for (int j = 0; j < 4 && col + j < p.N; ++j)
                    dst[j] = accumulate ? __fadd_rn(dst[j], e[j]) : e[j];
                }
              }
            }
            __syncwarp();
          }
        } else {
#pragma unroll
          for (int g = 0; g < 8; ++g)
            store16(base, ld, p.M, p.N, row, col_base + g * 16, &S[g * 16], false, accumulate);
        }
      };
      const bool split_out = (NTERMS == 3) && !FUSED && (p.Phh != nullptr);
      if (split_out) store_tile(p.Phh + (long long)slice * p.pstride, p.ldp, true, 0);
      if (NTERMS == 3 && p.order == 0) {
        // Termwise: the correction stream meets the dominant stream once: here, or (split-K) in
        // the reduction kernel, which gets the raw correction sums of this slice.
        if (!wait_tfull(1)) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        const uint32_t t_x = tmem_base + lane_addr + kBN + half * 128;
#pragma unroll
        for (int g = 0; g < 128 / GW; ++g) {
          uint32_t v[GW];
          tmem_ld_cols(t_x + g * GW, v);
          tmem_ld_wait();
          if (split_out) {
#pragma unroll
            for (int j = 0; j < GW; ++j) S[g * GW + j] = __uint_as_float(v[j]);
          } else {
#pragma unroll
            for (int j = 0; j < GW; ++j)
              S[g * GW + j] = __fmaf_rn(__uint_as_float(v[j]), p.inv_scale, S[g * GW + j]);
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) arrive_tempty(1);
        drains[1]++;
        if (split_out) store_tile(p.Px + (long long)slice * p.pstride, p.ldp, true, 0);
      }
      if (!split_out) store_tile(p.D, p.ldd, vec_ok, (NTERMS == 1) ? p.accumulate : 0);
      SGC_TADD(8, blockIdx.x == 0 && threadIdx.x == 0);
    }
  } else if (warp == kMmaWarp) {
    if (FUSED) setmaxnreg_dec<SGC_FUSED_OTHER_REGS>();
    else setmaxnreg_dec<56>();
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && leader) {
      constexpr uint32_t idesc =
          umma_idesc_f16(PAIR ? 2 * kBM : kBM, kBN, /*A MN-major*/ false, /*B MN-major*/ true);
      auto mma = [&](uint32_t d, uint64_t da, uint64_t db, uint32_t acc) {
        if (PAIR) umma_f16_ss_pair(d, da, db, idesc, acc);
        else umma_f16_ss(d, da, db, idesc, acc);
      };
      auto commit_both = [&](uint64_t* bar) {            // barrier at this offset in every CTA
        if (PAIR) umma_commit_pair_both(bar);
        else umma_commit(bar);
      };
      auto wait = [&](uint64_t* bar, uint32_t parity, unsigned int code) {
        return PAIR ? mbar_wait_bounded_cluster(bar, parity, abort_flag, p.err, code, peer_abort)
                    : mbar_wait_bounded(bar, parity, abort_flag, p.err, code);
      };
      constexpr uint64_t a_swz = (Cfg::A_ROW_BYTES == 128) ? kSwizzle128
                                 : (Cfg::A_ROW_BYTES == 64) ? kSwizzle64 : kSwizzle32;
      constexpr uint64_t b_swz = FUSED ? kSwizzle64 : kSwizzle128;
      constexpr uint32_t a_sbo = Cfg::A_SBO, b_lbo = Cfg::B_LBO, b_sbo = Cfg::B_SBO;
      // The issuing thread is a single lane: every instruction it spends on a descriptor delays
      // the next MMA.  Only the start-address field (low word, in units of 16 bytes) changes from
      // one MMA to the next, so the constant fields are folded at compile time and a descriptor
      // costs one 32-bit add.
      constexpr uint32_t a_desc_hi =
          ((a_sbo >> 4) & 0x3FFFu) | (1u << 14) | ((uint32_t)a_swz << 29);
      constexpr uint32_t b_desc_hi =
          ((b_sbo >> 4) & 0x3FFFu) | (1u << 14) | ((uint32_t)b_swz << 29);
      constexpr uint32_t a_desc_lo0 = ((16u >> 4) & 0x3FFFu) << 16;
      constexpr uint32_t b_desc_lo0 = ((b_lbo >> 4) & 0x3FFFu) << 16;
      auto desc = [](uint32_t lo, uint32_t hi) -> uint64_t {
        uint64_t d;
        asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
        return d;
      };
      uint32_t it = 0;
      uint32_t fills[2] = {0, 0};     // how many times each TMEM region has been handed over
      uint32_t gchunk = 0;            // running k-block counter (NTERMS == 1 region choice)
      bool ok = true;
      for (int unit = first_tile; unit < num_units && ok; unit += tile_stride) {
        int tm_, tn_, kb0, kb1, slice_;
        unit_rc(unit, tm_, tn_, kb0, kb1, slice_);
        const int unit_chunks = (kb1 - kb0 + chunk - 1) / chunk;
        for (int c = 0; c < unit_chunks && ok; ++c, ++gchunk) {
          const int kb_begin = kb0 + c * chunk;
          const int kb_end = min(kb1, kb_begin + chunk);
          // Region(s) this k-block accumulates into, and which of them start from zero here.
          const int r_main = (NTERMS == 1) ? (int)(gchunk & 1) : 0;
          const bool x_fresh = (NTERMS == 3) && (p.order != 0 || c == 0);
          bool main_ready = false, x_ready = !x_fresh;
          const uint32_t d_x = tmem_base + kBN;
          const uint32_t d_main = tmem_base + r_main * kBN;
          // Wait for stage `i` (running stage counter) to be filled; returns its base address.
          auto stage_ready = [&](uint32_t i, uint32_t& st) -> bool {
            const int s = i % STAGES;
            SGC_T0();
            if (!wait(&full_bar[s], (i / STAGES) & 1, kErrMmaFullWait)) return false;
            SGC_TADD(4, blockIdx.x == 0);
            tc_fence_after_sync();
            st = smem_u32(smem + s * Cfg::STAGE_BYTES);
            return true;
          };
          // lo_A hi_B and hi_A lo_B of one stage into the correction accumulator.
          auto issue_cross = [&](uint32_t st, bool first_kb) -> bool {
            if (!x_ready) {
              if (!wait(&tempty_bar[1], (fills[1] & 1) ^ 1, kErrMmaTmemEmptyWait)) return false;
              tc_fence_after_sync();
              x_ready = true;
            }
            const uint32_t a_hi = a_desc_lo0 + (st >> 4), a_lo = a_hi + (Cfg::A_LO_OFF >> 4);
            const uint32_t b_hi = b_desc_lo0 + ((st + Cfg::B_OFF) >> 4);
            const uint32_t b_lo = b_hi + (Cfg::B_LO_OFF >> 4);
            // Order inside the correction chain: per 32 k-steps, lo*hi of both k16 steps, then
            // hi*lo of both.  Fixed whatever the stage depth, so that every variant of the
            // kernel rounds the chain identically.
            constexpr int G = (BK < 32 ? BK : 32) / 16;
#pragma unroll
            for (int j0 = 0; j0 < BK / 16; j0 += G) {
#pragma unroll
              for (int j = j0; j < j0 + G; ++j) {
                const uint64_t da = desc(a_lo + 2 * j, a_desc_hi);
                const uint64_t db = desc(b_hi + 128 * j, b_desc_hi);
                mma(d_x, da, db, (x_fresh && first_kb && j == 0) ? 0u : 1u);
              }
#pragma unroll
              for (int j = j0; j < j0 + G; ++j) {
                const uint64_t da = desc(a_hi + 2 * j, a_desc_hi);
                const uint64_t db = desc(b_lo + 128 * j, b_desc_hi);
                mma(d_x, da, db, 1u);
              }
            }
            return true;
          };
          // hi_A hi_B (or the single product) of one stage into the main region; frees the stage.
          auto issue_main = [&](uint32_t st, uint32_t i, bool first_kb, bool release = true) -> bool {
            if (!main_ready) {
              SGC_T0();
              if (!wait(&tempty_bar[r_main], (fills[r_main] & 1) ^ 1, kErrMmaTmemEmptyWait)) return false;
              SGC_TADD(5, blockIdx.x == 0);
              tc_fence_after_sync();
              main_ready = true;
            }
            const uint32_t a_hi = a_desc_lo0 + (st >> 4);
            const uint32_t b_hi = b_desc_lo0 + ((st + Cfg::B_OFF) >> 4);
#pragma unroll
            for (int j = 0; j < BK / 16; ++j) {
              const uint64_t da = desc(a_hi + 2 * j, a_desc_hi);
              const uint64_t db = desc(b_hi + 128 * j, b_desc_hi);
              mma(d_main, da, db, (first_kb && j == 0) ? 0u : 1u);
            }
            // the stage may be refilled once these MMAs retire
            if (release) commit_both(&empty_bar[i % STAGES]);
            return true;
          };
          if constexpr (REORD && NTERMS == 3) {
            if (reord_fast) {
              // One region per k-block, alternating: all correction products of the block first
              // (from zero), then its hi*hi products, the first of which takes the accumulator
              // scaled by 2^-s:  D = P_hh + 2^-s P_x.  The order inside each chain is the usual one.
              const int r = (int)(gchunk & 1);
              const uint32_t d = tmem_base + r * kBN;
              if (!wait(&tempty_bar[r], (fills[r] & 1) ^ 1, kErrMmaTmemEmptyWait)) { ok = false; break; }
              tc_fence_after_sync();
              const int n = kb_end - kb_begin;
              constexpr int kMaxN = STAGES / 2 > 0 ? STAGES / 2 : 1;
              uint32_t stv[kMaxN];
#pragma unroll
              for (int l = 0; l < kMaxN; ++l) {
                if (l < n && ok) {
                  ok = stage_ready(it + l, stv[l]);
                  if (ok) {
                    const uint32_t a_hi = a_desc_lo0 + (stv[l] >> 4), a_lo = a_hi + (Cfg::A_LO_OFF >> 4);
                    const uint32_t b_hi = b_desc_lo0 + ((stv[l] + Cfg::B_OFF) >> 4);
                    const uint32_t b_lo = b_hi + (Cfg::B_LO_OFF >> 4);
                    constexpr int G = (BK < 32 ? BK : 32) / 16;
#pragma unroll
                    for (int j0 = 0; j0 < BK / 16; j0 += G) {
#pragma unroll
                      for (int j = j0; j < j0 + G; ++j)
                        mma(d, desc(a_lo + 2 * j, a_desc_hi), desc(b_hi + 128 * j, b_desc_hi),
                            (l == 0 && j == 0) ? 0u : 1u);
#pragma unroll
                      for (int j = j0; j < j0 + G; ++j)
                        mma(d, desc(a_hi + 2 * j, a_desc_hi), desc(b_lo + 128 * j, b_desc_hi), 1u);
                    }
                  }
                }
              }
#pragma unroll
              for (int l = 0; l < kMaxN; ++l) {
                if (l < n && ok) {
                  const uint32_t a_hi = a_desc_lo0 + (stv[l] >> 4);
                  const uint32_t b_hi = b_desc_lo0 + ((stv[l] + Cfg::B_OFF) >> 4);
#pragma unroll
                  for (int j = 0; j < BK / 16; ++j) {
                    const uint64_t da = desc(a_hi + 2 * j, a_desc_hi);
                    const uint64_t db = desc(b_hi + 128 * j, b_desc_hi);
                    if (l == 0 && j == 0) umma_f16_ss_scale_d_rt(scale_exp, d, da, db, idesc, PAIR);
                    else mma(d, da, db, 1u);
                  }
                  commit_both(&empty_bar[(it + l) % STAGES]);
                }
              }
              if (!ok) break;
              commit_both(&tfull_bar[r]);
              fills[r]++;
              it += n;
              continue;
            }
          }
          int kb = kb_begin;
          // stages whose correction products go first (64 k-steps' worth)
#ifdef SGC_KLOOK
          constexpr int kLook = SGC_KLOOK;
#else
          constexpr int kLook = (2 * 32 + BK - 1) / BK;
#endif
          if (NTERMS == 3 && p.order == 0 && kb + kLook <= kb_end) {
            // Start of a termwise k-block: the correction products of the first kLook stages go
            // first.  They do not touch region 0, so the accumulate warps get 8 kLook MMAs' worth
            // of time to add the previous k-block into their sums before hi*hi needs the region.
            uint32_t st[kLook];
#pragma unroll
            for (int l = 0; l < kLook; ++l)
              ok = ok && stage_ready(it + l, st[l]) && issue_cross(st[l], l == 0);
#pragma unroll
            for (int l = 0; l < kLook; ++l) ok = ok && issue_main(st[l], it + l, l == 0);
            kb += kLook;
            it += kLook;
          }
          bool handed_over = false;
          for (; kb < kb_end && ok; ++kb, ++it) {
            uint32_t st;
            const bool first_kb = (kb == kb_begin);
#ifndef SGC_NO_TAIL_SWAP
            if (NTERMS == 3 && p.order == 0 && kb == kb_end - 1 && !first_kb) {
              // Last stage of a termwise k-block of two or more stages: hi*hi first, so that
              // region 0 goes to the accumulate warps eight MMAs earlier; this stage's correction
              // products and those of the next block's first stage then run while it is drained.
              // The order inside each chain is unchanged.
              ok = stage_ready(it, st) && issue_main(st, it, false, /*release*/ false);
              if (!ok) break;
              commit_both(&tfull_bar[r_main]);
              fills[r_main]++;
              handed_over = true;
              ok = issue_cross(st, false);
              commit_both(&empty_bar[it % STAGES]);
              continue;
            }
#endif
            if (NTERMS == 3 && p.order != 0) {
              // Elementwise: both regions go to the accumulate warps after every k-block.  hi*hi
              // first and handed over at once: it is drained while the correction products run,
              // and the corrections are drained while the next block's hi*hi products run.
              ok = stage_ready(it, st) && issue_main(st, it, first_kb, /*release*/ false);
              if (!ok) break;
              if (kb == kb_end - 1) {
                commit_both(&tfull_bar[r_main]);
                fills[r_main]++;
                handed_over = true;
              }
              ok = issue_cross(st, first_kb);
              commit_both(&empty_bar[it % STAGES]);
              continue;
            }
            ok = stage_ready(it, st) && (NTERMS != 3 || issue_cross(st, first_kb)) &&
                 issue_main(st, it, first_kb);
          }
          if (!ok) break;
          // Hand the finished region(s) to the accumulate warps.
          if (!handed_over) {
            commit_both(&tfull_bar[r_main]);
            fills[r_main]++;
          }
          if (NTERMS == 3 && (p.order != 0 || c == unit_chunks - 1)) {
            commit_both(&tfull_bar[1]);
            fills[1]++;
          }
        }
      }
      // Bounded drain: all issued MMAs must have retired before TMEM is freed.
      if (PAIR) umma_commit_pair_local(drain_bar);
      else umma_commit(drain_bar);
      mbar_wait_bounded(drain_bar, 0, nullptr, p.err, kErrDrainWait);
    }
  } else if (warp == kProducerWarp) {
    if (FUSED) setmaxnreg_dec<SGC_FUSED_OTHER_REGS>();
    else setmaxnreg_dec<56>();
    // ------------------------------------------------------------------ TMA producer
    // not FUSED: FP16 operand tiles, read by the MMA thread.  FUSED: FP32 tiles of A and B, which
    // the converter warps turn into FP16 words in place (this CTA's own rows of A and its own
    // columns of B; the "filled" barrier is local to the CTA also in a pair, the "free" barrier
    // is the MMA thread's commit, which arrives in both CTAs).
    if (lane == 0) {
      constexpr int RING = STAGES;
      uint64_t* const ring_full = FUSED ? full32_bar : full_bar;
      uint64_t* const ring_empty = empty_bar;
      uint32_t it = 0;
      bool ok = true;
      auto load = [&](void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
        if (PAIR && !FUSED) tma_load_2d_pair(dst, map, x, y, bar);   // bytes counted on the leader's barrier
        else tma_load_2d(dst, map, x, y, bar);
      };
      for (int unit = first_tile; unit < num_units && ok; unit += tile_stride) {
        int tm, tn, kb0, kb1, slice;
        unit_rc(unit, tm, tn, kb0, kb1, slice);
        const int n0 = tn * kBN + (PAIR ? (int)cta_rank * Cfg::BN_CTA : 0);   // this CTA's B columns
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % RING;
          const uint32_t ph = (it / RING) & 1;
          {
            SGC_T0();
            if (!mbar_wait_bounded(&ring_empty[s], ph ^ 1, abort_flag, p.err, kErrProducerEmptyWait, peer_abort)) {
              ok = false;
              break;
            }
            SGC_TADD(14, blockIdx.x == 0);
          }
          const int k0 = kb * BK;
          if constexpr (FUSED) {
            // A: one box {32 k (128 bytes), 128 rows}; B: boxes {32 columns (128 bytes), 32 k-rows}.
            // Rows and columns outside the matrices arrive as zeros, and split(0) = (0, 0).
            uint8_t* st = smem + s * Cfg::STAGE_BYTES;
            mbar_arrive_expect_tx(&ring_full[s], Cfg::STAGE_BYTES);
            load(st, &tmA0, k0, tm * kBM, &ring_full[s]);
#pragma unroll
            for (int a = 0; a < Cfg::BN_CTA / 32; ++a)
              load(st + Cfg::A32_TILE + a * (BK * 128), &tmB0, n0 + a * 32, k0, &ring_full[s]);
          } else {
            uint8_t* st = smem + s * Cfg::STAGE_BYTES;
            // The leader announces the bytes of both CTAs' copies; the peer's copies may land first
            // (the phase cannot complete before the leader's arrival).
            if (leader) mbar_arrive_expect_tx(&ring_full[s], Cfg::STAGE_BYTES * (PAIR ? 2 : 1));
            // A tiles: box {BK (k), 128 rows}.  B tiles: boxes {64 (n), BK (k rows)}.
            load(st, &tmA0, k0, tm * kBM, &ring_full[s]);
            uint8_t* bdst = st + Cfg::A_TILE;
            if (NTERMS == 3) {
              load(st + Cfg::A_TILE, &tmA1, k0, tm * kBM, &ring_full[s]);
              bdst = st + 2 * Cfg::A_TILE;
            }
#pragma unroll
            for (int a = 0; a < Cfg::BN_CTA / 64; ++a)
              load(bdst + a * (BK * 128), &tmB0, n0 + a * 64, k0, &ring_full[s]);
            if (NTERMS == 3) {
#pragma unroll
              for (int a = 0; a < Cfg::BN_CTA / 64; ++a)
                load(bdst + Cfg::B_TILE + a * (BK * 128), &tmB1, n0 + a * 64, k0, &ring_full[s]);
            }
          }
        }
      }
      // No bulk copy may be in flight into this CTA's shared memory when it exits.  Normal end:
      // wait until the consumer has released every stage that was filled.  After an abort the
      // consumers no longer release anything: wait (bounded) for the copies themselves, on the
      // barriers that count their bytes where this CTA can see them, else for a fixed time that
      // is long against any copy's latency.
      if (ok) {
        for (int d = 0; d < RING && d < (int)it; ++d, ++it) {
          const int s = it % RING;
          const uint32_t ph = (it / RING) & 1;
          if (!mbar_wait_bounded(&ring_empty[s], ph ^ 1, abort_flag, p.err, kErrDrainWait, peer_abort)) {
            ok = false;
            break;
          }
        }
      }
      if (!ok) {
        const uint32_t issued = it < (uint32_t)RING ? it : (uint32_t)RING;
        if (FUSED || !PAIR || leader) {
          for (uint32_t d = 1; d <= issued; ++d) {
            const uint32_t j = it - d;
            mbar_wait_clocks(&ring_full[j % RING], (j / RING) & 1, kAbortDrainClocks);
          }
        } else {
          const long long t0 = clock64();
          while (clock64() - t0 < kAbortDrainClocks) {}
        }
      }
    }
  } else if (FUSED && warp >= kNumEpiWarps && warp < kNumEpiWarps + kNumConvWarps) {
    setmaxnreg_dec<SGC_FUSED_OTHER_REGS>();
    // ------------------------------------------------------------------ converter warps
    // A stage is STAGE_BYTES / 1024 regions of 1 KB: 8 rows of 128 bytes (32 FP32 elements: 8 rows
    // of A over 32 k, or 8 k-rows of B over 32 columns), 16-byte chunk j of row r at position
    // j ^ r (TMA's 128-byte swizzle).  A warp converts a region in place: lane l takes the item
    // (8 elements) q = l % 4 of row r = l / 4, reads its two chunks, and after the whole warp has
    // read (__syncwarp) writes the hi chunk to r * 64 + ((q ^ (r / 2)) << 4) (rows of 64 bytes,
    // 64-byte swizzle: the K-major atom of A, the MN-major atom of B) and the lo chunk 512 bytes
    // further.  A quarter warp reads 8 distinct chunk positions (rows of both parities) and
    // writes 128 contiguous bytes: no bank conflicts.  Warp w takes regions w, w + NW, ...; its
    // offsets inside a region are per-thread constants and the rest of each address is an
    // immediate.
    constexpr int NW = kNumConvWarps;
    constexpr int kRegions = Cfg::STAGE_BYTES / 1024;             // 32 (pair) or 48
    static_assert(kRegions % NW == 0, "regions per converter warp");
    constexpr int R = kRegions / NW;
    constexpr int kBatch = SGC_CONV_BATCH;                        // regions loaded before converting
    static_assert(R % kBatch == 0, "batches");
    const int cw = warp - kNumEpiWarps;
    const int ar = lane >> 2, aq = lane & 3;
    const uint32_t src_c = (uint32_t)(cw * 1024 + ar * 128 + (((2 * aq) ^ ar) << 4));
    const uint32_t dst_c = (uint32_t)(cw * 1024 + ar * 64 + ((aq ^ ((ar >> 1) & 3)) << 4));
    const int total_stages = (first_tile < num_tiles)
        ? ((num_tiles - first_tile + tile_stride - 1) / tile_stride) * num_kb : 0;
    ConvScale cs;
    cs.scale = p.scale;
    cs.fast = p.scale <= 32768.f;
    asm("mov.b64 %0, {%1, %1};" : "=l"(cs.scale2) : "f"(p.scale));
    cs.neg_scale_h = __half_as_ushort(__float2half_rn(cs.fast ? -p.scale : -1.f));
    const uint32_t ring = smem_u32(smem);
    const bool timed = (blockIdx.x == 0 && threadIdx.x == kNumEpiWarps * 32);
    const bool timed1 = (blockIdx.x == 1 && threadIdx.x == (kNumEpiWarps + kNumConvWarps - 1) * 32);
    (void)timed; (void)timed1;
    auto convert_stage = [&](uint32_t st, auto fast_tag) {
      constexpr bool FAST = decltype(fast_tag)::value;
      const uint32_t s0 = st + src_c, s1 = s0 ^ 16u, d = st + dst_c;
#pragma unroll
      for (int b = 0; b < R; b += kBatch) {
        ConvItem x[kBatch];
#pragma unroll
        for (int r = 0; r < kBatch; ++r) load_item(x[r], s0 + (b + r) * NW * 1024, s1 + (b + r) * NW * 1024);
        __syncwarp();       // every lane has read its part of these regions: they may be overwritten
#pragma unroll
        for (int r = 0; r < kBatch; ++r) convert_store<FAST>(x[r], d + (b + r) * NW * 1024, 512, cs);
      }
    };
    for (int it = 0; it < total_stages; ++it) {
      const int s = it % STAGES;
      const uint32_t ph = (it / STAGES) & 1;
      {
        SGC_T0();
        if (!mbar_wait_bounded(&full32_bar[s], ph, abort_flag, p.err, kErrConvFullWait, peer_abort)) break;
        SGC_TADD(11, timed);
      }
      SGC_T0();
      const uint32_t st = ring + s * Cfg::STAGE_BYTES;
      if (cs.fast) convert_stage(st, std::true_type{});
      else convert_stage(st, std::false_type{});
      SGC_TADD(1, timed);
      // Hand the stage to the relay thread, which makes it visible to the tensor core.
      {
        SGC_T0();
        __syncwarp();
        if (lane == 0) mbar_arrive(&conv_bar[s]);
        SGC_TADD(2, timed);
        SGC_TADD(15, timed1);
      }
#ifdef SGC_ROLE_TIMING
      if (timed) atomicAdd(&g_role_timing[3], 1ull);
#endif
    }
  } else if (FUSED) {
    setmaxnreg_dec<SGC_FUSED_OTHER_REGS>();
    // ------------------------------------------------------------------ relay threads
    // The converters' stores go through the generic proxy and the tensor core reads through the
    // async proxy, so a proxy fence has to lie between the two.  Inside a cluster that fence
    // costs several hundred clocks (and the peer's arrival on the leader's barrier as much
    // again), which the converter warps cannot afford once per stage.  The fence may be executed
    // by any thread on the path from the stores to the MMA: the converter warps arrive on a
    // local barrier, one lane of each of the two spare warps takes every other stage, acquires
    // that barrier, fences and tells the MMA thread (in a pair: the leader's) that this CTA's
    // part of the stage is ready.
    const int rw = warp - (kProducerWarp + 1);         // 0 or 1
    if (lane == 0 && rw >= 0 && rw < 2) {
      const int total_stages = (first_tile < num_tiles)
          ? ((num_tiles - first_tile + tile_stride - 1) / tile_stride) * num_kb : 0;
      for (int it = rw; it < total_stages; it += 2) {
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        if (!mbar_wait_bounded(&conv_bar[s], ph, abort_flag, p.err, kErrRelayWait, peer_abort)) break;
        SGC_T0();
        fence_proxy_async_smem();
        if (!PAIR || leader) mbar_arrive(&full_bar[s]);
        // remote arrival with the default (CTA-scope) release: what it publishes was made visible
        // to the async proxy by the fence above, before the arrive was issued
        else mbar_arrive_remote_cta(mapa_u32(smem_u32(&full_bar[s]), 0));
        SGC_TADD(12, blockIdx.x == 1 && rw == 0);
        SGC_TADD(13, blockIdx.x == 0 && rw == 0);
      }
    }
  } else {
    setmaxnreg_dec<56>();      // idle warps of the last warpgroup
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before_sync();
  __syncthreads();
  if (kclock_on) {
    unsigned long long ns1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns1));
    p.kclock[0] = (unsigned long long)(clock64() - kclock_clk0);
    p.kclock[1] = ns1 - kclock_ns0;
  }
#ifdef SGC_ROLE_TIMING
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    unsigned long long ns1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns1));
    atomicAdd(&g_role_timing[9], (unsigned long long)(clock64() - sgc_k_clk0));
    atomicAdd(&g_role_timing[10], ns1 - sgc_k_ns0);
  }
#endif
  if (PAIR) cluster_sync_all();      // neither CTA exits (or frees TMEM) while its peer still runs
  if (warp == kMmaWarp) {
    __syncwarp();
    tc_fence_after_sync();
    if (PAIR) tmem_dealloc_pair(tmem_base, kTmemCols);
    else tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Diagnostic kernel (one CTA): thread 0 waits, with the bounded wait that every role of the
// kernels above uses, on an mbarrier that nothing ever signals, so the wait runs into its clock
// limit, publishes kErrProbeWait in the error word and raises the CTA's abort flag; the second
// warp waits on the same barrier with the full limit and must leave as soon as the flag is up.
// Lets a test walk the path device wait -> error word -> host status without making any real
// pipeline fail.  `limit` is a few thousand clocks.
__global__ void wait_timeout_probe_kernel(unsigned int* err, long long limit) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0u;
    fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait_bounded(&bar, 0, &abort_flag, err, kErrProbeWait, 0u, limit);
  if (threadIdx.x == 32) mbar_wait_bounded(&bar, 0, &abort_flag, err, kErrProbeWait + 1, 0u, kWaitLimitClocks);
}

}  // namespace sgc
