// Weight-only variant of step 3 (Appendix "Weight-only Quantization", Table "wquant": W4A16 / W3A16):
//   Y[t, c] = fp16((sum_k Z16[t, k] * code[c, k]) * s_w[c])
// with the rotated activations Z16 in fp16, the pre-rotated weights as b-bit two's-complement codes
// (b = 4 or 3, one nibble each) and fp32 accumulation.
//
// Tensor-core kernel (sm_100a): the activation tile is the A operand exactly as TMA delivers it (128
// tokens x 64 channels, 128-byte swizzled rows); the packed weights arrive by TMA into a staging
// ring and eight warps widen them to fp16 in shared memory, written in the swizzled K-major layout
// the MMA descriptors expect; one thread issues tcgen05.mma kind::f16 into an fp32 accumulator in
// tensor memory; four warps read it back, multiply by the channel step and store fp16 while the next
// tile's main loop runs into the other accumulator buffer.
//
// Widening a nibble to fp16 without a conversion: for a two's-complement nibble u of the code c,
// u ^ 8 = c + 8, and the fp16 bit pattern 0x6400 | v is the number 1024 + v (0 <= v < 1024).  So
// (u ^ 0x6408) read as fp16 is 1032 + c, and one exact fp16 subtraction of 1032 leaves c.  The
// weight-only storage order puts channels (2s, 2s+1) of every eight at nibble positions (s, s+4) of a
// 32-bit word, so that (word >> 4s) & 0x000F000F is one such pair in the two halves of a register:
// a shift, one three-input logic operation and one half2 subtraction per two weights (half of the pairs
// need no shift: see widen_high).
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

constexpr int WO_BM = 128;              // tokens per tile (UMMA M)
constexpr int WO_UNPACK_WARPS = 8;
constexpr int WO_EPI_WARPS = 4;
constexpr int WO_THREADS = (2 + WO_UNPACK_WARPS + WO_EPI_WARPS) * 32;

enum WoSite : uint32_t { WO_A_EMPTY = 80, WO_A_FULL, WO_ST_EMPTY, WO_ST_FULL, WO_B_EMPTY, WO_B_FULL, WO_TMEM_FULL, WO_TMEM_EMPTY };

// Shared-memory plan: SA activation k-blocks (64 channels, 16 KB), SB widened weight k-blocks
// (BN rows x 128 bytes), SS staging blocks of packed weights (BN rows x 128 bytes = 256 channels).
template <int BN, int SA, int SS, int SB>
struct WoSmem {
  static constexpr int A_TILE = WO_BM * 128;
  static constexpr int B_OP = BN * 128;
  static constexpr int B_ST = BN * 128;
  static constexpr int OFF_A = 0;
  static constexpr int OFF_B_OP = OFF_A + SA * A_TILE;
  static constexpr int OFF_B_ST = OFF_B_OP + SB * B_OP;
  static constexpr int OFF_BAR = OFF_B_ST + SS * B_ST;
  static constexpr int NUM_BARS = 2 * SA + 2 * SS + 2 * SB + 4;
  static constexpr int OFF_TMEM = OFF_BAR + NUM_BARS * 8;
  static constexpr int TOTAL = OFF_TMEM + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;      // slack for the 1024-byte alignment
};

// Eight weights of one packed word as four half2 (channel pairs (0,1), (2,3), (4,5), (6,7)).  Nibble
// positions 0 and 4 sit in the low four mantissa bits of the two halves: (w & 0x000F000F) ^ 0x64086408 is
// (1032 + code) twice, minus 1032.  Positions 1 and 5 sit four bits higher: (w & 0x00F000F0) ^ 0x64806480
// is 1024 + 16 (code + 8), and one fused multiply-add, x / 16 - 72, leaves the code -- exact in fp16, and
// it spares the shift (the logic pipe is the busier one here).  One shift by 8 brings positions 2, 3, 6, 7
// to where 0, 1, 4, 5 were.
__device__ __forceinline__ uint32_t widen_low(uint32_t w) {
  const uint32_t x = (w & 0x000F000Fu) ^ 0x64086408u;
  const __half2 v = __hsub2(*reinterpret_cast<const __half2*>(&x), __half2half2(__ushort_as_half(0x6408)));
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t widen_high(uint32_t w) {
  const uint32_t x = (w & 0x00F000F0u) ^ 0x64806480u;
  const __half2 v = __hfma2(*reinterpret_cast<const __half2*>(&x), __half2half2(__ushort_as_half(0x2C00)),   // 1/16
                            __half2half2(__ushort_as_half(0xD480)));                                      // -72
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t widen_pair(uint32_t word, int s) {
  const uint32_t w = (s & 2) ? (word >> 8) : word;
  return (s & 1) ? widen_high(w) : widen_low(w);
}

__device__ __forceinline__ uint4 widen_word(uint32_t word) {
  const uint32_t w8 = word >> 8;
  return make_uint4(widen_low(word), widen_high(word), widen_low(w8), widen_high(w8));
}

// Widens k-block h (64 channels = 32 packed bytes) of BN staged rows into BN x 64 fp16.  Staging and
// operand rows are 128 bytes with the 128-byte swizzle (16-byte chunk c of row r sits at chunk
// c ^ (r & 7)).  Thread t takes source chunk j = (t >> 3) & 1 of rows 8 * (t >> 4) + (t & 7) + 128 i:
// a quarter-warp covers eight consecutive rows, so its eight 16-byte loads and each round of eight
// 16-byte stores fall into eight different bank groups.
template <int BN>
__device__ __forceinline__ void widen_tile(const unsigned char* __restrict__ st, unsigned char* __restrict__ op, int t,
                                           int h) {
  static_assert(BN % 128 == 0, "tile rows must be a multiple of 128");
  const int j = (t >> 3) & 1;
  const int r0 = ((t >> 4) << 3) + (t & 7);
  const int sw = r0 & 7;
#pragma unroll
  for (int i = 0; i < BN / 128; ++i) {
    const int r = r0 + i * 128;
    const uint4 w = *reinterpret_cast<const uint4*>(st + r * 128 + ((((h << 1) + j) ^ sw) << 4));
    unsigned char* dst = op + r * 128;
    *reinterpret_cast<uint4*>(dst + ((((j << 2) + 0) ^ sw) << 4)) = widen_word(w.x);
    *reinterpret_cast<uint4*>(dst + ((((j << 2) + 1) ^ sw) << 4)) = widen_word(w.y);
    *reinterpret_cast<uint4*>(dst + ((((j << 2) + 2) ^ sw) << 4)) = widen_word(w.z);
    *reinterpret_cast<uint4*>(dst + ((((j << 2) + 3) ^ sw) << 4)) = widen_word(w.w);
  }
}

// Persistent kernel: CTA b works on tiles b, b + gridDim.x, ...; tile index = m_tile * tiles_n + n_tile.
// Warp 0 lane 0: TMA producer.  Warp 1 lane 0: MMA issuer.  Warps 2..9: widen.  Warps 10..13: epilogue.
template <int BN, int SA, int SS, int SB>
__global__ void __launch_bounds__(WO_THREADS, 1)
wo_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_z, const __grid_constant__ CUtensorMap tmap_w,
                  const __half* __restrict__ sw, int M, int N, int K, __half* __restrict__ Y) {
  using L = WoSmem<BN, SA, SS, SB>;
  griddep_launch_dependents();          // a rotate kernel launched behind this one may set itself up
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* a_full = bars;
  uint64_t* a_empty = a_full + SA;
  uint64_t* st_full = a_empty + SA;
  uint64_t* st_empty = st_full + SS;
  uint64_t* b_full = st_empty + SS;
  uint64_t* b_empty = b_full + SB;
  uint64_t* tmem_full = b_empty + SB;         // [2]
  uint64_t* tmem_empty = tmem_full + 2;       // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_TMEM);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = K / 64;                  // fp16 k-blocks of 64 channels
  const int num_sb = (num_kb + 3) / 4;        // staging blocks of 256 channels (the last may be partly used)
  const int tiles_n = (N + BN - 1) / BN, tiles_m = (M + WO_BM - 1) / WO_BM;
  const int num_tiles = tiles_n * tiles_m;
  const uint32_t limit = wait_limit();

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmap_z);
    tma_prefetch_desc(&tmap_w);
    for (int s = 0; s < SA; ++s) {
      mbar_init(&a_full[s], 1);
      mbar_init(&a_empty[s], 1);
    }
    for (int s = 0; s < SS; ++s) {
      mbar_init(&st_full[s], 1);
      mbar_init(&st_empty[s], WO_UNPACK_WARPS);
    }
    for (int s = 0; s < SB; ++s) {
      mbar_init(&b_full[s], WO_UNPACK_WARPS);
      mbar_init(&b_empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&tmem_full[b], 1);
      mbar_init(&tmem_empty[b], WO_EPI_WARPS);
    }
    mbar_fence_init();
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  griddep_wait();                                     // Z16 may come from the kernel launched before this one

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (elect_one()) {
      uint32_t ait = 0, sit = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile / tiles_n) * WO_BM, n0 = (tile % tiles_n) * BN;
        for (int sb = 0; sb < num_sb && ok; ++sb, ++sit) {
          const int ss = sit % SS;
          ok = mbar_wait(&st_empty[ss], ((sit / SS) & 1) ^ 1, WO_ST_EMPTY, limit);
          if (!ok) break;
          mbar_arrive_expect_tx(&st_full[ss], L::B_ST);
          tma_load_2d(smem + L::OFF_B_ST + ss * L::B_ST, &tmap_w, &st_full[ss], sb * 128, n0);
          for (int h = 0; h < 4 && 4 * sb + h < num_kb; ++h, ++ait) {
            const int sa = ait % SA;
            ok = mbar_wait(&a_empty[sa], ((ait / SA) & 1) ^ 1, WO_A_EMPTY, limit);
            if (!ok) break;
            mbar_arrive_expect_tx(&a_full[sa], L::A_TILE);
            tma_load_2d(smem + L::OFF_A + sa * L::A_TILE, &tmap_z, &a_full[sa], (4 * sb + h) * 64, m0);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------------------
    if (elect_one()) {
      constexpr uint32_t idesc = umma_idesc(/*c=f32*/ 1, /*a=f16*/ 0, /*b=f16*/ 0, WO_BM, BN);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tcount) {
        const uint32_t b = tcount & 1;
        ok = mbar_wait(&tmem_empty[b], ((tcount >> 1) & 1) ^ 1, WO_TMEM_EMPTY, limit);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + b * BN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int sa = it % SA, sbo = it % SB;
          ok = mbar_wait(&a_full[sa], (it / SA) & 1, WO_A_FULL, limit) &&
               mbar_wait(&b_full[sbo], (it / SB) & 1, WO_B_FULL, limit);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t a_base = smem_u32(smem + L::OFF_A + sa * L::A_TILE);
          const uint32_t b_base = smem_u32(smem + L::OFF_B_OP + sbo * L::B_OP);
#pragma unroll
          for (int k = 0; k < 4; ++k) {                // 4 x (K = 16 fp16) per 128-byte row
            umma_f16(tmem_d, umma_desc_sw128(a_base + k * 32), umma_desc_sw128(b_base + k * 32), idesc,
                     (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&a_empty[sa]);                    // both operand stages are free when the MMAs retire
          umma_commit(&b_empty[sbo]);
        }
        umma_commit(&tmem_full[b]);                     // accumulator complete (or abandoned)
      }
    }
  } else if (warp < 2 + WO_UNPACK_WARPS) {
    // ------------------------------ widening warps ------------------------------------------
    const int t = threadIdx.x - 64;                    // 0 .. 255
    uint32_t it = 0, sit = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      for (int sb = 0; sb < num_sb && ok; ++sb, ++sit) {
        const int ss = sit % SS;
        ok = mbar_wait(&st_full[ss], (sit / SS) & 1, WO_ST_FULL, limit);
        if (!ok) break;
        for (int h = 0; h < 4 && 4 * sb + h < num_kb; ++h, ++it) {
          const int s = it % SB;
          ok = mbar_wait(&b_empty[s], ((it / SB) & 1) ^ 1, WO_B_EMPTY, limit);
          if (!ok) break;
          widen_tile<BN>(smem + L::OFF_B_ST + ss * L::B_ST, smem + L::OFF_B_OP + s * L::B_OP, t, h);
          fence_proxy_async_smem();                     // generic-proxy stores -> visible to the MMA
          __syncwarp();
          if (lane == 0) mbar_arrive(&b_full[s]);
        }
        if (!ok) break;
        __syncwarp();
        if (lane == 0) mbar_arrive(&st_empty[ss]);
      }
    }
  } else {
    // ------------------------------ epilogue warps ------------------------------------------
    const int quarter = warp & 3;                       // TMEM lanes this warp may read
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tcount) {
      const int m0 = (tile / tiles_n) * WO_BM, n0 = (tile % tiles_n) * BN;
      const uint32_t b = tcount & 1;
      ok = mbar_wait(&tmem_full[b], (tcount >> 1) & 1, WO_TMEM_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      const int row = m0 + quarter * 32 + lane;
      const uint32_t tmem_d = tmem_base + b * BN + (static_cast<uint32_t>(quarter * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem_d + c * 32, r);
        tmem_wait_ld();
        const int col0 = n0 + c * 32;
        if (row < M && col0 < N) {
          __half* yrow = Y + static_cast<size_t>(row) * N + col0;
#pragma unroll
          for (int g = 0; g < 4; ++g) {                 // groups of 8 columns (N % 8 == 0)
            if (col0 + g * 8 < N) {
              const uint4 swraw = __ldg(reinterpret_cast<const uint4*>(sw + col0 + g * 8));
              const __half2* swh = reinterpret_cast<const __half2*>(&swraw);
              uint4 out;
              uint32_t* o = reinterpret_cast<uint32_t*>(&out);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float2 sc = __half22float2(swh[e]);
                const __half2 hv = __floats2half2_rn(__uint_as_float(r[g * 8 + 2 * e]) * sc.x,
                                                     __uint_as_float(r[g * 8 + 2 * e + 1]) * sc.y);
                o[e] = *reinterpret_cast<const uint32_t*>(&hv);
              }
              *reinterpret_cast<uint4*>(yrow + g * 8) = out;
            }
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[b]);       // this warp's quarter of the buffer is drained
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 2 * BN);
  }
}

// The main kernel.  Its design comes from decode-sized batches (M <= 64), where the product is bound by
// reading the packed weights once; with 128-token tiles it also takes the larger batches (see the
// dispatch at the end of the file), because the weights as a tensor-memory operand cost no
// shared-memory traffic.  The operands swap roles.  A tile is 128 OUTPUT CHANNELS (the MMA's M and the accumulator's lanes), the
// tokens are the MMA's N (16, 32 or 64): the token tiles are a few KB straight from TMA, and an MMA
// with a narrow N takes a third of the time.  The widened weights never touch shared memory: each
// thread of a converter group reads the 128 packed bytes of "its" channel from the staging ring,
// widens them in registers and stores them into a ring in tensor memory (tcgen05.st), from where the
// MMA takes its A operand -- through shared memory the fp16 operand alone cost 128 KB of traffic per
// 256 channels and bounded the kernel (20 us on 14336 x 4096 against 28.7 us with 64-channel stages,
// whose hand-overs cost 920 cycles each).  A stage is a whole staging block: 256 channels, sixteen
// MMAs.  Two converter groups alternate stages (a third group and a third operand stage changed
// nothing).  What bounds a stage now, at about 1300 cycles: two things of about the same size -- the
// sixteen MMAs of a stage take about 76 cycles each (with the converters idle a stage still takes 1220
// cycles; a second issuing thread with an accumulator of its own, with or without a third converter
// group, changed nothing, so it is the tensor pipe reading its 4 KB A operand out of tensor memory per
// MMA, not the issue), and a converter group needs about as long to widen and move
// the 64 KB fp16 operand of a stage into tensor memory.  Where the tiles alone leave most SMs idle
// (4096 channels: 32 tiles) K is split over a cluster of 2 or 4 CTAs.  The accumulator holds one channel
// per thread and the tokens along its registers; a warp's stores of one token cover 32 consecutive
// channels.
constexpr int WOD_CONV_GROUPS = 2;
constexpr int WOD_CONV_WARPS = 4 * WOD_CONV_GROUPS;
constexpr int WOD_THREADS = (2 + WOD_CONV_WARPS + WO_EPI_WARPS) * 32;
constexpr int WOD_A_STAGES = 2;           // tensor-memory operand stages of 128 columns (256 fp16 channels)
// accumulators: columns [0, 2 NT); operand ring: two stages of 128 columns from column max(128, 2 NT) on

template <int NT, int ST, int SS>
struct WoDecSmem {
  static constexpr int T_KB = NT * 128;               // tokens x 64 channels fp16 (one k-block)
  static constexpr int T_TILE = 4 * T_KB;             // a stage: four k-blocks
  static constexpr int W_ST = 128 * 128;              // 128 channels x 256 packed codes
  static constexpr int OFF_T = 0;
  static constexpr int OFF_W_ST = OFF_T + ST * T_TILE;
  static constexpr int OFF_BAR = OFF_W_ST + SS * W_ST;
  static constexpr int NUM_BARS = 2 * ST + 2 * SS + 2 * WOD_A_STAGES + 4;
  static constexpr int OFF_TMEM = OFF_BAR + NUM_BARS * 8;
  static constexpr int TOTAL = OFF_TMEM + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

template <int NT, int ST, int SS, int CT>
__global__ void __launch_bounds__(WOD_THREADS, 1)
wo_gemm_tmem_kernel(const __grid_constant__ CUtensorMap tmap_z, const __grid_constant__ CUtensorMap tmap_w,
                      const __half* __restrict__ sw, int M, int N, int K, __half* __restrict__ Y, int splits) {
  using L = WoDecSmem<NT, ST, SS>;
  // CT = channel tiles of 128 that share a token tile (1 or 2).  With one, two accumulators alternate
  // between tiles (the epilogue of a tile runs under the next tile's MMAs); with two, both accumulators
  // belong to the same tile -- channels [0, 128) and [128, 256) of it -- and every token block that
  // reaches shared memory feeds two MMAs instead of one.
  static_assert(CT == 1 || CT == 2, "one or two channel tiles per token tile");
  static_assert(2 * NT + 128 * WOD_A_STAGES <= 512, "tensor-memory plan does not fit");
  constexpr int NBUF = 2 / CT;                           // accumulator sets that alternate between tiles
  constexpr int WOD_A_COL0 = 2 * NT > 128 ? 2 * NT : 128;
  griddep_launch_dependents();
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* t_full = bars;
  uint64_t* t_empty = t_full + ST;
  uint64_t* st_full = t_empty + ST;
  uint64_t* st_empty = st_full + SS;
  uint64_t* a_full = st_empty + SS;
  uint64_t* a_empty = a_full + WOD_A_STAGES;
  uint64_t* tmem_full = a_empty + WOD_A_STAGES;   // [2]
  uint64_t* tmem_empty = tmem_full + 2;           // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_TMEM);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = K / 64;
  const int num_sb = (num_kb + 3) / 4;        // stages per tile (the last may hold fewer than four k-blocks)
  // A tile is 128 channels x NT tokens; the channel tiles run fastest, so that the CTAs at work at one
  // time share a few token tiles (which stay in L2) and stream different weights.
  const int tiles_n = (N + 128 * CT - 1) / (128 * CT);
  const int num_tiles = tiles_n * ((M + NT - 1) / NT);
  const uint32_t limit = wait_limit();
  // K split over a cluster of `splits` CTAs (1, 2 or 4) where the tiles alone leave most SMs idle: the
  // cluster's CTAs work on the same tile, CTA r of it on the stages [sb0, sb1); the launcher then gives
  // every cluster exactly one tile, and the partial tiles meet in CTA 0 at the end (see the epilogue).
  const uint32_t crank = splits > 1 ? cluster_ctarank() : 0u;
  const int cid = static_cast<int>(blockIdx.x) / splits, ncl = static_cast<int>(gridDim.x) / splits;
  const int sb0 = static_cast<int>(crank) * num_sb / splits, sb1 = (static_cast<int>(crank) + 1) * num_sb / splits;

  // The weights do not depend on the kernel before this one: the first ring-full of them is requested
  // before anything else is set up and before that kernel's completion is awaited.
  int pre = 0;
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmap_w);
    for (int s = 0; s < SS; ++s) mbar_init(&st_full[s], 1);
    mbar_fence_init();
    {
      int t = cid, sb = sb0, half = 0;
      while (pre < SS && t < num_tiles && sb < sb1) {
        mbar_arrive_expect_tx(&st_full[pre], L::W_ST);
        tma_load_2d(smem + L::OFF_W_ST + pre * L::W_ST, &tmap_w, &st_full[pre], sb * 128,
                    ((t % tiles_n) * CT + half) * 128);
        ++pre;
        if (++half < CT) continue;
        half = 0;
        if (++sb >= sb1) {
          sb = sb0;
          t += ncl;
        }
      }
    }
    tma_prefetch_desc(&tmap_z);
    for (int s = 0; s < ST; ++s) {
      mbar_init(&t_full[s], 1);
      mbar_init(&t_empty[s], 1);
    }
    for (int s = 0; s < SS; ++s) mbar_init(&st_empty[s], 4);          // the four warps of one converter group
    for (int s = 0; s < WOD_A_STAGES; ++s) {
      mbar_init(&a_full[s], 4);
      mbar_init(&a_empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&tmem_full[b], 1);
      mbar_init(&tmem_empty[b], WO_EPI_WARPS);
    }
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  griddep_wait();                                     // Z16 may come from the kernel launched before this one

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      uint32_t sit = 0;
      bool ok = true;
      for (int tile = cid; tile < num_tiles && ok; tile += ncl) {
        for (int sb = sb0; sb < sb1 && ok; ++sb) {
          for (int half = 0; half < CT && ok; ++half, ++sit) {
            if (sit >= static_cast<uint32_t>(pre)) {        // the first `pre` blocks are on their way already
              const int ss = sit % SS;
              ok = mbar_wait(&st_empty[ss], ((sit / SS) & 1) ^ 1, WO_ST_EMPTY, limit);
              if (!ok) break;
              mbar_arrive_expect_tx(&st_full[ss], L::W_ST);
              tma_load_2d(smem + L::OFF_W_ST + ss * L::W_ST, &tmap_w, &st_full[ss], sb * 128,
                          ((tile % tiles_n) * CT + half) * 128);
            }
            if (half != 0) continue;                        // the token block serves both channel tiles
            const uint32_t tit = sit / CT;
            const int st = tit % ST;
            const int nk = (num_kb - 4 * sb) < 4 ? (num_kb - 4 * sb) : 4;
            ok = mbar_wait(&t_empty[st], ((tit / ST) & 1) ^ 1, WO_A_EMPTY, limit);
            if (!ok) break;
            mbar_arrive_expect_tx(&t_full[st], static_cast<uint32_t>(nk * L::T_KB));
            for (int h = 0; h < nk; ++h)
              tma_load_2d(smem + L::OFF_T + st * L::T_TILE + h * L::T_KB, &tmap_z, &t_full[st], (4 * sb + h) * 64,
                          (tile / tiles_n) * NT);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------------------
    if (elect_one()) {
      constexpr uint32_t idesc = umma_idesc(/*c=f32*/ 1, /*a=f16*/ 0, /*b=f16*/ 0, 128, NT);
      // descriptors of a stage differ from the ring's first by constants in the start-address field
      // (16-byte units, no carry out of it): formed once, the stage's MMAs unrolled
      const uint64_t t_desc0 = umma_desc_sw128(smem_u32(smem + L::OFF_T));
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = cid; tile < num_tiles && ok; tile += ncl, ++tcount) {
        const uint32_t b = tcount % NBUF;
        ok = mbar_wait(&tmem_empty[b], ((tcount / NBUF) & 1) ^ 1, WO_TMEM_EMPTY, limit);
        if (!ok) break;
        tc_fence_after_sync();
        for (int sb = sb0; sb < sb1 && ok; ++sb) {
#pragma unroll
          for (int half = 0; half < CT; ++half, ++it) {
            const uint32_t tit = it / CT;
            const int st = tit % ST, sa = it % WOD_A_STAGES;
            const int nk = (num_kb - 4 * sb) < 4 ? (num_kb - 4 * sb) : 4;
            if (half == 0) ok = mbar_wait(&t_full[st], (tit / ST) & 1, WO_A_FULL, limit);
            ok = ok && mbar_wait(&a_full[sa], (it / WOD_A_STAGES) & 1, WO_B_FULL, limit);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t tmem_d = tmem_base + (b * CT + half) * NT;
            const uint32_t a_tmem = tmem_base + WOD_A_COL0 + sa * 128;
            const uint64_t td = t_desc0 + static_cast<uint64_t>((st * L::T_TILE) >> 4);
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              if (h < nk) {
#pragma unroll
                for (int k = 0; k < 4; ++k)       // K = 16 fp16: eight 32-bit columns of A, 32 bytes of a token row
                  umma_f16_ts(tmem_d, a_tmem + 32 * h + 8 * k, td + ((h * L::T_KB + k * 32) >> 4), idesc,
                              ((sb - sb0) | h | k) != 0 ? 1u : 0u);
              }
            }
            if (half == CT - 1) umma_commit(&t_empty[st]);
            umma_commit(&a_empty[sa]);
          }
        }
        if (!ok) break;
        umma_commit(&tmem_full[b]);
      }
    }
  } else if (warp < 2 + WOD_CONV_WARPS) {
    // ------------------------------ weight converters: staging -> registers -> tensor memory ------
    const int q = warp & 3;
    const int grp = (warp - 2) >> 2;                    // this group's stages: it % WOD_CONV_GROUPS == grp
    const int r = q * 32 + lane;                        // channel of the tile = TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = cid; tile < num_tiles && ok; tile += ncl) {
      for (int sbh = sb0 * CT; sbh < sb1 * CT && ok; ++sbh, ++it) {
        if ((it % WOD_CONV_GROUPS) != static_cast<uint32_t>(grp)) continue;
        const int sb = sbh / CT;
        const int ss = it % SS, sa = it % WOD_A_STAGES;
        const int nk = (num_kb - 4 * sb) < 4 ? (num_kb - 4 * sb) : 4;
        ok = mbar_wait(&st_full[ss], (it / SS) & 1, WO_ST_FULL, limit);
        if (!ok) break;
        const unsigned char* row = smem + L::OFF_W_ST + ss * L::W_ST + r * 128;
        uint4 w[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) w[c] = *reinterpret_cast<const uint4*>(row + ((c ^ (r & 7)) << 4));
        ok = mbar_wait(&a_empty[sa], ((it / WOD_A_STAGES) & 1) ^ 1, WO_B_EMPTY, limit);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll
        for (int h = 0; h < 4; ++h) {                   // k-block h: chunks 2h, 2h+1 -> 32 columns
          if (h < nk) {
            uint32_t v[32];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              const uint4 x = w[2 * h + j];
              const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                const uint4 f = widen_word(xs[g]);
                v[16 * j + 4 * g + 0] = f.x;
                v[16 * j + 4 * g + 1] = f.y;
                v[16 * j + 4 * g + 2] = f.z;
                v[16 * j + 4 * g + 3] = f.w;
              }
            }
            tmem_st_32x32b_x32(tmem_base + lane_addr + WOD_A_COL0 + sa * 128 + h * 32, v);
          }
        }
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&a_full[sa]);
          mbar_arrive(&st_empty[ss]);
        }
      }
    }
  } else {
    // ------------------------------ epilogue warps ------------------------------------------
    const int quarter = warp & 3;
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = cid; tile < num_tiles && ok; tile += ncl, ++tcount) {
      const uint32_t b = tcount % NBUF;
      const int ch0 = (tile % tiles_n) * (128 * CT) + quarter * 32 + lane;
      const int tok0 = (tile / tiles_n) * NT;
      float swh[CT];
#pragma unroll
      for (int half = 0; half < CT; ++half) swh[half] = (ch0 + 128 * half < N) ? __half2float(sw[ch0 + 128 * half]) : 0.0f;
      ok = mbar_wait(&tmem_full[b], (tcount / NBUF) & 1, WO_TMEM_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tmem_d = tmem_base + b * CT * NT + (static_cast<uint32_t>(quarter * 32) << 16);
      if (splits > 1) {                                   // (launched with CT = 1 only)
        // K split over the cluster (one tile per cluster): CTAs other than the first leave their partial
        // tile in their own shared memory, [token][channel] fp32 over the token ring (every load into it
        // has been consumed once the accumulator is complete); the first CTA adds them after the cluster
        // barrier below.  Nothing is stored here.
        if (crank != 0) {
          float* part = reinterpret_cast<float*>(smem + L::OFF_T);
#pragma unroll
          for (int c = 0; c < NT / 16; ++c) {
            uint32_t r[16];
            tmem_ld_32x32b_x16(tmem_d + c * 16, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) part[(c * 16 + e) * 128 + quarter * 32 + lane] = __uint_as_float(r[e]);
          }
        }
        continue;
      }
#pragma unroll
      for (int half = 0; half < CT; ++half) {
        const int ch = ch0 + 128 * half;
        const float swv = swh[half];
#pragma unroll
        for (int c = 0; c < NT / 16; ++c) {
          uint32_t r[16];
          tmem_ld_32x32b_x16(tmem_d + half * NT + c * 16, r);
          tmem_wait_ld();
          if (ch < N) {
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const int tok = tok0 + c * 16 + e;
              if (tok < M) Y[static_cast<size_t>(tok) * N + ch] = __float2half_rn(__uint_as_float(r[e]) * swv);
            }
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[b]);
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (splits > 1) {
    // Every thread of every CTA of the cluster comes through here, whatever happened above: the two
    // barriers are hardware barriers, not polled waits.
    cluster_sync_all();                                 // the partial tiles are in place
    if (crank == 0 && warp >= 2 + WOD_CONV_WARPS && cid < num_tiles) {
      tc_fence_after_sync();
      const int quarter = warp & 3;
      const int ch = (cid % tiles_n) * 128 + quarter * 32 + lane;                          // CT = 1 here
      const int tok0 = (cid / tiles_n) * NT;
      const float swv = (ch < N) ? __half2float(sw[ch]) : 0.0f;
      const uint32_t tmem_d = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);     // accumulator 0: one tile
      const float* part = reinterpret_cast<const float*>(smem + L::OFF_T);
#pragma unroll
      for (int c = 0; c < NT / 16; ++c) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(tmem_d + c * 16, r);
        tmem_wait_ld();
        // all of a chunk's remote reads are issued before the first is used (each is a round trip to
        // another SM); the sums are taken in a fixed order: deterministic
        float a[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) a[e] = __uint_as_float(r[e]);
        for (int pr = 1; pr < splits; ++pr) {
          const uint32_t base = cluster_map(part + (c * 16) * 128 + quarter * 32 + lane, static_cast<uint32_t>(pr));
          float v[16];
#pragma unroll
          for (int e = 0; e < 16; ++e)
            asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v[e]) : "r"(base + e * 512) : "memory");
#pragma unroll
          for (int e = 0; e < 16; ++e) a[e] += v[e];
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const int tok = tok0 + c * 16 + e;
          if (ch < N && tok < M) Y[static_cast<size_t>(tok) * N + ch] = __float2half_rn(a[e] * swv);
        }
      }
      tc_fence_before_sync();
    }
    cluster_sync_all();                                 // the others' shared memory has been read
  }
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// The CTA-pair form of the kernel above for batches above 128 tokens (tcgen05 cta_group::2, M = 256,
// N = 256).  In the single-CTA form an MMA of M = 128, N = 128 with its A operand in tensor memory
// takes about 96 cycles instead of 64 (reading the 4 KB of A costs as much as the arithmetic), and every
// 128 x 128 tile pulls its 128 tokens out of L2 again.  Here two CTAs share a tile of 256 channels x 256
// tokens: CTA r widens channels [128 r, 128 r + 128) of the tile into its own tensor memory (its half of
// the M operand, its accumulator lanes) and loads tokens [128 r, 128 r + 128) of the tile (its half of
// the N operand).  An MMA then does 128 cycles of arithmetic per 4 KB of A, and a CTA reads 128 tokens per
// 256 tokens' worth of work.  The accumulator (128 lanes x 256 columns per CTA) is single-buffered: the
// operand ring needs the other 256 columns; eight epilogue warps (two per lane quarter, 128 columns
// each) hand it back after their last read.
//   warp 0        TMA: packed weights of this CTA's channels (staging ring), this CTA's tokens (ring
//                 stage s = four 64-channel k-blocks)
//   warps 2..9    two converter groups, alternating stages: staging -> registers -> tensor-memory ring
//                 stage s; a warp reports the stage to the leader once its part is stored AND this
//                 CTA's tokens of the stage have landed
//   warp 1        (leader CTA) sixteen MMAs per stage; the commit frees stage s in both CTAs
//   warps 10..17  epilogue: tensor memory -> scale -> fp16 stores
constexpr int WP_EPI_WARPS = 8;
constexpr int WP_THREADS = (2 + WOD_CONV_WARPS + WP_EPI_WARPS) * 32;
constexpr int WP_S = 2;                  // ring stages: 256 channels of K (tokens in shared, weights in tensor memory)
constexpr int WP_A_COL0 = 256;           // first column of the operand ring (0..255: accumulator)
static_assert(WP_S == WOD_CONV_GROUPS, "a converter group owns one ring stage");

enum WoPairSite : uint32_t {
  WP_ST_EMPTY = 96, WP_ST_FULL, WP_T_FULL, WP_EMPTY_T, WP_EMPTY_A, WP_FULL, WP_TMEM_FULL, WP_TMEM_EMPTY
};

template <int SS>
struct WoPairSmem {
  static constexpr int T_KB = 128 * 128;              // 128 tokens x 64 channels fp16 (one k-block)
  static constexpr int T_TILE = 4 * T_KB;             // a stage: four k-blocks
  static constexpr int W_ST = 128 * 128;              // 128 channels x 256 packed codes
  static constexpr int OFF_T = 0;
  static constexpr int OFF_W_ST = OFF_T + WP_S * T_TILE;
  static constexpr int OFF_BAR = OFF_W_ST + SS * W_ST;
  static constexpr int NUM_BARS = 2 * SS + 3 * WP_S + 2;
  static constexpr int OFF_TMEM = OFF_BAR + NUM_BARS * 8;
  static constexpr int TOTAL = OFF_TMEM + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

template <int SS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(WP_THREADS, 1)
wo_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_z, const __grid_constant__ CUtensorMap tmap_w,
                    const __half* __restrict__ sw, int M, int N, int K, __half* __restrict__ Y) {
  using L = WoPairSmem<SS>;
  griddep_launch_dependents();
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* st_full = bars;                           // [SS]    packed weights landed (local)
  uint64_t* st_empty = st_full + SS;                  // [SS]    a converter group has read them (local)
  uint64_t* t_full = st_empty + SS;                   // [WP_S]  tokens landed (local)
  uint64_t* full = t_full + WP_S;                     // [WP_S]  stage complete in both CTAs (the leader's copy is used)
  uint64_t* empty = full + WP_S;                      // [WP_S]  the stage's MMAs have retired (each CTA's own copy)
  uint64_t* tmem_full = empty + WP_S;                 // accumulator complete (each CTA's own copy)
  uint64_t* tmem_empty = tmem_full + 1;               // epilogue warps of the pair (the leader's copy is used)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_TMEM);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();            // 0 = leader (issues the MMAs)
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int num_kb = K / 64;
  const int num_sb = (num_kb + 3) / 4;                // stages per tile (the last may hold fewer than four k-blocks)
  // channel tiles run fastest: the pairs at work at one time share a few token tiles, which stay in L2
  const int tiles_n = (N + 255) / 256;
  const int num_tiles = tiles_n * ((M + 255) / 256);
  const uint32_t limit = wait_limit();

  // The weights do not depend on the kernel before this one: the first ring-full of them is requested
  // (local barriers only) before anything else is set up and before that kernel's completion is awaited.
  int pre = 0;
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmap_w);
    for (int s = 0; s < SS; ++s) mbar_init(&st_full[s], 1);
    mbar_fence_init();
    {
      int t = pair, sb = 0;
      while (pre < SS && t < num_tiles) {
        mbar_arrive_expect_tx(&st_full[pre], L::W_ST);
        tma_load_2d(smem + L::OFF_W_ST + pre * L::W_ST, &tmap_w, &st_full[pre], sb * 128,
                    (t % tiles_n) * 256 + static_cast<int>(rank) * 128);
        ++pre;
        if (++sb >= num_sb) {
          sb = 0;
          t += npairs;
        }
      }
    }
    tma_prefetch_desc(&tmap_z);
    for (int s = 0; s < SS; ++s) mbar_init(&st_empty[s], 4);          // the four warps of one converter group
    for (int s = 0; s < WP_S; ++s) {
      mbar_init(&t_full[s], 1);
      mbar_init(&full[s], 2 * 4);                                      // one converter group in each CTA
      mbar_init(&empty[s], 1);
    }
    mbar_init(tmem_full, 1);
    mbar_init(tmem_empty, 2 * WP_EPI_WARPS);
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();                                 // both CTAs' barriers exist before any remote arrival
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  griddep_wait();                                     // Z16 may come from the kernel launched before this one

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {                                  // thread 0: it knows how many blocks are on their way
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
        const int ch0 = (tile % tiles_n) * 256 + static_cast<int>(rank) * 128;
        const int tok0 = (tile / tiles_n) * 256 + static_cast<int>(rank) * 128;
        for (int sb = 0; sb < num_sb && ok; ++sb, ++it) {
          if (it >= static_cast<uint32_t>(pre)) {
            const int ss = it % SS;
            ok = mbar_wait(&st_empty[ss], ((it / SS) & 1) ^ 1, WP_ST_EMPTY, limit);
            if (!ok) break;
            mbar_arrive_expect_tx(&st_full[ss], L::W_ST);
            tma_load_2d(smem + L::OFF_W_ST + ss * L::W_ST, &tmap_w, &st_full[ss], sb * 128, ch0);
          }
          const int s = it % WP_S;
          const int nk = (num_kb - 4 * sb) < 4 ? (num_kb - 4 * sb) : 4;
          ok = mbar_wait(&empty[s], ((it / WP_S) & 1) ^ 1, WP_EMPTY_T, limit);
          if (!ok) break;
          mbar_arrive_expect_tx(&t_full[s], static_cast<uint32_t>(nk * L::T_KB));
          for (int h = 0; h < nk; ++h)
            tma_load_2d(smem + L::OFF_T + s * L::T_TILE + h * L::T_KB, &tmap_z, &t_full[s], (4 * sb + h) * 64, tok0);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader CTA) -------------------------------
    if (rank == 0 && elect_one()) {
      constexpr uint32_t idesc = umma_idesc(/*c=f32*/ 1, /*a=f16*/ 0, /*b=f16*/ 0, 256, 256);
      const uint64_t t_desc0 = umma_desc_sw128(smem_u32(smem + L::OFF_T));
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += npairs, ++tcount) {
        ok = mbar_wait(tmem_empty, (tcount & 1) ^ 1, WP_TMEM_EMPTY, limit);
        if (!ok) break;
        tc_fence_after_sync();
        for (int sb = 0; sb < num_sb; ++sb, ++it) {
          const int s = it % WP_S;
          const int nk = (num_kb - 4 * sb) < 4 ? (num_kb - 4 * sb) : 4;
          ok = mbar_wait(&full[s], (it / WP_S) & 1, WP_FULL, limit);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t a_tmem = tmem_base + WP_A_COL0 + s * 128;
          const uint64_t td = t_desc0 + static_cast<uint64_t>((s * L::T_TILE) >> 4);
#pragma unroll
          for (int h = 0; h < 4; ++h) {
            if (h < nk) {
#pragma unroll
              for (int k = 0; k < 4; ++k)         // K = 16 fp16: eight 32-bit columns of A, 32 bytes of a token row
                umma_f16_ts_pair(tmem_base, a_tmem + 32 * h + 8 * k, td + ((h * L::T_KB + k * 32) >> 4), idesc,
                                 (sb | h | k) != 0 ? 1u : 0u);
            }
          }
          umma_commit_pair_mc(&empty[s], 3);          // frees ring stage s in both CTAs
        }
        umma_commit_pair_mc(tmem_full, 3);            // accumulator complete (or abandoned)
      }
    }
  } else if (warp < 2 + WOD_CONV_WARPS) {
    // ------------------------------ weight converters: staging -> registers -> tensor memory ------
    const int q = warp & 3;
    const int grp = (warp - 2) >> 2;                    // this group's ring stage
    const int r = q * 32 + lane;                        // channel of the CTA's 128 = TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
      for (int sb = 0; sb < num_sb && ok; ++sb, ++it) {
        if ((it % WP_S) != static_cast<uint32_t>(grp)) continue;
        const int ss = it % SS, s = grp;
        const int nk = (num_kb - 4 * sb) < 4 ? (num_kb - 4 * sb) : 4;
        ok = mbar_wait(&st_full[ss], (it / SS) & 1, WP_ST_FULL, limit);
        if (!ok) break;
        const unsigned char* row = smem + L::OFF_W_ST + ss * L::W_ST + r * 128;
        uint4 w[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) w[c] = *reinterpret_cast<const uint4*>(row + ((c ^ (r & 7)) << 4));
        ok = mbar_wait(&empty[s], ((it / WP_S) & 1) ^ 1, WP_EMPTY_A, limit);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll
        for (int h = 0; h < 4; ++h) {                   // k-block h: chunks 2h, 2h+1 -> 32 columns
          if (h < nk) {
            uint32_t v[32];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              const uint4 x = w[2 * h + j];
              const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                const uint4 f = widen_word(xs[g]);
                v[16 * j + 4 * g + 0] = f.x;
                v[16 * j + 4 * g + 1] = f.y;
                v[16 * j + 4 * g + 2] = f.z;
                v[16 * j + 4 * g + 3] = f.w;
              }
            }
            tmem_st_32x32b_x32(tmem_base + lane_addr + WP_A_COL0 + s * 128 + h * 32, v);
          }
        }
        tmem_wait_st();
        tc_fence_before_sync();
        // the stage also needs this CTA's tokens: the leader learns of both with one arrival
        ok = mbar_wait(&t_full[s], (it / WP_S) & 1, WP_T_FULL, limit);
        if (!ok) break;
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_cluster(&full[s], 0);
          mbar_arrive(&st_empty[ss]);
        }
      }
    }
  } else {
    // ------------------------------ epilogue warps ------------------------------------------
    const int q = warp & 3;                             // TMEM lane quarter this warp may read
    const int half = (warp - (2 + WOD_CONV_WARPS)) >> 2;  // its 128 of the 256 token columns
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = pair; tile < num_tiles && ok; tile += npairs, ++tcount) {
      const int ch = (tile % tiles_n) * 256 + static_cast<int>(rank) * 128 + q * 32 + lane;
      const int tok0 = (tile / tiles_n) * 256 + half * 128;
      const float swv = (ch < N) ? __half2float(sw[ch]) : 0.0f;
      ok = mbar_wait(tmem_full, tcount & 1, WP_TMEM_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tmem_d = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + half * 128;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(tmem_d + c * 16, r);
        tmem_wait_ld();
        if (c == 7) {                                   // last read of this warp: hand the accumulator back
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(tmem_empty, 0);
        }
        if (ch < N) {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const int tok = tok0 + c * 16 + e;
            if (tok < M) Y[static_cast<size_t>(tok) * N + ch] = __float2half_rn(__uint_as_float(r[e]) * swv);
          }
        }
      }
    }
  }

  // Neither CTA may leave while its partner can still reach its shared memory, barriers or TMEM.
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

// One or two tokens: dot products on the CUDA cores.  The product is pure streaming then (29 MB of
// packed weights against a few MFLOP), and the tensor-core forms pay more in hand-overs than the read
// costs.  Each warp takes four weight rows at a time; every lane reads 16-byte pieces of them straight
// from global memory (coalesced, several in flight), widens the nibbles to half2 as above, converts to
// fp32 and multiplies with the tokens, which the CTA holds in shared memory as fp32.  Accumulation is
// fp32 throughout; a row's sum is completed by one warp (shuffle reduction): deterministic.
constexpr int WOV_ROWS = 4, WOV_UNROLL = 2;

template <int MT>
__global__ void __launch_bounds__(512)
wo_gemv_kernel(const __half* __restrict__ Z16, const uint8_t* __restrict__ Wq, const __half* __restrict__ sw, int M,
               int N, int K, __half* __restrict__ Y) {
  // No early start for whatever follows: its CTAs would sit on the SMs beside this kernel's (a second
  // large shared-memory allocation per SM) and slow the streaming down (36 us instead of 18 on
  // 1 x 4096 x 14336 in back-to-back launches).
  griddep_wait();                                        // Z16 may come from the kernel launched before this one
  // Tokens as fp32, laid out [token][word of a piece g][half h][piece c][4]: the lanes of a warp work on
  // consecutive pieces c, so their 16-byte reads for one (g, h) are contiguous (no bank conflicts).
  extern __shared__ __align__(16) float zs[];
  const int nchunk = K / 32;                             // 16-byte pieces of packed weights per row
  for (int i = threadIdx.x; i < MT * (K / 8); i += blockDim.x) {
    const int t = i / (K / 8), c = i % (K / 8);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (t < M) v = __ldg(reinterpret_cast<const uint4*>(Z16 + static_cast<size_t>(t) * K) + c);
    const __half2* h = reinterpret_cast<const __half2*>(&v);
    const float2 a = __half22float2(h[0]), b = __half22float2(h[1]), c2 = __half22float2(h[2]), d = __half22float2(h[3]);
    const int piece = c >> 2, g = c & 3;
    float* base = zs + static_cast<size_t>(t) * K;
    *reinterpret_cast<float4*>(base + ((g * 2 + 0) * nchunk + piece) * 4) = make_float4(a.x, a.y, b.x, b.y);
    *reinterpret_cast<float4*>(base + ((g * 2 + 1) * nchunk + piece) * 4) = make_float4(c2.x, c2.y, d.x, d.y);
  }
  __syncthreads();

  const int lane = threadIdx.x & 31;
  const int warps_per_cta = blockDim.x >> 5;
  const long long ntask = (N + WOV_ROWS - 1) / WOV_ROWS;
  const long long wstride = static_cast<long long>(gridDim.x) * warps_per_cta;
  for (long long task = static_cast<long long>(threadIdx.x >> 5) * gridDim.x + blockIdx.x; task < ntask; task += wstride) {
    const int row0 = static_cast<int>(task) * WOV_ROWS;
    float acc[WOV_ROWS][MT];
#pragma unroll
    for (int r = 0; r < WOV_ROWS; ++r)
#pragma unroll
      for (int t = 0; t < MT; ++t) acc[r][t] = 0.0f;
    const uint4* wrow[WOV_ROWS];
#pragma unroll
    for (int r = 0; r < WOV_ROWS; ++r)
      wrow[r] = reinterpret_cast<const uint4*>(Wq + static_cast<size_t>(min(row0 + r, N - 1)) * (K / 2));
    for (int c0 = lane; c0 < nchunk; c0 += 32 * WOV_UNROLL) {
      uint4 wv[WOV_UNROLL][WOV_ROWS];
#pragma unroll
      for (int u = 0; u < WOV_UNROLL; ++u) {
        const int c = c0 + 32 * u;
#pragma unroll
        for (int r = 0; r < WOV_ROWS; ++r)
          wv[u][r] = (c < nchunk) ? __ldcs(wrow[r] + c) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < WOV_UNROLL; ++u) {
        const int c = c0 + 32 * u;
        if (c < nchunk) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {                   // word g of the piece: channels 32 c + 8 g .. + 7
            float zf[MT][8];
#pragma unroll
            for (int t = 0; t < MT; ++t) {
              const float4 z0 = *reinterpret_cast<const float4*>(zs + static_cast<size_t>(t) * K + ((g * 2 + 0) * nchunk + c) * 4);
              const float4 z1 = *reinterpret_cast<const float4*>(zs + static_cast<size_t>(t) * K + ((g * 2 + 1) * nchunk + c) * 4);
              zf[t][0] = z0.x; zf[t][1] = z0.y; zf[t][2] = z0.z; zf[t][3] = z0.w;
              zf[t][4] = z1.x; zf[t][5] = z1.y; zf[t][6] = z1.z; zf[t][7] = z1.w;
            }
#pragma unroll
            for (int r = 0; r < WOV_ROWS; ++r) {
              const uint32_t word = g == 0 ? wv[u][r].x : (g == 1 ? wv[u][r].y : (g == 2 ? wv[u][r].z : wv[u][r].w));
              const uint4 f = widen_word(word);
              const float2 w01 = __half22float2(*reinterpret_cast<const __half2*>(&f.x));
              const float2 w23 = __half22float2(*reinterpret_cast<const __half2*>(&f.y));
              const float2 w45 = __half22float2(*reinterpret_cast<const __half2*>(&f.z));
              const float2 w67 = __half22float2(*reinterpret_cast<const __half2*>(&f.w));
#pragma unroll
              for (int t = 0; t < MT; ++t) {
                float a = acc[r][t];
                a = fmaf(zf[t][0], w01.x, a); a = fmaf(zf[t][1], w01.y, a);
                a = fmaf(zf[t][2], w23.x, a); a = fmaf(zf[t][3], w23.y, a);
                a = fmaf(zf[t][4], w45.x, a); a = fmaf(zf[t][5], w45.y, a);
                a = fmaf(zf[t][6], w67.x, a); a = fmaf(zf[t][7], w67.y, a);
                acc[r][t] = a;
              }
            }
          }
        }
      }
    }
#pragma unroll
    for (int r = 0; r < WOV_ROWS; ++r)
#pragma unroll
      for (int t = 0; t < MT; ++t) {
        float a = acc[r][t];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        acc[r][t] = a;
      }
    if (lane < WOV_ROWS * MT) {
      const int r = lane / MT, t = lane % MT;
      float a = 0.0f;
#pragma unroll
      for (int rr = 0; rr < WOV_ROWS; ++rr)
#pragma unroll
        for (int tt = 0; tt < MT; ++tt)
          if (rr == r && tt == t) a = acc[rr][tt];
      const int row = row0 + r;
      if (row < N && t < M) Y[static_cast<size_t>(t) * N + row] = __float2half_rn(a * __half2float(__ldg(sw + row)));
    }
  }
}

// Plain kernel for shapes the tensor-core path does not take (K % 64 != 0, N % 8 != 0): one thread per
// output channel, fp32 multiply-adds in channel order; gridDim.y strides over the token rows.
__global__ void wo_gemm_simple_kernel(const __half* __restrict__ Z16, const uint8_t* __restrict__ Wq,
                                      const __half* __restrict__ sw, int M, int N, int K, __half* __restrict__ Y) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= N) return;
  const uint32_t* wrow = reinterpret_cast<const uint32_t*>(Wq + static_cast<size_t>(c) * (K / 2));
  const float swv = __half2float(sw[c]);
  for (int t = blockIdx.y; t < M; t += gridDim.y) {
    const __half* z = Z16 + static_cast<size_t>(t) * K;
    float acc = 0.0f;
    for (int g = 0; g < K / 8; ++g) {
      const uint32_t word = wrow[g];
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        const int c0 = (static_cast<int>(word << (28 - 4 * s))) >> 28;          // nibble position s: channel 2s
        const int c1 = (static_cast<int>(word << (12 - 4 * s))) >> 28;          // nibble position s + 4: channel 2s + 1
        acc = fmaf(__half2float(z[8 * g + 2 * s]), static_cast<float>(c0), acc);
        acc = fmaf(__half2float(z[8 * g + 2 * s + 1]), static_cast<float>(c1), acc);
      }
    }
    Y[static_cast<size_t>(t) * N + c] = __float2half_rn(acc * swv);
  }
}

// Channel order -> weight-only storage order, one 32-bit word (eight channels) per thread, in place.
__global__ void interleave_nibbles_kernel(uint32_t* __restrict__ words, long long count) {
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < count;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const uint32_t w = words[i];
    uint32_t o = 0;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      o |= ((w >> (8 * s)) & 0xFu) << (4 * s);               // channel 2s     -> position s
      o |= ((w >> (8 * s + 4)) & 0xFu) << (4 * s + 16);      // channel 2s + 1 -> position s + 4
    }
    words[i] = o;
  }
}

template <int BN, int SA, int SS, int SB>
sq_status_t launch_wo_tc(const void* Z16, const void* Wq, const void* sw, int M, int N, int K, void* Y, cudaStream_t s) {
  using L = WoSmem<BN, SA, SS, SB>;
  static_assert(L::DYN_BYTES <= 227 * 1024, "shared-memory plan does not fit");
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return SQ_ERR_CUDA;
  CUtensorMap mz, mw;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(M)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * 2};
  const cuuint32_t box[2] = {64, WO_BM};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&mz, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(Z16), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return SQ_ERR_CUDA;
  if (!make_packed_map(&mw, Wq, N, K / 2, BN)) return SQ_ERR_CUDA;
  auto kern = wo_gemm_tc_kernel<BN, SA, SS, SB>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), L::DYN_BYTES)) return SQ_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const int tiles = ((N + BN - 1) / BN) * ((M + WO_BM - 1) / WO_BM);
  const int grid = tiles < sms ? tiles : sms;
  const cudaError_t err = launch_maybe_pdl(kern, dim3(grid), dim3(WO_THREADS), L::DYN_BYTES, s, mz, mw,
                                           static_cast<const __half*>(sw), M, N, K, static_cast<__half*>(Y));
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SQ_OK : SQ_ERR_CUDA;
}

template <int NT, int ST, int SS, int CT = 1>
sq_status_t launch_wo_decode(const void* Z16, const void* Wq, const void* sw, int M, int N, int K, void* Y,
                             cudaStream_t s) {
  using L = WoDecSmem<NT, ST, SS>;
  static_assert(L::DYN_BYTES <= 227 * 1024, "shared-memory plan does not fit");
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return SQ_ERR_CUDA;
  CUtensorMap mz, mw;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(M)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * 2};
  const cuuint32_t box[2] = {64, NT};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&mz, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(Z16), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return SQ_ERR_CUDA;
  if (!make_packed_map(&mw, Wq, N, K / 2, 128)) return SQ_ERR_CUDA;
  auto kern = wo_gemm_tmem_kernel<NT, ST, SS, CT>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), L::DYN_BYTES)) return SQ_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const int tiles = ((N + 128 * CT - 1) / (128 * CT)) * ((M + NT - 1) / NT);
  // K over clusters of 2 or 4 CTAs where the tiles alone would leave more than half of the SMs idle and
  // every CTA still gets at least four 256-channel stages; each cluster then has exactly one tile.
  const int num_sb = (K / 64 + 3) / 4;
  int splits = 1;
  while (CT == 1 && splits < 4 && tiles * splits * 2 <= sms && num_sb / (splits * 2) >= 4) splits *= 2;
  const int grid = splits > 1 ? tiles * splits : (tiles < sms ? tiles : sms);
  const cudaError_t err = launch_cluster_maybe_pdl(kern, dim3(grid), dim3(WOD_THREADS), L::DYN_BYTES, s,
                                                   static_cast<unsigned>(splits), mz, mw, static_cast<const __half*>(sw),
                                                   M, N, K, static_cast<__half*>(Y), splits);
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SQ_OK : SQ_ERR_CUDA;
}

template <int SS>
sq_status_t launch_wo_pair(const void* Z16, const void* Wq, const void* sw, int M, int N, int K, void* Y, cudaStream_t s) {
  using L = WoPairSmem<SS>;
  static_assert(L::DYN_BYTES <= 227 * 1024, "shared-memory plan does not fit");
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return SQ_ERR_CUDA;
  CUtensorMap mz, mw;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(M)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * 2};
  const cuuint32_t box[2] = {64, 128};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&mz, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(Z16), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return SQ_ERR_CUDA;
  if (!make_packed_map(&mw, Wq, N, K / 2, 128)) return SQ_ERR_CUDA;
  auto kern = wo_gemm_pair_kernel<SS>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), L::DYN_BYTES)) return SQ_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const int tiles = ((N + 255) / 256) * ((M + 255) / 256);
  const int pairs = tiles < sms / 2 ? tiles : sms / 2;
  const cudaError_t err = launch_maybe_pdl(kern, dim3(2 * pairs), dim3(WP_THREADS), L::DYN_BYTES, s, mz, mw,
                                           static_cast<const __half*>(sw), M, N, K, static_cast<__half*>(Y));
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SQ_OK : SQ_ERR_CUDA;
}

template <int MT>
sq_status_t launch_wo_gemv(const void* Z16, const void* Wq, const void* sw, int M, int N, int K, void* Y, cudaStream_t s) {
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const long long ntask = (N + WOV_ROWS - 1) / WOV_ROWS;
  const int warps = gemv_warps(ntask, sms);
  const int smem = MT * K * 4;
  auto kern = wo_gemv_kernel<MT>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) return SQ_ERR_CUDA;
  const unsigned grid = static_cast<unsigned>(std::min<long long>(sms, (ntask + warps - 1) / warps));
  const cudaError_t err = launch_maybe_pdl(kern, dim3(grid), dim3(warps * 32), static_cast<size_t>(smem), s,
                                           static_cast<const __half*>(Z16), static_cast<const uint8_t*>(Wq),
                                           static_cast<const __half*>(sw), M, N, K, static_cast<__half*>(Y));
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace

sq_status_t launch_wo_gemm(const void* Z16, const void* Wq, const void* sw, int64_t M, int64_t N, int64_t K, void* Y,
                           cudaStream_t s) {
  if (M == 0 || N == 0) return SQ_OK;
  const bool tc_ok = (K % 64 == 0) && (N % 8 == 0);
  if (M <= 2 && K % 32 == 0 && static_cast<int64_t>(M) * K * 4 <= 200 * 1024) {
    // one or two tokens: dot products on the CUDA cores
    if (M == 1) return launch_wo_gemv<1>(Z16, Wq, sw, (int)M, (int)N, (int)K, Y, s);
    return launch_wo_gemv<2>(Z16, Wq, sw, (int)M, (int)N, (int)K, Y, s);
  }
  if (tc_ok && M <= 64 && N >= 128) {
    // decode-sized batches: weights as the M operand, a deep ring of packed weights in flight
    if (M <= 16) return launch_wo_decode<16, 4, 8>(Z16, Wq, sw, (int)M, (int)N, (int)K, Y, s);
    if (M <= 32) return launch_wo_decode<32, 4, 8>(Z16, Wq, sw, (int)M, (int)N, (int)K, Y, s);
    return launch_wo_decode<64, 3, 6>(Z16, Wq, sw, (int)M, (int)N, (int)K, Y, s);
  }
  if (tc_ok && N >= 128) {
    // Larger batches through the same kernel with 128-token tiles: the weights as the tensor-memory
    // operand cost no shared-memory traffic at all, which is what bounds the kernel below (2048 x 4096 x
    // 4096: 76 us there).  From 256 channels on, two channel tiles share every token block (half the
    // token traffic out of L2 per flop: 65 -> 61 us on that shape, 1.85 -> 1.65 ms on 4096 x 28672 x 8192).
    // Above 128 tokens: CTA pairs on 256 x 256 tiles (an MMA's 4 KB of A then feed twice the arithmetic).
    if (M > 128 && N >= 256) return launch_wo_pair<4>(Z16, Wq, sw, (int)M, (int)N, (int)K, Y, s);
    if (N >= 256) return launch_wo_decode<128, 2, 4, 2>(Z16, Wq, sw, (int)M, (int)N, (int)K, Y, s);
    return launch_wo_decode<128, 2, 4>(Z16, Wq, sw, (int)M, (int)N, (int)K, Y, s);
  }
  if (tc_ok) {
    // 256-channel tiles wherever there are enough token rows and channels: the kernel is bound by shared
    // memory (the fp16 operand is written and read there), and a wider tile moves fewer bytes per flop
    // (2048 x 4096 x 4096: 103 us with 128-channel tiles)
    if (M > 128 && N >= 256) return launch_wo_tc<256, 4, 2, 3>(Z16, Wq, sw, (int)M, (int)N, (int)K, Y, s);
    return launch_wo_tc<128, 6, 2, 4>(Z16, Wq, sw, (int)M, (int)N, (int)K, Y, s);
  }
  dim3 block(128), grid((unsigned)((N + 127) / 128), (unsigned)(M < 65535 ? M : 65535));
  wo_gemm_simple_kernel<<<grid, block, 0, s>>>(static_cast<const __half*>(Z16), static_cast<const uint8_t*>(Wq),
                                               static_cast<const __half*>(sw), (int)M, (int)N, (int)K,
                                               static_cast<__half*>(Y));
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

sq_status_t launch_interleave_nibbles(void* Wq, int64_t rows, int64_t K, cudaStream_t s) {
  const long long count = static_cast<long long>(rows) * (K / 8);
  if (count == 0) return SQ_OK;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const long long want = (count + 255) / 256;
  const unsigned grid = static_cast<unsigned>(want < static_cast<long long>(sms) * 16 ? want : static_cast<long long>(sms) * 16);
  interleave_nibbles_kernel<<<grid, 256, 0, s>>>(static_cast<uint32_t*>(Wq), count);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace sq
