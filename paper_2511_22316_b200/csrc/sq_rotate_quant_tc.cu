// Steps 1+2 on the tensor cores (sm_100a): Z_t = R1^T X~_t R2 (Eq. "eq18"), per-token absmax,
// INT4 quantisation (Section 3.2) and packing, one fused kernel.
//
// Both small contractions run as tcgen05.mma kind::f16 with fp32 accumulation in TMEM, with the
// operands split so that the result keeps fp32 accuracy:
//   stage 1  D1[p'][q]  = sum_p R1[p][p'] X~[p][q]     A = R1^T (shared memory, fp16 hi + lo),
//                                                      B = X~   (the TMA tile as it lands, used as
//                                                               an MN-major operand; exact fp16)
//   stage 2  D2[p'][q'] = sum_q D1[p'][q] R2[q][q']    A = D1   (TMEM, fp16 hi + lo, per-lane
//                                                               power-of-two scale),
//                                                      B = R2^T (shared memory, fp16 hi + lo)
// (hi*hi + lo*hi + hi*lo; the lo*lo term is below fp32 resolution).  TMEM lanes are the p' index,
// so a thread of the epilogue owns n2 CONSECUTIVE channels of one token: it packs them in
// registers and writes 16-byte pieces of the packed row straight to global memory, and a warp's
// stores cover one contiguous kilobyte.  128 / LS tokens share one accumulator (LS = lanes per
// token, a power of two >= n1); in stage 1 each of them uses the image of R1^T shifted to its own
// lane range, with zero rows elsewhere.  Both factors are stored pre-multiplied by 2^10 to keep
// the lo parts out of the fp16 subnormal range; every power-of-two factor is divided out exactly.
//
// Warp roles: warp 0 lane 0 = TMA producer, warp 1 lane 0 = MMA issuer, then one group of four
// warps per accumulator slot (256 / n2 slots).  Group w handles the token groups w, w + S, ...:
// it converts D1 in place to fp16 hi/lo, and after stage 2 reduces the absmax, quantises, packs
// and stores.  While one group waits for its MMAs the others compute.  With n2 = 128 a slot has eight
// warps, two per lane quarter, each on half of the columns (more warps to issue from while others wait).
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <vector>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

constexpr float kFactorScale = 1024.0f;           // 2^10 applied to R1 and R2 in the images
constexpr int kFactorScaleLog2 = 10;
constexpr int kMaxDynSmem = 227 * 1024;
constexpr int kHalfDynSmem = 113 * 1024;        // two CTAs per SM

enum RqSite : uint32_t { RQ_X_EMPTY = 16, RQ_X_FULL, RQ_D_FREE, RQ_A2_READY, RQ_D1_FULL, RQ_D2_FULL, RQ_IMG };

// Byte offset of element (row r, k) inside a K-major tile with 128-byte rows and 128-byte swizzle.
inline size_t sw128_offset(int r, int k) { return static_cast<size_t>(r) * 128 + ((((k >> 3) ^ (r & 7))) << 4) + (k & 7) * 2; }

struct RqLayout {
  int LS, G, N1, KA1, XQ, S, XS, rowsA;
  int a1_tile, a1_part, a1_bytes, b2_tile, b2_part, b2_bytes, x_tile, x_token, x_bytes;
  int off_a1, off_b2, off_x, off_misc, total;
};

__host__ __device__ inline RqLayout rq_layout(int n1, int n2, int budget = kMaxDynSmem) {
  RqLayout L;
  L.LS = n1 <= 32 ? 32 : (n1 <= 64 ? 64 : 128);   // TMEM lanes per token
  L.G = 128 / L.LS;                               // tokens per accumulator
  L.N1 = (n1 + 15) & ~15;                         // K of stage 1, padded to the MMA's K = 16
  L.KA1 = (L.N1 + 63) / 64;                       // 64-wide K atoms of stage 1
  L.XQ = n2 / 64;                                 // 64-wide column blocks of a token
  L.S = 256 / n2;                                 // accumulator slots
  L.rowsA = 256 - L.LS;
  L.a1_tile = L.rowsA * 128;
  L.a1_part = L.KA1 * L.a1_tile;
  L.a1_bytes = 2 * L.a1_part;
  L.b2_tile = n2 * 128;
  L.b2_part = L.XQ * L.b2_tile;
  L.b2_bytes = 2 * L.b2_part;
  L.x_tile = L.N1 * 128;
  L.x_token = L.XQ * L.x_tile;
  L.x_bytes = L.G * L.x_token;
  L.off_a1 = 0;
  L.off_b2 = L.off_a1 + L.a1_bytes;
  L.off_x = L.off_b2 + L.b2_bytes;
  const int extra = (n2 == 128) ? 2048 : 0;       // per-lane absmax swap of the eight-warp slot form
  const int room = budget - 1024 - 512 - extra - L.off_x;
  const int xs = room / L.x_bytes;
  L.XS = xs > 4 ? 4 : xs;                         // X ring depth
  L.off_misc = L.off_x + L.XS * L.x_bytes;
  L.total = L.off_misc + 512 + extra;
  return L;
}

// Shared-memory descriptor of an MN-major operand with the 128-byte swizzle: 64 elements along
// N are contiguous (one 128-byte row), 8 consecutive K rows form a 1024-byte atom, `lbo_bytes`
// separates successive groups of 64 along N.
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t smem_addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

// Untiled bulk copy global -> shared, completion counted on an mbarrier (16-byte aligned, size a
// multiple of 16).
__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gmem_src)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Eight consecutive codes -> one packed word.  u_i = floor(t_i) + 8 is taken from the low bits of
// t_i + (2^23 + 8) rounded towards -inf (no conversion instruction); the words' common high bits
// cancel in `kBias`; flipping bit 3 of every nibble turns the offset code into two's complement.
__device__ __forceinline__ uint32_t pack8_codes(const float* t) {
  constexpr uint32_t kBias = 0x4B000000u * 0x11111111u;
  uint32_t w = __float_as_uint(__fadd_rd(t[7], 8388616.0f));
#pragma unroll
  for (int i = 6; i >= 0; --i) w = w * 16u + __float_as_uint(__fadd_rd(t[i], 8388616.0f));
  return (w - kBias) ^ 0x88888888u;
}

// max |r[e]| over 32 fp32 bit patterns, as a tree (four independent chains).
__device__ __forceinline__ float absmax32(const uint32_t (&r)[32]) {
  float m[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
  for (int e = 0; e < 32; e += 8)
#pragma unroll
    for (int x = 0; x < 4; ++x)
      m[x] = fmaxf(m[x], fmaxf(fabsf(__uint_as_float(r[e + 2 * x])), fabsf(__uint_as_float(r[e + 2 * x + 1]))));
  return fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3]));
}

// The kernel's body, for CTA `cta` of `ncta` that share the token groups (the fused decode kernel of
// sq_linear_fused.cu runs it in its first CTAs, with more warps in the block than the roles below use).
template <int N2, int S, int CW = 1, bool F16OUT = false>
__device__ __forceinline__ void rotate_quant_tc_body(const CUtensorMap& tmap_x, const RqLayout& L,
                                                     const unsigned char* __restrict__ a1_img,
                                                     const unsigned char* __restrict__ b2_img, int n1, int rows,
                                                     uint8_t* __restrict__ Xq, __half* __restrict__ scales,
                                                     float* __restrict__ Zdbg, int cta, int ncta) {
  constexpr int TM_COLS = S * 2 * N2;             // 256 or 512
  constexpr int XQ = N2 / 64;
  constexpr int SLOT_COLS = 2 * N2;              // D1 (N2 columns) + D2 (N2 columns)
  // The layout comes from the host (the same rq_layout call that sized the shared memory); group
  // counts are 32-bit: the set-up is on the critical path of a decode step.
  const int n = n1 * N2;
  const int G = L.G, LS = L.LS;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* a1s = smem + L.off_a1;
  unsigned char* b2s = smem + L.off_b2;
  unsigned char* xs = smem + L.off_x;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.off_misc);
  uint64_t* x_full = bars;             // [4]
  uint64_t* x_empty = bars + 4;        // [4]
  uint64_t* d1_full = bars + 8;        // [4]
  uint64_t* a2_ready = bars + 12;      // [4]
  uint64_t* d2_full = bars + 16;       // [4]
  uint64_t* img_full = bars + 24;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 25);
  float* amax_x = reinterpret_cast<float*>(bars + 26);      // [S groups][2 parities][4 warps]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ngroups = (rows + G - 1) / G;
  const int my_groups = (ngroups > cta) ? (ngroups - cta + ncta - 1) / ncta : 0;
  const uint32_t limit = wait_limit();

  // One X tile set per token group: G tokens, XQ 64-column blocks each.
  auto load_group = [&](int i) {
    const int g = cta + i * ncta;
    const int s = i % L.XS;
    mbar_arrive_expect_tx(&x_full[s], static_cast<uint32_t>(L.x_bytes));
    for (int tk = 0; tk < G; ++tk)
      for (int a = 0; a < XQ; ++a)
        tma_load_3d(xs + s * L.x_bytes + tk * L.x_token + a * L.x_tile, &tmap_x, &x_full[s], a * 64, 0,
                    g * G + tk);
  };
  const int preload = my_groups < L.XS ? my_groups : L.XS;

  if (threadIdx.x == 0) {
    // The first loads go out before anything else is set up: the factor images (they belong to the
    // handle, so they may be fetched while the kernel before this one in the stream still runs), then,
    // once that kernel has completed (it may have produced X, and may still be reading the buffers this
    // one writes), the whole X ring.  Every store of this kernel depends on X having landed.  Only the
    // barriers the loads complete on exist at that point; nobody else touches a barrier before the
    // __syncthreads below.
    for (int b = 0; b < 4; ++b) mbar_init(&x_full[b], 1);
    mbar_init(img_full, 1);
    mbar_fence_init();
    mbar_arrive_expect_tx(img_full, static_cast<uint32_t>(L.a1_bytes + L.b2_bytes));
    for (int o = 0; o < L.a1_bytes; o += 16384)
      bulk_load_1d(a1s + o, a1_img + o, static_cast<uint32_t>(min(16384, L.a1_bytes - o)), img_full);
    for (int o = 0; o < L.b2_bytes; o += 16384)
      bulk_load_1d(b2s + o, b2_img + o, static_cast<uint32_t>(min(16384, L.b2_bytes - o)), img_full);
    griddep_wait();
    // Only now may a GEMM launched behind this kernel start: it requests its weights before it waits for
    // this kernel, and whatever precedes this kernel (sq_pack_weight, say) may have been writing them.
    griddep_launch_dependents();
    for (int i = 0; i < preload; ++i) load_group(i);
    for (int b = 0; b < 4; ++b) {
      mbar_init(&x_empty[b], 1);
      mbar_init(&d1_full[b], 1);
      mbar_init(&a2_ready[b], 4 * CW);
      mbar_init(&d2_full[b], 1);
    }
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, TM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------ producer: keeps the X ring full -------------------------------------
    if (lane == 0) {
      for (int i = preload; i < my_groups; ++i) {
        if (!mbar_wait(&x_empty[i % L.XS], ((i / L.XS) & 1) ^ 1, RQ_X_EMPTY, limit)) break;
        load_group(i);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------------------------------
    if (elect_one()) {
      // stage 1: A K-major (shared), B MN-major (bit 16); stage 2: A from TMEM, B K-major
      const uint32_t idesc1 = umma_idesc(/*c=f32*/ 1, /*a=f16*/ 0, /*b=f16*/ 0, 128, N2) | (1u << 16);
      const uint32_t idesc2 = umma_idesc(/*c=f32*/ 1, /*a=f16*/ 0, /*b=f16*/ 0, 128, N2);
      const uint64_t a1_desc0 = umma_desc_sw128(smem_u32(a1s)), b2_desc0 = umma_desc_sw128(smem_u32(b2s));
      const uint64_t x_desc0 = umma_desc_sw128_mn(smem_u32(xs), static_cast<uint32_t>(L.x_tile));
      const int ksteps1 = L.N1 / 16;                 // K = p, 16 per MMA
      bool ok = mbar_wait(img_full, 0, RQ_IMG, limit);
      auto stage1 = [&](int i) {
        const int slot = i % S, xs_i = i % L.XS;
        tc_fence_after_sync();
        const uint32_t d1 = tmem_base + slot * SLOT_COLS;
        uint32_t acc = 0;
        // descriptors differ only in their start-address field (16-byte units, no carry out of it)
        for (int tk = 0; tk < G; ++tk) {
          uint64_t bd = x_desc0 + ((xs_i * L.x_bytes + tk * L.x_token) >> 4);
          const uint64_t ad = a1_desc0 + (((128 - LS - tk * LS) * 128) >> 4);
          for (int ks = 0; ks < ksteps1; ++ks, bd += 2048 >> 4) {
            const uint64_t ah = ad + (((ks >> 2) * L.a1_tile + (ks & 3) * 32) >> 4);
            umma_f16(d1, ah, bd, idesc1, acc);                         // hi
            umma_f16(d1, ah + (L.a1_part >> 4), bd, idesc1, 1u);       // lo
            acc = 1;
          }
        }
        umma_commit(&x_empty[xs_i]);
        umma_commit(&d1_full[slot]);
      };
      auto stage2 = [&](int i) {
        const int slot = i % S;
        tc_fence_after_sync();
        const uint32_t d1 = tmem_base + slot * SLOT_COLS, d2 = d1 + N2;
#pragma unroll
        for (int j = 0; j < N2 / 16; ++j) {
          const uint64_t bh = b2_desc0 + (((j >> 2) * L.b2_tile + (j & 3) * 32) >> 4), bl = bh + (L.b2_part >> 4);
          umma_f16_ts(d2, d1 + 16 * j, bh, idesc2, j > 0 ? 1u : 0u);      // hi * hi
          umma_f16_ts(d2, d1 + 16 * j + 8, bh, idesc2, 1u);               // lo * hi
          umma_f16_ts(d2, d1 + 16 * j, bl, idesc2, 1u);                   // hi * lo
        }
        umma_commit(&d2_full[slot]);
      };
      // Whichever is ready goes: stage 1 of the next group whose X tile has landed and whose slot's D1
      // columns are free, and stage 2 of the oldest group whose operand has been converted.  D1 is free
      // as soon as stage 2 of the slot's previous group has completed (it was that stage's A operand),
      // so stage 1 of the next group runs while the previous one is still being quantised out of the D2
      // columns; D2 is not written again before the group's warps have finished reading it, because
      // they convert the next group (which is what lets its stage 2 go) only after that.
      int i1 = 0, i2 = 0;
      uint32_t idle = 0;
      while (ok && i2 < my_groups) {
        bool did = false;
        if (i1 < my_groups && i1 < i2 + S &&
            mbar_test_wait(&x_full[i1 % L.XS], (i1 / L.XS) & 1) &&
            mbar_test_wait(&d2_full[i1 % S], ((i1 / S) & 1) ^ 1)) {
          stage1(i1++);
          did = true;
        }
        if (i2 < i1 && mbar_test_wait(&a2_ready[i2 % S], (i2 / S) & 1)) {
          stage2(i2++);
          did = true;
        }
        if (did) {
          idle = 0;
        } else if (++idle > limit) {
          atomicCAS(&g_device_status, 0u, (static_cast<uint32_t>(RQ_A2_READY) << 8) | 1u);
          ok = false;
        }
      }
    }
  } else if (CW == 2 && warp < 2 + 4 * S * CW) {
    // ------------------------------ compute groups, two warps per lane quarter ---------------------
    // Eight warps per accumulator slot: warp (quarter, cp) owns columns [cp * N2/2, (cp+1) * N2/2) of
    // its lane quarter and works through them 16 at a time (the register budget of 18 warps per CTA).
    // Twice as many warps are there to issue while others wait for tensor memory or a barrier.
    constexpr int HC = N2 / 2;                     // columns per warp
    const int gi = (warp - 2) >> 2;
    const int w = gi >> 1, cp = gi & 1;
    const int quarter = warp & 3;
    const int lane_g = quarter * 32 + lane;
    const int tk = lane_g / LS, pp = lane_g % LS;
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t d1 = tmem_base + w * SLOT_COLS + lane_addr + cp * HC, d2 = d1 + N2;
    const int wpt = LS / 32;
    const int q0 = (quarter / wpt) * wpt;
    float* lane_m = reinterpret_cast<float*>(smem + L.off_misc + 512);       // [S][2][128 lanes]
    bool ok = true;
    for (int i = w; i < my_groups && ok; i += S) {
      const int g = cta + i * ncta;
      const long long token = static_cast<long long>(g) * G + tk;
      const uint32_t ph = (i / S) & 1;
      ok = mbar_wait(&d1_full[w], ph, RQ_D1_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      // The lane's scale must be the same in the two warps that share the lane: each takes the absmax of
      // its own columns and they swap through shared memory.  The barrier also keeps either from
      // overwriting a column of D1 that the other has yet to read (it reads only its own: nothing to keep).
      float m = 0.0f;
#pragma unroll
      for (int c = 0; c < HC / 16; ++c) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(d1 + 16 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 16; e += 2)
          m = fmaxf(m, fmaxf(fabsf(__uint_as_float(r[e])), fabsf(__uint_as_float(r[e + 1]))));
      }
      lane_m[(w * 2 + cp) * 128 + lane_g] = m;
      named_barrier(1 + w, 256);
      m = fmaxf(m, lane_m[(w * 2 + (cp ^ 1)) * 128 + lane_g]);
      int ebits = static_cast<int>((__float_as_uint(m) >> 23) & 0xFF);
      int k = 13 - (ebits - 127);
      if (m == 0.0f) k = 0;
      k = max(-126, min(127, k));
      const float sc = __uint_as_float(static_cast<uint32_t>(k + 127) << 23);
      const int uexp = -(k + 2 * kFactorScaleLog2) + 127;
      const float un = (uexp >= 1) ? __uint_as_float(static_cast<uint32_t>(min(uexp, 254)) << 23) : 0.0f;
#pragma unroll
      for (int c = 0; c < HC / 16; ++c) {
        uint32_t r[16], o[16];
        tmem_ld_32x32b_x16(d1 + 16 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float v0 = __uint_as_float(r[2 * e]), v1 = __uint_as_float(r[2 * e + 1]);
          const __half2 hh = __floats2half2_rn(v0 * sc, v1 * sc);
          const float2 hf = __half22float2(hh);
          o[e] = *reinterpret_cast<const uint32_t*>(&hh);
          o[8 + e] = pack_half2(fmaf(v0, sc, -hf.x), fmaf(v1, sc, -hf.y));
        }
        tmem_st_32x32b_x16(d1 + 16 * c, o);
      }
      tmem_wait_st();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&a2_ready[w]);

      ok = mbar_wait(&d2_full[w], ph, RQ_D2_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      if constexpr (F16OUT) {
        // rotation only: the rotated row leaves as fp16 (weight-only variant), nothing is quantised
        const bool live16 = (pp < n1) && (token < rows);
        __half* zrow16 = reinterpret_cast<__half*>(Xq) + token * n + pp * N2 + cp * HC;
#pragma unroll
        for (int c = 0; c < HC / 16; ++c) {
          uint32_t r[16];
          tmem_ld_32x32b_x16(d2 + 16 * c, r);
          tmem_wait_ld();
          uint4 lo, hi;
          lo.x = pack_half2(__uint_as_float(r[0]) * un, __uint_as_float(r[1]) * un);
          lo.y = pack_half2(__uint_as_float(r[2]) * un, __uint_as_float(r[3]) * un);
          lo.z = pack_half2(__uint_as_float(r[4]) * un, __uint_as_float(r[5]) * un);
          lo.w = pack_half2(__uint_as_float(r[6]) * un, __uint_as_float(r[7]) * un);
          hi.x = pack_half2(__uint_as_float(r[8]) * un, __uint_as_float(r[9]) * un);
          hi.y = pack_half2(__uint_as_float(r[10]) * un, __uint_as_float(r[11]) * un);
          hi.z = pack_half2(__uint_as_float(r[12]) * un, __uint_as_float(r[13]) * un);
          hi.w = pack_half2(__uint_as_float(r[14]) * un, __uint_as_float(r[15]) * un);
          if (live16) {
            *reinterpret_cast<uint4*>(zrow16 + 16 * c) = lo;
            *reinterpret_cast<uint4*>(zrow16 + 16 * c + 8) = hi;
          }
        }
        continue;
      }
      float zm = 0.0f;
#pragma unroll
      for (int c = 0; c < HC / 16; ++c) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(d2 + 16 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 16; e += 2)
          zm = fmaxf(zm, fmaxf(fabsf(__uint_as_float(r[e])), fabsf(__uint_as_float(r[e + 1]))));
      }
      zm *= un;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) zm = fmaxf(zm, __shfl_xor_sync(0xffffffffu, zm, o));
      float* amax_w = amax_x + (w * 2 + ph) * 8;
      if (lane == 0) amax_w[quarter * 2 + cp] = zm;
      named_barrier(1 + w, 256);
      float amax = fmaxf(amax_w[q0 * 2], amax_w[q0 * 2 + 1]);
      for (int x = 1; x < wpt; ++x) amax = fmaxf(amax, fmaxf(amax_w[(q0 + x) * 2], amax_w[(q0 + x) * 2 + 1]));
      __half delta;
      float inv;
      row_scale(amax, delta, inv);
      const float inv_un = inv * un;
      const bool live = (pp < n1) && (token < rows);
      const bool clamp = __half2float(delta) < 6.103515625e-05f;
      uint8_t* orow = Xq + token * (n / 2) + pp * (N2 / 2) + cp * (HC / 2);
      float* zrow = (Zdbg != nullptr && live) ? Zdbg + token * n + pp * N2 + cp * HC : nullptr;
#pragma unroll
      for (int c = 0; c < HC / 16; ++c) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(d2 + 16 * c, r);
        tmem_wait_ld();
        float t[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          t[e] = __fadd_rn(__fmul_rn(__uint_as_float(r[e]), inv_un), 0.5f);
          if (clamp) t[e] = fminf(fmaxf(t[e], -8.0f), 7.5f);
        }
        uint2 pk;
        pk.x = pack8_codes(t);
        pk.y = pack8_codes(t + 8);
        if (live) {
          *reinterpret_cast<uint2*>(orow + 8 * c) = pk;
          if (zrow) {
#pragma unroll
            for (int e = 0; e < 16; e += 4)
              *reinterpret_cast<float4*>(zrow + 16 * c + e) =
                  make_float4(__uint_as_float(r[e]) * un, __uint_as_float(r[e + 1]) * un,
                              __uint_as_float(r[e + 2]) * un, __uint_as_float(r[e + 3]) * un);
          }
        }
      }
      if (live && pp == 0 && cp == 0) scales[token] = delta;
    }
  } else if (CW == 1 && warp < 2 + 4 * S) {
    // ------------------------------ compute groups ------------------------------------------------
    const int w = (warp - 2) >> 2;                 // accumulator slot of this group
    const int quarter = warp & 3;                  // TMEM lane quarter this warp may touch
    const int lane_g = quarter * 32 + lane;        // accumulator lane = token-in-group * LS + p'
    const int tk = lane_g / LS, pp = lane_g % LS;
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t d1 = tmem_base + w * SLOT_COLS + lane_addr, d2 = d1 + N2;
    const int wpt = LS / 32;                       // warps that share a token
    const int q0 = (quarter / wpt) * wpt;
    bool ok = true;
    for (int i = w; i < my_groups && ok; i += S) {
      const int g = cta + i * ncta;
      const long long token = static_cast<long long>(g) * G + tk;
      const uint32_t ph = (i / S) & 1;

      // ---- D1 -> fp16 hi/lo in place, with a per-lane power-of-two scale --------------------------
      ok = mbar_wait(&d1_full[w], ph, RQ_D1_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      float m = 0.0f;
#pragma unroll
      for (int c = 0; c < N2 / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(d1 + 32 * c, r);
        tmem_wait_ld();
        m = fmaxf(m, absmax32(r));
      }
      // scale so that the lane's largest entry lands in [2^13, 2^14)
      int ebits = static_cast<int>((__float_as_uint(m) >> 23) & 0xFF);
      int k = 13 - (ebits - 127);
      if (m == 0.0f) k = 0;
      k = max(-126, min(127, k));
      const float sc = __uint_as_float(static_cast<uint32_t>(k + 127) << 23);
      // z = D2 * 2^-(k + 20): the two factor scales and the lane scale, divided out exactly
      const int uexp = -(k + 2 * kFactorScaleLog2) + 127;
      const float un = (uexp >= 1) ? __uint_as_float(static_cast<uint32_t>(min(uexp, 254)) << 23) : 0.0f;
#pragma unroll
      for (int c = 0; c < N2 / 32; ++c) {
        uint32_t r[32], o[32];
        tmem_ld_32x32b_x32(d1 + 32 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int h = 0; h < 2; ++h)                  // 16 fp32 columns -> 8 columns of hi + 8 of lo
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float v0 = __uint_as_float(r[16 * h + 2 * e]), v1 = __uint_as_float(r[16 * h + 2 * e + 1]);
            const __half2 hh = __floats2half2_rn(v0 * sc, v1 * sc);
            const float2 hf = __half22float2(hh);
            o[16 * h + e] = *reinterpret_cast<const uint32_t*>(&hh);
            o[16 * h + 8 + e] = pack_half2(fmaf(v0, sc, -hf.x), fmaf(v1, sc, -hf.y));
          }
        tmem_st_32x32b_x32(d1 + 32 * c, o);
      }
      tmem_wait_st();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&a2_ready[w]);

      // ---- D2: absmax over the token, quantise, pack, store ------------------------------------------
      ok = mbar_wait(&d2_full[w], ph, RQ_D2_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      if constexpr (F16OUT) {
        // rotation only: the rotated row leaves as fp16 (weight-only variant), nothing is quantised
        const bool live16 = (pp < n1) && (token < rows);
        __half* zrow16 = reinterpret_cast<__half*>(Xq) + token * n + pp * N2;
#pragma unroll
        for (int c = 0; c < N2 / 32; ++c) {
          uint32_t r[32];
          tmem_ld_32x32b_x32(d2 + 32 * c, r);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            uint4 v;
            v.x = pack_half2(__uint_as_float(r[e]) * un, __uint_as_float(r[e + 1]) * un);
            v.y = pack_half2(__uint_as_float(r[e + 2]) * un, __uint_as_float(r[e + 3]) * un);
            v.z = pack_half2(__uint_as_float(r[e + 4]) * un, __uint_as_float(r[e + 5]) * un);
            v.w = pack_half2(__uint_as_float(r[e + 6]) * un, __uint_as_float(r[e + 7]) * un);
            if (live16) *reinterpret_cast<uint4*>(zrow16 + 32 * c + e) = v;
          }
        }
        continue;
      }
      float zm = 0.0f;
#pragma unroll
      for (int c = 0; c < N2 / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(d2 + 32 * c, r);
        tmem_wait_ld();
        zm = fmaxf(zm, absmax32(r));
      }
      zm *= un;                                      // lanes of padding rows hold exact zeros
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) zm = fmaxf(zm, __shfl_xor_sync(0xffffffffu, zm, o));
      float* amax_w = amax_x + (w * 2 + ph) * 4;
      if (lane == 0) amax_w[quarter] = zm;
      named_barrier(1 + w, 128);
      float amax = amax_w[q0];
      for (int x = 1; x < wpt; ++x) amax = fmaxf(amax, amax_w[q0 + x]);
      __half delta;
      float inv;
      row_scale(amax, delta, inv);
      const float inv_un = inv * un;                 // exact: un is a power of two
      const bool live = (pp < n1) && (token < rows);
      // Delta >= 2^-14 (a normal fp16) bounds |z / Delta| by 7 (1 + 2^-11): no clamp is needed then.
      const bool clamp = __half2float(delta) < 6.103515625e-05f;
      uint8_t* orow = Xq + token * (n / 2) + pp * (N2 / 2);
      float* zrow = (Zdbg != nullptr && live) ? Zdbg + token * n + pp * N2 : nullptr;
#pragma unroll
      for (int c = 0; c < N2 / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(d2 + 32 * c, r);
        tmem_wait_ld();
        float t[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          t[e] = __fadd_rn(__fmul_rn(__uint_as_float(r[e]), inv_un), 0.5f);
          if (clamp) t[e] = fminf(fmaxf(t[e], -8.0f), 7.5f);
        }
        uint4 pk;
        pk.x = pack8_codes(t);
        pk.y = pack8_codes(t + 8);
        pk.z = pack8_codes(t + 16);
        pk.w = pack8_codes(t + 24);
        if (live) {
          *reinterpret_cast<uint4*>(orow + 16 * c) = pk;
          if (zrow) {
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              *reinterpret_cast<float4*>(zrow + 32 * c + e) =
                  make_float4(__uint_as_float(r[e]) * un, __uint_as_float(r[e + 1]) * un,
                              __uint_as_float(r[e + 2]) * un, __uint_as_float(r[e + 3]) * un);
          }
        }
      }
      if (live && pp == 0) scales[token] = delta;
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, TM_COLS);
  }
}

// S accumulator slots (= compute groups) per CTA.  With S * 2 * N2 = 256 TMEM columns two CTAs share
// an SM (each with its own producer and MMA issuer); with 512 a CTA has the SM to itself.
template <int N2, int S, int CW = 1, bool F16OUT = false>
__global__ void __launch_bounds__((2 + 4 * S * CW) * 32, (S * 2 * N2 <= 256) ? 2 : 1)
rotate_quant_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ RqLayout L,
                       const unsigned char* __restrict__ a1_img, const unsigned char* __restrict__ b2_img, int n1,
                       int rows, uint8_t* __restrict__ Xq, __half* __restrict__ scales, float* __restrict__ Zdbg) {
  rotate_quant_tc_body<N2, S, CW, F16OUT>(tmap_x, L, a1_img, b2_img, n1, rows, Xq, scales, Zdbg, static_cast<int>(blockIdx.x),
                              static_cast<int>(gridDim.x));
}

// ---------------------------------------------------------------------------------------------
// Host: factor images (the exact shared-memory bytes: fp16 hi/lo, 2^10 pre-scale, swizzled)
// ---------------------------------------------------------------------------------------------
void split_half(float v, __half& hi, __half& lo) {
  hi = __float2half_rn(v);
  lo = __float2half_rn(v - __half2float(hi));
}

void put_half(std::vector<unsigned char>& img, size_t off, __half h) {
  const unsigned short u = __half_as_ushort(h);
  img[off] = static_cast<unsigned char>(u & 0xFF);
  img[off + 1] = static_cast<unsigned char>(u >> 8);
}

}  // namespace

bool rotate_quant_tc_supported(int n1, int n2) {
  if (n2 != 64 && n2 != 128) return false;
  if (n1 < 1 || n1 > 128) return false;
  return rq_layout(n1, n2).XS >= 2;
}

// Builds and uploads the two images for a handle.  Returns false on a CUDA failure.
bool rotate_quant_tc_prepare(sq_rotation* h) {
  const int n1 = h->n1, n2 = h->n2;
  const RqLayout L = rq_layout(n1, n2);
  std::vector<unsigned char> a1(L.a1_bytes, 0), b2(L.b2_bytes, 0);
  // A1 (stage-1 A operand): rows = lanes, K = p.  R1^T sits at rows [128 - LS, 128 - LS + n1) of a
  // (256 - LS)-row image; token slot g reads it from row (128 - LS) - g * LS on, which puts R1^T
  // on lanes [g * LS, g * LS + n1) and zero rows on every other lane.
  for (int pp = 0; pp < n1; ++pp)
    for (int p = 0; p < n1; ++p) {
      __half hi, lo;
      split_half(kFactorScale * h->R1[static_cast<size_t>(p) * n1 + pp], hi, lo);
      const size_t off = static_cast<size_t>(p / 64) * L.a1_tile + sw128_offset(128 - L.LS + pp, p % 64);
      put_half(a1, off, hi);
      put_half(a1, static_cast<size_t>(L.a1_part) + off, lo);
    }
  // B2 (stage-2 B operand): rows q', K = q, value 2^10 * R2[q][q']
  for (int qp = 0; qp < n2; ++qp)
    for (int q = 0; q < n2; ++q) {
      __half hi, lo;
      split_half(kFactorScale * h->R2[static_cast<size_t>(q) * n2 + qp], hi, lo);
      const size_t off = static_cast<size_t>(q / 64) * L.b2_tile + sw128_offset(qp, q % 64);
      put_half(b2, off, hi);
      put_half(b2, static_cast<size_t>(L.b2_part) + off, lo);
    }
  if (cudaMalloc(&h->dA1img, a1.size()) != cudaSuccess || cudaMalloc(&h->dB2img, b2.size()) != cudaSuccess ||
      cudaMemcpy(h->dA1img, a1.data(), a1.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(h->dB2img, b2.data(), b2.size(), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  h->tc_ready = true;
  return true;
}

sq_status_t launch_rotate_quant_tc(const sq_rotation* h, const void* X, int64_t rows, void* Xq, void* scales,
                                   float* Zdbg, cudaStream_t s, bool f16out) {
  const int n1 = h->n1, n2 = h->n2;
  if (rows > 0x7FFFFFFF) return SQ_ERR_UNSUPPORTED;   // the kernel counts token groups in 32 bits
  // n2 = 64 with images small enough: two CTAs per SM, two accumulator slots each.
  const RqLayout Lh = rq_layout(n1, n2, kHalfDynSmem);
  const bool dual = (n2 == 64) && Lh.XS >= 2;
  const RqLayout L = dual ? Lh : rq_layout(n1, n2);
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return SQ_ERR_CUDA;
  CUtensorMap mx;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(n2), static_cast<cuuint64_t>(n1), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(n2) * 2, static_cast<cuuint64_t>(n1) * n2 * 2};
  const cuuint32_t box[3] = {64, static_cast<cuuint32_t>(L.N1), 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (enc(&mx, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(X), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return SQ_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const long long ngroups = (rows + L.G - 1) / L.G;
  const unsigned char* a1 = static_cast<const unsigned char*>(h->dA1img);
  const unsigned char* b2 = static_cast<const unsigned char*>(h->dB2img);
  auto launch = [&](auto kern, int slots, int ctas_per_sm, int cw = 1) -> bool {
    // A CTA that wants all of TMEM asks for more than half of the shared memory, so that it is alone.
    const int smem = ctas_per_sm == 1 ? std::max(L.total + 1024, 120 * 1024) : L.total + 1024;
    if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) return false;
    const unsigned grid = static_cast<unsigned>(std::min<long long>(ngroups, static_cast<long long>(sms) * ctas_per_sm));
    return launch_dependent(kern, dim3(grid), dim3((2 + 4 * slots * cw) * 32), static_cast<size_t>(smem), s, mx, L, a1, b2, n1,
                            static_cast<int>(rows), static_cast<uint8_t*>(Xq), static_cast<__half*>(scales),
                            Zdbg) == cudaSuccess;
  };
  bool ok;
  // n2 = 128 (one CTA per SM, two slots): eight warps per slot, 18 in all instead of 10 -- measured 10 %
  // faster on 4096 x 8192 (39.7 -> 35.5 us) and 0.8 us on the decode batches (6.6 -> 5.8 us).  With n2 = 64
  // and two CTAs per SM the same split leaves 56 registers per thread and was slower (12.0 -> 15.9 us).
  if (f16out) {
    // rotation only: Xq receives the rotated rows as fp16 [rows x n], `scales` is not touched
    if (n2 == 64 && dual) ok = launch(rotate_quant_tc_kernel<64, 2, 1, true>, 2, 2);
    else if (n2 == 64) ok = launch(rotate_quant_tc_kernel<64, 4, 1, true>, 4, 1);
    else ok = launch(rotate_quant_tc_kernel<128, 2, 2, true>, 2, 1, 2);
  } else if (n2 == 64 && dual) ok = launch(rotate_quant_tc_kernel<64, 2>, 2, 2);
  else if (n2 == 64) ok = launch(rotate_quant_tc_kernel<64, 4>, 4, 1);
  else ok = launch(rotate_quant_tc_kernel<128, 2, 2>, 2, 1, 2);
  if (!ok) return SQ_ERR_CUDA;
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace sq
