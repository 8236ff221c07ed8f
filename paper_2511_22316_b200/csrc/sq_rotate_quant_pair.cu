// Steps 1+2 on the tensor cores for reshaped tokens with more than 128 rows (128 < n1 <= 256):
// the same two split-fp16 contractions as sq_rotate_quant_tc.cu, run by a CTA pair
// (tcgen05 cta_group::2, M = 256).  CTA r of the pair owns the rows p' in [128 r, 128 r + 128) of
// every token (its TMEM lanes) and therefore holds only its half of the image of R1^T, which
// would not fit into one SM's shared memory whole.  The B operands are split the way the pair
// MMA wants them: each CTA loads its half of the token's columns (stage 1, MN-major, straight
// from TMA) and holds its half of the rows of R2^T (stage 2).  One token per accumulator slot.
//
// Warp roles per CTA: warp 0 = TMA producer; warp 1 = MMA issuer in the leader CTA and a relay in
// the other (it tells the leader when its half of a tile has landed); then one group of four
// warps per accumulator slot (eight, two per lane quarter, when n2 = 128).  The per-token absmax spans both CTAs: each group reduces its 128
// lanes and swaps the result with its partner group through the other CTA's shared memory.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <vector>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

enum RqPairSite : uint32_t {
  RQP_X_EMPTY = 48, RQP_X_FULL, RQP_XP_FULL, RQP_D_FREE, RQP_A2_READY, RQP_D1_FULL, RQP_D2_FULL, RQP_IMG,
  RQP_AMAX, RQP_ISSUE
};

struct RqPairLayout {
  int N1, KA1, HQ, KA2, S, XS;
  int a1_part, a1_bytes, b2_tile, b2_part, b2_bytes, x_row, x_tile;
  int off_a1, off_b2, off_x, off_misc, total;
};

__host__ __device__ inline RqPairLayout rq_pair_layout(int n1, int n2) {
  RqPairLayout L;
  L.N1 = (n1 + 15) & ~15;                         // K of stage 1
  L.KA1 = (L.N1 + 63) / 64;
  L.HQ = n2 / 2;                                  // columns of a token held by one CTA
  L.KA2 = n2 / 64;                                // 64-wide K atoms of stage 2
  L.S = 256 / n2;
  L.a1_part = L.KA1 * 128 * 128;                  // this CTA's 128 rows of R1^T, one part (hi or lo)
  L.a1_bytes = 2 * L.a1_part;
  L.b2_tile = L.HQ * 128;                         // this CTA's n2/2 rows of R2^T, one K atom
  L.b2_part = L.KA2 * L.b2_tile;
  L.b2_bytes = 2 * L.b2_part;
  L.x_row = L.HQ * 2;                             // bytes per row of the half tile (64 or 128)
  L.x_tile = L.N1 * L.x_row;
  L.off_a1 = 0;
  L.off_b2 = L.a1_bytes;
  L.off_x = L.off_b2 + L.b2_bytes;
  const int extra = (n2 == 128) ? 2048 : 0;       // per-lane absmax swap of the eight-warp slot form
  const int room = kMaxDynSmem - 1024 - 1024 - extra - L.off_x;
  const int xs = room / L.x_tile;
  L.XS = xs > 4 ? 4 : xs;
  L.off_misc = L.off_x + L.XS * L.x_tile;
  L.total = L.off_misc + 1024 + extra;
  return L;
}

// MN-major operand descriptor for 128-byte (layout 2) or 64-byte (layout 4) swizzled rows: the
// rows are K, 8 of them form an atom, `sbo_bytes` separates atoms along K.
__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t smem_addr, uint32_t sbo_bytes, uint32_t layout) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;                                  // one group along N: unused
  d |= static_cast<uint64_t>(sbo_bytes >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(layout) << 61;
  return d;
}

template <int N2, int CW, bool F16OUT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__((2 + 4 * CW * (256 / N2)) * 32, 1)
rotate_quant_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const unsigned char* __restrict__ a1_img,
                         const unsigned char* __restrict__ b2_img, int n1, long long rows,
                         uint8_t* __restrict__ Xq, __half* __restrict__ scales, float* __restrict__ Zdbg) {
  constexpr int S = 256 / N2;
  constexpr int SLOT_COLS = 2 * N2;
  const RqPairLayout L = rq_pair_layout(n1, N2);
  const int n = n1 * N2;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* a1s = smem + L.off_a1;
  unsigned char* b2s = smem + L.off_b2;
  unsigned char* xs = smem + L.off_x;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.off_misc);
  uint64_t* x_full = bars;             // [4] this CTA's half tile has landed (local)
  uint64_t* x_empty = bars + 4;        // [4] stage-1 MMAs retired (each CTA's own copy)
  uint64_t* xp_full = bars + 8;        // [4] the partner's half tile has landed (leader's copy is used)
  uint64_t* d1_full = bars + 12;       // [4] each CTA's own copy
  uint64_t* a2_ready = bars + 16;      // [4] 8 warps of the pair (leader's copy is used)
  uint64_t* d2_full = bars + 20;       // [4] each CTA's own copy
  uint64_t* amax_bar = bars + 28;      // [4] the partner group's absmax has arrived (local)
  uint64_t* img_full = bars + 32;      // this CTA's factor images (local)
  uint64_t* peer_img = bars + 33;      // the partner's factor images (leader's copy is used)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 34);
  float* amax_x = reinterpret_cast<float*>(bars + 35);      // [S][2 parities][4 warps]
  float* amax_peer = amax_x + 32;                           // [S][2 parities], written by the partner

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const long long pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const long long my_tokens = (rows > pair) ? (rows - pair + npairs - 1) / npairs : 0;
  const uint32_t limit = wait_limit();

  auto load_token = [&](long long i) {
    const long long t = pair + i * npairs;
    const int s = static_cast<int>(i % L.XS);
    mbar_arrive_expect_tx(&x_full[s], static_cast<uint32_t>(L.x_tile));
    tma_load_3d(xs + s * L.x_tile, &tmap_x, &x_full[s], static_cast<int32_t>(rank) * L.HQ, 0, static_cast<int32_t>(t));
  };
  const long long preload = my_tokens < L.XS ? my_tokens : L.XS;

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmap_x);
    for (int b = 0; b < 4; ++b) {
      mbar_init(&x_full[b], 1);
      mbar_init(&x_empty[b], 1);
      mbar_init(&xp_full[b], 1);
      mbar_init(&d1_full[b], 1);
      mbar_init(&a2_ready[b], 8 * CW);
      mbar_init(&d2_full[b], 1);
      mbar_init(&amax_bar[b], 1);
    }
    mbar_init(img_full, 1);
    mbar_init(peer_img, 1);
    mbar_fence_init();
    // The factor images belong to the handle: fetched at once.  X may come from the kernel before this
    // one in the stream, which may also still read the buffers this kernel writes: its completion is
    // awaited before the first token is requested (every store here depends on a token having landed).
    mbar_arrive_expect_tx(img_full, static_cast<uint32_t>(L.a1_bytes + L.b2_bytes));
    const unsigned char* a1g = a1_img + static_cast<size_t>(rank) * L.a1_bytes;
    const unsigned char* b2g = b2_img + static_cast<size_t>(rank) * L.b2_bytes;
    for (int o = 0; o < L.a1_bytes; o += 16384)
      bulk_load_1d(a1s + o, a1g + o, static_cast<uint32_t>(min(16384, L.a1_bytes - o)), img_full);
    for (int o = 0; o < L.b2_bytes; o += 16384)
      bulk_load_1d(b2s + o, b2g + o, static_cast<uint32_t>(min(16384, L.b2_bytes - o)), img_full);
    griddep_wait();
    // only now may a GEMM launched behind this kernel start (it requests its weights before it waits for
    // this kernel, and this kernel's predecessor may have been writing them)
    griddep_launch_dependents();
    for (long long i = 0; i < preload; ++i) load_token(i);
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();                   // both CTAs' barriers exist before any remote arrival
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------ producer: keeps this CTA's half of the X ring full --------------
    if (lane == 0) {
      for (long long i = preload; i < my_tokens; ++i) {
        if (!mbar_wait(&x_empty[i % L.XS], ((i / L.XS) & 1) ^ 1, RQP_X_EMPTY, limit)) break;
        load_token(i);
      }
    }
  } else if (warp == 1) {
    if (rank != 0) {
      // ------------------------------ relay: tells the leader what has landed here ------------------
      if (lane == 0) {
        bool ok = mbar_wait(img_full, 0, RQP_IMG, limit);
        if (ok) mbar_arrive_cluster(peer_img, 0);
        for (long long i = 0; i < my_tokens && ok; ++i) {
          ok = mbar_wait(&x_full[i % L.XS], (i / L.XS) & 1, RQP_X_FULL, limit);
          if (ok) mbar_arrive_cluster(&xp_full[i % L.XS], 0);
        }
      }
    } else if (elect_one()) {
      // ------------------------------ MMA issuer (leader CTA) ----------------------------------------
      const uint32_t idesc1 = umma_idesc(/*c=f32*/ 1, /*a=f16*/ 0, /*b=f16*/ 0, 256, N2) | (1u << 16);
      const uint32_t idesc2 = umma_idesc(/*c=f32*/ 1, /*a=f16*/ 0, /*b=f16*/ 0, 256, N2);
      const uint64_t a1_desc0 = umma_desc_sw128(smem_u32(a1s)), b2_desc0 = umma_desc_sw128(smem_u32(b2s));
      const uint64_t x_desc0 = umma_desc_mn(smem_u32(xs), 8u * L.x_row, N2 == 128 ? 2u : 4u);
      const int ksteps1 = L.N1 / 16;
      bool ok = mbar_wait(img_full, 0, RQP_IMG, limit) && mbar_wait(peer_img, 0, RQP_IMG, limit);
      auto stage1 = [&](long long i) {
        const int slot = static_cast<int>(i % S), xs_i = static_cast<int>(i % L.XS);
        tc_fence_after_sync();
        const uint32_t d1 = tmem_base + slot * SLOT_COLS;
        uint64_t bd = x_desc0 + ((xs_i * L.x_tile) >> 4);
        for (int ks = 0; ks < ksteps1; ++ks, bd += (16 * L.x_row) >> 4) {
          const uint64_t ah = a1_desc0 + (((ks >> 2) * (128 * 128) + (ks & 3) * 32) >> 4);
          umma_f16_pair(d1, ah, bd, idesc1, ks > 0 ? 1u : 0u);           // hi
          umma_f16_pair(d1, ah + (L.a1_part >> 4), bd, idesc1, 1u);      // lo
        }
        umma_commit_pair_mc(&x_empty[xs_i], 3);
        umma_commit_pair_mc(&d1_full[slot], 3);
      };
      auto stage2 = [&](long long i) {
        const int slot = static_cast<int>(i % S);
        tc_fence_after_sync();
        const uint32_t d1 = tmem_base + slot * SLOT_COLS, d2 = d1 + N2;
#pragma unroll
        for (int j = 0; j < N2 / 16; ++j) {
          const uint64_t bh = b2_desc0 + (((j >> 2) * L.b2_tile + (j & 3) * 32) >> 4), bl = bh + (L.b2_part >> 4);
          umma_f16_ts_pair(d2, d1 + 16 * j, bh, idesc2, j > 0 ? 1u : 0u);      // hi * hi
          umma_f16_ts_pair(d2, d1 + 16 * j + 8, bh, idesc2, 1u);               // lo * hi
          umma_f16_ts_pair(d2, d1 + 16 * j, bl, idesc2, 1u);                   // hi * lo
        }
        umma_commit_pair_mc(&d2_full[slot], 3);
      };
      long long i1 = 0, i2 = 0;
      uint32_t idle = 0;
      while (ok && i2 < my_tokens) {
        bool did = false;
        if (i1 < my_tokens && i1 < i2 + S &&
            mbar_test_wait(&x_full[i1 % L.XS], (i1 / L.XS) & 1) &&
            mbar_test_wait(&xp_full[i1 % L.XS], (i1 / L.XS) & 1) &&
            mbar_test_wait(&d2_full[i1 % S], ((i1 / S) & 1) ^ 1)) {   // D1 free: the slot's previous stage 2 is done
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
          atomicCAS(&g_device_status, 0u, (static_cast<uint32_t>(RQP_ISSUE) << 8) | 1u);
          ok = false;
        }
      }
    }
  } else if (CW == 2) {
    // ------------------------------ compute groups, two warps per lane quarter ---------------------
    // Eight warps per accumulator slot: warp (quarter, cp) owns columns [cp * N2/2, (cp+1) * N2/2) of its
    // lane quarter, 16 at a time; the lane's scale is the larger of the two halves' (swapped through
    // shared memory behind the group barrier, which also orders the reads of D1 before its overwrite).
    constexpr int HC = N2 / 2;
    const int gi = (warp - 2) >> 2;
    const int w = gi >> 1, cp = gi & 1;
    const int quarter = warp & 3;
    const int lane_g = quarter * 32 + lane;
    const int pp = static_cast<int>(rank) * 128 + lane_g;
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t d1 = tmem_base + w * SLOT_COLS + lane_addr + cp * HC, d2 = d1 + N2;
    const bool live = pp < n1;
    float* lane_m = reinterpret_cast<float*>(smem + L.off_misc + 1024);       // [S][2][128 lanes]
    bool ok = true;
    for (long long i = w; i < my_tokens && ok; i += S) {
      const long long token = pair + i * npairs;
      const uint32_t ph = (i / S) & 1;
      ok = mbar_wait(&d1_full[w], ph, RQP_D1_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
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
      if (lane == 0) mbar_arrive_cluster(&a2_ready[w], 0);

      ok = mbar_wait(&d2_full[w], ph, RQP_D2_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      if constexpr (F16OUT) {
        // rotation only: the rotated row leaves as fp16 (weight-only variant), nothing is quantised
        __half* zrow16 = reinterpret_cast<__half*>(Xq) + token * n + static_cast<long long>(pp) * N2 + cp * HC;
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
          if (live) {
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
      float amax = fmaxf(fmaxf(fmaxf(amax_w[0], amax_w[1]), fmaxf(amax_w[2], amax_w[3])),
                         fmaxf(fmaxf(amax_w[4], amax_w[5]), fmaxf(amax_w[6], amax_w[7])));
      if (lane_g == 0 && cp == 0) st_f32_peer_and_arrive(&amax_peer[w * 2 + ph], amax, &amax_bar[w], rank ^ 1u);
      ok = mbar_wait_acq_cluster(&amax_bar[w], ph, RQP_AMAX, limit);
      if (!ok) break;
      amax = fmaxf(amax, amax_peer[w * 2 + ph]);
      __half delta;
      float inv;
      row_scale(amax, delta, inv);
      const float inv_un = inv * un;
      const bool clamp = __half2float(delta) < 6.103515625e-05f;
      uint8_t* orow = Xq + token * (n / 2) + static_cast<long long>(pp) * (N2 / 2) + cp * (HC / 2);
      float* zrow = (Zdbg != nullptr && live) ? Zdbg + token * n + static_cast<long long>(pp) * N2 + cp * HC : nullptr;
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
      if (pp == 0 && cp == 0) scales[token] = delta;
    }
  } else {
    // ------------------------------ compute groups ------------------------------------------------
    const int w = (warp - 2) >> 2;                 // accumulator slot of this group
    const int quarter = warp & 3;
    const int lane_g = quarter * 32 + lane;        // TMEM lane
    const int pp = static_cast<int>(rank) * 128 + lane_g;    // row p' of the reshaped token
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t d1 = tmem_base + w * SLOT_COLS + lane_addr, d2 = d1 + N2;
    const bool live = pp < n1;
    bool ok = true;
    for (long long i = w; i < my_tokens && ok; i += S) {
      const long long token = pair + i * npairs;
      const uint32_t ph = (i / S) & 1;

      // ---- D1 -> fp16 hi/lo in place, with a per-lane power-of-two scale --------------------------
      ok = mbar_wait(&d1_full[w], ph, RQP_D1_FULL, limit);
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
      int ebits = static_cast<int>((__float_as_uint(m) >> 23) & 0xFF);
      int k = 13 - (ebits - 127);                  // the lane's largest entry lands in [2^13, 2^14)
      if (m == 0.0f) k = 0;
      k = max(-126, min(127, k));
      const float sc = __uint_as_float(static_cast<uint32_t>(k + 127) << 23);
      const int uexp = -(k + 2 * kFactorScaleLog2) + 127;
      const float un = (uexp >= 1) ? __uint_as_float(static_cast<uint32_t>(min(uexp, 254)) << 23) : 0.0f;
#pragma unroll
      for (int c = 0; c < N2 / 32; ++c) {
        uint32_t r[32], o[32];
        tmem_ld_32x32b_x32(d1 + 32 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int h = 0; h < 2; ++h)
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
      if (lane == 0) mbar_arrive_cluster(&a2_ready[w], 0);

      // ---- D2: absmax over the token (both CTAs), quantise, pack, store --------------------------
      ok = mbar_wait(&d2_full[w], ph, RQP_D2_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      if constexpr (F16OUT) {
        // rotation only: the rotated row leaves as fp16 (weight-only variant), nothing is quantised
        __half* zrow16 = reinterpret_cast<__half*>(Xq) + token * n + static_cast<long long>(pp) * N2;
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
            if (live) *reinterpret_cast<uint4*>(zrow16 + 32 * c + e) = v;
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
      float amax = fmaxf(fmaxf(amax_w[0], amax_w[1]), fmaxf(amax_w[2], amax_w[3]));
      if (lane_g == 0) st_f32_peer_and_arrive(&amax_peer[w * 2 + ph], amax, &amax_bar[w], rank ^ 1u);
      ok = mbar_wait_acq_cluster(&amax_bar[w], ph, RQP_AMAX, limit);
      if (!ok) break;
      amax = fmaxf(amax, amax_peer[w * 2 + ph]);
      __half delta;
      float inv;
      row_scale(amax, delta, inv);
      const float inv_un = inv * un;
      const bool clamp = __half2float(delta) < 6.103515625e-05f;   // see sq_rotate_quant_tc.cu
      uint8_t* orow = Xq + token * (n / 2) + static_cast<long long>(pp) * (N2 / 2);
      float* zrow = (Zdbg != nullptr && live) ? Zdbg + token * n + static_cast<long long>(pp) * N2 : nullptr;
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
      if (pp == 0) scales[token] = delta;
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

}  // namespace

bool rotate_quant_pair_supported(int n1, int n2) {
  if (n2 != 64 && n2 != 128) return false;
  if (n1 <= 128 || n1 > 256) return false;
  return rq_pair_layout(n1, n2).XS >= 2;
}

// Builds and uploads the images of both CTAs of the pair.  Returns false on a CUDA failure.
bool rotate_quant_pair_prepare(sq_rotation* h) {
  const int n1 = h->n1, n2 = h->n2;
  const RqPairLayout L = rq_pair_layout(n1, n2);
  std::vector<unsigned char> a1(2 * static_cast<size_t>(L.a1_bytes), 0), b2(2 * static_cast<size_t>(L.b2_bytes), 0);
  // A1 of CTA r: row l = p' - 128 r, K = p, value 2^10 * R1[p][p']
  for (int pp = 0; pp < n1; ++pp)
    for (int p = 0; p < n1; ++p) {
      __half hi, lo;
      split_half(kFactorScale * h->R1[static_cast<size_t>(p) * n1 + pp], hi, lo);
      const size_t base = static_cast<size_t>(pp / 128) * L.a1_bytes;
      const size_t off = static_cast<size_t>(p / 64) * (128 * 128) + sw128_offset(pp % 128, p % 64);
      put_half(a1, base + off, hi);
      put_half(a1, base + L.a1_part + off, lo);
    }
  // B2 of CTA r: row j = q' - r * n2/2, K = q, value 2^10 * R2[q][q']
  for (int qp = 0; qp < n2; ++qp)
    for (int q = 0; q < n2; ++q) {
      __half hi, lo;
      split_half(kFactorScale * h->R2[static_cast<size_t>(q) * n2 + qp], hi, lo);
      const size_t base = static_cast<size_t>(qp / L.HQ) * L.b2_bytes;
      const size_t off = static_cast<size_t>(q / 64) * L.b2_tile + sw128_offset(qp % L.HQ, q % 64);
      put_half(b2, base + off, hi);
      put_half(b2, base + L.b2_part + off, lo);
    }
  if (cudaMalloc(&h->dA1img, a1.size()) != cudaSuccess || cudaMalloc(&h->dB2img, b2.size()) != cudaSuccess ||
      cudaMemcpy(h->dA1img, a1.data(), a1.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(h->dB2img, b2.data(), b2.size(), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  h->tc_pair = true;
  return true;
}

sq_status_t launch_rotate_quant_pair(const sq_rotation* h, const void* X, int64_t rows, void* Xq, void* scales,
                                     float* Zdbg, cudaStream_t s, bool f16out) {
  const int n1 = h->n1, n2 = h->n2;
  const RqPairLayout L = rq_pair_layout(n1, n2);
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return SQ_ERR_CUDA;
  CUtensorMap mx;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(n2), static_cast<cuuint64_t>(n1), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(n2) * 2, static_cast<cuuint64_t>(n1) * n2 * 2};
  const cuuint32_t box[3] = {static_cast<cuuint32_t>(L.HQ), static_cast<cuuint32_t>(L.N1), 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (enc(&mx, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(X), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, n2 == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return SQ_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const int smem = L.total + 1024;
  const long long pairs = std::min<long long>(rows, sms / 2);
  const unsigned grid = static_cast<unsigned>(2 * pairs);
  const unsigned char* a1 = static_cast<const unsigned char*>(h->dA1img);
  const unsigned char* b2 = static_cast<const unsigned char*>(h->dB2img);
  if (n2 == 64) {
    auto kern = f16out ? rotate_quant_pair_kernel<64, 1, true> : rotate_quant_pair_kernel<64, 1, false>;
    if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) return SQ_ERR_CUDA;
    if (launch_dependent(kern, dim3(grid), dim3((2 + 4 * 4) * 32), static_cast<size_t>(smem), s, mx, a1, b2, n1, rows,
                         static_cast<uint8_t*>(Xq), static_cast<__half*>(scales), Zdbg) != cudaSuccess)
      return SQ_ERR_CUDA;
  } else {
    // two slots of eight warps (18 warps in the CTA instead of 10)
    auto kern = f16out ? rotate_quant_pair_kernel<128, 2, true> : rotate_quant_pair_kernel<128, 2, false>;
    if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) return SQ_ERR_CUDA;
    if (launch_dependent(kern, dim3(grid), dim3((2 + 4 * 2 * 2) * 32), static_cast<size_t>(smem), s, mx, a1, b2, n1, rows,
                         static_cast<uint8_t*>(Xq), static_cast<__half*>(scales), Zdbg) != cudaSuccess)
      return SQ_ERR_CUDA;
  }
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace sq
