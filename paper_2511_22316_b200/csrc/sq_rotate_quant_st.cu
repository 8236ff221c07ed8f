// Steps 1+2 with R2 applied through its structure (sm_100a): Z_t = R1^T X~_t R2 (Eq. "eq18") with
// R2 = H R2^U, R2^U = R_map R'_map^T (paragraphs "Uniformity Rotation Transformation" and "The
// Overall SingleQuant Method"), then the per-token absmax, INT4 quantisation (Section 3.2) and packing.
//
// Only R1^T, which holds the dense random block of ART, is a dense contraction: it runs as
// tcgen05.mma kind::f16 with the factor split into fp16 hi + lo and fp32 accumulation in TMEM,
// exactly as stage 1 of the dense kernel (sq_rotate_quant_tc.cu).  TMEM lanes are the p' index, so
// afterwards one thread owns the n2 consecutive channels (p', 0 .. n2-1) of one token, and R2 acts
// on exactly those: the thread applies it in registers, in fp32, piece by piece --
//   x H          the Sylvester Hadamard matrix as log2(n2) levels of butterflies;
//   . R_map      the chain of n2-1 plane rotations on adjacent coordinates that takes v to ||v|| e_1.
//                Written out, row k >= 1 of the product is a_k x_{k-1} + b_k S_k with the suffix sums
//                S_k = sum_{j >= k} v_j x_j, and row 0 is S_0 / ||v||.  The kernel keeps the rows
//                unscaled, y~_k = S_k + (a_k / b_k) x_{k-1} (two multiply-adds per element, only the
//                running sum is a dependent chain), and b_k goes into the next set of coefficients;
//   . R'_map^T   the transposed chain for the target u: z_j = u_j Q_j + a'_{j+1} y_{j+1} with the prefix
//                sums Q_j = y_0 / ||u|| + sum_{1 <= k <= j} g_k y_k (three per element).
// The coefficients come from v and u in float64 (st_coefficients below); the 1/sqrt(n2) of H and the
// 2^10 pre-scale of the R1 image are folded into the last set.  No second MMA stage, no conversion of
// the intermediate to fp16, one TMEM read per element.
//
// Warp roles: warp 0 lane 0 = TMA producer (ring of X tiles), warp 1 lane 0 = MMA issuer (one
// accumulator slot of n2 columns per token group, 512 / n2 slots, so the tensor cores run ahead of the
// arithmetic), then NG groups of four warps; group g takes the token groups g, g + NG, ...: it reads
// its slot into registers, hands the slot back, and computes, quantises and stores from registers.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

enum StSite : uint32_t { ST_X_EMPTY = 32, ST_X_FULL, ST_D_FREE, ST_D_FULL, ST_IMG };

constexpr int kStMaxRing = 6;          // X ring stages (barrier arrays are sized for it)
constexpr int kStSlots = 4;            // accumulator slots of 128 TMEM columns

// Coefficients of the structured R2, read by the kernel as immediate constant-bank operands.
template <int N2>
struct StCoef {
  float sv[N2];    // v_k: S_k = sum_{j >= k} v_j x_j
  float rho[N2];   // k >= 1: y~_k = S_k + rho_k x_{k-1} (last row: x_{N2-1} in place of S_k);  rho[0] unused
  float uu[N2];    // c0 u_j
  float a2[N2];    // k >= 1: c0 x coefficient of y~_k in z_{k-1};   a2[0]: Q_0 = a2[0] y~_0
  float g2[N2];    // 1 <= k <= N2-2: coefficient of y~_k in Q_k;   g2[N2-1]: c0 x coefficient of y~_{N2-1} in z_{N2-1}
  float c0;        // 2^-10 (the image's pre-scale) x 1/sqrt(n2) when H is present
};

// An accumulator slot is 128 TMEM columns wide, so that every MMA has N = 128 (an MMA of N = 64 costs
// the issuing thread as much as one of N = 128 and the tensor pipe three quarters of it).  Its lanes
// hold G = 128 / LS tokens side by side (LS = lanes per token, a power of two >= n1); its columns
// hold CH = 128 / n2 tokens side by side: one "super-group" is TPS = G * CH consecutive tokens.
struct StLayout {
  int LS, G, CH, TPS, N1, KA1, XS;
  int a1_tile, a1_part, a1_bytes, x_tile, x_half, x_bytes;
  int off_a1, off_x, off_misc, total;
};

inline StLayout st_layout(int n1, int n2) {
  StLayout L;
  L.LS = n1 <= 32 ? 32 : (n1 <= 64 ? 64 : 128);
  L.G = 128 / L.LS;
  L.CH = 128 / n2;
  L.TPS = L.G * L.CH;
  L.N1 = (n1 + 15) & ~15;                         // K of the contraction, padded to the MMA's K = 16
  L.KA1 = (L.N1 + 63) / 64;
  L.a1_tile = (256 - L.LS) * 128;
  L.a1_part = L.KA1 * L.a1_tile;
  L.a1_bytes = 2 * L.a1_part;
  L.x_tile = L.N1 * 128;                          // one token's rows x 64 columns
  L.x_half = L.G * L.x_tile;                      // one 64-column group of the slot: G tokens
  L.x_bytes = 2 * L.x_half;                       // one ring stage: both 64-column groups
  L.off_a1 = 0;
  L.off_x = L.a1_bytes;
  const int room = kMaxDynSmem - 1024 - 4096 - L.off_x;
  const int xs = room / L.x_bytes;
  L.XS = xs > kStMaxRing ? kStMaxRing : xs;
  L.off_misc = L.off_x + L.XS * L.x_bytes;
  L.total = L.off_misc + 4096;                    // barriers, TMEM address, absmax exchange, coefficients
  return L;
}

// A 64-bit MMA descriptor from its constant high word and a low word (start address + LBO fields).
__device__ __forceinline__ uint64_t desc_from(uint32_t hi, uint32_t lo) {
  return (static_cast<uint64_t>(hi) << 32) | lo;
}

template <int N2, int NG, bool HAD, bool URT>
__global__ void __launch_bounds__((2 + 4 * NG) * 32, 1)
rotate_quant_st_kernel(const __grid_constant__ StLayout L, int n1, int rows, const unsigned char* __restrict__ a1_img,
                       uint8_t* __restrict__ Xq, __half* __restrict__ scales, float* __restrict__ Zdbg,
                       const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ StCoef<N2> cf) {
  constexpr int NS = kStSlots;
  constexpr int CH = 128 / N2;                    // tokens side by side in a slot's columns
  const int n = n1 * N2;
  const int G = L.G, LS = L.LS;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* a1s = smem + L.off_a1;
  unsigned char* xs = smem + L.off_x;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.off_misc);
  uint64_t* x_full = bars;                        // [8]
  uint64_t* x_empty = bars + 8;                   // [8]
  uint64_t* d_full = bars + 16;                   // [4]
  uint64_t* d_free = bars + 20;                   // [4]
  uint64_t* img_full = bars + 24;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 25);
  float* amax_x = reinterpret_cast<float*>(bars + 26);      // [NG groups][2 parities][4 warps]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Work item = the G tokens of one 64-column group (n2 = 64) or of one slot (n2 = 128).  The items are
  // dealt out in contiguous, nearly equal runs: CTA b takes the items [i0, i0 + cnt); CH consecutive
  // items of a run share a slot (a super-group); a run's last super-group may be half filled.
  const int nitems = (rows + G - 1) / G;
  const int per = nitems / static_cast<int>(gridDim.x), extra = nitems % static_cast<int>(gridDim.x);
  const int b = static_cast<int>(blockIdx.x);
  const int i0 = b * per + (b < extra ? b : extra), cnt = per + (b < extra ? 1 : 0);
  const int my_sg = (cnt + CH - 1) / CH;
  const uint32_t limit = wait_limit();

  // One ring stage per super-group: two boxes of 64 columns x N1 rows x G tokens.  n2 = 64: the boxes are
  // the super-group's two items (the second one may not belong to this CTA: then it is not loaded, and
  // what the MMAs make of the stale bytes lands in columns nobody reads); n2 = 128: they are the two
  // column halves of the one item.
  auto load_sg = [&](int k) {
    const int it0 = i0 + k * CH;
    const int s = k % L.XS;
    unsigned char* dst = xs + s * L.x_bytes;
    const bool both = (CH == 1) || (it0 + 1 < i0 + cnt);
    mbar_arrive_expect_tx(&x_full[s], static_cast<uint32_t>(both ? L.x_bytes : L.x_half));
    tma_load_3d(dst, &tmap_x, &x_full[s], 0, 0, it0 * G);
    if (CH == 1) tma_load_3d(dst + L.x_half, &tmap_x, &x_full[s], 64, 0, it0 * G);
    else if (both) tma_load_3d(dst + L.x_half, &tmap_x, &x_full[s], 0, 0, (it0 + 1) * G);
  };
  // The first two stages are requested at once; the rest of the ring follows when the first has landed,
  // so that every SM's first tokens are not queued behind everybody's later ones.
  const int preload = my_sg < 2 ? my_sg : 2;

  if (warp == 0) {
    // Every lane sets up "its" barriers, then the loads go out at once: the factor image first (it
    // gates the first MMA and comes from L2), then one ring stage per lane.
    if (lane < 8) {
      mbar_init(&x_full[lane], 1);
      mbar_init(&x_empty[lane], 1);
    }
    if (lane < NS) {
      mbar_init(&d_full[lane], 1);
      mbar_init(&d_free[lane], 4 * CH);
    }
    if (lane == 0) mbar_init(img_full, 1);
    mbar_fence_init();
    __syncwarp();
    if (lane == 0) {
      tma_prefetch_desc(&tmap_x);
      mbar_arrive_expect_tx(img_full, static_cast<uint32_t>(L.a1_bytes));
      for (int o = 0; o < L.a1_bytes; o += 16384)
        bulk_load_1d(a1s + o, a1_img + o, static_cast<uint32_t>(min(16384, L.a1_bytes - o)), img_full);
    }
    __syncwarp();
    // X may come from the kernel before this one in the stream, which may also still read the buffers
    // this kernel writes: its completion is awaited before the first tokens are requested (every store
    // of this kernel depends on tokens having landed; the image above belongs to the handle).
    if (lane < preload || lane == 0) {
      griddep_wait();
      // only now may a GEMM launched behind this kernel start (it requests its weights before it waits
      // for this kernel, and this kernel's predecessor may have been writing them)
      if (lane == 0) griddep_launch_dependents();
      if (lane < preload) load_sg(lane);
    }
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------ producer: keeps the X ring full -------------------------------------
    if (lane == 0 && my_sg > preload) {
      bool ok = mbar_wait(&x_full[0], 0, ST_X_FULL, limit);
      for (int i = preload; i < my_sg && ok; ++i) {
        if (i >= L.XS) ok = mbar_wait(&x_empty[i % L.XS], ((i / L.XS) & 1) ^ 1, ST_X_EMPTY, limit);
        if (ok) load_sg(i);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer: D[p'][q] = sum_p R1[p][p'] X~[p][q] --------------------
    if (elect_one()) {
      // A K-major (shared: the image of R1^T shifted to the token's lanes), B MN-major (bit 16): the
      // tokens' TMA tiles as they landed, two 64-column groups x_half apart.  Descriptors of one
      // super-group differ only in the start-address field of their low word (no carry out of it).
      constexpr uint32_t idesc1 = umma_idesc(/*c=f32*/ 1, /*a=f16*/ 0, /*b=f16*/ 0, 128, 128) | (1u << 16);
      const uint64_t a1_desc0 = umma_desc_sw128(smem_u32(a1s));
      const uint64_t x_desc0 = umma_desc_sw128_mn(smem_u32(xs), static_cast<uint32_t>(L.x_half));
      const uint32_t a_hi = static_cast<uint32_t>(a1_desc0 >> 32), b_hi = static_cast<uint32_t>(x_desc0 >> 32);
      const uint32_t a_lo0 = static_cast<uint32_t>(a1_desc0), b_lo0 = static_cast<uint32_t>(x_desc0);
      const uint32_t lo_part = static_cast<uint32_t>(L.a1_part >> 4), a_tile = static_cast<uint32_t>(L.a1_tile >> 4);
      const int ksteps1 = L.N1 / 16;
      bool ok = mbar_wait(img_full, 0, ST_IMG, limit);
      int slot = 0, xs_i = 0;
      uint32_t xph = 0, dph = 1;                  // phases: X stage "full", slot "free" (free at first)
      for (int i = 0; i < my_sg && ok; ++i) {
        ok = mbar_wait(&x_full[xs_i], xph, ST_X_FULL, limit) && mbar_wait(&d_free[slot], dph, ST_D_FREE, limit);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t d = tmem_base + slot * 128;
        uint32_t acc = 0;
        for (int tk = 0; tk < G; ++tk) {
          uint32_t b_lo = b_lo0 + static_cast<uint32_t>((xs_i * L.x_bytes + tk * L.x_tile) >> 4);
          uint32_t a_lo = a_lo0 + static_cast<uint32_t>(((128 - LS - tk * LS) * 128) >> 4);
          for (int k4 = 0; k4 < ksteps1; k4 += 4, a_lo += a_tile) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              if (k4 + kk < ksteps1) {
                umma_f16(d, desc_from(a_hi, a_lo + 2 * kk), desc_from(b_hi, b_lo), idesc1, acc);             // hi
                umma_f16(d, desc_from(a_hi, a_lo + 2 * kk + lo_part), desc_from(b_hi, b_lo), idesc1, 1u);   // lo
                acc = 1;
                b_lo += 2048 >> 4;
              }
            }
          }
        }
        umma_commit(&x_empty[xs_i]);
        umma_commit(&d_full[slot]);
        if (++xs_i == L.XS) { xs_i = 0; xph ^= 1; }
        if (++slot == NS) { slot = 0; dph ^= 1; }
      }
    }
  } else {
    // ------------------------------ compute groups ------------------------------------------------
    // Work item j = (super-group j / CH, 64-column group j % CH of its slot when n2 = 64): the rows
    // (p', all q) of G tokens, one row per thread.  Group w takes the items w, w + NG, ...
    const int w = (warp - 2) >> 2;                 // group
    const int quarter = warp & 3;                  // TMEM lane quarter this warp may touch
    const int lane_g = quarter * 32 + lane;        // accumulator lane = token-in-group * LS + p'
    const int tk = lane_g / LS, pp = lane_g % LS;
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    const int wpt = LS / 32;                       // warps that share a token
    const int q0 = (quarter / wpt) * wpt;
    uint32_t it = 0;
    for (int j = w; j < cnt; j += NG, ++it) {
      const int sg = j / CH, c = j % CH;
      const int slot = sg % NS;
      const long long token = static_cast<long long>(i0 + j) * G + tk;
      if (!mbar_wait(&d_full[slot], (sg / NS) & 1, ST_D_FULL, limit)) break;
      tc_fence_after_sync();
      float x[N2];
      {
        const uint32_t d = tmem_base + slot * 128 + c * N2 + lane_addr;
        uint32_t r[N2 / 32][32];
#pragma unroll
        for (int b = 0; b < N2 / 32; ++b) tmem_ld_32x32b_x32(d + 32 * b, r[b]);
        tmem_wait_ld();
#pragma unroll
        for (int b = 0; b < N2 / 32; ++b)
#pragma unroll
          for (int e = 0; e < 32; ++e) x[32 * b + e] = __uint_as_float(r[b][e]);
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&d_free[slot]);   // this warp's part of the slot is in registers

      // ---- x H: butterflies ---------------------------------------------------------------------------
      if (HAD) {
#pragma unroll
        for (int len = 1; len < N2; len <<= 1)
#pragma unroll
          for (int b = 0; b < N2; b += 2 * len)
#pragma unroll
            for (int e = b; e < b + len; ++e) {
              const float lo = x[e], hi = x[e + len];
              x[e] = lo + hi;
              x[e + len] = lo - hi;
            }
      }
      if (URT) {
        // ---- . R_map: suffix sums S_k, unscaled rows y~_k from the last one down ----------------------
        float S = cf.sv[N2 - 1] * x[N2 - 1];
        x[N2 - 1] = fmaf(cf.rho[N2 - 1], x[N2 - 2], x[N2 - 1]);
#pragma unroll
        for (int k = N2 - 2; k >= 1; --k) {
          S = fmaf(cf.sv[k], x[k], S);
          x[k] = fmaf(cf.rho[k], x[k - 1], S);
        }
        x[0] = fmaf(cf.sv[0], x[0], S);
        // ---- . R'_map^T: prefix sums Q_j, rows from the first one up -----------------------------------
        float Q = x[0] * cf.a2[0];
#pragma unroll
        for (int e = 0; e < N2 - 2; ++e) {
          const float y = x[e + 1];
          x[e] = fmaf(cf.uu[e], Q, cf.a2[e + 1] * y);
          Q = fmaf(cf.g2[e + 1], y, Q);
        }
        const float yl = x[N2 - 1];
        x[N2 - 2] = fmaf(cf.uu[N2 - 2], Q, cf.a2[N2 - 1] * yl);
        x[N2 - 1] = fmaf(cf.uu[N2 - 1], Q, cf.g2[N2 - 1] * yl);
      } else {
#pragma unroll
        for (int e = 0; e < N2; ++e) x[e] *= cf.c0;
      }

      // ---- absmax over the token, quantise, pack, store ----------------------------------------------
      float m4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
      for (int b = 0; b < N2; b += 4)
#pragma unroll
        for (int e = 0; e < 4; ++e) m4[e] = fmaxf(m4[e], fabsf(x[b + e]));
      float zm = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));   // lanes of padding rows hold exact zeros
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) zm = fmaxf(zm, __shfl_xor_sync(0xffffffffu, zm, o));
      float amax = zm;
      if (wpt > 1) {
        float* amax_w = amax_x + (w * 2 + (it & 1)) * 4;
        if (lane == 0) amax_w[quarter] = zm;
        named_barrier(1 + w, 128);
        amax = amax_w[q0];
        for (int e = 1; e < wpt; ++e) amax = fmaxf(amax, amax_w[q0 + e]);
      }
      __half delta;
      float inv;
      row_scale(amax, delta, inv);
      const bool live = (pp < n1) && (token < rows);
      // Delta >= 2^-14 (a normal fp16) bounds |z / Delta| by 7 (1 + 2^-11): no clamp is needed then.
      const bool clamp = __half2float(delta) < 6.103515625e-05f;
      uint8_t* orow = Xq + token * (n / 2) + pp * (N2 / 2);
      float* zrow = (Zdbg != nullptr && live) ? Zdbg + token * n + pp * N2 : nullptr;
      if (zrow) {
#pragma unroll
        for (int e = 0; e < N2; e += 4) *reinterpret_cast<float4*>(zrow + e) = make_float4(x[e], x[e + 1], x[e + 2], x[e + 3]);
      }
#pragma unroll
      for (int b = 0; b < N2 / 32; ++b) {
        float t[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          t[e] = __fadd_rn(__fmul_rn(x[32 * b + e], inv), 0.5f);
          if (clamp) t[e] = fminf(fmaxf(t[e], -8.0f), 7.5f);
        }
        uint4 pk;
        pk.x = pack8_codes(t);
        pk.y = pack8_codes(t + 8);
        pk.z = pack8_codes(t + 16);
        pk.w = pack8_codes(t + 24);
        if (live) *reinterpret_cast<uint4*>(orow + 16 * b) = pk;
      }
      if (live && pp == 0) scales[token] = delta;
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------------
// Host: coefficients of the two chains (float64 -> fp32) and the launch
// ---------------------------------------------------------------------------------------------
// h[k] (k = 1 .. n-1) = the value the chain of plane rotations leaves at position k-1 after the step
// on the plane (k-1, k): h[n-1] = hypot(v[n-2], v[n-1]), h[k] = hypot(v[k-1], h[k+1]); h[1] = ||v||.
std::vector<double> chain_norms(const std::vector<double>& v) {
  const int n = static_cast<int>(v.size());
  std::vector<double> h(n + 1, 0.0);
  double w = v[n - 1];
  for (int k = n - 1; k >= 1; --k) {
    h[k] = std::hypot(v[k - 1], w);
    w = h[k];
  }
  return h;
}

// Fills the coefficient block; returns false when the closed forms would divide by zero (a vanishing
// partial norm of a chain, or an entry of v that is zero where a row is scaled by it): such a handle
// keeps the dense kernels.
template <int N2>
bool st_coefficients(const R2Structure& s2, StCoef<N2>& cf) {
  const int n = N2;
  const double c0 = std::ldexp(1.0, -kFactorScaleLog2) * (s2.hadamard ? 1.0 / std::sqrt(static_cast<double>(n)) : 1.0);
  std::memset(&cf, 0, sizeof(cf));
  cf.c0 = static_cast<float>(c0);
  if (!s2.urt) return true;
  if (static_cast<int>(s2.v.size()) != n || static_cast<int>(s2.u.size()) != n) return false;
  const std::vector<double>&v = s2.v, &u = s2.u;
  const std::vector<double> h = chain_norms(v), g = chain_norms(u);
  for (int k = 1; k <= n - 1; ++k)
    if (!(h[k] > 1e-18 * h[1]) || !(g[k] > 1e-18 * g[1])) return false;
  if (!(h[1] > 1e-18 && h[1] < 1e18 && g[1] > 1e-18 && g[1] < 1e18)) return false;
  // Row k of x R_map is a_k x_{k-1} + b_k S_k (k <= n-2), b_{n-1} x_{n-1} + a_{n-1} x_{n-2} (the chain's
  // first step works on the untouched last coordinate), S_0 / h_1 for k = 0.  The kernel computes
  // y~_k = S_k + (a_k / b_k) x_{k-1} and the factor sc_k = b_k multiplies the coefficients of y_k below.
  std::vector<double> sc(n), rho(n, 0.0);
  sc[0] = 1.0 / h[1];
  for (int k = 1; k <= n - 2; ++k) {
    const double a = -h[k + 1] / h[k], bk = v[k - 1] / (h[k + 1] * h[k]);
    sc[k] = bk;
    rho[k] = a / bk;
  }
  sc[n - 1] = v[n - 2] / h[n - 1];
  rho[n - 1] = (-v[n - 1] / h[n - 1]) / sc[n - 1];
  for (int k = 1; k <= n - 1; ++k)
    if (!(std::fabs(sc[k]) > 1e-20 / h[1]) || !std::isfinite(rho[k]) || std::fabs(rho[k]) > 1e30) return false;
  // z_j = u_j Q_j + a'_{j+1} y_{j+1}, Q_j = Q_{j-1} + g_j y_j, Q_0 = y_0 / g_1norm; the last two rows use the
  // untouched last coordinate of u.  All of c0 goes into u_j and a'.
  for (int k = 0; k < n; ++k) {
    cf.sv[k] = static_cast<float>(v[k]);
    cf.rho[k] = static_cast<float>(rho[k]);
    cf.uu[k] = static_cast<float>(c0 * u[k]);
  }
  cf.a2[0] = static_cast<float>(sc[0] / g[1]);
  for (int k = 1; k <= n - 2; ++k) {
    cf.a2[k] = static_cast<float>(c0 * (-g[k + 1] / g[k]) * sc[k]);
    cf.g2[k] = static_cast<float>(u[k - 1] / (g[k] * g[k + 1]) * sc[k]);
  }
  cf.a2[n - 1] = static_cast<float>(c0 * (-u[n - 1] / g[n - 1]) * sc[n - 1]);
  cf.g2[n - 1] = static_cast<float>(c0 * (u[n - 2] / g[n - 1]) * sc[n - 1]);
  for (int k = 0; k < n; ++k) {
    const float all[5] = {cf.sv[k], cf.rho[k], cf.uu[k], cf.a2[k], cf.g2[k]};
    for (float f : all)
      if (!std::isfinite(f)) return false;
  }
  return true;
}

template <int N2, int NG>
sq_status_t launch_st(const sq_rotation* h, const StLayout& L, const CUtensorMap& mx, const void* X, int rows, void* Xq,
                      void* scales, float* Zdbg, cudaStream_t s) {
  StCoef<N2> cf;
  if (h->st_coef.size() * sizeof(float) != sizeof(cf)) return SQ_ERR_INVALID_ARG;
  std::memcpy(&cf, h->st_coef.data(), sizeof(cf));
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  // one CTA per SM, but no CTA with less than one full slot of tokens
  const long long nsg = (static_cast<long long>(rows) + L.TPS - 1) / L.TPS;
  const unsigned grid = static_cast<unsigned>(std::min<long long>(nsg, sms));
  const int smem = L.total + 1024;
  const unsigned char* a1 = static_cast<const unsigned char*>(h->dA1img);
  auto go = [&](auto kern) -> sq_status_t {
    if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) return SQ_ERR_CUDA;
    const cudaError_t err = launch_dependent(kern, dim3(grid), dim3((2 + 4 * NG) * 32), static_cast<size_t>(smem), s, L,
                                             h->n1, rows, a1, static_cast<uint8_t*>(Xq), static_cast<__half*>(scales),
                                             Zdbg, mx, cf);
    count_launch();
    return err == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
  };
  const bool had = h->s2.hadamard, urt = h->s2.urt;
  if (had && urt) return go(rotate_quant_st_kernel<N2, NG, true, true>);
  if (had) return go(rotate_quant_st_kernel<N2, NG, true, false>);
  if (urt) return go(rotate_quant_st_kernel<N2, NG, false, true>);
  return go(rotate_quant_st_kernel<N2, NG, false, false>);
}

}  // namespace

// The handle must already hold the R1^T image of the dense kernel (rotate_quant_tc_prepare).
bool rotate_quant_st_prepare(sq_rotation* h) {
  h->st_ready = false;
  if (!h->s2.known || !h->tc_ready || h->dA1img == nullptr) return true;
  if (h->n2 != 64 && h->n2 != 128) return true;
  if (st_layout(h->n1, h->n2).XS < 2) return true;
  bool ok;
  if (h->n2 == 64) {
    StCoef<64> cf;
    ok = st_coefficients<64>(h->s2, cf);
    if (ok) h->st_coef.assign(reinterpret_cast<const float*>(&cf), reinterpret_cast<const float*>(&cf) + sizeof(cf) / 4);
  } else {
    StCoef<128> cf;
    ok = st_coefficients<128>(h->s2, cf);
    if (ok) h->st_coef.assign(reinterpret_cast<const float*>(&cf), reinterpret_cast<const float*>(&cf) + sizeof(cf) / 4);
  }
  h->st_ready = ok;
  return true;
}

sq_status_t launch_rotate_quant_st(const sq_rotation* h, const void* X, int64_t rows, void* Xq, void* scales,
                                   float* Zdbg, cudaStream_t s) {
  const int n1 = h->n1, n2 = h->n2;
  if (rows > 0x7FFFFFFF) return SQ_ERR_UNSUPPORTED;   // the kernel counts token groups in 32 bits
  const StLayout L = st_layout(n1, n2);
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return SQ_ERR_CUDA;
  CUtensorMap mx;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(n2), static_cast<cuuint64_t>(n1), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(n2) * 2, static_cast<cuuint64_t>(n1) * n2 * 2};
  const cuuint32_t box[3] = {64, static_cast<cuuint32_t>(L.N1), static_cast<cuuint32_t>(L.G)};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (enc(&mx, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(X), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return SQ_ERR_CUDA;
  if (n2 == 64) return launch_st<64, 3>(h, L, mx, X, static_cast<int>(rows), Xq, scales, Zdbg, s);
  return launch_st<128, 2>(h, L, mx, X, static_cast<int>(rows), Xq, scales, Zdbg, s);
}

}  // namespace sq
