// Steps 1+2 on the tensor cores (sm_100a): Z_t = R1^T X~_t R2 (Eq. "eq18"), per-token absmax,
// INT4 quantisation (Section 3.2) and packing, one fused kernel.
//
// Both small contractions run as tcgen05.mma kind::f16 with fp32 accumulation in TMEM, with the
// operands split so that the result keeps fp32 accuracy:
//   stage 1  D1[q'][p]  = sum_q R2[q][q'] X~[p][q]          A = R2^T (shared memory, fp16 hi + lo),
//                                                            B = X~   (TMA tile, exact fp16)
//   stage 2  D2[q'][p'] = sum_p D1[q'][p]  R1[p][p']        A = D1   (TMEM, fp16 hi + lo, per-lane
//                                                                     power-of-two scale),
//                                                            B = R1^T (shared memory, fp16 hi + lo)
// (hi*hi + lo*hi + hi*lo; the lo*lo term is below fp32 resolution).  Lanes of TMEM are the q'
// index, so 128 / n2 tokens share one accumulator; their R2^T blocks sit on disjoint lane ranges.
// Both factors are stored pre-multiplied by 2^10 to keep the lo parts out of the fp16 subnormal
// range; every power-of-two factor is divided out exactly in the epilogue.
//
// Warp roles: warp 0 lane 0 = TMA producer, warp 1 lane 0 = MMA issuer, warps 2..5 and 6..9 = two
// compute groups that alternate token groups (each converts D1 in place to fp16 hi/lo, then
// reduces the absmax, quantises, packs into a shared-memory row and bulk-stores it).
#include <cuda.h>
#include <cuda_fp16.h>

#include <vector>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

constexpr int RQ_THREADS = 320;
constexpr float kFactorScale = 1024.0f;           // 2^10 applied to R1 and R2 in the images
constexpr int kFactorScaleLog2 = 10;

enum RqSite : uint32_t { RQ_X_EMPTY = 16, RQ_X_FULL, RQ_D_FREE, RQ_A2_READY, RQ_D1_FULL, RQ_D2_FULL };

__host__ __device__ inline int rq_align1024(int v) { return (v + 1023) & ~1023; }

// Byte offset of element (row r, k) inside a K-major tile with 128-byte rows and 128-byte swizzle.
inline size_t sw128_offset(int r, int k) { return static_cast<size_t>(r) * 128 + ((((k >> 3) ^ (r & 7))) << 4) + (k & 7) * 2; }

struct RqLayout {
  int a1_bytes, b2_bytes, b2_tile, x_tile, x_bytes, out_bytes;
  int off_a1, off_b2, off_x, off_out, off_misc, total;
};

__host__ __device__ inline RqLayout rq_layout(int n1, int N1, int n2) {
  RqLayout L;
  const int G = 128 / n2, XA = n2 / 64, KA2 = (N1 + 63) / 64;
  L.a1_bytes = (n2 == 64) ? 2 * 192 * 128 : 2 * 2 * 128 * 128;
  L.b2_tile = N1 * 128;
  L.b2_bytes = 2 * KA2 * L.b2_tile;
  L.x_tile = N1 * 128;
  L.x_bytes = G * XA * L.x_tile;
  L.out_bytes = rq_align1024(G * (n1 * n2 / 2));
  L.off_a1 = 0;
  L.off_b2 = L.off_a1 + L.a1_bytes;
  L.off_x = L.off_b2 + rq_align1024(L.b2_bytes);
  L.off_out = L.off_x + 2 * L.x_bytes;
  L.off_misc = L.off_out + 2 * L.out_bytes;
  L.total = L.off_misc + 256;
  return L;
}

template <int N2>
__global__ void __launch_bounds__(RQ_THREADS, 1)
rotate_quant_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const uint4* __restrict__ a1_img,
                       const uint4* __restrict__ b2_img, int n1, int N1, long long rows,
                       uint8_t* __restrict__ Xq, __half* __restrict__ scales, float* __restrict__ Zdbg) {
  constexpr int G = 128 / N2;                    // tokens per accumulator
  constexpr int XA = N2 / 64;                    // 64-wide K atoms of stage 1
  const int n = n1 * N2;
  const RqLayout L = rq_layout(n1, N1, N2);

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* a1s = smem + L.off_a1;
  unsigned char* b2s = smem + L.off_b2;
  unsigned char* xs = smem + L.off_x;
  unsigned char* outs = smem + L.off_out;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.off_misc);
  uint64_t* x_full = bars;            // [2]
  uint64_t* x_empty = bars + 2;       // [2]
  uint64_t* d1_full = bars + 4;       // [2]
  uint64_t* a2_ready = bars + 6;      // [2]
  uint64_t* d2_full = bars + 8;       // [2]
  uint64_t* d_free = bars + 10;       // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 12);
  float* amax_x = reinterpret_cast<float*>(bars + 13);      // [2 groups][4 warps]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long ngroups = (rows + G - 1) / G;
  const long long my_groups = (ngroups > blockIdx.x) ? (ngroups - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  const uint32_t limit = wait_limit();

  // ---- one-time setup: factor images into shared memory, barriers, TMEM --------------------------
  {
    uint4* dst = reinterpret_cast<uint4*>(a1s);
    for (int i = threadIdx.x; i < L.a1_bytes / 16; i += RQ_THREADS) dst[i] = __ldg(a1_img + i);
    dst = reinterpret_cast<uint4*>(b2s);
    for (int i = threadIdx.x; i < L.b2_bytes / 16; i += RQ_THREADS) dst[i] = __ldg(b2_img + i);
  }
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmap_x);
    for (int b = 0; b < 2; ++b) {
      mbar_init(&x_full[b], 1);
      mbar_init(&x_empty[b], 1);
      mbar_init(&d1_full[b], 1);
      mbar_init(&a2_ready[b], 4);
      mbar_init(&d2_full[b], 1);
      mbar_init(&d_free[b], 4);
    }
    mbar_fence_init();
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  fence_proxy_async_smem();          // the factor images were written through the generic proxy
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------ TMA producer: one X tile set per token group ------------------
    if (elect_one()) {
      for (long long i = 0; i < my_groups; ++i) {
        const long long g = blockIdx.x + i * gridDim.x;
        const int s = static_cast<int>(i & 1);
        if (!mbar_wait(&x_empty[s], ((i >> 1) & 1) ^ 1, RQ_X_EMPTY, limit)) break;
        mbar_arrive_expect_tx(&x_full[s], L.x_bytes);
        for (int tk = 0; tk < G; ++tk)
          for (int a = 0; a < XA; ++a)
            tma_load_3d(xs + s * L.x_bytes + (tk * XA + a) * L.x_tile, &tmap_x, &x_full[s], a * 64, 0,
                        static_cast<int32_t>(g * G + tk));
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------------------------------
    if (elect_one()) {
      const uint32_t idesc = umma_idesc(/*c=f32*/ 1, /*a=f16*/ 0, /*b=f16*/ 0, 128, static_cast<uint32_t>(N1));
      const uint32_t a1_addr = smem_u32(a1s), b2_addr = smem_u32(b2s), x_addr = smem_u32(xs);
      const int ksteps2 = N1 / 16;
      const int b2_lo = ((N1 + 63) / 64) * L.b2_tile;
      bool ok = true;
      auto stage1 = [&](long long i) {
        const int b = static_cast<int>(i & 1);
        const uint32_t ph = (i >> 1) & 1;
        ok = mbar_wait(&x_full[b], ph, RQ_X_FULL, limit) && mbar_wait(&d_free[b], ph ^ 1, RQ_D_FREE, limit);
        if (!ok) return;
        tc_fence_after_sync();
        const uint32_t d1 = tmem_base + b * 256;
        uint32_t acc = 0;
        for (int tk = 0; tk < G; ++tk)
          for (int a = 0; a < XA; ++a)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint32_t xb = x_addr + b * L.x_bytes + (tk * XA + a) * L.x_tile + ks * 32;
#pragma unroll
              for (int part = 0; part < 2; ++part) {
                uint32_t aa;
                if (N2 == 64) aa = a1_addr + part * (192 * 128) + (tk == 0 ? 64 * 128 : 0) + ks * 32;
                else aa = a1_addr + part * (2 * 128 * 128) + a * (128 * 128) + ks * 32;
                umma_f16(d1, umma_desc_sw128(aa), umma_desc_sw128(xb), idesc, acc);
                acc = 1;
              }
            }
        umma_commit(&x_empty[b]);
        umma_commit(&d1_full[b]);
      };
      auto stage2 = [&](long long i) {
        const int b = static_cast<int>(i & 1);
        ok = mbar_wait(&a2_ready[b], (i >> 1) & 1, RQ_A2_READY, limit);
        if (!ok) return;
        tc_fence_after_sync();
        const uint32_t d1 = tmem_base + b * 256, d2 = d1 + 128;
        for (int j = 0; j < ksteps2; ++j) {
          const uint32_t off = (j >> 2) * L.b2_tile + (j & 3) * 32;
          const uint64_t bh = umma_desc_sw128(b2_addr + off), bl = umma_desc_sw128(b2_addr + b2_lo + off);
          umma_f16_ts(d2, d1 + 16 * j, bh, idesc, j > 0 ? 1u : 0u);      // hi * hi
          umma_f16_ts(d2, d1 + 16 * j + 8, bh, idesc, 1u);               // lo * hi
          umma_f16_ts(d2, d1 + 16 * j, bl, idesc, 1u);                   // hi * lo
        }
        umma_commit(&d2_full[b]);
      };
      if (my_groups > 0) stage1(0);
      for (long long i = 0; i < my_groups && ok; ++i) {
        if (i + 1 < my_groups) stage1(i + 1);
        if (!ok) break;
        stage2(i);
      }
    }
  } else {
    // ------------------------------ compute groups ------------------------------------------------
    const int w = (warp - 2) >> 2;                 // 0 or 1: which accumulator buffer / token groups
    const int quarter = warp & 3;                  // TMEM lane quarter this warp may touch
    const int lane_g = quarter * 32 + lane;        // accumulator lane = token-in-group * N2 + q'
    const int tk = lane_g / N2, qp = lane_g % N2;
    const bool wg_leader = ((warp - 2) & 3) == 0 && lane == 0;
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    unsigned char* out = outs + w * L.out_bytes;
    float* amax_w = amax_x + w * 4;
    const int chunks = N1 / 16;
    bool ok = true;
    for (long long i = w; i < my_groups && ok; i += 2) {
      const long long g = blockIdx.x + i * gridDim.x;
      const long long token = g * G + tk;
      const uint32_t ph = (i >> 1) & 1;
      const uint32_t d1 = tmem_base + w * 256 + lane_addr, d2 = d1 + 128;

      // ---- D1 -> fp16 hi/lo in place, with a per-lane power-of-two scale --------------------------
      ok = mbar_wait(&d1_full[w], ph, RQ_D1_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      float m = 0.0f;
      for (int c = 0; c < chunks; ++c) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(d1 + 16 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 16; ++e) m = fmaxf(m, fabsf(__uint_as_float(r[e])));
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
      for (int c = 0; c < chunks; ++c) {
        uint32_t r[16], hi[8], lo[8];
        tmem_ld_32x32b_x16(d1 + 16 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float v0 = __uint_as_float(r[2 * e]) * sc, v1 = __uint_as_float(r[2 * e + 1]) * sc;
          const __half h0 = __float2half_rn(v0), h1 = __float2half_rn(v1);
          const __half l0 = __float2half_rn(v0 - __half2float(h0)), l1 = __float2half_rn(v1 - __half2float(h1));
          hi[e] = static_cast<uint32_t>(__half_as_ushort(h0)) | (static_cast<uint32_t>(__half_as_ushort(h1)) << 16);
          lo[e] = static_cast<uint32_t>(__half_as_ushort(l0)) | (static_cast<uint32_t>(__half_as_ushort(l1)) << 16);
        }
        tmem_st_32x32b_x8(d1 + 16 * c, hi);
        tmem_st_32x32b_x8(d1 + 16 * c + 8, lo);
      }
      tmem_wait_st();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&a2_ready[w]);

      // ---- D2: absmax over the token, quantise, pack -----------------------------------------------
      ok = mbar_wait(&d2_full[w], ph, RQ_D2_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      float zm = 0.0f;
      for (int c = 0; c < chunks; ++c) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(d2 + 16 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 16; ++e) zm = fmaxf(zm, fabsf(__uint_as_float(r[e])));   // padded columns are exactly 0
      }
      zm *= un;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) zm = fmaxf(zm, __shfl_xor_sync(0xffffffffu, zm, o));
      if (lane == 0) amax_w[quarter] = zm;
      if (wg_leader) tma_store_wait_read();          // the previous bulk store has finished reading `out`
      named_barrier(1 + w, 128);
      float amax;
      if (N2 == 128) amax = fmaxf(fmaxf(amax_w[0], amax_w[1]), fmaxf(amax_w[2], amax_w[3]));
      else amax = fmaxf(amax_w[quarter & 2], amax_w[(quarter & 2) + 1]);
      __half delta;
      float inv;
      row_scale(amax, delta, inv);
      const float inv_un = inv * un;                 // exact: un is a power of two
      unsigned char* orow = out + tk * (n / 2) + (qp >> 1);
      float* zrow = (Zdbg != nullptr && token < rows) ? Zdbg + token * n + qp : nullptr;
      for (int c = 0; c < chunks; ++c) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(d2 + 16 * c, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const int pp = 16 * c + e;
          const float v = __uint_as_float(r[e]);
          const int code = quant_code(v, inv_un);
          const int nb = __shfl_down_sync(0xffffffffu, code, 1);
          if (pp < n1) {
            if ((lane & 1) == 0) orow[pp * (N2 / 2)] = static_cast<unsigned char>((code & 15) | ((nb & 15) << 4));
            if (zrow) zrow[pp * N2] = v * un;
          }
        }
      }
      tc_fence_before_sync();
      fence_proxy_async_smem();                      // packed bytes -> visible to the bulk store
      named_barrier(1 + w, 128);
      if (lane == 0) mbar_arrive(&d_free[w]);
      if (qp == 0 && token < rows) scales[token] = delta;
      if (wg_leader) {
        for (int t2 = 0; t2 < G; ++t2) {
          const long long tok2 = g * G + t2;
          if (tok2 < rows) bulk_store_1d(Xq + tok2 * (n / 2), out + t2 * (n / 2), static_cast<uint32_t>(n / 2));
        }
        tma_store_commit();
      }
    }
    if (wg_leader) tma_store_wait_all();
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
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
  const int N1 = (n1 + 15) & ~15;
  if (n1 < 1 || N1 > 128) return false;
  return rq_layout(n1, N1, n2).total + 1024 <= 227 * 1024;
}

// Builds and uploads the two images for a handle.  Returns false on a CUDA failure.
bool rotate_quant_tc_prepare(sq_rotation* h) {
  const int n1 = h->n1, n2 = h->n2, N1 = (n1 + 15) & ~15;
  const RqLayout L = rq_layout(n1, N1, n2);
  std::vector<unsigned char> a1(L.a1_bytes, 0), b2(L.b2_bytes, 0);
  // A1: rows q', columns q, value 2^10 * R2[q][q']
  for (int qp = 0; qp < n2; ++qp)
    for (int q = 0; q < n2; ++q) {
      __half hi, lo;
      split_half(kFactorScale * h->R2[static_cast<size_t>(q) * n2 + qp], hi, lo);
      if (n2 == 64) {                       // [192 x 64]: zero rows, R2^T at rows 64..127, zero rows
        const size_t off = sw128_offset(64 + qp, q);
        put_half(a1, off, hi);
        put_half(a1, 192 * 128 + off, lo);
      } else {                              // two [128 x 64] atoms per part
        const size_t off = static_cast<size_t>(q / 64) * (128 * 128) + sw128_offset(qp, q % 64);
        put_half(a1, off, hi);
        put_half(a1, 2 * 128 * 128 + off, lo);
      }
    }
  // B2: rows p', columns p, value 2^10 * R1[p][p'], zero padded to N1 x (64 * atoms)
  const int KA2 = (N1 + 63) / 64;
  for (int pp = 0; pp < n1; ++pp)
    for (int p = 0; p < n1; ++p) {
      __half hi, lo;
      split_half(kFactorScale * h->R1[static_cast<size_t>(p) * n1 + pp], hi, lo);
      const size_t off = static_cast<size_t>(p / 64) * L.b2_tile + sw128_offset(pp, p % 64);
      put_half(b2, off, hi);
      put_half(b2, static_cast<size_t>(KA2) * L.b2_tile + off, lo);
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
                                   float* Zdbg, cudaStream_t s) {
  const int n1 = h->n1, n2 = h->n2, N1 = (n1 + 15) & ~15;
  const RqLayout L = rq_layout(n1, N1, n2);
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return SQ_ERR_CUDA;
  CUtensorMap mx;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(n2), static_cast<cuuint64_t>(n1), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(n2) * 2, static_cast<cuuint64_t>(n1) * n2 * 2};
  const cuuint32_t box[3] = {64, static_cast<cuuint32_t>(N1), 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (enc(&mx, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(X), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return SQ_ERR_CUDA;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SQ_ERR_CUDA;
  // More than half of an SM's shared memory, so that two CTAs (each wanting all of TMEM) never share one.
  const int smem = std::max(L.total + 1024, 120 * 1024);
  const long long G = 128 / n2, ngroups = (rows + G - 1) / G;
  const unsigned grid = static_cast<unsigned>(std::min<long long>(ngroups, sms));
  if (n2 == 64) {
    auto kern = rotate_quant_tc_kernel<64>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return SQ_ERR_CUDA;
    kern<<<grid, RQ_THREADS, smem, s>>>(mx, static_cast<const uint4*>(h->dA1img), static_cast<const uint4*>(h->dB2img),
                                        n1, N1, rows, static_cast<uint8_t*>(Xq), static_cast<__half*>(scales), Zdbg);
  } else {
    auto kern = rotate_quant_tc_kernel<128>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return SQ_ERR_CUDA;
    kern<<<grid, RQ_THREADS, smem, s>>>(mx, static_cast<const uint4*>(h->dA1img), static_cast<const uint4*>(h->dB2img),
                                        n1, N1, rows, static_cast<uint8_t*>(Xq), static_cast<__half*>(scales), Zdbg);
  }
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace sq
