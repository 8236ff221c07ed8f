// Steps 1+2 of the hot path, fused: Kronecker rotation of each row, per-row absmax, INT4
// quantisation and nibble packing (Eq. "eq18"; Section 3.2 for Q_Delta).
//
// Generic fp32 kernel: one CTA owns one row at a time.  The row (n = n1*n2 halves) is staged in
// shared memory, T = X~ R2 is formed in shared memory, Z = R1^T T is formed in registers (each
// thread keeps its 4x4 tiles until the row's absmax is known), then quantised and stored.
// The rotated row never touches HBM unless the debug output is requested.
#include <cuda_fp16.h>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

constexpr int TP = 4;   // tile rows (p or p')
constexpr int TQ = 4;   // tile columns (q')

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide maximum; `red` holds one float per warp.  All threads get the result.
__device__ __forceinline__ float block_max(float v, float* red) {
  v = warp_max(v);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = (blockDim.x + 31) >> 5;
  __syncthreads();                 // protects `red` against the previous use
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float r = (lane < nwarps) ? red[lane] : 0.0f;
  r = warp_max(r);
  return r;
}

// The quantiser's decision, in fp32 and in this order of operations:
//   Delta = fp16(amax / 7); inv = 1 / Delta; code = floor(fl(fl(z * inv) + 0.5)) clamped to [-8, 7].
// With b bits the 7 becomes qmax = 2^(b-1) - 1 and the clamp [-qmax - 1, qmax] (weight-only variant).
__device__ __forceinline__ int quant_code(float z, float inv, int qmax = 7) {
  const float t = __fadd_rn(__fmul_rn(z, inv), 0.5f);
  int c = static_cast<int>(floorf(t));
  return max(-qmax - 1, min(qmax, c));
}

__device__ __forceinline__ void row_scale(float amax, __half& delta, float& inv, int qmax = 7) {
  delta = __float2half_rn(__fdiv_rn(amax, static_cast<float>(qmax)));
  const float d = __half2float(delta);
  inv = (d > 0.0f) ? __fdiv_rn(1.0f, d) : 0.0f;
}

// `qmax` = 7 for INT4.  F16OUT: rotation only, Xq then receives the rotated rows as fp16 [rows x n]
// and `scales` is not touched (weight-only variant); a separate instantiation, so that the quantising
// kernel's code is what it was without it (as a run-time branch it cost that kernel half of its speed:
// the compiler stopped software-pipelining its two product loops).
template <int MAXT, bool VEC, bool F16OUT>
__global__ void __launch_bounds__(512)
rotate_quant_kernel(const float* __restrict__ R1, const float* __restrict__ R2, int n1, int n2,
                    const __half* __restrict__ X, long long rows, uint8_t* __restrict__ Xq,
                    __half* __restrict__ scales, float* __restrict__ Zdbg, int qmax) {
  griddep_wait();                    // X may come from the kernel before this one in the stream
  griddep_launch_dependents();       // a GEMM launched behind this kernel may set itself up from here on
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n = n1 * n2;
  float* Ts = reinterpret_cast<float*>(smem_raw);                       // [n1][n2] fp32
  __half* Xs = reinterpret_cast<__half*>(smem_raw + sizeof(float) * n);  // [n1][n2] fp16
  float* red = reinterpret_cast<float*>(smem_raw + sizeof(float) * n + ((sizeof(__half) * n + 15) & ~size_t(15)));

  const int tiles_q = (n2 + TQ - 1) / TQ;
  const int tiles_p = (n1 + TP - 1) / TP;
  const int ntiles = tiles_p * tiles_q;
  const int tid = threadIdx.x, nthr = blockDim.x;

  for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
    // ---- stage the row -------------------------------------------------------------------
    const __half* xrow = X + row * n;
    if ((n & 7) == 0) {
      const uint4* src = reinterpret_cast<const uint4*>(xrow);
      uint4* dst = reinterpret_cast<uint4*>(Xs);
      for (int i = tid; i < n / 8; i += nthr) dst[i] = __ldg(src + i);
    } else {
      for (int i = tid; i < n; i += nthr) Xs[i] = xrow[i];
    }
    __syncthreads();

    // ---- T = X~ R2 : T[p][q'] = sum_q X~[p][q] R2[q][q'] --------------------------------
    for (int tile = tid; tile < ntiles; tile += nthr) {
      const int p0 = (tile / tiles_q) * TP, q0 = (tile % tiles_q) * TQ;
      float acc[TP][TQ];
#pragma unroll
      for (int i = 0; i < TP; ++i)
#pragma unroll
        for (int j = 0; j < TQ; ++j) acc[i][j] = 0.0f;
      for (int q = 0; q < n2; ++q) {
        float r[TQ];
        if (VEC) {
          const float4 v = __ldg(reinterpret_cast<const float4*>(R2 + (size_t)q * n2 + q0));
          r[0] = v.x; r[1] = v.y; r[2] = v.z; r[3] = v.w;
        } else {
#pragma unroll
          for (int j = 0; j < TQ; ++j) r[j] = (q0 + j < n2) ? __ldg(R2 + (size_t)q * n2 + q0 + j) : 0.0f;
        }
#pragma unroll
        for (int i = 0; i < TP; ++i) {
          const float x = (VEC || p0 + i < n1) ? __half2float(Xs[(p0 + i) * n2 + q]) : 0.0f;
#pragma unroll
          for (int j = 0; j < TQ; ++j) acc[i][j] = fmaf(x, r[j], acc[i][j]);
        }
      }
#pragma unroll
      for (int i = 0; i < TP; ++i) {
        if (VEC) {
          *reinterpret_cast<float4*>(Ts + (p0 + i) * n2 + q0) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        } else if (p0 + i < n1) {
#pragma unroll
          for (int j = 0; j < TQ; ++j)
            if (q0 + j < n2) Ts[(p0 + i) * n2 + q0 + j] = acc[i][j];
        }
      }
    }
    __syncthreads();

    // ---- Z = R1^T T : Z[p'][q'] = sum_p R1[p][p'] T[p][q'] ; kept in registers -------------
    float z[MAXT][TP][TQ];
    float amax = 0.0f;
#pragma unroll
    for (int t = 0; t < MAXT; ++t) {
      const int tile = tid + t * nthr;
#pragma unroll
      for (int i = 0; i < TP; ++i)
#pragma unroll
        for (int j = 0; j < TQ; ++j) z[t][i][j] = 0.0f;
      if (tile < ntiles) {
        const int p0 = (tile / tiles_q) * TP, q0 = (tile % tiles_q) * TQ;
        for (int p = 0; p < n1; ++p) {
          float a[TP], b[TQ];
          if (VEC) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(R1 + (size_t)p * n1 + p0));
            a[0] = v.x; a[1] = v.y; a[2] = v.z; a[3] = v.w;
            const float4 w = *reinterpret_cast<const float4*>(Ts + p * n2 + q0);
            b[0] = w.x; b[1] = w.y; b[2] = w.z; b[3] = w.w;
          } else {
#pragma unroll
            for (int i = 0; i < TP; ++i) a[i] = (p0 + i < n1) ? __ldg(R1 + (size_t)p * n1 + p0 + i) : 0.0f;
#pragma unroll
            for (int j = 0; j < TQ; ++j) b[j] = (q0 + j < n2) ? Ts[p * n2 + q0 + j] : 0.0f;
          }
#pragma unroll
          for (int i = 0; i < TP; ++i)
#pragma unroll
            for (int j = 0; j < TQ; ++j) z[t][i][j] = fmaf(a[i], b[j], z[t][i][j]);
        }
#pragma unroll
        for (int i = 0; i < TP; ++i)
#pragma unroll
          for (int j = 0; j < TQ; ++j) amax = fmaxf(amax, fabsf(z[t][i][j]));   // padded entries are 0
      }
    }
    if constexpr (F16OUT) {
      // ---- rotation only: the row leaves as fp16 ---------------------------------------------------
      __half* zrow16 = reinterpret_cast<__half*>(Xq) + row * (long long)n;
#pragma unroll
      for (int t = 0; t < MAXT; ++t) {
        const int tile = tid + t * nthr;
        if (tile < ntiles) {
          const int p0 = (tile / tiles_q) * TP, q0 = (tile % tiles_q) * TQ;
#pragma unroll
          for (int i = 0; i < TP; ++i) {
            if (!VEC && p0 + i >= n1) continue;
            const int c0 = (p0 + i) * n2 + q0;
#pragma unroll
            for (int j = 0; j < TQ; ++j)
              if (VEC || q0 + j < n2) zrow16[c0 + j] = __float2half_rn(z[t][i][j]);
          }
        }
      }
      __syncthreads();
      continue;
    }
    amax = block_max(amax, red);

    // ---- quantise, pack, store ---------------------------------------------------------------
    __half delta;
    float inv;
    row_scale(amax, delta, inv, qmax);
    if (tid == 0) scales[row] = delta;
    uint8_t* qrow = Xq + row * (long long)(n / 2);
#pragma unroll
    for (int t = 0; t < MAXT; ++t) {
      const int tile = tid + t * nthr;
      if (tile < ntiles) {
        const int p0 = (tile / tiles_q) * TP, q0 = (tile % tiles_q) * TQ;
#pragma unroll
        for (int i = 0; i < TP; ++i) {
          if (!VEC && p0 + i >= n1) continue;
          const int c0 = (p0 + i) * n2 + q0;     // even: n2 is even and q0 is a multiple of 4
          const int k0 = quant_code(z[t][i][0], inv, qmax), k1 = quant_code(z[t][i][1], inv, qmax);
          const int k2 = quant_code(z[t][i][2], inv, qmax), k3 = quant_code(z[t][i][3], inv, qmax);
          const uint8_t b0 = static_cast<uint8_t>((k0 & 15) | ((k1 & 15) << 4));
          const uint8_t b1 = static_cast<uint8_t>((k2 & 15) | ((k3 & 15) << 4));
          if (VEC) {
            *reinterpret_cast<uint16_t*>(qrow + c0 / 2) = static_cast<uint16_t>(b0 | (b1 << 8));
          } else {
            if (q0 + 1 < n2) qrow[c0 / 2] = b0;
            if (q0 + 3 < n2) qrow[c0 / 2 + 1] = b1;
          }
          if (Zdbg != nullptr) {
            float* zr = Zdbg + row * (long long)n + c0;
            if (VEC) {
              *reinterpret_cast<float4*>(zr) = make_float4(z[t][i][0], z[t][i][1], z[t][i][2], z[t][i][3]);
            } else {
#pragma unroll
              for (int j = 0; j < TQ; ++j)
                if (q0 + j < n2) zr[j] = z[t][i][j];
            }
          }
        }
      }
    }
    __syncthreads();    // Xs/Ts are rewritten by the next row
  }
}

// Identity rotation: quantise the fp16 rows as they are (used by sq_pack_weight with no handle).
__global__ void __launch_bounds__(256)
quant_rows_kernel(const __half* __restrict__ X, long long rows, int n, uint8_t* __restrict__ Xq,
                  __half* __restrict__ scales, float* __restrict__ Zdbg, int qmax) {
  __shared__ float red[32];
  for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
    const __half* xrow = X + row * n;
    float amax = 0.0f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) amax = fmaxf(amax, fabsf(__half2float(xrow[i])));
    amax = block_max(amax, red);
    __half delta;
    float inv;
    row_scale(amax, delta, inv, qmax);
    if (threadIdx.x == 0) scales[row] = delta;
    uint8_t* qrow = Xq + row * (long long)(n / 2);
    for (int i = threadIdx.x; i < n / 2; i += blockDim.x) {
      const float z0 = __half2float(xrow[2 * i]), z1 = __half2float(xrow[2 * i + 1]);
      const int k0 = quant_code(z0, inv, qmax), k1 = quant_code(z1, inv, qmax);
      qrow[i] = static_cast<uint8_t>((k0 & 15) | ((k1 & 15) << 4));
      if (Zdbg != nullptr) {
        Zdbg[row * (long long)n + 2 * i] = z0;
        Zdbg[row * (long long)n + 2 * i + 1] = z1;
      }
    }
  }
}

template <int MAXT, bool VEC>
sq_status_t launch_generic(const float* dR1, const float* dR2, int n1, int n2, const void* X, int64_t rows,
                           void* Xq, void* scales, float* Zdbg, int threads, size_t smem, int sms,
                           cudaStream_t s, int qmax) {
  auto kern = qmax == 0 ? rotate_quant_kernel<MAXT, VEC, true> : rotate_quant_kernel<MAXT, VEC, false>;
  if (smem > 48 * 1024) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
      return SQ_ERR_CUDA;
  }
  int per_sm = 1;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem) != cudaSuccess || per_sm < 1)
    per_sm = 1;
  const long long grid = std::min<long long>(rows, static_cast<long long>(sms) * per_sm);
  kern<<<static_cast<unsigned>(grid), threads, smem, s>>>(dR1, dR2, n1, n2, static_cast<const __half*>(X), rows,
                                                         static_cast<uint8_t*>(Xq), static_cast<__half*>(scales),
                                                         Zdbg, qmax);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace

sq_status_t launch_rotate_quant(const float* dR1, const float* dR2, int n1, int n2, const void* X,
                                int64_t rows, void* Xq, void* scales, float* Zdbg, cudaStream_t s, int qmax) {
  if (rows == 0) return SQ_OK;
  const long long n = static_cast<long long>(n1) * n2;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;

  if (dR1 == nullptr || dR2 == nullptr) {
    if (qmax == 0) return SQ_ERR_INVALID_ARG;          // rotation only with no rotation: nothing to do here
    const long long grid = std::min<long long>(rows, static_cast<long long>(sms) * 8);
    quant_rows_kernel<<<static_cast<unsigned>(grid), 256, 0, s>>>(static_cast<const __half*>(X), rows,
                                                                   static_cast<int>(n), static_cast<uint8_t*>(Xq),
                                                                   static_cast<__half*>(scales), Zdbg, qmax);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
  }

  const int ntiles = ((n1 + TP - 1) / TP) * ((n2 + TQ - 1) / TQ);
  const bool vec = (n1 % 4 == 0) && (n2 % 4 == 0);
  const size_t smem = sizeof(float) * n + ((sizeof(__half) * n + 15) & ~size_t(15)) + 32 * sizeof(float);
  int threads, maxt;
  if (ntiles <= 128) { threads = 128; maxt = 1; }
  else if (ntiles <= 256) { threads = 256; maxt = 1; }
  else if (ntiles <= 512) { threads = 512; maxt = 1; }
  else if (ntiles <= 1024) { threads = 512; maxt = 2; }
  else if (ntiles <= 2048) { threads = 512; maxt = 4; }
  else return SQ_ERR_UNSUPPORTED;
  if (smem > 227 * 1024) return SQ_ERR_UNSUPPORTED;

#define SQ_DISPATCH(MT)                                                                                      \
  return vec ? launch_generic<MT, true>(dR1, dR2, n1, n2, X, rows, Xq, scales, Zdbg, threads, smem, sms, s, qmax)  \
             : launch_generic<MT, false>(dR1, dR2, n1, n2, X, rows, Xq, scales, Zdbg, threads, smem, sms, s, qmax)
  if (maxt == 1) { SQ_DISPATCH(1); }
  if (maxt == 2) { SQ_DISPATCH(2); }
  SQ_DISPATCH(4);
#undef SQ_DISPATCH
}

}  // namespace sq
