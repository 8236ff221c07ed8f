// Step 3 for one to four tokens: the INT4 x INT4 product as dot products on the CUDA cores.
//
// With M <= 4 the work is 2 M N K <= 0.5 GOP against 29 MB of packed weights: pure streaming, and
// every tensor-core arrangement pays more in pipeline hand-overs and MMA issue than the whole
// read costs.  Here each warp takes two weight rows at a time, every lane reads 16-byte pieces of
// them straight from global memory (coalesced, several in flight), widens the nibbles to
// 16 x code in the top of each byte -- the same trick as the tensor-core kernels, so the dp4a
// accumulator holds 256 x acc and the shift at the end is exact -- and multiplies them with the
// tokens' codes, widened the same way once per CTA into shared memory.  No workspace, no split K:
// a row's sum is completed by one warp (shuffle reduction), so the result is deterministic.
#include <cuda_fp16.h>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

constexpr int GV_UNROLL = 4;          // 16-byte pieces of each row in flight per lane
// Weight rows per warp task: four for one or two tokens (more bytes in flight per lane), two for four.
template <int MT> struct GvRows { static constexpr int value = MT <= 2 ? 4 : 2; };

__device__ __forceinline__ int dp4a_s8(uint32_t a, uint32_t b, int c) {
  int d;
  asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// xs: shared memory, [2][MT][K / 8] words: for token t and packed word j, the even channels
// (16 x code per byte) at xs[(0 * MT + t) * kw + j], the odd channels at xs[(1 * MT + t) * kw + j].
template <int MT>
__global__ void __launch_bounds__(512)
w4a4_gemv_kernel(const uint8_t* __restrict__ Xq, const __half* __restrict__ sx, const uint8_t* __restrict__ Wq,
                 const __half* __restrict__ sw, int M, int N, int K, __half* __restrict__ Y,
                 int32_t* __restrict__ accdbg) {
  griddep_launch_dependents();                           // a rotate kernel launched behind this one may set itself up
  griddep_wait();                                        // Xq and sx may come from the kernel launched before this one
  extern __shared__ __align__(16) uint32_t xs[];
  constexpr int GV_ROWS = GvRows<MT>::value;
  const int kw = K / 8;                                  // packed words per row
  const int nchunk = K / 32;                             // 16-byte pieces per row
  // tokens -> shared memory, four 16-byte pieces per thread in flight
  for (int i0 = threadIdx.x; i0 < MT * nchunk; i0 += 4 * blockDim.x) {
    uint4 w[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * blockDim.x;
      const int t = i / nchunk, c = i % nchunk;
      w[u] = (i < MT * nchunk && t < M) ? __ldg(reinterpret_cast<const uint4*>(Xq + static_cast<size_t>(t) * (K / 2)) + c)
                                        : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * blockDim.x;
      if (i < MT * nchunk) {
        const int t = i / nchunk, c = i % nchunk;
        *reinterpret_cast<uint4*>(xs + (0 * MT + t) * kw + 4 * c) =
            make_uint4((w[u].x << 4) & 0xF0F0F0F0u, (w[u].y << 4) & 0xF0F0F0F0u, (w[u].z << 4) & 0xF0F0F0F0u,
                       (w[u].w << 4) & 0xF0F0F0F0u);
        *reinterpret_cast<uint4*>(xs + (1 * MT + t) * kw + 4 * c) =
            make_uint4(w[u].x & 0xF0F0F0F0u, w[u].y & 0xF0F0F0F0u, w[u].z & 0xF0F0F0F0u, w[u].w & 0xF0F0F0F0u);
      }
    }
  }
  __syncthreads();

  const int lane = threadIdx.x & 31;
  const int warps_per_cta = blockDim.x >> 5;
  const long long ntask = (N + GV_ROWS - 1) / GV_ROWS;
  const long long wstride = static_cast<long long>(gridDim.x) * warps_per_cta;
  // task index interleaved over CTAs first, so that the warps of all SMs work on neighbouring rows
  for (long long task = static_cast<long long>(threadIdx.x >> 5) * gridDim.x + blockIdx.x; task < ntask; task += wstride) {
    const int row0 = static_cast<int>(task) * GV_ROWS;
    int acc[GV_ROWS][MT];
#pragma unroll
    for (int r = 0; r < GV_ROWS; ++r)
#pragma unroll
      for (int t = 0; t < MT; ++t) acc[r][t] = 0;
    const uint4* wrow[GV_ROWS];
#pragma unroll
    for (int r = 0; r < GV_ROWS; ++r)
      wrow[r] = reinterpret_cast<const uint4*>(Wq + static_cast<size_t>(min(row0 + r, N - 1)) * (K / 2));
    for (int c0 = lane; c0 < nchunk; c0 += 32 * GV_UNROLL) {
      uint4 wv[GV_UNROLL][GV_ROWS];
#pragma unroll
      for (int u = 0; u < GV_UNROLL; ++u) {
        const int c = c0 + 32 * u;
#pragma unroll
        for (int r = 0; r < GV_ROWS; ++r)
          wv[u][r] = (c < nchunk) ? __ldcs(wrow[r] + c) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < GV_UNROLL; ++u) {
        const int c = c0 + 32 * u;
        if (c < nchunk) {
#pragma unroll
          for (int t = 0; t < MT; ++t) {
            const uint4 xe = *reinterpret_cast<const uint4*>(xs + (0 * MT + t) * kw + 4 * c);
            const uint4 xo = *reinterpret_cast<const uint4*>(xs + (1 * MT + t) * kw + 4 * c);
#pragma unroll
            for (int r = 0; r < GV_ROWS; ++r) {
              const uint4 w = wv[u][r];
              int a = acc[r][t];
              a = dp4a_s8((w.x << 4) & 0xF0F0F0F0u, xe.x, a); a = dp4a_s8(w.x & 0xF0F0F0F0u, xo.x, a);
              a = dp4a_s8((w.y << 4) & 0xF0F0F0F0u, xe.y, a); a = dp4a_s8(w.y & 0xF0F0F0F0u, xo.y, a);
              a = dp4a_s8((w.z << 4) & 0xF0F0F0F0u, xe.z, a); a = dp4a_s8(w.z & 0xF0F0F0F0u, xo.z, a);
              a = dp4a_s8((w.w << 4) & 0xF0F0F0F0u, xe.w, a); a = dp4a_s8(w.w & 0xF0F0F0F0u, xo.w, a);
              acc[r][t] = a;
            }
          }
        }
      }
    }
#pragma unroll
    for (int r = 0; r < GV_ROWS; ++r)
#pragma unroll
      for (int t = 0; t < MT; ++t) {
        int a = acc[r][t];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        acc[r][t] = a >> 8;                                // exact: the sum is 256 * acc
      }
    if (lane < GV_ROWS * MT) {
      const int r = lane / MT, t = lane % MT;
      int a = 0;
#pragma unroll
      for (int rr = 0; rr < GV_ROWS; ++rr)
#pragma unroll
        for (int tt = 0; tt < MT; ++tt)
          if (rr == r && tt == t) a = acc[rr][tt];
      const int row = row0 + r;
      if (row < N && t < M) {
        const float f = __int_as_float(0x4B400000 + a) - 12582912.0f;
        Y[static_cast<size_t>(t) * N + row] = __float2half_rn(f * (__half2float(__ldg(sx + t)) * __half2float(__ldg(sw + row))));
        if (accdbg) accdbg[static_cast<size_t>(t) * N + row] = a;
      }
    }
  }
}

// Warps per CTA such that the tasks fill sms * warps warps as evenly as possible.
int gemv_warps(long long ntask, int sms) {
  int best = 16;
  double best_eff = 0.0;
  for (int w = 16; w >= 8; --w) {                        // more warps = more bytes in flight: prefer many
    const long long total = static_cast<long long>(sms) * w;
    const long long waves = (ntask + total - 1) / total;
    const double eff = static_cast<double>(ntask) / static_cast<double>(waves * total);
    if (eff > best_eff + 0.01) {
      best_eff = eff;
      best = w;
    }
  }
  return best;
}

template <int MT>
sq_status_t launch_gemv(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N, int K, void* Y,
                        int32_t* accdbg, cudaStream_t s) {
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  constexpr int GV_ROWS = GvRows<MT>::value;
  const long long ntask = (N + GV_ROWS - 1) / GV_ROWS;
  const int warps = gemv_warps(ntask, sms);
  const int smem = MT * K;                               // 2 * MT * (K / 8) words
  auto kern = w4a4_gemv_kernel<MT>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) return SQ_ERR_CUDA;
  const unsigned grid = static_cast<unsigned>(std::min<long long>(sms, (ntask + warps - 1) / warps));
  const cudaError_t err = launch_maybe_pdl(kern, dim3(grid), dim3(warps * 32), static_cast<size_t>(smem), s,
                                           static_cast<const uint8_t*>(Xq), static_cast<const __half*>(sx),
                                           static_cast<const uint8_t*>(Wq), static_cast<const __half*>(sw), M, N, K,
                                           static_cast<__half*>(Y), accdbg);
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace

bool gemv_supported(int64_t M, int64_t N, int64_t K) {
  return M >= 1 && M <= 4 && N >= 1 && (K % 32 == 0) && K >= 32 && K <= 32768;
}

sq_status_t launch_w4a4_gemv(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N, int K,
                             void* Y, int32_t* accdbg, cudaStream_t s) {
  if (M == 1) return launch_gemv<1>(Xq, sx, Wq, sw, M, N, K, Y, accdbg, s);
  if (M == 2) return launch_gemv<2>(Xq, sx, Wq, sw, M, N, K, Y, accdbg, s);
  return launch_gemv<4>(Xq, sx, Wq, sw, M, N, K, Y, accdbg, s);
}

}  // namespace sq
