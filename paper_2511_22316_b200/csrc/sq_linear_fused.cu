// sq_linear for decode-sized batches (M <= 64) as ONE launch: steps 1+2 (Eq. "eq18", Section 3.2) and
// step 3 (X W = Flat(X~_R) Flat(W~_R)^T) run side by side in one grid.
//
// With a handful of tokens the layer is bound by streaming the packed weights once, and the two-kernel
// form pays a second launch, a second set-up and a hand-over through the end of a kernel.  Here the
// grid's first `rot_ctas` CTAs rotate and quantise the tokens (the body of the dense rotate kernel, one
// token group each) while all the others are CTAs of the decode GEMM (its body, unchanged): they set
// themselves up and pull the weights of their whole staging ring in at once, and only their token loads
// and the reads of the token steps wait -- on a counter in device memory that every rotating CTA bumps,
// with release semantics, after its last store.  The packed tokens travel through L2 (a few KB), not
// through a kernel boundary.
//
// Ordering between the two kinds of CTA: a rotating CTA's threads store Xq and sx, meet at the block
// barrier, then one thread does `red.release.gpu` on the counter; a GEMM thread that needs the tokens
// polls it with `ld.acquire.gpu`, then issues a proxy fence before its TMA loads.  The rotating CTAs
// have the lowest block indices, so they are on an SM before any CTA that waits for them; every wait is
// bounded all the same.  The counters (one slot per call, taken round-robin from 64 in the handle) are
// put back to zero by the last GEMM CTA to finish, so a slot is clean when its turn comes again.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <atomic>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

constexpr int kFusedSlots = 64;          // counter pairs per handle

template <int N2, int NT>
__global__ void __launch_bounds__(D_THREADS, 1)
linear_decode_fused_kernel(const __grid_constant__ CUtensorMap tmap_xin, const __grid_constant__ RqLayout L,
                           const unsigned char* __restrict__ a1_img, const unsigned char* __restrict__ b2_img, int n1,
                           int M, uint8_t* __restrict__ Xq, __half* __restrict__ sx,
                           const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_xq,
                           const __half* __restrict__ sw, int N, int K, int splits, __half* __restrict__ Y,
                           int rot_ctas, uint32_t* __restrict__ counters) {
  uint32_t* ready = counters;            // rotating CTAs that have stored their tokens
  uint32_t* done = counters + 1;         // GEMM CTAs that have finished
  const int cta = static_cast<int>(blockIdx.x);
  if (cta < rot_ctas) {
    rotate_quant_tc_body<N2, 2>(tmap_xin, L, a1_img, b2_img, n1, M, Xq, sx, nullptr, cta, rot_ctas);
    // every thread's stores precede the block barrier at the end of the body; the release is cumulative
    if (threadIdx.x == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ready) : "memory");
  } else {
    const int gemm_ctas = static_cast<int>(gridDim.x) - rot_ctas;
    w4a4_gemm_decode_body<NT>(tmap_w, tmap_xq, sx, sw, M, N, K, splits, Y, nullptr, cta - rot_ctas, gemm_ctas, ready,
                              static_cast<uint32_t>(rot_ctas));
    // The last GEMM CTA to get here clears the slot: every CTA has passed its waits on `ready` by then.
    __syncthreads();
    if (threadIdx.x == 0) {
      const uint32_t before = atomicAdd(done, 1u);
      if (before == static_cast<uint32_t>(gemm_ctas) - 1u) {
        *ready = 0u;
        *done = 0u;
      }
    }
  }
}

template <int N2, int NT>
int fused_max_clusters(int s, int sms, int smem) {
  static std::atomic<int> cache[64][4];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  const int slot = s == 2 ? 1 : (s == 4 ? 2 : (s == 8 ? 3 : 0));
  if (slot == 0) return sms;
  int v = cache[dev][slot].load(std::memory_order_relaxed);
  if (v != 0) return v > 0 ? v : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(sms / s * s));
  cfg.blockDim = dim3(D_THREADS);
  cfg.dynamicSmemBytes = static_cast<size_t>(smem);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(s);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, linear_decode_fused_kernel<N2, NT>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    n = 0;
  }
  cache[dev][slot].store(n > 0 ? n : -1, std::memory_order_relaxed);
  return n;
}

template <int N2, int NT>
sq_status_t launch_fused(const sq_rotation* h, const void* X, int M, const void* Wq, const void* sw, int N, int K,
                         void* Xq, void* sx, void* Y, cudaStream_t s) {
  using DL = DecSmem<NT>;
  const int n1 = h->n1, n2 = h->n2;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const RqLayout L = rq_layout(n1, n2);
  const int smem = std::max(L.total + 1024, DL::DYN_BYTES);
  auto kern = linear_decode_fused_kernel<N2, NT>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) return SQ_ERR_CUDA;
  const int tiles = (N + 127) / 128, blocks = (K / 128 + 1) / 2;
  // choose_splits asks how many clusters of the plain decode kernel fit the device; that query needs the
  // kernel's shared-memory limit raised first, as its own launcher does
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(w4a4_gemm_decode_kernel<NT>), DL::DYN_BYTES)) return SQ_ERR_CUDA;
  const int splits = choose_splits<NT>(tiles, blocks, sms);
  const int ncl_max = fused_max_clusters<N2, NT>(splits, sms, smem);
  if (ncl_max <= 0) return SQ_ERR_CUDA;
  // One rotating CTA per token group where the device has room for more clusters beside the GEMM's
  // (every CTA of the grid must be resident at once: the GEMM CTAs wait for the rotating ones).  The
  // GEMM gives up a cluster when it fills the device and that costs it no extra wave of tiles.  When a
  // rotating CTA would get more than four token groups, the two-kernel form is the better one: nothing
  // is launched and the caller falls back to it.
  const int groups = (M + L.G - 1) / L.G;
  int ncl = tiles < ncl_max ? tiles : ncl_max;
  int avail_cl = (splits == 1 ? sms : ncl_max) - ncl;
  if (avail_cl < 1) {
    if (ncl < 2 || (tiles + ncl - 2) / (ncl - 1) != (tiles + ncl - 1) / ncl) return SQ_ERR_UNSUPPORTED;
    --ncl;
    avail_cl = 1;
  }
  const int want_cl = (groups + splits - 1) / splits;
  const int rot_cl = want_cl < avail_cl ? want_cl : avail_cl;
  const int rot_ctas = rot_cl * splits;
  if ((groups + rot_ctas - 1) / rot_ctas > 4) return SQ_ERR_UNSUPPORTED;
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return SQ_ERR_CUDA;
  CUtensorMap mxin, mw, mxq;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(n2), static_cast<cuuint64_t>(n1), static_cast<cuuint64_t>(M)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(n2) * 2, static_cast<cuuint64_t>(n1) * n2 * 2};
  const cuuint32_t box[3] = {64, static_cast<cuuint32_t>(L.N1), 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (enc(&mxin, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(X), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return SQ_ERR_CUDA;
  if (!make_packed_map(&mw, Wq, N, K / 2, 128) || !make_packed_map(&mxq, Xq, M, K / 2, NT)) return SQ_ERR_CUDA;
  const uint32_t slot = h->fused_calls.fetch_add(1u, std::memory_order_relaxed) % kFusedSlots;
  uint32_t* counters = h->dFusedCounters + 2 * slot;
  const unsigned grid = static_cast<unsigned>(rot_ctas + ncl * splits);
  const bool pdl = g_pdl_next;
  g_pdl_next = false;                      // nothing precedes this kernel that it may overlap
  const cudaError_t err = launch_cluster_maybe_pdl(
      kern, dim3(grid), dim3(D_THREADS), static_cast<size_t>(smem), s, static_cast<unsigned>(splits), mxin, L,
      static_cast<const unsigned char*>(h->dA1img), static_cast<const unsigned char*>(h->dB2img), n1, M,
      static_cast<uint8_t*>(Xq), static_cast<__half*>(sx), mw, mxq, static_cast<const __half*>(sw), N, K, splits,
      static_cast<__half*>(Y), rot_ctas, counters);
  g_pdl_next = pdl;
  count_launch();
  return err == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace

bool linear_fused_prepare(sq_rotation* h) {
  if (!h->tc_ready) return true;           // only handles that take the dense tensor-core rotate kernel
  if (cudaMalloc(&h->dFusedCounters, sizeof(uint32_t) * 2 * kFusedSlots) != cudaSuccess ||
      cudaMemset(h->dFusedCounters, 0, sizeof(uint32_t) * 2 * kFusedSlots) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return true;
}

bool linear_fused_supported(const sq_rotation* h, int64_t M, int64_t N, int64_t K) {
  if (!h->tc_ready || h->st_ready || h->dFusedCounters == nullptr) return false;
  if (M < 1 || M > 64) return false;
  return gemm_decode_supported(M, N, K);
}

sq_status_t launch_linear_fused(const sq_rotation* h, const void* X, int64_t M, const void* Wq, const void* sw,
                                int64_t N, int64_t K, void* Xq, void* sx, void* Y, cudaStream_t s) {
  const int m = static_cast<int>(M), n = static_cast<int>(N), k = static_cast<int>(K);
  if (h->n2 == 64) {
    if (M <= 16) return launch_fused<64, 16>(h, X, m, Wq, sw, n, k, Xq, sx, Y, s);
    if (M <= 32) return launch_fused<64, 32>(h, X, m, Wq, sw, n, k, Xq, sx, Y, s);
    return launch_fused<64, 64>(h, X, m, Wq, sw, n, k, Xq, sx, Y, s);
  }
  if (M <= 16) return launch_fused<128, 16>(h, X, m, Wq, sw, n, k, Xq, sx, Y, s);
  if (M <= 32) return launch_fused<128, 32>(h, X, m, Wq, sw, n, k, Xq, sx, Y, s);
  return launch_fused<128, 64>(h, X, m, Wq, sw, n, k, Xq, sx, Y, s);
}

}  // namespace sq
