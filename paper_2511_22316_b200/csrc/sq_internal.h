// Internal declarations shared by the translation units of libsinglequant.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <utility>
#include <vector>

#include "../../include/singlequant.h"

// How R2 = H R2^U was composed (paragraphs "Uniformity Rotation Transformation", "The Overall
// SingleQuant Method"): R2^U = R_map R'_map^T, R_map the chain of plane rotations on adjacent
// coordinates with v R_map = ||v|| e_1, R'_map the same for the target u.  Known for handles made
// by sq_build_rotation, unknown for factors injected by the caller.
struct R2Structure {
  bool known = false;
  bool hadamard = false;        // H is the Sylvester Hadamard matrix / sqrt(n2) (else the identity)
  bool urt = false;             // R2^U is present (else the identity)
  std::vector<double> v, u;     // URT's source vector and its target, length n2 (when urt)
};

struct sq_rotation {
  int32_t n1 = 0, n2 = 0;
  int device = -1;
  std::vector<float> R1;   // host fp32 [n1 x n1]
  std::vector<float> R2;   // host fp32 [n2 x n2]
  float* dR1 = nullptr;    // device fp32 [n1 x n1]
  float* dR2 = nullptr;    // device fp32 [n2 x n2]
  // tensor-core rotate+quant: shared-memory images of the split factors (device), if supported
  void* dA1img = nullptr;
  void* dB2img = nullptr;
  bool tc_ready = false;   // images for the single-CTA kernel (n1 <= 128)
  bool tc_pair = false;    // images for the CTA-pair kernel (128 < n1 <= 256)
  // structured application of R2 (sq_rotate_quant_st.cu): composition and kernel coefficients
  R2Structure s2;
  bool st_ready = false;
  std::vector<float> st_coef;   // the kernel's coefficient block (host copy, passed by value)
  // fused decode layer (sq_linear_fused.cu): pairs of device counters, one pair per call in turn
  uint32_t* dFusedCounters = nullptr;
  mutable std::atomic<uint32_t> fused_calls{0};
};

namespace sq {

extern std::atomic<uint64_t> g_launches;
inline void count_launch(uint64_t k = 1) { g_launches.fetch_add(k, std::memory_order_relaxed); }

// Multiprocessor count of the current device (cached per device; <= 0 on failure).
int sm_count();

// True except around the launch of the one-launch decode layer: every GEMM kernel is launched as a
// programmatic dependent of the kernel before it in the stream.  It may then set itself up and request
// its first weight blocks while that kernel is still running (a rotate kernel, or another GEMM in a run
// of projections); it waits on the device before it reads activations, steps or writes anything.  Weights
// written by this library are complete by then: sq_pack_weight and sq_pack_weight_wo end with an ordinary
// kernel, which never lets dependents start early.
extern thread_local bool g_pdl_next;

// Launches `kern` with thread-block clusters of `cluster` CTAs along x (1: no clusters), and as a
// programmatic dependent of the stream's previous kernel when g_pdl_next is set.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_cluster_maybe_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                            unsigned cluster, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (g_pdl_next) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_maybe_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    Args&&... args) {
  return launch_cluster_maybe_pdl(kern, grid, block, smem, s, 1u, static_cast<Args&&>(args)...);
}

// Launches `kern` as a programmatic dependent of whatever precedes it in the stream: it may start while
// that kernel still runs, once all of that kernel's CTAs have allowed it (griddepcontrol.launch_dependents)
// or exited, and must not touch memory the predecessor reads or writes before its own
// griddepcontrol.wait returns.  After a predecessor that never allows it, this is an ordinary launch.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Raises a kernel's dynamic shared-memory limit to `bytes` if it is lower.  Function attributes
// belong to a device: the sizes already set are remembered per (device, kernel).
bool ensure_dyn_smem(const void* kern, int bytes);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Host-side construction of the factors in float64 (sq_rotation_host.cu).
sq_status_t build_factors_host(const float* calib, int64_t T, int64_t n, int32_t n1, int32_t n2,
                               uint32_t flags, uint64_t seed, const double* O,
                               std::vector<float>& R1, std::vector<float>& R2, R2Structure* s2);

// Steps 1+2 (sq_rotate_quant.cu).  R1/R2 device fp32 or both nullptr for the identity.
// qmax = 2^(b-1) - 1 for b-bit codes (7: INT4); qmax = 0: rotation only, Xq receives fp16 rows.
sq_status_t launch_rotate_quant(const float* dR1, const float* dR2, int n1, int n2, const void* X,
                                int64_t rows, void* Xq, void* scales, float* Zdbg, cudaStream_t s, int qmax = 7);

// Tensor-core variant of steps 1+2 (sq_rotate_quant_tc.cu).
bool rotate_quant_tc_supported(int n1, int n2);
bool rotate_quant_tc_prepare(sq_rotation* h);
sq_status_t launch_rotate_quant_tc(const sq_rotation* h, const void* X, int64_t rows, void* Xq, void* scales,
                                   float* Zdbg, cudaStream_t s, bool f16out = false);
// Tensor-core variant for 128 < n1 <= 256 on CTA pairs (sq_rotate_quant_pair.cu).
bool rotate_quant_pair_supported(int n1, int n2);
bool rotate_quant_pair_prepare(sq_rotation* h);
sq_status_t launch_rotate_quant_pair(const sq_rotation* h, const void* X, int64_t rows, void* Xq, void* scales,
                                     float* Zdbg, cudaStream_t s, bool f16out = false);
// Steps 1+2 with R2 applied through its structure (sq_rotate_quant_st.cu): R1^T on the tensor cores,
// then the Hadamard butterflies and the two rotation chains of URT in registers.
bool rotate_quant_st_prepare(sq_rotation* h);
sq_status_t launch_rotate_quant_st(const sq_rotation* h, const void* X, int64_t rows, void* Xq, void* scales,
                                   float* Zdbg, cudaStream_t s);
// The whole layer for M <= 64 as one launch (sq_linear_fused.cu): rotating CTAs and decode-GEMM CTAs in
// one grid, the tokens handed over through L2 behind a device counter.
bool linear_fused_prepare(sq_rotation* h);
bool linear_fused_supported(const sq_rotation* h, int64_t M, int64_t N, int64_t K);
sq_status_t launch_linear_fused(const sq_rotation* h, const void* X, int64_t M, const void* Wq, const void* sw,
                                int64_t N, int64_t K, void* Xq, void* sx, void* Y, cudaStream_t s);
// Picks the tensor-core kernel when the handle has its images, else the generic fp32 kernel.
sq_status_t rotate_quant_dispatch(const sq_rotation* h, const void* X, int64_t rows, void* Xq, void* scales,
                                  float* Zdbg, cudaStream_t s);

// Step 1 alone with fp16 rows out (the rotation-only form of the kernels above).
sq_status_t rotate_f16_dispatch(const sq_rotation* h, const void* X, int64_t rows, void* Z16, cudaStream_t s);

// Step 3 (sq_gemm.cu).
sq_status_t launch_w4a4_gemm(const void* Xq, const void* sx, const void* Wq, const void* sw,
                             int64_t M, int64_t N, int64_t K, void* Y, int32_t* accdbg, cudaStream_t s);

// Step 3 on CTA pairs (sq_gemm_pair.cu): prefill-sized problems.
bool gemm_pair_supported(int64_t M, int64_t N, int64_t K);
sq_status_t launch_w4a4_gemm_pair(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N,
                                  int K, void* Y, int32_t* accdbg, cudaStream_t s);

// Step 3 for decode-sized problems (sq_gemm_decode.cu): weights as the A operand, K split over a
// thread-block cluster with the partial tiles exchanged on chip (no scratch in global memory).
bool gemm_decode_supported(int64_t M, int64_t N, int64_t K);
// The CTA-pair kernel over the experts of a grouped layer in one launch (any number of rows per expert).
int gemm_pair_max_groups();
sq_status_t launch_w4a4_gemm_pair_grouped(const void* Xq, const void* sx, int64_t M_total, int count,
                                          const void* const* Wq, const void* const* sw, const int64_t* r0,
                                          const int64_t* rows, int N, int K, void* Y, cudaStream_t s);
// The decode kernel over the experts of a grouped layer in one launch (a tile = expert x 128 channels).
int gemm_decode_max_groups();
sq_status_t launch_w4a4_gemm_decode_grouped(const void* Xq, const void* sx, int64_t M_total, int count,
                                            const void* const* Wq, const void* const* sw, const int64_t* r0,
                                            const int64_t* rows, int N, int K, void* Y, cudaStream_t s);
sq_status_t launch_w4a4_gemm_decode(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N, int K,
                                    void* Y, int32_t* accdbg, cudaStream_t s);

// Step 3 for one to four tokens (sq_gemv.cu): dot products on the CUDA cores.
bool gemv_supported(int64_t M, int64_t N, int64_t K);
sq_status_t launch_w4a4_gemv(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N, int K,
                             void* Y, int32_t* accdbg, cudaStream_t s);

// Weight-only variant (sq_gemm_wo.cu): fp16 activations x b-bit weight codes in the weight-only
// storage order, fp32 accumulation, one rounding of acc * s_w to fp16.
sq_status_t launch_wo_gemm(const void* Z16, const void* Wq, const void* sw, int64_t M, int64_t N, int64_t K, void* Y,
                           cudaStream_t s);
// Rewrites packed rows [rows x K/2] from channel order into the weight-only storage order, in place.
sq_status_t launch_interleave_nibbles(void* Wq, int64_t rows, int64_t K, cudaStream_t s);

// Device status word helpers (sq_api.cu).
sq_status_t read_and_clear_device_status(cudaStream_t s);

}  // namespace sq
