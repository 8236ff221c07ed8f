// C ABI entry points: argument validation on the host, then the kernel launchers.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>
#include <vector>
#include <new>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
std::atomic<uint64_t> g_launches{0};
thread_local bool g_pdl_next = true;

bool ensure_dyn_smem(const void* kern, int bytes) {
  struct Entry { int dev; const void* kern; int bytes; };
  static std::mutex mu;
  static std::vector<Entry> set;
  if (bytes <= 48 * 1024) return true;                 // within every kernel's default limit
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  std::lock_guard<std::mutex> lock(mu);
  for (Entry& e : set)
    if (e.dev == dev && e.kern == kern) {
      if (e.bytes >= bytes) return true;
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
      e.bytes = bytes;
      return true;
    }
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
  set.push_back({dev, kern, bytes});
  return true;
}

int sm_count() {
  static std::atomic<int> cache[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return -1;
  if (dev >= 0 && dev < 64) {
    const int c = cache[dev].load(std::memory_order_relaxed);
    if (c > 0) return c;
  }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
  if (dev >= 0 && dev < 64) cache[dev].store(sms, std::memory_order_relaxed);
  return sms;
}

sq_status_t read_and_clear_device_status(cudaStream_t s) {
  if (cudaStreamSynchronize(s) != cudaSuccess) return SQ_ERR_CUDA;
  unsigned int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(v)) != cudaSuccess) return SQ_ERR_CUDA;
  if (v != 0) {
    const unsigned int zero = 0;
    if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(zero)) != cudaSuccess) return SQ_ERR_CUDA;
    return SQ_ERR_TIMEOUT;
  }
  return SQ_OK;
}
}  // namespace sq

extern "C" void sq_rotation_destroy(sq_rotation_t* rot);

namespace sq {
// Ends sq_pack_weight: an ordinary launch that never lets dependents start early.  The GEMM kernels are
// launched as programmatic dependents and request their first weight blocks before they wait for their
// predecessor; the rotate kernels that wrote those weights allow dependents while they are still
// writing, this kernel does not, so a GEMM queued right behind sq_pack_weight starts after the weights
// are complete.
__global__ void weights_complete_kernel() {}

// One thread, one barrier that nobody arrives at, the library's own bounded wait: it gives up after
// `polls` polls, records its site in the status word and returns.  No copy, MMA or TMEM allocation
// is in flight when it does.
__global__ void bounded_wait_probe_kernel(uint32_t polls) {
  __shared__ uint64_t bar;
  mbar_init(&bar, 1);
  mbar_fence_init();
  mbar_wait(&bar, 0, /*site=*/255u, polls);
}
}  // namespace sq

namespace sq {
sq_status_t rotate_quant_dispatch(const sq_rotation* h, const void* X, int64_t rows, void* Xq, void* scales,
                                  float* Zdbg, cudaStream_t s) {
  if (h->st_ready) return launch_rotate_quant_st(h, X, rows, Xq, scales, Zdbg, s);
  if (h->tc_ready) return launch_rotate_quant_tc(h, X, rows, Xq, scales, Zdbg, s);
  if (h->tc_pair) return launch_rotate_quant_pair(h, X, rows, Xq, scales, Zdbg, s);
  return launch_rotate_quant(h->dR1, h->dR2, h->n1, h->n2, X, rows, Xq, scales, Zdbg, s);
}
// Step 1 alone, fp16 rows out (weight-only variant): the same kernels in their rotation-only form.
sq_status_t rotate_f16_dispatch(const sq_rotation* h, const void* X, int64_t rows, void* Z16, cudaStream_t s) {
  if (h->tc_ready) return launch_rotate_quant_tc(h, X, rows, Z16, nullptr, nullptr, s, true);
  if (h->tc_pair) return launch_rotate_quant_pair(h, X, rows, Z16, nullptr, nullptr, s, true);
  return launch_rotate_quant(h->dR1, h->dR2, h->n1, h->n2, X, rows, Z16, nullptr, nullptr, s, 0);
}
}  // namespace sq

namespace {

constexpr int64_t kMaxN = 32768;       // rotate+quant: the row and its fp32 image stay in shared memory
constexpr int64_t kMaxK = 65536;       // GEMM: 256 * 64 * K must fit in int32
constexpr int64_t kMaxRows = (1ll << 31) - 1;

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

sq_status_t make_handle(std::vector<float>&& R1, std::vector<float>&& R2, int32_t n1, int32_t n2,
                        const R2Structure* s2, bool fuse_decode, sq_rotation_t** out) {
  sq_rotation* h = new (std::nothrow) sq_rotation();
  if (!h) return SQ_ERR_NOMEM;
  h->n1 = n1;
  h->n2 = n2;
  if (s2) h->s2 = *s2;
  h->R1 = std::move(R1);
  h->R2 = std::move(R2);
  if (cudaGetDevice(&h->device) != cudaSuccess) {
    delete h;
    return SQ_ERR_CUDA;
  }
  const size_t b1 = sizeof(float) * h->R1.size(), b2 = sizeof(float) * h->R2.size();
  if (cudaMalloc(&h->dR1, b1) != cudaSuccess || cudaMalloc(&h->dR2, b2) != cudaSuccess ||
      cudaMemcpy(h->dR1, h->R1.data(), b1, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(h->dR2, h->R2.data(), b2, cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    if (h->dR1) cudaFree(h->dR1);
    if (h->dR2) cudaFree(h->dR2);
    delete h;
    return SQ_ERR_CUDA;
  }
  const bool prepared = (sq::rotate_quant_tc_supported(n1, n2)     ? sq::rotate_quant_tc_prepare(h)
                         : sq::rotate_quant_pair_supported(n1, n2) ? sq::rotate_quant_pair_prepare(h)
                                                                   : true) &&
                        sq::rotate_quant_st_prepare(h) && (!fuse_decode || sq::linear_fused_prepare(h));
  if (!prepared) {
    sq_rotation_destroy(h);
    return SQ_ERR_CUDA;
  }
  *out = h;
  return SQ_OK;
}

sq_status_t check_rows_args(const void* in, const void* q, const void* sc, const void* dbg, int64_t rows,
                            int64_t n) {
  if (rows < 0 || rows > kMaxRows) return SQ_ERR_INVALID_ARG;
  if (n < 2 || (n & 1)) return SQ_ERR_SHAPE;
  if (n > kMaxN) return SQ_ERR_UNSUPPORTED;
  if (rows == 0) return SQ_OK;
  if (!in || !q || !sc) return SQ_ERR_INVALID_ARG;
  if (!sq::aligned16(in) || !sq::aligned16(q) || !sq::aligned16(sc) || !sq::aligned16(dbg)) return SQ_ERR_ALIGN;
  return SQ_OK;
}

sq_status_t check_gemm_args(const void* Xq, const void* sx, const void* Wq, const void* sw, int64_t M, int64_t N,
                            int64_t K, const void* Y, const void* acc) {
  if (M < 0 || N < 0 || M > kMaxRows || N > kMaxRows) return SQ_ERR_INVALID_ARG;
  if (K < 2 || (K & 1)) return SQ_ERR_SHAPE;
  if (K > kMaxK) return SQ_ERR_UNSUPPORTED;
  if (M == 0 || N == 0) return SQ_OK;
  if (!Xq || !sx || !Wq || !sw || !Y) return SQ_ERR_INVALID_ARG;
  if (!sq::aligned16(Xq) || !sq::aligned16(sx) || !sq::aligned16(Wq) || !sq::aligned16(sw) || !sq::aligned16(Y) ||
      !sq::aligned16(acc))
    return SQ_ERR_ALIGN;
  return SQ_OK;
}

// A handle's factors live on the device that was current when it was made; a call with another
// device current would hand that GPU's kernels pointers into this one's memory.
sq_status_t check_handle_device(const sq_rotation* rot) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return SQ_ERR_CUDA;
  return dev == rot->device ? SQ_OK : SQ_ERR_INVALID_ARG;
}

}  // namespace

extern "C" {

sq_status_t sq_factorize(int64_t n, int32_t* n1, int32_t* n2) {
  if (!n1 || !n2 || n < 1 || n > (1ll << 40)) return SQ_ERR_INVALID_ARG;
  // The powers of two that divide n are 2^0 .. 2^v, v = number of trailing zero bits of n.  The one
  // nearest to sqrt(n) is one of the two powers of two that bracket sqrt(n), each clipped to 2^v:
  // lo = 2^e with 4^e <= n < 4^(e+1), hi = 2 lo.  "lo is at least as near as hi" is
  // sqrt(n) - lo <= hi - sqrt(n), i.e. 4 n <= 9 lo^2 in exact integer arithmetic; the smaller power
  // wins a tie (Algorithm 1 keeps the first candidate it meets, and it meets them in rising order).
  const int v = __builtin_ctzll(static_cast<unsigned long long>(n));
  int e = 0;
  while ((4ll << (2 * e)) <= n) ++e;                       // largest e with 4^e <= n
  int64_t lo = 1ll << (e < v ? e : v);
  int64_t hi = 1ll << (e + 1 < v ? e + 1 : v);
  const int64_t best = (hi == lo || 4 * n <= 9 * lo * lo) ? lo : hi;
  if (n / best > INT32_MAX) return SQ_ERR_UNSUPPORTED;
  *n1 = static_cast<int32_t>(n / best);
  *n2 = static_cast<int32_t>(best);
  return SQ_OK;
}

sq_status_t sq_build_rotation(const float* calib, int64_t T, int64_t n, int32_t n1, int32_t n2, uint32_t flags,
                              uint64_t seed, const double* O_or_null, sq_rotation_t** out) {
  if (!out) return SQ_ERR_INVALID_ARG;
  *out = nullptr;
  if (!calib || T < 1 || n1 < 1 || n2 < 1 || (flags & ~(7u | (0x7FFu << 8) | SQ_ROT_APPLY_STRUCTURED | SQ_ROT_FUSE_DECODE)))
    return SQ_ERR_INVALID_ARG;
  if (static_cast<int64_t>(n1) * n2 != n) return SQ_ERR_SHAPE;
  if ((flags & SQ_ROT_HADAMARD) && (n2 & (n2 - 1)) != 0) return SQ_ERR_SHAPE;
  if (n1 > 4096 || n2 > 4096) return SQ_ERR_UNSUPPORTED;
  std::vector<float> R1, R2;
  R2Structure s2;
  sq_status_t st = sq::build_factors_host(calib, T, n, n1, n2, flags, seed, O_or_null, R1, R2, &s2);
  if (st != SQ_OK) return st;
  return make_handle(std::move(R1), std::move(R2), n1, n2, (flags & SQ_ROT_APPLY_STRUCTURED) ? &s2 : nullptr,
                     (flags & SQ_ROT_FUSE_DECODE) != 0, out);
}

sq_status_t sq_rotation_from_factors(const float* R1, const float* R2, int32_t n1, int32_t n2,
                                     sq_rotation_t** out) {
  if (!out) return SQ_ERR_INVALID_ARG;
  *out = nullptr;
  if (!R1 || !R2 || n1 < 1 || n2 < 1) return SQ_ERR_INVALID_ARG;
  if (n1 > 4096 || n2 > 4096) return SQ_ERR_UNSUPPORTED;
  std::vector<float> a(R1, R1 + static_cast<size_t>(n1) * n1), b(R2, R2 + static_cast<size_t>(n2) * n2);
  return make_handle(std::move(a), std::move(b), n1, n2, nullptr, false, out);
}

sq_status_t sq_rotation_get_factors(const sq_rotation_t* rot, float* R1, float* R2) {
  if (!rot || !R1 || !R2) return SQ_ERR_INVALID_ARG;
  std::memcpy(R1, rot->R1.data(), sizeof(float) * rot->R1.size());
  std::memcpy(R2, rot->R2.data(), sizeof(float) * rot->R2.size());
  return SQ_OK;
}

sq_status_t sq_rotation_dims(const sq_rotation_t* rot, int32_t* n1, int32_t* n2) {
  if (!rot || !n1 || !n2) return SQ_ERR_INVALID_ARG;
  *n1 = rot->n1;
  *n2 = rot->n2;
  return SQ_OK;
}

int32_t sq_rotation_is_structured(const sq_rotation_t* rot) { return (rot && rot->st_ready) ? 1 : 0; }

void sq_rotation_destroy(sq_rotation_t* rot) {
  if (!rot) return;
  if (rot->dR1) cudaFree(rot->dR1);
  if (rot->dR2) cudaFree(rot->dR2);
  if (rot->dA1img) cudaFree(rot->dA1img);
  if (rot->dB2img) cudaFree(rot->dB2img);
  if (rot->dFusedCounters) cudaFree(rot->dFusedCounters);
  delete rot;
}

sq_status_t sq_rotate_quant_act(const sq_rotation_t* rot, const void* X, int64_t M, void* Xq, void* sx,
                                void* Zdbg_or_null, void* stream) {
  if (!rot) return SQ_ERR_INVALID_ARG;
  const int64_t n = static_cast<int64_t>(rot->n1) * rot->n2;
  if (rot->n2 & 1) return SQ_ERR_SHAPE;
  sq_status_t st = check_rows_args(X, Xq, sx, Zdbg_or_null, M, n);
  if (st != SQ_OK || M == 0) return st;
  if ((st = check_handle_device(rot)) != SQ_OK) return st;
  return sq::rotate_quant_dispatch(rot, X, M, Xq, sx, static_cast<float*>(Zdbg_or_null),
                                   static_cast<cudaStream_t>(stream));
}

sq_status_t sq_pack_weight(const sq_rotation_t* rot_or_null, const void* W, int64_t N, int64_t K, void* Wq,
                           void* sw, void* stream) {
  if (rot_or_null) {
    if (static_cast<int64_t>(rot_or_null->n1) * rot_or_null->n2 != K) return SQ_ERR_SHAPE;
    if (rot_or_null->n2 & 1) return SQ_ERR_SHAPE;
  }
  sq_status_t st = check_rows_args(W, Wq, sw, nullptr, N, K);
  if (st != SQ_OK || N == 0) return st;
  if (rot_or_null && (st = check_handle_device(rot_or_null)) != SQ_OK) return st;
  if (!rot_or_null)
    return sq::launch_rotate_quant(nullptr, nullptr, 1, static_cast<int>(K), W, N, Wq, sw, nullptr,
                                   static_cast<cudaStream_t>(stream));
  st = sq::rotate_quant_dispatch(rot_or_null, W, N, Wq, sw, nullptr, static_cast<cudaStream_t>(stream));
  if (st != SQ_OK) return st;
  sq::weights_complete_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>();
  sq::count_launch();
  return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

sq_status_t sq_w4a4_gemm(const void* Xq, const void* sx, const void* Wq, const void* sw, int64_t M, int64_t N,
                         int64_t K, void* Y, void* accdbg_or_null, void* stream) {
  sq_status_t st = check_gemm_args(Xq, sx, Wq, sw, M, N, K, Y, accdbg_or_null);
  if (st != SQ_OK || M == 0 || N == 0) return st;
  return sq::launch_w4a4_gemm(Xq, sx, Wq, sw, M, N, K, Y, static_cast<int32_t*>(accdbg_or_null),
                              static_cast<cudaStream_t>(stream));
}

// Workspace layout of sq_linear: [Xq: M*K/2][sx: 2*M], each 256-byte aligned.
size_t sq_linear_workspace_bytes(int64_t M, int64_t K) {
  if (M <= 0 || K <= 0) return 0;
  return align_up(static_cast<size_t>(M) * (K / 2), 256) + align_up(static_cast<size_t>(M) * 2, 256);
}

sq_status_t sq_linear(const sq_rotation_t* rot, const void* X, int64_t M, const void* Wq, const void* sw,
                      int64_t N, int64_t K, void* workspace, size_t workspace_bytes, void* Y, void* stream) {
  if (!rot) return SQ_ERR_INVALID_ARG;
  if (static_cast<int64_t>(rot->n1) * rot->n2 != K) return SQ_ERR_SHAPE;
  if (rot->n2 & 1) return SQ_ERR_SHAPE;
  if (M < 0 || N < 0) return SQ_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return SQ_OK;
  if (!workspace) return SQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SQ_ERR_ALIGN;
  if (workspace_bytes < sq_linear_workspace_bytes(M, K)) return SQ_ERR_NOMEM;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  void* Xq = ws;
  void* sx = ws + align_up(static_cast<size_t>(M) * (K / 2), 256);
  // Both halves are validated before anything is queued.
  sq_status_t st = check_rows_args(X, Xq, sx, nullptr, M, K);
  if (st != SQ_OK) return st;
  if ((st = check_gemm_args(Xq, sx, Wq, sw, M, N, K, Y, nullptr)) != SQ_OK) return st;
  if ((st = check_handle_device(rot)) != SQ_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // A decode-sized batch: rotation, quantisation and GEMM as one launch.
  if (sq::linear_fused_supported(rot, M, N, K)) {
    st = sq::launch_linear_fused(rot, X, M, Wq, sw, N, K, Xq, sx, Y, s);
    if (st != SQ_ERR_UNSUPPORTED) return st;          // else: nothing was launched, take the two-kernel form
  }
  st = sq::rotate_quant_dispatch(rot, X, M, Xq, sx, nullptr, s);
  if (st != SQ_OK) return st;
  // Every tensor-core GEMM kernel and the dot-product kernel start their set-up (and their weight
  // loads) while the rotate kernel drains; they wait for it before they read Xq or sx.
  return sq::launch_w4a4_gemm(Xq, sx, Wq, sw, M, N, K, Y, nullptr, s);
}

// Workspace layout of sq_linear_host: [X: 2*M*K][Y: 2*M*N][sq_linear workspace].
size_t sq_linear_host_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M <= 0 || N <= 0 || K <= 0) return 0;
  return align_up(static_cast<size_t>(M) * K * 2, 256) + align_up(static_cast<size_t>(M) * N * 2, 256) +
         sq_linear_workspace_bytes(M, K);
}

namespace {
// Copy streams and events of sq_linear_host, made once per device and kept until exit.
constexpr int kHostChunks = 4;
struct HostPipe {
  bool ready = false;
  cudaStream_t h2d = nullptr, d2h = nullptr;
  cudaEvent_t start = nullptr, landed[kHostChunks] = {}, done[kHostChunks] = {};
};
HostPipe* host_pipe() {
  static HostPipe pipes[64];
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  HostPipe& p = pipes[dev];
  if (!p.ready) {
    bool ok = cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess;
    for (int c = 0; c < kHostChunks && ok; ++c)
      ok = cudaEventCreateWithFlags(&p.landed[c], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&p.done[c], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      return nullptr;
    }
    p.ready = true;
  }
  return &p;
}
}  // namespace

// Large batches are cut into up to four row chunks: chunk c + 1 travels to the device while chunk c
// is computed and chunk c - 1 travels back (the two copy directions use separate streams, the link
// is full duplex), so the call takes about one direction's copy time instead of the sum of both.
sq_status_t sq_linear_host(const sq_rotation_t* rot, const void* X_host, int64_t M, const void* Wq, const void* sw,
                           int64_t N, int64_t K, void* workspace, size_t workspace_bytes, void* Y_host,
                           void* stream) {
  if (!rot || M < 0 || N < 0 || K < 2) return SQ_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return SQ_OK;
  if (!X_host || !Y_host || !workspace) return SQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SQ_ERR_ALIGN;
  if (workspace_bytes < sq_linear_host_workspace_bytes(M, N, K)) return SQ_ERR_NOMEM;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  const size_t xb = static_cast<size_t>(M) * K * 2, yb = static_cast<size_t>(M) * N * 2;
  unsigned char* dX = ws;
  unsigned char* dY = ws + align_up(xb, 256);
  void* lws = dY + align_up(yb, 256);
  const size_t lws_bytes = sq_linear_workspace_bytes(M, K);
  // Everything sq_linear would refuse is refused here, before the first copy is queued.
  if (static_cast<int64_t>(rot->n1) * rot->n2 != K || (rot->n2 & 1)) return SQ_ERR_SHAPE;
  {
    unsigned char* lw = static_cast<unsigned char*>(lws);
    sq_status_t pre = check_rows_args(dX, lw, lw + align_up(static_cast<size_t>(M) * (K / 2), 256), nullptr, M, K);
    if (pre == SQ_OK) pre = check_gemm_args(lw, lw, Wq, sw, M, N, K, dY, nullptr);
    if (pre == SQ_OK) pre = check_handle_device(rot);
    if (pre != SQ_OK) return pre;
  }
  // Up to four chunks, a multiple of 256 rows each.  The link is some ten times slower than the kernels,
  // so what counts is how little of it idles: one chunk's copy in before the first kernel and one
  // chunk's copy out after the last are exposed.  Measured on two hosts (2048 x 4096 -> 4096, 16.8 MB each
  // way): 0.68 ms unchunked, 0.56 / 0.59 / 0.67 / 0.72 ms with 2 / 4 / 8 / 16 chunks -- each queued copy
  // costs the link more than the finer overlap returns, although one 16.8 MB copy per direction, both at
  // once, takes 0.35 ms.
  // From 1024 rows on the first and the last chunk are small (an eighth of the rows each): they are the
  // two copies nothing overlaps (2048 rows: 0.563 -> 0.532 ms; a sixteenth each measured 0.545 ms).
  int64_t bound[kHostChunks + 1];
  int chunks = 1;
  bound[0] = 0;
  bound[1] = M;
  if (M >= 1024) {
    const int64_t edge = std::max<int64_t>(256, (M / 8 + 255) / 256 * 256);
    const int64_t mid = ((M - 2 * edge) / 2 + 255) / 256 * 256;
    chunks = 4;
    bound[1] = edge;
    bound[2] = edge + mid;
    bound[3] = M - edge;
    bound[4] = M;
    if (bound[2] >= bound[3]) {             // cannot happen for M >= 1024; keeps the bounds monotone anyway
      bound[2] = bound[3];
    }
  } else if (M >= 512) {
    chunks = 2;
    bound[1] = (M / 2 + 255) / 256 * 256;
    bound[2] = M;
  }
  HostPipe* p = chunks > 1 ? host_pipe() : nullptr;
  if (chunks == 1 || p == nullptr) {
    // Whatever fails after the first copy is queued, the stream is drained before returning: no
    // copy from or to the caller's host buffers outlives the call.
    sq_status_t st = SQ_OK;
    if (cudaMemcpyAsync(dX, X_host, xb, cudaMemcpyHostToDevice, s) != cudaSuccess) return SQ_ERR_CUDA;
    st = sq_linear(rot, dX, M, Wq, sw, N, K, lws, lws_bytes, dY, stream);
    if (st == SQ_OK && cudaMemcpyAsync(Y_host, dY, yb, cudaMemcpyDeviceToHost, s) != cudaSuccess) st = SQ_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess && st == SQ_OK) st = SQ_ERR_CUDA;
    return st;
  }
  // Everything follows what is already queued on the caller's stream.
  if (cudaEventRecord(p->start, s) != cudaSuccess || cudaStreamWaitEvent(p->h2d, p->start, 0) != cudaSuccess ||
      cudaStreamWaitEvent(p->d2h, p->start, 0) != cudaSuccess)
    return SQ_ERR_CUDA;
  sq_status_t st = SQ_OK;
  // All copies in are queued first: the host needs some twenty microseconds per chunk to queue the
  // kernels and the copy out, and the inbound link must not idle meanwhile.
  for (int c = 0; c < chunks && st == SQ_OK; ++c) {
    const int64_t r0 = bound[c], r = bound[c + 1] - bound[c];
    const size_t xo = static_cast<size_t>(r0) * K * 2;
    if (cudaMemcpyAsync(dX + xo, static_cast<const unsigned char*>(X_host) + xo, static_cast<size_t>(r) * K * 2,
                        cudaMemcpyHostToDevice, p->h2d) != cudaSuccess ||
        cudaEventRecord(p->landed[c], p->h2d) != cudaSuccess)
      st = SQ_ERR_CUDA;
  }
  for (int c = 0; c < chunks && st == SQ_OK; ++c) {
    const int64_t r0 = bound[c], r = bound[c + 1] - bound[c];
    const size_t xo = static_cast<size_t>(r0) * K * 2, yo = static_cast<size_t>(r0) * N * 2;
    if (cudaStreamWaitEvent(s, p->landed[c], 0) != cudaSuccess) {
      st = SQ_ERR_CUDA;
      break;
    }
    st = sq_linear(rot, dX + xo, r, Wq, sw, N, K, lws, lws_bytes, dY + yo, stream);
    if (st != SQ_OK) break;
    if (cudaEventRecord(p->done[c], s) != cudaSuccess || cudaStreamWaitEvent(p->d2h, p->done[c], 0) != cudaSuccess ||
        cudaMemcpyAsync(static_cast<unsigned char*>(Y_host) + yo, dY + yo, static_cast<size_t>(r) * N * 2,
                        cudaMemcpyDeviceToHost, p->d2h) != cudaSuccess)
      st = SQ_ERR_CUDA;
  }
  // Wait for all three streams whatever happened, so that no copy outlives the call.
  const bool synced = cudaStreamSynchronize(p->h2d) == cudaSuccess && cudaStreamSynchronize(s) == cudaSuccess &&
                      cudaStreamSynchronize(p->d2h) == cudaSuccess;
  if (st != SQ_OK) return st;
  return synced ? SQ_OK : SQ_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Weight-only variant and the grouped layer
// ---------------------------------------------------------------------------------------------
sq_status_t sq_pack_weight_wo(const sq_rotation_t* rot_or_null, const void* W, int64_t N, int64_t K, int32_t bits,
                              void* Wq, void* sw, void* stream) {
  if (bits != 3 && bits != 4) return SQ_ERR_INVALID_ARG;
  if (rot_or_null) {
    if (static_cast<int64_t>(rot_or_null->n1) * rot_or_null->n2 != K) return SQ_ERR_SHAPE;
    if (rot_or_null->n2 & 1) return SQ_ERR_SHAPE;
  }
  if (K % 8 != 0) return SQ_ERR_SHAPE;
  sq_status_t st = check_rows_args(W, Wq, sw, nullptr, N, K);
  if (st != SQ_OK || N == 0) return st;
  if (rot_or_null && (st = check_handle_device(rot_or_null)) != SQ_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int qmax = (1 << (bits - 1)) - 1;
  if (!rot_or_null)
    st = sq::launch_rotate_quant(nullptr, nullptr, 1, static_cast<int>(K), W, N, Wq, sw, nullptr, s, qmax);
  else if (bits == 4)
    st = sq::rotate_quant_dispatch(rot_or_null, W, N, Wq, sw, nullptr, s);
  else      // other widths: the fp32 kernel, which takes the number of levels as an argument (offline path)
    st = sq::launch_rotate_quant(rot_or_null->dR1, rot_or_null->dR2, rot_or_null->n1, rot_or_null->n2, W, N, Wq, sw,
                                 nullptr, s, qmax);
  if (st != SQ_OK) return st;
  return sq::launch_interleave_nibbles(Wq, N, K, s);
}

sq_status_t sq_rotate_act_f16(const sq_rotation_t* rot, const void* X, int64_t M, void* Z16, void* stream) {
  if (!rot) return SQ_ERR_INVALID_ARG;
  const int64_t n = static_cast<int64_t>(rot->n1) * rot->n2;
  if (rot->n2 & 1) return SQ_ERR_SHAPE;
  sq_status_t st = check_rows_args(X, Z16, Z16, nullptr, M, n);
  if (st != SQ_OK || M == 0) return st;
  if (X == Z16) return SQ_ERR_INVALID_ARG;
  if ((st = check_handle_device(rot)) != SQ_OK) return st;
  return sq::rotate_f16_dispatch(rot, X, M, Z16, static_cast<cudaStream_t>(stream));
}

namespace {
sq_status_t check_wo_gemm_args(const void* Z16, const void* Wq, const void* sw, int64_t M, int64_t N, int64_t K,
                               const void* Y) {
  if (M < 0 || N < 0 || M > kMaxRows || N > kMaxRows) return SQ_ERR_INVALID_ARG;
  if (K < 8 || (K % 8) != 0) return SQ_ERR_SHAPE;
  if (K > kMaxK) return SQ_ERR_UNSUPPORTED;
  if (M == 0 || N == 0) return SQ_OK;
  if (!Z16 || !Wq || !sw || !Y) return SQ_ERR_INVALID_ARG;
  if (!sq::aligned16(Z16) || !sq::aligned16(Wq) || !sq::aligned16(sw) || !sq::aligned16(Y)) return SQ_ERR_ALIGN;
  return SQ_OK;
}
}  // namespace

sq_status_t sq_w4a16_gemm(const void* Z16, const void* Wq, const void* sw, int64_t M, int64_t N, int64_t K, void* Y,
                          void* stream) {
  sq_status_t st = check_wo_gemm_args(Z16, Wq, sw, M, N, K, Y);
  if (st != SQ_OK || M == 0 || N == 0) return st;
  return sq::launch_wo_gemm(Z16, Wq, sw, M, N, K, Y, static_cast<cudaStream_t>(stream));
}

size_t sq_linear_wo_workspace_bytes(int64_t M, int64_t K) {
  if (M <= 0 || K <= 0) return 0;
  return align_up(static_cast<size_t>(M) * K * 2, 256);
}

sq_status_t sq_linear_wo(const sq_rotation_t* rot, const void* X, int64_t M, const void* Wq, const void* sw,
                         int64_t N, int64_t K, void* workspace, size_t workspace_bytes, void* Y, void* stream) {
  if (!rot) return SQ_ERR_INVALID_ARG;
  if (static_cast<int64_t>(rot->n1) * rot->n2 != K) return SQ_ERR_SHAPE;
  if (rot->n2 & 1) return SQ_ERR_SHAPE;
  if (M < 0 || N < 0) return SQ_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return SQ_OK;
  if (!workspace) return SQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SQ_ERR_ALIGN;
  if (workspace_bytes < sq_linear_wo_workspace_bytes(M, K)) return SQ_ERR_NOMEM;
  void* Z16 = workspace;
  sq_status_t st = check_rows_args(X, Z16, Z16, nullptr, M, K);
  if (st != SQ_OK) return st;
  if ((st = check_wo_gemm_args(Z16, Wq, sw, M, N, K, Y)) != SQ_OK) return st;
  if ((st = check_handle_device(rot)) != SQ_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = sq::rotate_f16_dispatch(rot, X, M, Z16, s);
  if (st != SQ_OK) return st;
  return sq::launch_wo_gemm(Z16, Wq, sw, M, N, K, Y, s);     // sets itself up while the rotation drains
}

sq_status_t sq_linear_grouped(const sq_rotation_t* const* rots, int32_t E, const int64_t* offsets, const void* X,
                              const void* const* Wq, const void* const* sw, int64_t N, int64_t K, void* workspace,
                              size_t workspace_bytes, void* Y, void* stream) {
  if (!rots || !offsets || !Wq || !sw || E < 1 || N < 0) return SQ_ERR_INVALID_ARG;
  if (offsets[0] != 0) return SQ_ERR_INVALID_ARG;
  for (int32_t e = 0; e < E; ++e)
    if (offsets[e + 1] < offsets[e]) return SQ_ERR_INVALID_ARG;
  const int64_t M = offsets[E];
  if (M > kMaxRows) return SQ_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return SQ_OK;
  if (!workspace || !X || !Y) return SQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SQ_ERR_ALIGN;
  if (workspace_bytes < sq_linear_workspace_bytes(M, K)) return SQ_ERR_NOMEM;
  const unsigned char* Xb = static_cast<const unsigned char*>(X);
  unsigned char* Yb = static_cast<unsigned char*>(Y);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  // Everything any expert's call would refuse is refused here, before the first kernel is queued.
  for (int32_t e = 0; e < E; ++e) {
    const int64_t r0 = offsets[e], r = offsets[e + 1] - r0;
    if (r == 0) continue;
    const sq_rotation_t* rot = rots[e];
    if (!rot) return SQ_ERR_INVALID_ARG;
    if (static_cast<int64_t>(rot->n1) * rot->n2 != K || (rot->n2 & 1)) return SQ_ERR_SHAPE;
    void* Xq = ws;
    void* sx = ws + align_up(static_cast<size_t>(r) * (K / 2), 256);
    sq_status_t st = check_rows_args(Xb + static_cast<size_t>(r0) * K * 2, Xq, sx, nullptr, r, K);
    if (st == SQ_OK) st = check_gemm_args(Xq, sx, Wq[e], sw[e], r, N, K, Yb + static_cast<size_t>(r0) * N * 2, nullptr);
    if (st == SQ_OK) st = check_handle_device(rot);
    if (st != SQ_OK) return st;
  }
  // All rows share one Xq and one sx in the workspace (row slices of Xq start on 16-byte boundaries when
  // K % 32 == 0; the kernels read and write the token steps one by one, so a slice of sx may start
  // anywhere).  Experts that share one handle (one rotation for the block's common input): steps 1 and 2 run
  // once over all rows -- one launch that fills the SMs instead of one small launch per expert; experts with
  // handles of their own: one launch each, into their rows.  A token's codes do not depend on which rows
  // are rotated with it, so the result is that of the per-expert calls.  Step 3 then runs over the experts.
  const sq_rotation_t* shared = nullptr;
  int with_rows = 0;
  bool same = true;
  for (int32_t e = 0; e < E; ++e) {
    if (offsets[e + 1] == offsets[e]) continue;
    ++with_rows;
    if (!shared) shared = rots[e];
    else if (rots[e] != shared) same = false;
  }
  if (with_rows >= 2 && K % 32 == 0) {
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned char* Xq = ws;
    unsigned char* sx = ws + align_up(static_cast<size_t>(M) * (K / 2), 256);
    sq_status_t st = SQ_OK;
    if (same) {
      st = sq::rotate_quant_dispatch(shared, X, M, Xq, sx, nullptr, s);
    } else {
      for (int32_t e = 0; e < E && st == SQ_OK; ++e) {
        const int64_t r0 = offsets[e], r = offsets[e + 1] - r0;
        if (r > 0)
          st = sq::rotate_quant_dispatch(rots[e], Xb + static_cast<size_t>(r0) * K * 2, r,
                                         Xq + static_cast<size_t>(r0) * (K / 2), sx + static_cast<size_t>(r0) * 2, nullptr, s);
      }
    }
    if (st != SQ_OK) return st;
    // Decode-sized expert batches (at most 64 rows each): step 3 for up to sixteen experts per launch, a
    // tile being (expert, 128 channels) -- one start-up and one stream of weights instead of one per expert.
    bool small = true;
    for (int32_t e = 0; e < E && small; ++e) {
      const int64_t r = offsets[e + 1] - offsets[e];
      if (r > 0 && !sq::gemm_decode_supported(r, N, K)) small = false;
    }
    // Larger expert batches: the CTA-pair kernel over up to sixteen experts per launch (one tile list: the
    // last wave of one expert's tiles no longer leaves SMs idle, and there is one start-up instead of E).
    const bool pairs = !small && sq::gemm_pair_supported(129, N, K);
    if (small || pairs) {
      const int cap = small ? sq::gemm_decode_max_groups() : sq::gemm_pair_max_groups();
      std::vector<const void*> gw, gs;
      std::vector<int64_t> g0, gr;
      auto flush = [&]() -> sq_status_t {
        if (gw.empty()) return SQ_OK;
        const sq_status_t fs =
            small ? sq::launch_w4a4_gemm_decode_grouped(Xq, sx, M, static_cast<int>(gw.size()), gw.data(), gs.data(),
                                                        g0.data(), gr.data(), static_cast<int>(N), static_cast<int>(K), Y, s)
                  : sq::launch_w4a4_gemm_pair_grouped(Xq, sx, M, static_cast<int>(gw.size()), gw.data(), gs.data(),
                                                      g0.data(), gr.data(), static_cast<int>(N), static_cast<int>(K), Y, s);
        gw.clear(); gs.clear(); g0.clear(); gr.clear();
        return fs;
      };
      for (int32_t e = 0; e < E; ++e) {
        const int64_t r0 = offsets[e], r = offsets[e + 1] - r0;
        if (r == 0) continue;
        gw.push_back(Wq[e]); gs.push_back(sw[e]); g0.push_back(r0); gr.push_back(r);
        if (static_cast<int>(gw.size()) == cap && (st = flush()) != SQ_OK) return st;
      }
      return flush();
    }
    for (int32_t e = 0; e < E; ++e) {
      const int64_t r0 = offsets[e], r = offsets[e + 1] - r0;
      if (r == 0) continue;
      st = sq::launch_w4a4_gemm(Xq + static_cast<size_t>(r0) * (K / 2), sx + static_cast<size_t>(r0) * 2, Wq[e], sw[e],
                                r, N, K, Yb + static_cast<size_t>(r0) * N * 2, nullptr, s);
      if (st != SQ_OK) return st;
    }
    return SQ_OK;
  }
  for (int32_t e = 0; e < E; ++e) {
    const int64_t r0 = offsets[e], r = offsets[e + 1] - r0;
    if (r == 0) continue;
    const sq_status_t st = sq_linear(rots[e], Xb + static_cast<size_t>(r0) * K * 2, r, Wq[e], sw[e], N, K, workspace,
                                     workspace_bytes, Yb + static_cast<size_t>(r0) * N * 2, stream);
    if (st != SQ_OK) return st;
  }
  return SQ_OK;
}

sq_status_t sq_last_device_status(void* stream) {
  return sq::read_and_clear_device_status(static_cast<cudaStream_t>(stream));
}

sq_status_t sq_debug_bounded_wait(uint32_t polls, void* stream) {
  if (polls < 1 || polls > 1000000u) return SQ_ERR_INVALID_ARG;
  sq::bounded_wait_probe_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(polls);
  sq::count_launch();
  return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

uint64_t sq_kernel_launch_count(void) { return sq::g_launches.load(std::memory_order_relaxed); }

const char* sq_status_string(sq_status_t s) {
  switch (s) {
    case SQ_OK: return "ok";
    case SQ_ERR_INVALID_ARG: return "invalid argument";
    case SQ_ERR_SHAPE: return "shape mismatch";
    case SQ_ERR_ALIGN: return "pointer not 16-byte aligned";
    case SQ_ERR_UNSUPPORTED: return "size not supported";
    case SQ_ERR_NOMEM: return "out of memory or workspace too small";
    case SQ_ERR_CUDA: return "CUDA call failed";
    case SQ_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

}  // extern "C"
