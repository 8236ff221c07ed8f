/*
 * singlequant.h - C ABI of the B200 (sm_100a) W4A4 linear hot path of SingleQuant.
 *
 * The path (paper, Section "SingleQuant"):
 *   step 1  Kronecker rotation of every activation token: the length-n row is viewed as an
 *           n1 x n2 row-major matrix X~_t and Z_t = R1^T X~_t R2       (Eq. "eq18", and the
 *           per-slice form of the mode products that follows it);
 *   step 2  per-token symmetric INT4 quantisation Q_Delta(z) = Delta*floor(z/Delta + 1/2)
 *           (Section 3.2) with Delta_t = fp16(max|Z_t| / 7), two codes per byte;
 *   step 3  INT4 x INT4 GEMM against weights rotated offline by the same operator
 *           (Flat(W~_R) = W^T R), int32 accumulation, dequantisation by token step x channel
 *           step to fp16                                  (X W = Flat(X~_R) Flat(W~_R)^T).
 *
 * General conventions
 *   - Pointers marked HOST are ordinary host memory; pointers marked DEVICE are CUDA device
 *     memory of the device that was current when the rotation handle was created.  A call that
 *     takes a handle while another device is current returns SQ_ERR_INVALID_ARG.  The
 *     caller owns every buffer; the library allocates only the sq_rotation_t handle (and the
 *     device copies of R1, R2 inside it), freed by sq_rotation_destroy.
 *   - All matrices are dense row-major.  X is [M x n] (one token per row, ld = n), W is
 *     [N x K] with K = n (one OUTPUT channel per row), Y is [M x N].
 *   - Packed INT4 layout (public, canonical): row r, byte j holds channel 2j in its low nibble
 *     and channel 2j+1 in its high nibble, two's complement, row stride K/2 bytes.
 *   - Steps (scales) are IEEE fp16.  The step used to quantise is the ROUNDED fp16 value.
 *   - DEVICE pointers must be 16-byte aligned; K (= n) must be even.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Device
 *     calls only enqueue work and never synchronise, except where stated.
 *   - Every call validates its arguments on the host before any launch and reports problems
 *     through the return code; nothing throws, aborts or traps.  M = 0 or N = 0 is SQ_OK and
 *     a no-op.
 *   - Kernels wait on hardware barriers with bounded spins; a wait that runs out sets a
 *     device status word that sq_last_device_status returns as SQ_ERR_TIMEOUT.
 */
#ifndef SINGLEQUANT_H_
#define SINGLEQUANT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SQ_OK = 0,
  SQ_ERR_INVALID_ARG = 1,   /* NULL pointer, negative size, bad flag                         */
  SQ_ERR_SHAPE = 2,         /* n1*n2 != n, odd K, K mismatch with the rotation, ...          */
  SQ_ERR_ALIGN = 3,         /* a DEVICE pointer is not 16-byte aligned                       */
  SQ_ERR_UNSUPPORTED = 4,   /* a size beyond what the kernels handle (stated per call)       */
  SQ_ERR_NOMEM = 5,         /* allocation of the handle failed / workspace too small         */
  SQ_ERR_CUDA = 6,          /* a CUDA runtime or driver call failed                          */
  SQ_ERR_TIMEOUT = 7        /* a bounded device-side wait ran out (see sq_last_device_status) */
} sq_status_t;

typedef struct sq_rotation sq_rotation_t;   /* opaque: host + device copies of R1 and R2 */

/* Components of R = (R1^U R^A)^T (x) (H R2^U); a cleared bit replaces that component by the
 * identity (the paper's ablation of ART and URT). */
enum { SQ_ROT_ART = 1, SQ_ROT_URT = 2, SQ_ROT_HADAMARD = 4, SQ_ROT_DEFAULT = 7 };
/* Repeated ART rotations (paragraph "Effect of ART Steps"): OR this into `flags` to apply k >= 1
 * ART steps (k <= 2048); each step after the first is the closed-form Givens rotation of Lemma 1
 * in the plane (outlier, minimum) of the column as rotated so far.  The paper finds one step
 * sufficient; the default is one. */
#define SQ_ROT_ART_STEPS(k) ((uint32_t)((k) - 1) << 8)
/* A handle made by sq_build_rotation knows how R2 = H R2^U was composed.  With this bit in `flags`
 * (and n2 = 64 or 128, n1 <= 128) the kernel of steps 1+2 applies R2 piece by piece in fp32 registers
 * -- Hadamard butterflies, then the two chains of plane rotations of URT in closed form -- instead of
 * as a dense matrix on the tensor cores: the same operator with about a tenth of the multiply-adds.
 * Without the bit (the default, and always for handles made by sq_rotation_from_factors) R2 is applied
 * as the dense matrix, which measures as fast or faster on a B200 at every benchmark shape (the
 * structured form trades idle tensor cores for busy arithmetic pipes). */
#define SQ_ROT_APPLY_STRUCTURED (1u << 20)
/* With this bit in `flags`, sq_linear (and sq_linear_static / sq_linear_host) evaluate batches of up to
 * 64 tokens as ONE launch: some CTAs of the grid rotate and quantise the tokens while the others, CTAs
 * of the decode GEMM, already pull their weights in, and the packed tokens are handed over through L2
 * behind a device counter instead of through the end of a kernel.  Same results bit for bit.  Off by
 * default: on a B200 the two-kernel form, whose GEMM is launched as a programmatic dependent of the
 * rotate kernel, measures as fast or faster at the benchmark's decode shapes.  A handle built with this
 * bit keeps 64 pairs of device counters; calls that use one handle concurrently from more than 64
 * streams at a time would share a pair.  After SQ_ERR_TIMEOUT such a handle should be destroyed (a
 * counter may be left non-zero). */
#define SQ_ROT_FUSE_DECODE (1u << 21)

/* Algorithm 1 (Kronecker Dimension Factorization).  Host only.  n2 = the power of two dividing
 * n closest to sqrt(n), the first found winning ties; n1 = n / n2.  n >= 1. */
sq_status_t sq_factorize(int64_t n, int32_t* n1, int32_t* n2);

/* Builds R1 = (R1^U R^A)^T [n1 x n1] and R2 = H R2^U [n2 x n2] (paragraphs "Alignment Rotation
 * Transformation", "Uniformity Rotation Transformation", "The Overall SingleQuant Method") in
 * float64 on the host from one calibration batch, stores them as fp32, copies them to the
 * current device and returns a handle.  Host-synchronous.
 *   calib      HOST fp32 [T x n] row-major, T >= 1
 *   n1, n2     n1*n2 == n; n2 must be a power of two when SQ_ROT_HADAMARD is set
 *   flags      SQ_ROT_* bits
 *   seed       seeds the library's own generator for the random orthogonal block O of ART when
 *              O_or_null is NULL
 *   O_or_null  HOST fp64 [(n1-2) x (n1-2)] orthogonal block for ART, or NULL
 *   out        receives the handle
 * The vectors ART/URT are built from: the calibration token with the largest |entry| is
 * reshaped to n1 x n2; ART and URT_1 use the column holding that entry; URT_2 uses the row of
 * the left-rotated token with the largest |entry|, after the Hadamard mix. */
sq_status_t sq_build_rotation(const float* calib, int64_t T, int64_t n, int32_t n1, int32_t n2,
                              uint32_t flags, uint64_t seed, const double* O_or_null,
                              sq_rotation_t** out);

/* Wraps caller-made factors (HOST fp32, row-major, R1 [n1 x n1], R2 [n2 x n2]) in a handle.
 * No orthogonality check is made. */
sq_status_t sq_rotation_from_factors(const float* R1, const float* R2, int32_t n1, int32_t n2,
                                     sq_rotation_t** out);

/* Copies the fp32 factors back to HOST buffers of n1*n1 and n2*n2 floats. */
sq_status_t sq_rotation_get_factors(const sq_rotation_t* rot, float* R1, float* R2);
sq_status_t sq_rotation_dims(const sq_rotation_t* rot, int32_t* n1, int32_t* n2);
/* 1 when steps 1+2 with this handle apply R2 through its composition (see SQ_ROT_APPLY_STRUCTURED), 0 when
 * they apply it as a dense matrix (also for a NULL handle). */
int32_t sq_rotation_is_structured(const sq_rotation_t* rot);
void sq_rotation_destroy(sq_rotation_t* rot);

/* Steps 1+2, fused: Z_t = R1^T X~_t R2 in fp32 on chip, Delta_t = fp16(max|Z_t|/7),
 * code = clamp(floor(fl(fl(z * fl(1/Delta)) + 0.5)), -8, 7) in fp32 arithmetic, packed.
 *   rot           handle; n = n1*n2 of the handle.  Supported: n2 even (SQ_ERR_SHAPE otherwise),
 *                 n <= 32768.
 *   X             DEVICE fp16 [M x n]
 *   Xq            DEVICE uint8 [M x n/2]   (out)
 *   sx            DEVICE fp16 [M]          (out; Delta_t; 0 for an all-zero row)
 *   Zdbg_or_null  DEVICE fp32 [M x n]      (out, optional: the rotated rows, for parity tests) */
sq_status_t sq_rotate_quant_act(const sq_rotation_t* rot, const void* X, int64_t M,
                                void* Xq, void* sx, void* Zdbg_or_null, void* stream);

/* Offline weight path: the same operator on the rows of W (Flat(W~_R) = W^T R), then
 * round-to-nearest INT4 with one step per output channel.
 *   rot_or_null   NULL = identity rotation (plain per-channel INT4)
 *   W             DEVICE fp16 [N x K], K == n of the handle
 *   Wq            DEVICE uint8 [N x K/2]   (out)
 *   sw            DEVICE fp16 [N]          (out) */
sq_status_t sq_pack_weight(const sq_rotation_t* rot_or_null, const void* W, int64_t N, int64_t K,
                           void* Wq, void* sw, void* stream);

/* Step 3: acc[t,c] = sum_k Xq[t,k] * Wq[c,k] (int32, exact), Y[t,c] = fp16(acc * sx[t] * sw[c]).
 *   Xq  DEVICE uint8 [M x K/2]     sx  DEVICE fp16 [M]
 *   Wq  DEVICE uint8 [N x K/2]     sw  DEVICE fp16 [N]
 *   Y   DEVICE fp16  [M x N] (out)
 *   accdbg_or_null  DEVICE int32 [M x N] (out, optional: the raw accumulators)
 * No scratch memory: every kernel keeps its intermediates on chip (split-K partial tiles are
 * exchanged through cluster shared memory).
 * Supported: K even, K <= 65536 (so that the 256x-scaled int32 accumulator cannot overflow).
 * The tensor-core path needs K % 128 == 0 and N % 8 == 0; other shapes run a plain integer
 * kernel with the same results.
 * Ordering: the kernel is queued as a programmatic dependent of the kernel before it in `stream`: it
 * may request its first blocks of Wq while that kernel still runs, and waits for it before it reads Xq
 * or sx or writes Y.  Weights packed by sq_pack_weight / sq_pack_weight_wo on the same stream are
 * complete by then (those calls end with an ordinary kernel).  A caller that produces Wq with a
 * kernel of its own which lets dependents start early must not let it do so before Wq is written. */
sq_status_t sq_w4a4_gemm(const void* Xq, const void* sx, const void* Wq, const void* sw,
                         int64_t M, int64_t N, int64_t K, void* Y, void* accdbg_or_null,
                         void* stream);

/* The whole layer on one stream: steps 1+2 into the workspace (Xq, sx), then step 3.
 *   workspace  DEVICE, at least sq_linear_workspace_bytes(M, K) bytes, 256-byte aligned
 * Every argument of both halves is validated before the first kernel is queued. */
size_t sq_linear_workspace_bytes(int64_t M, int64_t K);
sq_status_t sq_linear(const sq_rotation_t* rot, const void* X, int64_t M,
                      const void* Wq, const void* sw, int64_t N, int64_t K,
                      void* workspace, size_t workspace_bytes, void* Y, void* stream);

/* sq_linear without a caller workspace and without any allocation on the call path.
 * (The paper has no counterpart: this is a deployment variant of sq_linear.)
 *
 * For callers that cannot obtain device memory where they evaluate a layer: a serving loop that
 * must stay out of cudaMalloc (which synchronises the device and may fail under memory pressure),
 * a plugin that is handed input and output tensors by its host framework but no allocator, a
 * process whose device memory is already split into fixed pools.  The packed activations and
 * their steps go to a scratch array of SQ_LINEAR_STATIC_SCRATCH_BYTES that is part of the library
 * image; every GPU that loads the library holds it until the process exits.
 *   - Arguments as sq_linear, minus the workspace.  All pointers DEVICE; the caller owns X, Wq,
 *     sw and Y.
 *   - Limit: sq_linear_workspace_bytes(M, K) <= SQ_LINEAR_STATIC_SCRATCH_BYTES, i.e. roughly
 *     M * K / 2 + 2 * M bytes (LLaMA-2-7B prefill, 2048 x 4096, needs 4.2 MB).  Larger problems
 *     return SQ_ERR_UNSUPPORTED before anything is launched: split M, or use sq_linear.
 *   - The first call on each device looks up the scratch's device address (a CUDA runtime query,
 *     no allocation).  Make that first call outside any stream capture; later calls only launch.
 *   - The call itself never calls cudaMalloc, cudaFree or any allocating routine.
 *   - One array serves every call on a device, and it keeps what the last call wrote.  Nothing in
 *     it needs clearing (each call rewrites all it reads), but two calls that overlap on the GPU
 *     (different streams, or two host threads) race on it: serialise them, e.g. on one stream. */
#define SQ_LINEAR_STATIC_SCRATCH_BYTES (8u << 20)
sq_status_t sq_linear_static(const sq_rotation_t* rot, const void* X, int64_t M,
                             const void* Wq, const void* sw, int64_t N, int64_t K,
                             void* Y, void* stream);

/* The whole layer from HOST activations to HOST outputs: copies X (HOST fp16 [M x n], pinned
 * memory recommended) to the device, runs sq_linear, copies Y back (HOST fp16 [M x N]) and
 * waits for the stream.  Weights stay on the device.  Batches of 512 rows or more are cut into up
 * to four chunks whose copies in, computation and copies out overlap (two internal copy streams
 * and a few events per device, created at the first such call and kept until exit; both are
 * ordered after the work already queued on `stream`).  The result does not depend on the cut:
 * every row is rotated, quantised and multiplied on its own.  Concurrent calls on one device
 * share those copy streams and therefore serialise.
 *   workspace  DEVICE, at least sq_linear_host_workspace_bytes(M, N, K) bytes */
size_t sq_linear_host_workspace_bytes(int64_t M, int64_t N, int64_t K);
sq_status_t sq_linear_host(const sq_rotation_t* rot, const void* X_host, int64_t M,
                           const void* Wq, const void* sw, int64_t N, int64_t K,
                           void* workspace, size_t workspace_bytes, void* Y_host, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Weight-only variant (Appendix "Weight-only Quantization", Table "wquant": W4A16 and W3A16): the
 * same rotation, weights quantised to b = 4 or 3 bits with one step per output channel, activations
 * left in 16 bits.  The paper states the setting only; taken here: the activations are rotated
 * online as in the W4A4 path and rounded once to fp16; a b-bit code is the W4A4 quantiser with 7
 * replaced by 2^(b-1) - 1 and the clamp by [-2^(b-1), 2^(b-1) - 1]; the product is accumulated in
 * fp32 and rounded once to fp16.
 *
 * Storage of the codes ("weight-only order"): one two's-complement nibble per code, for 3 bits too
 * (the codes then lie in [-4, 3]; the 25 % a 3-bit packing would save is not taken).  Within every
 * eight consecutive channels, read as a little-endian 32-bit word, nibble position i (bits 4i..4i+3)
 * holds channel (0, 2, 4, 6, 1, 3, 5, 7)[i]: (word >> 4s) & 0x000F000F is then the pair of channels
 * (2s, 2s+1) in the two 16-bit halves, which is what the kernel widens to a half2.  This differs from
 * the channel order sq_pack_weight writes for the W4A4 path; the two formats are not interchangeable.
 * ------------------------------------------------------------------------------------------- */

/* Offline: rotate the rows of W, quantise to `bits` (4 or 3; else SQ_ERR_INVALID_ARG), store in the
 * weight-only order.  K % 8 == 0 (SQ_ERR_SHAPE otherwise).
 *   rot_or_null   NULL = identity rotation
 *   W             DEVICE fp16 [N x K], K == n of the handle
 *   Wq            DEVICE uint8 [N x K/2]   (out)
 *   sw            DEVICE fp16 [N]          (out; Delta_c = fp16(max|row| / (2^(bits-1) - 1))) */
sq_status_t sq_pack_weight_wo(const sq_rotation_t* rot_or_null, const void* W, int64_t N, int64_t K,
                              int32_t bits, void* Wq, void* sw, void* stream);

/* Step 1 alone: Z16_t = fp16(R1^T X~_t R2), the rotation accurate to fp32 on chip, one rounding.
 *   X    DEVICE fp16 [M x n]        Z16  DEVICE fp16 [M x n] (out; may not alias X)
 * Supported sizes as sq_rotate_quant_act. */
sq_status_t sq_rotate_act_f16(const sq_rotation_t* rot, const void* X, int64_t M, void* Z16, void* stream);

/* Step 3 of the variant: Y[t,c] = fp16((sum_k Z16[t,k] * code[c,k]) * sw[c]), fp32 accumulation.
 *   Z16 DEVICE fp16 [M x K]      Wq DEVICE uint8 [N x K/2] (weight-only order)     sw DEVICE fp16 [N]
 *   Y   DEVICE fp16 [M x N] (out)
 * K % 8 == 0, K <= 65536.  The tensor-core path needs K % 64 == 0 and N % 8 == 0; other shapes run a
 * plain fp32 kernel (same definition, another summation order). */
sq_status_t sq_w4a16_gemm(const void* Z16, const void* Wq, const void* sw, int64_t M, int64_t N, int64_t K,
                          void* Y, void* stream);

/* The weight-only layer on one stream: rotation into the workspace (Z16), then the product.
 *   workspace  DEVICE, at least sq_linear_wo_workspace_bytes(M, K) bytes, 256-byte aligned
 * Every argument of both halves is validated before the first kernel is queued. */
size_t sq_linear_wo_workspace_bytes(int64_t M, int64_t K);
sq_status_t sq_linear_wo(const sq_rotation_t* rot, const void* X, int64_t M, const void* Wq, const void* sw,
                         int64_t N, int64_t K, void* workspace, size_t workspace_bytes, void* Y, void* stream);

/* The W4A4 layer of a mixture-of-experts block (Section "Results on Mixtral Models": the method is
 * applied to each expert's linear layers).  The tokens are sorted by expert: expert e owns rows
 * offsets[e] .. offsets[e+1]-1 of X and of Y and has its own packed weights and its own rotation
 * handle (experts that share an input distribution may share a handle).  Each expert's rows go
 * through the same kernels as sq_linear, queued back to back on `stream`; experts without tokens
 * cost nothing.  With K % 32 == 0, steps 1 and 2 run once over all M rows when every expert with
 * tokens has the SAME handle (else once per expert), and step 3 runs over up to sixteen experts per
 * launch (one list of tiles over the experts); the outputs are the same bits as those of sq_linear
 * on each expert's rows.
 *   rots          HOST array of E handles (all with n1*n2 == K)
 *   offsets       HOST array of E+1 non-decreasing row offsets, offsets[0] == 0, offsets[E] == M
 *   X             DEVICE fp16 [M x K]
 *   Wq, sw        HOST arrays of E DEVICE pointers: uint8 [N x K/2] and fp16 [N] per expert
 *   workspace     DEVICE, at least sq_linear_workspace_bytes(M, K) bytes, 256-byte aligned (shared by
 *                 the experts, which run one after the other)
 *   Y             DEVICE fp16 [M x N] (out)
 * Every expert's slice must start on a 16-byte boundary (K % 8 == 0 and N % 8 == 0 make every offset
 * valid; otherwise SQ_ERR_ALIGN).  All arguments are validated before the first kernel is queued. */
sq_status_t sq_linear_grouped(const sq_rotation_t* const* rots, int32_t E, const int64_t* offsets,
                              const void* X, const void* const* Wq, const void* const* sw, int64_t N, int64_t K,
                              void* workspace, size_t workspace_bytes, void* Y, void* stream);

/* Synchronises `stream`, then returns and clears the device status word: SQ_OK, or
 * SQ_ERR_TIMEOUT if any kernel since the last call gave up a bounded wait, or SQ_ERR_CUDA. */
sq_status_t sq_last_device_status(void* stream);

/* Diagnostic (the paper has no counterpart): enqueues a one-thread kernel that waits, with the
 * same bounded-wait routine the production kernels use, on a hardware barrier that nothing ever
 * completes, for `polls` polls (1 .. 1000000), and then gives up.  Nothing else is in flight in
 * that kernel.  A following sq_last_device_status(stream) therefore returns SQ_ERR_TIMEOUT once
 * and SQ_OK afterwards, and the context stays usable: this is how the time-out reporting path is
 * checked without hanging or faulting anything. */
sq_status_t sq_debug_bounded_wait(uint32_t polls, void* stream);

/* Number of kernels this library has launched in the calling process (monotonic counter). */
uint64_t sq_kernel_launch_count(void);

const char* sq_status_string(sq_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* SINGLEQUANT_H_ */
