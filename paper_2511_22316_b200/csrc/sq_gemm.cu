// Step 3 of the hot path: INT4 x INT4 GEMM with int32 accumulation and the dequantisation
// (token step x channel step -> fp16) fused into the epilogue:
//   acc[t, c] = sum_k Xq[t, k] Wq[c, k],   Y[t, c] = fp16(acc * sx[t] * sw[c])
// i.e. the "NT" product Flat(X~_R) Flat(W~_R)^T on the integer codes.
//
// Tensor-core kernel (sm_100a): packed nibbles arrive by TMA into a staging ring; eight unpack
// warps widen them to int8 in shared memory, written directly in the 128-byte-swizzled K-major
// layout the UMMA descriptors expect; one thread issues tcgen05.mma kind::i8 into a TMEM int32
// accumulator; four epilogue warps read TMEM, dequantise and store fp16 while the next tile's main
// loop runs into the other accumulator buffer.
//
// Widening without arithmetic: a nibble moved to the top of a byte is the int8 value 16*code
// (two's complement keeps the sign), so  lo = (w << 4) & 0xF0F0F0F0  and  hi = w & 0xF0F0F0F0
// turn one packed word into eight int8 operands.  Both operands carry the factor 16, so the
// accumulator holds 256 * acc; the epilogue shifts it out exactly.  Within a k-block the even
// and odd channels land in different 16-byte chunks; A and B use the same permutation, which
// leaves every dot product unchanged.
#include <cuda.h>
#include <cuda_fp16.h>

#include <cstring>
#include <mutex>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {

namespace {

constexpr int BM = 128;          // tokens per tile (UMMA M)
constexpr int BK = 128;          // int4 channels per k-block: 64 packed bytes -> one 128-byte int8 row
constexpr int PACKED_ROW = BK / 2;
constexpr int UNPACK_WARPS = 8;
constexpr int EPI_WARPS = 4;
constexpr int UNPACK_THREADS = UNPACK_WARPS * 32;
constexpr int GEMM_THREADS = (2 + UNPACK_WARPS + EPI_WARPS) * 32;

enum WaitSite : uint32_t {
  SITE_STAGE_EMPTY = 1, SITE_STAGE_FULL, SITE_OP_EMPTY, SITE_OP_FULL, SITE_TMEM_FULL, SITE_TMEM_EMPTY
};

// Shared-memory plan.  The staging ring holds TMA blocks of 256 channels (128 packed bytes per
// row, 128-byte swizzle); the operand ring holds int8 k-blocks of 128 channels (one 128-byte
// swizzled row per matrix row), two per staging block.
template <int BN, int S_OP, int S_ST>
struct GemmSmem {
  static constexpr int A_OP = BM * 128;               // int8 operand tile (one k-block)
  static constexpr int B_OP = BN * 128;
  static constexpr int A_ST = BM * 128;               // packed staging tile (two k-blocks)
  static constexpr int B_ST = BN * 128;
  static constexpr int OFF_A_OP = 0;
  static constexpr int OFF_B_OP = OFF_A_OP + S_OP * A_OP;
  static constexpr int OFF_A_ST = OFF_B_OP + S_OP * B_OP;
  static constexpr int OFF_B_ST = OFF_A_ST + S_ST * A_ST;
  static constexpr int OFF_BAR = OFF_B_ST + S_ST * B_ST;
  static constexpr int NUM_BARS = 2 * S_OP + 2 * S_ST + 4;
  static constexpr int OFF_TMEM = OFF_BAR + NUM_BARS * 8;
  static constexpr int TOTAL = OFF_TMEM + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;      // slack for the 1024-byte alignment
};

// Widens half h (64 packed bytes = 128 channels) of ROWS staged rows into ROWS x 128 int8.
// Staging rows are 128 bytes with the 128-byte swizzle (16-byte chunk c of row r sits at chunk
// c ^ (r & 7)); operand rows use the same swizzle.  Even channels of the k-block go to operand
// chunks 0..3 and odd channels to chunks 4..7, for A and B alike.
// Thread t works on chunk j = t & 3 of rows r0 + 64*i, r0 = 8*(t >> 5) + ((t >> 3) & 3) + 4*((t >> 2) & 1):
// a quarter-warp covers rows {a, a+4} of one 8-row group, which makes its eight 16-byte loads
// and each of its two rounds of eight 16-byte stores fall into eight different bank groups.
template <int ROWS>
__device__ __forceinline__ void unpack_tile(const unsigned char* __restrict__ st, unsigned char* __restrict__ op,
                                            int t, int h) {
  static_assert(ROWS % 64 == 0, "tile rows must be a multiple of 64");
  constexpr int PER_THREAD = ROWS / 64;
  const int j = t & 3;
  const int r0 = ((t >> 5) << 3) + ((t >> 3) & 3) + (((t >> 2) & 1) << 2);
  const int sw = r0 & 7;
  const unsigned char* src = st + r0 * 128 + ((((h << 2) + j) ^ sw) << 4);
  unsigned char* dst_lo = op + r0 * 128 + ((j ^ sw) << 4);
  unsigned char* dst_hi = op + r0 * 128 + (((4 + j) ^ sw) << 4);
  uint4 w[PER_THREAD];
#pragma unroll
  for (int i = 0; i < PER_THREAD; ++i) w[i] = *reinterpret_cast<const uint4*>(src + i * (64 * 128));
#pragma unroll
  for (int i = 0; i < PER_THREAD; ++i) {
    uint4 lo, hi;
    lo.x = (w[i].x << 4) & 0xF0F0F0F0u; hi.x = w[i].x & 0xF0F0F0F0u;
    lo.y = (w[i].y << 4) & 0xF0F0F0F0u; hi.y = w[i].y & 0xF0F0F0F0u;
    lo.z = (w[i].z << 4) & 0xF0F0F0F0u; hi.z = w[i].z & 0xF0F0F0F0u;
    lo.w = (w[i].w << 4) & 0xF0F0F0F0u; hi.w = w[i].w & 0xF0F0F0F0u;
    *reinterpret_cast<uint4*>(dst_lo + i * (64 * 128)) = lo;
    *reinterpret_cast<uint4*>(dst_hi + i * (64 * 128)) = hi;
  }
}

// Dequantises eight accumulators (each 256 * acc, |acc| <= 2^22) of one token: exact shift, exact
// int -> float through the 1.5 * 2^23 trick (one integer add and one float subtract instead of a
// conversion instruction, whose throughput is a quarter of the ALU's), one fp32 product with the
// combined step, one rounding to fp16 (two values per cvt.rn.f16x2).
__device__ __forceinline__ uint4 dequant8(const uint32_t* r, float sxv, uint4 swraw, int32_t* a) {
  const __half2* swh = reinterpret_cast<const __half2*>(&swraw);
  uint4 out;
  uint32_t* o = reinterpret_cast<uint32_t*>(&out);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 sc = __half22float2(swh[e]);
    a[2 * e] = static_cast<int32_t>(r[2 * e]) >> 8;
    a[2 * e + 1] = static_cast<int32_t>(r[2 * e + 1]) >> 8;
    const float f0 = __int_as_float(0x4B400000 + a[2 * e]) - 12582912.0f;
    const float f1 = __int_as_float(0x4B400000 + a[2 * e + 1]) - 12582912.0f;
    const __half2 h = __floats2half2_rn(f0 * (sxv * sc.x), f1 * (sxv * sc.y));
    o[e] = *reinterpret_cast<const uint32_t*>(&h);
  }
  return out;
}

// Persistent kernel: CTA b works on tiles b, b + gridDim.x, ...; tile index = m_tile * tiles_n +
// n_tile.  Warp 0 lane 0: TMA producer.  Warp 1 lane 0: MMA issuer.  Warps 2..9: unpack.
// Warps 10..13: epilogue (TMEM -> dequant -> fp16 stores), overlapped with the next tile's main
// loop through two TMEM accumulator buffers.
template <int BN, int S_OP, int S_ST>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
w4a4_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                    const __half* __restrict__ sx, const __half* __restrict__ sw, int M, int N, int K,
                    __half* __restrict__ Y, int32_t* __restrict__ accdbg) {
  using L = GemmSmem<BN, S_OP, S_ST>;
  griddep_launch_dependents();          // a rotate kernel launched behind this one may set itself up
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* stage_full = bars;
  uint64_t* stage_empty = bars + S_ST;
  uint64_t* op_full = bars + 2 * S_ST;
  uint64_t* op_empty = bars + 2 * S_ST + S_OP;
  uint64_t* tmem_full = bars + 2 * S_ST + 2 * S_OP;        // [2]
  uint64_t* tmem_empty = tmem_full + 2;                     // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_TMEM);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = K / BK;                  // int8 k-blocks of 128 channels
  const int num_sb = (num_kb + 1) / 2;        // staging blocks of 256 channels (the last may be half used)
  const int tiles_n = (N + BN - 1) / BN, tiles_m = (M + BM - 1) / BM;
  const int num_tiles = tiles_n * tiles_m;
  const uint32_t limit = wait_limit();

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmap_x);
    tma_prefetch_desc(&tmap_w);
    for (int s = 0; s < S_ST; ++s) {
      mbar_init(&stage_full[s], 1);
      mbar_init(&stage_empty[s], UNPACK_WARPS);
    }
    for (int s = 0; s < S_OP; ++s) {
      mbar_init(&op_full[s], UNPACK_WARPS);
      mbar_init(&op_empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&tmem_full[b], 1);
      mbar_init(&tmem_empty[b], EPI_WARPS);
    }
    mbar_fence_init();
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  griddep_wait();                                     // Xq and sx may come from the kernel launched before this one

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------
    if (elect_one()) {
      uint32_t sit = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile / tiles_n) * BM, n0 = (tile % tiles_n) * BN;
        for (int sb = 0; sb < num_sb; ++sb, ++sit) {
          const int s = sit % S_ST;
          const uint32_t ph = (sit / S_ST) & 1;
          ok = mbar_wait(&stage_empty[s], ph ^ 1, SITE_STAGE_EMPTY, limit);
          if (!ok) break;
          mbar_arrive_expect_tx(&stage_full[s], L::A_ST + L::B_ST);
          tma_load_2d(smem + L::OFF_A_ST + s * L::A_ST, &tmap_x, &stage_full[s], sb * 128, m0);
          tma_load_2d(smem + L::OFF_B_ST + s * L::B_ST, &tmap_w, &stage_full[s], sb * 128, n0);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------------------
    if (elect_one()) {
      constexpr uint32_t idesc = umma_idesc(/*c=s32*/ 2, /*a=s8*/ 1, /*b=s8*/ 1, BM, BN);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tcount) {
        const uint32_t b = tcount & 1;
        ok = mbar_wait(&tmem_empty[b], ((tcount >> 1) & 1) ^ 1, SITE_TMEM_EMPTY, limit);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + b * BN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % S_OP;
          const uint32_t ph = (it / S_OP) & 1;
          ok = mbar_wait(&op_full[s], ph, SITE_OP_FULL, limit);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t a_base = smem_u32(smem + L::OFF_A_OP + s * L::A_OP);
          const uint32_t b_base = smem_u32(smem + L::OFF_B_OP + s * L::B_OP);
#pragma unroll
          for (int k = 0; k < 4; ++k) {                // 4 x (K = 32 int8) per 128-byte row
            umma_i8(tmem_d, umma_desc_sw128(a_base + k * 32), umma_desc_sw128(b_base + k * 32), idesc,
                    (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&op_empty[s]);                    // frees the operand stage when the MMAs retire
        }
        umma_commit(&tmem_full[b]);                     // accumulator complete (or abandoned)
      }
    }
  } else if (warp < 2 + UNPACK_WARPS) {
    // ------------------------------ unpack warps --------------------------------------------
    const int t = threadIdx.x - 64;                    // 0 .. UNPACK_THREADS-1
    uint32_t it = 0, sit = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      for (int sb = 0; sb < num_sb && ok; ++sb, ++sit) {
        const int ss = sit % S_ST;
        ok = mbar_wait(&stage_full[ss], (sit / S_ST) & 1, SITE_STAGE_FULL, limit);
        if (!ok) break;
        for (int h = 0; h < 2 && 2 * sb + h < num_kb; ++h, ++it) {
          const int s = it % S_OP;
          ok = mbar_wait(&op_empty[s], ((it / S_OP) & 1) ^ 1, SITE_OP_EMPTY, limit);
          if (!ok) break;
          unpack_tile<BM>(smem + L::OFF_A_ST + ss * L::A_ST, smem + L::OFF_A_OP + s * L::A_OP, t, h);
          unpack_tile<BN>(smem + L::OFF_B_ST + ss * L::B_ST, smem + L::OFF_B_OP + s * L::B_OP, t, h);
          fence_proxy_async_smem();                     // generic-proxy stores -> visible to the MMA
          __syncwarp();
          if (lane == 0) mbar_arrive(&op_full[s]);
        }
        if (!ok) break;
        __syncwarp();
        if (lane == 0) mbar_arrive(&stage_empty[ss]);
      }
    }
  } else {
    // ------------------------------ epilogue warps ------------------------------------------
    const int quarter = warp & 3;                       // TMEM lanes this warp may read
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tcount) {
      const int m0 = (tile / tiles_n) * BM, n0 = (tile % tiles_n) * BN;
      const uint32_t b = tcount & 1;
      ok = mbar_wait(&tmem_full[b], (tcount >> 1) & 1, SITE_TMEM_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      const int row = m0 + quarter * 32 + lane;
      const float sxv = (row < M) ? __half2float(sx[row]) : 0.0f;
      const uint32_t tmem_d = tmem_base + b * BN + (static_cast<uint32_t>(quarter * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem_d + c * 32, r);
        tmem_wait_ld();
        const int col0 = n0 + c * 32;
        if (row < M && col0 < N) {
          __half* yrow = Y + static_cast<size_t>(row) * N + col0;
          int32_t* arow = accdbg ? accdbg + static_cast<size_t>(row) * N + col0 : nullptr;
#pragma unroll
          for (int g = 0; g < 4; ++g) {                 // groups of 8 columns (N % 8 == 0)
            if (col0 + g * 8 < N) {
              const uint4 swraw = __ldg(reinterpret_cast<const uint4*>(sw + col0 + g * 8));
              int32_t a[8];
              *reinterpret_cast<uint4*>(yrow + g * 8) = dequant8(&r[g * 8], sxv, swraw, a);
              if (arow) {
                *reinterpret_cast<int4*>(arow + g * 8) = make_int4(a[0], a[1], a[2], a[3]);
                *reinterpret_cast<int4*>(arow + g * 8 + 4) = make_int4(a[4], a[5], a[6], a[7]);
              }
            }
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[b]);       // this warp's quarter of the buffer is drained
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 2 * BN);
  }
}

// Plain integer kernel for shapes the tensor-core path does not take (K % 128 != 0, N % 8 != 0):
// one thread per output, byte-wise; gridDim.y strides over the token rows (a grid's y extent stops
// at 65535).  Same results, bit for bit.
__global__ void w4a4_gemm_simple_kernel(const uint8_t* __restrict__ Xq, const __half* __restrict__ sx,
                                        const uint8_t* __restrict__ Wq, const __half* __restrict__ sw,
                                        int M, int N, int K, __half* __restrict__ Y, int32_t* __restrict__ accdbg) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= N) return;
  const uint8_t* b = Wq + static_cast<size_t>(c) * (K / 2);
  const float swv = __half2float(sw[c]);
  for (int t = blockIdx.y; t < M; t += gridDim.y) {
    const uint8_t* a = Xq + static_cast<size_t>(t) * (K / 2);
    int32_t acc = 0;
    for (int j = 0; j < K / 2; ++j) {
      const int av = a[j], bv = b[j];
      const int a0 = (av << 28) >> 28, a1 = (av << 24) >> 28;      // sign-extended nibbles
      const int b0 = (bv << 28) >> 28, b1 = (bv << 24) >> 28;
      acc += a0 * b0 + a1 * b1;
    }
    const float s = __half2float(sx[t]) * swv;
    Y[static_cast<size_t>(t) * N + c] = __float2half_rn(static_cast<float>(acc) * s);
    if (accdbg) accdbg[static_cast<size_t>(t) * N + c] = acc;
  }
}

// ---------------------------------------------------------------------------------------------
// Tensor maps (driver entry point fetched at run time, so the library has no link-time
// dependency on libcuda and still loads on a machine without a driver).
// ---------------------------------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn driver_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// A tensor map is a pure function of the arguments it is encoded from, and a layer that is evaluated
// again and again asks for the same few maps every time (same buffers, same shapes).  Each host thread
// keeps the maps it encoded last, keyed by all of the arguments, so that a steady-state call encodes
// nothing: the driver call costs about a microsecond per map, several per layer call.
struct MapKey {
  const void* base;
  cuuint64_t dims[3], strides[2];
  cuuint32_t box[3], estr[3];
  int dtype, rank, interleave, swizzle, promo, oob;
};
struct MapEntry {
  bool valid = false;
  MapKey key;
  CUtensorMap map;
};

CUresult cached_encode(CUtensorMap* out, CUtensorMapDataType dtype, cuuint32_t rank, void* base,
                       const cuuint64_t* dims, const cuuint64_t* strides, const cuuint32_t* box,
                       const cuuint32_t* estr, CUtensorMapInterleave interleave, CUtensorMapSwizzle swizzle,
                       CUtensorMapL2promotion promo, CUtensorMapFloatOOBfill oob) {
  EncodeTiledFn enc = driver_encode_fn();
  if (!enc) return CUDA_ERROR_NOT_SUPPORTED;
  if (rank < 1 || rank > 3) return enc(out, dtype, rank, base, dims, strides, box, estr, interleave, swizzle, promo, oob);
  constexpr int kEntries = 128;
  thread_local MapEntry cache[kEntries];
  MapKey key;
  std::memset(&key, 0, sizeof(key));
  key.base = base;
  for (cuuint32_t d = 0; d < rank; ++d) {
    key.dims[d] = dims[d];
    key.box[d] = box[d];
    key.estr[d] = estr[d];
    if (d + 1 < rank) key.strides[d] = strides[d];
  }
  key.dtype = static_cast<int>(dtype);
  key.rank = static_cast<int>(rank);
  key.interleave = static_cast<int>(interleave);
  key.swizzle = static_cast<int>(swizzle);
  key.promo = static_cast<int>(promo);
  key.oob = static_cast<int>(oob);
  uint64_t hsh = reinterpret_cast<uintptr_t>(base) >> 8;
  hsh = (hsh ^ (hsh >> 17)) * 0x9E3779B97F4A7C15ull + key.dims[rank - 1] * 31 + key.box[rank - 1] * 7 + key.box[0];
  MapEntry& e = cache[(hsh >> 20) % kEntries];
  if (e.valid && std::memcmp(&e.key, &key, sizeof(key)) == 0) {
    *out = e.map;
    return CUDA_SUCCESS;
  }
  const CUresult r = enc(out, dtype, rank, base, dims, strides, box, estr, interleave, swizzle, promo, oob);
  if (r == CUDA_SUCCESS) {
    e.valid = true;
    e.key = key;
    e.map = *out;
  }
  return r;
}

// The encoder every launcher uses (nullptr when the driver entry point is missing).
EncodeTiledFn get_encode_fn() { return driver_encode_fn() ? &cached_encode : nullptr; }

// 2-D uint8 map over a packed [rows x row_bytes] matrix; box = box_rows x 128 bytes with the
// 128-byte swizzle; out-of-range rows and bytes read as zero.
bool make_packed_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t row_bytes, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[2] = {row_bytes, rows};
  const cuuint64_t strides[1] = {row_bytes};
  const cuuint32_t box[2] = {128, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int S_OP, int S_ST>
sq_status_t launch_tc(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N, int K, void* Y,
                      int32_t* accdbg, cudaStream_t s) {
  using L = GemmSmem<BN, S_OP, S_ST>;
  CUtensorMap mx, mw;
  if (!make_packed_map(&mx, Xq, M, K / 2, BM) || !make_packed_map(&mw, Wq, N, K / 2, BN)) return SQ_ERR_CUDA;
  auto kern = w4a4_gemm_tc_kernel<BN, S_OP, S_ST>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), L::DYN_BYTES)) return SQ_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const int tiles = ((N + BN - 1) / BN) * ((M + BM - 1) / BM);
  const int grid = tiles < sms ? tiles : sms;
  const cudaError_t err = launch_maybe_pdl(kern, dim3(grid), dim3(GEMM_THREADS), L::DYN_BYTES, s, mx, mw,
                                           static_cast<const __half*>(sx), static_cast<const __half*>(sw), M, N, K,
                                           static_cast<__half*>(Y), accdbg);
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace

// One or two tokens are pure streaming: dot products on the CUDA cores.  With three or four the
// dot-product kernel is bound by its dp4a and shared-memory issue and the tensor-core decode kernel
// (whose time does not depend on M up to 16) is as fast or faster, where it supports the shape.
static bool use_gemv(int64_t M, int64_t N, int64_t K) {
  return gemv_supported(M, N, K) && (M <= 2 || !gemm_decode_supported(M, N, K));
}

sq_status_t launch_w4a4_gemm(const void* Xq, const void* sx, const void* Wq, const void* sw, int64_t M, int64_t N,
                             int64_t K, void* Y, int32_t* accdbg, cudaStream_t s) {
  if (M == 0 || N == 0) return SQ_OK;
  if (use_gemv(M, N, K)) return launch_w4a4_gemv(Xq, sx, Wq, sw, (int)M, (int)N, (int)K, Y, accdbg, s);
  if (gemm_decode_supported(M, N, K))
    return launch_w4a4_gemm_decode(Xq, sx, Wq, sw, (int)M, (int)N, (int)K, Y, accdbg, s);
  const bool tc_ok = (K % BK == 0) && (N % 8 == 0) && K >= BK;
  if (gemm_pair_supported(M, N, K))
    return launch_w4a4_gemm_pair(Xq, sx, Wq, sw, (int)M, (int)N, (int)K, Y, accdbg, s);
  if (M > 64 && M <= 128 && gemm_decode_supported(64, N, K)) {
    // 65 to 128 tokens: the CTA-pair kernel with its tile half empty, or the decode kernel twice
    // (64 tokens, then the rest; the weights are read twice).  Estimates in microseconds from
    // measured rates: a 256-channel block costs a pair 0.54 and a decode CTA 0.46; fixed costs 6
    // and 8 per launch.  The pair kernel wins when its 256-channel tiles fill the 74 pairs or K is
    // short; the decode kernel wins on long K with few output channels (it splits K).
    const int sms = sm_count();
    if (sms <= 0) return SQ_ERR_CUDA;
    const int num_sb = static_cast<int>((K / 128 + 1) / 2);
    const int pair_tiles = static_cast<int>((N + 255) / 256), pairs = sms / 2 > 0 ? sms / 2 : 1;
    const double pair_us = 6.0 + 0.54 * num_sb * ((pair_tiles + pairs - 1) / pairs);
    const int dec_tiles = static_cast<int>((N + 127) / 128);
    int split = 1;
    while (split < 8 && dec_tiles * split * 2 <= sms && num_sb / (split * 2) >= 2) split *= 2;
    const int clusters = sms / split > 0 ? sms / split : 1;
    const double dec_us = 2.0 * (8.0 + 0.46 * ((num_sb + split - 1) / split) * ((dec_tiles + clusters - 1) / clusters));
    if (pair_us <= dec_us) return launch_w4a4_gemm_pair(Xq, sx, Wq, sw, (int)M, (int)N, (int)K, Y, accdbg, s);
    const sq_status_t st = launch_w4a4_gemm_decode(Xq, sx, Wq, sw, 64, (int)N, (int)K, Y, accdbg, s);
    if (st != SQ_OK) return st;
    const size_t half = 64;
    return launch_w4a4_gemm_decode(static_cast<const unsigned char*>(Xq) + half * (K / 2),
                                   static_cast<const __half*>(sx) + half, Wq, sw, (int)(M - 64), (int)N, (int)K,
                                   static_cast<__half*>(Y) + half * N, accdbg ? accdbg + half * N : nullptr, s);
  }
  if (tc_ok) {
    if (N >= 256 && M > 64)
      return launch_tc<256, 2, 2>(Xq, sx, Wq, sw, (int)M, (int)N, (int)K, Y, accdbg, s);
    return launch_tc<128, 3, 3>(Xq, sx, Wq, sw, (int)M, (int)N, (int)K, Y, accdbg, s);
  }
  dim3 block(128), grid((unsigned)((N + 127) / 128), (unsigned)(M < 65535 ? M : 65535));
  w4a4_gemm_simple_kernel<<<grid, block, 0, s>>>(static_cast<const uint8_t*>(Xq), static_cast<const __half*>(sx),
                                                 static_cast<const uint8_t*>(Wq), static_cast<const __half*>(sw),
                                                 (int)M, (int)N, (int)K, static_cast<__half*>(Y), accdbg);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace sq
