// Step 3 for prefill-sized problems: the INT4 x INT4 GEMM on CTA pairs (tcgen05 cta_group::2).
//
// Two CTAs of a cluster share one 256 x 256 output tile: CTA r owns token rows [128 r, 128 r + 128)
// of the tile (its TMEM lanes) and stages weight rows [128 r, 128 r + 128) of the tile (its half
// of the B operand), so every widened weight byte is written to shared memory once per pair and
// feeds both SMs' tensor cores.  The activation codes never pass through shared memory as int8:
// four warps read the packed bytes of "their" token row, widen them in registers and store the
// int8 operand straight into tensor memory (tcgen05.st), from where the MMA takes its A operand.
//
// Pipeline per CTA (block = 256 channels = 128 packed bytes per row = two k-blocks of 128):
//   warp 0        TMA: packed A rows and packed B rows, one block per staging stage
//   warps 2..5    A: staging -> registers -> widen -> TMEM ring stage        } arrive on the
//   warps 6..9    B: staging -> registers -> widen -> swizzled operand ring  } leader's full[s]
//   warp 1        (leader CTA only) 8 MMAs of K = 32 per block; commit frees the ring stage in
//                 both CTAs; the last commit of a tile publishes the accumulator to both CTAs
//   warps 10..25  epilogue: TMEM -> dequantise -> fp16 tile in shared memory -> TMA store (which
//                 also clips the ragged edges); four warps per TMEM lane quarter, two 32-column
//                 chunks each, so that the single accumulator is handed back after one chunk's
//                 worth of work and the next tile's MMAs wait as briefly as possible
// Every hand-over costs each warp a few hundred cycles of barrier and fence latency whatever the
// amount of data, which is why a ring stage holds two k-blocks.
// The widening and the operand byte order are those of the single-CTA kernel (sq_gemm.cu).
#include <cuda.h>
#include <cuda_fp16.h>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

constexpr int P_A_WARPS = 4;
constexpr int P_B_WARPS = 4;             // one weight row of the CTA's 128 per thread
constexpr int P_EPI_WARPS = 16;          // four per TMEM lane quarter, two 32-column chunks each
constexpr int P_THREADS = (2 + P_A_WARPS + P_B_WARPS + P_EPI_WARPS) * 32;
constexpr int P_TILE_M = 256;            // tokens per pair tile (128 per CTA)
constexpr int P_TILE_N = 256;            // output channels per pair tile (128 staged per CTA)
constexpr int P_A_COL0 = 256;            // first TMEM column of the A operand ring (0..255: accumulator)
constexpr int P_A_COLS_PER_STAGE = 64;   // 256 int8 per lane = 64 columns

enum PairSite : uint32_t {
  PSITE_ST_EMPTY = 32, PSITE_ST_FULL_A, PSITE_ST_FULL_B, PSITE_EMPTY_A, PSITE_EMPTY_B, PSITE_FULL,
  PSITE_TMEM_FULL, PSITE_TMEM_EMPTY
};

template <int S_OP, int S_ST>
struct PairSmem {
  static_assert(S_OP >= 2 && S_OP <= 4, "the A ring has room for at most 4 blocks in TMEM");
  static constexpr int B_OP = 2 * 128 * 128;         // int8 B half, two k-blocks
  static constexpr int A_ST = 128 * 128;             // packed A rows, two k-blocks
  static constexpr int B_ST = 128 * 128;             // packed B rows, two k-blocks
  static constexpr int OFF_B_OP = 0;
  static constexpr int OFF_A_ST = OFF_B_OP + S_OP * B_OP;
  static constexpr int OFF_B_ST = OFF_A_ST + S_ST * A_ST;
  static constexpr int OUT_BUF = 32 * 64;            // fp16 [32 rows x 32 columns], 64-byte swizzle
  static constexpr int OFF_OUT = OFF_B_ST + S_ST * B_ST;
  static constexpr int OFF_BAR = OFF_OUT + P_EPI_WARPS * OUT_BUF;     // one staging tile per epilogue warp
  static constexpr int NUM_BARS = 2 * S_OP + 2 * S_ST + 2;
  static constexpr int OFF_TMEM = OFF_BAR + NUM_BARS * 8;
  static constexpr int TOTAL = OFF_TMEM + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

// 2-D fp16 map over Y [M x N]; box = 32 rows x 32 columns (64 bytes) with the 64-byte swizzle.
bool make_out_map(CUtensorMap* map, void* Y, uint64_t M, uint64_t N) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[2] = {N, M};
  const cuuint64_t strides[1] = {N * 2};
  const cuuint32_t box[2] = {32, 32};
  const cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, Y, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The grouped form (one launch for the experts of a mixture-of-experts layer): expert g has its own packed
// weights, channel steps and output map (Y restricted to its rows, so that the TMA store clips there) and
// owns rows[g] consecutive token rows from r0[g] on of a common Xq and sx.  Its tiles are tile0[g] ..
// tile0[g + 1] - 1 of the launch, token tiles innermost as in the plain form.
constexpr int P_MAX_GROUPS = 16;
struct alignas(64) PairGroups {
  CUtensorMap wmap[P_MAX_GROUPS];
  CUtensorMap ymap[P_MAX_GROUPS];
  const __half* sw[P_MAX_GROUPS];
  int r0[P_MAX_GROUPS];
  int rows[P_MAX_GROUPS];
  int tile0[P_MAX_GROUPS + 1];
  int count;
};

// GROUPED: the tiles run over the experts of `G`; tmap_w, tmap_y, sw and M are unused.
template <int S_OP, int S_ST, bool GROUPED>
__device__ __forceinline__ void w4a4_gemm_pair_body(const CUtensorMap& tmap_x, const CUtensorMap& tmap_w,
                                                    const CUtensorMap& tmap_y, const __half* __restrict__ sx,
                                                    const __half* __restrict__ sw, int M, int N, int K,
                                                    int32_t* __restrict__ accdbg, const PairGroups* G) {
  using L = PairSmem<S_OP, S_ST>;
  griddep_launch_dependents();          // a rotate kernel launched behind this one may set itself up on SMs that fall idle
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* st_full = bars;                           // [S_ST]  TMA landed (local)
  uint64_t* st_empty = bars + S_ST;                   // [S_ST]  12 converter warps done (local)
  uint64_t* full = bars + 2 * S_ST;                   // [S_OP]  24 converter warps of the pair (leader's copy is used)
  uint64_t* empty = bars + 2 * S_ST + S_OP;           // [S_OP]  MMAs retired (each CTA's own copy)
  uint64_t* tmem_full = bars + 2 * S_ST + 2 * S_OP;   // accumulator complete (each CTA's own copy)
  uint64_t* tmem_empty = tmem_full + 1;               // epilogue warps of the pair (leader's copy is used)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_TMEM);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();            // 0 = leader (issues the MMAs)
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int num_kb = K / 128;
  const int num_sb = (num_kb + 1) / 2;
  const int tiles_n = (N + P_TILE_N - 1) / P_TILE_N, tiles_m = (M + P_TILE_M - 1) / P_TILE_M;
  const int num_tiles = GROUPED ? G->tile0[G->count] : tiles_n * tiles_m;
  // tile -> expert g, first token row of the tile within the expert, first channel of the tile
  auto locate = [&](int tile, int& g, int& mrow, int& ncol) {
    if constexpr (GROUPED) {
      g = 0;
      while (g + 1 < G->count && tile >= G->tile0[g + 1]) ++g;
      const int local = tile - G->tile0[g], tm = (G->rows[g] + P_TILE_M - 1) / P_TILE_M;
      mrow = (local % tm) * P_TILE_M;
      ncol = (local / tm) * P_TILE_N;
    } else {
      g = 0;
      mrow = (tile % tiles_m) * P_TILE_M;
      ncol = (tile / tiles_m) * P_TILE_N;
    }
  };
  const uint32_t limit = wait_limit();
  const int pre_sb = num_sb < S_ST ? num_sb : S_ST;    // blocks whose weights are requested during set-up

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmap_x);
    tma_prefetch_desc(&tmap_w);
    tma_prefetch_desc(&tmap_y);
    for (int s = 0; s < S_ST; ++s) {
      mbar_init(&st_full[s], 1);
      mbar_init(&st_empty[s], P_A_WARPS + P_B_WARPS);
    }
    for (int s = 0; s < S_OP; ++s) {
      mbar_init(&full[s], 2 * (P_A_WARPS + P_B_WARPS));
      mbar_init(&empty[s], 1);
    }
    mbar_init(tmem_full, 1);
    mbar_init(tmem_empty, 2 * P_EPI_WARPS);
    mbar_fence_init();
    // The weights of the first tile's first blocks do not depend on the kernel launched before this
    // one: they are requested now (local barriers only), the activations after the wait below.
    if (pair < num_tiles) {
      int g, mrow, ncol;
      locate(pair, g, mrow, ncol);
      const int n0 = ncol + static_cast<int>(rank) * 128;
      for (int sb = 0; sb < pre_sb; ++sb) {
        mbar_arrive_expect_tx(&st_full[sb], L::A_ST + L::B_ST);
        tma_load_2d(smem + L::OFF_B_ST + sb * L::B_ST, GROUPED ? &G->wmap[g] : &tmap_w, &st_full[sb], sb * 128, n0);
      }
    }
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();                                 // both CTAs' barriers exist before any remote arrival
  tc_fence_after_sync();
  griddep_wait();                                     // Xq and sx may come from the kernel launched before this one
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------------
    if (elect_one()) {
      uint32_t it = 0;
      bool ok = true;
      // Tile order: token tiles innermost.  The pairs that run at the same time then share a few weight
      // tiles and all of X, which stays in L2; with the channel tiles innermost every token tile
      // streamed the whole weight matrix from HBM again once it no longer fitted L2.
      for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
        int g, mrow, ncol;
        locate(tile, g, mrow, ncol);
        const int m0 = (GROUPED ? G->r0[g] : 0) + mrow + static_cast<int>(rank) * 128;    // row of Xq
        const int n0 = ncol + static_cast<int>(rank) * 128;
        const CUtensorMap* wm = GROUPED ? &G->wmap[g] : &tmap_w;
        for (int sb = 0; sb < num_sb; ++sb, ++it) {
          const int ss = it % S_ST;
          if (it < static_cast<uint32_t>(pre_sb)) {     // armed and half loaded during set-up
            tma_load_2d(smem + L::OFF_A_ST + ss * L::A_ST, &tmap_x, &st_full[ss], sb * 128, m0);
            continue;
          }
          ok = mbar_wait(&st_empty[ss], ((it / S_ST) & 1) ^ 1, PSITE_ST_EMPTY, limit);
          if (!ok) break;
          mbar_arrive_expect_tx(&st_full[ss], L::A_ST + L::B_ST);
          tma_load_2d(smem + L::OFF_A_ST + ss * L::A_ST, &tmap_x, &st_full[ss], sb * 128, m0);
          tma_load_2d(smem + L::OFF_B_ST + ss * L::B_ST, wm, &st_full[ss], sb * 128, n0);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader CTA) -------------------------------------
    if (rank == 0 && elect_one()) {
      constexpr uint32_t idesc = umma_idesc(/*c=s32*/ 2, /*a=s8*/ 1, /*b=s8*/ 1, P_TILE_M, P_TILE_N);
      // The issuing thread pays several cycles per instruction: descriptors are formed once and
      // differ from block to block by constants in the start-address field (no carry out of it).
      const uint64_t b_desc0 = umma_desc_sw128(smem_u32(smem + L::OFF_B_OP));
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += npairs, ++tcount) {
        ok = mbar_wait(tmem_empty, (tcount & 1) ^ 1, PSITE_TMEM_EMPTY, limit);
        if (!ok) break;
        tc_fence_after_sync();
        for (int sb = 0; sb < num_sb; ++sb, ++it) {
          const int s = it % S_OP;
          ok = mbar_wait(&full[s], (it / S_OP) & 1, PSITE_FULL, limit);
          if (!ok) break;
          tc_fence_after_sync();
          // K = 32 int8 per MMA: 8 TMEM columns, 32 shared-memory bytes (2 in the descriptor's
          // 16-byte units; the second k-block tile lies 128 * 128 bytes further on).
          const uint32_t a_tmem = tmem_base + P_A_COL0 + s * P_A_COLS_PER_STAGE;
          const uint64_t bd = b_desc0 + static_cast<uint64_t>(s * (L::B_OP >> 4));
          constexpr uint32_t KB1 = (128 * 128) >> 4;
          umma_i8_ts_pair(tmem_base, a_tmem, bd, idesc, sb != 0 ? 1u : 0u);
          umma_i8_ts_pair(tmem_base, a_tmem + 8, bd + 2, idesc, 1u);
          umma_i8_ts_pair(tmem_base, a_tmem + 16, bd + 4, idesc, 1u);
          umma_i8_ts_pair(tmem_base, a_tmem + 24, bd + 6, idesc, 1u);
          if (2 * sb + 1 < num_kb) {
            umma_i8_ts_pair(tmem_base, a_tmem + 32, bd + KB1, idesc, 1u);
            umma_i8_ts_pair(tmem_base, a_tmem + 40, bd + (KB1 + 2), idesc, 1u);
            umma_i8_ts_pair(tmem_base, a_tmem + 48, bd + (KB1 + 4), idesc, 1u);
            umma_i8_ts_pair(tmem_base, a_tmem + 56, bd + (KB1 + 6), idesc, 1u);
          }
          umma_commit_pair_mc(&empty[s], 3);            // frees ring stage s in both CTAs
        }
        umma_commit_pair_mc(tmem_full, 3);              // accumulator complete (or abandoned)
      }
    }
  } else if (warp < 2 + P_A_WARPS) {
    // ------------------------------ A converters: staging -> registers -> TMEM ------------------
    const int q = warp & 3;                             // TMEM lane quarter this warp may touch
    const int r = q * 32 + lane;                        // row of the CTA's 128 tokens = TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
      for (int sb = 0; sb < num_sb && ok; ++sb, ++it) {
        const int ss = it % S_ST, s = it % S_OP;
        ok = mbar_wait(&st_full[ss], (it / S_ST) & 1, PSITE_ST_FULL_A, limit);
        if (!ok) break;
        const unsigned char* row = smem + L::OFF_A_ST + ss * L::A_ST + r * 128;
        const int nh = (2 * sb + 1 < num_kb) ? 2 : 1;
        uint4 w[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) w[c] = *reinterpret_cast<const uint4*>(row + ((c ^ (r & 7)) << 4));
        ok = mbar_wait(&empty[s], ((it / S_OP) & 1) ^ 1, PSITE_EMPTY_A, limit);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (h < nh) {
            uint32_t v[32];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint4 x = w[4 * h + j];
              v[4 * j + 0] = (x.x << 4) & 0xF0F0F0F0u; v[16 + 4 * j + 0] = x.x & 0xF0F0F0F0u;
              v[4 * j + 1] = (x.y << 4) & 0xF0F0F0F0u; v[16 + 4 * j + 1] = x.y & 0xF0F0F0F0u;
              v[4 * j + 2] = (x.z << 4) & 0xF0F0F0F0u; v[16 + 4 * j + 2] = x.z & 0xF0F0F0F0u;
              v[4 * j + 3] = (x.w << 4) & 0xF0F0F0F0u; v[16 + 4 * j + 3] = x.w & 0xF0F0F0F0u;
            }
            tmem_st_32x32b_x32(tmem_base + lane_addr + P_A_COL0 + s * P_A_COLS_PER_STAGE + h * 32, v);
          }
        }
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_cluster(&full[s], 0);
          mbar_arrive(&st_empty[ss]);
        }
      }
    }
  } else if (warp < 2 + P_A_WARPS + P_B_WARPS) {
    // ------------------------------ B unpackers: staging -> registers -> operand ring -----------
    // Thread t widens row t of the CTA's 128 weight rows: eight 16-byte loads (both k-blocks) first,
    // then the sixteen stores.  Consecutive lanes take consecutive rows, whose swizzled chunks fall
    // into different bank groups.
    const int br = threadIdx.x - (2 + P_A_WARPS) * 32;  // 0 .. 127
    const int bsw = br & 7;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
      for (int sb = 0; sb < num_sb && ok; ++sb, ++it) {
        const int ss = it % S_ST, s = it % S_OP;
        ok = mbar_wait(&st_full[ss], (it / S_ST) & 1, PSITE_ST_FULL_B, limit);
        if (!ok) break;
        const int nh = (2 * sb + 1 < num_kb) ? 2 : 1;
        const unsigned char* row = smem + L::OFF_B_ST + ss * L::B_ST + br * 128;
        uint4 w[8];
#pragma unroll
        for (int c = 0; c < 8; ++c)
          if (c < 4 * nh) w[c] = *reinterpret_cast<const uint4*>(row + ((c ^ bsw) << 4));
        ok = mbar_wait(&empty[s], ((it / S_OP) & 1) ^ 1, PSITE_EMPTY_B, limit);
        if (!ok) break;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c < 4 * nh) {
            const int h = c >> 2, j = c & 3;
            uint4 lo, hi;
            lo.x = (w[c].x << 4) & 0xF0F0F0F0u; hi.x = w[c].x & 0xF0F0F0F0u;
            lo.y = (w[c].y << 4) & 0xF0F0F0F0u; hi.y = w[c].y & 0xF0F0F0F0u;
            lo.z = (w[c].z << 4) & 0xF0F0F0F0u; hi.z = w[c].z & 0xF0F0F0F0u;
            lo.w = (w[c].w << 4) & 0xF0F0F0F0u; hi.w = w[c].w & 0xF0F0F0F0u;
            unsigned char* orow = smem + L::OFF_B_OP + s * L::B_OP + h * (128 * 128) + br * 128;
            *reinterpret_cast<uint4*>(orow + ((j ^ bsw) << 4)) = lo;
            *reinterpret_cast<uint4*>(orow + (((4 + j) ^ bsw) << 4)) = hi;
          }
        }
        fence_proxy_async_smem();                       // generic-proxy stores -> visible to the MMA
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_cluster(&full[s], 0);
          mbar_arrive(&st_empty[ss]);
        }
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------------------------
    const int e = warp - (2 + P_A_WARPS + P_B_WARPS);   // 0 .. 15
    const int q = warp & 3;                             // TMEM lane quarter this warp may read
    const int c_first = (e >> 2) * 2;                   // this warp's two 32-column chunks
    unsigned char* obuf = smem + L::OFF_OUT + e * L::OUT_BUF;
    uint32_t tcount = 0, nstore = 0;
    bool ok = true;
    for (int tile = pair; tile < num_tiles && ok; tile += npairs, ++tcount) {
      int tg, mrow, n0;
      locate(tile, tg, mrow, n0);
      const int Mt = GROUPED ? G->rows[tg] : M;            // token rows of the tile's expert
      const int trow0 = GROUPED ? G->r0[tg] : 0;           // the first of them in Xq and sx
      const int m0 = mrow + static_cast<int>(rank) * 128;
      // Fetched while the MMAs still run: this row's token step, and the channel steps of the warp's
      // 128 columns, four per lane (handed round by shuffles when a chunk needs them).
      const int row0 = m0 + q * 32, row = row0 + lane;     // rows within the expert (= rows of its Y map)
      const float sxv = (row < Mt) ? __half2float(sx[trow0 + row]) : 0.0f;
      const int swcol = n0 + c_first * 32 + 4 * lane;
      const uint2 swp = (swcol < N) ? __ldg(reinterpret_cast<const uint2*>((GROUPED ? G->sw[tg] : sw) + swcol))
                                    : make_uint2(0u, 0u);
      ok = mbar_wait(tmem_full, tcount & 1, PSITE_TMEM_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tmem_d = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
#pragma unroll 1
      for (int j = 0; j < 2; ++j, ++nstore) {
        const int c = c_first + j;
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem_d + c * 32, r);
        tmem_wait_ld();
        if (j == 1) {                                   // last read of this warp: hand the accumulator back
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(tmem_empty, 0);
        }
        const int col0 = n0 + c * 32;
        unsigned char* buf = obuf;
        if (nstore >= 1) {                              // the previous chunk's store has read `buf`
          if (lane == 0) tma_store_wait_read_0();
          __syncwarp();
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {                   // groups of 8 columns (N % 8 == 0)
          uint4 swraw;
          swraw.x = __shfl_sync(0xffffffffu, swp.x, 8 * j + 2 * g);
          swraw.y = __shfl_sync(0xffffffffu, swp.y, 8 * j + 2 * g);
          swraw.z = __shfl_sync(0xffffffffu, swp.x, 8 * j + 2 * g + 1);
          swraw.w = __shfl_sync(0xffffffffu, swp.y, 8 * j + 2 * g + 1);
          int32_t a[8];
          *reinterpret_cast<uint4*>(buf + lane * 64 + ((g ^ ((lane >> 1) & 3)) << 4)) = dequant8(&r[g * 8], sxv, swraw, a);
          if (accdbg != nullptr && row < Mt && col0 + g * 8 < N) {
            int32_t* arow = accdbg + static_cast<size_t>(trow0 + row) * N + col0 + g * 8;
            *reinterpret_cast<int4*>(arow) = make_int4(a[0], a[1], a[2], a[3]);
            *reinterpret_cast<int4*>(arow + 4) = make_int4(a[4], a[5], a[6], a[7]);
          }
        }
        fence_proxy_async_smem();                       // the tile in `buf` -> visible to the TMA store
        __syncwarp();
        if (lane == 0) {
          if (row0 < Mt && col0 < N) tma_store_2d(GROUPED ? &G->ymap[tg] : &tmap_y, buf, col0, row0);
          tma_store_commit();
        }
      }
    }
    if (lane == 0) tma_store_wait_all();
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

template <int S_OP, int S_ST>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(P_THREADS, 1)
w4a4_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                      const __grid_constant__ CUtensorMap tmap_y, const __half* __restrict__ sx, const __half* __restrict__ sw, int M, int N, int K,
                      __half* __restrict__ Y, int32_t* __restrict__ accdbg) {
  (void)Y;                                              // the output goes through tmap_y
  w4a4_gemm_pair_body<S_OP, S_ST, false>(tmap_x, tmap_w, tmap_y, sx, sw, M, N, K, accdbg, nullptr);
}

template <int S_OP, int S_ST>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(P_THREADS, 1)
w4a4_gemm_pair_grouped_kernel(const __grid_constant__ PairGroups G, const __grid_constant__ CUtensorMap tmap_x,
                              const __half* __restrict__ sx, int N, int K) {
  w4a4_gemm_pair_body<S_OP, S_ST, true>(tmap_x, G.wmap[0], G.ymap[0], sx, nullptr, 0, N, K, nullptr, &G);
}

}  // namespace

int gemm_pair_max_groups() { return P_MAX_GROUPS; }

// Step 3 for up to P_MAX_GROUPS experts in one launch: expert g owns rows[g] >= 1 token rows from r0[g] on of
// Xq [M_total x K/2], sx and Y, and has its own Wq[g], sw[g].  Shapes as gemm_pair_supported (whatever rows[g]).
sq_status_t launch_w4a4_gemm_pair_grouped(const void* Xq, const void* sx, int64_t M_total, int count,
                                          const void* const* Wq, const void* const* sw, const int64_t* r0,
                                          const int64_t* rows, int N, int K, void* Y, cudaStream_t s) {
  constexpr int S_OP = 3, S_ST = 3;
  using L = PairSmem<S_OP, S_ST>;
  if (count < 1 || count > P_MAX_GROUPS) return SQ_ERR_INVALID_ARG;
  PairGroups G;
  CUtensorMap mx;
  if (!make_packed_map(&mx, Xq, static_cast<uint64_t>(M_total), K / 2, 128)) return SQ_ERR_CUDA;
  const int tiles_n = (N + P_TILE_N - 1) / P_TILE_N;
  long long total = 0;
  for (int g = 0; g < P_MAX_GROUPS; ++g) {
    const int src = g < count ? g : 0;                   // unused entries repeat the first (never read)
    if (rows[src] < 1) return SQ_ERR_INVALID_ARG;
    void* Yg = static_cast<unsigned char*>(Y) + static_cast<size_t>(r0[src]) * N * 2;
    if (!make_packed_map(&G.wmap[g], Wq[src], N, K / 2, 128) ||
        !make_out_map(&G.ymap[g], Yg, static_cast<uint64_t>(rows[src]), N))
      return SQ_ERR_CUDA;
    G.sw[g] = static_cast<const __half*>(sw[src]);
    G.r0[g] = static_cast<int>(r0[src]);
    G.rows[g] = static_cast<int>(rows[src]);
    if (g < count) {
      G.tile0[g] = static_cast<int>(total);
      total += static_cast<long long>(tiles_n) * ((rows[src] + P_TILE_M - 1) / P_TILE_M);
    }
  }
  if (total > 0x7fffffffll) return SQ_ERR_UNSUPPORTED;
  for (int g = count; g <= P_MAX_GROUPS; ++g) G.tile0[g] = static_cast<int>(total);
  G.count = count;
  auto kern = w4a4_gemm_pair_grouped_kernel<S_OP, S_ST>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), L::DYN_BYTES)) return SQ_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const int pairs = total < sms / 2 ? static_cast<int>(total) : sms / 2;
  const cudaError_t err = launch_maybe_pdl(kern, dim3(2 * pairs), dim3(P_THREADS), L::DYN_BYTES, s, G, mx,
                                           static_cast<const __half*>(sx), N, K);
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SQ_OK : SQ_ERR_CUDA;
}

bool gemm_pair_supported(int64_t M, int64_t N, int64_t K) {
  return M > 128 && N >= 128 && (K % 128 == 0) && K >= 128 && (N % 8 == 0);
}

sq_status_t launch_w4a4_gemm_pair(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N,
                                  int K, void* Y, int32_t* accdbg, cudaStream_t s) {
  constexpr int S_OP = 3, S_ST = 3;
  using L = PairSmem<S_OP, S_ST>;
  CUtensorMap mx, mw, my;
  if (!make_packed_map(&mx, Xq, M, K / 2, 128) || !make_packed_map(&mw, Wq, N, K / 2, 128) ||
      !make_out_map(&my, Y, M, N))
    return SQ_ERR_CUDA;
  auto kern = w4a4_gemm_pair_kernel<S_OP, S_ST>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), L::DYN_BYTES)) return SQ_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const int tiles = ((N + P_TILE_N - 1) / P_TILE_N) * ((M + P_TILE_M - 1) / P_TILE_M);
  const int pairs = tiles < sms / 2 ? tiles : sms / 2;
  const cudaError_t err = launch_maybe_pdl(kern, dim3(2 * pairs), dim3(P_THREADS), L::DYN_BYTES, s, mx, mw, my,
                                           static_cast<const __half*>(sx), static_cast<const __half*>(sw), M, N, K,
                                           static_cast<__half*>(Y), accdbg);
  count_launch();
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace sq
