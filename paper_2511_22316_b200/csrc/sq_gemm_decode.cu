// Step 3 for decode-sized problems (M <= 64 tokens): the INT4 x INT4 GEMM with the operands
// swapped and K split, so that every SM streams weights.
//
// With a handful of tokens the GEMM is bound by reading the packed weights once (N K / 2 bytes).
// The weights therefore take the role of the MMA's A operand: a tile is 128 OUTPUT CHANNELS (the
// TMEM lanes), the tokens are the MMA's N (16, 32 or 64).  Four warps read the packed bytes of
// "their" weight row from the TMA staging ring, widen them in registers and store the int8
// operand into a TMEM ring (tcgen05.st); the few token rows are widened through shared memory.
// A work item is (tile of 128 channels, chunk of K); the chunk count is chosen so that the items
// fill the SMs evenly.  Each item leaves an exact int32 partial tile in the caller's workspace;
// the item that completes a tile (a counter per tile) adds the partials in a fixed order,
// dequantises and writes fp16 -- the result does not depend on which item came last.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer, warps 2..9 = two groups of weight
// converters and warps 10..13 = two groups of token unpackers (a group takes every other block:
// a block costs a warp several hundred cycles of waits and fences whatever its size), warps
// 14..21 = two epilogue groups that take the items in turn (four accumulators, so epilogues,
// whose global-memory round trips are long, overlap the main loop of the following items).
#include <cuda.h>
#include <cuda_fp16.h>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

constexpr int D_CONV_GROUPS = 2;          // converter groups; group g takes the blocks g, g + 2, ...
constexpr int D_A_WARPS = 4 * D_CONV_GROUPS, D_B_WARPS = 2 * D_CONV_GROUPS;
constexpr int D_EPI_GROUPS = 2, D_EPI_WARPS = 4 * D_EPI_GROUPS;
constexpr int D_THREADS = (2 + D_A_WARPS + D_B_WARPS + D_EPI_WARPS) * 32;
constexpr int D_S_ST = 6;                // staging stages (256 channels each)
constexpr int D_S_OP = 4;                // operand stages (TMEM A ring: 4 x 64 columns)
constexpr int D_A_COL0 = 256;
constexpr int D_MAX_SPLITS = 16;           // partial tiles of one output tile, all in flight when they are summed
constexpr int D_ACCS = 4;                 // accumulators in TMEM (columns 0 .. 4 * NT)

enum DecSite : uint32_t {
  DSITE_ST_EMPTY = 64, DSITE_ST_FULL_A, DSITE_ST_FULL_B, DSITE_EMPTY_A, DSITE_EMPTY_B, DSITE_FULL,
  DSITE_TMEM_FULL, DSITE_TMEM_EMPTY
};

template <int NT>
struct DecSmem {
  static constexpr int W_ST = 128 * 128;             // packed weight rows, two k-blocks
  static constexpr int X_ST = NT * 128;              // packed token rows, two k-blocks
  static constexpr int X_OP = 2 * NT * 128;          // int8 token rows, two k-block tiles
  static constexpr int OFF_X_OP = 0;
  static constexpr int OFF_W_ST = OFF_X_OP + D_S_OP * X_OP;
  static constexpr int OFF_X_ST = OFF_W_ST + D_S_ST * W_ST;
  static constexpr int OFF_BAR = OFF_X_ST + D_S_ST * X_ST;
  static constexpr int NUM_BARS = 2 * D_S_ST + 2 * D_S_OP + 2 * D_ACCS;
  static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;
  static constexpr int TOTAL = OFF_MISC + 32;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

// Splits the K blocks of every tile into `splits` chunks.  Cost model (cycles, measured): a block of
// 256 channels takes about 1250 cycles of the main loop; splitting K adds about 8000 cycles once
// (partial tiles, fence, counter, the sum by the last item).  The cheapest count wins.
int choose_splits(int tiles, int blocks, int sms) {
  int best = 1;
  double best_cost = 0.0;
  for (int s = 1; s <= D_MAX_SPLITS && s * 2 <= blocks + 1; ++s) {
    if (s > 1 && blocks / s < 2) break;
    const long long items = static_cast<long long>(tiles) * s;
    const long long waves = (items + sms - 1) / sms;
    const double per_item = static_cast<double>((blocks + s - 1) / s);
    const double cost = static_cast<double>(waves) * per_item * 1250.0 + (s > 1 ? 8000.0 : 0.0);
    if (s == 1 || cost < best_cost * 0.97) {
      best_cost = cost;
      best = s;
    }
  }
  return best;
}

// Widens the 128 staged bytes of `rows` token rows into two int8 k-block tiles (rows x 128 B each,
// 128-byte swizzle), same byte order as unpack_tile.  Task = (row, 16-byte chunk).
__device__ __forceinline__ void unpack_rows(const unsigned char* __restrict__ st, unsigned char* __restrict__ op,
                                            int rows, int t, int nthreads, bool second) {
  const int ntask = rows * (second ? 8 : 4);
  for (int task = t; task < ntask; task += nthreads) {
    const int r = task % rows, c = task / rows;          // c: chunk of the staged row (0..7)
    const int h = c >> 2, j = c & 3, sw = r & 7;
    const uint4 w = *reinterpret_cast<const uint4*>(st + r * 128 + ((c ^ sw) << 4));
    uint4 lo, hi;
    lo.x = (w.x << 4) & 0xF0F0F0F0u; hi.x = w.x & 0xF0F0F0F0u;
    lo.y = (w.y << 4) & 0xF0F0F0F0u; hi.y = w.y & 0xF0F0F0F0u;
    lo.z = (w.z << 4) & 0xF0F0F0F0u; hi.z = w.z & 0xF0F0F0F0u;
    lo.w = (w.w << 4) & 0xF0F0F0F0u; hi.w = w.w & 0xF0F0F0F0u;
    unsigned char* tile = op + h * (rows * 128) + r * 128;
    *reinterpret_cast<uint4*>(tile + ((j ^ sw) << 4)) = lo;
    *reinterpret_cast<uint4*>(tile + (((4 + j) ^ sw) << 4)) = hi;
  }
}

template <int NT>
__global__ void __launch_bounds__(D_THREADS, 1)
w4a4_gemm_decode_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                        const __half* __restrict__ sx, const __half* __restrict__ sw, int M, int N, int K,
                        int splits, __half* __restrict__ Y, int32_t* __restrict__ accdbg,
                        int32_t* __restrict__ partials, unsigned int* __restrict__ counters) {
  using L = DecSmem<NT>;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* st_full = bars;
  uint64_t* st_empty = bars + D_S_ST;
  uint64_t* full = bars + 2 * D_S_ST;
  uint64_t* empty = bars + 2 * D_S_ST + D_S_OP;
  uint64_t* tmem_full = bars + 2 * D_S_ST + 2 * D_S_OP;      // [D_ACCS]
  uint64_t* tmem_empty = tmem_full + D_ACCS;                  // [D_ACCS]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
  uint32_t* last_flag = tmem_slot + 1;                        // [D_EPI_GROUPS]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = K / 128;
  const int num_sb = (num_kb + 1) / 2;                 // blocks of 256 channels (the last may be half)
  const int tiles = (N + 127) / 128;
  const int num_items = tiles * splits;
  const uint32_t limit = wait_limit();

  // item -> (tile, first block, one-past-last block)
  auto item_range = [&](int item, int& tile, int& b0, int& b1) {
    tile = item / splits;
    const int sp = item % splits;
    b0 = static_cast<int>(static_cast<long long>(sp) * num_sb / splits);
    b1 = static_cast<int>(static_cast<long long>(sp + 1) * num_sb / splits);
  };
  // The producer's walk over (item, block); `budget` blocks are issued per call (waiting for the
  // staging stage of each), so that the first ring-full can go out before the CTA has set up.
  int p_item = blockIdx.x, p_sb = -1, p_b1 = 0, p_tile = 0;
  uint32_t p_it = 0;
  auto produce = [&](uint32_t budget) -> bool {
    while (budget > 0 && p_item < num_items) {
      if (p_sb < 0) {
        int b0;
        item_range(p_item, p_tile, b0, p_b1);
        p_sb = b0;
      }
      const int ss = p_it % D_S_ST;
      if (!mbar_wait(&st_empty[ss], ((p_it / D_S_ST) & 1) ^ 1, DSITE_ST_EMPTY, limit)) return false;
      mbar_arrive_expect_tx(&st_full[ss], L::W_ST + L::X_ST);
      tma_load_2d(smem + L::OFF_W_ST + ss * L::W_ST, &tmap_w, &st_full[ss], p_sb * 128, p_tile * 128);
      tma_load_2d(smem + L::OFF_X_ST + ss * L::X_ST, &tmap_x, &st_full[ss], p_sb * 128, 0);
      ++p_it;
      --budget;
      if (++p_sb >= p_b1) {
        p_sb = -1;
        p_item += gridDim.x;
      }
    }
    return true;
  };

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmap_w);
    tma_prefetch_desc(&tmap_x);
    for (int s = 0; s < D_S_ST; ++s) {
      mbar_init(&st_full[s], 1);
      mbar_init(&st_empty[s], 6);                      // one converter group + one unpacker group
    }
    for (int s = 0; s < D_S_OP; ++s) {
      mbar_init(&full[s], 6);
      mbar_init(&empty[s], 1);
    }
    for (int b = 0; b < D_ACCS; ++b) {
      mbar_init(&tmem_full[b], 1);
      mbar_init(&tmem_empty[b], 4);
    }
    mbar_fence_init();
    produce(D_S_ST);                                   // the whole staging ring, before anyone else is ready
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
    // ------------------------------ TMA producer ------------------------------------------------
    if (lane == 0) produce(0xFFFFFFFFu);
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------------------------
    if (elect_one()) {
      constexpr uint32_t idesc = umma_idesc(/*c=s32*/ 2, /*a=s8*/ 1, /*b=s8*/ 1, 128, NT);
      uint32_t it = 0, icount = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x, ++icount) {
        int tile, b0, b1;
        item_range(item, tile, b0, b1);
        const uint32_t acc = icount % D_ACCS;
        ok = mbar_wait(&tmem_empty[acc], ((icount / D_ACCS) & 1) ^ 1, DSITE_TMEM_EMPTY, limit);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * NT;
        for (int sb = b0; sb < b1; ++sb, ++it) {
          const int s = it % D_S_OP;
          ok = mbar_wait(&full[s], (it / D_S_OP) & 1, DSITE_FULL, limit);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t a_tmem = tmem_base + D_A_COL0 + s * 64;
          const uint32_t b_base = smem_u32(smem + L::OFF_X_OP + s * L::X_OP);
          const int nk = (2 * sb + 1 < num_kb) ? 8 : 4;
#pragma unroll 4
          for (int k = 0; k < nk; ++k)
            umma_i8_ts(d_tmem, a_tmem + k * 8, umma_desc_sw128(b_base + (k >> 2) * (NT * 128) + (k & 3) * 32), idesc,
                       (sb > b0 || k > 0) ? 1u : 0u);
          umma_commit(&empty[s]);
        }
        umma_commit(&tmem_full[acc]);
      }
    }
  } else if (warp < 2 + D_A_WARPS) {
    // ------------------------------ weight converters: staging -> registers -> TMEM --------------
    const int q = warp & 3;
    const int grp = (warp - 2) >> 2;                    // this group's blocks: it % D_CONV_GROUPS == grp
    const int r = q * 32 + lane;
    const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
    uint32_t it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
      int tile, b0, b1;
      item_range(item, tile, b0, b1);
      for (int sb = b0; sb < b1 && ok; ++sb, ++it) {
        if ((it % D_CONV_GROUPS) != static_cast<uint32_t>(grp)) continue;
        const int ss = it % D_S_ST, s = it % D_S_OP;
        ok = mbar_wait(&st_full[ss], (it / D_S_ST) & 1, DSITE_ST_FULL_A, limit);
        if (!ok) break;
        const unsigned char* row = smem + L::OFF_W_ST + ss * L::W_ST + r * 128;
        const int nh = (2 * sb + 1 < num_kb) ? 2 : 1;
        uint4 w[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) w[c] = *reinterpret_cast<const uint4*>(row + ((c ^ (r & 7)) << 4));
        ok = mbar_wait(&empty[s], ((it / D_S_OP) & 1) ^ 1, DSITE_EMPTY_A, limit);
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
            tmem_st_32x32b_x32(tmem_base + lane_addr + D_A_COL0 + s * 64 + h * 32, v);
          }
        }
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&full[s]);
          mbar_arrive(&st_empty[ss]);
        }
      }
    }
  } else if (warp < 2 + D_A_WARPS + D_B_WARPS) {
    // ------------------------------ token unpackers: staging -> operand ring ----------------------
    const int grp = (warp - (2 + D_A_WARPS)) >> 1;
    const int t = (threadIdx.x - (2 + D_A_WARPS) * 32) & 63;
    uint32_t it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
      int tile, b0, b1;
      item_range(item, tile, b0, b1);
      for (int sb = b0; sb < b1 && ok; ++sb, ++it) {
        if ((it % D_CONV_GROUPS) != static_cast<uint32_t>(grp)) continue;
        const int ss = it % D_S_ST, s = it % D_S_OP;
        ok = mbar_wait(&st_full[ss], (it / D_S_ST) & 1, DSITE_ST_FULL_B, limit) &&
             mbar_wait(&empty[s], ((it / D_S_OP) & 1) ^ 1, DSITE_EMPTY_B, limit);
        if (!ok) break;
        unpack_rows(smem + L::OFF_X_ST + ss * L::X_ST, smem + L::OFF_X_OP + s * L::X_OP, NT, t, 64,
                    2 * sb + 1 < num_kb);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&full[s]);
          mbar_arrive(&st_empty[ss]);
        }
      }
    }
  } else {
    // ------------------------------ epilogue groups -----------------------------------------------
    const int q = warp & 3;
    const int eg = (warp - (2 + D_A_WARPS + D_B_WARPS)) >> 2;        // this group takes items eg, eg + 2, ...
    const int et = (threadIdx.x - (2 + D_A_WARPS + D_B_WARPS) * 32) & 127;
    const int rowl = q * 32 + lane;                                  // row of the tile = TMEM lane
    bool ok = true;
    uint32_t icount = 0;
    for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x, ++icount) {
      if ((icount % D_EPI_GROUPS) != static_cast<uint32_t>(eg)) continue;
      int tile, b0, b1;
      item_range(item, tile, b0, b1);
      const uint32_t acc = icount % D_ACCS;
      ok = mbar_wait(&tmem_full[acc], (icount / D_ACCS) & 1, DSITE_TMEM_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tmem_d = tmem_base + acc * NT + (static_cast<uint32_t>(q * 32) << 16);
      const int ch = tile * 128 + rowl;                    // output channel of this thread
      const float swv = (ch < N) ? __half2float(sw[ch]) : 0.0f;
      // Partial tiles are stored as [item][4-column chunk][row][4]: a warp's 16-byte accesses are contiguous.
      int4* mine = reinterpret_cast<int4*>(partials) + static_cast<size_t>(item) * (NT / 4) * 128 + rowl;
#pragma unroll
      for (int c16 = 0; c16 < NT / 16; ++c16) {
        uint32_t r[16];
        tmem_ld_32x32b_x16(tmem_d + 16 * c16, r);
        tmem_wait_ld();
        if (c16 == NT / 16 - 1) {                          // last read: hand the accumulator back
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty[acc]);
        }
        if (splits == 1) {
#pragma unroll
          for (int x = 0; x < 16; ++x) {
            const int e = 16 * c16 + x;
            if (e < M && ch < N) {
              const int32_t a = static_cast<int32_t>(r[x]) >> 8;          // exact: the accumulator is 256 * acc
              const float f = __int_as_float(0x4B400000 + a) - 12582912.0f;
              Y[static_cast<size_t>(e) * N + ch] = __float2half_rn(f * (__half2float(__ldg(sx + e)) * swv));
              if (accdbg) accdbg[static_cast<size_t>(e) * N + ch] = a;
            }
          }
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c)
            mine[(4 * c16 + c) * 128] =
                make_int4(static_cast<int32_t>(r[4 * c]) >> 8, static_cast<int32_t>(r[4 * c + 1]) >> 8,
                          static_cast<int32_t>(r[4 * c + 2]) >> 8, static_cast<int32_t>(r[4 * c + 3]) >> 8);
        }
      }
      if (splits == 1) continue;
      named_barrier(1 + eg, 128);                            // the group's stores happen before ...
      if (et == 0) {
        __threadfence();                                     // ... this fence, which orders them before the count
        const unsigned int old = atomicAdd(&counters[tile], 1u);
        const bool last = (old == static_cast<unsigned int>(splits - 1));
        if (last) {
          counters[tile] = 0u;                               // ready for the next call
          __threadfence();                                   // the other items' partials are visible from here on
        }
        last_flag[eg] = last ? 1u : 0u;
      }
      named_barrier(1 + eg, 128);
      const bool finish = (last_flag[eg] != 0u);
      if (finish) {
        // Sum the tile's partials in the fixed order sp = 0, 1, ...: the result does not depend on
        // which item came last.  All loads of a chunk are issued before any is used.
        const int4* base = reinterpret_cast<const int4*>(partials) + static_cast<size_t>(tile) * splits * (NT / 4) * 128 + rowl;
#pragma unroll 1
        for (int c = 0; c < NT / 4; ++c) {
          int4 a = make_int4(0, 0, 0, 0);
#pragma unroll
          for (int h = 0; h < D_MAX_SPLITS; h += 8) {      // eight loads in flight at a time
            if (h < splits) {
              int4 v[8];
#pragma unroll
              for (int sp = 0; sp < 8; ++sp)
                if (h + sp < splits) v[sp] = __ldcg(base + (static_cast<size_t>(h + sp) * (NT / 4) + c) * 128);
#pragma unroll
              for (int sp = 0; sp < 8; ++sp)
                if (h + sp < splits) { a.x += v[sp].x; a.y += v[sp].y; a.z += v[sp].z; a.w += v[sp].w; }
            }
          }
          const int32_t av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const int e = 4 * c + x;
            if (e < M && ch < N) {
              const float f = __int_as_float(0x4B400000 + av[x]) - 12582912.0f;
              Y[static_cast<size_t>(e) * N + ch] = __float2half_rn(f * (__half2float(__ldg(sx + e)) * swv));
              if (accdbg) accdbg[static_cast<size_t>(e) * N + ch] = av[x];
            }
          }
        }
      }
      named_barrier(1 + eg, 128);                            // last_flag may be rewritten by the group's next item
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

template <int NT>
sq_status_t launch_decode(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N, int K, void* Y,
                          int32_t* accdbg, void* workspace, size_t workspace_bytes, cudaStream_t s) {
  using L = DecSmem<NT>;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  const int tiles = (N + 127) / 128, blocks = (K / 128 + 1) / 2;
  int splits = choose_splits(tiles, blocks, sms);
  const size_t part_bytes = static_cast<size_t>(tiles) * splits * 128 * NT * sizeof(int32_t);
  const size_t cnt_off = (part_bytes + 255) / 256 * 256;
  if (splits > 1 && (workspace == nullptr || workspace_bytes < cnt_off + static_cast<size_t>(tiles) * 4)) splits = 1;
  int32_t* partials = nullptr;
  unsigned int* counters = nullptr;
  if (splits > 1) {
    partials = static_cast<int32_t*>(workspace);
    counters = reinterpret_cast<unsigned int*>(static_cast<unsigned char*>(workspace) + cnt_off);
    if (cudaMemsetAsync(counters, 0, static_cast<size_t>(tiles) * 4, s) != cudaSuccess) return SQ_ERR_CUDA;
  }
  CUtensorMap mw, mx;
  if (!make_packed_map(&mw, Wq, N, K / 2, 128) || !make_packed_map(&mx, Xq, M, K / 2, NT)) return SQ_ERR_CUDA;
  auto kern = w4a4_gemm_decode_kernel<NT>;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES) != cudaSuccess)
      return SQ_ERR_CUDA;
    attr_set = true;
  }
  const int items = tiles * splits;
  const int grid = items < sms ? items : sms;
  kern<<<grid, D_THREADS, L::DYN_BYTES, s>>>(mw, mx, static_cast<const __half*>(sx), static_cast<const __half*>(sw), M, N,
                                             K, splits, static_cast<__half*>(Y), accdbg, partials, counters);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace

bool gemm_decode_supported(int64_t M, int64_t N, int64_t K) {
  return M >= 1 && M <= 64 && N >= 128 && (K % 128 == 0) && K >= 256 && (N % 8 == 0);
}

// Workspace of the split-K path: int32 partial tiles, then one counter per tile.
size_t gemm_decode_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (!gemm_decode_supported(M, N, K)) return 0;
  const int sms = sm_count();
  if (sms <= 0) return 0;
  const int NT = M <= 16 ? 16 : (M <= 32 ? 32 : 64);
  const int tiles = static_cast<int>((N + 127) / 128), blocks = static_cast<int>((K / 128 + 1) / 2);
  const int splits = choose_splits(tiles, blocks, sms);
  if (splits == 1) return 0;
  const size_t part_bytes = static_cast<size_t>(tiles) * splits * 128 * NT * sizeof(int32_t);
  return (part_bytes + 255) / 256 * 256 + (static_cast<size_t>(tiles) * 4 + 255) / 256 * 256;
}

sq_status_t launch_w4a4_gemm_decode(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N, int K,
                                    void* Y, int32_t* accdbg, void* workspace, size_t workspace_bytes, cudaStream_t s) {
  if (M <= 16) return launch_decode<16>(Xq, sx, Wq, sw, M, N, K, Y, accdbg, workspace, workspace_bytes, s);
  if (M <= 32) return launch_decode<32>(Xq, sx, Wq, sw, M, N, K, Y, accdbg, workspace, workspace_bytes, s);
  return launch_decode<64>(Xq, sx, Wq, sw, M, N, K, Y, accdbg, workspace, workspace_bytes, s);
}

}  // namespace sq
