// Step 3 for decode-sized problems (M <= 64 tokens): the INT4 x INT4 GEMM with the operands
// swapped and K split, so that every SM streams weights.
//
// With a handful of tokens the GEMM is bound by reading the packed weights once (N K / 2 bytes).
// The weights therefore take the role of the MMA's A operand: a tile is 128 OUTPUT CHANNELS (the
// TMEM lanes), the tokens are the MMA's N (16, 32 or 64).  Four warps read the packed bytes of
// "their" weight row from the TMA staging ring, widen them in registers and store the int8
// operand into a TMEM ring (tcgen05.st); the few token rows are widened through shared memory.
//
// Where the tiles alone do not fill the SMs, K is split over a thread-block cluster of 2, 4 or 8
// CTAs: every CTA of the cluster accumulates its chunk of K for the same tile, then the cluster
// reduce-scatters the exact int32 partial tiles through distributed shared memory -- CTA r of s
// receives, from each of the others, the 128 / s rows it finishes (one slot per source, written
// with st.shared::cluster and handed over with a cluster-scope release/acquire barrier), adds
// them to its own rows, dequantises and writes fp16.  Integer addition makes the result
// independent of any order; no partial tile, counter or scratch exists in global memory.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer, warps 2..9 = two groups of weight
// converters and warps 10..13 = two groups of token unpackers (a group takes every other block:
// a block costs a warp several hundred cycles of waits and fences whatever its size), warps
// 14..21 = epilogue: all eight work on every tile, each on a quarter of the channels and half of
// the tokens (four accumulators, so the epilogue overlaps the main loop of the following tiles).
#include <cuda.h>
#include <cuda_fp16.h>

#include <atomic>

#include "sq_internal.h"
#include "sq_ptx.cuh"

namespace sq {
namespace {

constexpr int D_CONV_GROUPS = 2;          // converter groups; group g takes the blocks g, g + 2, ...
constexpr int D_A_WARPS = 4 * D_CONV_GROUPS, D_B_WARPS = 2 * D_CONV_GROUPS;
constexpr int D_EPI_GROUPS = 2, D_EPI_WARPS = 4 * D_EPI_GROUPS;
constexpr int D_THREADS = (2 + D_A_WARPS + D_B_WARPS + D_EPI_WARPS) * 32;
constexpr int D_S_OP = 4;                // operand stages (TMEM A ring: 4 x 64 columns)
constexpr int D_A_COL0 = 256;
constexpr int D_MAX_SPLITS = 8;            // largest cluster (the portable limit)
constexpr int D_ACCS = 4;                 // accumulators in TMEM (columns 0 .. 4 * NT)

enum DecSite : uint32_t {
  DSITE_ST_EMPTY = 64, DSITE_ST_FULL_A, DSITE_ST_FULL_B, DSITE_EMPTY_A, DSITE_EMPTY_B, DSITE_FULL,
  DSITE_TMEM_FULL, DSITE_TMEM_EMPTY, DSITE_RED_FULL, DSITE_RED_EMPTY, DSITE_TOKENS
};

// Bounded wait until the counter at `flag` (device memory, bumped with release semantics by the CTAs
// that produce the tokens) has reached `target`; what those CTAs wrote before is then visible to this
// thread's loads, and after the proxy fence also to the TMA loads it issues.
__device__ __forceinline__ bool wait_counter(const uint32_t* flag, uint32_t target, uint32_t site, uint32_t limit) {
  for (uint32_t it = 0; it < limit; ++it) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v >= target) {
      asm volatile("fence.proxy.async;" ::: "memory");
      return true;
    }
    __nanosleep(it < 8 ? 100 : 250);       // one thread per CTA polls; keep the counter's L2 line quiet
  }
  atomicCAS(&g_device_status, 0u, (site << 8) | 1u);
  return false;
}

template <int NT>
struct DecSmem {
  static constexpr int S_ST = NT == 64 ? 5 : 6;      // staging stages (256 channels each); deeper rings measured no faster
  static_assert(NT == 16 || NT == 32 || NT == 64, "token-count classes");
  static constexpr int W_ST = 128 * 128;             // packed weight rows, two k-blocks
  static constexpr int X_ST = NT * 128;              // packed token rows, two k-blocks
  static constexpr int X_OP = 2 * NT * 128;          // int8 token rows, two k-block tiles
  // Reduce-scatter slots of one epilogue group: (s - 1) sources x 128 / s rows x NT int32, largest at s = 8.
  static constexpr int RED_GROUP = 128 * NT * 4 / D_MAX_SPLITS * (D_MAX_SPLITS - 1);
  static constexpr int OFF_X_OP = 0;
  static constexpr int OFF_W_ST = OFF_X_OP + D_S_OP * X_OP;
  static constexpr int OFF_X_ST = OFF_W_ST + S_ST * W_ST;
  static constexpr int OFF_RED = OFF_X_ST + S_ST * X_ST;
  static constexpr int OFF_OUT = OFF_RED + RED_GROUP;     // per epilogue warp: 16 tokens x 32 channels fp16
  static constexpr int OFF_BAR = OFF_OUT + D_EPI_WARPS * 1024;
  static constexpr int NUM_BARS = 2 * S_ST + 2 * D_S_OP + 2 * D_ACCS + 2 * D_EPI_GROUPS + 1;
  static constexpr int OFF_MISC = (OFF_BAR + NUM_BARS * 8 + 15) / 16 * 16;   // the scales below are read as float4
  static constexpr int TOTAL = OFF_MISC + 32 + NT * 4;   // TMEM address, then the tokens' scales as floats
  static constexpr int DYN_BYTES = TOTAL + 1024;
  static_assert(DYN_BYTES <= 227 * 1024, "shared memory of one SM");
  static_assert((OFF_MISC + 32) % 16 == 0, "the token scales are read with 16-byte loads");
};

// Widens the 128 staged bytes of NT token rows into two int8 k-block tiles (NT x 128 B each,
// 128-byte swizzle), same byte order as unpack_tile.  64 threads: thread t takes NT / 8 16-byte
// chunks of row t % NT, all loads first.  `second` false: only the first k-block is there.
template <int NT>
__device__ __forceinline__ void unpack_rows(const unsigned char* __restrict__ st, unsigned char* __restrict__ op,
                                            int t, bool second) {
  constexpr int CPT = NT / 8;                              // chunks per thread: 2, 4 or 8
  const int r = t % NT, c0 = (t / NT) * CPT, sw = r & 7;
  const unsigned char* row = st + r * 128;
  uint4 w[CPT];
#pragma unroll
  for (int i = 0; i < CPT; ++i)
    if (second || c0 + i < 4) w[i] = *reinterpret_cast<const uint4*>(row + (((c0 + i) ^ sw) << 4));
#pragma unroll
  for (int i = 0; i < CPT; ++i) {
    const int c = c0 + i, h = c >> 2, j = c & 3;
    if (second || c < 4) {
      uint4 lo, hi;
      lo.x = (w[i].x << 4) & 0xF0F0F0F0u; hi.x = w[i].x & 0xF0F0F0F0u;
      lo.y = (w[i].y << 4) & 0xF0F0F0F0u; hi.y = w[i].y & 0xF0F0F0F0u;
      lo.z = (w[i].z << 4) & 0xF0F0F0F0u; hi.z = w[i].z & 0xF0F0F0F0u;
      lo.w = (w[i].w << 4) & 0xF0F0F0F0u; hi.w = w[i].w & 0xF0F0F0F0u;
      unsigned char* tile = op + h * (NT * 128) + r * 128;
      *reinterpret_cast<uint4*>(tile + ((j ^ sw) << 4)) = lo;
      *reinterpret_cast<uint4*>(tile + (((4 + j) ^ sw) << 4)) = hi;
    }
  }
}

// The grouped form (one launch for the experts of a mixture-of-experts layer): expert g has its own
// packed weights and channel steps and owns `rows[g]` <= NT consecutive token rows from `r0[g]` on, of a
// common Xq, sx and Y.  A tile is (expert, 128 channels); nothing else changes.
constexpr int D_MAX_GROUPS = 16;
struct alignas(64) DecGroups {
  CUtensorMap wmap[D_MAX_GROUPS];
  const __half* sw[D_MAX_GROUPS];
  int r0[D_MAX_GROUPS];
  int rows[D_MAX_GROUPS];
  int count;
};

// The kernel's body for CTA `cta` of `ncta` (a multiple of the cluster size `splits`).  `tokens_ready`:
// nullptr when the tokens come from the kernel before this one in the stream (programmatic dependent
// launch); else a counter that the token-producing CTAs of the SAME launch bump to `tokens_target`
// (the fused kernel of sq_linear_fused.cu).
// GROUPED: the tiles run over the experts of `G` (splits == 1, no token counter); M, sw and tmap_w are unused.
template <int NT, bool GROUPED = false>
__device__ __forceinline__ void w4a4_gemm_decode_body(const CUtensorMap& tmap_w, const CUtensorMap& tmap_x,
                                                      const __half* __restrict__ sx, const __half* __restrict__ sw,
                                                      int M, int N, int K, int splits, __half* __restrict__ Y,
                                                      int32_t* __restrict__ accdbg, int cta, int ncta,
                                                      const uint32_t* tokens_ready, uint32_t tokens_target,
                                                      const DecGroups* G = nullptr) {
  using L = DecSmem<NT>;
  constexpr int S_ST = L::S_ST;
  griddep_launch_dependents();          // a rotate kernel launched behind this one may set itself up on the idle SMs
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* st_full = bars;
  uint64_t* st_empty = bars + S_ST;
  uint64_t* full = bars + 2 * S_ST;
  uint64_t* empty = bars + 2 * S_ST + D_S_OP;
  uint64_t* tmem_full = bars + 2 * S_ST + 2 * D_S_OP;        // [D_ACCS]
  uint64_t* tmem_empty = tmem_full + D_ACCS;                  // [D_ACCS]
  uint64_t* red_full = tmem_empty + D_ACCS;                   // the others' rows have arrived in this CTA's slots (entry 0; entry 1 unused)
  uint64_t* red_empty = red_full + D_EPI_GROUPS;              // the others have read what this CTA sent them
  uint64_t* tok_seen = red_empty + D_EPI_GROUPS;              // the producer has seen the tokens' counter (fused form)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
  float* sxs = reinterpret_cast<float*>(smem + L::OFF_MISC + 32);   // [NT], zero beyond M

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = K / 128;
  const int num_sb = (num_kb + 1) / 2;                 // blocks of 256 channels (the last may be half)
  const int tiles_pe = (N + 127) / 128;                // channel tiles (per expert)
  const int tiles = GROUPED ? tiles_pe * G->count : tiles_pe;
  const uint32_t limit = wait_limit();

  // The cluster (a single CTA when splits == 1) takes the tiles cid, cid + ncl, ...; CTA `crank`
  // of it accumulates the blocks [b0, b1) of every one of them.
  const uint32_t crank = (splits > 1) ? cluster_ctarank() : 0u;
  const int cid = cta / splits, ncl = ncta / splits;
  const int b0 = static_cast<int>(crank * static_cast<uint32_t>(num_sb) / static_cast<uint32_t>(splits));
  const int b1 = static_cast<int>((crank + 1u) * static_cast<uint32_t>(num_sb) / static_cast<uint32_t>(splits));

  // The producer's walk over (tile, block); `budget` blocks are issued per call (waiting for the
  // staging stage of each, except on the first lap of the ring, when every stage is free and the
  // "empty" barriers may not exist yet).  The weights do not depend on the kernel before this
  // one, the tokens do: with `defer_x` only the weights are requested and the blocks are noted.
  int p_tile = cid, p_sb = b0, pre_n = 0;
  int pre_sb[S_ST], pre_row[S_ST];
  uint32_t p_it = 0;
  auto produce = [&](uint32_t budget, bool defer_x) -> bool {
    while (budget > 0 && p_tile < tiles) {
      const int ss = p_it % S_ST;
      if (p_it >= static_cast<uint32_t>(S_ST) &&
          !mbar_wait(&st_empty[ss], ((p_it / S_ST) & 1) ^ 1, DSITE_ST_EMPTY, limit)) return false;
      mbar_arrive_expect_tx(&st_full[ss], L::W_ST + L::X_ST);
      const int pg = GROUPED ? p_tile / tiles_pe : 0;                  // expert of the tile
      const int xrow = GROUPED ? G->r0[pg] : 0;                        // its first token row
      tma_load_2d(smem + L::OFF_W_ST + ss * L::W_ST, GROUPED ? &G->wmap[pg] : &tmap_w, &st_full[ss], p_sb * 128,
                  (GROUPED ? p_tile % tiles_pe : p_tile) * 128);
      if (defer_x) {
        pre_sb[pre_n] = p_sb;
        pre_row[pre_n++] = xrow;
      } else {
        tma_load_2d(smem + L::OFF_X_ST + ss * L::X_ST, &tmap_x, &st_full[ss], p_sb * 128, xrow);
      }
      ++p_it;
      --budget;
      if (++p_sb >= b1) {
        p_sb = b0;
        p_tile += ncl;
      }
    }
    return true;
  };

  if (threadIdx.x == 0) {
    // First of all the weights of the whole staging ring: nothing else is on the critical path.
    for (int s = 0; s < S_ST; ++s) mbar_init(&st_full[s], 1);
    mbar_fence_init();
    produce(S_ST, true);
    tma_prefetch_desc(&tmap_x);
    for (int s = 0; s < S_ST; ++s) mbar_init(&st_empty[s], 6);   // one converter group + one unpacker group
    for (int s = 0; s < D_S_OP; ++s) {
      mbar_init(&full[s], 6);
      mbar_init(&empty[s], 1);
    }
    for (int b = 0; b < D_ACCS; ++b) {
      mbar_init(&tmem_full[b], 1);
      mbar_init(&tmem_empty[b], D_EPI_WARPS);
    }
    // red_full: armed by one thread with the bytes that cross into this CTA; red_empty: one
    // arrival per epilogue group and row that crossed out of it, (s - 1) readers x 128 / s rows.
    const uint32_t crossing = splits > 1 ? static_cast<uint32_t>(D_EPI_GROUPS * (splits - 1) * (128 / splits)) : 1u;
    for (int g = 0; g < D_EPI_GROUPS; ++g) {
      mbar_init(&red_full[g], 1);
      mbar_init(&red_empty[g], crossing);
    }
    mbar_init(tok_seen, 1);
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  // Every CTA's barriers must exist before another CTA stores or arrives on them: only the
  // epilogue warps do that, so only they wait here; the others pick the barrier up at the end.
  if (splits > 1) cluster_arrive_release();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  if (tokens_ready == nullptr) griddep_wait();         // the tokens and their scales come from the kernel before

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------------------------
    // In the fused form this one thread polls the counter of the token-producing CTAs for the whole
    // CTA; the epilogue warps, which read the token steps, wait for its arrival on a local barrier.
    if (lane == 0 && (tokens_ready == nullptr || wait_counter(tokens_ready, tokens_target, DSITE_TOKENS, limit))) {
      if (tokens_ready != nullptr) mbar_arrive(tok_seen);
      for (int i = 0; i < pre_n; ++i)
        tma_load_2d(smem + L::OFF_X_ST + i * L::X_ST, &tmap_x, &st_full[i], pre_sb[i] * 128, pre_row[i]);
      produce(0xFFFFFFFFu, false);
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------------------------
    if (elect_one()) {
      constexpr uint32_t idesc = umma_idesc(/*c=s32*/ 2, /*a=s8*/ 1, /*b=s8*/ 1, 128, NT);
      // One thread issues every MMA, and each instruction it executes costs it several cycles: the
      // descriptors are formed once (those of a block differ from the ring's first by constants in
      // the start-address field, 16-byte units, no carry out of it) and the block's MMAs unrolled.
      const uint64_t b_desc0 = umma_desc_sw128(smem_u32(smem + L::OFF_X_OP));
      constexpr uint32_t KB1 = (NT * 128) >> 4;           // second k-block tile of a stage
      uint32_t it = 0, icount = 0;
      bool ok = true;
      for (int tile = cid; tile < tiles && ok; tile += ncl, ++icount) {
        const uint32_t acc = icount % D_ACCS;
        ok = mbar_wait(&tmem_empty[acc], ((icount / D_ACCS) & 1) ^ 1, DSITE_TMEM_EMPTY, limit);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * NT;
        for (int sb = b0; sb < b1; ++sb, ++it) {
          const uint32_t s = it % D_S_OP;
          ok = mbar_wait(&full[s], (it / D_S_OP) & 1, DSITE_FULL, limit);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t a_tmem = tmem_base + D_A_COL0 + s * 64;
          const uint64_t bd = b_desc0 + static_cast<uint64_t>(s * (L::X_OP >> 4));
          umma_i8_ts(d_tmem, a_tmem, bd, idesc, sb > b0 ? 1u : 0u);
          umma_i8_ts(d_tmem, a_tmem + 8, bd + 2, idesc, 1u);
          umma_i8_ts(d_tmem, a_tmem + 16, bd + 4, idesc, 1u);
          umma_i8_ts(d_tmem, a_tmem + 24, bd + 6, idesc, 1u);
          if (2 * sb + 1 < num_kb) {
            umma_i8_ts(d_tmem, a_tmem + 32, bd + KB1, idesc, 1u);
            umma_i8_ts(d_tmem, a_tmem + 40, bd + (KB1 + 2), idesc, 1u);
            umma_i8_ts(d_tmem, a_tmem + 48, bd + (KB1 + 4), idesc, 1u);
            umma_i8_ts(d_tmem, a_tmem + 56, bd + (KB1 + 6), idesc, 1u);
          }
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
    for (int tile = cid; tile < tiles && ok; tile += ncl) {
      for (int sb = b0; sb < b1 && ok; ++sb, ++it) {
        if ((it % D_CONV_GROUPS) != static_cast<uint32_t>(grp)) continue;
        const int ss = it % S_ST, s = it % D_S_OP;
        ok = mbar_wait(&st_full[ss], (it / S_ST) & 1, DSITE_ST_FULL_A, limit);
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
    for (int tile = cid; tile < tiles && ok; tile += ncl) {
      for (int sb = b0; sb < b1 && ok; ++sb, ++it) {
        if ((it % D_CONV_GROUPS) != static_cast<uint32_t>(grp)) continue;
        const int ss = it % S_ST, s = it % D_S_OP;
        ok = mbar_wait(&st_full[ss], (it / S_ST) & 1, DSITE_ST_FULL_B, limit) &&
             mbar_wait(&empty[s], ((it / D_S_OP) & 1) ^ 1, DSITE_EMPTY_B, limit);
        if (!ok) break;
        unpack_rows<NT>(smem + L::OFF_X_ST + ss * L::X_ST, smem + L::OFF_X_OP + s * L::X_OP, t, 2 * sb + 1 < num_kb);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&full[s]);
          mbar_arrive(&st_empty[ss]);
        }
      }
    }
  } else {
    // ------------------------------ epilogue ------------------------------------------------------
    // Eight warps share every tile: warp q of group eg reads the TMEM lanes 32 q .. 32 q + 31 (all a
    // warp may touch) of the columns [eg * NT / 2, (eg + 1) * NT / 2) -- a single warp per scheduler
    // is bound by its own instruction issue, so the columns are spread over as many as there are.
    constexpr int HALF = NT / 2;                                     // columns (tokens) per group
    constexpr int CH = HALF >= 16 ? 16 : 8;                          // columns per TMEM load
    const int q = warp & 3;
    const int eg = (warp - (2 + D_A_WARPS + D_B_WARPS)) >> 2;
    const int et = static_cast<int>(threadIdx.x) - (2 + D_A_WARPS + D_B_WARPS) * 32;   // 0 .. 255
    const int rowl = q * 32 + lane;                                  // row of the tile = TMEM lane
    // Reduce-scatter geometry: CTA `owner` finishes this thread's row; this CTA finishes the rows
    // [crank * rows_per, (crank + 1) * rows_per).  Slots are [source][4-column chunk][row][4] int32:
    // a warp's 16-byte accesses are contiguous.  One buffer, reused by the CTA's tiles in turn.
    const int rows_per = 128 / splits;
    const uint32_t owner = static_cast<uint32_t>(rowl / rows_per);
    const int rloc = rowl % rows_per;
    const bool mine = (owner == crank);
    const bool warp_owns = __any_sync(0xFFFFFFFFu, mine);
    const bool warp_sends = __any_sync(0xFFFFFFFFu, !mine);
    const uint32_t my_slot = crank < owner ? crank : crank - 1u;     // this CTA's slot in `owner`'s buffer
    const uint32_t send_base = mine ? 0u : cluster_map(smem + L::OFF_RED, owner) + ((my_slot * (NT / 4)) * rows_per + rloc) * 16u;
    const uint32_t send_bar0 = mine ? 0u : cluster_map(&red_full[0], owner);
    const uint32_t red_bytes = static_cast<uint32_t>((splits - 1) * rows_per * NT * 4);   // what crosses into this CTA per tile
    // Output staging of this warp: the accumulator has one channel per thread and the tokens along
    // its registers, Y has the channels contiguous.  A chunk of CH tokens x 32 channels is turned in
    // shared memory -- written as words of two tokens, [token pair][channel] -- so that a thread
    // stores 8 channels (16 bytes) of one token.
    uint32_t* outw = reinterpret_cast<uint32_t*>(smem + L::OFF_OUT + (warp - (2 + D_A_WARPS + D_B_WARPS)) * 1024);
    const int piece = lane & 3, prow = lane >> 2;                    // reader: channels 8 * piece .., token prow (+ 8)
    const bool piece_mine = static_cast<uint32_t>((q * 32 + piece * 8) / rows_per) == crank;
    const uint32_t pick = (prow & 1) ? 0x7632u : 0x5410u;            // the odd or the even token of a pair
    // The tokens' scales as floats (zero beyond M): read once, before any accumulator is ready.
    if (!GROUPED && et < NT) {
      const bool there = tokens_ready == nullptr || mbar_wait(tok_seen, 0, DSITE_TOKENS, limit);
      // written during this launch by another CTA in the fused form: read past the L1 / read-only path
      const __half v = (et < M && there)
                           ? (tokens_ready == nullptr ? sx[et]
                                                      : __ushort_as_half(__ldcg(reinterpret_cast<const unsigned short*>(sx) + et)))
                           : __float2half(0.0f);
      sxs[et] = __half2float(v);
    }
    named_barrier(1, D_EPI_WARPS * 32);
    if (splits > 1) cluster_wait_acquire();                            // the other CTAs' barriers exist
    bool ok = true;
    uint32_t icount = 0;
    for (int tile = cid; tile < tiles && ok; tile += ncl, ++icount) {
      const uint32_t acc = icount % D_ACCS;
      const uint32_t par = 0u, g = icount;                            // reduce buffer and its use count
      const int tg = GROUPED ? tile / tiles_pe : 0;        // expert of the tile
      const int ct = GROUPED ? tile % tiles_pe : tile;     // channel tile
      const int Mt = GROUPED ? G->rows[tg] : M;            // token rows of the tile
      const int trow0 = GROUPED ? G->r0[tg] : 0;           // the first of them in Xq, sx and Y
      const __half* swp = GROUPED ? G->sw[tg] : sw;
      const int ch = ct * 128 + rowl;                      // output channel of this thread
      const float swv = (ch < N) ? __half2float(swp[ch]) : 0.0f;     // in flight while the accumulator is awaited
      if (splits > 1 && eg == 0 && mine && rloc == 0) mbar_arrive_expect_tx(&red_full[par], red_bytes);
      ok = mbar_wait(&tmem_full[acc], (icount / D_ACCS) & 1, DSITE_TMEM_FULL, limit);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tmem_d = tmem_base + acc * NT + eg * HALF + (static_cast<uint32_t>(q * 32) << 16);
      if (warp_sends) {
        // This CTA's chunk of K for rows that another CTA finishes: into that CTA's slot, once it
        // has read what was sent for the CTA's previous tile.
        if (!mine) ok = mbar_wait_acq_cluster(&red_empty[par], (g & 1) ^ 1, DSITE_RED_EMPTY, limit);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        const uint32_t dst = send_base + par * L::RED_GROUP, bar = send_bar0 + par * 8u;
#pragma unroll
        for (int k = 0; k < HALF / CH; ++k) {
          uint32_t r[CH];
          __syncwarp();
          if constexpr (CH == 16) tmem_ld_32x32b_x16(tmem_d + CH * k, r);
          else tmem_ld_32x32b_x8(tmem_d + CH * k, r);
          tmem_wait_ld();
          if (!mine) {
#pragma unroll
            for (int c = 0; c < CH / 4; ++c)
              st_async_v4_cluster(dst + static_cast<uint32_t>(((eg * HALF + CH * k) / 4 + c) * rows_per) * 16u,
                                  static_cast<int32_t>(r[4 * c]) >> 8, static_cast<int32_t>(r[4 * c + 1]) >> 8,
                                  static_cast<int32_t>(r[4 * c + 2]) >> 8, static_cast<int32_t>(r[4 * c + 3]) >> 8, bar);
          }
        }
      }
      if (!warp_owns) {                                      // nothing to finish here: hand the accumulator back
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tmem_empty[acc]);
        continue;
      }
      if (splits > 1) {
        if (mine) ok = mbar_wait_acq_cluster(&red_full[par], g & 1, DSITE_RED_FULL, limit);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
      }
      const int4* red = reinterpret_cast<const int4*>(smem + L::OFF_RED + par * L::RED_GROUP);
#pragma unroll
      for (int k = 0; k < HALF / CH; ++k) {
        uint32_t r[CH];
        __syncwarp();
        if constexpr (CH == 16) tmem_ld_32x32b_x16(tmem_d + CH * k, r);
        else tmem_ld_32x32b_x8(tmem_d + CH * k, r);
        tmem_wait_ld();
        if (k == HALF / CH - 1) {                          // last read: hand the accumulator back
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty[acc]);
        }
        const int t0 = eg * HALF + CH * k;                 // first token of the chunk
        if (mine) {
#pragma unroll
          for (int c = 0; c < CH / 4; ++c) {
            // exact: the accumulator is 256 * (sum of products)
            int4 a = make_int4(static_cast<int32_t>(r[4 * c]) >> 8, static_cast<int32_t>(r[4 * c + 1]) >> 8,
                               static_cast<int32_t>(r[4 * c + 2]) >> 8, static_cast<int32_t>(r[4 * c + 3]) >> 8);
            // The other CTAs' partial sums, four loads in flight at a time.
            const int4* slot = red + (t0 / 4 + c) * rows_per + rloc;
#pragma unroll
            for (int h = 0; h < D_MAX_SPLITS - 1; h += 4) {
              if (h + 1 < splits) {
                int4 v[4];
#pragma unroll
                for (int sp = 0; sp < 4; ++sp)
                  v[sp] = (h + sp + 1 < splits) ? slot[(h + sp) * (NT / 4) * rows_per] : make_int4(0, 0, 0, 0);
#pragma unroll
                for (int sp = 0; sp < 4; ++sp) {
                  a.x += v[sp].x; a.y += v[sp].y; a.z += v[sp].z; a.w += v[sp].w;
                }
              }
            }
            const int e0 = t0 + 4 * c;
            float4 s4;
            if constexpr (GROUPED) {                     // the experts' token steps straight from global memory
              const __half* sxg = sx + trow0;
              s4.x = (e0 + 0 < Mt) ? __half2float(sxg[e0 + 0]) : 0.0f;
              s4.y = (e0 + 1 < Mt) ? __half2float(sxg[e0 + 1]) : 0.0f;
              s4.z = (e0 + 2 < Mt) ? __half2float(sxg[e0 + 2]) : 0.0f;
              s4.w = (e0 + 3 < Mt) ? __half2float(sxg[e0 + 3]) : 0.0f;
            } else {
              s4 = *reinterpret_cast<const float4*>(sxs + e0);
            }
            const __half2 h01 = __floats2half2_rn((__int_as_float(0x4B400000 + a.x) - 12582912.0f) * (s4.x * swv),
                                                  (__int_as_float(0x4B400000 + a.y) - 12582912.0f) * (s4.y * swv));
            const __half2 h23 = __floats2half2_rn((__int_as_float(0x4B400000 + a.z) - 12582912.0f) * (s4.z * swv),
                                                  (__int_as_float(0x4B400000 + a.w) - 12582912.0f) * (s4.w * swv));
            outw[(2 * c) * 32 + lane] = *reinterpret_cast<const uint32_t*>(&h01);
            outw[(2 * c + 1) * 32 + lane] = *reinterpret_cast<const uint32_t*>(&h23);
            if (accdbg && ch < N) {
              const int32_t av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
              for (int x = 0; x < 4; ++x)
                if (e0 + x < Mt) accdbg[static_cast<size_t>(trow0 + e0 + x) * N + ch] = av[x];
            }
          }
        }
        __syncwarp();
        {
          const int ch0 = ct * 128 + q * 32 + piece * 8;
#pragma unroll
          for (int pass = 0; pass < CH / 8; ++pass) {
            const int e = t0 + 8 * pass + prow;
            const uint4* src = reinterpret_cast<const uint4*>(outw + (4 * pass + (prow >> 1)) * 32 + piece * 8);
            const uint4 w0 = src[0], w1 = src[1];
            uint4 v;
            v.x = __byte_perm(w0.x, w0.y, pick);
            v.y = __byte_perm(w0.z, w0.w, pick);
            v.z = __byte_perm(w1.x, w1.y, pick);
            v.w = __byte_perm(w1.z, w1.w, pick);
            if (piece_mine && e < Mt && ch0 < N)
              *reinterpret_cast<uint4*>(Y + static_cast<size_t>(trow0 + e) * N + ch0) = v;
          }
        }
      }
      // The slots may be rewritten -- if the CTA has another tile (nobody waits otherwise).
      if (splits > 1 && mine && tile + ncl < tiles) {
        for (uint32_t d = 0; d < static_cast<uint32_t>(splits); ++d)
          if (d != crank) mbar_arrive_release_cluster(cluster_map(&red_empty[par], d));
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
  if (splits > 1) {
    // Nobody leaves while another CTA may still store or arrive here.  No memory is ordered by
    // this barrier: what crossed CTAs was handed over by the red_* barriers.
    if (warp < 2 + D_A_WARPS + D_B_WARPS) cluster_wait_acquire();      // the set-up barrier, long complete
    cluster_arrive_relaxed();
    cluster_wait_acquire();
  }
}

template <int NT>
__global__ void __launch_bounds__(D_THREADS, 1)
w4a4_gemm_decode_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                        const __half* __restrict__ sx, const __half* __restrict__ sw, int M, int N, int K,
                        int splits, __half* __restrict__ Y, int32_t* __restrict__ accdbg) {
  w4a4_gemm_decode_body<NT>(tmap_w, tmap_x, sx, sw, M, N, K, splits, Y, accdbg, static_cast<int>(blockIdx.x),
                            static_cast<int>(gridDim.x), nullptr, 0u);
}

template <int NT>
__global__ void __launch_bounds__(D_THREADS, 1)
w4a4_gemm_decode_grouped_kernel(const __grid_constant__ DecGroups G, const __grid_constant__ CUtensorMap tmap_x,
                                const __half* __restrict__ sx, int N, int K, __half* __restrict__ Y) {
  w4a4_gemm_decode_body<NT, true>(G.wmap[0], tmap_x, sx, nullptr, 0, N, K, 1, Y, nullptr, static_cast<int>(blockIdx.x),
                                  static_cast<int>(gridDim.x), nullptr, 0u, &G);
}

// Largest number of clusters of `s` CTAs of this kernel that the device holds at once.
template <int NT>
int max_clusters(int s, int sms) {
  using L = DecSmem<NT>;
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
  cfg.dynamicSmemBytes = L::DYN_BYTES;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(s);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, w4a4_gemm_decode_kernel<NT>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    n = 0;
  }
  cache[dev][slot].store(n > 0 ? n : -1, std::memory_order_relaxed);
  return n;
}

// Chooses the cluster size s in {1, 2, 4, 8} over which K is split.  Cost model (cycles, measured):
// a block of 256 channels costs the main loop BLOCK_CYCLES; the exchange through shared memory
// adds SPLIT_CYCLES per tile (the cluster's CTAs meet at every tile); tiles beyond the clusters
// the device holds at once take further waves.
template <int NT>
int choose_splits(int tiles, int blocks, int sms) {
  constexpr double BLOCK_CYCLES = NT == 64 ? 1100.0 : (NT == 32 ? 900.0 : 700.0);
  constexpr double SPLIT_CYCLES = 2500.0;
  int best = 1;
  double best_cost = 0.0;
  for (int s = 1; s <= D_MAX_SPLITS; s *= 2) {
    if (s > 1 && blocks / s < 2) break;
    const int ncl = max_clusters<NT>(s, sms);
    if (ncl <= 0) continue;
    const int waves = (tiles + ncl - 1) / ncl;
    const double cost = static_cast<double>(waves) * (((blocks + s - 1) / s) * BLOCK_CYCLES + (s > 1 ? SPLIT_CYCLES : 0.0));
    if (s == 1 || cost < best_cost * 0.97) {
      best_cost = cost;
      best = s;
    }
  }
  return best;
}

template <int NT>
sq_status_t launch_decode(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N, int K, void* Y,
                          int32_t* accdbg, cudaStream_t s) {
  using L = DecSmem<NT>;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  auto kern = w4a4_gemm_decode_kernel<NT>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), L::DYN_BYTES)) return SQ_ERR_CUDA;
  const int tiles = (N + 127) / 128, blocks = (K / 128 + 1) / 2;
  const int splits = choose_splits<NT>(tiles, blocks, sms);
  const int ncl_max = max_clusters<NT>(splits, sms);
  if (ncl_max <= 0) return SQ_ERR_CUDA;
  CUtensorMap mw, mx;
  if (!make_packed_map(&mw, Wq, N, K / 2, 128) || !make_packed_map(&mx, Xq, M, K / 2, NT)) return SQ_ERR_CUDA;
  const int ncl = tiles < ncl_max ? tiles : ncl_max;
  const cudaError_t err = launch_cluster_maybe_pdl(kern, dim3(static_cast<unsigned>(ncl * splits)), dim3(D_THREADS),
                                                   static_cast<size_t>(L::DYN_BYTES), s, static_cast<unsigned>(splits), mw,
                                                   mx, static_cast<const __half*>(sx), static_cast<const __half*>(sw), M, N,
                                                   K, splits, static_cast<__half*>(Y), accdbg);
  count_launch();
  return err == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

template <int NT>
sq_status_t launch_decode_grouped(const void* Xq, const void* sx, int64_t M_total, int count, const void* const* Wq,
                                  const void* const* sw, const int64_t* r0, const int64_t* rows, int N, int K, void* Y,
                                  cudaStream_t s) {
  using L = DecSmem<NT>;
  const int sms = sm_count();
  if (sms <= 0) return SQ_ERR_CUDA;
  auto kern = w4a4_gemm_decode_grouped_kernel<NT>;
  if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), L::DYN_BYTES)) return SQ_ERR_CUDA;
  DecGroups G;
  CUtensorMap mx;
  if (!make_packed_map(&mx, Xq, static_cast<uint64_t>(M_total), K / 2, NT)) return SQ_ERR_CUDA;
  for (int g = 0; g < D_MAX_GROUPS; ++g) {
    const int src = g < count ? g : 0;                   // unused entries repeat the first (never read)
    if (!make_packed_map(&G.wmap[g], Wq[src], N, K / 2, 128)) return SQ_ERR_CUDA;
    G.sw[g] = static_cast<const __half*>(sw[src]);
    G.r0[g] = static_cast<int>(r0[src]);
    G.rows[g] = static_cast<int>(rows[src]);
  }
  G.count = count;
  const int tiles = ((N + 127) / 128) * count;
  const int grid = tiles < sms ? tiles : sms;
  const cudaError_t err = launch_maybe_pdl(kern, dim3(static_cast<unsigned>(grid)), dim3(D_THREADS),
                                           static_cast<size_t>(L::DYN_BYTES), s, G, mx, static_cast<const __half*>(sx), N,
                                           K, static_cast<__half*>(Y));
  count_launch();
  return err == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace

int gemm_decode_max_groups() { return D_MAX_GROUPS; }

// Step 3 for up to D_MAX_GROUPS experts in one launch: expert g owns rows[g] (1..64) token rows from r0[g]
// on of Xq [M_total x K/2], sx and Y, and has its own Wq[g], sw[g].  Shapes as gemm_decode_supported.
sq_status_t launch_w4a4_gemm_decode_grouped(const void* Xq, const void* sx, int64_t M_total, int count,
                                            const void* const* Wq, const void* const* sw, const int64_t* r0,
                                            const int64_t* rows, int N, int K, void* Y, cudaStream_t s) {
  if (count < 1 || count > D_MAX_GROUPS) return SQ_ERR_INVALID_ARG;
  int64_t most = 0;
  for (int g = 0; g < count; ++g) most = rows[g] > most ? rows[g] : most;
  if (most < 1 || most > 64) return SQ_ERR_INVALID_ARG;
  if (most <= 16) return launch_decode_grouped<16>(Xq, sx, M_total, count, Wq, sw, r0, rows, N, K, Y, s);
  if (most <= 32) return launch_decode_grouped<32>(Xq, sx, M_total, count, Wq, sw, r0, rows, N, K, Y, s);
  return launch_decode_grouped<64>(Xq, sx, M_total, count, Wq, sw, r0, rows, N, K, Y, s);
}

bool gemm_decode_supported(int64_t M, int64_t N, int64_t K) {
  return M >= 1 && M <= 64 && N >= 128 && (K % 128 == 0) && K >= 256 && (N % 8 == 0);
}

sq_status_t launch_w4a4_gemm_decode(const void* Xq, const void* sx, const void* Wq, const void* sw, int M, int N, int K,
                                    void* Y, int32_t* accdbg, cudaStream_t s) {
  if (M <= 16) return launch_decode<16>(Xq, sx, Wq, sw, M, N, K, Y, accdbg, s);
  if (M <= 32) return launch_decode<32>(Xq, sx, Wq, sw, M, N, K, Y, accdbg, s);
  return launch_decode<64>(Xq, sx, Wq, sw, M, N, K, Y, accdbg, s);
}

}  // namespace sq
