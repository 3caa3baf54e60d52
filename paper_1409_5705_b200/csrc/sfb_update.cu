// Reconstruct-and-apply step of SFB on sm_100a (Section 3, Figure 1: every worker rebuilds the K rank-1 updates
// from the gathered sufficient factors and applies them):   W <- W + alpha * U^T V,   alpha = -eta,
// as ONE pass over W: the tensor-core product of a tile is combined with the fp32 tile of W while both are on
// the SM, so the reconstructed update matrix never exists in memory and W makes one HBM round trip.
//
// Kernel shape.  Clusters of two CTAs on the two SMs of a TPC drive one tcgen05.mma.cta_group::2: the pair owns a
// 256 x 256 tile of W, CTA r of the pair holds rows [128 r, 128 r + 128) of it in its TMEM (fp32, two accumulator
// stages of 256 columns), loads its own 128 x 64 slice of U^T and its own 128 x 64 half of the V^T slice per
// k-block (32 KB per stage instead of the 48 KB a single-CTA 128 x 256 tile needs), and streams its own
// 128 x 256 fp32 half of the W tile.
// Warps of a CTA: 0 = TMA producer, 1 = MMA issuer (leader CTA only) and TMEM owner, 2..9 = epilogue.
// Epilogue warp (q, h): TMEM lane quarter q (32 rows of W), column half h (128 columns), in four chunks of
// 32 x 32.  Each warp owns a ring of three 4 KB slots: the W chunk lands there by TMA (two chunks in flight per
// warp, 64 KB per SM), is combined in place with the accumulator chunk and goes back by TMA from the same slot;
// the bf16 copy of the new chunk is read back from the slot and stored as 64-byte row pieces.  Shared memory is
// the scarce resource: 4 operand stages (128 KB) + the rings (96 KB).  Measured: a fourth operand stage gains
// more (the operand loads slow down when they share L2 with the stream of W) than a fourth ring slot.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>

#include "sfb_ptx.cuh"
#include "sfb_tc.h"

namespace sfb {
namespace {

using namespace ptx;

constexpr int UM = 128;                 // rows of W per CTA (256 per pair)
constexpr int UN = 256;                 // columns of W per tile
constexpr int UK = 64, UMMA_K = 16;
constexpr int kStages = 4;
constexpr int kBytesA = UM * UK * 2;          // 16 KB: this CTA's rows of U^T
constexpr int kBytesB = (UN / 2) * UK * 2;    // 16 KB: this CTA's half of the V^T rows
constexpr int kStageBytes = kBytesA + kBytesB;
constexpr int kChunk = 32;
constexpr int kSlotBytes = 32 * kChunk * 4;   // 4 KB
constexpr int kRing = 3;                      // slots per epilogue warp
constexpr int kPend = 1;                      // TMA stores of a warp that may still be reading their slots
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kChunksPerWarp = (UN / 2) / kChunk;   // 4
constexpr int kTmemCols = 512;
constexpr int kBars = 2 * kStages + 4 + kEpiWarps * kRing;
constexpr int kSmem = kStages * kStageBytes + kEpiWarps * kRing * kSlotBytes + kBars * 8 + 16 + 1024;

struct UpdParams {
  int32_t rows, cols;          // shape of W
  int32_t tilesM, tilesN;      // pair tiles: 256 rows x 256 columns
  int32_t nseg, kseg;          // contraction: nseg segments of kseg k-blocks (3 segments: split-bf16 product)
  // Segment s reads U^T from column a_off<s> and V^T from column b_off<s>.  Scalars, not arrays: indexing an
  // array of a kernel parameter with a run-time index moves the whole parameter block to local memory.
  int32_t a_off0, a_off1, a_off2, b_off0, b_off1, b_off2;
  float alpha;
  int32_t prox_kind;           // entry-wise prox applied to the updated value (0 none, 1 soft-threshold, 2 scale)
  float prox_a;
  __nv_bfloat16* shadow;       // bf16 copy of the updated W (or null), row pitch shadow_ld elements
  float* shadow32;             // (big | small) tf32 copy of the updated W: big at column c, small at shadow_half + c
  int64_t shadow_ld;
  int64_t shadow_half;
  uint32_t* status;
  unsigned long long* copy_counters;   // [0] row pieces of the bf16 copy visited, [1] of them rewritten (or null)
};

__device__ __forceinline__ float to_tf32(float x) {
  uint32_t u;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
  return __uint_as_float(u);
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Tile order: row blocks are taken in groups of kGroup; within a group the tiles are numbered row block fastest,
// then column block.  The pairs that run at the same time therefore work on kGroup blocks of U^T (512 KB each) and
// on about 74 / kGroup blocks of V^T: every operand line has a handful of readers at a time instead of one block of
// U^T having forty (measured: groups of 8 are 4-5 % faster than column-block-fastest order, groups of 37 or more
// slower again).  All of V^T (marked evict_last) and the group's blocks of U^T stay in L2.
constexpr int kGroup = 8;
__device__ __forceinline__ void tile_origin(const UpdParams& p, int tile, int& m0, int& n0) {
  const int per_group = kGroup * p.tilesN;
  const int grp = tile / per_group, within = tile - grp * per_group;
  const int gsz = min(kGroup, p.tilesM - grp * kGroup);       // the last group may be smaller
  const int tm = grp * kGroup + within % gsz, tn = within / gsz;
  m0 = tm * (2 * UM);
  n0 = tn * UN;
}

// TF32: the operands are 32-bit words read as tf32 (32 elements per 128-byte k-block), see the forward kernel.
// SHADOW: the operand copy of the new W that the epilogue writes beside it for the next forward product:
// 0 none, 1 bf16, 2 the (big | small) pair of tf32 words of the fp32-on-tensor-cores mode.
template <int SHADOW, bool TF32 = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
update_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                   const __grid_constant__ CUtensorMap tmC, const UpdParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = smem + kStages * kBytesA;
  uint8_t* sRing = smem + kStages * kStageBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sRing + kEpiWarps * kRing * kSlotBytes);
  uint64_t* full = bars;                       // leader's copy is the one in use: both CTAs' loads signal it
  uint64_t* empty = bars + kStages;            // one per CTA: the MMA's commit arrives on both
  uint64_t* tfull = bars + 2 * kStages;        // one per CTA (commit arrives on both)
  uint64_t* tempty = bars + 2 * kStages + 2;   // leader's copy: 8 epilogue warps of each CTA arrive on it
  uint64_t* rfull = bars + 2 * kStages + 4;    // per epilogue warp and ring slot
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kBars);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int ntiles = p.tilesM * p.tilesN;
  const int my_tiles = pair < ntiles ? (ntiles - 1 - pair) / npairs + 1 : 0;
  const int numK = p.nseg * p.kseg;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], 2 * kEpiWarps); }
    for (int i = 0; i < kEpiWarps * kRing; ++i) mbar_init(&rfull[i], 1);
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmA); prefetch_tmap(&tmB); prefetch_tmap(&tmC);
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, kTmemCols); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_arrive();          // both CTAs' barriers exist and both have their TMEM before anyone signals the peer
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer (each CTA loads its own rows of U^T and its own half of the V^T rows) ---------
    if (lane == 0) {
      const uint64_t pol_keep = policy_evict_last(), pol_norm = policy_evict_normal();
      uint32_t it = 0;
      bool ok = true;
      for (int tl = 0; tl < my_tiles && ok; ++tl) {
        int m0, n0;
        tile_origin(p, pair + tl * npairs, m0, n0);
        for (int seg = 0; seg < p.nseg && ok; ++seg) {
          for (int kl = 0; kl < p.kseg; ++kl, ++it) {
            const uint32_t s = it % kStages, ph = (it / kStages) & 1;
            if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; break; }
            if (rank == 0) mbar_expect_tx(&full[s], 2 * kStageBytes);
            const uint32_t full_leader = mapa_u32(smem_u32(&full[s]), 0);
            const int xa = (seg == 0 ? p.a_off0 : seg == 1 ? p.a_off1 : p.a_off2) + kl * (TF32 ? UK / 2 : UK);
            const int xb = (seg == 0 ? p.b_off0 : seg == 1 ? p.b_off1 : p.b_off2) + kl * (TF32 ? UK / 2 : UK);
            tma_load_2d_pair(sA + s * kBytesA, &tmA, xa, m0 + static_cast<int>(rank) * UM, full_leader, pol_norm);
            tma_load_2d_pair(sB + s * kBytesB, &tmB, xb, n0 + static_cast<int>(rank) * (UN / 2), full_leader, pol_keep);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: one thread of the leader CTA drives both SMs ----------------
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = TF32 ? umma_idesc_tf32(2 * UM, UN) : umma_idesc_bf16(2 * UM, UN);
      uint32_t it = 0;
      bool ok = true;
      for (int tl = 0; tl < my_tiles && ok; ++tl) {
        const uint32_t a = tl & 1, aph = (tl >> 1) & 1;
        if (!mbar_wait(&tempty[a], aph ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * UN;
        for (int kb = 0; kb < numK; ++kb, ++it) {
          const uint32_t s = it % kStages, ph = (it / kStages) & 1;
          if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = umma_desc_k128(smem_u32(sA + s * kBytesA));
          const uint64_t db = umma_desc_k128(smem_u32(sB + s * kBytesB));
#pragma unroll
          for (int k = 0; k < UK / UMMA_K; ++k) {          // four MMAs of 32 bytes of contraction each, either kind
            const uint64_t adv = static_cast<uint64_t>(k * UMMA_K * 2 / 16);
            if (TF32) umma_tf32_pair(d_tmem, da + adv, db + adv, idesc, (kb | k) != 0 ? 1u : 0u);
            else umma_bf16_pair(d_tmem, da + adv, db + adv, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit_pair(&empty[s], 3);          // both CTAs' stage s is free once these MMAs have read it
        }
        if (ok) umma_commit_pair(&tfull[a], 3);    // both CTAs' halves of the accumulator are complete
      }
    }
  } else {
    // ---------------- epilogue: warp (q, h) = TMEM lane quarter q, column half h ----------------
    const int e = warp - 2, q = warp & 3, h = e >> 2;
    uint8_t* ring = sRing + e * kRing * kSlotBytes;
    uint64_t* rf = rfull + e * kRing;
    const uint32_t nchunks = static_cast<uint32_t>(my_tiles) * kChunksPerWarp;
    // Default L2 priority for the tiles of W: with evict_first on this traffic the written lines are pushed to
    // HBM at once, in small pieces between the reads, and the measured rate drops by a quarter.
    const uint64_t pol_w = policy_evict_normal();
    const uint32_t tempty_leader0 = mapa_u32(smem_u32(&tempty[0]), 0), tempty_leader1 = mapa_u32(smem_u32(&tempty[1]), 0);
    const int row_in_tile = static_cast<int>(rank) * UM + q * 32;
    bool ok = true;
    uint32_t copy_written = 0;           // row pieces of the bf16 copy this warp rewrote
    uint32_t lg = 0;                     // next chunk to request
    auto issue_load = [&]() {
      if (lg >= nchunks) return;
      int m0, n0;
      tile_origin(p, pair + static_cast<int>(lg / kChunksPerWarp) * npairs, m0, n0);
      const uint32_t slot = lg % kRing;
      mbar_expect_tx(&rf[slot], kSlotBytes);
      tma_load_2d_hint(ring + slot * kSlotBytes, &tmC, n0 + h * (UN / 2) + static_cast<int>(lg % kChunksPerWarp) * kChunk,
                       m0 + row_in_tile, &rf[slot], pol_w);
      ++lg;
    };
    if (lane == 0)
      for (int i = 0; i < kRing - kPend; ++i) issue_load();
    uint32_t g = 0;
    for (int tl = 0; tl < my_tiles && ok; ++tl) {
      int m0, n0;
      tile_origin(p, pair + tl * npairs, m0, n0);
      const uint32_t a = tl & 1, aph = (tl >> 1) & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&tfull[a], aph, abort_flag))) { ok = false; break; }
      tc_fence_after();
      const int y0 = m0 + row_in_tile;
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + a * UN + h * (UN / 2);
      uint32_t acc0[32], acc1[32];
      tmem_ld_32x32(t_addr, acc0);
      auto process = [&](uint32_t (&acc)[32], uint32_t (&nxt)[32], int c) -> bool {
        tmem_ld_wait();                                      // chunk c's accumulators are in registers
        if (c + 1 < kChunksPerWarp) {
          tmem_ld_32x32(t_addr + (c + 1) * kChunk, nxt);     // chunk c+1 streams in during this chunk's work
        } else {
          tc_fence_before();                                 // last TMEM read of the tile by this warp: hand the
          __syncwarp();                                      // accumulator stage back to the leader's MMA warp
          if (lane == 0) mbar_arrive_cluster(a ? tempty_leader1 : tempty_leader0);
        }
        const uint32_t slot = g % kRing;
        uint8_t* sl = ring + slot * kSlotBytes;
        if (!__all_sync(0xffffffffu, mbar_wait(&rf[slot], (g / kRing) & 1, abort_flag))) return false;
        const int x0 = n0 + h * (UN / 2) + c * kChunk;
        uint32_t differs = 0;      // SHADOW == 1: does the bf16 rounding of any of this row's 32 values change?
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          float4* wp = reinterpret_cast<float4*>(sl + lane * 128 + ((j ^ (lane & 7)) << 4));
          float4 w = *wp;
          uint32_t o01 = 0, o23 = 0;
          if (SHADOW == 1) { o01 = pack2(w.x, w.y); o23 = pack2(w.z, w.w); }
          w.x = fmaf(p.alpha, __uint_as_float(acc[4 * j + 0]), w.x);
          w.y = fmaf(p.alpha, __uint_as_float(acc[4 * j + 1]), w.y);
          w.z = fmaf(p.alpha, __uint_as_float(acc[4 * j + 2]), w.z);
          w.w = fmaf(p.alpha, __uint_as_float(acc[4 * j + 3]), w.w);
          if (p.prox_kind != 0) {
            w.x = prox_entry(w.x, p.prox_kind, p.prox_a); w.y = prox_entry(w.y, p.prox_kind, p.prox_a);
            w.z = prox_entry(w.z, p.prox_kind, p.prox_a); w.w = prox_entry(w.w, p.prox_kind, p.prox_a);
          }
          *wp = w;
          if (SHADOW == 1) differs |= (o01 ^ pack2(w.x, w.y)) | (o23 ^ pack2(w.z, w.w));
        }
        // The bf16 copy holds bf16(W) when the pass starts (set-up, refresh, label rows and this kernel keep it so): a
        // row piece whose 32 roundings all stay the same already holds bf16 of the new values and is not rewritten.
        // With updates of a few fp32 spacings per entry that is most of the matrix; the copy stays exact either way.
        const uint32_t rowmask = SHADOW == 1 ? __ballot_sync(0xffffffffu, differs != 0) : 0u;
        fence_proxy_async_smem();
        __syncwarp();                                        // every lane has rewritten its row of the slot
        if (lane == 0) {
          if (x0 < p.cols && y0 < p.rows) tma_store_2d_hint(&tmC, sl, x0, y0, pol_w);
          tma_commit_group();
          if (g >= kPend) tma_wait_group_read<kPend>();      // the store of chunk g-kPend has read its slot:
          issue_load();                                      // refill it with chunk g + kRing - kPend
        }
        if (SHADOW == 2) {
          // (big | small) tf32 copy of the chunk, read back from the slot with 8 lanes per row: 128-byte row pieces
          const int sub = lane >> 3, jj = lane & 7;
#pragma unroll
          for (int r0 = 0; r0 < 32; r0 += 4) {
            const int r = r0 + sub;
            const float4 w = *reinterpret_cast<const float4*>(sl + r * 128 + ((jj ^ (r & 7)) << 4));
            const int col = x0 + 4 * jj;
            if (y0 + r < p.rows && col < p.cols) {
              const float4 b = make_float4(to_tf32(w.x), to_tf32(w.y), to_tf32(w.z), to_tf32(w.w));
              float* d = p.shadow32 + static_cast<int64_t>(y0 + r) * p.shadow_ld + col;
              *reinterpret_cast<float4*>(d) = b;
              *reinterpret_cast<float4*>(d + p.shadow_half) =
                  make_float4(to_tf32(w.x - b.x), to_tf32(w.y - b.y), to_tf32(w.z - b.z), to_tf32(w.w - b.w));
            }
          }
        }
        if (SHADOW == 1) {
          // bf16 copy of the chunk, read back from the slot with 8 lanes per row (4 rows per pass): each row's
          // 32 values leave as one 64-byte piece instead of 32 lanes storing 16 bytes to 32 different rows.
          const int sub = lane >> 3, jj = lane & 7;
          if (__popc(rowmask) > 12) {
            // most rows changed: all 32 in eight fixed passes (cheaper than picking them one by one)
            copy_written += 32;
#pragma unroll
            for (int r0 = 0; r0 < 32; r0 += 4) {
              const int r = r0 + sub;
              const float4 w = *reinterpret_cast<const float4*>(sl + r * 128 + ((jj ^ (r & 7)) << 4));
              const int col = x0 + 4 * jj;
              if (y0 + r < p.rows && col < p.shadow_ld)
                *reinterpret_cast<uint2*>(p.shadow + static_cast<int64_t>(y0 + r) * p.shadow_ld + col) =
                    make_uint2(pack2(w.x, w.y), pack2(w.z, w.w));
            }
          } else {
          copy_written += __popc(rowmask);
          // the changed rows, four per pass: lane group `sub` takes the (sub+1)-th changed row still to do
#pragma unroll 1
          for (uint32_t todo = rowmask; todo != 0;) {
            const uint32_t r = __fns(todo, 0, sub + 1);           // 0xffffffff when fewer than sub+1 rows are left
            if (r < 32u) {
              const float4 w = *reinterpret_cast<const float4*>(sl + r * 128 + ((jj ^ (r & 7)) << 4));
              const int col = x0 + 4 * jj;
              if (y0 + static_cast<int>(r) < p.rows && col < p.shadow_ld)
                *reinterpret_cast<uint2*>(p.shadow + static_cast<int64_t>(y0 + r) * p.shadow_ld + col) =
                    make_uint2(pack2(w.x, w.y), pack2(w.z, w.w));
            }
            todo &= todo - 1; todo &= todo - 1; todo &= todo - 1; todo &= todo - 1;    // drop the four lowest set bits
          }
          }
        }
        ++g;
        return true;
      };
#pragma unroll 1
      for (int c = 0; c < kChunksPerWarp && ok; c += 2) {
        ok = process(acc0, acc1, c);
        if (ok) ok = process(acc1, acc0, c + 1);
      }
    }
    if (lane == 0) tma_wait_group<0>();
    if (SHADOW == 1 && lane == 0 && p.copy_counters) {
      atomicAdd(&p.copy_counters[0], 32ull * nchunks);
      atomicAdd(&p.copy_counters[1], static_cast<unsigned long long>(copy_written));
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // A wait ran out: report it and give copies in flight a bounded time to land.
    if (threadIdx.x == 0) atomicOr(p.status, SFB_STATUS_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  cluster_arrive();          // neither CTA frees its TMEM or exits while the other may still signal or write it
  cluster_wait();
  if (warp == 1) { tc_fence_after(); tmem_dealloc_pair(tmem_base, kTmemCols); }
}

// The label entries of the K factors, u_iy = p_iy - 1, which the bf16 operand leaves out (it holds 0 there):
//   W[y] <- W[y] + eta * sum_{i : y_i = y} (1 - p_iy) x_i     in fp32, from the fp32 copy of the samples.
// One block per (sample, 1024 columns); the blocks of the first sample of each class list that class's samples
// (ascending, so the sum has the same order every run; no atomics), sum them and refresh the bf16 copy of the row.
constexpr int kLabelList = 1024;
__global__ void __launch_bounds__(256) label_rows_kernel(float* __restrict__ W, int64_t rows, int64_t cols,
                                                         const float* __restrict__ Xf, const int32_t* __restrict__ labels,
                                                         const float* __restrict__ coef, int K, float eta, __nv_bfloat16* __restrict__ shadow,
                                                         int64_t shadow_ld) {
  __shared__ int first;
  __shared__ int count;
  __shared__ int list[kLabelList];
  __shared__ int warp_tot[8];
  const int i = blockIdx.x;
  const int32_t y = labels[i];
  if (y < 0 || y >= rows) return;              // out-of-range ids were flagged by the softmax pass
  if (threadIdx.x == 0) first = 1;
  __syncthreads();
  for (int j = threadIdx.x; j < i; j += 256)
    if (labels[j] == y) first = 0;
  __syncthreads();
  if (!first) return;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int64_t c = static_cast<int64_t>(threadIdx.x) * 4 + static_cast<int64_t>(blockIdx.y) * 1024;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int base = i; base < K; base += kLabelList) {
    // ordered compaction of the matching sample indices in [base, base + kLabelList)
    if (threadIdx.x == 0) count = 0;
    __syncthreads();
    for (int off = 0; off < kLabelList; off += 256) {
      const int j = base + off + threadIdx.x;
      const bool hit = j < K && labels[j] == y;
      const unsigned m = __ballot_sync(0xffffffffu, hit);
      if (lane == 0) warp_tot[wid] = __popc(m);
      __syncthreads();
      int pre = count;
      for (int w = 0; w < wid; ++w) pre += warp_tot[w];
      if (hit) list[pre + __popc(m & ((1u << lane) - 1))] = j;
      __syncthreads();
      if (threadIdx.x == 0) {
        int t = 0;
        for (int w = 0; w < 8; ++w) t += warp_tot[w];
        count += t;
      }
      __syncthreads();
    }
    if (c < cols) {
      const int n = count;
      for (int k = 0; k < n; ++k) {
        const int j = list[k];
        const float4 x = *reinterpret_cast<const float4*>(Xf + static_cast<int64_t>(j) * cols + c);
        const float cf = coef[j];
        acc.x = fmaf(cf, x.x, acc.x); acc.y = fmaf(cf, x.y, acc.y);
        acc.z = fmaf(cf, x.z, acc.z); acc.w = fmaf(cf, x.w, acc.w);
      }
    }
    __syncthreads();
  }
  if (c < cols) {
    float4* wp = reinterpret_cast<float4*>(W + static_cast<int64_t>(y) * cols + c);
    float4 w = *wp;
    w.x = fmaf(eta, acc.x, w.x); w.y = fmaf(eta, acc.y, w.y);
    w.z = fmaf(eta, acc.z, w.z); w.w = fmaf(eta, acc.w, w.w);
    *wp = w;
    if (shadow)
      *reinterpret_cast<uint2*>(shadow + static_cast<int64_t>(y) * shadow_ld + c) =
          make_uint2(pack2(w.x, w.y), pack2(w.z, w.w));
  }
}

}  // namespace

#define CKC(call)                                       \
  do {                                                  \
    cudaError_t e__ = (call);                           \
    if (e__ != cudaSuccess) {                           \
      ctx->last_cuda = static_cast<int>(e__);           \
      return SFB_ERR_CUDA;                              \
    }                                                   \
  } while (0)

template <int SHADOW, bool TF32 = false>
static cudaError_t prepare_kernel(int* max_pairs) {
  cudaError_t e = cudaFuncSetAttribute(update_pair_kernel<SHADOW, TF32>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmem;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  int n = 0;
  e = cudaOccupancyMaxActiveClusters(&n, update_pair_kernel<SHADOW, TF32>, &cfg);
  if (e != cudaSuccess) return e;
  *max_pairs = n;
  return cudaSuccess;
}

int tc_update_init(sfb_ctx* ctx, TcState* st) {
  int a = 0, b = 0, t = 0;
  CKC(prepare_kernel<1>(&a));
  CKC(prepare_kernel<0>(&b));
  CKC((prepare_kernel<2, true>(&t)));
  st->max_pairs = std::min(std::min(a, b), t);
  if (st->max_pairs < 1) return SFB_ERR_ARCH;     // the device cannot host a CTA pair of this kernel
  return SFB_OK;
}

// fp32 mode on the tensor cores (MLR): U^T and V^T are (big | small) pairs of tf32 words, [rows x 2 Kp] and
// [cols x 2 Kp] with Kp the pair count rounded up to 32;  U^T V = Ub Vb + Ub Vs + Us Vb  (Us Vs, 2^-22 of the product,
// is dropped).  The label entries are part of U here: no separate label-row pass, no bf16 copy of W.
int tc32_update(sfb_ctx* ctx) {
  if (ctx->sparse_v) return sparse_update(ctx);         // writes the (big | small) copy as well
  const sfb_config& c = ctx->cfg;
  const TcState* st = static_cast<const TcState*>(ctx->tc);
  const Layout& L = ctx->lay;
  const int64_t Kp = L.Kp;                                  // a multiple of 32
  CUtensorMap ma, mb, mc;
  if (!make_map(st, &ma, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, ctx->at<float>(L.UT), 2 * Kp, c.rows, 2 * Kp * 4, UK / 2, UM) ||
      !make_map(st, &mb, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, ctx->at<float>(L.VT), 2 * Kp, c.cols, 2 * Kp * 4, UK / 2, UN / 2) ||
      !make_map(st, &mc, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, ctx->W, c.cols, c.rows, c.cols * 4, kChunk, 32))
    return SFB_ERR_CUDA;
  UpdParams p{};
  p.rows = static_cast<int32_t>(c.rows); p.cols = static_cast<int32_t>(c.cols);
  p.tilesM = static_cast<int32_t>((c.rows + 2 * UM - 1) / (2 * UM));
  p.tilesN = static_cast<int32_t>((c.cols + UN - 1) / UN);
  p.kseg = static_cast<int32_t>(Kp / (UK / 2));
  p.alpha = -ctx->step;
  p.prox_kind = ctx->prox_kind; p.prox_a = ctx->prox_a;
  p.status = ctx->at<uint32_t>(L.status);
  // The two cross terms first, big*big last: the tensor core rounds its fp32 accumulator at every instruction, by an
  // amount relative to what the accumulator holds, so the many roundings of the small terms should happen while it is
  // still small (measured: 3 times less error than with big*big first).
  p.nseg = 3;
  p.a_off0 = 0; p.a_off1 = static_cast<int32_t>(Kp); p.a_off2 = 0;
  p.b_off0 = static_cast<int32_t>(Kp); p.b_off1 = 0; p.b_off2 = 0;
  // the epilogue also writes the (big | small) copy of the new W, the operand of the next forward product
  p.shadow = nullptr; p.shadow32 = ctx->at<float>(L.Ws); p.shadow_ld = 2 * L.colsp; p.shadow_half = L.colsp;
  const int64_t tiles = static_cast<int64_t>(p.tilesM) * p.tilesN;
  const unsigned grid = 2u * static_cast<unsigned>(std::min<int64_t>(tiles, st->max_pairs));
  update_pair_kernel<2, true><<<grid, kThreads, kSmem, ctx->stream>>>(ma, mb, mc, p);
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

int tc_update(sfb_ctx* ctx) {
  const sfb_config& c = ctx->cfg;
  const TcState* st = static_cast<const TcState*>(ctx->tc);
  const Layout& L = ctx->lay;
  const bool split = c.model != SFB_MLR;
  const int64_t kw = split ? 2 * L.Kp : ctx->K;       // operand width in elements; pitch is Kp or 2*Kp
  const int64_t pitch = (split ? 2 * L.Kp : L.Kp) * 2;
  CUtensorMap ma, mb, mc;
  if (!make_map(st, &ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, ctx->at<__nv_bfloat16>(L.UT), kw, c.rows, pitch, UK, UM) ||
      !make_map(st, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, ctx->at<__nv_bfloat16>(L.VT), kw, c.cols, pitch, UK, UN / 2) ||
      !make_map(st, &mc, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, ctx->W, c.cols, c.rows, c.cols * 4, kChunk, 32))
    return SFB_ERR_CUDA;
  UpdParams p{};
  p.rows = static_cast<int32_t>(c.rows); p.cols = static_cast<int32_t>(c.cols);
  p.tilesM = static_cast<int32_t>((c.rows + 2 * UM - 1) / (2 * UM));
  p.tilesN = static_cast<int32_t>((c.cols + UN - 1) / UN);
  p.kseg = static_cast<int32_t>(L.Kp / UK);
  p.alpha = -ctx->step;
  p.prox_kind = ctx->prox_kind; p.prox_a = ctx->prox_a;
  p.status = ctx->at<uint32_t>(L.status);
  const int64_t tiles = static_cast<int64_t>(p.tilesM) * p.tilesN;
  const unsigned grid = 2u * static_cast<unsigned>(std::min<int64_t>(tiles, st->max_pairs));
  if (split) {
    // U^T V = Uhi Vhi + Uhi Vlo + Ulo Vhi (+ Ulo Vlo, dropped: 2^-16 of the product)
    p.nseg = 3;
    p.a_off0 = 0; p.a_off1 = 0; p.a_off2 = static_cast<int32_t>(L.Kp);
    p.b_off0 = 0; p.b_off1 = static_cast<int32_t>(L.Kp); p.b_off2 = 0;
    p.shadow = nullptr; p.shadow_ld = 0;
    update_pair_kernel<0><<<grid, kThreads, kSmem, ctx->stream>>>(ma, mb, mc, p);
    count_launch();
    CKC(cudaGetLastError());
    return SFB_OK;
  }
  p.nseg = 1;
  p.shadow = ctx->at<__nv_bfloat16>(L.Wb); p.shadow_ld = L.colsb;
  p.copy_counters = &ctx->at<Scalars>(L.scalars)->copy_pieces;
  if ((c.cols + 1023) / 1024 > 65535) return SFB_ERR_SHAPE;
  dim3 lgrid(static_cast<unsigned>(ctx->K), static_cast<unsigned>((c.cols + 1023) / 1024));
  // With a fused prox the fp32 label-row term has to be in W before the pass that applies the operator, so it goes
  // first (both terms are sums into W).  Either way the label-row kernel rewrites the bf16 copy of its rows, so the
  // copy equals bf16(W) whenever the main pass starts.
  const bool labels_first = ctx->prox_kind != 0;
  for (int pass = 0; pass < 2; ++pass) {
    if ((pass == 0) == labels_first) {
      label_rows_kernel<<<lgrid, 256, 0, ctx->stream>>>(
          ctx->W, c.rows, c.cols, ctx->at<float>(L.Xf), ctx->at<int32_t>(L.labels), ctx->at<float>(L.coef),
          static_cast<int>(ctx->K), ctx->step, ctx->at<__nv_bfloat16>(L.Wb), L.colsb);   // keeps the copy = bf16(W)
    } else if (ctx->sparse_v) {
      const int rc = sparse_update(ctx);                                                // the same sum over the non-zeros of V
      if (rc) return rc;
      continue;
    } else {
      update_pair_kernel<1><<<grid, kThreads, kSmem, ctx->stream>>>(ma, mb, mc, p);     // W += -eta * P^T V
    }
    count_launch();
    CKC(cudaGetLastError());
  }
  return SFB_OK;
}

}  // namespace sfb
