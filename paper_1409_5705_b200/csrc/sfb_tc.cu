// Tensor-core (bf16 operand) path of the SFB step on sm_100a: sufficient-factor computation for multiclass
// logistic regression (Sections 1 and 2: u = softmax(W x) - onehot(y), v = x) and the operand packing of the
// update product.  The update product itself is in sfb_update.cu.
//
// Forward product: one persistent, warp-specialised kernel computes  Z (K x rows) = X (K x cols) * W^T  with bf16
// operands staged by TMA into 128-byte-swizzled shared memory, tcgen05.mma accumulating in TMEM (two 128 x 256
// fp32 accumulators, so the epilogue of one tile overlaps the main loop of the next).  The epilogue stores Z as
// fp32 and, per (sample, 256-row block), the softmax partials (max, sum of exp).
// Roles: warp 0 TMA producer, warp 1 MMA issuer (and TMEM owner), warps 2-5 epilogue (one TMEM lane quarter each).
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdint>
#include <new>

#include "sfb_ptx.cuh"
#include "sfb_tc.h"

#ifndef SFB_SPLIT_PREFETCH
#define SFB_SPLIT_PREFETCH 4
#endif

namespace sfb {
namespace {

using namespace ptx;

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int kBytesA = BM * BK * 2, kBytesB = BN * BK * 2;
constexpr int kChunk = 32;                 // accumulator columns handled per epilogue step
constexpr int kSlotBytes = 32 * kChunk * 4;  // one warp's 32 rows x 32 fp32 columns
constexpr int kTmemCols = 512;
constexpr int S = 4;                      // operand pipeline stages
constexpr int R = 2;                      // epilogue ring slots per warp
constexpr int kEpiWarps = 4;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kBars = 2 * S + 4;
constexpr int kSmem = S * (kBytesA + kBytesB) + kEpiWarps * R * kSlotBytes + kBars * 8 + 16 + 1024;

// Epilogues of the product  D (samples x N) = A * B^T:
//   F_SOFTMAX  store D as fp32 logits and the per (sample, 256-column block) softmax partials      (MLR; forward_kernel)
// and, in forward_split_kernel:
//   F_STORE    store D as fp32                                                                     (DML: z = W v)
//   F_SUB      store D - aux as fp32 and as a (hi | lo) bf16 pair                                  (SC: r = W a - x)
//   F_ISTA     C <- soft(C - D / L, lambda / L) in place, also as a (hi | lo) bf16 pair            (SC: ISTA step)
enum FwdEpi { F_SOFTMAX = 0, F_STORE = 1, F_SUB = 2, F_ISTA = 3 };

struct TcParams {
  int32_t M, N, Kc;            // extents of the product: samples, output columns, contraction
  int32_t m_off;               // first sample handled by this launch (per-worker slices)
  int32_t tilesM, tilesN;
  int32_t bn;                  // columns per tile, at most BN (chosen so that the tiles fill the SMs): a multiple of 32
                               // in forward_kernel, of 16 in forward_split_kernel
  // The contraction runs over nseg segments of kseg k-blocks; segment s reads A from column a_off<s> and B from
  // column b_off<s> of their tensors: one segment is the plain product, three segments over [hi | lo] operand
  // halves form the split-bf16 product hi*hi + hi*lo + lo*hi.  (Scalars: an indexed array would send the whole
  // parameter block to local memory.)
  int32_t nseg, kseg;
  int32_t a_off0, a_off1, a_off2, b_off0, b_off1, b_off2;
  float2* part;                // F_SOFTMAX: [tilesN][part_ld] (max, sum exp) per sample and 256-row block
  int64_t part_ld;
  const float* aux;            // F_SUB: the matrix subtracted, [M x ldaux]; F_ISTA: the matrix updated, [M x ldaux]
  int64_t ldaux;
  int32_t prefetch;            // k-blocks by which the producer asks L2 for the B operand ahead of its loads (0: off)
  int32_t ksplit;              // forward_split_kernel, F_STORE: the contraction is cut into this many parts, each a work
  int64_t c_split_stride;      //   unit of its own writing its partial product to C + part * c_split_stride (else 1, 0)
  const Scalars* sc;           // F_ISTA: 1 / L
  float lam;                   // F_ISTA: lambda
  __nv_bfloat16* split;        // F_SUB, F_ISTA: [M x ld_split] receives hi at column n and lo at column split_half + n
  int64_t ld_split;
  int32_t split_half;          // padded N (a multiple of 64); columns N..split_half-1 are written as zeros
  uint32_t* status;
};

// Tiles are numbered with the sample block fastest: consecutive tiles (which run on different SMs at the same
// time) share one block of W, which therefore stays hot in L2 while all K samples are swept past it.
__device__ __forceinline__ void tile_coords(const TcParams& p, int tile, int& m0, int& n0) {
  const int tm = tile % p.tilesM, tn = tile / p.tilesM;
  m0 = p.m_off + tm * BM;
  n0 = tn * p.bn;
}

__device__ __forceinline__ float soft_threshold(float w, float t) {
  const float a = fabsf(w) - t;
  return a > 0.f ? copysignf(a, w) : 0.f;
}

// TF32: the operands are 32-bit words read as tf32 (a k-block of 128 bytes is then 32 elements and one MMA contracts
// 8 of them); everything else -- stages, descriptors, epilogues -- is the same.
template <int EPI, bool TF32 = false>
__global__ void __launch_bounds__(kThreads, 1)
forward_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmC, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = smem + S * kBytesA;
  uint8_t* sRing = smem + S * (kBytesA + kBytesB);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sRing + 4 * R * kSlotBytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + S;
  uint64_t* tfull = bars + 2 * S;
  uint64_t* tempty = bars + 2 * S + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kBars);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ntiles = p.tilesM * p.tilesN;
  const int numK = p.nseg * p.kseg;

  if (threadIdx.x == 0) {
    for (int i = 0; i < S; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], 4); }
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmA); prefetch_tmap(&tmB); prefetch_tmap(&tmC);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      // A (the K samples) is the small operand every tile re-reads: pinned in L2.
      const uint64_t pol_keep = policy_evict_last();
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
        int m0, n0;
        tile_coords(p, tile, m0, n0);
        for (int seg = 0; seg < p.nseg && ok; ++seg) {
          const int xa0 = seg == 0 ? p.a_off0 : seg == 1 ? p.a_off1 : p.a_off2;
          const int xb0 = seg == 0 ? p.b_off0 : seg == 1 ? p.b_off1 : p.b_off2;
          for (int kl = 0; kl < p.kseg; ++kl, ++it) {
            const uint32_t s = it % S, ph = (it / S) & 1;
            if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; break; }
            // B streams from HBM when it is larger than L2: with the box asked for a few k-blocks early, the load
            // that fills the stage finds it in L2 and the four stages cover the latency
            if (p.prefetch > 0 && kl + p.prefetch < p.kseg)
              tma_prefetch_2d(&tmB, xb0 + (kl + p.prefetch) * (TF32 ? BK / 2 : BK), n0);
            mbar_expect_tx(&full[s], kBytesA + p.bn * BK * 2);
            tma_load_2d_hint(sA + s * kBytesA, &tmA, xa0 + kl * (TF32 ? BK / 2 : BK), m0, &full[s], pol_keep);
            tma_load_2d(sB + s * kBytesB, &tmB, xb0 + kl * (TF32 ? BK / 2 : BK), n0, &full[s]);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = TF32 ? umma_idesc_tf32(BM, p.bn) : umma_idesc_bf16(BM, p.bn);
      uint32_t it = 0, tl = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++tl) {
        const uint32_t a = tl & 1, aph = (tl >> 1) & 1;
        if (!mbar_wait(&tempty[a], aph ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * BN;
        for (int kb = 0; kb < numK; ++kb, ++it) {
          const uint32_t s = it % S, ph = (it / S) & 1;
          if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = umma_desc_k128(smem_u32(sA + s * kBytesA));
          const uint64_t db = umma_desc_k128(smem_u32(sB + s * kBytesB));
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {          // four MMAs of 32 bytes of contraction each, either kind
            const uint64_t adv = static_cast<uint64_t>(k * UMMA_K * 2 / 16);
            if (TF32) umma_tf32(d_tmem, da + adv, db + adv, idesc, (kb | k) != 0 ? 1u : 0u);
            else umma_bf16(d_tmem, da + adv, db + adv, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&empty[s]);          // the stage is free once these MMAs have read it
        }
        if (ok) umma_commit(&tfull[a]);    // the accumulator is complete once every MMA of the tile is
      }
    }
  } else {
    // ---------------- epilogue: warps 2..5, TMEM lane quarter q ----------------
    const int q = warp & 3;
    uint8_t* ring = sRing + q * R * kSlotBytes;
    const int my_tiles = blockIdx.x < ntiles ? (ntiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;
    bool ok = true;

    {
      // The fp32 result goes out through the ring by TMA; F_SOFTMAX keeps a running (max, sum exp) per sample.
      uint32_t gs = 0;                       // stores issued so far: consecutive stores alternate ring slots
      for (int tl = 0; tl < my_tiles && ok; ++tl) {
        int m0, n0;
        tile_coords(p, blockIdx.x + tl * gridDim.x, m0, n0);
        const uint32_t a = tl & 1, aph = (tl >> 1) & 1;
        if (!__all_sync(0xffffffffu, mbar_wait(&tfull[a], aph, abort_flag))) { ok = false; break; }
        tc_fence_after();
        const int row = m0 + q * 32 + lane;
        float mx = -INFINITY, sum = 0.f;
        for (int c = 0; c < p.bn / kChunk; ++c) {
          uint8_t* sl = ring + (gs % R) * kSlotBytes;
          uint32_t acc[32];
          tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + a * BN + c * kChunk, acc);
          tmem_ld_wait();
          const int col0 = n0 + c * kChunk;
          if (col0 < p.N) {
            if constexpr (EPI == F_SOFTMAX) {
              float cm = -INFINITY;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) cm = fmaxf(cm, __uint_as_float(acc[j]));
              const float nm = fmaxf(mx, cm);
              float cs = 0.f;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) cs += __expf(__uint_as_float(acc[j]) - nm);
              sum = sum * __expf(mx - nm) + cs;
              mx = nm;
            }
            if (lane == 0) tma_wait_group_read<R - 1>();   // the store that last used this slot has read it
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              *reinterpret_cast<uint4*>(sl + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                  make_uint4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&tmC, sl, col0, m0 + q * 32);
              tma_commit_group();
            }
            ++gs;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty[a]);
        if (EPI == F_SOFTMAX && row < p.M) p.part[static_cast<int64_t>(n0 / p.bn) * p.part_ld + row] = make_float2(mx, sum);
      }
      if (lane == 0) tma_wait_group<0>();
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // A wait ran out: report it, give copies in flight a bounded time to land, then release TMEM.
    if (threadIdx.x == 0) atomicOr(p.status, SFB_STATUS_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, kTmemCols); }
}

// ---------------------------------------------------------------------------------------------------------
// Split-bf16 products of distance metric learning and sparse coding:  D (samples x N) = A * B^T  with both operands
// stored as [hi | lo] bf16 halves,  A_hi B_hi + A_lo B_hi + A_hi B_lo  (fp32-class accuracy; A_lo B_lo, 2^-16 of the
// product, is dropped).  One pipeline stage holds the k-block of all four halves, and the three products of that
// k-block are issued from it: 72 KB of operands per three k-blocks of tensor work instead of 108 KB when the three
// products run as separate passes over the contraction (these products are bound by their operand loads: a 128 x 160
// tile takes 36 KB per 320 cycles of MMA).  Three stages of 72 KB fill the shared memory, so the epilogue writes its
// results straight from registers (the outputs are small: samples x N).
// Roles as in forward_kernel: warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2-5 epilogue.
// ---------------------------------------------------------------------------------------------------------
constexpr int FS_BN = 160;                          // widest tile of this kernel (columns of the accumulator)
constexpr int FS_STAGES = 3;
constexpr int kFsBytesB = FS_BN * BK * 2;           // 20 KB
constexpr int kFsStage = 2 * kBytesA + 2 * kFsBytesB;
constexpr int kFsBars = 2 * FS_STAGES + 4;
constexpr int kFsSmem = FS_STAGES * kFsStage + kFsBars * 8 + 16 + 1024;

template <int EPI>
__global__ void __launch_bounds__(kThreads, 1)
forward_split_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, float* __restrict__ C,
                     int64_t ldc, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + FS_STAGES * kFsStage);
  uint64_t* full = bars;
  uint64_t* empty = bars + FS_STAGES;
  uint64_t* tfull = bars + 2 * FS_STAGES;
  uint64_t* tempty = bars + 2 * FS_STAGES + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kFsBars);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = p.ksplit > 1 ? p.ksplit : 1;
  const int ntiles = p.tilesM * p.tilesN * S;       // work units: (tile, part of the contraction), parts of a tile adjacent
  const int numKall = p.kseg;                       // k-blocks of the contraction (each serves three products)
  const int a_hi = p.a_off0, a_lo = p.a_off2, b_hi = p.b_off0, b_lo = p.b_off1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < FS_STAGES; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], 4); }
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmA); prefetch_tmap(&tmB);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer: the four operand halves of a k-block per stage ----------------
    if (lane == 0) {
      const uint64_t pol_keep = policy_evict_last();
      const uint32_t stage_bytes = 2 * kBytesA + 2 * static_cast<uint32_t>(p.bn) * BK * 2;
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
        int m0, n0;
        tile_coords(p, tile / S, m0, n0);
        const int part = tile % S, kbeg = part * numKall / S, numK = (part + 1) * numKall / S;
        for (int kl = kbeg; kl < numK; ++kl, ++it) {
          const uint32_t s = it % FS_STAGES, ph = (it / FS_STAGES) & 1;
          if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; break; }
          if (p.prefetch > 0 && kl + p.prefetch < numK) {          // B streams from HBM when it is larger than L2
            tma_prefetch_2d(&tmB, b_hi + (kl + p.prefetch) * BK, n0);
            tma_prefetch_2d(&tmB, b_lo + (kl + p.prefetch) * BK, n0);
          }
          uint8_t* st = smem + s * kFsStage;
          mbar_expect_tx(&full[s], stage_bytes);
          tma_load_2d_hint(st, &tmA, a_hi + kl * BK, m0, &full[s], pol_keep);
          tma_load_2d_hint(st + kBytesA, &tmA, a_lo + kl * BK, m0, &full[s], pol_keep);
          tma_load_2d(st + 2 * kBytesA, &tmB, b_hi + kl * BK, n0, &full[s]);
          tma_load_2d(st + 2 * kBytesA + kFsBytesB, &tmB, b_lo + kl * BK, n0, &full[s]);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: three products per stage ----------------
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(BM, p.bn);
      uint32_t it = 0, tl = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++tl) {
        const uint32_t a = tl & 1, aph = (tl >> 1) & 1;
        if (!mbar_wait(&tempty[a], aph ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * BN;
        const int part = tile % S, numK = (part + 1) * numKall / S - part * numKall / S;
        for (int kb = 0; kb < numK; ++kb, ++it) {
          const uint32_t s = it % FS_STAGES, ph = (it / FS_STAGES) & 1;
          if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          uint8_t* st = smem + s * kFsStage;
          const uint64_t dah = umma_desc_k128(smem_u32(st));
          const uint64_t dal = umma_desc_k128(smem_u32(st + kBytesA));
          const uint64_t dbh = umma_desc_k128(smem_u32(st + 2 * kBytesA));
          const uint64_t dbl = umma_desc_k128(smem_u32(st + 2 * kBytesA + kFsBytesB));
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t adv = static_cast<uint64_t>(k * UMMA_K * 2 / 16);
            umma_bf16(d_tmem, dal + adv, dbh + adv, idesc, (kb | k) != 0 ? 1u : 0u);     // A_lo B_hi
            umma_bf16(d_tmem, dah + adv, dbl + adv, idesc, 1u);                          // A_hi B_lo
            umma_bf16(d_tmem, dah + adv, dbh + adv, idesc, 1u);                          // A_hi B_hi
          }
          umma_commit(&empty[s]);
        }
        if (ok) umma_commit(&tfull[a]);
      }
    }
  } else {
    // ---------------- epilogue: warps 2..5, TMEM lane quarter q; results leave straight from registers ----------------
    const int q = warp & 3;
    const int my_tiles = blockIdx.x < ntiles ? (ntiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;
    bool ok = true;
    float invL = 0.f, thr = 0.f;
    if (EPI == F_ISTA) { invL = p.sc->invL; thr = p.lam * invL; }
    for (int tl = 0; tl < my_tiles && ok; ++tl) {
      int m0, n0;
      const int unit = blockIdx.x + tl * gridDim.x;
      tile_coords(p, unit / S, m0, n0);
      float* Cp = C + static_cast<int64_t>(unit % S) * p.c_split_stride;
      const uint32_t a = tl & 1, aph = (tl >> 1) & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&tfull[a], aph, abort_flag))) { ok = false; break; }
      tc_fence_after();
      const int row = m0 + q * 32 + lane;
      // the tile's columns end at nlim; its width is a multiple of 16, so the last 32-column chunk may be half used
      const int nlim = min(p.N, n0 + p.bn);
      for (int c = 0; c < (p.bn + kChunk - 1) / kChunk; ++c) {
        uint32_t acc[32];
        tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + a * BN + c * kChunk, acc);
        tmem_ld_wait();
        const int col0 = n0 + c * kChunk;
        if (col0 >= nlim || row >= p.M) continue;
        if constexpr (EPI == F_SUB || EPI == F_ISTA) {
          // the sample's values of aux (x, or the current code a) are contiguous: up to 128 bytes per lane
          float xv[32];
          const float* ap = p.aux + static_cast<int64_t>(row) * p.ldaux + col0;
          const bool ap16 = (reinterpret_cast<uintptr_t>(ap) & 15u) == 0;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (ap16 && col0 + 4 * j + 4 <= nlim) {
              const float4 v4 = *reinterpret_cast<const float4*>(ap + 4 * j);
              xv[4 * j] = v4.x; xv[4 * j + 1] = v4.y; xv[4 * j + 2] = v4.z; xv[4 * j + 3] = v4.w;
            } else {
#pragma unroll
              for (int e = 0; e < 4; ++e) xv[4 * j + e] = col0 + 4 * j + e < nlim ? ap[4 * j + e] : 0.f;
            }
          }
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float d = __uint_as_float(acc[j]);
            const float v = EPI == F_SUB ? d - xv[j] : soft_threshold(fmaf(-d, invL, xv[j]), thr);
            acc[j] = __float_as_uint(col0 + j < p.N ? v : 0.f);
          }
          // (hi | lo) bf16 pair of the result: the operand of the next product (zero in the padding past N; the
          // columns past this tile's width belong to the next tile)
          __nv_bfloat16* hp = p.split + static_cast<int64_t>(row) * p.ld_split + col0;
          const int split_lim = min(p.split_half, n0 + p.bn);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (col0 + 8 * j < split_lim) {
              uint32_t hi[4], lo[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float f0 = __uint_as_float(acc[8 * j + 2 * e]), f1 = __uint_as_float(acc[8 * j + 2 * e + 1]);
                const __nv_bfloat16 h0 = __float2bfloat16_rn(f0), h1 = __float2bfloat16_rn(f1);
                hi[e] = static_cast<uint32_t>(__bfloat16_as_ushort(h0)) |
                        (static_cast<uint32_t>(__bfloat16_as_ushort(h1)) << 16);
                const __nv_bfloat162 l2 = __floats2bfloat162_rn(f0 - __bfloat162float(h0), f1 - __bfloat162float(h1));
                lo[e] = *reinterpret_cast<const uint32_t*>(&l2);
              }
              *reinterpret_cast<uint4*>(hp + 8 * j) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
              *reinterpret_cast<uint4*>(hp + p.split_half + 8 * j) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
          }
        }
        // the fp32 result: this lane's consecutive columns of its row
        float* cp = Cp + static_cast<int64_t>(row) * ldc + col0;
        const bool cp16 = (reinterpret_cast<uintptr_t>(cp) & 15u) == 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (cp16 && col0 + 4 * j + 4 <= nlim) {
            *reinterpret_cast<uint4*>(cp + 4 * j) = make_uint4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
          } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if (col0 + 4 * j + e < nlim) cp[4 * j + e] = __uint_as_float(acc[4 * j + e]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty[a]);
    }
  }

  // ---------------- teardown ----------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, SFB_STATUS_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, kTmemCols); }
}

// ---------------------------------------------------------------------------------------------------------
// Bandwidth-bound companions of the tensor-core products
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// fp32 [rows x cols] -> bf16 [rows x ld] (row-major), 8 elements per thread; cols is a multiple of 4.
__global__ void __launch_bounds__(256) convert_rows_kernel(const float* __restrict__ src, int64_t rows, int64_t cols,
                                                           __nv_bfloat16* __restrict__ dst, int64_t ld) {
  const int64_t quads = cols / 4;
  const int64_t total = rows * quads;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total; i += stride) {
    const int64_t r = i / quads, qd = i % quads;
    const float4 v = *reinterpret_cast<const float4*>(src + r * cols + qd * 4);
    *reinterpret_cast<uint2*>(dst + r * ld + qd * 4) = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
  }
}

// Pack of the inputs of n samples starting at pair index off (Section 2.1: v = a_i):
//   Xb[off + i][:]  = bf16(x_i)          forward operand, sample-major
//   VT[:][off + i]  = bf16(x_i)          update operand, feature-major (V^T)
// 64 x 64 tiles through shared memory so that both sides are written in 16-byte pieces.
__global__ void __launch_bounds__(256) pack_mlr_kernel(const float* __restrict__ X, int64_t n, int64_t cols,
                                                       __nv_bfloat16* __restrict__ Xb, int64_t ldx,
                                                       __nv_bfloat16* __restrict__ VT, int64_t ldv, int64_t off,
                                                       float* __restrict__ Xf, const int32_t* __restrict__ labels,
                                                       int32_t* __restrict__ labels_out) {
  __shared__ float tile[64][65];
  const int64_t i0 = static_cast<int64_t>(blockIdx.y) * 64, c0 = static_cast<int64_t>(blockIdx.x) * 64;
  const int t = threadIdx.x;
#pragma unroll
  for (int v = 0; v < 4; ++v) {
    const int idx = t + v * 256;            // 64 samples x 16 quads
    const int i = idx / 16, cq = (idx % 16) * 4;
    float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i0 + i < n && c0 + cq < cols) val = *reinterpret_cast<const float4*>(X + (i0 + i) * cols + c0 + cq);
    tile[i][cq + 0] = val.x; tile[i][cq + 1] = val.y; tile[i][cq + 2] = val.z; tile[i][cq + 3] = val.w;
    if (i0 + i < n && c0 + cq < cols) {
      *reinterpret_cast<uint2*>(Xb + (off + i0 + i) * ldx + c0 + cq) =
          make_uint2(pack_bf16(val.x, val.y), pack_bf16(val.z, val.w));
      *reinterpret_cast<float4*>(Xf + (off + i0 + i) * cols + c0 + cq) = val;
    }
  }
  if (blockIdx.x == 0 && t < 64 && i0 + t < n) labels_out[off + i0 + t] = labels[i0 + t];
  __syncthreads();
#pragma unroll
  for (int v = 0; v < 2; ++v) {
    const int idx = t + v * 256;            // 64 features x 8 groups of 8 samples
    const int c = idx / 8, ig = (idx % 8) * 8;
    if (c0 + c >= cols) continue;
    __nv_bfloat16* dst = VT + (c0 + c) * ldv + off + i0 + ig;
    if (i0 + ig + 7 < n && ((off + i0 + ig) & 7) == 0) {
      *reinterpret_cast<uint4*>(dst) =
          make_uint4(pack_bf16(tile[ig][c], tile[ig + 1][c]), pack_bf16(tile[ig + 2][c], tile[ig + 3][c]),
                     pack_bf16(tile[ig + 4][c], tile[ig + 5][c]), pack_bf16(tile[ig + 6][c], tile[ig + 7][c]));
    } else {
      for (int k = 0; k < 8; ++k)
        if (i0 + ig + k < n) dst[k] = __float2bfloat16_rn(tile[ig + k][c]);
    }
  }
}

// Gathered fp32 factors F [n x dim] (pair-major) -> the split-bf16 operand of the update product,
// FT [dim x 2*Kp] (samples contiguous): FT[c][i] = hi(F[i][c]), FT[c][Kp + i] = lo(F[i][c]) with
// hi = bf16(f), lo = bf16(f - hi); samples n..Kp-1 are written as zeros.  64 x 64 tiles through shared memory.
__global__ void __launch_bounds__(256) pack_split_t_kernel(const float* __restrict__ F, int64_t n, int64_t dim,
                                                           int64_t ld, __nv_bfloat16* __restrict__ FT, int64_t Kp) {
  __shared__ float tile[64][65];
  const int64_t i0 = static_cast<int64_t>(blockIdx.y) * 64, c0 = static_cast<int64_t>(blockIdx.x) * 64;
  const int t = threadIdx.x;
  const bool vec = (ld % 4) == 0;
#pragma unroll
  for (int v = 0; v < 4; ++v) {
    const int idx = t + v * 256;            // 64 samples x 16 quads
    const int i = idx / 16, cq = (idx % 16) * 4;
    float f[4] = {0.f, 0.f, 0.f, 0.f};
    if (i0 + i < n) {
      const float* src = F + (i0 + i) * ld + c0 + cq;
      if (vec && c0 + cq + 3 < dim) {
        const float4 q4 = *reinterpret_cast<const float4*>(src);
        f[0] = q4.x; f[1] = q4.y; f[2] = q4.z; f[3] = q4.w;
      } else {
        for (int k = 0; k < 4; ++k)
          if (c0 + cq + k < dim) f[k] = src[k];
      }
    }
    tile[i][cq + 0] = f[0]; tile[i][cq + 1] = f[1]; tile[i][cq + 2] = f[2]; tile[i][cq + 3] = f[3];
  }
  __syncthreads();
#pragma unroll
  for (int v = 0; v < 2; ++v) {
    const int idx = t + v * 256;            // 64 features x 8 groups of 8 samples
    const int c = idx / 8, ig = (idx % 8) * 8;
    if (c0 + c >= dim) continue;
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float f0 = tile[ig + 2 * k][c], f1 = tile[ig + 2 * k + 1][c];
      const __nv_bfloat16 h0 = __float2bfloat16_rn(f0), h1 = __float2bfloat16_rn(f1);
      hi[k] = static_cast<uint32_t>(__bfloat16_as_ushort(h0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(h1)) << 16);
      lo[k] = pack_bf16(f0 - __bfloat162float(h0), f1 - __bfloat162float(h1));
    }
    __nv_bfloat16* dst = FT + (c0 + c) * 2 * Kp + i0 + ig;     // Kp is a multiple of 64: 16-byte aligned
    *reinterpret_cast<uint4*>(dst) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<uint4*>(dst + Kp) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
}

// fp32 [n x dim] (row pitch ld) -> the (hi | lo) bf16 operand [n x 2*dimp], no transpose: dst[r][c] = hi,
// dst[r][dimp + c] = lo with hi = bf16(f), lo = bf16(f - hi).  Columns dim..dimp-1 are left as they are (zero since
// set-up).  dim and ld are multiples of 4.
__global__ void __launch_bounds__(256) pack_split_rows_kernel(const float* __restrict__ F, int64_t n, int64_t dim,
                                                              int64_t ld, __nv_bfloat16* __restrict__ dst, int64_t dimp) {
  const int64_t quads = dim / 4, total = n * quads;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total; i += stride) {
    const int64_t r = i / quads, qd = i % quads;
    const float4 v = *reinterpret_cast<const float4*>(F + r * ld + qd * 4);
    const __nv_bfloat16 h0 = __float2bfloat16_rn(v.x), h1 = __float2bfloat16_rn(v.y), h2 = __float2bfloat16_rn(v.z),
                        h3 = __float2bfloat16_rn(v.w);
    __nv_bfloat16* d = dst + r * 2 * dimp + qd * 4;
    *reinterpret_cast<uint2*>(d) =
        make_uint2(static_cast<uint32_t>(__bfloat16_as_ushort(h0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(h1)) << 16),
                   static_cast<uint32_t>(__bfloat16_as_ushort(h2)) | (static_cast<uint32_t>(__bfloat16_as_ushort(h3)) << 16));
    *reinterpret_cast<uint2*>(d + dimp) = make_uint2(pack_bf16(v.x - __bfloat162float(h0), v.y - __bfloat162float(h1)),
                                                     pack_bf16(v.z - __bfloat162float(h2), v.w - __bfloat162float(h3)));
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// One warp per sample: merge the per-block (max, sum exp) partials into log sum exp; loss = lse - z_y;
// coef = 1 - p_y, the size of the label entry of u, kept in fp32 for label_rows_kernel.
__global__ void __launch_bounds__(256) mlr_lse_kernel(const float2* __restrict__ part, int64_t part_ld, int nblocks,
                                                      const float* __restrict__ Z, int64_t ldz, int64_t rows,
                                                      const int32_t* __restrict__ labels, int64_t off, int64_t n,
                                                      float* __restrict__ lse, float* __restrict__ loss,
                                                      float* __restrict__ coef, uint32_t* status) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (i >= n) return;
  const int lane = threadIdx.x & 31;
  const int64_t s = off + i;
  float m = -INFINITY;
  for (int b = lane; b < nblocks; b += 32) m = fmaxf(m, part[static_cast<int64_t>(b) * part_ld + s].x);
  m = warp_max(m);
  float sum = 0.f;
  for (int b = lane; b < nblocks; b += 32) {
    const float2 v = part[static_cast<int64_t>(b) * part_ld + s];
    sum += v.y * __expf(v.x - m);
  }
  sum = warp_sum(sum);
  if (lane == 0) {
    const float l = m + logf(sum);
    lse[s] = l;
    const int32_t y = labels[i];
    const bool okl = y >= 0 && y < rows;
    if (!okl) atomicOr(status, SFB_STATUS_LABEL_RANGE);
    const float zy = okl ? Z[s * ldz + y] : 0.f;
    loss[s] = okl ? l - zy : 0.f;
    coef[s] = okl ? -expm1f(zy - l) : 0.f;        // 1 - p_y = -u_y, formed in fp32 without cancellation
  }
}

// Row-sharded form, first half: one warp per sample merges the forward's per-block (max, sum exp) partials over the
// shard's rows into the shard's partial (m_i, s_i, zy_i, has_i); zy_i = z_{i,y_i} and has_i = 1 when the shard owns
// class y_i (labels are global ids; the shard holds rows [row_off, row_off + rows)).
__global__ void __launch_bounds__(256) mlr_shard_partials_tc_kernel(const float2* __restrict__ part, int64_t part_ld, int nblocks,
                                                                    const float* __restrict__ Z, int64_t ldz, int64_t rows,
                                                                    const int32_t* __restrict__ labels, int64_t row_off,
                                                                    int64_t n, float4* __restrict__ out) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (i >= n) return;
  const int lane = threadIdx.x & 31;
  float m = -INFINITY;
  for (int b = lane; b < nblocks; b += 32) m = fmaxf(m, part[static_cast<int64_t>(b) * part_ld + i].x);
  m = warp_max(m);
  float sum = 0.f;
  for (int b = lane; b < nblocks; b += 32) {
    const float2 v = part[static_cast<int64_t>(b) * part_ld + i];
    sum += v.y * __expf(v.x - m);
  }
  sum = warp_sum(sum);
  if (lane == 0) {
    const int64_t yl = static_cast<int64_t>(labels[i]) - row_off;
    const bool mine = yl >= 0 && yl < rows;
    out[i] = make_float4(m, sum, mine ? Z[i * ldz + yl] : 0.f, mine ? 1.f : 0.f);
  }
}

// Second half, one thread per sample: merge the partials of all shards ([shards][n], shard order) into the global
// log-partition; loss = lse - z_y; coef = 1 - p_y for the samples whose class this shard owns (0 otherwise); the class
// ids are rewritten as row indices of this shard (-1: another shard's row).  A class no shard owns sets the status bit.
__global__ void __launch_bounds__(256) mlr_shard_finish_tc_kernel(const float4* __restrict__ parts, int shards, int64_t n,
                                                                  int64_t rows, int64_t row_off, int32_t* __restrict__ labels,
                                                                  float* __restrict__ lse, float* __restrict__ loss,
                                                                  float* __restrict__ coef, uint32_t* status) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (i >= n) return;
  float M = -INFINITY;
  for (int g = 0; g < shards; ++g) M = fmaxf(M, parts[static_cast<int64_t>(g) * n + i].x);
  float S = 0.f, zy = 0.f, has = 0.f;
  for (int g = 0; g < shards; ++g) {
    const float4 v = parts[static_cast<int64_t>(g) * n + i];
    S += v.y * expf(v.x - M);
    zy += v.z;
    has += v.w;
  }
  const float l = M + logf(S);
  const bool ok = has > 0.5f;
  if (!ok) atomicOr(status, SFB_STATUS_LABEL_RANGE);
  const int64_t yl = static_cast<int64_t>(labels[i]) - row_off;
  const bool mine = ok && yl >= 0 && yl < rows;
  lse[i] = l;
  loss[i] = ok ? l - zy : 0.f;
  coef[i] = mine ? -expm1f(zy - l) : 0.f;
  labels[i] = mine ? static_cast<int32_t>(yl) : -1;
}

// P^T[r][off + i] = bf16( exp(z_ir - lse_i) ) for r != y_i and 0 for r = y_i: 64 samples x 64 rows per block,
// transposed through shared memory (Z is sample-major, the update operand is row-major with samples
// contiguous).  The factor is u_i = p_i - onehot(y_i); its label entry u_iy = p_iy - 1 is left out of the bf16
// operand and applied to W in fp32 by label_rows_kernel, because bf16 cannot hold it when p_iy is close to 1
// (spacing 2^-8 next to 1) and a rounded p_iy with an exact -1 would not cancel.
// PLAIN: the values of Z themselves instead of exp(z - lse) (the dual changes of the SDCA step), same layout and
// the same zero at the label entry.
template <bool PLAIN>
__global__ void __launch_bounds__(256) mlr_emit_ut_kernel(const float* __restrict__ Z, int64_t ldz, int64_t rows,
                                                          const float* __restrict__ lse, int64_t off, int64_t n,
                                                          const int32_t* __restrict__ labels,
                                                          __nv_bfloat16* __restrict__ UT, int64_t ldu) {
  __shared__ float tile[64][65];
  const int64_t i0 = static_cast<int64_t>(blockIdx.y) * 64, r0 = static_cast<int64_t>(blockIdx.x) * 64;
  const int t = threadIdx.x;
  const bool vec = (ldz % 4) == 0;
#pragma unroll
  for (int v = 0; v < 4; ++v) {
    const int idx = t + v * 256;
    const int i = idx / 16, rq = (idx % 16) * 4;
    if (i0 + i >= n) continue;
    const int64_t s = off + i0 + i;
    const float l = PLAIN ? 0.f : lse[s];
    const int64_t yrel = static_cast<int64_t>(labels[i0 + i]) - (r0 + rq);     // label row relative to this quad
    const float* zp = Z + s * ldz + r0 + rq;
    float z[4] = {0.f, 0.f, 0.f, 0.f};
    if (vec && r0 + rq + 3 < rows) {
      const float4 q4 = *reinterpret_cast<const float4*>(zp);
      z[0] = q4.x; z[1] = q4.y; z[2] = q4.z; z[3] = q4.w;
    } else {
      for (int k = 0; k < 4; ++k)
        if (r0 + rq + k < rows) z[k] = zp[k];
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      tile[i][rq + k] = k == yrel ? 0.f : (PLAIN ? z[k] : __expf(z[k] - l));
    }
  }
  __syncthreads();
#pragma unroll
  for (int v = 0; v < 2; ++v) {
    const int idx = t + v * 256;
    const int r = idx / 8, ig = (idx % 8) * 8;
    if (r0 + r >= rows) continue;
    __nv_bfloat16* dst = UT + (r0 + r) * ldu + off + i0 + ig;
    if (i0 + ig + 7 < n && ((off + i0 + ig) & 7) == 0) {
      *reinterpret_cast<uint4*>(dst) =
          make_uint4(pack_bf16(tile[ig][r], tile[ig + 1][r]), pack_bf16(tile[ig + 2][r], tile[ig + 3][r]),
                     pack_bf16(tile[ig + 4][r], tile[ig + 5][r]), pack_bf16(tile[ig + 6][r], tile[ig + 7][r]));
    } else {
      for (int k = 0; k < 8; ++k)
        if (i0 + ig + k < n) dst[k] = __float2bfloat16_rn(tile[ig + k][r]);
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// fp32 mode on the tensor cores: every fp32 value x is carried as two tf32 words, big = tf32(x) and
// small = tf32(x - big) (x = big + small to about 2^-22 |x|), and a product runs as big*big + big*small + small*big.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_tf32(float x) {
  uint32_t u;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
  return __uint_as_float(u);
}

// fp32 [n x dim] (row pitch ld) -> [n x 2*dimp] fp32 words: dst[r][c] = big, dst[r][dimp + c] = small.  Columns
// dim..dimp-1 keep the zeros of set-up.  dim and ld are multiples of 4.
__global__ void __launch_bounds__(256) split32_rows_kernel(const float* __restrict__ F, int64_t n, int64_t dim, int64_t ld,
                                                           float* __restrict__ dst, int64_t dimp) {
  const int64_t quads = dim / 4, total = n * quads;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total; i += stride) {
    const int64_t r = i / quads, qd = i % quads;
    const float4 v = *reinterpret_cast<const float4*>(F + r * ld + qd * 4);
    const float4 b = make_float4(to_tf32(v.x), to_tf32(v.y), to_tf32(v.z), to_tf32(v.w));
    float* d = dst + r * 2 * dimp + qd * 4;
    *reinterpret_cast<float4*>(d) = b;
    *reinterpret_cast<float4*>(d + dimp) = make_float4(to_tf32(v.x - b.x), to_tf32(v.y - b.y), to_tf32(v.z - b.z),
                                                       to_tf32(v.w - b.w));
  }
}

// Gathered fp32 factors F [n x dim] (pair-major, row pitch ld) -> FT [dim x 2*Kp] (pairs contiguous):
// FT[c][i] = big, FT[c][Kp + i] = small; pairs n..Kp-1 are written as zeros.  64 x 64 tiles through shared memory.
__global__ void __launch_bounds__(256) split32_t_kernel(const float* __restrict__ F, int64_t n, int64_t dim, int64_t ld,
                                                        float* __restrict__ FT, int64_t Kp) {
  __shared__ float tile[64][65];
  const int64_t i0 = static_cast<int64_t>(blockIdx.y) * 64, c0 = static_cast<int64_t>(blockIdx.x) * 64;
  const int t = threadIdx.x;
#pragma unroll
  for (int v = 0; v < 16; ++v) {
    const int idx = t + v * 256;            // 64 pairs x 64 columns
    const int i = idx / 64, c = idx % 64;
    tile[i][c] = (i0 + i < n && c0 + c < dim) ? F[(i0 + i) * ld + c0 + c] : 0.f;
  }
  __syncthreads();
#pragma unroll
  for (int v = 0; v < 4; ++v) {
    const int idx = t + v * 256;            // 64 columns x 16 groups of 4 pairs
    const int c = idx / 16, ig = (idx % 16) * 4;
    if (c0 + c >= dim || i0 + ig >= Kp) continue;
    const float f0 = tile[ig][c], f1 = tile[ig + 1][c], f2 = tile[ig + 2][c], f3 = tile[ig + 3][c];
    const float4 b = make_float4(to_tf32(f0), to_tf32(f1), to_tf32(f2), to_tf32(f3));
    float* dst = FT + (c0 + c) * 2 * Kp + i0 + ig;          // Kp is a multiple of 32: 16-byte aligned
    *reinterpret_cast<float4*>(dst) = b;
    *reinterpret_cast<float4*>(dst + Kp) = make_float4(to_tf32(f0 - b.x), to_tf32(f1 - b.y), to_tf32(f2 - b.z), to_tf32(f3 - b.w));
  }
}

// u_ij = exp(z_ij - lse_i) - [j = y_i], from the logits Z [n x ldz] to the pair-major fp32 factors U [n x rows]
// (Section 2.1: u = d f / d (W a)).  PLAIN copies Z instead (the dual changes of the SDCA step already are the factors).
template <bool PLAIN>
__global__ void __launch_bounds__(256) mlr_finish_u_kernel(const float* __restrict__ Z, int64_t ldz, int64_t rows,
                                                           const float* __restrict__ lse, const int32_t* __restrict__ labels,
                                                           float* __restrict__ U) {
  const int64_t i = blockIdx.y;
  const float l = PLAIN ? 0.f : lse[i];
  const int64_t y = PLAIN ? -1 : static_cast<int64_t>(labels[i]);
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t j = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; j < rows; j += stride) {
    const float z = Z[i * ldz + j];
    U[i * rows + j] = PLAIN ? z : expf(z - l) - (j == y ? 1.f : 0.f);
  }
}

// ---------------------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------------------
template <int EPI, bool TF32 = false>
cudaError_t launch_forward(sfb_ctx* ctx, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c, TcParams p) {
  const TcState* st = static_cast<const TcState*>(ctx->tc);
  const int64_t tiles = static_cast<int64_t>(p.tilesM) * p.tilesN;
  if (tiles <= 0) return cudaSuccess;
  const int grid = static_cast<int>(tiles < st->sms ? tiles : st->sms);
  forward_kernel<EPI, TF32><<<grid, kThreads, kSmem, ctx->stream>>>(a, b, c, p);
  count_launch();
  return cudaGetLastError();
}

template <int EPI>
cudaError_t launch_forward_split(sfb_ctx* ctx, const CUtensorMap& a, const CUtensorMap& b, float* C, int64_t ldc, TcParams p) {
  const TcState* st = static_cast<const TcState*>(ctx->tc);
  const int64_t tiles = static_cast<int64_t>(p.tilesM) * p.tilesN * (p.ksplit > 1 ? p.ksplit : 1);
  if (tiles <= 0) return cudaSuccess;
  const int grid = static_cast<int>(tiles < st->sms ? tiles : st->sms);
  forward_split_kernel<EPI><<<grid, kThreads, kFsSmem, ctx->stream>>>(a, b, C, ldc, p);
  count_launch();
  return cudaGetLastError();
}

// The shared-memory opt-in is a per-device attribute of each kernel: set for every instantiation when a context is
// created (with its device current), not once per process.
cudaError_t prepare_forward_kernels() {
  cudaError_t e = cudaFuncSetAttribute(forward_kernel<F_SOFTMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(forward_split_kernel<F_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFsSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(forward_split_kernel<F_SUB>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFsSmem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(forward_split_kernel<F_ISTA>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFsSmem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(forward_kernel<F_SOFTMAX, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
  return e;
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

// fp32 mode on the tensor cores (MLR): fp32 pair-major factors as in the FFMA path, plus the (big | small) tf32
// operands of the two products and the logits.
void tc32_extend_layout(const sfb_config& c, Layout& L, size_t& off) {
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + kAlign - 1) / kAlign * kAlign; return o; };
  const size_t K = static_cast<size_t>(c.workers) * c.batch;
  L.Kp = round_up(static_cast<int64_t>(K), 32);
  L.colsp = round_up(c.cols, 32);
  const size_t ldz = static_cast<size_t>(round_up(c.rows, 32));
  const size_t nblk = static_cast<size_t>((c.rows + BN - 1) / BN);
  L.V = take(K * static_cast<size_t>(c.cols) * 4);
  L.U = take(K * static_cast<size_t>(c.rows) * 4);
  L.Ws = take(static_cast<size_t>(c.rows) * 2 * L.colsp * 4);        // W, rows x (big | small)
  L.As = take(K * 2 * static_cast<size_t>(L.colsp) * 4);             // the samples, K x (big | small)
  L.VT = take(static_cast<size_t>(c.cols) * 2 * L.Kp * 4);
  L.UT = take(static_cast<size_t>(c.rows) * 2 * L.Kp * 4);
  L.ZT = take(K * ldz * 4);
  L.part = take(nblk * K * 8);
  L.lse = take(K * 4);
  L.coef = take(K * 4);
  L.labels = take(K * 4);
}

void tc_extend_layout(const sfb_config& c, Layout& L, size_t& off) {
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + kAlign - 1) / kAlign * kAlign; return o; };
  const size_t K = static_cast<size_t>(c.workers) * c.batch;
  L.Kp = round_up(static_cast<int64_t>(K), 64);
  L.colsb = round_up(c.cols, 64);
  if (c.model != SFB_MLR) {
    // fp32 factors as the workers write them, their split-bf16 transposes for the update product, and the
    // split-bf16 operands of the forward products
    L.colsp = round_up(c.cols, 64);
    L.rowsp = round_up(c.rows, 64);
    L.ldu = round_up(c.rows, 4);                                        // TMA stores need a 16-byte row pitch
    L.V = take(K * static_cast<size_t>(c.cols) * 4);
    L.U = take(K * static_cast<size_t>(L.ldu) * 4);
    L.U2 = take(c.model == SFB_DML ? K * static_cast<size_t>(L.ldu) * 4 : 0);
    L.UT = take(static_cast<size_t>(c.rows) * 2 * L.Kp * 2);
    L.VT = take(static_cast<size_t>(c.cols) * 2 * L.Kp * 2);
    L.Ws = take(static_cast<size_t>(c.rows) * 2 * L.colsp * 2);         // W, rows x (hi | lo)
    L.As = take(K * 2 * static_cast<size_t>(L.colsp) * 2);              // v (DML) or the codes a (SC)
    if (c.model == SFB_SC) {
      L.WTs = take(static_cast<size_t>(c.cols) * 2 * L.rowsp * 2);      // W^T, atoms x (hi | lo)
      L.Rs = take(K * 2 * static_cast<size_t>(L.rowsp) * 2);            // residual r = W a - x
    }
    return;
  }
  const size_t ldz = static_cast<size_t>(round_up(c.rows, 32));
  const size_t nblk = static_cast<size_t>((c.rows + BN - 1) / BN);
  L.Wb = take(static_cast<size_t>(c.rows) * L.colsb * 2);
  L.Xb = take(K * L.colsb * 2);
  L.VT = take(static_cast<size_t>(c.cols) * L.Kp * 2);
  L.ZT = take(K * ldz * 4);                      // logits Z, sample-major [K x ldz]
  L.UT = take(static_cast<size_t>(c.rows) * L.Kp * 2);
  L.part = take(nblk * K * 8);
  L.V = take(K * 4);                             // log-sum-exp per sample
  L.Xf = take(K * static_cast<size_t>(c.cols) * 4);   // fp32 copy of the K samples (exact label-row term)
  L.labels = take(K * 4);                        // class ids of the K samples
  L.coef = take(K * 4);                          // 1 - p_y per sample (fp32 label entry of u)
  L.U = 0;
}

int tc_init(sfb_ctx* ctx) {
  TcState* st = new (std::nothrow) TcState();
  if (!st) return SFB_ERR_ARG;
  ctx->tc = st;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  CKC(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (qres != cudaDriverEntryPointSuccess || !fn) return SFB_ERR_CUDA;
  st->encode = reinterpret_cast<EncodeTiledFn>(fn);
  int dev = 0;
  CKC(cudaGetDevice(&dev));
  CKC(cudaDeviceGetAttribute(&st->sms, cudaDevAttrMultiProcessorCount, dev));
  CKC(prepare_forward_kernels());
  {
    const int rc = tc_update_init(ctx, st);
    if (rc) return rc;
  }
  const sfb_config& c = ctx->cfg;
  if (ctx->tf32) {
    // pad columns of the split operands are never written by the kernels: clear the buffers once
    const Layout& L = ctx->lay;
    CKC(cudaMemsetAsync(ctx->at<char>(L.Ws), 0, static_cast<size_t>(c.rows) * 2 * L.colsp * 4, ctx->stream));
    CKC(cudaMemsetAsync(ctx->at<char>(L.As), 0, static_cast<size_t>(ctx->K) * 2 * L.colsp * 4, ctx->stream));
    return tc_refresh_operands(ctx);
  }
  if (c.model != SFB_MLR) {
    // pad columns of the split operands are never written by the kernels: clear the buffers once
    const Layout& L = ctx->lay;
    const size_t K = static_cast<size_t>(ctx->K);
    CKC(cudaMemsetAsync(ctx->at<char>(L.Ws), 0, static_cast<size_t>(c.rows) * 2 * L.colsp * 2, ctx->stream));
    CKC(cudaMemsetAsync(ctx->at<char>(L.As), 0, K * 2 * L.colsp * 2, ctx->stream));
    if (c.model == SFB_SC) {
      CKC(cudaMemsetAsync(ctx->at<char>(L.WTs), 0, static_cast<size_t>(c.cols) * 2 * L.rowsp * 2, ctx->stream));
      CKC(cudaMemsetAsync(ctx->at<char>(L.Rs), 0, K * 2 * L.rowsp * 2, ctx->stream));
    }
    return SFB_OK;
  }
  // bf16 copy of W for the forward product; afterwards the update's epilogue keeps it current
  return tc_refresh_operands(ctx);
}

int tc_refresh_operands(sfb_ctx* ctx) {
  const sfb_config& c = ctx->cfg;
  if (c.model != SFB_MLR) return SFB_OK;          // the split copies of W are rebuilt by the first factors call of a step
  const TcState* st = static_cast<const TcState*>(ctx->tc);
  if (ctx->tf32) {
    split32_rows_kernel<<<static_cast<unsigned>(st->sms * 16), 256, 0, ctx->stream>>>(ctx->W, c.rows, c.cols, c.cols,
                                                                                     ctx->at<float>(ctx->lay.Ws), ctx->lay.colsp);
    count_launch();
    CKC(cudaGetLastError());
    return SFB_OK;
  }
  convert_rows_kernel<<<st->sms * 8, 256, 0, ctx->stream>>>(ctx->W, c.rows, c.cols, ctx->at<__nv_bfloat16>(ctx->lay.Wb),
                                                            ctx->lay.colsb);
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

void tc_destroy(sfb_ctx* ctx) {
  delete static_cast<TcState*>(ctx->tc);
  ctx->tc = nullptr;
}

namespace {

inline unsigned grid1d(int64_t items, int per_block) {
  int64_t g = (items + per_block - 1) / per_block;
  return static_cast<unsigned>(std::max<int64_t>(1, std::min<int64_t>(g, static_cast<int64_t>(sm_count()) * 16)));
}

// Tile width (a multiple of `step` columns, at most `widest`) for a product with tilesM row blocks and N columns on
// `sms` SMs.  The
// persistent kernel runs ceil(tiles / sms) rounds of tiles; measured, a tile costs about max(width, 128) + 16
// column-equivalents (below 128 columns a k-block is bound by the latency of its operand loads, not by the MMA).
// Narrower tiles fill the SMs of small products, where 256-wide ones leave many idle or need a nearly empty
// second round; ties go to the wider tile.
inline int pick_tile_width(int sms, int64_t tilesM, int64_t N, int widest, int step = 32) {
  int best = widest;
  int64_t best_cost = INT64_MAX;
  for (int bn = widest; bn >= 128; bn -= step) {
    const int64_t tiles = tilesM * ((N + bn - 1) / bn);
    const int64_t cost = ((tiles + sms - 1) / sms) * (bn + 16);
    if (cost < best_cost) { best_cost = cost; best = bn; }
  }
  return best;
}

constexpr int kSplitPrefetch = SFB_SPLIT_PREFETCH;    // k-blocks of look-ahead of the L2 prefetch in the split products

// One split-bf16 product  D[off..off+n) = A * B^T  with A = [*, 2*Cp] and B = [N x 2*Cp] (hi | lo) operands:
// hi*hi + hi*lo + lo*hi over a contraction of Cp.
template <int EPI>
int split_product(sfb_ctx* ctx, int64_t off, int64_t n, __nv_bfloat16* A, __nv_bfloat16* B, int64_t N, int64_t Cp,
                  float* C, int64_t ldc, TcParams p, int64_t c_split_stride = 0, int* parts_out = nullptr) {
  const TcState* st = static_cast<const TcState*>(ctx->tc);
  const int bn = pick_tile_width(st->sms, (n + BM - 1) / BM, N, FS_BN, 16);
  CUtensorMap ma, mb;
  if (!make_map(st, &ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, A, 2 * Cp, off + n, 2 * Cp * 2, BK, BM) ||
      !make_map(st, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, B, 2 * Cp, N, 2 * Cp * 2, BK, bn))
    return SFB_ERR_CUDA;
  p.M = static_cast<int32_t>(off + n); p.N = static_cast<int32_t>(N); p.Kc = static_cast<int32_t>(Cp);
  p.m_off = static_cast<int32_t>(off);
  p.tilesM = static_cast<int32_t>((n + BM - 1) / BM);
  p.bn = bn;
  p.tilesN = static_cast<int32_t>((N + bn - 1) / bn);
  p.nseg = 3; p.kseg = static_cast<int32_t>(Cp / BK);
  p.prefetch = kSplitPrefetch;
  // a product whose tiles fill less than half of the SMs is cut along its contraction (plain store epilogue only: the
  // partial products are added, in a fixed order, by the kernel that consumes them)
  const int64_t tiles = static_cast<int64_t>(p.tilesM) * p.tilesN;
  p.ksplit = (EPI == F_STORE && c_split_stride > 0 && 2 * tiles <= st->sms && p.kseg >= 8) ? 2 : 1;
  p.c_split_stride = p.ksplit > 1 ? c_split_stride : 0;
  if (parts_out) *parts_out = p.ksplit;
  p.a_off0 = 0; p.a_off1 = 0; p.a_off2 = static_cast<int32_t>(Cp);
  p.b_off0 = 0; p.b_off1 = static_cast<int32_t>(Cp); p.b_off2 = 0;
  p.status = ctx->at<uint32_t>(ctx->lay.status);
  CKC(launch_forward_split<EPI>(ctx, ma, mb, C, ldc, p));
  ctx->stats.flops += 3.0 * 2.0 * n * N * Cp;
  return SFB_OK;
}

// Sufficient factors of distance metric learning and sparse coding in bf16 mode: the same steps as the fp32
// path (Section 2: z = W v with v = x - y; Figure 3: ISTA codes, u = W a - x), every product on the tensor cores
// with (hi | lo) bf16 operands.
int factors_split(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const float* Y, const int32_t* labels,
                  float* dml_norm_out = nullptr) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  const int64_t rows = c.rows, cols = c.cols;
  cudaStream_t s = ctx->stream;
  float* V = ctx->at<float>(L.V);
  float* U = ctx->at<float>(L.U);
  __nv_bfloat16* Ws = ctx->at<__nv_bfloat16>(L.Ws);
  __nv_bfloat16* As = ctx->at<__nv_bfloat16>(L.As);
  if (ctx->committed == 0) {
    // first factors of the step: refresh the split copies of the W every worker sees (BSP)
    pack_split_rows_kernel<<<grid1d(rows * cols / 4, 256), 256, 0, s>>>(ctx->W, rows, cols, cols, Ws, L.colsp);
    count_launch();
    if (c.model == SFB_SC) {
      pack_split_t_kernel<<<dim3(static_cast<unsigned>((cols + 63) / 64), static_cast<unsigned>(L.rowsp / 64)), 256, 0, s>>>(
          ctx->W, rows, cols, cols, ctx->at<__nv_bfloat16>(L.WTs), L.rowsp);
      count_launch();
    }
    CKC(cudaGetLastError());
  }
  TcParams p{};
  if (c.model == SFB_DML) {
    CKC(pack_copy(s, V + off * cols, X, Y, n * cols));                                   // v = x - y
    pack_split_rows_kernel<<<grid1d(n * cols / 4, 256), 256, 0, s>>>(V + off * cols, n, cols, cols,
                                                                     As + off * 2 * L.colsp, L.colsp);
    count_launch();
    CKC(cudaGetLastError());
    float* U2 = ctx->at<float>(L.U2);
    int parts = 1;
    int rc = split_product<F_STORE>(ctx, off, n, As, Ws, rows, L.colsp, U, L.ldu, p, U2 - U, &parts);   // z_i = W v_i
    if (rc) return rc;
    CKC(dml_scale_rows(s, U + off * L.ldu, n, rows, L.ldu, labels, c.dml_margin, parts > 1 ? U2 + off * L.ldu : nullptr,
                       dml_norm_out));
    return SFB_OK;
  }
  // sparse coding: ISTA from a = 0, then u = W a - x, v = a
  __nv_bfloat16* WTs = ctx->at<__nv_bfloat16>(L.WTs);
  __nv_bfloat16* Rs = ctx->at<__nv_bfloat16>(L.Rs);
  CKC(cudaMemsetAsync(V + off * cols, 0, static_cast<size_t>(n) * cols * 4, s));
  CKC(cudaMemsetAsync(As + off * 2 * L.colsp, 0, static_cast<size_t>(n) * 2 * L.colsp * 2, s));
  for (int it = 0; it <= c.sc_ista_iters; ++it) {
    p = TcParams{};
    p.aux = X - off * rows; p.ldaux = rows;          // X holds this worker's samples: index it by the global row
    p.split = Rs; p.ld_split = 2 * L.rowsp; p.split_half = static_cast<int32_t>(L.rowsp);
    int rc = split_product<F_SUB>(ctx, off, n, As, Ws, rows, L.colsp, U, L.ldu, p);     // r = W a - x
    if (rc) return rc;
    if (it == c.sc_ista_iters) break;
    p = TcParams{};
    p.aux = V; p.ldaux = cols;
    p.sc = ctx->at<Scalars>(L.scalars); p.lam = c.sc_lambda;
    p.split = As; p.ld_split = 2 * L.colsp; p.split_half = static_cast<int32_t>(L.colsp);
    rc = split_product<F_ISTA>(ctx, off, n, Rs, WTs, cols, L.rowsp, V, cols, p);        // a <- soft(a - W^T r / L)
    if (rc) return rc;
  }
  return SFB_OK;
}

}  // namespace

// v = x, the (big | small) samples, and the logits of n samples at pair offset off against this context's rows as
// the three-term tf32 product, with the per-(sample, 256-row block) softmax partials.
static int mlr32_forward(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, int* tiles_n) {
  const sfb_config& c = ctx->cfg;
  const TcState* st = static_cast<const TcState*>(ctx->tc);
  const Layout& L = ctx->lay;
  const int64_t rows = c.rows, cols = c.cols, K = ctx->K;
  const int64_t ldz = round_up(rows, 32);
  cudaStream_t s = ctx->stream;
  float* Ws = ctx->at<float>(L.Ws);
  float* As = ctx->at<float>(L.As);
  float* Z = ctx->at<float>(L.ZT);
  float* V = ctx->at<float>(L.V) + off * cols;
  // Ws, the (big | small) copy of W, is built at set-up and rewritten by the update's epilogue together with W
  CKC(pack_copy(s, V, X, nullptr, n * cols));                                              // v = x
  split32_rows_kernel<<<grid1d(n * cols / 4, 256), 256, 0, s>>>(X, n, cols, cols, As + off * 2 * L.colsp, L.colsp);
  count_launch();
  CKC(cudaGetLastError());
  CUtensorMap ma, mb, mc;
  if (!make_map(st, &ma, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, As, 2 * L.colsp, off + n, 2 * L.colsp * 4, BK / 2, BM) ||
      !make_map(st, &mb, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Ws, 2 * L.colsp, rows, 2 * L.colsp * 4, BK / 2, BN) ||
      !make_map(st, &mc, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Z, rows, off + n, ldz * 4, kChunk, 32))
    return SFB_ERR_CUDA;
  TcParams p{};
  p.M = static_cast<int32_t>(off + n); p.N = static_cast<int32_t>(rows); p.Kc = static_cast<int32_t>(L.colsp);
  p.m_off = static_cast<int32_t>(off);
  p.tilesM = static_cast<int32_t>((n + BM - 1) / BM);
  p.bn = BN;
  p.tilesN = static_cast<int32_t>((rows + BN - 1) / BN);
  p.part = ctx->at<float2>(L.part); p.part_ld = K; p.status = ctx->at<uint32_t>(L.status);
  p.nseg = 3; p.kseg = static_cast<int32_t>(L.colsp / (BK / 2));          // cross terms first, big*big last
  p.a_off0 = 0; p.a_off1 = static_cast<int32_t>(L.colsp); p.a_off2 = 0;
  p.b_off0 = static_cast<int32_t>(L.colsp); p.b_off1 = 0; p.b_off2 = 0;
  CKC((launch_forward<F_SOFTMAX, true>(ctx, ma, mb, mc, p)));                                // z_i = W x_i
  ctx->stats.flops += 3.0 * 2.0 * n * rows * cols;
  *tiles_n = p.tilesN;
  return SFB_OK;
}

// Row-sharded form in the tensor-core fp32 mode: partials of all K samples against this shard's rows ...
int tc32_forward_partials(sfb_ctx* ctx, const float* X, const int32_t* labels, float* part_out) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  int tiles_n = 0;
  const int rc = mlr32_forward(ctx, 0, ctx->K, X, &tiles_n);
  if (rc) return rc;
  CKC(cudaMemcpyAsync(ctx->at<int32_t>(L.labels), labels, static_cast<size_t>(ctx->K) * 4, cudaMemcpyDeviceToDevice, ctx->stream));
  mlr_shard_partials_tc_kernel<<<static_cast<unsigned>((ctx->K + 7) / 8), 256, 0, ctx->stream>>>(
      ctx->at<float2>(L.part), ctx->K, tiles_n, ctx->at<float>(L.ZT), round_up(c.rows, 32), c.rows,
      ctx->at<int32_t>(L.labels), ctx->row_offset, ctx->K, reinterpret_cast<float4*>(part_out));
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

// ... and the fp32 factors from the partials of all shards.
int tc32_finish_factors(sfb_ctx* ctx, const float* parts, int shards) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  const int64_t K = ctx->K, rows = c.rows;
  mlr_shard_finish_tc_kernel<<<static_cast<unsigned>((K + 255) / 256), 256, 0, ctx->stream>>>(
      reinterpret_cast<const float4*>(parts), shards, K, rows, ctx->row_offset, ctx->at<int32_t>(L.labels),
      ctx->at<float>(L.lse), ctx->at<float>(L.loss), ctx->at<float>(L.coef), ctx->at<uint32_t>(L.status));
  count_launch();
  dim3 ugrid(static_cast<unsigned>(std::min<int64_t>((rows + 255) / 256, 64)), static_cast<unsigned>(K));
  mlr_finish_u_kernel<false><<<ugrid, 256, 0, ctx->stream>>>(ctx->at<float>(L.ZT), round_up(rows, 32), rows, ctx->at<float>(L.lse),
                                                             ctx->at<int32_t>(L.labels), ctx->at<float>(L.U));
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

// fp32 mode on the tensor cores: factors of n MLR samples at pair offset off.  The logits are the three-term tf32
// product of the (big | small) samples and the (big | small) rows of W; softmax, loss and the factors in fp32.
// sdca_ids != nullptr: the dual changes of the SDCA step instead of softmax - onehot.
int tc32_factors(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const int32_t* labels, const int32_t* sdca_ids,
                 float inv_lam_n) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  const int64_t rows = c.rows, cols = c.cols, K = ctx->K;
  const int64_t ldz = round_up(rows, 32);
  cudaStream_t s = ctx->stream;
  float* Z = ctx->at<float>(L.ZT);
  float* U = ctx->at<float>(L.U) + off * rows;
  int tiles_n = 0;
  {
    const int rc = mlr32_forward(ctx, off, n, X, &tiles_n);
    if (rc) return rc;
  }
  dim3 ugrid(static_cast<unsigned>(std::min<int64_t>((rows + 255) / 256, 64)), static_cast<unsigned>(n));
  if (sdca_ids) {
    CKC(sdca_dual_rows(s, Z + off * ldz, n, rows, ldz, X, cols, labels, sdca_ids, ctx->dualQ, ctx->dual_n, inv_lam_n, c.eta,
                       nullptr, ctx->at<float>(L.loss) + off, ctx->at<uint32_t>(L.status)));
    mlr_finish_u_kernel<true><<<ugrid, 256, 0, s>>>(Z + off * ldz, ldz, rows, nullptr, nullptr, U);
  } else {
    float* lse = ctx->at<float>(L.lse);
    mlr_lse_kernel<<<static_cast<unsigned>((n + 7) / 8), 256, 0, s>>>(ctx->at<float2>(L.part), K, tiles_n, Z, ldz, rows, labels,
                                                                     off, n, lse, ctx->at<float>(L.loss),
                                                                     ctx->at<float>(L.coef), ctx->at<uint32_t>(L.status));
    count_launch();
    mlr_finish_u_kernel<false><<<ugrid, 256, 0, s>>>(Z + off * ldz, ldz, rows, lse + off, labels, U);
  }
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

// The gathered fp32 pairs (computed here or received) become the (big | small) operands of the update product.
int tc32_gather(sfb_ctx* ctx) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  const unsigned gy = static_cast<unsigned>((L.Kp + 63) / 64);
  split32_t_kernel<<<dim3(static_cast<unsigned>((c.rows + 63) / 64), gy), 256, 0, ctx->stream>>>(
      ctx->at<float>(L.U), ctx->K, c.rows, c.rows, ctx->at<float>(L.UT), L.Kp);
  count_launch();
  split32_t_kernel<<<dim3(static_cast<unsigned>((c.cols + 63) / 64), gy), 256, 0, ctx->stream>>>(
      ctx->at<float>(L.V), ctx->K, c.cols, c.cols, ctx->at<float>(L.VT), L.Kp);
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

// Pack of n samples at pair offset off and their logits against the rows of this context's W:
// Z[off .. off+n) = X W^T with the per-(sample, 256-row block) softmax partials.
static int mlr_forward(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const int32_t* labels, int* tiles_n) {
  const sfb_config& c = ctx->cfg;
  const TcState* st = static_cast<const TcState*>(ctx->tc);
  const Layout& L = ctx->lay;
  const int64_t rows = c.rows, cols = c.cols, K = ctx->K;
  const int64_t ldz = round_up(rows, 32);
  __nv_bfloat16* Xb = ctx->at<__nv_bfloat16>(L.Xb);
  dim3 pgrid(static_cast<unsigned>((cols + 63) / 64), static_cast<unsigned>((n + 63) / 64));
  pack_mlr_kernel<<<pgrid, 256, 0, ctx->stream>>>(X, n, cols, Xb, L.colsb, ctx->at<__nv_bfloat16>(L.VT), L.Kp, off,
                                                  ctx->at<float>(L.Xf), labels, ctx->at<int32_t>(L.labels));
  count_launch();
  CKC(cudaGetLastError());
  // samples on the lanes (A), rows of W on the accumulator columns (B)
  CUtensorMap ma, mb, mc;
  if (!make_map(st, &ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Xb, cols, off + n, L.colsb * 2, BK, BM) ||
      !make_map(st, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, ctx->at<__nv_bfloat16>(L.Wb), cols, rows, L.colsb * 2, BK, BN) ||
      !make_map(st, &mc, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, ctx->at<float>(L.ZT), rows, off + n, ldz * 4, kChunk, 32))
    return SFB_ERR_CUDA;
  TcParams p{};
  p.M = static_cast<int32_t>(off + n); p.N = static_cast<int32_t>(rows); p.Kc = static_cast<int32_t>(cols);
  p.m_off = static_cast<int32_t>(off);
  p.tilesM = static_cast<int32_t>((n + BM - 1) / BM);
  p.bn = BN;
  p.tilesN = static_cast<int32_t>((rows + BN - 1) / BN);
  p.part = ctx->at<float2>(L.part); p.part_ld = K; p.status = ctx->at<uint32_t>(L.status);
  p.nseg = 1; p.kseg = (p.Kc + BK - 1) / BK;
  CKC(launch_forward<F_SOFTMAX>(ctx, ma, mb, mc, p));
  ctx->stats.flops += 2.0 * n * rows * cols;
  *tiles_n = p.tilesN;
  return SFB_OK;
}

int tc_forward_partials(sfb_ctx* ctx, const float* X, const int32_t* labels, float* part_out) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  int tiles_n = 0;
  const int rc = mlr_forward(ctx, 0, ctx->K, X, labels, &tiles_n);
  if (rc) return rc;
  mlr_shard_partials_tc_kernel<<<static_cast<unsigned>((ctx->K + 7) / 8), 256, 0, ctx->stream>>>(
      ctx->at<float2>(L.part), ctx->K, tiles_n, ctx->at<float>(L.ZT), round_up(c.rows, 32), c.rows,
      ctx->at<int32_t>(L.labels), ctx->row_offset, ctx->K, reinterpret_cast<float4*>(part_out));
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

int tc_finish_factors(sfb_ctx* ctx, const float* parts, int shards) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  const int64_t K = ctx->K;
  mlr_shard_finish_tc_kernel<<<static_cast<unsigned>((K + 255) / 256), 256, 0, ctx->stream>>>(
      reinterpret_cast<const float4*>(parts), shards, K, c.rows, ctx->row_offset, ctx->at<int32_t>(L.labels),
      ctx->at<float>(L.V), ctx->at<float>(L.loss), ctx->at<float>(L.coef), ctx->at<uint32_t>(L.status));
  count_launch();
  dim3 egrid(static_cast<unsigned>((c.rows + 63) / 64), static_cast<unsigned>((K + 63) / 64));
  mlr_emit_ut_kernel<false><<<egrid, 256, 0, ctx->stream>>>(ctx->at<float>(L.ZT), round_up(c.rows, 32), c.rows, ctx->at<float>(L.V), 0, K,
                                                     ctx->at<int32_t>(L.labels), ctx->at<__nv_bfloat16>(L.UT), L.Kp);
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

// What a worker sends (Section 3) in bf16 mode: u_ij = exp(z_ij - lse_i) - [j = y_i] in fp32 from the logits and the
// log-partition it holds; one block row per sample.
__global__ void __launch_bounds__(256) mlr_export_u_kernel(const float* __restrict__ Z, int64_t ldz, int64_t rows,
                                                           const float* __restrict__ lse, const int32_t* __restrict__ labels,
                                                           int64_t off, float* __restrict__ U_out) {
  const int64_t i = blockIdx.y;
  const float l = lse[off + i];
  const int32_t y = labels[off + i];
  const float* z = Z + (off + i) * ldz;
  float* u = U_out + i * rows;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t j = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; j < rows; j += stride)
    u[j] = expf(z[j] - l) - (j == y ? 1.f : 0.f);
}

// A received u = p - onehot(y): its smallest entry is the (only negative) one at y.  Per sample: the class, the fp32
// label coefficient 1 - p_y = -u_y and the loss -log p_y, as the local softmax pass leaves them.  One block per sample;
// ties (none for a valid u) go to the smaller index.
__global__ void __launch_bounds__(256) mlr_import_labels_kernel(const float* __restrict__ U_in, int64_t rows, int64_t off,
                                                                int32_t* __restrict__ labels, float* __restrict__ coef,
                                                                float* __restrict__ loss) {
  __shared__ float sv[256];
  __shared__ int32_t si[256];
  const int64_t i = blockIdx.x;
  const float* u = U_in + i * rows;
  float best = INFINITY;
  int32_t arg = 0;
  for (int64_t j = threadIdx.x; j < rows; j += 256) {
    const float v = u[j];
    if (v < best) { best = v; arg = static_cast<int32_t>(j); }
  }
  sv[threadIdx.x] = best; si[threadIdx.x] = arg;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      const float v = sv[threadIdx.x + o];
      const int32_t a = si[threadIdx.x + o];
      if (v < sv[threadIdx.x] || (v == sv[threadIdx.x] && a < si[threadIdx.x])) { sv[threadIdx.x] = v; si[threadIdx.x] = a; }
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float c = fminf(fmaxf(-sv[0], 0.f), 1.f);
    labels[off + i] = si[0];
    coef[off + i] = c;
    loss[off + i] = -logf(fmaxf(1.f - c, 1e-37f));
  }
}

int tc_export_factors(sfb_ctx* ctx, int64_t off, int64_t n, float* U_out, float* V_out) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  const int64_t ldz = round_up(c.rows, 32);
  dim3 grid(static_cast<unsigned>(std::min<int64_t>((c.rows + 255) / 256, 64)), static_cast<unsigned>(n));
  mlr_export_u_kernel<<<grid, 256, 0, ctx->stream>>>(ctx->at<float>(L.ZT), ldz, c.rows, ctx->at<float>(L.V),
                                                     ctx->at<int32_t>(L.labels), off, U_out);
  count_launch();
  CKC(cudaGetLastError());
  CKC(cudaMemcpyAsync(V_out, ctx->at<float>(L.Xf) + off * c.cols, static_cast<size_t>(n) * c.cols * 4, cudaMemcpyDeviceToDevice,
                      ctx->stream));
  return SFB_OK;
}

// Received fp32 factors take a worker's place in the bf16 layout: v into V^T (bf16) and the fp32 sample copy, u into U^T
// (bf16, 0 at the class entry), the class entry into the fp32 label coefficients.
int tc_import_factors(sfb_ctx* ctx, int64_t off, int64_t n, const float* U_in, const float* V_in) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  const int64_t rows = c.rows, cols = c.cols;
  const int64_t ldz = round_up(rows, 32);
  cudaStream_t s = ctx->stream;
  int32_t* labels = ctx->at<int32_t>(L.labels);
  mlr_import_labels_kernel<<<static_cast<unsigned>(n), 256, 0, s>>>(U_in, rows, off, labels, ctx->at<float>(L.coef),
                                                                   ctx->at<float>(L.loss));
  count_launch();
  float* Z = ctx->at<float>(L.ZT);
  CKC(cudaMemcpy2DAsync(Z + off * ldz, static_cast<size_t>(ldz) * 4, U_in, static_cast<size_t>(rows) * 4,
                        static_cast<size_t>(rows) * 4, static_cast<size_t>(n), cudaMemcpyDeviceToDevice, s));
  dim3 pgrid(static_cast<unsigned>((cols + 63) / 64), static_cast<unsigned>((n + 63) / 64));
  pack_mlr_kernel<<<pgrid, 256, 0, s>>>(V_in, n, cols, ctx->at<__nv_bfloat16>(L.Xb), L.colsb, ctx->at<__nv_bfloat16>(L.VT), L.Kp,
                                        off, ctx->at<float>(L.Xf), labels + off, labels);
  count_launch();
  dim3 egrid(static_cast<unsigned>((rows + 63) / 64), static_cast<unsigned>((n + 63) / 64));
  mlr_emit_ut_kernel<true><<<egrid, 256, 0, s>>>(Z, ldz, rows, nullptr, off, n, labels + off, ctx->at<__nv_bfloat16>(L.UT), L.Kp);
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

// SDCA factors in bf16 mode: logits by the forward product, the dual changes in fp32 in place of the logits, then the
// bf16 operand U^T = du (0 at the label entry, which goes to W in fp32 through coef, as for MLR).
int tc_sdca_factors(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const int32_t* labels, const int32_t* ids,
                    float inv_lam_n) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  const int64_t rows = c.rows;
  const int64_t ldz = round_up(rows, 32);
  float* Z = ctx->at<float>(L.ZT);
  int tiles_n = 0;
  const int rc = mlr_forward(ctx, off, n, X, labels, &tiles_n);
  if (rc) return rc;
  CKC(sdca_dual_rows(ctx->stream, Z + off * ldz, n, rows, ldz, X, c.cols, labels, ids, ctx->dualQ, ctx->dual_n, inv_lam_n,
                     c.eta, ctx->at<float>(L.coef) + off, ctx->at<float>(L.loss) + off, ctx->at<uint32_t>(L.status)));
  dim3 egrid(static_cast<unsigned>((rows + 63) / 64), static_cast<unsigned>((n + 63) / 64));
  mlr_emit_ut_kernel<true><<<egrid, 256, 0, ctx->stream>>>(Z, ldz, rows, nullptr, off, n, labels, ctx->at<__nv_bfloat16>(L.UT),
                                                           L.Kp);
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

int tc_factors(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const float* Y, const int32_t* labels,
               float* dml_norm_out) {
  if (ctx->cfg.model != SFB_MLR) return factors_split(ctx, off, n, X, Y, labels, dml_norm_out);
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  const int64_t rows = c.rows, K = ctx->K;
  const int64_t ldz = round_up(rows, 32);
  float* Z = ctx->at<float>(L.ZT);
  float* lse = ctx->at<float>(L.V);
  int tiles_n = 0;
  const int rc = mlr_forward(ctx, off, n, X, labels, &tiles_n);
  if (rc) return rc;
  mlr_lse_kernel<<<static_cast<unsigned>((n + 7) / 8), 256, 0, ctx->stream>>>(
      ctx->at<float2>(L.part), K, tiles_n, Z, ldz, rows, labels, off, n, lse, ctx->at<float>(L.loss), ctx->at<float>(L.coef),
      ctx->at<uint32_t>(L.status));
  count_launch();
  dim3 egrid(static_cast<unsigned>((rows + 63) / 64), static_cast<unsigned>((n + 63) / 64));
  mlr_emit_ut_kernel<false><<<egrid, 256, 0, ctx->stream>>>(Z, ldz, rows, lse, off, n, labels, ctx->at<__nv_bfloat16>(L.UT), L.Kp);
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

// MLR: every worker wrote at its offset of U^T and V^T, nothing to move.  DML, SC: the workers' fp32 factors
// are transposed into the split-bf16 operands of the update product.
int tc_gather(sfb_ctx* ctx) {
  const sfb_config& c = ctx->cfg;
  if (c.model == SFB_MLR) return SFB_OK;
  const Layout& L = ctx->lay;
  const unsigned gy = static_cast<unsigned>(L.Kp / 64);
  pack_split_t_kernel<<<dim3(static_cast<unsigned>((c.rows + 63) / 64), gy), 256, 0, ctx->stream>>>(
      ctx->at<float>(L.U), ctx->K, c.rows, L.ldu, ctx->at<__nv_bfloat16>(L.UT), L.Kp);
  count_launch();
  pack_split_t_kernel<<<dim3(static_cast<unsigned>((c.cols + 63) / 64), gy), 256, 0, ctx->stream>>>(
      ctx->at<float>(L.V), ctx->K, c.cols, c.cols, ctx->at<__nv_bfloat16>(L.VT), L.Kp);
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

int tc_get_factors(sfb_ctx* ctx, const void** U, const void** V, int32_t* dtype, int32_t* layout, int64_t* ldu,
                   int64_t* ldv) {
  if (ctx->cfg.model != SFB_MLR) {   // the workers' fp32 factors, pair-major
    if (U) *U = ctx->at<float>(ctx->lay.U);
    if (V) *V = ctx->at<float>(ctx->lay.V);
    if (dtype) *dtype = 0;
    if (layout) *layout = 0;
    if (ldu) *ldu = ctx->lay.ldu;
    if (ldv) *ldv = ctx->cfg.cols;
    return SFB_OK;
  }
  if (U) *U = ctx->at<__nv_bfloat16>(ctx->lay.UT);
  if (V) *V = ctx->at<__nv_bfloat16>(ctx->lay.VT);
  if (dtype) *dtype = 1;
  if (layout) *layout = 1;
  if (ldu) *ldu = ctx->lay.Kp;
  if (ldv) *ldv = ctx->lay.Kp;
  return SFB_OK;
}

}  // namespace sfb
