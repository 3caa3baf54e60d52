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
#include <new>

#include "sfb_ptx.cuh"
#include "sfb_tc.h"

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

struct TcParams {
  int32_t M, N, Kc;            // extents of the product: samples, rows of W, features
  int32_t m_off;               // first sample handled by this launch (per-worker slices)
  int32_t tilesM, tilesN;
  float2* part;                // [tilesN][part_ld] (max, sum exp) per sample and 256-row block
  int64_t part_ld;
  uint32_t* status;
};

// Tiles are numbered with the sample block fastest: consecutive tiles (which run on different SMs at the same
// time) share one block of W, which therefore stays hot in L2 while all K samples are swept past it.
__device__ __forceinline__ void tile_coords(const TcParams& p, int tile, int& m0, int& n0) {
  const int tm = tile % p.tilesM, tn = tile / p.tilesM;
  m0 = p.m_off + tm * BM;
  n0 = tn * BN;
}

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
  const int numK = (p.Kc + BK - 1) / BK;

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
        for (int kb = 0; kb < numK; ++kb, ++it) {
          const uint32_t s = it % S, ph = (it / S) & 1;
          if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; break; }
          mbar_expect_tx(&full[s], kBytesA + kBytesB);
          tma_load_2d_hint(sA + s * kBytesA, &tmA, kb * BK, m0, &full[s], pol_keep);
          tma_load_2d(sB + s * kBytesB, &tmB, kb * BK, n0, &full[s]);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(BM, BN);
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
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16(d_tmem, da + static_cast<uint64_t>(k * UMMA_K * 2 / 16), db + static_cast<uint64_t>(k * UMMA_K * 2 / 16),
                      idesc, (kb | k) != 0 ? 1u : 0u);
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
      // Forward: store Z through the ring and keep a running (max, sum exp) per sample over the tile's columns.
      uint32_t gs = 0;                       // stores issued so far: consecutive stores alternate ring slots
      for (int tl = 0; tl < my_tiles && ok; ++tl) {
        int m0, n0;
        tile_coords(p, blockIdx.x + tl * gridDim.x, m0, n0);
        const uint32_t a = tl & 1, aph = (tl >> 1) & 1;
        if (!__all_sync(0xffffffffu, mbar_wait(&tfull[a], aph, abort_flag))) { ok = false; break; }
        tc_fence_after();
        const int row = m0 + q * 32 + lane;
        float mx = -INFINITY, sum = 0.f;
        for (int c = 0; c < BN / kChunk; ++c) {
          uint8_t* sl = ring + (gs % R) * kSlotBytes;
          uint32_t acc[32];
          tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + a * BN + c * kChunk, acc);
          tmem_ld_wait();
          const int col0 = n0 + c * kChunk;
          if (col0 < p.N) {
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
        if (row < p.M) p.part[static_cast<int64_t>(n0 / BN) * p.part_ld + row] = make_float2(mx, sum);
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
                                                           __nv_bfloat16* __restrict__ FT, int64_t Kp) {
  __shared__ float tile[64][65];
  const int64_t i0 = static_cast<int64_t>(blockIdx.y) * 64, c0 = static_cast<int64_t>(blockIdx.x) * 64;
  const int t = threadIdx.x;
  const bool vec = (dim % 4) == 0;
#pragma unroll
  for (int v = 0; v < 4; ++v) {
    const int idx = t + v * 256;            // 64 samples x 16 quads
    const int i = idx / 16, cq = (idx % 16) * 4;
    float f[4] = {0.f, 0.f, 0.f, 0.f};
    if (i0 + i < n) {
      const float* src = F + (i0 + i) * dim + c0 + cq;
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

// One warp per sample: merge the per-block (max, sum exp) partials into log sum exp; loss = lse - z_y.
__global__ void __launch_bounds__(256) mlr_lse_kernel(const float2* __restrict__ part, int64_t part_ld, int nblocks,
                                                      const float* __restrict__ Z, int64_t ldz, int64_t rows,
                                                      const int32_t* __restrict__ labels, int64_t off, int64_t n,
                                                      float* __restrict__ lse, float* __restrict__ loss,
                                                      uint32_t* status) {
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
    loss[s] = okl ? l - Z[s * ldz + y] : 0.f;
  }
}

// P^T[r][off + i] = bf16( exp(z_ir - lse_i) ): 64 samples x 64 rows per block, transposed through shared
// memory (Z is sample-major, the update operand is row-major with samples contiguous).  The factor is
// u_i = p_i - onehot(y_i); its onehot part is not rounded to bf16 but applied exactly by label_rows_kernel.
__global__ void __launch_bounds__(256) mlr_emit_ut_kernel(const float* __restrict__ Z, int64_t ldz, int64_t rows,
                                                          const float* __restrict__ lse, int64_t off, int64_t n,
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
    const float l = lse[s];
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
      tile[i][rq + k] = __expf(z[k] - l);
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
// Host side
// ---------------------------------------------------------------------------------------------------------
cudaError_t launch_forward(sfb_ctx* ctx, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c, TcParams p) {
  const TcState* st = static_cast<const TcState*>(ctx->tc);
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int64_t tiles = static_cast<int64_t>(p.tilesM) * p.tilesN;
  if (tiles <= 0) return cudaSuccess;
  const int grid = static_cast<int>(tiles < st->sms ? tiles : st->sms);
  forward_kernel<<<grid, kThreads, kSmem, ctx->stream>>>(a, b, c, p);
  count_launch();
  return cudaGetLastError();
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

void tc_extend_layout(const sfb_config& c, Layout& L, size_t& off) {
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + kAlign - 1) / kAlign * kAlign; return o; };
  const size_t K = static_cast<size_t>(c.workers) * c.batch;
  L.Kp = round_up(static_cast<int64_t>(K), 64);
  L.colsb = round_up(c.cols, 64);
  if (c.model != SFB_MLR) {
    // fp32 factors as the workers write them, and their split-bf16 transposes for the update product
    L.V = take(K * static_cast<size_t>(c.cols) * 4);
    L.U = take(K * static_cast<size_t>(c.rows) * 4);
    L.UT = take(static_cast<size_t>(c.rows) * 2 * L.Kp * 2);
    L.VT = take(static_cast<size_t>(c.cols) * 2 * L.Kp * 2);
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
  {
    const int rc = tc_update_init(ctx, st);
    if (rc) return rc;
  }
  const sfb_config& c = ctx->cfg;
  if (c.model != SFB_MLR) return SFB_OK;        // the forward products of DML and SC run on fp32 operands
  // bf16 copy of W for the forward product; afterwards the update's epilogue keeps it current
  convert_rows_kernel<<<148 * 8, 256, 0, ctx->stream>>>(ctx->W, c.rows, c.cols, ctx->at<__nv_bfloat16>(ctx->lay.Wb),
                                                        ctx->lay.colsb);
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

void tc_destroy(sfb_ctx* ctx) {
  delete static_cast<TcState*>(ctx->tc);
  ctx->tc = nullptr;
}

int tc_factors(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const float* /*Y*/, const int32_t* labels) {
  const sfb_config& c = ctx->cfg;
  const TcState* st = static_cast<const TcState*>(ctx->tc);
  const Layout& L = ctx->lay;
  const int64_t rows = c.rows, cols = c.cols, K = ctx->K;
  const int64_t ldz = round_up(rows, 32);
  __nv_bfloat16* Xb = ctx->at<__nv_bfloat16>(L.Xb);
  __nv_bfloat16* VT = ctx->at<__nv_bfloat16>(L.VT);
  __nv_bfloat16* Wb = ctx->at<__nv_bfloat16>(L.Wb);
  __nv_bfloat16* UT = ctx->at<__nv_bfloat16>(L.UT);
  float* Z = ctx->at<float>(L.ZT);
  float2* part = ctx->at<float2>(L.part);
  float* lse = ctx->at<float>(L.V);
  float* loss = ctx->at<float>(L.loss);
  uint32_t* status = ctx->at<uint32_t>(L.status);

  dim3 pgrid(static_cast<unsigned>((cols + 63) / 64), static_cast<unsigned>((n + 63) / 64));
  pack_mlr_kernel<<<pgrid, 256, 0, ctx->stream>>>(X, n, cols, Xb, L.colsb, VT, L.Kp, off, ctx->at<float>(L.Xf), labels,
                                                  ctx->at<int32_t>(L.labels));
  count_launch();
  CKC(cudaGetLastError());

  // Z[off .. off+n) = X W^T : samples on the lanes (A), rows of W on the accumulator columns (B)
  CUtensorMap ma, mb, mc;
  if (!make_map(st, &ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Xb, cols, off + n, L.colsb * 2, BK, BM) ||
      !make_map(st, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Wb, cols, rows, L.colsb * 2, BK, BN) ||
      !make_map(st, &mc, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Z, rows, off + n, ldz * 4, kChunk, 32))
    return SFB_ERR_CUDA;
  TcParams p{};
  p.M = static_cast<int32_t>(off + n); p.N = static_cast<int32_t>(rows); p.Kc = static_cast<int32_t>(cols);
  p.m_off = static_cast<int32_t>(off);
  p.tilesM = static_cast<int32_t>((n + BM - 1) / BM);
  p.tilesN = static_cast<int32_t>((rows + BN - 1) / BN);
  p.part = part; p.part_ld = K; p.status = status;
  CKC(launch_forward(ctx, ma, mb, mc, p));
  ctx->stats.flops += 2.0 * n * rows * cols;

  mlr_lse_kernel<<<static_cast<unsigned>((n + 7) / 8), 256, 0, ctx->stream>>>(part, K, p.tilesN, Z, ldz, rows, labels, off,
                                                                              n, lse, loss, status);
  count_launch();
  dim3 egrid(static_cast<unsigned>((rows + 63) / 64), static_cast<unsigned>((n + 63) / 64));
  mlr_emit_ut_kernel<<<egrid, 256, 0, ctx->stream>>>(Z, ldz, rows, lse, off, n, UT, L.Kp);
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
      ctx->at<float>(L.U), ctx->K, c.rows, ctx->at<__nv_bfloat16>(L.UT), L.Kp);
  count_launch();
  pack_split_t_kernel<<<dim3(static_cast<unsigned>((c.cols + 63) / 64), gy), 256, 0, ctx->stream>>>(
      ctx->at<float>(L.V), ctx->K, c.cols, ctx->at<__nv_bfloat16>(L.VT), L.Kp);
  count_launch();
  CKC(cudaGetLastError());
  return SFB_OK;
}

int tc_after_update(sfb_ctx*) { return SFB_OK; }

int tc_get_factors(sfb_ctx* ctx, const void** U, const void** V, int32_t* dtype, int32_t* layout, int64_t* ldu,
                   int64_t* ldv) {
  if (ctx->cfg.model != SFB_MLR) {   // the workers' fp32 factors, pair-major
    if (U) *U = ctx->at<float>(ctx->lay.U);
    if (V) *V = ctx->at<float>(ctx->lay.V);
    if (dtype) *dtype = 0;
    if (layout) *layout = 0;
    if (ldu) *ldu = ctx->cfg.rows;
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
