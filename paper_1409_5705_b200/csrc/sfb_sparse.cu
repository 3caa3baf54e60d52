// Sparse sufficient factors of multiclass logistic regression (Section 6: the features of the paper's data sets are
// sparse; Section 3: a factor v_i = a_i with few non-zeros is sent as its (index, value) pairs).
//
// The samples arrive in compressed-sparse-row form.  Their logits still need every column of W (the union of the
// non-zero columns of a mini-batch covers the matrix): the tensor-core modes keep the dense forward product over the
// scattered samples, the fp32 FMA mode has a row-wise product over the non-zeros (sparse_forward_kernel).  What the
// zeros remove is the work of the update:
//     W[j][d] <- prox( W[j][d] - eta * sum_{i : x_id != 0} u_ij x_id )
// has as many terms per entry as column d has non-zeros in the mini-batch (K * density) instead of K.  The kernel here
// streams W once, as the dense update does, and sums only those terms, from the column-major (CSC) form of the
// mini-batch that the gather step builds.
#include <cuda_bf16.h>

#include <algorithm>

#include "sfb_internal.h"

namespace sfb {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kSuWarps = 16;                       // warps per block of the update kernel
constexpr int kSuThreads = kSuWarps * 32;
constexpr int kSuStage = 32 * 33;                  // floats of one warp's 32 x 32 buffer of sums
constexpr int kSuChunk = 176;                      // entries (8 bytes each) of a column block staged at a time, per warp
constexpr int kSuWarpBytes = kSuStage * 4 + kSuChunk * 8;
constexpr int kSmemOptIn = 232448 - 1024;          // dynamic shared memory asked for: what a block may opt into, less the static part

inline unsigned grid1d(int64_t n, int block, int cap = 148 * 16) {
  return static_cast<unsigned>(std::max<int64_t>(1, std::min<int64_t>((n + block - 1) / block, cap)));
}

// Shared-memory reads of the inner loop through 32-bit shared-space addresses (one integer multiply-add per address).
__device__ __forceinline__ uint32_t shared_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ float lds_f32(uint32_t a) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t a) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts_f32(uint32_t a, float v) {
  asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(v) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ int4 lds_v4(uint32_t a) {
  int4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}

// ---------------------------------------------------------------------------------------------------------
// Staging of a worker's CSR block: the dense fp32 samples for the forward product, and (sample, column, value)
// triples appended to the step's list for the column-major form.  One warp per sample.
// ---------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) csr_stage_kernel(const int64_t* __restrict__ indptr, const int32_t* __restrict__ idx,
                                                        const float* __restrict__ val, int64_t n, int64_t nnz, int64_t cols,
                                                        int64_t off, float* __restrict__ Xd, int32_t* __restrict__ coo_i,
                                                        int32_t* __restrict__ coo_c, float* __restrict__ coo_x,
                                                        int2* __restrict__ coo_cx, int32_t fill, int32_t* __restrict__ row_beg,
                                                        int32_t* __restrict__ row_end, uint32_t* __restrict__ status) {
  const int64_t i = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (i >= n) return;
  const int64_t base = indptr[0];
  const int64_t b = indptr[i] - base, e = indptr[i + 1] - base;
  if (b < 0 || e < b || e > nnz) {                 // row pointers that do not describe nnz entries: sample left empty
    if (lane == 0) {
      atomicOr(status, SFB_STATUS_INDEX_RANGE);
      row_beg[off + i] = row_end[off + i] = fill;
    }
    return;
  }
  if (lane == 0) {                                 // the sample's range in the step's list (for the row-wise forward)
    row_beg[off + i] = fill + static_cast<int32_t>(b);
    row_end[off + i] = fill + static_cast<int32_t>(e);
  }
  for (int64_t t = b + lane; t < e; t += 32) {
    const int32_t c = idx[base + t];
    const float x = val[base + t];
    if (c < 0 || c >= cols) {                      // entry skipped (its slot keeps the "no entry" mark)
      atomicOr(status, SFB_STATUS_INDEX_RANGE);
      coo_cx[t] = make_int2(0, 0);                 // value 0 at column 0: adds nothing to a logit
      continue;
    }
    coo_cx[t] = make_int2(c, __float_as_int(x));
    Xd[(off + i) * cols + c] = x;
    coo_i[t] = static_cast<int32_t>(off + i);
    coo_c[t] = c;
    coo_x[t] = x;
  }
}

// ---------------------------------------------------------------------------------------------------------
// Column-major form of the step's K samples: a counting sort of the triples by column, then every column's
// entries in ascending sample order (so that the sums of the update have one order, whatever order the atomics
// of the fill took).  Column d owns ent[ptr[d] .. ptr[d+1]); its length is rounded up to an even number with a
// (sample K, value 0) entry, which points at an all-zero row of the factor slab.
// ---------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) csc_count_kernel(const int32_t* __restrict__ coo_c, int64_t nnz, int32_t* __restrict__ cnt) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t t = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; t < nnz; t += stride) {
    const int32_t c = coo_c[t];
    if (c >= 0) atomicAdd(&cnt[c], 1);
  }
}

__global__ void __launch_bounds__(1024) csc_scan_kernel(const int32_t* __restrict__ cnt, int64_t cols, int32_t* __restrict__ ptr) {
  __shared__ int32_t part[1024];
  const int t = threadIdx.x;
  const int64_t chunk = (cols + 1023) / 1024;
  const int64_t lo = t * chunk < cols ? t * chunk : cols, hi = lo + chunk < cols ? lo + chunk : cols;
  int32_t s = 0;
  for (int64_t d = lo; d < hi; ++d) s += (cnt[d] + 1) & ~1;
  part[t] = s;
  __syncthreads();
  for (int o = 1; o < 1024; o <<= 1) {             // inclusive scan of the 1024 chunk sums
    const int32_t v = t >= o ? part[t - o] : 0;
    __syncthreads();
    part[t] += v;
    __syncthreads();
  }
  int32_t run = t > 0 ? part[t - 1] : 0;
  for (int64_t d = lo; d < hi; ++d) {
    ptr[d] = run;
    run += (cnt[d] + 1) & ~1;
  }
  if (t == 1023) ptr[cols] = part[1023];
}

__global__ void __launch_bounds__(256) csc_fill_kernel(const int32_t* __restrict__ coo_i, const int32_t* __restrict__ coo_c,
                                                       const float* __restrict__ coo_x, int64_t nnz,
                                                       const int32_t* __restrict__ ptr, int32_t* __restrict__ cur,
                                                       int2* __restrict__ tmp) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t t = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; t < nnz; t += stride) {
    const int32_t c = coo_c[t];
    if (c < 0) continue;
    const int32_t pos = ptr[c] + atomicAdd(&cur[c], 1);
    tmp[pos] = make_int2(coo_i[t], __float_as_int(coo_x[t]));
  }
}

// One block per column (grid-stride): rank of every entry among the column's entries by sample index.
__global__ void __launch_bounds__(128) csc_sort_kernel(const int2* __restrict__ tmp, const int32_t* __restrict__ ptr,
                                                       const int32_t* __restrict__ cnt, int64_t cols, int32_t K,
                                                       int2* __restrict__ ent) {
  for (int64_t d = blockIdx.x; d < cols; d += gridDim.x) {
    const int32_t n = cnt[d], b = ptr[d];
    for (int32_t e = threadIdx.x; e < n; e += blockDim.x) {
      const int2 me = tmp[b + e];
      int32_t rank = 0;
      for (int32_t f = 0; f < n; ++f) {
        const int32_t o = tmp[b + f].x;
        rank += (o < me.x || (o == me.x && f < e)) ? 1 : 0;
      }
      ent[b + rank] = me;
    }
    if (threadIdx.x == 0 && (n & 1)) ent[b + n] = make_int2(K, 0);
  }
}

// ---------------------------------------------------------------------------------------------------------
// Row-wise forward product for sparse samples in the fp32 FMA mode:  z_ij = sum_t x_it W[j][c_it]  (Section 2.1: the
// logits W a_i), the sparse counterpart of the FFMA product (the tensor-core modes keep their dense product over the
// scattered samples, which is faster than any gather).  A block holds RB whole rows of W in shared memory; a warp takes
// one sample at a time with its lanes as RB rows x 32/RB entries: each lane multiplies every (32/RB)-th entry of the
// sample with its row's value at that column, the partial sums of a row are added by shuffles.  The entries of a
// sample come through a small per-warp buffer in shared memory, filled by asynchronous copies two samples ahead.  Sums
// are in a fixed order.
// ---------------------------------------------------------------------------------------------------------
constexpr int kSfWarps = 16;
constexpr int kSfThreads = kSfWarps * 32;
constexpr int kSfChunk = 128;                        // entries of a sample staged at once (a warp's buffer: 1 KB)
constexpr int kSfBufs = 3;                           // the samples one and two ahead are in flight

__device__ __forceinline__ void cp_async_8(uint32_t dst, const void* src, bool valid) {
  const uint32_t n = valid ? 8u : 0u;                // 0: nothing is read, the 8 bytes are filled with zeros
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ int2 lds_v2(uint32_t a) {
  int2 v;
  asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}

// The first kSfChunk entries [b, e) of a sample into a warp's buffer, zeros after the last one.
__device__ __forceinline__ void stage_entries(uint32_t buf, const int2* __restrict__ cx, int32_t b, int32_t e, int lane) {
#pragma unroll
  for (int k = 0; k < kSfChunk / 32; ++k) {
    const int32_t t = b + k * 32 + lane;
    cp_async_8(buf + static_cast<uint32_t>(k * 32 + lane) * 8u, cx + (t < e ? t : b), t < e);
  }
  cp_async_commit();
}

template <int RB>
__global__ void __launch_bounds__(kSfThreads, 1) sparse_forward_kernel(const float* __restrict__ W, int64_t rows, int64_t cols,
                                                                       int32_t pitch, const int32_t* __restrict__ row_beg,
                                                                       const int32_t* __restrict__ row_end,
                                                                       const int2* __restrict__ cx, int64_t off, int32_t n,
                                                                       float* __restrict__ Z, int64_t ldz) {
  extern __shared__ __align__(16) uint8_t sf_smem[];
  constexpr int EP = 32 / RB;                        // entries of a sample worked on at once
  float* ws = reinterpret_cast<float*>(sf_smem);     // RB rows of W, row pitch `pitch` floats
  int2* ranges = reinterpret_cast<int2*>(ws + static_cast<size_t>(RB) * pitch);   // (begin, end) of the n samples
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane % RB, e = lane / RB;
  const uint32_t ebuf = shared_addr(ranges + n) + static_cast<uint32_t>(warp) * (kSfBufs * kSfChunk * 8);
  for (int s = threadIdx.x; s < n; s += kSfThreads) ranges[s] = make_int2(row_beg[off + s], row_end[off + s]);
  const uint32_t wrow = shared_addr(ws) + static_cast<uint32_t>(r) * pitch * 4u;
  const int64_t nblk = (rows + RB - 1) / RB;
  const int quads = static_cast<int>(cols / 4);

  for (int64_t blk = blockIdx.x; blk < nblk; blk += gridDim.x) {
    const int64_t j0 = blk * RB;
    __syncthreads();                                 // every warp is done with the previous rows (and ranges is filled)
    for (int q = threadIdx.x; q < RB * quads; q += kSfThreads) {
      const int rr = q / quads, cc = (q - rr * quads) * 4;
      const float4 v = j0 + rr < rows ? *reinterpret_cast<const float4*>(W + (j0 + rr) * cols + cc)
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
      *reinterpret_cast<float4*>(ws + static_cast<size_t>(rr) * pitch + cc) = v;
    }
    __syncthreads();

    // samples warp, warp + 16, ...: buffer (it % 3) holds the entries of the it-th of them
    int2 rg = warp < n ? ranges[warp] : make_int2(0, 0);
    stage_entries(ebuf, cx, rg.x, rg.y, lane);
    {
      const int2 r1 = warp + kSfWarps < n ? ranges[warp + kSfWarps] : make_int2(0, 0);
      stage_entries(ebuf + kSfChunk * 8, cx, r1.x, r1.y, lane);
    }
    int it = 0;
    for (int s = warp; s < n; s += kSfWarps, ++it) {
      {
        const int2 r2 = s + 2 * kSfWarps < n ? ranges[s + 2 * kSfWarps] : make_int2(0, 0);
        stage_entries(ebuf + static_cast<uint32_t>((it + 2) % kSfBufs) * (kSfChunk * 8), cx, r2.x, r2.y, lane);
      }
      cp_async_wait<2>();                            // all but the two newest groups: this sample's entries are in
      __syncwarp();
      const uint32_t q0 = ebuf + static_cast<uint32_t>(it % kSfBufs) * (kSfChunk * 8) + static_cast<uint32_t>(e) * 8u;
      const int32_t len = rg.y - rg.x;
      const int32_t cnt = len < kSfChunk ? len : kSfChunk;
      float acc = 0.f;
      uint32_t q = q0;
      int32_t m = 0;
      for (; m + 4 * EP <= cnt; m += 4 * EP, q += 4 * EP * 8) {
        const int2 a0 = lds_v2(q), a1 = lds_v2(q + EP * 8), a2 = lds_v2(q + 2 * EP * 8), a3 = lds_v2(q + 3 * EP * 8);
        const float w0 = lds_f32(wrow + static_cast<uint32_t>(a0.x) * 4u), w1 = lds_f32(wrow + static_cast<uint32_t>(a1.x) * 4u);
        const float w2 = lds_f32(wrow + static_cast<uint32_t>(a2.x) * 4u), w3 = lds_f32(wrow + static_cast<uint32_t>(a3.x) * 4u);
        acc = fmaf(__int_as_float(a0.y), w0, acc); acc = fmaf(__int_as_float(a1.y), w1, acc);
        acc = fmaf(__int_as_float(a2.y), w2, acc); acc = fmaf(__int_as_float(a3.y), w3, acc);
      }
      for (; m < cnt; m += EP, q += EP * 8) {       // the rest: groups of EP entries, zeros after the last entry
        const int2 a0 = lds_v2(q);
        acc = fmaf(__int_as_float(a0.y), lds_f32(wrow + static_cast<uint32_t>(a0.x) * 4u), acc);
      }
      for (int32_t t = rg.x + kSfChunk + e; t < rg.y; t += EP) {     // a sample of more than kSfChunk entries: the rest
        const int2 a0 = __ldg(cx + t);
        acc = fmaf(__int_as_float(a0.y), lds_f32(wrow + static_cast<uint32_t>(a0.x) * 4u), acc);
      }
#pragma unroll
      for (int o = RB; o < 32; o <<= 1) acc += __shfl_xor_sync(kFull, acc, o);
      if (e == 0 && j0 + r < rows) Z[(off + s) * ldz + j0 + r] = acc;
      __syncwarp();                                  // the buffer may be refilled two iterations from now
      rg = s + kSfWarps < n ? ranges[s + kSfWarps] : make_int2(0, 0);
    }
    cp_async_wait<0>();
  }
}

// ---------------------------------------------------------------------------------------------------------
// The update.  A block owns 32 rows of W at a time and keeps their factor slab u[i][row] (all K samples) in shared
// memory; its warps take 32-column blocks of those rows.  Within a block of 32 x 32 entries a lane first is a ROW:
// for each of the 32 columns it sums x_id * u[i][row] over the column's entries (the entries are read by all lanes at
// once, the slab row by row without bank conflicts).  The 32 x 32 sums are then transposed through shared memory so
// that a lane is a COLUMN and each row's 32 entries of W leave as one 128-byte piece.
//   USRC 0: factors fp32, sample-major [K x ldu] (fp32 modes);  1: bf16, transposed [rows x ldut] (bf16 mode, whose
//           label entries are applied separately in fp32).
//   SHADOW 0: none;  1: bf16 operand copy of W, a 64-byte row piece rewritten only if one of its roundings changed;
//           2: the (big | small) tf32 copy.
// ---------------------------------------------------------------------------------------------------------
struct SuParams {
  float* W;
  int64_t rows, cols;
  const int32_t* ptr;
  const int2* ent;
  const float* U;
  int64_t ldu;
  const __nv_bfloat16* UT;
  int64_t ldut;
  int32_t K;
  float alpha;
  int32_t prox_kind;
  float prox_a;
  __nv_bfloat16* shadow;
  int64_t shadow_ld;
  float* shadow32;
  int64_t shadow32_ld, shadow_half;
  unsigned long long* copy_counters;
};

template <int USRC>
struct Slab {
  static constexpr int kPitch = USRC == 0 ? 33 * 4 : 34 * 2;      // bytes per sample: 32 rows, padded to an odd word count
  // base: shared address of this lane's row in sample 0
  static __device__ __forceinline__ float load(uint32_t base, int32_t i) {
    if (USRC == 0) return lds_f32(base + i * kPitch);
    return __uint_as_float(lds_u16(base + i * kPitch) << 16);
  }
};

__device__ __forceinline__ float tf32_round(float x) {
  uint32_t u;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
  return __uint_as_float(u);
}

template <int USRC, int SHADOW, bool PROX>
__global__ void __launch_bounds__(kSuThreads, 1) sparse_update_kernel(const SuParams p) {
  extern __shared__ __align__(16) uint8_t su_smem[];
  __shared__ int next_cb;
  using S = Slab<USRC>;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* us = su_smem;
  const int slab_bytes = ((p.K + 1) * S::kPitch + 15) & ~15;
  float* stg = reinterpret_cast<float*>(su_smem + slab_bytes + warp * kSuWarpBytes);
  int2* ebuf = reinterpret_cast<int2*>(stg + kSuStage);
  const uint32_t ebuf_s = shared_addr(ebuf);
  const uint32_t stg_s = shared_addr(stg) + lane * 4;                      // this lane's row of column 0 of the sums
  const uint32_t us_s = shared_addr(us) + lane * (USRC == 0 ? 4 : 2);     // this lane's row of sample 0
  const int nrb = static_cast<int>((p.rows + 31) / 32), ncb = static_cast<int>((p.cols + 31) / 32);
  // second role of a lane, for the pass over W: 8 lanes x 4 columns cover a row's 32 columns, 4 rows per step
  const int sub = lane >> 3, jj = lane & 7;
  // sample K of the slab is all zero: the padding entries of odd columns point there
  for (int t = threadIdx.x; t < S::kPitch / 2; t += kSuThreads) reinterpret_cast<uint16_t*>(us + p.K * S::kPitch)[t] = 0;
  unsigned long long pieces = 0, written = 0;

  for (int rb = blockIdx.x; rb < nrb; rb += gridDim.x) {
    const int64_t r0 = static_cast<int64_t>(rb) * 32;
    const int nrows = p.rows - r0 < 32 ? static_cast<int>(p.rows - r0) : 32;
    __syncthreads();                                   // every warp is done with the previous slab
    if (USRC == 0) {
      const bool rv = lane < nrows;
#pragma unroll 8
      for (int i = warp; i < p.K; i += kSuWarps)
        *reinterpret_cast<float*>(us + i * S::kPitch + lane * 4) = rv ? p.U[static_cast<int64_t>(i) * p.ldu + r0 + lane] : 0.f;
    } else {
      for (int r = warp; r < 32; r += kSuWarps) {
        const bool rv = r < nrows;
        const uint16_t* src = reinterpret_cast<const uint16_t*>(p.UT) + (r0 + r) * p.ldut;
#pragma unroll 8
        for (int i = lane; i < p.K; i += 32)
          *reinterpret_cast<uint16_t*>(us + i * S::kPitch + r * 2) = rv ? src[i] : static_cast<uint16_t>(0);
      }
    }
    if (threadIdx.x == 0) next_cb = 0;
    __syncthreads();

    for (;;) {
      int cb = 0;
      if (lane == 0) cb = atomicAdd(&next_cb, 1);       // which warp takes which block does not change any result
      cb = __shfl_sync(kFull, cb, 0);
      if (cb >= ncb) break;
      // the block's 32 x 32 entries of W, asked for before the sums so that they arrive meanwhile
      const int64_t dq = static_cast<int64_t>(cb) * 32 + 4 * jj;        // cols is a multiple of 4: a quad is in or out
      const bool qv = dq < p.cols;
      float4 wv[8];
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int r = 4 * it + sub;
        wv[it] = (qv && r < nrows) ? *reinterpret_cast<const float4*>(p.W + (r0 + r) * p.cols + dq)
                                   : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      // first role of a lane: a ROW.  The sum over the entries of each of the 32 columns goes to the warp's 32 x 32
      // buffer (column-major with an odd pitch: conflict-free both ways).  The entries of the block are contiguous
      // (column after column); a window of kSuChunk of them is staged in a second small buffer and moved on when a
      // column runs past its end (one trip to L2 per window).  The column loop is deliberately not unrolled: sixteen
      // warps at sixteen places of a long unrolled body starve on instruction fetch.
      const int64_t d = static_cast<int64_t>(cb) * 32 + lane;
      const int32_t pb = p.ptr[d < p.cols ? d : p.cols], pe = p.ptr[d + 1 < p.cols ? d + 1 : p.cols];
      const int32_t len = pe - pb;
      const int32_t E1 = __shfl_sync(kFull, pe, 31);
      int32_t b = __shfl_sync(kFull, pb, 0);                       // running entry index
      int32_t wlo = 0, whi = 0;                                    // staged window of entries [wlo, whi)
      uint32_t sacc = stg_s;
#pragma unroll 1
      for (int c = 0; c < 32; ++c, sacc += 33 * 4) {
        int32_t left = __shfl_sync(kFull, len, c);
        float a = 0.f;
        while (left > 0) {
          if (b >= whi) {
            __syncwarp();                                          // every lane is done with the old window
            wlo = b;
            whi = b + kSuChunk < E1 ? b + kSuChunk : E1;
            for (int32_t t = wlo + 2 * lane; t < whi; t += 64)
              *reinterpret_cast<int4*>(ebuf + (t - wlo)) = __ldg(reinterpret_cast<const int4*>(p.ent + t));
            __syncwarp();
          }
          int32_t n = left < whi - b ? left : whi - b;
          uint32_t q = ebuf_s + static_cast<uint32_t>(b - wlo) * 8u;
          b += n;
          left -= n;
          for (; n >= 8; n -= 8, q += 64) {
            const int4 t0 = lds_v4(q), t1 = lds_v4(q + 16), t2 = lds_v4(q + 32), t3 = lds_v4(q + 48);
            const float u0 = S::load(us_s, t0.x), u1 = S::load(us_s, t0.z);
            const float u2 = S::load(us_s, t1.x), u3 = S::load(us_s, t1.z);
            const float u4 = S::load(us_s, t2.x), u5 = S::load(us_s, t2.z);
            const float u6 = S::load(us_s, t3.x), u7 = S::load(us_s, t3.z);
            a = fmaf(__int_as_float(t0.y), u0, a); a = fmaf(__int_as_float(t0.w), u1, a);
            a = fmaf(__int_as_float(t1.y), u2, a); a = fmaf(__int_as_float(t1.w), u3, a);
            a = fmaf(__int_as_float(t2.y), u4, a); a = fmaf(__int_as_float(t2.w), u5, a);
            a = fmaf(__int_as_float(t3.y), u6, a); a = fmaf(__int_as_float(t3.w), u7, a);
          }
          if (n >= 4) {
            const int4 t0 = lds_v4(q), t1 = lds_v4(q + 16);
            const float u0 = S::load(us_s, t0.x), u1 = S::load(us_s, t0.z);
            const float u2 = S::load(us_s, t1.x), u3 = S::load(us_s, t1.z);
            a = fmaf(__int_as_float(t0.y), u0, a); a = fmaf(__int_as_float(t0.w), u1, a);
            a = fmaf(__int_as_float(t1.y), u2, a); a = fmaf(__int_as_float(t1.w), u3, a);
            n -= 4; q += 32;
          }
          if (n >= 2) {
            const int4 t0 = lds_v4(q);
            const float u0 = S::load(us_s, t0.x), u1 = S::load(us_s, t0.z);
            a = fmaf(__int_as_float(t0.y), u0, a); a = fmaf(__int_as_float(t0.w), u1, a);
          }
        }
        sts_f32(sacc, a);
      }
      __syncwarp();                                    // all sums are in the buffer
      // second role: the pass over W, 4 rows of 32 columns per step, every lane a quad of columns
      if (SHADOW == 1 && lane == 0) pieces += nrows;
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int r = 4 * it + sub;
        const bool ok = qv && r < nrows;
        const float4 wo = wv[it];
        const float* sp = stg + (4 * jj) * 33 + r;
        float4 wn = make_float4(fmaf(p.alpha, sp[0], wo.x), fmaf(p.alpha, sp[33], wo.y), fmaf(p.alpha, sp[66], wo.z),
                                fmaf(p.alpha, sp[99], wo.w));
        if (PROX) {
          wn.x = prox_entry(wn.x, p.prox_kind, p.prox_a); wn.y = prox_entry(wn.y, p.prox_kind, p.prox_a);
          wn.z = prox_entry(wn.z, p.prox_kind, p.prox_a); wn.w = prox_entry(wn.w, p.prox_kind, p.prox_a);
        }
        if (ok) *reinterpret_cast<float4*>(p.W + (r0 + r) * p.cols + dq) = wn;
        if (SHADOW == 1) {
          const uint32_t o01 = pack_bf16x2(wo.x, wo.y), o23 = pack_bf16x2(wo.z, wo.w);
          const uint32_t n01 = pack_bf16x2(wn.x, wn.y), n23 = pack_bf16x2(wn.z, wn.w);
          const unsigned bal = __ballot_sync(kFull, ok && (o01 != n01 || o23 != n23));
          if ((bal >> (8 * sub)) & 0xffu) {             // this row's 64-byte piece changes: rewrite it
            if (jj == 0) ++written;
            if (ok) *reinterpret_cast<uint2*>(p.shadow + (r0 + r) * p.shadow_ld + dq) = make_uint2(n01, n23);
          }
        }
        if (SHADOW == 2 && ok) {
          const float4 big = make_float4(tf32_round(wn.x), tf32_round(wn.y), tf32_round(wn.z), tf32_round(wn.w));
          float* s32 = p.shadow32 + (r0 + r) * p.shadow32_ld + dq;
          *reinterpret_cast<float4*>(s32) = big;
          *reinterpret_cast<float4*>(s32 + p.shadow_half) =
              make_float4(tf32_round(wn.x - big.x), tf32_round(wn.y - big.y), tf32_round(wn.z - big.z), tf32_round(wn.w - big.w));
        }
      }
      __syncwarp();                                    // the buffer of sums is free again
    }
  }
  if (SHADOW == 1 && p.copy_counters) {
    if (lane == 0) atomicAdd(p.copy_counters, pieces);
    if (jj == 0 && written) atomicAdd(p.copy_counters + 1, written);
  }
}

template <int USRC, int SHADOW, bool PROX>
cudaError_t launch_sparse_update_k(cudaStream_t s, const SuParams& p, int smem) {
  static std::atomic<uint64_t> prepared{0};            // one bit per device ordinal
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const uint64_t bit = 1ull << (dev & 63);
  if (!(prepared.load(std::memory_order_acquire) & bit)) {
    e = cudaFuncSetAttribute(sparse_update_kernel<USRC, SHADOW, PROX>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemOptIn);
    if (e != cudaSuccess) return e;
    prepared.fetch_or(bit, std::memory_order_release);
  }
  const int nrb = static_cast<int>((p.rows + 31) / 32);
  sparse_update_kernel<USRC, SHADOW, PROX><<<std::min(nrb, sm_count()), kSuThreads, smem, s>>>(p);
  count_launch();
  return cudaGetLastError();
}

template <int USRC, int SHADOW>
cudaError_t launch_sparse_update(cudaStream_t s, const SuParams& p, int smem) {
  return p.prox_kind != 0 ? launch_sparse_update_k<USRC, SHADOW, true>(s, p, smem)
                          : launch_sparse_update_k<USRC, SHADOW, false>(s, p, smem);
}

int slab_smem(int64_t K, bool bf16) {
  const int64_t pitch = bf16 ? 34 * 2 : 33 * 4;
  const int64_t bytes = (((K + 1) * pitch + 15) & ~int64_t(15)) + static_cast<int64_t>(kSuWarps) * kSuWarpBytes;
  return bytes <= kSmemOptIn ? static_cast<int>(bytes) : -1;
}

}  // namespace

#define CKS(call)                                       \
  do {                                                  \
    cudaError_t e__ = (call);                           \
    if (e__ != cudaSuccess) {                           \
      ctx->last_cuda = static_cast<int>(e__);           \
      return SFB_ERR_CUDA;                              \
    }                                                   \
  } while (0)

void sparse_extend_layout(const sfb_config& c, Layout& L, size_t& off) {
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + kAlign - 1) / kAlign * kAlign; return o; };
  const size_t nnz = static_cast<size_t>(c.csr_nnz_max), cols = static_cast<size_t>(c.cols);
  L.coo_i = take(nnz * 4);
  L.coo_c = take(nnz * 4);
  L.coo_x = take(nnz * 4);
  L.coo_cx = take((nnz + 128) * 8);
  L.row_beg = take(static_cast<size_t>(c.workers) * c.batch * 4);
  L.row_end = take(static_cast<size_t>(c.workers) * c.batch * 4);
  L.csc_cnt = take((cols + 1) * 4);
  L.csc_cur = take((cols + 1) * 4);
  L.csc_ptr = take((cols + 1) * 4);
  L.csc_tmp = take((nnz + cols) * 8);
  L.csc_ent = take((nnz + cols + 8) * 8);
}

// Cost model, in time per entry of W relative to the dense update of K = 1024 pairs in bf16 (measured at 325,000 x
// 10,000 on one B200: 8.5 ms): the sparse update costs a fixed 0.83 for its pass over W (1.57 in the tensor-core fp32
// mode, whose 8-byte operand copy it also writes) plus 0.089 per non-zero of an average column; the dense update
// costs K/1024 in bf16 mode, 4.4 K/1024 with tf32 pairs, and far more on the FMA kernels.
bool sparse_update_wanted(const sfb_ctx* ctx) {
  const sfb_config& c = ctx->cfg;
  const bool bf16 = c.precision == SFB_PREC_BF16;
  if (c.csr_update == 2 || slab_smem(ctx->K, bf16) < 0) return false;
  if (c.csr_update == 1 || (!bf16 && !ctx->tf32)) return true;
  const double per_col = static_cast<double>(ctx->csr_fill) / static_cast<double>(c.cols);
  const double k = static_cast<double>(ctx->K) / 1024.0;
  const double sparse = (bf16 ? 0.83 : 1.57) + 0.089 * per_col;
  return sparse < (bf16 ? 1.0 : 4.4) * k;
}

int sparse_stage(sfb_ctx* ctx, int64_t off, int64_t n, const int64_t* indptr, const int32_t* idx, const float* val,
                 int64_t nnz) {
  const Layout& L = ctx->lay;
  const int64_t cols = ctx->cfg.cols;
  cudaStream_t s = ctx->stream;
  float* Xd = ctx->at<float>(L.stageX);
  CKS(cudaMemsetAsync(Xd + off * cols, 0, static_cast<size_t>(n) * cols * 4, s));
  if (nnz > 0) CKS(cudaMemsetAsync(ctx->at<int32_t>(L.coo_c) + ctx->csr_fill, 0xff, static_cast<size_t>(nnz) * 4, s));   // "no entry"
  csr_stage_kernel<<<static_cast<unsigned>((n * 32 + 255) / 256), 256, 0, s>>>(
      indptr, idx, val, n, nnz, cols, off, Xd, ctx->at<int32_t>(L.coo_i) + ctx->csr_fill,
      ctx->at<int32_t>(L.coo_c) + ctx->csr_fill, ctx->at<float>(L.coo_x) + ctx->csr_fill,
      ctx->at<int2>(L.coo_cx) + ctx->csr_fill, static_cast<int32_t>(ctx->csr_fill), ctx->at<int32_t>(L.row_beg),
      ctx->at<int32_t>(L.row_end), ctx->at<uint32_t>(L.status));
  count_launch();
  CKS(cudaGetLastError());
  ctx->last_stage_nnz = nnz;
  return SFB_OK;
}

namespace {

template <int RB>
cudaError_t launch_sparse_forward(sfb_ctx* ctx, int64_t off, int64_t n, float* Z, int64_t ldz, int pitch, int smem) {
  static std::atomic<uint64_t> prepared{0};            // one bit per device ordinal
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const uint64_t bit = 1ull << (dev & 63);
  if (!(prepared.load(std::memory_order_acquire) & bit)) {
    e = cudaFuncSetAttribute(sparse_forward_kernel<RB>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemOptIn);
    if (e != cudaSuccess) return e;
    prepared.fetch_or(bit, std::memory_order_release);
  }
  const Layout& L = ctx->lay;
  const sfb_config& c = ctx->cfg;
  const int64_t nblk = (c.rows + RB - 1) / RB;
  sparse_forward_kernel<RB><<<static_cast<unsigned>(std::min<int64_t>(nblk, sm_count())), kSfThreads, smem, ctx->stream>>>(
      ctx->W, c.rows, c.cols, pitch, ctx->at<int32_t>(L.row_beg), ctx->at<int32_t>(L.row_end), ctx->at<int2>(L.coo_cx), off,
      static_cast<int32_t>(n), Z, ldz);
  count_launch();
  return cudaGetLastError();
}

// Row pitch (floats) of the rows of W in shared memory: at least cols, and congruent to 32/RB modulo 32 so that the RB
// rows of one column fall into different banks.
int forward_pitch(int64_t cols, int rb) {
  const int64_t want = rb == 1 ? 0 : 32 / rb;
  int64_t p = (cols + 31) / 32 * 32 + want;
  return static_cast<int>(p);
}

}  // namespace

// Rows of W a block of the row-wise forward can hold (4, 2 or 1), or 0 when even one row does not fit.
int sparse_forward_rows(const sfb_ctx* ctx, int64_t n) {
  for (int rb = 4; rb >= 1; rb >>= 1) {
    const int64_t bytes = static_cast<int64_t>(rb) * forward_pitch(ctx->cfg.cols, rb) * 4 + n * 8 + kSfWarps * kSfBufs * kSfChunk * 8;
    if (bytes <= kSmemOptIn) return rb;
  }
  return 0;
}

// Z[off .. off+n) = X W^T for the n staged sparse samples at pair offset off (fp32, row pitch ldz).
int sparse_forward(sfb_ctx* ctx, int64_t off, int64_t n, float* Z, int64_t ldz) {
  const int rb = sparse_forward_rows(ctx, n);
  if (rb == 0) return SFB_ERR_SHAPE;
  const int pitch = forward_pitch(ctx->cfg.cols, rb);
  const int smem = static_cast<int>(static_cast<int64_t>(rb) * pitch * 4 + n * 8 + kSfWarps * kSfBufs * kSfChunk * 8);
  if (rb == 4) CKS(launch_sparse_forward<4>(ctx, off, n, Z, ldz, pitch, smem));
  else if (rb == 2) CKS(launch_sparse_forward<2>(ctx, off, n, Z, ldz, pitch, smem));
  else CKS(launch_sparse_forward<1>(ctx, off, n, Z, ldz, pitch, smem));
  ctx->stats.flops += 2.0 * static_cast<double>(ctx->cfg.rows) * static_cast<double>(ctx->last_stage_nnz);
  return SFB_OK;
}

int sparse_build_csc(sfb_ctx* ctx) {
  const Layout& L = ctx->lay;
  const int64_t cols = ctx->cfg.cols, nnz = ctx->csr_fill;
  cudaStream_t s = ctx->stream;
  int32_t* cnt = ctx->at<int32_t>(L.csc_cnt);
  int32_t* cur = ctx->at<int32_t>(L.csc_cur);
  int32_t* ptr = ctx->at<int32_t>(L.csc_ptr);
  CKS(cudaMemsetAsync(cnt, 0, static_cast<size_t>(cols + 1) * 4, s));
  CKS(cudaMemsetAsync(cur, 0, static_cast<size_t>(cols + 1) * 4, s));
  if (nnz > 0) {
    csc_count_kernel<<<grid1d(nnz, 256), 256, 0, s>>>(ctx->at<int32_t>(L.coo_c), nnz, cnt);
    count_launch();
  }
  csc_scan_kernel<<<1, 1024, 0, s>>>(cnt, cols, ptr);
  count_launch();
  if (nnz > 0) {
    csc_fill_kernel<<<grid1d(nnz, 256), 256, 0, s>>>(ctx->at<int32_t>(L.coo_i), ctx->at<int32_t>(L.coo_c), ctx->at<float>(L.coo_x),
                                                     nnz, ptr, cur, ctx->at<int2>(L.csc_tmp));
    count_launch();
    csc_sort_kernel<<<grid1d(cols, 1, 148 * 16), 128, 0, s>>>(ctx->at<int2>(L.csc_tmp), ptr, cnt, cols,
                                                              static_cast<int32_t>(ctx->K), ctx->at<int2>(L.csc_ent));
    count_launch();
  }
  CKS(cudaGetLastError());
  return SFB_OK;
}

// W <- prox(W - step * U^T V) with V in the column-major form built by sparse_build_csc.
int sparse_update(sfb_ctx* ctx) {
  const sfb_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  const bool bf16 = c.precision == SFB_PREC_BF16;
  const int smem = slab_smem(ctx->K, bf16);
  if (smem < 0) return SFB_ERR_SHAPE;
  SuParams p{};
  p.W = ctx->W; p.rows = c.rows; p.cols = c.cols;
  p.ptr = ctx->at<int32_t>(L.csc_ptr);
  p.ent = ctx->at<int2>(L.csc_ent);
  p.K = static_cast<int32_t>(ctx->K);
  p.alpha = -ctx->step;
  p.prox_kind = ctx->prox_kind; p.prox_a = ctx->prox_a;
  if (bf16) {
    p.UT = ctx->at<__nv_bfloat16>(L.UT); p.ldut = L.Kp;
    p.shadow = ctx->at<__nv_bfloat16>(L.Wb); p.shadow_ld = L.colsb;
    p.copy_counters = &ctx->at<Scalars>(L.scalars)->copy_pieces;
    CKS((launch_sparse_update<1, 1>(ctx->stream, p, smem)));
  } else {
    p.U = ctx->at<float>(L.U); p.ldu = c.rows;
    if (ctx->tf32) {
      p.shadow32 = ctx->at<float>(L.Ws); p.shadow32_ld = 2 * L.colsp; p.shadow_half = L.colsp;
      CKS((launch_sparse_update<0, 2>(ctx->stream, p, smem)));
    } else {
      CKS((launch_sparse_update<0, 0>(ctx->stream, p, smem)));
    }
  }
  return SFB_OK;
}

}  // namespace sfb
