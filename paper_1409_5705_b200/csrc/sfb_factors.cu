// Bandwidth-bound kernels of the SFB step in fp32: factor packing, the row softmax of multiclass logistic
// regression, the pair residual of distance metric learning, the column-norm prox of sparse coding and the
// power iteration that estimates the coder's step size.
#include "sfb_internal.h"

namespace sfb {
namespace {

constexpr int kThreads = 256;

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

// Block-wide sum in a fixed order (warp shuffles, then warp 0 over the per-warp values).
template <int NTHREADS>
__device__ __forceinline__ float block_sum(float v, float* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  float r = (threadIdx.x < NTHREADS / 32) ? sh[threadIdx.x] : 0.f;
  if (w == 0) r = warp_sum(r);
  if (threadIdx.x == 0) sh[0] = r;
  __syncthreads();
  return sh[0];
}
template <int NTHREADS>
__device__ __forceinline__ float block_max(float v, float* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  v = warp_max(v);
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  float r = (threadIdx.x < NTHREADS / 32) ? sh[threadIdx.x] : -INFINITY;
  if (w == 0) r = warp_max(r);
  if (threadIdx.x == 0) sh[0] = r;
  __syncthreads();
  return sh[0];
}

// v = x (MLR) or v = x - y (DML pair difference, Section 2), 16-byte vectors with a scalar tail.
__global__ void pack_kernel(float* __restrict__ dst, const float* __restrict__ x, const float* __restrict__ y,
                            int64_t n4, int64_t n) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n4; i += stride) {
    float4 a = reinterpret_cast<const float4*>(x)[i];
    if (y) {
      const float4 b = reinterpret_cast<const float4*>(y)[i];
      a.x -= b.x; a.y -= b.y; a.z -= b.z; a.w -= b.w;
    }
    reinterpret_cast<float4*>(dst)[i] = a;
  }
  for (int64_t i = n4 * 4 + blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n; i += stride)
    dst[i] = y ? x[i] - y[i] : x[i];
}

__global__ void zero_kernel(float* __restrict__ dst, int64_t n) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n; i += stride) dst[i] = 0.f;
}

__global__ void prox_entries_kernel(float* __restrict__ w, int64_t n, int kind, float a) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n; i += stride)
    w[i] = prox_entry(w[i], kind, a);
}

__global__ void axpy_kernel(float* __restrict__ y, const float* __restrict__ x, float alpha, int64_t n) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n; i += stride)
    y[i] = fmaf(alpha, x[i], y[i]);
}

// One block per sample: u = softmax(z) - onehot(y) in place over the sample's row of Z [nsamp x rows]
// (Section 1: u is the prediction vector; Section 2.1: u = d f / d (W a)).  A class id outside [0, rows)
// sets a status bit and subtracts nothing.  loss = log sum exp z - z_y.
template <int NTHREADS>
__global__ void __launch_bounds__(NTHREADS) mlr_softmax_kernel(float* __restrict__ Z, int64_t rows,
                                                               const int32_t* __restrict__ labels,
                                                               float* __restrict__ loss, uint32_t* status) {
  __shared__ float sh[32];
  float* z = Z + static_cast<int64_t>(blockIdx.x) * rows;
  float m = -INFINITY;
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) m = fmaxf(m, z[j]);
  m = block_max<NTHREADS>(m, sh);
  float s = 0.f;
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) s += expf(z[j] - m);
  s = block_sum<NTHREADS>(s, sh);
  const float inv = 1.f / s;
  const int32_t y = labels[blockIdx.x];
  const bool ok = y >= 0 && y < rows;
  if (threadIdx.x == 0) {
    if (!ok) atomicOr(status, SFB_STATUS_LABEL_RANGE);
    loss[blockIdx.x] = ok ? (m + logf(s)) - z[y] : 0.f;
  }
  __syncthreads();
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) {
    float u = expf(z[j] - m) * inv;
    if (ok && j == y) u -= 1.f;
    z[j] = u;
  }
}

// Row-sharded form of the same factor (the parameter matrix partitioned by rows; every shard holds all K samples'
// logits against its own rows only).  First half, one block per sample: the shard's softmax partial
//   part[i] = (m_i, s_i, zy_i, has_i):  m_i = max_j z_ij,  s_i = sum_j exp(z_ij - m_i)  over the shard's rows j,
//   zy_i = z_{i,y_i} and has_i = 1 when class y_i is one of the shard's rows, else 0 and 0.
// labels are global class ids; the shard holds rows [row_off, row_off + rows).
template <int NTHREADS>
__global__ void __launch_bounds__(NTHREADS) mlr_shard_partials_kernel(const float* __restrict__ Z, int64_t rows, int64_t ldz,
                                                                      const int32_t* __restrict__ labels, int64_t row_off,
                                                                      float4* __restrict__ part) {
  __shared__ float sh[32];
  const float* z = Z + static_cast<int64_t>(blockIdx.x) * ldz;
  float m = -INFINITY;
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) m = fmaxf(m, z[j]);
  m = block_max<NTHREADS>(m, sh);
  float s = 0.f;
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) s += expf(z[j] - m);
  s = block_sum<NTHREADS>(s, sh);
  if (threadIdx.x == 0) {
    const int64_t yl = static_cast<int64_t>(labels[blockIdx.x]) - row_off;
    const bool mine = yl >= 0 && yl < rows;
    part[blockIdx.x] = make_float4(m, s, mine ? z[yl] : 0.f, mine ? 1.f : 0.f);
  }
}

// Merge of the shards' partials of one sample, in shard order:  lse = M + log sum_g s_g exp(m_g - M),  M = max_g m_g;
// zy = sum_g zy_g (only the owning shard contributes).  parts is [shards][K].
__device__ __forceinline__ void merge_shard_partials(const float4* __restrict__ parts, int shards, int64_t K, int64_t i,
                                                     float& lse, float& zy, float& has) {
  float M = -INFINITY;
  for (int g = 0; g < shards; ++g) M = fmaxf(M, parts[static_cast<int64_t>(g) * K + i].x);
  float S = 0.f;
  zy = 0.f; has = 0.f;
  for (int g = 0; g < shards; ++g) {
    const float4 v = parts[static_cast<int64_t>(g) * K + i];
    S += v.y * expf(v.x - M);
    zy += v.z;
    has += v.w;
  }
  lse = M + logf(S);
}

// Second half, one block per sample: with the global log-partition, u_ij = exp(z_ij - lse_i) - [j is y_i's row] in
// place over the shard's rows; loss_i = lse_i - z_{i,y_i} (the same on every shard).  A class id that no shard owns
// sets the status bit and subtracts nothing.
template <int NTHREADS>
__global__ void __launch_bounds__(NTHREADS) mlr_shard_finish_kernel(float* __restrict__ Z, int64_t rows, int64_t ldz,
                                                                    const int32_t* __restrict__ labels, int64_t row_off,
                                                                    const float4* __restrict__ parts, int shards, int64_t K,
                                                                    float* __restrict__ loss, uint32_t* status) {
  __shared__ float sh_lse;
  float* z = Z + static_cast<int64_t>(blockIdx.x) * ldz;
  if (threadIdx.x == 0) {
    float lse, zy, has;
    merge_shard_partials(parts, shards, K, blockIdx.x, lse, zy, has);
    const bool ok = has > 0.5f;
    if (!ok) atomicOr(status, SFB_STATUS_LABEL_RANGE);
    loss[blockIdx.x] = ok ? lse - zy : 0.f;
    sh_lse = lse;
  }
  __syncthreads();
  const float lse = sh_lse;
  const int64_t yl = static_cast<int64_t>(labels[blockIdx.x]) - row_off;
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) {
    float u = expf(z[j] - lse);
    if (j == yl) u -= 1.f;
    z[j] = u;
  }
}

// SDCA for l2-regularised multiclass logistic regression (Section 2.1, "Stochastic DCA").  One block per sample:
// the new dual row q minimises  sum_j q_j log q_j - q.(z + kappa q_old) + kappa/2 ||q||^2  over the simplex, kappa =
// ||x||^2 / (lam N).  Stationarity: log q_j + kappa q_j = t_j - nu with t = z + kappa q_old, and nu such that the q_j sum
// to 1; nu lies in [lse(t) - kappa, lse(t)].
// q_j(nu): Newton on y = log q for  y + kappa e^y = c  (increasing and convex in y, so the iteration is monotone from
// the right of the root, where it starts).
__device__ __forceinline__ float sdca_coordinate(float c, float kappa) {
  if (kappa <= 0.f) return expf(c);
  float y = c;                                       // y + kappa e^y - c = kappa e^c >= 0 here: right of the root
  if (c > 0.f) y = fminf(c, logf((c + 1.f) / kappa));
#pragma unroll 1
  for (int it = 0; it < 24; ++it) {
    const float e = kappa * expf(y);
    const float d = (y + e - c) / (1.f + e);
    y -= d;
    if (fabsf(d) <= 1e-7f * fmaxf(1.f, fabsf(y))) break;
  }
  return expf(y);
}

template <int NTHREADS>
__global__ void __launch_bounds__(NTHREADS) sdca_dual_kernel(float* __restrict__ Z, int64_t rows, int64_t ldz,
                                                             const float* __restrict__ X, int64_t cols,
                                                             const int32_t* __restrict__ labels,
                                                             const int32_t* __restrict__ ids, float* __restrict__ Q,
                                                             int64_t n_samples, float inv_lam_n, float gamma,
                                                             float* __restrict__ coef, float* __restrict__ loss,
                                                             uint32_t* status) {
  __shared__ float sh[32];
  const int64_t i = blockIdx.x;
  float* z = Z + i * ldz;
  const int64_t id = ids[i];
  const int32_t y = labels[i];
  const bool ok = id >= 0 && id < n_samples && y >= 0 && y < rows;
  if (!ok) {                                         // uniform over the block: skip the sample, contribute nothing
    if (threadIdx.x == 0) {
      atomicOr(status, (id >= 0 && id < n_samples) ? SFB_STATUS_LABEL_RANGE : SFB_STATUS_SAMPLE_RANGE);
      if (coef) coef[i] = 0.f;
      loss[i] = 0.f;
    }
    for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) z[j] = 0.f;
    return;
  }
  float* q = Q + id * rows;
  const float* x = X + i * cols;
  float ss = 0.f;
  for (int64_t d = threadIdx.x; d < cols; d += NTHREADS) ss = fmaf(x[d], x[d], ss);
  const float kappa = block_sum<NTHREADS>(ss, sh) * inv_lam_n;
  // lse(t) and, for the read-out, lse(z)
  float m = -INFINITY, mz = -INFINITY;
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) {
    m = fmaxf(m, fmaf(kappa, q[j], z[j]));
    mz = fmaxf(mz, z[j]);
  }
  m = block_max<NTHREADS>(m, sh);
  mz = block_max<NTHREADS>(mz, sh);
  float s = 0.f, sz = 0.f;
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) {
    s += expf(fmaf(kappa, q[j], z[j]) - m);
    sz += expf(z[j] - mz);
  }
  s = block_sum<NTHREADS>(s, sh);
  sz = block_sum<NTHREADS>(sz, sh);
  const float lse = m + logf(s);
  if (threadIdx.x == 0) loss[i] = (mz + logf(sz)) - z[y];        // the sample's logistic loss at the W of this step
  // safeguarded Newton on nu: G(nu) = sum_j q_j(nu) is decreasing and convex, G(lse - kappa) >= 1 >= G(lse)
  float lo = lse - kappa, hi = lse, nu = lse;
#pragma unroll 1
  for (int it = 0; it < 12; ++it) {
    float G = 0.f, Dv = 0.f;
    for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) {
      const float qj = sdca_coordinate(fmaf(kappa, q[j], z[j]) - nu, kappa);
      G += qj;
      Dv += qj / fmaf(kappa, qj, 1.f);
    }
    G = block_sum<NTHREADS>(G, sh);
    Dv = block_sum<NTHREADS>(Dv, sh);
    const float g = G - 1.f;
    if (fabsf(g) <= 2e-7f) break;                    // uniform over the block: every thread holds the same sums
    if (g > 0.f) lo = fmaxf(lo, nu); else hi = fminf(hi, nu);
    float next = nu + g / Dv;
    if (!(next > lo && next < hi)) next = 0.5f * (lo + hi);
    nu = next;
  }
  float S = 0.f;
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) S += sdca_coordinate(fmaf(kappa, q[j], z[j]) - nu, kappa);
  S = block_sum<NTHREADS>(S, sh);
  const float invS = 1.f / S;
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) {
    const float qo = q[j];
    const float du = sdca_coordinate(fmaf(kappa, qo, z[j]) - nu, kappa) * invS - qo;      // du = q_new - q_old
    z[j] = du;
    q[j] = fmaf(gamma, du, qo);
    if (coef && j == y) coef[i] = -du;
  }
}

// One block per pair: q = ||z||^2; similar: u = 2z; dissimilar: u = -2z if q < margin else 0 (Section 2, DML).
// Row-sharded form: with norm_out the block only stores its shard's q (after merging Z2) and leaves z as it is; with
// norms_all it takes q as the sum, in shard order, of the shards' values and scales.
template <int NTHREADS>
__global__ void __launch_bounds__(NTHREADS) dml_scale_kernel(float* __restrict__ Z, const float* __restrict__ Z2,
                                                             int64_t rows, int64_t ld,
                                                             const int32_t* __restrict__ similar, float margin,
                                                             float* __restrict__ norm_out, const float* __restrict__ norms_all,
                                                             int shards, int64_t nstride) {
  __shared__ float sh[32];
  float* z = Z + static_cast<int64_t>(blockIdx.x) * ld;
  if (Z2) {                      // z arrives as two partial sums over halves of the contraction (fixed order: Z + Z2)
    const float* z2 = Z2 + static_cast<int64_t>(blockIdx.x) * ld;
    for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) z[j] += z2[j];
    __syncthreads();
  }
  float q = 0.f;
  if (norms_all) {
    for (int g = 0; g < shards; ++g) q += norms_all[g * nstride + blockIdx.x];
  } else {
    for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) q = fmaf(z[j], z[j], q);
    q = block_sum<NTHREADS>(q, sh);
  }
  if (norm_out) {
    if (threadIdx.x == 0) norm_out[blockIdx.x] = q;
    return;
  }
  const float c = similar[blockIdx.x] != 0 ? 2.f : (q < margin ? -2.f : 0.f);
  for (int64_t j = threadIdx.x; j < rows; j += NTHREADS) z[j] = c * z[j];
}

__global__ void mean_kernel(const float* __restrict__ v, int64_t n, float* out) {
  __shared__ float sh[32];
  float s = 0.f;
  for (int64_t i = threadIdx.x; i < n; i += 256) s += v[i];
  s = block_sum<256>(s, sh);
  if (threadIdx.x == 0) *out = s / static_cast<float>(n);
}

// Column reductions over W [rows x cols] in a fixed order: block (slab, column group of 128) sums
// w^2 (MODE 0) or w * yvec[row] (MODE 1) over its row slab into part[slab][col].
template <int MODE>
__global__ void __launch_bounds__(kThreads) col_partial_kernel(const float* __restrict__ W, int64_t rows,
                                                               int64_t cols, const float* __restrict__ yvec,
                                                               float* __restrict__ part, int64_t slab_rows) {
  __shared__ float sh[8][128];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int64_t c0 = static_cast<int64_t>(blockIdx.x) * 128 + tx * 4;
  const int64_t r0 = static_cast<int64_t>(blockIdx.y) * slab_rows;
  const int64_t r1 = min(rows, r0 + slab_rows);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  if (c0 < cols) {                       // cols is a multiple of 4, so a quad is in range as a whole
    for (int64_t r = r0 + ty; r < r1; r += 8) {
      const float4 w = *reinterpret_cast<const float4*>(W + r * cols + c0);
      if (MODE == 0) {
        acc.x = fmaf(w.x, w.x, acc.x); acc.y = fmaf(w.y, w.y, acc.y);
        acc.z = fmaf(w.z, w.z, acc.z); acc.w = fmaf(w.w, w.w, acc.w);
      } else {
        const float yv = yvec[r];
        acc.x = fmaf(w.x, yv, acc.x); acc.y = fmaf(w.y, yv, acc.y);
        acc.z = fmaf(w.z, yv, acc.z); acc.w = fmaf(w.w, yv, acc.w);
      }
    }
  }
  *reinterpret_cast<float4*>(&sh[ty][tx * 4]) = acc;
  __syncthreads();
  if (threadIdx.x < 128) {
    const int64_t c = static_cast<int64_t>(blockIdx.x) * 128 + threadIdx.x;
    if (c < cols) {
      float s = 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) s += sh[k][threadIdx.x];
      part[static_cast<int64_t>(blockIdx.y) * cols + c] = s;
    }
  }
}

// Column sums of squares in fp64 (the prox must resolve norms to far better than fp32's 6e-8, because the
// rescaling multiplies every entry of W while the step's update is ~1e-3 of ||W||).
__global__ void __launch_bounds__(kThreads) col_sumsq_kernel(const float* __restrict__ W, int64_t rows, int64_t cols,
                                                             double* __restrict__ part, int64_t slab_rows) {
  __shared__ double sh[8][128];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int64_t c0 = static_cast<int64_t>(blockIdx.x) * 128 + tx * 4;
  const int64_t r0 = static_cast<int64_t>(blockIdx.y) * slab_rows;
  const int64_t r1 = min(rows, r0 + slab_rows);
  double a0 = 0., a1 = 0., a2 = 0., a3 = 0.;
  if (c0 < cols) {
    for (int64_t r = r0 + ty; r < r1; r += 8) {
      const float4 w = *reinterpret_cast<const float4*>(W + r * cols + c0);
      a0 = fma(static_cast<double>(w.x), static_cast<double>(w.x), a0);
      a1 = fma(static_cast<double>(w.y), static_cast<double>(w.y), a1);
      a2 = fma(static_cast<double>(w.z), static_cast<double>(w.z), a2);
      a3 = fma(static_cast<double>(w.w), static_cast<double>(w.w), a3);
    }
  }
  sh[ty][tx * 4 + 0] = a0; sh[ty][tx * 4 + 1] = a1; sh[ty][tx * 4 + 2] = a2; sh[ty][tx * 4 + 3] = a3;
  __syncthreads();
  if (threadIdx.x < 128) {
    const int64_t c = static_cast<int64_t>(blockIdx.x) * 128 + threadIdx.x;
    if (c < cols) {
      double s = 0.;
#pragma unroll
      for (int k = 0; k < 8; ++k) s += sh[k][threadIdx.x];
      part[static_cast<int64_t>(blockIdx.y) * cols + c] = s;
    }
  }
}

// Prox of Figure 3: b <- b / ||b|| for the columns with ||b|| > 1, others untouched (bit-identical).
__global__ void __launch_bounds__(kThreads) prox_scale_kernel(float* __restrict__ W, int64_t rows, int64_t cols,
                                                              const double* __restrict__ part, int nslabs,
                                                              int64_t slab_rows) {
  __shared__ double scale[128];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  if (threadIdx.x < 128) {
    const int64_t c = static_cast<int64_t>(blockIdx.x) * 128 + threadIdx.x;
    double s = 0.;
    if (c < cols)
      for (int k = 0; k < nslabs; ++k) s += part[static_cast<int64_t>(k) * cols + c];
    scale[threadIdx.x] = s > 1. ? 1. / sqrt(s) : 1.;
  }
  __syncthreads();
  const int64_t c0 = static_cast<int64_t>(blockIdx.x) * 128 + tx * 4;
  if (c0 >= cols) return;
  const double s0 = scale[tx * 4], s1 = scale[tx * 4 + 1], s2 = scale[tx * 4 + 2], s3 = scale[tx * 4 + 3];
  if (s0 == 1. && s1 == 1. && s2 == 1. && s3 == 1.) return;
  const int64_t r0 = static_cast<int64_t>(blockIdx.y) * slab_rows;
  const int64_t r1 = min(rows, r0 + slab_rows);
  for (int64_t r = r0 + ty; r < r1; r += 8) {
    float4* p = reinterpret_cast<float4*>(W + r * cols + c0);
    float4 w = *p;
    if (s0 != 1.) w.x = static_cast<float>(static_cast<double>(w.x) * s0);
    if (s1 != 1.) w.y = static_cast<float>(static_cast<double>(w.y) * s1);
    if (s2 != 1.) w.z = static_cast<float>(static_cast<double>(w.z) * s2);
    if (s3 != 1.) w.w = static_cast<float>(static_cast<double>(w.w) * s3);
    *p = w;
  }
}

// y = W b : one warp per row.
__global__ void __launch_bounds__(kThreads) matvec_rows_kernel(const float* __restrict__ W, int64_t rows,
                                                               int64_t cols, const float* __restrict__ b,
                                                               float* __restrict__ y) {
  const int64_t r = static_cast<int64_t>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
  if (r >= rows) return;
  const int lane = threadIdx.x & 31;
  float s = 0.f;
  for (int64_t c = lane * 4; c < cols; c += 128) {
    const float4 w = *reinterpret_cast<const float4*>(W + r * cols + c);
    const float4 v = *reinterpret_cast<const float4*>(b + c);
    s = fmaf(w.x, v.x, s); s = fmaf(w.y, v.y, s); s = fmaf(w.z, v.z, s); s = fmaf(w.w, v.w, s);
  }
  s = warp_sum(s);
  if (lane == 0) y[r] = s;
}

// One block: c = sum of the slab partials; b = c / ||c||.
__global__ void __launch_bounds__(1024) pi_normalise_kernel(const float* __restrict__ part, int nslabs, int64_t cols,
                                                            float* __restrict__ b) {
  __shared__ float sh[32];
  float ss = 0.f;
  for (int64_t c = threadIdx.x; c < cols; c += 1024) {
    float s = 0.f;
    for (int k = 0; k < nslabs; ++k) s += part[static_cast<int64_t>(k) * cols + c];
    b[c] = s;
    ss = fmaf(s, s, ss);
  }
  ss = block_sum<1024>(ss, sh);
  const float inv = rsqrtf(ss);
  for (int64_t c = threadIdx.x; c < cols; c += 1024) b[c] *= inv;
}

__global__ void __launch_bounds__(1024) pi_init_kernel(float* __restrict__ b, int64_t cols) {
  const float v = rsqrtf(static_cast<float>(cols));
  for (int64_t c = threadIdx.x; c < cols; c += 1024) b[c] = v;
}

// L = ||W b||^2 (Rayleigh quotient of W^T W at the unit vector b).
__global__ void __launch_bounds__(1024) pi_rayleigh_kernel(const float* __restrict__ y, int64_t rows, Scalars* sc) {
  __shared__ float sh[32];
  float ss = 0.f;
  for (int64_t r = threadIdx.x; r < rows; r += 1024) ss = fmaf(y[r], y[r], ss);
  ss = block_sum<1024>(ss, sh);
  if (threadIdx.x == 0) { sc->L = ss; sc->invL = 1.f / ss; }
}

__global__ void set_L_kernel(Scalars* sc, float L) { sc->L = L; sc->invL = 1.f / L; }

inline unsigned grid_for(int64_t n, int per_block) {
  int64_t g = (n + per_block - 1) / per_block;
  if (g < 1) g = 1;
  const int64_t cap = static_cast<int64_t>(sm_count()) * 16;
  return static_cast<unsigned>(g > cap ? cap : g);
}

inline int64_t slab_rows_for(int64_t rows) { return (rows + kProxSlabs - 1) / kProxSlabs; }

}  // namespace

cudaError_t pack_copy(cudaStream_t s, float* dst, const float* x, const float* y, int64_t n) {
  if (n <= 0) return cudaSuccess;
  pack_kernel<<<grid_for(n / 4 + 1, kThreads), kThreads, 0, s>>>(dst, x, y, n / 4, n);
  count_launch();
  return cudaGetLastError();
}

cudaError_t fill_zero(cudaStream_t s, float* dst, int64_t n) {
  if (n <= 0) return cudaSuccess;
  zero_kernel<<<grid_for(n, kThreads), kThreads, 0, s>>>(dst, n);
  count_launch();
  return cudaGetLastError();
}

cudaError_t axpy(cudaStream_t s, float* y, const float* x, float alpha, int64_t n) {
  if (n <= 0) return cudaSuccess;
  axpy_kernel<<<grid_for(n, kThreads), kThreads, 0, s>>>(y, x, alpha, n);
  count_launch();
  return cudaGetLastError();
}

cudaError_t mlr_softmax_rows(cudaStream_t s, float* Z, int64_t nsamp, int64_t rows, const int32_t* labels,
                             float* loss, uint32_t* status) {
  if (nsamp <= 0) return cudaSuccess;
  mlr_softmax_kernel<512><<<static_cast<unsigned>(nsamp), 512, 0, s>>>(Z, rows, labels, loss, status);
  count_launch();
  return cudaGetLastError();
}

cudaError_t prox_entries(cudaStream_t s, float* w, int64_t n, int kind, float a) {
  if (n <= 0 || kind == 0) return cudaSuccess;
  prox_entries_kernel<<<grid_for(n, kThreads), kThreads, 0, s>>>(w, n, kind, a);
  count_launch();
  return cudaGetLastError();
}

cudaError_t mlr_shard_partials(cudaStream_t s, const float* Z, int64_t nsamp, int64_t rows, int64_t ldz,
                               const int32_t* labels, int64_t row_off, float* part) {
  if (nsamp <= 0) return cudaSuccess;
  mlr_shard_partials_kernel<512><<<static_cast<unsigned>(nsamp), 512, 0, s>>>(Z, rows, ldz, labels, row_off,
                                                                           reinterpret_cast<float4*>(part));
  count_launch();
  return cudaGetLastError();
}

cudaError_t mlr_shard_finish(cudaStream_t s, float* Z, int64_t nsamp, int64_t rows, int64_t ldz, const int32_t* labels,
                             int64_t row_off, const float* parts, int shards, float* loss, uint32_t* status) {
  if (nsamp <= 0) return cudaSuccess;
  mlr_shard_finish_kernel<512><<<static_cast<unsigned>(nsamp), 512, 0, s>>>(
      Z, rows, ldz, labels, row_off, reinterpret_cast<const float4*>(parts), shards, nsamp, loss, status);
  count_launch();
  return cudaGetLastError();
}

cudaError_t sdca_dual_rows(cudaStream_t s, float* Z, int64_t nsamp, int64_t rows, int64_t ldz, const float* X, int64_t cols,
                           const int32_t* labels, const int32_t* ids, float* Q, int64_t n_samples, float inv_lam_n,
                           float gamma, float* coef, float* loss, uint32_t* status) {
  if (nsamp <= 0) return cudaSuccess;
  sdca_dual_kernel<512><<<static_cast<unsigned>(nsamp), 512, 0, s>>>(Z, rows, ldz, X, cols, labels, ids, Q, n_samples,
                                                                  inv_lam_n, gamma, coef, loss, status);
  count_launch();
  return cudaGetLastError();
}

cudaError_t dml_scale_rows(cudaStream_t s, float* Z, int64_t nsamp, int64_t rows, int64_t ld,
                           const int32_t* similar, float margin, const float* Z2, float* norm_out, const float* norms_all,
                           int shards, int64_t nstride) {
  if (nsamp <= 0) return cudaSuccess;
  dml_scale_kernel<256><<<static_cast<unsigned>(nsamp), 256, 0, s>>>(Z, Z2, rows, ld, similar, margin, norm_out, norms_all,
                                                                     shards, nstride);
  count_launch();
  return cudaGetLastError();
}

cudaError_t mean_of(cudaStream_t s, const float* v, int64_t n, float* out) {
  mean_kernel<<<1, 256, 0, s>>>(v, n, out);
  count_launch();
  return cudaGetLastError();
}

cudaError_t prox_unit_columns(cudaStream_t s, float* W, int64_t rows, int64_t cols, float* colpart) {
  const int64_t sr = slab_rows_for(rows);
  dim3 grid(static_cast<unsigned>((cols + 127) / 128), kProxSlabs);
  double* part = reinterpret_cast<double*>(colpart);
  col_sumsq_kernel<<<grid, kThreads, 0, s>>>(W, rows, cols, part, sr);
  count_launch();
  prox_scale_kernel<<<grid, kThreads, 0, s>>>(W, rows, cols, part, kProxSlabs, sr);
  count_launch();
  return cudaGetLastError();
}

cudaError_t estimate_lipschitz(cudaStream_t s, const float* W, int64_t rows, int64_t cols, float* b, float* y,
                               float* colpart, Scalars* sc, int iters) {
  const int64_t sr = slab_rows_for(rows);
  dim3 cgrid(static_cast<unsigned>((cols + 127) / 128), kProxSlabs);
  const unsigned rgrid = static_cast<unsigned>((rows + kThreads / 32 - 1) / (kThreads / 32));
  pi_init_kernel<<<1, 1024, 0, s>>>(b, cols);
  count_launch();
  for (int it = 0; it < iters; ++it) {
    matvec_rows_kernel<<<rgrid, kThreads, 0, s>>>(W, rows, cols, b, y);
    count_launch();
    col_partial_kernel<1><<<cgrid, kThreads, 0, s>>>(W, rows, cols, y, colpart, sr);
    count_launch();
    pi_normalise_kernel<<<1, 1024, 0, s>>>(colpart, kProxSlabs, cols, b);
    count_launch();
  }
  matvec_rows_kernel<<<rgrid, kThreads, 0, s>>>(W, rows, cols, b, y);
  count_launch();
  pi_rayleigh_kernel<<<1, 1024, 0, s>>>(y, rows, sc);
  count_launch();
  return cudaGetLastError();
}

cudaError_t set_lipschitz(cudaStream_t s, Scalars* sc, float L) {
  set_L_kernel<<<1, 1, 0, s>>>(sc, L);
  count_launch();
  return cudaGetLastError();
}

}  // namespace sfb

// ---------------------------------------------------------------------------------------------------------
// Column prox without any allocation (sfb_prox_columns_noalloc in sfb.h)
// ---------------------------------------------------------------------------------------------------------
#include <mutex>

namespace {

constexpr int64_t kNoAllocMaxCols = SFB_NOALLOC_MAX_COLS;
constexpr int kNoAllocMaxDevices = 64;

// Per-slab column sums of squares of the no-allocation prox: kProxSlabs x kNoAllocMaxCols doubles (8 MB), resident
// on every device that loads the library until the process exits.  Shared by all calls.
static __device__ __align__(256) double g_noalloc_colpart[static_cast<size_t>(sfb::kProxSlabs) * kNoAllocMaxCols];

std::mutex g_noalloc_mutex;
double* g_noalloc_ptr[kNoAllocMaxDevices] = {};   // device address of the array above, per device ordinal

// The array's name is only a handle on the host; the address a kernel can use comes from the runtime, and it
// differs per device.  Looked up once per device, with that device current.
cudaError_t noalloc_scratch(double** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kNoAllocMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (g_noalloc_ptr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_colpart);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[dev] = static_cast<double*>(p);
  }
  *out = g_noalloc_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int sfb_prox_columns_noalloc(float* W_dev, int64_t rows, int64_t cols, void* stream) {
  if (!W_dev || rows <= 0 || cols <= 0) return SFB_ERR_ARG;
  if ((reinterpret_cast<uintptr_t>(W_dev) & 15u) != 0) return SFB_ERR_ALIGN;
  if (cols % 4 != 0 || rows > (1LL << 30)) return SFB_ERR_SHAPE;
  if (cols > kNoAllocMaxCols) return SFB_ERR_STATIC_LIMIT;
  // The scratch array looked up below belongs to the current device: W must live there too.
  {
    int dev = -1;
    cudaPointerAttributes attr{};
    if (cudaGetDevice(&dev) != cudaSuccess) return SFB_ERR_CUDA;
    if (cudaPointerGetAttributes(&attr, W_dev) != cudaSuccess) { cudaGetLastError(); return SFB_ERR_ARG; }
    if (attr.type != cudaMemoryTypeDevice || attr.device != dev) return SFB_ERR_ARG;
  }
  double* part = nullptr;
  if (noalloc_scratch(&part) != cudaSuccess) return SFB_ERR_CUDA;
  // Every partial that the second kernel reads is written by the first one in this call, so nothing has to start
  // at zero and what an earlier call left in the array does not matter.
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t sr = sfb::slab_rows_for(rows);
  dim3 grid(static_cast<unsigned>((cols + 127) / 128), sfb::kProxSlabs);
  sfb::col_sumsq_kernel<<<grid, sfb::kThreads, 0, s>>>(W_dev, rows, cols, part, sr);
  sfb::count_launch();
  sfb::prox_scale_kernel<<<grid, sfb::kThreads, 0, s>>>(W_dev, rows, cols, part, sfb::kProxSlabs, sr);
  sfb::count_launch();
  return cudaGetLastError() == cudaSuccess ? SFB_OK : SFB_ERR_CUDA;
}
