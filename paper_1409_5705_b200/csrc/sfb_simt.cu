// fp32 FMA matrix products for the fp32-operand mode of the SFB step:
//   forward  z_i = W v_i            (Section 2: the matrix-vector product W a_i, batched over the K samples)
//   update   W  -= eta * U^T V      (Section 3, Figure 1: reconstruction of the K rank-1 updates)
//   coder    r = W a - x, g = W^T r (ISTA iterations of the sparse coder, Figure 3's compute_sparse_code)
// One register-tiled kernel, 128 x 128 x 16 tiles, 256 threads, 8 x 8 outputs per thread, operands staged
// through shared memory with a register prefetch of the next k-block.
#include "sfb_internal.h"

namespace sfb {
namespace {

constexpr int BM = 128, BN = 128, BK = 16, NT = 256;

// Loads the [BK x BM] slice of an operand into registers (2 float4 per thread).
// KC: element (m,k) at p[m*ld + k]; else at p[k*ld + m].  Out-of-range elements read as 0.
template <bool KC>
__device__ __forceinline__ void load_tile(float4 (&r)[2], const float* __restrict__ p, int64_t ld, int64_t m0,
                                          int64_t M, int64_t k0, int64_t Kc, bool vec_ok, int t) {
#pragma unroll
  for (int v = 0; v < 2; ++v) {
    const int idx = t + v * NT;
    int64_t m, k;
    if (KC) { m = m0 + idx / (BK / 4); k = k0 + (idx % (BK / 4)) * 4; }
    else    { k = k0 + idx / (BM / 4); m = m0 + (idx % (BM / 4)) * 4; }
    float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
    if (KC) {
      if (m < M) {
        const float* q = p + m * ld + k;
        if (vec_ok && k + 3 < Kc) val = *reinterpret_cast<const float4*>(q);
        else {
          if (k + 0 < Kc) val.x = q[0];
          if (k + 1 < Kc) val.y = q[1];
          if (k + 2 < Kc) val.z = q[2];
          if (k + 3 < Kc) val.w = q[3];
        }
      }
    } else {
      if (k < Kc) {
        const float* q = p + k * ld + m;
        if (vec_ok && m + 3 < M) val = *reinterpret_cast<const float4*>(q);
        else {
          if (m + 0 < M) val.x = q[0];
          if (m + 1 < M) val.y = q[1];
          if (m + 2 < M) val.z = q[2];
          if (m + 3 < M) val.w = q[3];
        }
      }
    }
    r[v] = val;
  }
}

template <bool KC>
__device__ __forceinline__ void store_tile(float (*S)[BM + 4], const float4 (&r)[2], int t) {
#pragma unroll
  for (int v = 0; v < 2; ++v) {
    const int idx = t + v * NT;
    if (KC) {
      const int m = idx / (BK / 4), k = (idx % (BK / 4)) * 4;
      S[k + 0][m] = r[v].x; S[k + 1][m] = r[v].y; S[k + 2][m] = r[v].z; S[k + 3][m] = r[v].w;
    } else {
      const int k = idx / (BM / 4), m = (idx % (BM / 4)) * 4;
      *reinterpret_cast<float4*>(&S[k][m]) = r[v];
    }
  }
}

__device__ __forceinline__ float soft(float w, float t) {
  const float a = fabsf(w) - t;
  return a > 0.f ? copysignf(a, w) : 0.f;
}

template <int EPI>
__device__ __forceinline__ float epi_one(float acc, float cur, float aux, const EpiArgs& e, float invL) {
  if (EPI == EPI_STORE) return acc;
  if (EPI == EPI_SUB) return acc - aux;
  if (EPI == EPI_RMW) return prox_entry(fmaf(e.alpha, acc, cur), e.prox_kind, e.prox_a);
  return soft(fmaf(-acc, invL, cur), e.lam * invL);   // EPI_ISTA
}

template <bool A_KC, bool B_KC, int EPI>
__global__ void __launch_bounds__(NT) sgemm_kernel(int64_t M, int64_t N, int64_t Kc, const float* __restrict__ A,
                                                   int64_t lda, const float* __restrict__ B, int64_t ldb,
                                                   EpiArgs e, int64_t tilesM, bool a_vec, bool b_vec, bool c_vec) {
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int t = threadIdx.x;
  const int64_t tile = blockIdx.x;
  const int64_t m0 = (tile % tilesM) * BM, n0 = (tile / tilesM) * BN;
  const int ty = t / 16, tx = t % 16;

  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  float4 ra[2], rb[2];
  load_tile<A_KC>(ra, A, lda, m0, M, 0, Kc, a_vec, t);
  load_tile<B_KC>(rb, B, ldb, n0, N, 0, Kc, b_vec, t);
  for (int64_t k0 = 0; k0 < Kc; k0 += BK) {
    __syncthreads();
    store_tile<A_KC>(As, ra, t);
    store_tile<B_KC>(Bs, rb, t);
    __syncthreads();
    if (k0 + BK < Kc) {
      load_tile<A_KC>(ra, A, lda, m0, M, k0 + BK, Kc, a_vec, t);
      load_tile<B_KC>(rb, B, ldb, n0, N, k0 + BK, Kc, b_vec, t);
    }
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[k][64 + tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
  }

  float invL = 0.f;
  if (EPI == EPI_ISTA) invL = e.sc->invL;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int64_t m = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
    if (m >= M) continue;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int64_t n = n0 + h * 64 + tx * 4;
      if (n >= N) continue;
      float* c = e.C + m * e.ldc + n;
      const float* x = (EPI == EPI_SUB) ? e.aux + m * e.ldc + n : nullptr;
      if (c_vec && n + 3 < N) {
        float4 cur = make_float4(0.f, 0.f, 0.f, 0.f), aux = cur, out;
        if (EPI == EPI_RMW || EPI == EPI_ISTA) cur = *reinterpret_cast<const float4*>(c);
        if (EPI == EPI_SUB) aux = *reinterpret_cast<const float4*>(x);
        out.x = epi_one<EPI>(acc[i][h * 4 + 0], cur.x, aux.x, e, invL);
        out.y = epi_one<EPI>(acc[i][h * 4 + 1], cur.y, aux.y, e, invL);
        out.z = epi_one<EPI>(acc[i][h * 4 + 2], cur.z, aux.z, e, invL);
        out.w = epi_one<EPI>(acc[i][h * 4 + 3], cur.w, aux.w, e, invL);
        *reinterpret_cast<float4*>(c) = out;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (n + j < N) {
            const float cur = (EPI == EPI_RMW || EPI == EPI_ISTA) ? c[j] : 0.f;
            const float aux = (EPI == EPI_SUB) ? x[j] : 0.f;
            c[j] = epi_one<EPI>(acc[i][h * 4 + j], cur, aux, e, invL);
          }
        }
      }
    }
  }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <bool A_KC, bool B_KC>
cudaError_t launch(cudaStream_t s, Epilogue epi, int64_t M, int64_t N, int64_t Kc, const float* A, int64_t lda,
                   const float* B, int64_t ldb, const EpiArgs& e) {
  const int64_t tilesM = (M + BM - 1) / BM, tilesN = (N + BN - 1) / BN;
  const int64_t tiles = tilesM * tilesN;
  if (tiles <= 0) return cudaSuccess;
  if (tiles > 0x7fffffffLL) return cudaErrorInvalidValue;
  const bool a_vec = aligned16(A) && lda % 4 == 0;
  const bool b_vec = aligned16(B) && ldb % 4 == 0;
  const bool c_vec = aligned16(e.C) && e.ldc % 4 == 0 && (epi != EPI_SUB || aligned16(e.aux));
  dim3 grid(static_cast<unsigned>(tiles)), block(NT);
#define SFB_LAUNCH(E) sgemm_kernel<A_KC, B_KC, E><<<grid, block, 0, s>>>(M, N, Kc, A, lda, B, ldb, e, tilesM, \
                                                                            a_vec, b_vec, c_vec)
  switch (epi) {
    case EPI_STORE: SFB_LAUNCH(EPI_STORE); break;
    case EPI_SUB: SFB_LAUNCH(EPI_SUB); break;
    case EPI_RMW: SFB_LAUNCH(EPI_RMW); break;
    case EPI_ISTA: SFB_LAUNCH(EPI_ISTA); break;
  }
#undef SFB_LAUNCH
  count_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t sgemm(cudaStream_t s, bool a_kc, bool b_kc, Epilogue epi, int64_t M, int64_t N, int64_t Kc,
                  const float* A, int64_t lda, const float* B, int64_t ldb, const EpiArgs& e) {
  if (a_kc && b_kc) return launch<true, true>(s, epi, M, N, Kc, A, lda, B, ldb, e);
  if (a_kc && !b_kc) return launch<true, false>(s, epi, M, N, Kc, A, lda, B, ldb, e);
  if (!a_kc && !b_kc) return launch<false, false>(s, epi, M, N, Kc, A, lda, B, ldb, e);
  return cudaErrorInvalidValue;   // (m-contiguous A, k-contiguous B) is not used by any step
}

}  // namespace sfb
