// Internal declarations shared by the translation units of libsfb (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>

#include <atomic>
#include <stdint.h>

#include "sfb.h"

namespace sfb {

extern std::atomic<int64_t> g_kernel_launches;     // kernels launched by this library in this process
inline void count_launch(int n = 1) { g_kernel_launches.fetch_add(n, std::memory_order_relaxed); }

// Multiprocessors of the current device (looked up once per device ordinal).
int sm_count();

// ---------------------------------------------------------------------------------------------------------
// Workspace carve-up.  Every offset is a multiple of 1024 bytes so that any sub-buffer can be a TMA base.
// ---------------------------------------------------------------------------------------------------------
constexpr size_t kAlign = 1024;
constexpr int kProxSlabs = 64;        // row slabs of the deterministic column reductions

struct Layout {
  size_t status, scalars, loss, V, U, colpart, pib, piy, stageX, stageY, stageL;
  // bf16 tensor-core mode
  size_t Wb, Xb, VT, ZT, UT, part, Xf, labels, coef, lse;
  // bf16 mode, DML and SC: (hi | lo) bf16 operands of the split products
  size_t Ws, WTs, As, Rs;             // W by rows, W transposed, the A operand (v or the codes), the residual
  size_t U2;                          // DML: second partial of z when the forward product splits its contraction
  // sparse factors (MLR, csr_nnz_max > 0): the step's (sample, column, value) triples and their column-major form
  size_t coo_i, coo_c, coo_x, coo_cx, row_beg, row_end, csc_cnt, csc_cur, csc_ptr, csc_tmp, csc_ent;
  int64_t ldu;                        // row pitch of the fp32 U buffer (rows rounded up to 4 in bf16 mode)
  int64_t colsp, rowsp;               // cols, rows rounded up to 64
  int64_t Kp;                         // K rounded up to the contraction block of the update product
  int64_t colsb;                      // cols rounded up to the contraction block of the forward product
  size_t total;
};

Layout make_layout(const sfb_config& c);

// fp32 mode runs its products of multiclass logistic regression on the tensor cores (every fp32 value as a pair of
// tf32 words, three products per term) when asked to, or by itself when the shape is large enough to be worth the
// operand copies; small shapes and the other models use the FFMA kernels.
inline bool use_tf32(const sfb_config& c) {
  const bool mlr = c.model == SFB_MLR || c.model == SFB_L2MLR;
  if (c.precision == SFB_PREC_TF32X3) return mlr;
  if (c.precision != SFB_PREC_FP32 || !mlr) return false;
  return c.rows >= 2048 && c.cols >= 512 && static_cast<int64_t>(c.workers) * c.batch >= 128;
}

struct Scalars {                      // device-resident scalars
  float loss_mean;
  float L;                            // ||W||_2^2 used by the coder
  float invL;
  float tmp;
  unsigned long long copy_pieces;     // 64-byte row pieces of the bf16 operand copy the update passes went over ...
  unsigned long long copy_written;    // ... and how many of them they had to rewrite (the others already held bf16(W))
};

}  // namespace sfb

struct sfb_ctx {
  sfb_config cfg;
  sfb::Layout lay;
  float* W;
  char* ws;
  cudaStream_t stream;
  int64_t K;
  int64_t in_dim;
  int64_t row_offset;                 // row-sharded MLR: this context's W holds rows [row_offset, row_offset + rows)
  int64_t global_rows;                //   of a matrix with global_rows rows (class ids are global); 0, rows when unsharded
  bool partials_ready;                // sfb_forward_partials has run since the last update
  bool tf32;                          // fp32 mode with its products on the tensor cores (see use_tf32)
  bool sdca;                          // SFB_L2MLR: the factors are dual changes; cfg.model is kept as SFB_MLR internally
  float* dualQ;                       // SDCA dual state [dual_n x rows], caller-owned
  int64_t dual_n;
  float step;                         // multiplier of sum u v^T in the update: eta, or eta / (lam N) for SDCA
  int32_t prox_kind;                  // entry-wise prox of the update pass and its parameter (threshold or factor)
  float prox_a;
  uint64_t committed;                 // bit p set: worker p has written its factors since the last update
  uint64_t sparse_mask;               // bit p set: worker p's samples of this step came in compressed-sparse-row form
  int64_t csr_fill;                   // triples staged so far in this step
  int64_t last_stage_nnz;             // entries of the last staged block of samples
  bool sparse_v;                      // the gathered v are in column-major sparse form: the update sums only the non-zeros
  bool gathered;
  int last_cuda;
  cudaEvent_t ev[4];
  sfb_stats stats;
  void* tc;                           // tensor-core path state (tensor maps), owned

  template <typename T>
  T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
};

namespace sfb {

// ---------------------------------------------------------------------------------------------------------
// fp32 FMA matrix products:  C (M x N) = sum_k A(m,k) * B(n,k)  followed by an epilogue.
// A_KC: A(m,k) at A[m*lda + k] (k contiguous), else at A[k*lda + m].  Same for B with n.
// ---------------------------------------------------------------------------------------------------------
enum Epilogue { EPI_STORE = 0, EPI_SUB = 1, EPI_RMW = 2, EPI_ISTA = 3 };

// Entry-wise proximal operator fused into the update: kind 1 soft-threshold by a, kind 2 multiply by a.
__host__ __device__ __forceinline__ float prox_entry(float w, int kind, float a) {
  if (kind == 1) {
    const float m = fabsf(w) - a;
    return m > 0.f ? copysignf(m, w) : 0.f;
  }
  return kind == 2 ? w * a : w;
}

struct EpiArgs {
  int32_t prox_kind;   // EPI_RMW: entry-wise prox applied to the updated value (0 none)
  float prox_a;
  float* C;            // output, row-major [M x ldc]
  int64_t ldc;
  const float* aux;    // EPI_SUB: the matrix subtracted, same shape and ld as C
  float alpha;         // EPI_RMW: C += alpha * acc
  const Scalars* sc;   // EPI_ISTA: reads invL
  float lam;           // EPI_ISTA: C = soft(C - acc*invL, lam*invL)
};

cudaError_t sgemm(cudaStream_t s, bool a_kc, bool b_kc, Epilogue epi, int64_t M, int64_t N, int64_t Kc,
                  const float* A, int64_t lda, const float* B, int64_t ldb, const EpiArgs& e);

// ---------------------------------------------------------------------------------------------------------
// Factor kernels (pack, softmax, pair residual, prox, power iteration)
// ---------------------------------------------------------------------------------------------------------
cudaError_t pack_copy(cudaStream_t s, float* dst, const float* x, const float* y_or_null, int64_t n);
cudaError_t fill_zero(cudaStream_t s, float* dst, int64_t n);
cudaError_t mlr_softmax_rows(cudaStream_t s, float* Z, int64_t nsamp, int64_t rows, const int32_t* labels,
                             float* loss_per_sample, uint32_t* status);
// Row-sharded MLR: per-sample softmax partials (max, sum exp, label logit, owner flag) of a shard, and the finish with
// the partials of all shards ([shards][nsamp] float4).
cudaError_t mlr_shard_partials(cudaStream_t s, const float* Z, int64_t nsamp, int64_t rows, int64_t ldz,
                               const int32_t* labels, int64_t row_off, float* part);
cudaError_t mlr_shard_finish(cudaStream_t s, float* Z, int64_t nsamp, int64_t rows, int64_t ldz, const int32_t* labels,
                             int64_t row_off, const float* parts, int shards, float* loss, uint32_t* status);
// SDCA (l2-regularised MLR): per sample, from its logits z (row of Z, overwritten with du), its dual row of Q (advanced
// by gamma * du) and its features x: the change of the dual vector that minimises the dual objective.  coef (may be
// null) receives -du at the label entry.
cudaError_t sdca_dual_rows(cudaStream_t s, float* Z, int64_t nsamp, int64_t rows, int64_t ldz, const float* X, int64_t cols,
                           const int32_t* labels, const int32_t* ids, float* Q, int64_t n_samples, float inv_lam_n,
                           float gamma, float* coef, float* loss, uint32_t* status);
// Z2 (may be null): a second partial of z (the other half of the contraction), added to Z first.  Row-sharded form:
// norm_out (may be null) receives the shard's ||z_i||^2 and z is left unscaled; norms_all (may be null), [shards][nstride],
// supplies ||z_i||^2 as the sum over the shards instead of this context's own.
cudaError_t dml_scale_rows(cudaStream_t s, float* Z, int64_t nsamp, int64_t rows, int64_t ld,
                           const int32_t* similar, float margin, const float* Z2 = nullptr, float* norm_out = nullptr,
                           const float* norms_all = nullptr, int shards = 0, int64_t nstride = 0);
cudaError_t mean_of(cudaStream_t s, const float* v, int64_t n, float* out);
cudaError_t prox_unit_columns(cudaStream_t s, float* W, int64_t rows, int64_t cols, float* colpart);
cudaError_t estimate_lipschitz(cudaStream_t s, const float* W, int64_t rows, int64_t cols, float* b, float* y,
                               float* colpart, Scalars* sc, int iters);
cudaError_t set_lipschitz(cudaStream_t s, Scalars* sc, float L);
cudaError_t axpy(cudaStream_t s, float* y, const float* x, float alpha, int64_t n);  // y += alpha*x
cudaError_t prox_entries(cudaStream_t s, float* w, int64_t n, int kind, float a);      // w <- prox(w), entry-wise

// ---------------------------------------------------------------------------------------------------------
// Sparse sufficient factors (MLR): staging of compressed-sparse-row samples, their column-major form, the update
// ---------------------------------------------------------------------------------------------------------
void sparse_extend_layout(const sfb_config& c, Layout& L, size_t& off);
// The step's sparse samples take the sparse update: its factor slab of K samples fits the shared memory of a block and,
// unless the config forces either, the cost model prefers it to the tensor-core update over the scattered samples.
bool sparse_update_wanted(const sfb_ctx* ctx);
int sparse_stage(sfb_ctx* ctx, int64_t off, int64_t n, const int64_t* indptr, const int32_t* idx, const float* val,
                 int64_t nnz);
// fp32 FMA mode: rows of W per block of the row-wise forward over sparse samples (0: the rows do not fit), and that product
int sparse_forward_rows(const sfb_ctx* ctx, int64_t n);
int sparse_forward(sfb_ctx* ctx, int64_t off, int64_t n, float* Z, int64_t ldz);
int sparse_build_csc(sfb_ctx* ctx);
int sparse_update(sfb_ctx* ctx);

}  // namespace sfb
