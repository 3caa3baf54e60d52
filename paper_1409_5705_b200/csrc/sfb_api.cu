// C ABI of libsfb: argument checking, workspace carve-up, and the sequencing of one SFB step
// (Section 3, Figure 1: compute factors -> broadcast/gather -> reconstruct and apply -> prox).
#include <new>

#include "sfb_internal.h"
#include "sfb_tc.h"

namespace sfb {

std::atomic<int64_t> g_kernel_launches{0};

int sm_count() {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cache[kMaxDevices];          // zero-initialised: 0 = not looked up yet
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  int n = cache[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cache[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

static size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

Layout make_layout(const sfb_config& cfg) {
  sfb_config c = cfg;
  if (c.model == SFB_L2MLR) c.model = SFB_MLR;        // same buffers: the factors differ, the products do not
  Layout L{};
  const size_t K = static_cast<size_t>(c.workers) * c.batch;
  const size_t rows = c.rows, cols = c.cols;
  const size_t in_dim = c.model == SFB_SC ? rows : cols;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += up(bytes); return o; };
  L.status = take(sizeof(uint32_t));
  L.scalars = take(sizeof(Scalars));
  L.loss = take(K * 4);
  L.stageX = take(K * in_dim * 4);
  L.stageY = take(c.model == SFB_DML ? K * cols * 4 : 0);
  L.stageL = take(K * 4);
  L.colpart = take(c.model == SFB_SC ? static_cast<size_t>(kProxSlabs) * cols * 8 : 0);
  L.pib = take(c.model == SFB_SC ? cols * 4 : 0);
  L.piy = take(c.model == SFB_SC ? rows * 4 : 0);
  L.Kp = static_cast<int64_t>(K);
  L.colsb = static_cast<int64_t>(cols);
  L.ldu = static_cast<int64_t>(rows);
  if (use_tf32(cfg)) {
    tc32_extend_layout(c, L, off);
  } else if (c.precision != SFB_PREC_BF16) {
    L.V = take(K * cols * 4);
    L.U = take(K * rows * 4);
  } else {
    tc_extend_layout(c, L, off);
  }
  if (c.csr_nnz_max > 0 && c.model == SFB_MLR) sparse_extend_layout(c, L, off);
  L.total = off;
  return L;
}

}  // namespace sfb

using namespace sfb;

#define CK(call)                                        \
  do {                                                  \
    cudaError_t e__ = (call);                           \
    if (e__ != cudaSuccess) {                           \
      ctx->last_cuda = static_cast<int>(e__);           \
      return SFB_ERR_CUDA;                              \
    }                                                   \
  } while (0)

static bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_config(const sfb_config* c) {
  if (!c) return SFB_ERR_ARG;
  if (c->model < SFB_MLR || c->model > SFB_L2MLR) return SFB_ERR_ARG;
  if (c->model == SFB_L2MLR && (!(c->sdca_lambda > 0.f) || c->sdca_n < 1)) return SFB_ERR_ARG;
  if (c->precision < SFB_PREC_BF16 || c->precision > SFB_PREC_FP32_FFMA) return SFB_ERR_ARG;
  if (c->precision == SFB_PREC_TF32X3 && c->model != SFB_MLR && c->model != SFB_L2MLR) return SFB_ERR_UNSUPPORTED;
  if (c->rows <= 0 || c->cols <= 0 || c->workers <= 0 || c->batch <= 0) return SFB_ERR_ARG;
  if (c->workers > 64) return SFB_ERR_SHAPE;
  if (c->cols % 4 != 0) return SFB_ERR_SHAPE;
  if (c->rows > (1LL << 30) || c->cols > (1LL << 30)) return SFB_ERR_SHAPE;
  if (static_cast<int64_t>(c->workers) * c->batch > (1 << 20)) return SFB_ERR_SHAPE;
  if (c->model == SFB_SC && c->sc_ista_iters < 0) return SFB_ERR_ARG;
  if (c->model == SFB_SC && !(c->sc_lambda >= 0.f)) return SFB_ERR_ARG;
  if (c->sc_prox < 0 || c->sc_prox > 1) return SFB_ERR_ARG;
  if (c->prox_kind < 0 || c->prox_kind > 2 || !(c->prox_weight >= 0.f)) return SFB_ERR_ARG;
  if (c->model == SFB_L2MLR && c->prox_kind != 0) return SFB_ERR_UNSUPPORTED;
  if (c->csr_nnz_max < 0 || c->csr_nnz_max + c->cols > (1LL << 31) - 64) return SFB_ERR_SHAPE;
  if (c->csr_update < 0 || c->csr_update > 2) return SFB_ERR_ARG;
  return SFB_OK;
}

extern "C" int sfb_workspace_bytes(const sfb_config* cfg, size_t* out_bytes) {
  if (!out_bytes) return SFB_ERR_ARG;
  int rc = check_config(cfg);
  if (rc) return rc;
  *out_bytes = make_layout(*cfg).total;
  return SFB_OK;
}

extern "C" int sfb_init(const sfb_config* cfg, float* W_dev, void* workspace_dev, size_t workspace_bytes,
                        sfb_ctx** out) {
  if (!out) return SFB_ERR_ARG;
  *out = nullptr;
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!W_dev || !workspace_dev) return SFB_ERR_ARG;
  if (!al16(W_dev) || (reinterpret_cast<uintptr_t>(workspace_dev) & (kAlign - 1)) != 0) return SFB_ERR_ALIGN;
  Layout lay = make_layout(*cfg);
  if (workspace_bytes < lay.total) return SFB_ERR_WORKSPACE;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SFB_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SFB_ERR_CUDA;
  if (major != 10) return SFB_ERR_ARCH;

  sfb_ctx* ctx = new (std::nothrow) sfb_ctx();
  if (!ctx) return SFB_ERR_ARG;
  ctx->cfg = *cfg;
  ctx->tf32 = use_tf32(*cfg);
  if (cfg->precision != SFB_PREC_BF16) ctx->cfg.precision = SFB_PREC_FP32;      // one fp32 family; tf32 says which kernels
  ctx->sdca = cfg->model == SFB_L2MLR;
  if (ctx->sdca) ctx->cfg.model = SFB_MLR;            // the products, buffers and the update are those of MLR
  ctx->dualQ = nullptr;
  ctx->dual_n = 0;
  ctx->step = ctx->sdca ? static_cast<float>(static_cast<double>(cfg->eta) / (static_cast<double>(cfg->sdca_lambda) *
                                                                            static_cast<double>(cfg->sdca_n)))
                        : cfg->eta;
  // prox_{eta h}: threshold eta*w for the l1 norm, factor 1 / (1 + eta*w) for the squared l2 norm
  ctx->prox_kind = cfg->prox_kind;
  ctx->prox_a = cfg->prox_kind == 1 ? cfg->eta * cfg->prox_weight
              : cfg->prox_kind == 2 ? static_cast<float>(1.0 / (1.0 + static_cast<double>(cfg->eta) * cfg->prox_weight)) : 0.f;
  ctx->lay = lay;
  ctx->W = W_dev;
  ctx->ws = static_cast<char*>(workspace_dev);
  ctx->stream = static_cast<cudaStream_t>(cfg->stream);
  ctx->K = static_cast<int64_t>(cfg->workers) * cfg->batch;
  ctx->in_dim = cfg->model == SFB_SC ? cfg->rows : cfg->cols;
  ctx->committed = 0;
  ctx->sparse_mask = 0;
  ctx->csr_fill = 0;
  ctx->sparse_v = false;
  ctx->gathered = false;
  ctx->row_offset = 0;
  ctx->global_rows = cfg->rows;
  ctx->partials_ready = false;
  ctx->last_cuda = 0;
  ctx->stats = sfb_stats{};
  ctx->tc = nullptr;
  for (auto& e : ctx->ev) e = nullptr;
  for (auto& e : ctx->ev) {
    cudaError_t ce = cudaEventCreate(&e);
    if (ce != cudaSuccess) { sfb_destroy(ctx); return SFB_ERR_CUDA; }
  }
  // status word, scalars and per-sample losses are the first three (contiguous) regions
  cudaError_t ce = cudaMemsetAsync(ctx->ws + lay.status, 0, lay.stageX - lay.status, ctx->stream);
  if (ce != cudaSuccess) { sfb_destroy(ctx); return SFB_ERR_CUDA; }
  if (cfg->model == SFB_SC && cfg->sc_lipschitz > 0.f) {
    ce = set_lipschitz(ctx->stream, ctx->at<Scalars>(lay.scalars), cfg->sc_lipschitz);
    if (ce != cudaSuccess) { sfb_destroy(ctx); return SFB_ERR_CUDA; }
  }
  if (cfg->precision == SFB_PREC_BF16 || ctx->tf32) {
    rc = tc_init(ctx);
    if (rc) { sfb_destroy(ctx); return rc; }
  }
  *out = ctx;
  return SFB_OK;
}

extern "C" int sfb_destroy(sfb_ctx* ctx) {
  if (!ctx) return SFB_ERR_ARG;
  for (auto& e : ctx->ev)
    if (e) cudaEventDestroy(e);
  tc_destroy(ctx);
  delete ctx;
  return SFB_OK;
}

// ---------------------------------------------------------------------------------------------------------
// fp32-operand path
// ---------------------------------------------------------------------------------------------------------
static int factors_fp32(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const float* Y,
                        const int32_t* labels, bool sparse_fwd = false, float* dml_norm_out = nullptr) {
  const sfb_config& c = ctx->cfg;
  const int64_t rows = c.rows, cols = c.cols;
  float* V = ctx->at<float>(ctx->lay.V) + off * cols;
  float* U = ctx->at<float>(ctx->lay.U) + off * rows;
  Scalars* sc = ctx->at<Scalars>(ctx->lay.scalars);
  uint32_t* status = ctx->at<uint32_t>(ctx->lay.status);
  cudaStream_t s = ctx->stream;
  EpiArgs e{};
  if (c.model == SFB_MLR || c.model == SFB_DML) {
    CK(pack_copy(s, V, X, c.model == SFB_DML ? Y : nullptr, n * cols));                 // v = x | x - y
    e.C = U; e.ldc = rows;
    if (sparse_fwd) {                                                                   // z_i = W v_i over the non-zeros of v_i
      const int rc = sparse_forward(ctx, off, n, ctx->at<float>(ctx->lay.U), rows);
      if (rc) return rc;
    } else {
      CK(sgemm(s, true, true, EPI_STORE, n, rows, cols, V, cols, ctx->W, cols, e));     // z_i = W v_i
      ctx->stats.flops += 2.0 * n * rows * cols;
    }
    if (c.model == SFB_MLR)
      CK(mlr_softmax_rows(s, U, n, rows, labels, ctx->at<float>(ctx->lay.loss) + off, status));
    else
      CK(dml_scale_rows(s, U, n, rows, rows, labels, c.dml_margin, nullptr, dml_norm_out));
    return SFB_OK;
  }
  // sparse coding: ISTA from a = 0, then u = W a - x, v = a
  CK(fill_zero(s, V, n * cols));
  for (int it = 0; it <= c.sc_ista_iters; ++it) {
    e = EpiArgs{};
    e.C = U; e.ldc = rows; e.aux = X;
    CK(sgemm(s, true, true, EPI_SUB, n, rows, cols, V, cols, ctx->W, cols, e));         // r = W a - x
    ctx->stats.flops += 2.0 * n * rows * cols;
    if (it == c.sc_ista_iters) break;
    e = EpiArgs{};
    e.C = V; e.ldc = cols; e.sc = sc; e.lam = c.sc_lambda;
    CK(sgemm(s, true, false, EPI_ISTA, n, cols, rows, U, rows, ctx->W, cols, e));       // a <- soft(a - W^T r / L)
    ctx->stats.flops += 2.0 * n * rows * cols;
  }
  return SFB_OK;
}

static int update_fp32(sfb_ctx* ctx) {
  const sfb_config& c = ctx->cfg;
  if (ctx->sparse_v) return sparse_update(ctx);
  EpiArgs e{};
  e.C = ctx->W; e.ldc = c.cols; e.alpha = -ctx->step;
  e.prox_kind = ctx->prox_kind; e.prox_a = ctx->prox_a;
  CK(sgemm(ctx->stream, false, false, EPI_RMW, c.rows, c.cols, ctx->K, ctx->at<float>(ctx->lay.U), c.rows,
           ctx->at<float>(ctx->lay.V), c.cols, e));
  return SFB_OK;
}

// ---------------------------------------------------------------------------------------------------------
static int check_inputs(sfb_ctx* ctx, const float* X, const float* Y, const int32_t* labels) {
  if (!ctx || !X) return SFB_ERR_ARG;
  if (ctx->cfg.model == SFB_DML && (!Y || !labels)) return SFB_ERR_ARG;
  if (ctx->cfg.model == SFB_MLR && !labels) return SFB_ERR_ARG;
  if (!al16(X) || (Y && !al16(Y))) return SFB_ERR_ALIGN;
  return SFB_OK;
}

extern "C" int sfb_compute_factors(sfb_ctx* ctx, int32_t worker, const float* X_dev, const float* Y_dev,
                                   const int32_t* labels_dev) {
  int rc = check_inputs(ctx, X_dev, Y_dev, labels_dev);
  if (rc) return rc;
  const sfb_config& c = ctx->cfg;
  if (ctx->sdca) return SFB_ERR_UNSUPPORTED;          // the dual step needs the samples' ids: sfb_sdca_compute_factors
  if (worker < -1 || worker >= c.workers) return SFB_ERR_SHAPE;
  const int64_t off = worker < 0 ? 0 : static_cast<int64_t>(worker) * c.batch;
  const int64_t n = worker < 0 ? ctx->K : c.batch;
  if (ctx->committed == 0) {
    ctx->sparse_mask = 0;
    ctx->csr_fill = 0;
    CK(cudaEventRecord(ctx->ev[0], ctx->stream));
    // the coder's step size comes from the W every worker sees at the start of the step (BSP)
    if (c.model == SFB_SC && !(c.sc_lipschitz > 0.f))
      CK(estimate_lipschitz(ctx->stream, ctx->W, c.rows, c.cols, ctx->at<float>(ctx->lay.pib),
                            ctx->at<float>(ctx->lay.piy), ctx->at<float>(ctx->lay.colpart),
                            ctx->at<Scalars>(ctx->lay.scalars), 50));
  }
  // bf16 mode: every product runs on the tensor cores; DML and SC, whose u comes from a cancelling residual,
  // carry each value as a (hi, lo) pair of bf16 (fp32-class products)
  rc = ctx->tf32 ? tc32_factors(ctx, off, n, X_dev, labels_dev, nullptr, 0.f)
       : c.precision == SFB_PREC_FP32 ? factors_fp32(ctx, off, n, X_dev, Y_dev, labels_dev)
                                      : tc_factors(ctx, off, n, X_dev, Y_dev, labels_dev);
  if (rc) return rc;
  const uint64_t all = c.workers == 64 ? ~0ull : ((1ull << c.workers) - 1);
  ctx->committed |= worker < 0 ? all : (1ull << worker);
  ctx->sparse_mask &= ~(worker < 0 ? all : (1ull << worker));       // these samples are dense
  ctx->gathered = false;
  return SFB_OK;
}

// ---------------------------------------------------------------------------------------------------------
// Samples in compressed-sparse-row form (MLR): scattered for the dense forward product, and kept as triples for the
// column-major form that the update reads
// ---------------------------------------------------------------------------------------------------------
extern "C" int sfb_compute_factors_csr(sfb_ctx* ctx, int32_t worker, const int64_t* indptr_dev, const int32_t* indices_dev,
                                       const float* values_dev, int64_t nnz, const int32_t* labels_dev) {
  if (!ctx || !indptr_dev || !labels_dev || nnz < 0) return SFB_ERR_ARG;
  if (nnz > 0 && (!indices_dev || !values_dev)) return SFB_ERR_ARG;
  const sfb_config& c = ctx->cfg;
  if (c.model != SFB_MLR || ctx->sdca || c.csr_nnz_max <= 0) return SFB_ERR_UNSUPPORTED;
  if (worker < -1 || worker >= c.workers) return SFB_ERR_SHAPE;
  if (ctx->partials_ready) return SFB_ERR_STATE;
  const uint64_t all = c.workers == 64 ? ~0ull : ((1ull << c.workers) - 1);
  const uint64_t bits = worker < 0 ? all : (1ull << worker);
  if (ctx->committed == 0) {
    ctx->sparse_mask = 0;
    ctx->csr_fill = 0;
  }
  if (ctx->sparse_mask & bits) return SFB_ERR_STATE;                // its triples are already in the step's list
  if (ctx->csr_fill + nnz > c.csr_nnz_max) return SFB_ERR_SHAPE;
  const int64_t off = worker < 0 ? 0 : static_cast<int64_t>(worker) * c.batch;
  const int64_t n = worker < 0 ? ctx->K : c.batch;
  if (ctx->committed == 0) CK(cudaEventRecord(ctx->ev[0], ctx->stream));
  int rc = sparse_stage(ctx, off, n, indptr_dev, indices_dev, values_dev, nnz);
  if (rc) return rc;
  const float* X = ctx->at<float>(ctx->lay.stageX) + off * c.cols;
  rc = ctx->tf32 ? tc32_factors(ctx, off, n, X, labels_dev, nullptr, 0.f)
       : c.precision == SFB_PREC_FP32 ? factors_fp32(ctx, off, n, X, nullptr, labels_dev, sparse_forward_rows(ctx, n) > 0)
                                      : tc_factors(ctx, off, n, X, nullptr, labels_dev);
  if (rc) return rc;
  ctx->csr_fill += nnz;
  ctx->sparse_mask |= bits;
  ctx->committed |= bits;
  ctx->gathered = false;
  return SFB_OK;
}

extern "C" int sfb_step_csr(sfb_ctx* ctx, const int64_t* indptr_dev, const int32_t* indices_dev, const float* values_dev,
                            int64_t nnz, const int32_t* labels_dev) {
  if (!ctx) return SFB_ERR_ARG;
  ctx->committed = 0;
  int rc = sfb_compute_factors_csr(ctx, -1, indptr_dev, indices_dev, values_dev, nnz, labels_dev);
  if (rc) return rc;
  rc = sfb_gather_factors(ctx);
  if (rc) return rc;
  return sfb_apply_update(ctx);
}

// ---------------------------------------------------------------------------------------------------------
// Row-sharded MLR: the parameter matrix partitioned by rows over several contexts (one per GPU)
// ---------------------------------------------------------------------------------------------------------
extern "C" int sfb_set_row_shard(sfb_ctx* ctx, int64_t row_offset, int64_t global_rows) {
  if (!ctx) return SFB_ERR_ARG;
  if ((ctx->cfg.model != SFB_MLR && ctx->cfg.model != SFB_DML) || ctx->sdca) return SFB_ERR_UNSUPPORTED;
  if (row_offset < 0 || global_rows < row_offset + ctx->cfg.rows || global_rows > (1LL << 31) - 1) return SFB_ERR_SHAPE;
  if (ctx->committed != 0 || ctx->partials_ready) return SFB_ERR_STATE;
  ctx->row_offset = row_offset;
  ctx->global_rows = global_rows;
  return SFB_OK;
}

extern "C" int sfb_forward_partials(sfb_ctx* ctx, const float* X_dev, const int32_t* labels_dev, float* partials_dev) {
  int rc = check_inputs(ctx, X_dev, nullptr, labels_dev);
  if (rc) return rc;
  if (ctx->cfg.model != SFB_MLR || ctx->sdca) return SFB_ERR_UNSUPPORTED;
  if (!partials_dev) return SFB_ERR_ARG;
  if (!al16(partials_dev)) return SFB_ERR_ALIGN;
  const sfb_config& c = ctx->cfg;
  ctx->committed = 0;
  ctx->sparse_mask = 0;
  ctx->csr_fill = 0;
  ctx->gathered = false;
  CK(cudaEventRecord(ctx->ev[0], ctx->stream));
  if (c.precision == SFB_PREC_BF16 || ctx->tf32) {
    rc = ctx->tf32 ? tc32_forward_partials(ctx, X_dev, labels_dev, partials_dev)
                   : tc_forward_partials(ctx, X_dev, labels_dev, partials_dev);
    if (rc) return rc;
  } else {
    const int64_t K = ctx->K;
    float* V = ctx->at<float>(ctx->lay.V);
    float* U = ctx->at<float>(ctx->lay.U);
    CK(pack_copy(ctx->stream, V, X_dev, nullptr, K * c.cols));                                    // v = x
    EpiArgs e{};
    e.C = U; e.ldc = c.rows;
    CK(sgemm(ctx->stream, true, true, EPI_STORE, K, c.rows, c.cols, V, c.cols, ctx->W, c.cols, e));   // z_i = W_shard x_i
    ctx->stats.flops += 2.0 * K * c.rows * c.cols;
    // the class ids are kept for the finish (the caller's buffer may change before it)
    CK(cudaMemcpyAsync(ctx->at<int32_t>(ctx->lay.stageL), labels_dev, static_cast<size_t>(K) * 4, cudaMemcpyDeviceToDevice,
                       ctx->stream));
    CK(mlr_shard_partials(ctx->stream, U, K, c.rows, c.rows, ctx->at<int32_t>(ctx->lay.stageL), ctx->row_offset,
                          partials_dev));
  }
  ctx->partials_ready = true;
  return SFB_OK;
}

// DML by rows: z = W v splits over the shards, the hinge needs ||z||^2 = sum over the shards of ||z_shard||^2.
extern "C" int sfb_forward_partials_pairs(sfb_ctx* ctx, const float* X_dev, const float* Y_dev, const int32_t* similar_dev,
                                          float* partials_dev) {
  int rc = check_inputs(ctx, X_dev, Y_dev, similar_dev);
  if (rc) return rc;
  if (ctx->cfg.model != SFB_DML) return SFB_ERR_UNSUPPORTED;
  if (!partials_dev) return SFB_ERR_ARG;
  const sfb_config& c = ctx->cfg;
  ctx->committed = 0;
  ctx->sparse_mask = 0;
  ctx->csr_fill = 0;
  ctx->gathered = false;
  CK(cudaEventRecord(ctx->ev[0], ctx->stream));
  // the flags are kept for the finish (the caller's buffer may change before it)
  CK(cudaMemcpyAsync(ctx->at<int32_t>(ctx->lay.stageL), similar_dev, static_cast<size_t>(ctx->K) * 4, cudaMemcpyDeviceToDevice,
                     ctx->stream));
  rc = c.precision == SFB_PREC_FP32 ? factors_fp32(ctx, 0, ctx->K, X_dev, Y_dev, similar_dev, false, partials_dev)
                                    : tc_factors(ctx, 0, ctx->K, X_dev, Y_dev, similar_dev, partials_dev);
  if (rc) return rc;
  ctx->partials_ready = true;
  return SFB_OK;
}

extern "C" int sfb_finish_factors(sfb_ctx* ctx, const float* partials_all_dev, int32_t shards) {
  if (!ctx || !partials_all_dev) return SFB_ERR_ARG;
  if (ctx->cfg.model != SFB_MLR && ctx->cfg.model != SFB_DML) return SFB_ERR_UNSUPPORTED;
  if (shards < 1 || shards > 4096) return SFB_ERR_ARG;
  if (!al16(partials_all_dev)) return SFB_ERR_ALIGN;
  if (!ctx->partials_ready) return SFB_ERR_STATE;
  const sfb_config& c = ctx->cfg;
  if (c.model == SFB_DML) {
    const int64_t ldu = c.precision == SFB_PREC_FP32 ? c.rows : ctx->lay.ldu;
    CK(dml_scale_rows(ctx->stream, ctx->at<float>(ctx->lay.U), ctx->K, c.rows, ldu, ctx->at<int32_t>(ctx->lay.stageL),
                      c.dml_margin, nullptr, nullptr, partials_all_dev, shards, ctx->K));
    ctx->partials_ready = false;
    ctx->committed = c.workers == 64 ? ~0ull : ((1ull << c.workers) - 1);
    ctx->gathered = false;
    return SFB_OK;
  }
  if (c.precision == SFB_PREC_BF16 || ctx->tf32) {
    const int rc = ctx->tf32 ? tc32_finish_factors(ctx, partials_all_dev, shards)
                             : tc_finish_factors(ctx, partials_all_dev, shards);
    if (rc) return rc;
  } else {
    CK(mlr_shard_finish(ctx->stream, ctx->at<float>(ctx->lay.U), ctx->K, c.rows, c.rows, ctx->at<int32_t>(ctx->lay.stageL),
                        ctx->row_offset, partials_all_dev, shards, ctx->at<float>(ctx->lay.loss),
                        ctx->at<uint32_t>(ctx->lay.status)));
  }
  ctx->partials_ready = false;
  ctx->committed = c.workers == 64 ? ~0ull : ((1ull << c.workers) - 1);
  ctx->gathered = false;
  return SFB_OK;
}

// Sufficient factors computed elsewhere (another replica, another machine) take the place of a worker's own:
// the receiving side of the broadcast of Section 3.
extern "C" int sfb_set_factors(sfb_ctx* ctx, int32_t worker, const float* U_dev, const float* V_dev) {
  if (!ctx || !U_dev || !V_dev) return SFB_ERR_ARG;
  const sfb_config& c = ctx->cfg;
  if (worker < 0 || worker >= c.workers) return SFB_ERR_SHAPE;
  if (ctx->sdca) return SFB_ERR_UNSUPPORTED;
  if (ctx->partials_ready) return SFB_ERR_STATE;
  if (ctx->committed == 0) CK(cudaEventRecord(ctx->ev[0], ctx->stream));
  const int64_t off = static_cast<int64_t>(worker) * c.batch;
  if (c.precision == SFB_PREC_BF16 && c.model == SFB_MLR) {
    const int rc = tc_import_factors(ctx, off, c.batch, U_dev, V_dev);
    if (rc) return rc;
    ctx->committed |= 1ull << worker;
    ctx->sparse_mask &= ~(1ull << worker);
    ctx->gathered = false;
    return SFB_OK;
  }
  const int64_t ldu = c.precision == SFB_PREC_FP32 ? c.rows : ctx->lay.ldu;
  float* U = ctx->at<float>(ctx->lay.U) + off * ldu;
  float* V = ctx->at<float>(ctx->lay.V) + off * c.cols;
  CK(cudaMemcpy2DAsync(U, static_cast<size_t>(ldu) * 4, U_dev, static_cast<size_t>(c.rows) * 4, static_cast<size_t>(c.rows) * 4,
                       static_cast<size_t>(c.batch), cudaMemcpyDeviceToDevice, ctx->stream));
  CK(cudaMemcpyAsync(V, V_dev, static_cast<size_t>(c.batch) * c.cols * 4, cudaMemcpyDeviceToDevice, ctx->stream));
  ctx->committed |= 1ull << worker;
  ctx->sparse_mask &= ~(1ull << worker);             // received factors are dense
  ctx->gathered = false;
  return SFB_OK;
}

extern "C" int sfb_export_factors(sfb_ctx* ctx, int32_t worker, float* U_out_dev, float* V_out_dev) {
  if (!ctx || !U_out_dev || !V_out_dev) return SFB_ERR_ARG;
  const sfb_config& c = ctx->cfg;
  if (worker < 0 || worker >= c.workers) return SFB_ERR_SHAPE;
  if (ctx->sdca) return SFB_ERR_UNSUPPORTED;
  if (!(ctx->committed & (1ull << worker))) return SFB_ERR_STATE;
  const int64_t off = static_cast<int64_t>(worker) * c.batch;
  if (c.precision == SFB_PREC_BF16 && c.model == SFB_MLR) return tc_export_factors(ctx, off, c.batch, U_out_dev, V_out_dev);
  const int64_t ldu = c.precision == SFB_PREC_FP32 ? c.rows : ctx->lay.ldu;
  CK(cudaMemcpy2DAsync(U_out_dev, static_cast<size_t>(c.rows) * 4, ctx->at<float>(ctx->lay.U) + off * ldu,
                       static_cast<size_t>(ldu) * 4, static_cast<size_t>(c.rows) * 4, static_cast<size_t>(c.batch),
                       cudaMemcpyDeviceToDevice, ctx->stream));
  CK(cudaMemcpyAsync(V_out_dev, ctx->at<float>(ctx->lay.V) + off * c.cols, static_cast<size_t>(c.batch) * c.cols * 4,
                     cudaMemcpyDeviceToDevice, ctx->stream));
  return SFB_OK;
}

extern "C" int sfb_set_eta(sfb_ctx* ctx, float eta) {
  if (!ctx || !(eta >= 0.f)) return SFB_ERR_ARG;
  if (ctx->committed != 0 || ctx->partials_ready) return SFB_ERR_STATE;       // not between the factors and their update
  ctx->cfg.eta = eta;
  ctx->step = ctx->sdca ? static_cast<float>(static_cast<double>(eta) / (static_cast<double>(ctx->cfg.sdca_lambda) *
                                                                        static_cast<double>(ctx->cfg.sdca_n)))
                        : eta;
  ctx->prox_a = ctx->prox_kind == 1 ? eta * ctx->cfg.prox_weight
              : ctx->prox_kind == 2 ? static_cast<float>(1.0 / (1.0 + static_cast<double>(eta) * ctx->cfg.prox_weight)) : 0.f;
  return SFB_OK;
}

extern "C" int sfb_gather_factors(sfb_ctx* ctx) {
  if (!ctx) return SFB_ERR_ARG;
  const sfb_config& c = ctx->cfg;
  const uint64_t all = c.workers == 64 ? ~0ull : ((1ull << c.workers) - 1);
  if (ctx->committed != all) return SFB_ERR_STATE;
  CK(cudaEventRecord(ctx->ev[1], ctx->stream));
  // Every worker wrote its pairs at row offset p*B of the shared buffers, so the gathered operands are
  // complete; what remains is the per-step read-out over all K pairs.
  // all K samples sparse: the v become their column-major form (and the dense update operands are not needed)
  ctx->sparse_v = c.model == SFB_MLR && c.csr_nnz_max > 0 && ctx->sparse_mask == all && sparse_update_wanted(ctx);
  if (ctx->sparse_v) {
    int rc = sparse_build_csc(ctx);
    if (rc) return rc;
  } else if (c.precision == SFB_PREC_BF16 || ctx->tf32) {
    int rc = ctx->tf32 ? tc32_gather(ctx) : tc_gather(ctx);
    if (rc) return rc;
  }
  if (c.model == SFB_MLR)
    CK(mean_of(ctx->stream, ctx->at<float>(ctx->lay.loss), ctx->K,
               &ctx->at<Scalars>(ctx->lay.scalars)->loss_mean));
  // bytes per gathered value: fp32, bf16, or a (hi, lo) pair of bf16 for the split operands of DML and SC
  const double esz = (c.precision == SFB_PREC_FP32 || c.model != SFB_MLR) ? 4.0 : 2.0;
  // sparse v: 8 bytes (index, value) per non-zero instead of cols values per sample
  const double pair = ctx->sparse_v ? static_cast<double>(c.rows) * esz + 8.0 * static_cast<double>(ctx->csr_fill) / ctx->K
                                    : static_cast<double>(c.rows + c.cols) * esz;
  ctx->stats.gather_bytes += static_cast<double>(ctx->K) * pair;
  ctx->stats.gather_bytes_p2p += static_cast<double>(c.workers) * (c.workers - 1) * c.batch * pair;
  ctx->stats.dense_sync_bytes += static_cast<double>(c.workers) * c.rows * c.cols * 4.0;
  ctx->gathered = true;
  CK(cudaEventRecord(ctx->ev[2], ctx->stream));
  return SFB_OK;
}

static int apply_prox(sfb_ctx* ctx) {
  const sfb_config& c = ctx->cfg;
  if (c.model == SFB_SC && c.sc_prox == 1)
    CK(prox_unit_columns(ctx->stream, ctx->W, c.rows, c.cols, ctx->at<float>(ctx->lay.colpart)));
  return SFB_OK;
}

extern "C" int sfb_apply_update(sfb_ctx* ctx) {
  if (!ctx) return SFB_ERR_ARG;
  if (!ctx->gathered) return SFB_ERR_STATE;
  const sfb_config& c = ctx->cfg;
  int rc = ctx->tf32 ? tc32_update(ctx) : c.precision == SFB_PREC_FP32 ? update_fp32(ctx) : tc_update(ctx);
  if (rc) return rc;
  ctx->stats.flops += 2.0 * c.rows * c.cols * ctx->K;
  rc = apply_prox(ctx);
  if (rc) return rc;
  CK(cudaEventRecord(ctx->ev[3], ctx->stream));
  ctx->committed = 0;
  ctx->sparse_mask = 0;               // the next step starts with no sparse samples staged
  ctx->csr_fill = 0;
  ctx->gathered = false;
  ctx->stats.steps += 1;
  ctx->stats.samples += ctx->K;
  if (ctx->sparse_v) ctx->stats.sparse_updates += 1;
  return SFB_OK;
}

// ---------------------------------------------------------------------------------------------------------
// l2-regularised MLR by stochastic dual coordinate ascent
// ---------------------------------------------------------------------------------------------------------
extern "C" int sfb_sdca_set_dual(sfb_ctx* ctx, float* Q_dev, int64_t n_samples) {
  if (!ctx || !Q_dev) return SFB_ERR_ARG;
  if (!ctx->sdca) return SFB_ERR_UNSUPPORTED;
  if (n_samples != ctx->cfg.sdca_n) return SFB_ERR_SHAPE;
  if (!al16(Q_dev)) return SFB_ERR_ALIGN;
  ctx->dualQ = Q_dev;
  ctx->dual_n = n_samples;
  return SFB_OK;
}

extern "C" int sfb_sdca_compute_factors(sfb_ctx* ctx, int32_t worker, const float* X_dev, const int32_t* labels_dev,
                                        const int32_t* sample_ids_dev) {
  if (!ctx || !X_dev || !labels_dev || !sample_ids_dev) return SFB_ERR_ARG;
  if (!ctx->sdca) return SFB_ERR_UNSUPPORTED;
  if (!ctx->dualQ) return SFB_ERR_STATE;
  if (!al16(X_dev)) return SFB_ERR_ALIGN;
  const sfb_config& c = ctx->cfg;
  if (worker < -1 || worker >= c.workers) return SFB_ERR_SHAPE;
  const int64_t off = worker < 0 ? 0 : static_cast<int64_t>(worker) * c.batch;
  const int64_t n = worker < 0 ? ctx->K : c.batch;
  if (ctx->committed == 0) CK(cudaEventRecord(ctx->ev[0], ctx->stream));
  const float inv_lam_n = static_cast<float>(1.0 / (static_cast<double>(c.sdca_lambda) * static_cast<double>(c.sdca_n)));
  uint32_t* status = ctx->at<uint32_t>(ctx->lay.status);
  float* loss = ctx->at<float>(ctx->lay.loss) + off;
  if (ctx->tf32) {
    const int rc = tc32_factors(ctx, off, n, X_dev, labels_dev, sample_ids_dev, inv_lam_n);
    if (rc) return rc;
  } else if (c.precision == SFB_PREC_FP32) {
    float* V = ctx->at<float>(ctx->lay.V) + off * c.cols;
    float* U = ctx->at<float>(ctx->lay.U) + off * c.rows;
    CK(pack_copy(ctx->stream, V, X_dev, nullptr, n * c.cols));                                        // v = a_i
    EpiArgs e{};
    e.C = U; e.ldc = c.rows;
    CK(sgemm(ctx->stream, true, true, EPI_STORE, n, c.rows, c.cols, V, c.cols, ctx->W, c.cols, e));   // z_i = W a_i
    ctx->stats.flops += 2.0 * n * c.rows * c.cols;
    CK(sdca_dual_rows(ctx->stream, U, n, c.rows, c.rows, X_dev, c.cols, labels_dev, sample_ids_dev, ctx->dualQ, ctx->dual_n,
                      inv_lam_n, c.eta, nullptr, loss, status));                                      // u_i = du_i
  } else {
    const int rc = tc_sdca_factors(ctx, off, n, X_dev, labels_dev, sample_ids_dev, inv_lam_n);
    if (rc) return rc;
  }
  const uint64_t all = c.workers == 64 ? ~0ull : ((1ull << c.workers) - 1);
  ctx->committed |= worker < 0 ? all : (1ull << worker);
  ctx->gathered = false;
  return SFB_OK;
}

extern "C" int sfb_sdca_step(sfb_ctx* ctx, const float* X_dev, const int32_t* labels_dev, const int32_t* sample_ids_dev) {
  if (!ctx) return SFB_ERR_ARG;
  ctx->committed = 0;
  int rc = sfb_sdca_compute_factors(ctx, -1, X_dev, labels_dev, sample_ids_dev);
  if (rc) return rc;
  rc = sfb_gather_factors(ctx);
  if (rc) return rc;
  return sfb_apply_update(ctx);
}

extern "C" int sfb_refresh_operands(sfb_ctx* ctx) {
  if (!ctx) return SFB_ERR_ARG;
  if (ctx->committed != 0 || ctx->partials_ready) return SFB_ERR_STATE;      // not in the middle of a step
  if (ctx->cfg.precision != SFB_PREC_BF16 && !ctx->tf32) return SFB_OK;       // the FFMA kernels read W itself
  return tc_refresh_operands(ctx);
}

extern "C" int sfb_replay_update(sfb_ctx* ctx) {
  if (!ctx) return SFB_ERR_ARG;
  if (ctx->stats.steps < 1 || ctx->committed != 0 || ctx->partials_ready) return SFB_ERR_STATE;
  const sfb_config& c = ctx->cfg;
  CK(cudaEventRecord(ctx->ev[2], ctx->stream));
  int rc = ctx->tf32 ? tc32_update(ctx) : c.precision == SFB_PREC_FP32 ? update_fp32(ctx) : tc_update(ctx);
  if (rc) return rc;
  ctx->stats.flops += 2.0 * c.rows * c.cols * ctx->K;
  rc = apply_prox(ctx);
  if (rc) return rc;
  CK(cudaEventRecord(ctx->ev[3], ctx->stream));
  return SFB_OK;
}

extern "C" int sfb_step(sfb_ctx* ctx, const float* X_dev, const float* Y_dev, const int32_t* labels_dev) {
  if (!ctx) return SFB_ERR_ARG;
  ctx->committed = 0;
  int rc = sfb_compute_factors(ctx, -1, X_dev, Y_dev, labels_dev);
  if (rc) return rc;
  rc = sfb_gather_factors(ctx);
  if (rc) return rc;
  return sfb_apply_update(ctx);
}

extern "C" int sfb_step_host(sfb_ctx* ctx, const float* X_host, const float* Y_host, const int32_t* labels_host,
                             float* loss_out, uint32_t* status_out) {
  if (!ctx || !X_host) return SFB_ERR_ARG;
  if (ctx->sdca) return SFB_ERR_UNSUPPORTED;
  const sfb_config& c = ctx->cfg;
  if (c.model == SFB_DML && (!Y_host || !labels_host)) return SFB_ERR_ARG;
  if (c.model == SFB_MLR && !labels_host) return SFB_ERR_ARG;
  float* Xs = ctx->at<float>(ctx->lay.stageX);
  float* Ys = ctx->at<float>(ctx->lay.stageY);
  int32_t* Ls = ctx->at<int32_t>(ctx->lay.stageL);
  CK(cudaMemcpyAsync(Xs, X_host, static_cast<size_t>(ctx->K) * ctx->in_dim * 4, cudaMemcpyHostToDevice, ctx->stream));
  if (c.model == SFB_DML)
    CK(cudaMemcpyAsync(Ys, Y_host, static_cast<size_t>(ctx->K) * c.cols * 4, cudaMemcpyHostToDevice, ctx->stream));
  if (c.model != SFB_SC)
    CK(cudaMemcpyAsync(Ls, labels_host, static_cast<size_t>(ctx->K) * 4, cudaMemcpyHostToDevice, ctx->stream));
  int rc = sfb_step(ctx, Xs, c.model == SFB_DML ? Ys : nullptr, c.model != SFB_SC ? Ls : nullptr);
  if (rc) return rc;
  float loss = 0.f;
  uint32_t st = 0;
  CK(cudaMemcpyAsync(&loss, &ctx->at<Scalars>(ctx->lay.scalars)->loss_mean, 4, cudaMemcpyDeviceToHost, ctx->stream));
  CK(cudaMemcpyAsync(&st, ctx->at<uint32_t>(ctx->lay.status), 4, cudaMemcpyDeviceToHost, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));
  if (loss_out) *loss_out = loss;
  if (status_out) *status_out = st;
  return SFB_OK;
}

extern "C" int sfb_dense_sync_step(sfb_ctx* ctx, const float* X_dev, const float* Y_dev, const int32_t* labels_dev,
                                   float* scratch_dev, size_t scratch_bytes) {
  if (!ctx || !scratch_dev) return SFB_ERR_ARG;
  const sfb_config& c = ctx->cfg;
  if (c.precision != SFB_PREC_FP32) return SFB_ERR_UNSUPPORTED;
  if (!al16(scratch_dev)) return SFB_ERR_ALIGN;
  const size_t mat = static_cast<size_t>(c.rows) * c.cols;
  if (scratch_bytes < 2 * mat * 4) return SFB_ERR_WORKSPACE;
  ctx->committed = 0;
  int rc = sfb_compute_factors(ctx, -1, X_dev, Y_dev, labels_dev);
  if (rc) return rc;
  rc = sfb_gather_factors(ctx);   // loss read-out and byte accounting; the factors stay per worker below
  if (rc) return rc;
  float* sum = scratch_dev;
  float* one = scratch_dev + mat;
  const float* U = ctx->at<float>(ctx->lay.U);
  const float* V = ctx->at<float>(ctx->lay.V);
  for (int p = 0; p < c.workers; ++p) {
    // worker p's dense update matrix, as it would be sent to the server
    EpiArgs e{};
    e.C = p == 0 ? sum : one; e.ldc = c.cols;
    CK(sgemm(ctx->stream, false, false, EPI_STORE, c.rows, c.cols, c.batch, U + static_cast<int64_t>(p) * c.batch * c.rows,
             c.rows, V + static_cast<int64_t>(p) * c.batch * c.cols, c.cols, e));
    if (p > 0) CK(axpy(ctx->stream, sum, one, 1.f, static_cast<int64_t>(mat)));          // server-side aggregation
  }
  CK(axpy(ctx->stream, ctx->W, sum, -c.eta, static_cast<int64_t>(mat)));                 // W <- W - eta * sum_p dW_p
  CK(prox_entries(ctx->stream, ctx->W, static_cast<int64_t>(mat), ctx->prox_kind, ctx->prox_a));
  ctx->stats.flops += 2.0 * c.rows * c.cols * ctx->K;
  rc = apply_prox(ctx);
  if (rc) return rc;
  CK(cudaEventRecord(ctx->ev[3], ctx->stream));
  ctx->committed = 0;
  ctx->gathered = false;
  ctx->stats.steps += 1;
  ctx->stats.samples += ctx->K;
  return SFB_OK;
}

extern "C" int sfb_get_factors(sfb_ctx* ctx, const void** U_dev, const void** V_dev, int32_t* dtype, int32_t* layout,
                               int64_t* ldu, int64_t* ldv) {
  if (!ctx) return SFB_ERR_ARG;
  if (ctx->cfg.precision == SFB_PREC_FP32) {
    if (U_dev) *U_dev = ctx->at<float>(ctx->lay.U);
    if (V_dev) *V_dev = ctx->at<float>(ctx->lay.V);
    if (dtype) *dtype = 0;
    if (layout) *layout = 0;
    if (ldu) *ldu = ctx->cfg.rows;
    if (ldv) *ldv = ctx->cfg.cols;
    return SFB_OK;
  }
  return tc_get_factors(ctx, U_dev, V_dev, dtype, layout, ldu, ldv);
}

extern "C" int sfb_get_operand_copy(sfb_ctx* ctx, const void** copy_dev, int32_t* dtype, int64_t* ld) {
  if (!ctx || !copy_dev) return SFB_ERR_ARG;
  if (ctx->cfg.model != SFB_MLR) return SFB_ERR_UNSUPPORTED;
  if (ctx->tf32) {
    *copy_dev = ctx->at<float>(ctx->lay.Ws);
    if (dtype) *dtype = 2;
    if (ld) *ld = 2 * ctx->lay.colsp;
    return SFB_OK;
  }
  if (ctx->cfg.precision != SFB_PREC_BF16) return SFB_ERR_UNSUPPORTED;
  *copy_dev = ctx->at<char>(ctx->lay.Wb);
  if (dtype) *dtype = 1;
  if (ld) *ld = ctx->lay.colsb;
  return SFB_OK;
}

extern "C" int sfb_get_stats(sfb_ctx* ctx, sfb_stats* out) {
  if (!ctx || !out) return SFB_ERR_ARG;
  CK(cudaStreamSynchronize(ctx->stream));
  if (ctx->stats.steps > 0) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->ev[0], ctx->ev[1]) == cudaSuccess) ctx->stats.ms_factors = ms;
    if (cudaEventElapsedTime(&ms, ctx->ev[1], ctx->ev[2]) == cudaSuccess) ctx->stats.ms_gather = ms;
    if (cudaEventElapsedTime(&ms, ctx->ev[2], ctx->ev[3]) == cudaSuccess) ctx->stats.ms_update = ms;
    cudaGetLastError();
    Scalars h{};
    CK(cudaMemcpy(&h, ctx->at<Scalars>(ctx->lay.scalars), sizeof(h), cudaMemcpyDeviceToHost));
    ctx->stats.last_loss = h.loss_mean;
    ctx->stats.sc_lipschitz = h.L;
    ctx->stats.copy_pieces = static_cast<int64_t>(h.copy_pieces);
    ctx->stats.copy_written = static_cast<int64_t>(h.copy_written);
  }
  ctx->stats.kernel_launches = g_kernel_launches.load(std::memory_order_relaxed);
  *out = ctx->stats;
  return SFB_OK;
}

extern "C" int sfb_get_status(sfb_ctx* ctx, uint32_t* status_out) {
  if (!ctx || !status_out) return SFB_ERR_ARG;
  CK(cudaMemcpyAsync(status_out, ctx->at<uint32_t>(ctx->lay.status), 4, cudaMemcpyDeviceToHost, ctx->stream));
  CK(cudaMemsetAsync(ctx->at<uint32_t>(ctx->lay.status), 0, 4, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));
  return SFB_OK;
}

extern "C" int sfb_last_cuda_error(sfb_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }

extern "C" const char* sfb_strerror(int code) {
  switch (code) {
    case SFB_OK: return "ok";
    case SFB_ERR_ARG: return "invalid argument";
    case SFB_ERR_ALIGN: return "pointer not 16-byte aligned";
    case SFB_ERR_SHAPE: return "unsupported shape";
    case SFB_ERR_WORKSPACE: return "workspace or scratch too small";
    case SFB_ERR_CUDA: return "CUDA runtime error";
    case SFB_ERR_ARCH: return "device is not compute capability 10.x";
    case SFB_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case SFB_ERR_LABEL_RANGE: return "class id out of range";
    case SFB_ERR_STATE: return "call out of order";
    case SFB_ERR_UNSUPPORTED: return "model/precision combination not built";
    case SFB_ERR_STATIC_LIMIT: return "size beyond the library's built-in scratch array";
    default: return "unknown error";
  }
}
