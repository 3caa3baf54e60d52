/*
 * sfb.h -- C ABI of the B200 (sm_100a) Sufficient Factor Broadcasting step.
 *
 * One minibatch step of the paper's computation model (Section 3, Figure 1; mini-batch form in Section 3,
 * "Mini-batch proximal SGD"): P logical workers hold B samples each; every worker turns its samples into
 * sufficient-factor pairs (u_i, v_i) against the same parameter matrix W (bulk-synchronous consistency,
 * Section 4.1); the K = P*B pairs are gathered into one buffer (the on-device form of the broadcast), and
 * the reconstructed update is applied:   W <- prox( W - eta * sum_{i<K} u_i v_i^T ).
 *
 * Conventions that hold for every call:
 *  - "dev" pointers are CUDA device pointers, "host" pointers are host memory.  All buffers are owned by
 *    the caller; the library borrows them.  W is updated in place.  The context is freed only by
 *    sfb_destroy.  The library allocates no device memory: everything it needs is carved from the
 *    caller's workspace (size from sfb_workspace_bytes).
 *  - W is fp32, row-major [rows][cols]:  MLR classes x features, DML latent x features, SC features x atoms.
 *    cols must be a multiple of 4 and every device pointer 16-byte aligned.
 *  - Samples are worker-major: global pair index i = p*B + b for sample b of worker p.
 *  - All work is enqueued on config.stream.  Calls return 0 or a negative sfb_error; nothing aborts or traps.
 *    Errors detected on the device (a class id out of range, a pipeline wait that ran out) set bits of a
 *    device status word, read with sfb_get_status.
 *  - One context per stream; calls on one context are not re-entrant.
 */
#ifndef SFB_H_
#define SFB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sfb_ctx sfb_ctx;

/* SFB_L2MLR: multiclass logistic regression with the regulariser lam/2 ||W||_F^2, learnt by stochastic dual coordinate
 * ascent (Section 2.1 "Stochastic DCA"; the fourth model of Section 6).  See sfb_sdca_compute_factors. */
enum sfb_model { SFB_MLR = 0, SFB_DML = 1, SFB_SC = 2, SFB_L2MLR = 3 };

/* Operand precision of the matrix products.  The master copy of W is fp32 in every mode.
 * SFB_PREC_BF16: tensor-core products on bf16 operands with fp32 accumulation.  MLR: forward and update
 *                products on single bf16 operands (the label entry of u is kept in fp32).  DML, SC: u is a residual
 *                that cancels, so every product -- the forward W v, the products of the ISTA coder and the update --
 *                runs on the tensor cores with each value carried as a (hi, lo) pair of bf16, three bf16 products
 *                per term (about 2^-16 relative error per product).
 * SFB_PREC_FP32: fp32 operands.  MLR and SFB_L2MLR contexts of at least 2048 x 512 with K >= 128 run their two
 *                products on the tensor cores as SFB_PREC_TF32X3 does; everything else uses fp32 FMA kernels.
 * SFB_PREC_TF32X3: (MLR, SFB_L2MLR) fp32 operands on the tensor cores at any shape: every fp32 value x is carried as
 *                two tf32 words, big = tf32(x) and small = tf32(x - big), and a product runs as
 *                big*big + big*small + small*big with fp32 accumulation (relative error about 2^-21 per product);
 *                softmax, loss and the factors stay in fp32.  SFB_ERR_UNSUPPORTED for the other models.
 * SFB_PREC_FP32_FFMA: fp32 FMA kernels at any shape (the on-device cross-check of the tensor-core paths). */
enum sfb_precision { SFB_PREC_BF16 = 0, SFB_PREC_FP32 = 1, SFB_PREC_TF32X3 = 2, SFB_PREC_FP32_FFMA = 3 };

enum sfb_error {
  SFB_OK = 0,
  SFB_ERR_ARG = -1,          /* null pointer, bad enum, non-positive size                      */
  SFB_ERR_ALIGN = -2,        /* a pointer is not 16-byte aligned                               */
  SFB_ERR_SHAPE = -3,        /* cols not a multiple of 4, worker index out of range, ...       */
  SFB_ERR_WORKSPACE = -4,    /* workspace smaller than sfb_workspace_bytes reports             */
  SFB_ERR_CUDA = -5,         /* a CUDA runtime call failed (see sfb_last_cuda_error)           */
  SFB_ERR_ARCH = -6,         /* the current device is not compute capability 10.x              */
  SFB_ERR_TIMEOUT = -7,      /* a bounded device-side wait gave up (status word)               */
  SFB_ERR_LABEL_RANGE = -8,  /* a class id outside [0, rows) was skipped (status word)         */
  SFB_ERR_STATE = -9,        /* call order: gather before all workers committed, ...           */
  SFB_ERR_UNSUPPORTED = -10, /* this model / precision combination is not built                */
  SFB_ERR_STATIC_LIMIT = -11 /* size beyond what the library's built-in scratch array can hold  */
};

/* Bits of the device status word. */
#define SFB_STATUS_LABEL_RANGE 0x1u
#define SFB_STATUS_TIMEOUT     0x2u
#define SFB_STATUS_SAMPLE_RANGE 0x4u   /* SDCA: a sample id outside [0, sdca_n) was skipped */
#define SFB_STATUS_INDEX_RANGE 0x8u    /* sparse samples: a column index outside [0, cols), or row pointers that do not
                                          describe the stated number of entries; the entry or the sample was skipped */

typedef struct sfb_config {
  int32_t model;          /* enum sfb_model                                                            */
  int32_t precision;      /* enum sfb_precision                                                        */
  int64_t rows, cols;     /* shape of W                                                                */
  int32_t workers;        /* P                                                                         */
  int32_t batch;          /* B; K = P*B                                                                */
  float   eta;            /* W <- W - eta * sum u v^T (a plain sum: fold 1/B or 1/K into eta)          */
  float   dml_margin;     /* hinge margin of dissimilar pairs (Section 2, DML)                         */
  float   sc_lambda;      /* l1 weight of the sparse coder                                             */
  int32_t sc_ista_iters;  /* ISTA iterations per sample, from a = 0                                    */
  float   sc_lipschitz;   /* step is 1/L; <= 0: the library estimates L = ||W||_2^2 by 50 power
                             iterations at the start of every step                                     */
  int32_t sc_prox;        /* 0 none | 1 rescale columns of norm > 1 to norm 1 (Figure 3)               */
  float   sdca_lambda;    /* SFB_L2MLR: weight lam of the regulariser h(W) = lam/2 ||W||_F^2 (> 0)    */
  int64_t sdca_n;         /* SFB_L2MLR: N, the number of training samples (rows of the dual state)     */
  int32_t prox_kind;      /* entry-wise proximal operator applied with the update (Section 2.1, proximal SGD):
                             0 none | 1 h = w ||W||_1: entries shrunk towards 0 by eta*w | 2 h = w/2 ||W||_F^2:
                             entries divided by 1 + eta*w.  Fused into the update pass; for SC it comes before
                             the column rescaling.  Not for SFB_L2MLR (its regulariser lives in the dual).     */
  float   prox_weight;    /* the weight w of that regulariser (>= 0)                                  */
  int64_t csr_nnz_max;    /* MLR: room, in non-zeros per step over all K samples, for samples given in
                             compressed-sparse-row form (sfb_compute_factors_csr); 0: none                */
  int32_t csr_update;     /* which update a step of sparse samples takes: 0 the cheaper one by the library's
                             cost model (non-zeros per column against K) | 1 the sparse one whenever its
                             factor slab fits | 2 always the dense one                                    */
  void*   stream;         /* cudaStream_t                                                              */
} sfb_config;

typedef struct sfb_stats {
  int64_t steps;              /* completed sfb_step / sfb_apply_update calls                           */
  int64_t samples;            /* pairs applied                                                         */
  double  flops;              /* matrix-product flops issued (2*m*n*k each)                            */
  double  gather_bytes;       /* bytes of gathered factors, one copy: K*(rows+cols)*element size        */
  double  gather_bytes_p2p;   /* the paper's peer-to-peer count: P*(P-1)*B*(rows+cols)*element size     */
  double  dense_sync_bytes;   /* what full-matrix sync would move: P*rows*cols*4 (Section 5 cost table) */
  float   ms_factors, ms_gather, ms_update;  /* device time of the last step's phases (CUDA events)     */
  float   last_loss;          /* MLR: mean over the last step's K samples of -log p(y_i); else 0        */
  float   sc_lipschitz;       /* SC: the L = ||W||_2^2 the coder used in the last step                  */
  int64_t kernel_launches;    /* kernels this library has launched in this process                      */
  int64_t copy_pieces;        /* MLR, bf16 mode: 64-byte row pieces of the bf16 operand copy of W that the update
                                 passes went over since sfb_init, and                                          */
  int64_t copy_written;       /* how many of them they rewrote (a piece whose 32 bf16 roundings did not change
                                 already holds bf16 of the new values and is left alone)                      */
  int64_t sparse_updates;     /* steps whose update summed only the non-zeros of sparse samples                */
} sfb_stats;

/* Bytes of device workspace a context with this config needs.  Host-only; no CUDA call. */
int sfb_workspace_bytes(const sfb_config* cfg, size_t* out_bytes);

/* Create a context over caller-owned W_dev [rows x cols] fp32 and workspace_dev.  Enqueues the set-up
 * work (status word clear, bf16 shadow of W in bf16 mode) on cfg->stream.  Problem (P), Section 2. */
int sfb_init(const sfb_config* cfg, float* W_dev, void* workspace_dev, size_t workspace_bytes, sfb_ctx** out);

/* Sufficient factors of worker `worker` (0..P-1; X_dev is that worker's [B x in_dim] fp32 block), or of all
 * P workers at once (worker = -1; X_dev is [K x in_dim]).  in_dim = cols (MLR, DML) or rows (SC).
 *   MLR: labels_dev = int32 class ids;   u = softmax(W x) - onehot(y), v = x       (Sections 1, 2.1)
 *   DML: Y_dev = pair partner, labels_dev = 1 similar / 0 dissimilar;
 *        v = x - y, u = 2 W v (similar), -2 W v if ||W v||^2 < margin else 0       (Section 2, DML)
 *   SC : v = a = ISTA code of x, u = W a - x                                        (Figure 3)
 * Factors are written at the worker's row offset p*B of the gathered buffers.  All P workers of a step see the
 * same W (bulk-synchronous consistency, Section 4.1).
 * Copies of W that the library derives: in bf16 mode the forward product reads a bf16 operand copy of W.  DML and SC
 * rebuild theirs from W in the first factors call of every step.  MLR (and the tensor-core fp32 mode, whose copy is
 * the pair of tf32 words per entry) builds it once in sfb_init and afterwards the
 * update pass rewrites it together with W (W makes one trip through the SM per step), so it tracks every change the
 * LIBRARY makes to W -- but not writes the caller makes to W_dev between steps (loading weights, rescaling, a prox of
 * its own): after such a write call sfb_refresh_operands, or the next forward product runs on the stale copy. */
int sfb_compute_factors(sfb_ctx* ctx, int32_t worker, const float* X_dev, const float* Y_dev,
                        const int32_t* labels_dev);

/* ---- sparse sufficient factors (MLR) --------------------------------------------------------------------------------
 * Section 6: the features of the paper's data sets are sparse; the factor v_i = a_i of such a sample is its (index,
 * value) pairs (Section 3: what a worker broadcasts).  sfb_compute_factors_csr is sfb_compute_factors for samples in
 * compressed-sparse-row form: sample i of the call holds the entries indices_dev[indptr_dev[i] .. indptr_dev[i+1]) /
 * values_dev[same range], column indices int32 in [0, cols), distinct within a sample, in any order; indptr_dev has
 * B + 1 (worker >= 0) or K + 1 (worker = -1) int64 entries, and nnz = indptr[last] - indptr[0] is stated by the caller
 * (the library does not read device memory on the host).  The entries of all workers of a step must fit
 * cfg.csr_nnz_max (SFB_ERR_SHAPE otherwise; SFB_ERR_UNSUPPORTED when it is 0 or the model is not SFB_MLR).  A worker
 * commits once per step in this form (SFB_ERR_STATE on a second call).  A column index out of range, or row pointers
 * that are not ascending within [indptr[0], indptr[0] + nnz], set SFB_STATUS_INDEX_RANGE and the entry (the sample) is
 * left out.  All arrays are copied or consumed before the call returns control of them to the stream order: they may
 * be reused once later work on the stream may overwrite them.
 *
 * u is computed as for dense samples.  The logits need every column of W (the non-zero columns of a mini-batch cover
 * it), so in the tensor-core modes the forward product is the dense one over the scattered samples; in the fp32 FMA
 * mode it is a row-wise product over the non-zeros (z_ij = sum_t x_it W[j][c_it], rows of W held on chip, cols up to
 * about 55,000; the dense FMA product beyond).
 * When every worker of the step committed in this form, sfb_gather_factors builds the column-major form of the K
 * samples (entries of a column in ascending sample order, so the result does not depend on scheduling) and
 * sfb_apply_update sums, per entry of W, only the samples that have a non-zero in that column:
 *     W[j][d] <- prox( W[j][d] - eta * sum_{i : x_id != 0} u_ij x_id ),
 * one pass over W as in the dense update, the derived operand copies of W rewritten with it.  sfb_stats.gather_bytes
 * then counts K*rows*element size for the u and 8 bytes per non-zero for the v.  A mini-batch too large for the
 * kernel's on-chip factor slab (K above about 1200 in the fp32 modes, 2400 in bf16 mode) takes the dense update, and
 * so does, unless cfg.csr_update says otherwise, one whose columns hold so many non-zeros that the tensor-core update
 * over the scattered samples is the faster of the two (in bf16 mode from about 2 non-zeros per column at K = 1024; in
 * the fp32 modes from about 30). */
int sfb_compute_factors_csr(sfb_ctx* ctx, int32_t worker, const int64_t* indptr_dev, const int32_t* indices_dev,
                            const float* values_dev, int64_t nnz, const int32_t* labels_dev);

/* sfb_compute_factors_csr(worker = -1) -> sfb_gather_factors -> sfb_apply_update. */
int sfb_step_csr(sfb_ctx* ctx, const int64_t* indptr_dev, const int32_t* indices_dev, const float* values_dev,
                 int64_t nnz, const int32_t* labels_dev);

/* ---- l2-regularised MLR by stochastic dual coordinate ascent (model SFB_L2MLR) ------------------------------------
 * Section 2.1 "Stochastic DCA": with the dual matrix U = [u_1 .. u_N], Z = 1/N U A^T and W = grad h^*(Z) = Z / lam, a
 * step picks samples i, finds the change du_i that minimises the dual (D) over u_i with the other dual vectors fixed,
 * and applies  u_i <- u_i - du_i,  Z <- Z - 1/N du_i a_i^T,  W <- grad h^*(Z).  The sufficient factors of the step are
 * (du_i, a_i) (Section 3: "the above procedure is instead used to broadcast SFs for the auxiliary matrix Z").
 *
 * Dual state: the caller owns Q_dev [sdca_n x rows] fp32 with rows q_i = e_{y_i} - u_i, points of the probability
 * simplex (for the multiclass logistic loss f_i^*(-u_i) = sum_j q_ij log q_ij); q_i = e_{y_i} (u_i = 0) with W = 0 is
 * the usual start.  The caller keeps W_dev = 1/(lam N) sum_i (e_{y_i} - q_i) a_i^T consistent with it at set-up; the
 * steps keep it so.
 *
 * sfb_sdca_compute_factors: for every sample of the worker (or of all workers, worker = -1), against the same W:
 *     z = W a_i,  kappa = ||a_i||^2 / (lam N),  q_new = argmin over the simplex of
 *         sum_j q_j log q_j - q.(z + kappa q_old) + kappa/2 ||q||^2
 *     (stationarity: log q_j + kappa q_j = z_j + kappa q_old_j - nu, sum_j q_j = 1; solved by a safeguarded Newton
 *     iteration on nu with a Newton solve per class), du_i = q_new - q_old, and, averaging the K changes of a
 *     mini-batch with the weight eta of the config (Section 3, "Mini-batch proximal SGD/SDCA": 1/K sum u_i v_i^T, so
 *     eta = 1/K; eta = 1 with K = 1 is the single-sample step),   q_i <- q_old + eta * du_i   in Q_dev.
 *     sample_ids_dev [B or K] int32: the rows of Q_dev of the samples, distinct within a step; an id outside
 *     [0, sdca_n) sets SFB_STATUS_SAMPLE_RANGE and contributes nothing.  labels_dev: class ids.
 * sfb_gather_factors, then sfb_apply_update:   W <- W - eta/(lam N) * sum_i du_i a_i^T   (the fused update pass).
 * sfb_sdca_step = the three calls for all K samples.  sfb_compute_factors / sfb_step on such a context and these
 * calls on any other return SFB_ERR_UNSUPPORTED; SFB_ERR_STATE before sfb_sdca_set_dual. */
int sfb_sdca_set_dual(sfb_ctx* ctx, float* Q_dev, int64_t n_samples);
int sfb_sdca_compute_factors(sfb_ctx* ctx, int32_t worker, const float* X_dev, const int32_t* labels_dev,
                             const int32_t* sample_ids_dev);
int sfb_sdca_step(sfb_ctx* ctx, const float* X_dev, const int32_t* labels_dev, const int32_t* sample_ids_dev);

/* The two sides of the broadcast (Section 3: every worker sends its sufficient factors to the others and applies the
 * ones it receives).
 * sfb_export_factors: the fp32 factors of worker `worker` as they are sent, U_out_dev [B x rows], V_out_dev [B x cols]
 * (pair-major, dense rows).  Valid between that worker's sfb_compute_factors and the update (SFB_ERR_STATE otherwise).
 * In bf16 mode MLR holds logits and log-partitions rather than u:  u_ij = exp(z_ij - lse_i) - [j = y_i]  is formed here
 * in fp32.
 * sfb_set_factors: B pairs U_dev, V_dev of the same form, computed elsewhere -- by another replica, under another
 * consistency model (Section 4.1), on another machine -- take worker `worker`'s place in the gathered buffers and the
 * worker counts as committed.  For MLR in bf16 mode a received u is split the way a local one is: the class of the
 * sample is read off it (u = p - onehot(y) has its one negative, hence smallest, entry at y), that entry goes to W in
 * fp32, the rest as bf16.
 * Both: SFB_ERR_UNSUPPORTED for SFB_L2MLR. */
int sfb_export_factors(sfb_ctx* ctx, int32_t worker, float* U_out_dev, float* V_out_dev);
int sfb_set_factors(sfb_ctx* ctx, int32_t worker, const float* U_dev, const float* V_dev);

/* Changes the step size eta of the following updates (step-size schedules, e.g. the decreasing eta_c of the
 * convergence analysis in Section 5).  SFB_ERR_STATE between the factors of a step and their update. */
int sfb_set_eta(sfb_ctx* ctx, float eta);

/* The broadcast of Section 3 as an on-device gather: after it, U [K x rows] and V [K x cols] of all P workers
 * sit in one buffer in the operand layout of the update.  Fails with SFB_ERR_STATE unless every worker has
 * computed its factors since the last update.  Accounts the bytes of Section 5's cost table. */
int sfb_gather_factors(sfb_ctx* ctx);

/* Reconstruct and apply:  W <- W - eta * U^T V  in one pass over W, then the proximal operator (SC, when
 * sc_prox = 1).  Section 2.1 (proximal SGD) and Figure 1. */
int sfb_apply_update(sfb_ctx* ctx);

/* Re-derives the library's operand copies of W from the caller's W_dev (enqueued on the stream): to be called after
 * the caller itself has written W_dev between two steps.  MLR in bf16 mode: one conversion pass over W (reads 4,
 * writes 2 bytes per entry; 8 bytes in the tensor-core fp32 mode); a no-op for the other models and for the FFMA
 * kernels.  SFB_ERR_STATE in the middle of a step. */
int sfb_refresh_operands(sfb_ctx* ctx);

/* Measurement hook (the paper has no counterpart): applies the factors gathered by the last completed step once
 * more, W <- prox(W - eta * U^T V) with the same U and V, so that the reconstruct-and-apply pass can be timed on its
 * own, back to back.  It moves W a second time by the same update: for benchmarks, not for training.  Counts flops
 * but no step.  SFB_ERR_STATE before the first completed step or while a step is under way. */
int sfb_replay_update(sfb_ctx* ctx);

/* compute_factors(all workers) + gather + apply_update for K samples resident on the device. */
int sfb_step(sfb_ctx* ctx, const float* X_dev, const float* Y_dev, const int32_t* labels_dev);

/* The same step for callers whose minibatch lives in HOST memory (pinned memory recommended): copies
 * X_host [K x in_dim] (and Y_host, labels_host when the model uses them) to staging buffers inside the
 * workspace, runs the step, copies the step's mean loss (MLR; 0 otherwise) and the status word back, and
 * waits for the stream.  loss_out and status_out may be NULL. */
int sfb_step_host(sfb_ctx* ctx, const float* X_host, const float* Y_host, const int32_t* labels_host,
                  float* loss_out, uint32_t* status_out);

/* ---- The parameter matrix partitioned by rows over several contexts (multiclass logistic regression) -------------
 * Section 3 assumes every worker holds a full copy of W and notes (footnote to the set-up of SFB) that a W too large
 * for that can be partitioned across machines.  On GPUs the partition also removes the redundant work of the replicas:
 * each context (one per GPU) owns rows [row_offset, row_offset + rows) of a matrix with global_rows classes, computes
 * the logits of ALL K samples against its own rows, and updates only those rows.  The softmax couples the shards
 * through one small exchange per step, which the caller performs (an all-gather of K*16 bytes per shard):
 *
 *   sfb_set_row_shard       once after sfb_init (rows of the config = this shard's row count; class ids stay global)
 *   sfb_forward_partials    logits of the K samples against this shard's rows and, per sample i, the shard's softmax
 *                           partial  partials_dev[i] = { m_i, s_i, zy_i, has_i }  (4 floats):  m_i = max_j z_ij and
 *                           s_i = sum_j exp(z_ij - m_i) over the shard's rows j;  zy_i = z_{i,y_i} and has_i = 1 if
 *                           the shard owns class y_i, else 0 and 0.   X_dev [K x cols], labels_dev [K] (global ids).
 *   (caller)                gathers the partials of all shards into partials_all_dev [shards][K][4], shard order
 *   sfb_finish_factors      log-partition lse_i = M + log sum_g s_gi exp(m_gi - M), M = max_g m_gi;  this shard's part
 *                           of the factor, u_ij = exp(z_ij - lse_i) - [j = y_i] (Section 2.1), v_i = x_i;  the loss
 *                           lse_i - z_{i,y_i}, identical on every shard.  A class id no shard owns sets
 *                           SFB_STATUS_LABEL_RANGE.  Afterwards every worker counts as committed:
 *   sfb_gather_factors, sfb_apply_update   as for an unsharded context, on this shard's rows.
 *
 * With one shard (row_offset 0, global_rows = rows) the three calls compute what sfb_compute_factors(-1) computes.
 * Errors: SFB_ERR_UNSUPPORTED for other models, SFB_ERR_STATE for calls out of order, SFB_ERR_SHAPE for a row range
 * outside [0, global_rows). */
int sfb_set_row_shard(sfb_ctx* ctx, int64_t row_offset, int64_t global_rows);
int sfb_forward_partials(sfb_ctx* ctx, const float* X_dev, const int32_t* labels_dev, float* partials_dev);
int sfb_finish_factors(sfb_ctx* ctx, const float* partials_all_dev, int32_t shards);

/* The same partition for DML (Section 2, DML; W is the k x D map): a context holds latent rows [row_offset, row_offset +
 * rows) of W (sfb_set_row_shard), z_i = W v_i splits over the shards and the hinge of a dissimilar pair needs
 * ||z_i||^2 = the sum over the shards of ||z_i,shard||^2.  sfb_forward_partials_pairs: v = x - y and this shard's z for all
 * K pairs, partials_dev [K] fp32 = this shard's squared norms.  sfb_finish_factors with partials_all_dev [shards][K] (all
 * shards' values, shard-major, summed in that order): u = 2 z (similar), -2 z if ||z||^2 < margin else 0.  Then
 * sfb_gather_factors and sfb_apply_update as usual; u and the update stay local to the shard. */
int sfb_forward_partials_pairs(sfb_ctx* ctx, const float* X_dev, const float* Y_dev, const int32_t* similar_dev,
                               float* partials_dev);

/* Full-matrix-synchronisation comparison path (Section 3 "SFB vs client-server", Section 5): every worker
 * materialises its dense update U_p^T V_p in scratch, the P matrices are summed, and W <- W - eta * sum.
 * scratch_dev: at least 2*rows*cols*4 bytes.  Same result as sfb_step up to summation order.  Built for
 * SFB_PREC_FP32 contexts only (a comparison path, not a product path); SFB_ERR_UNSUPPORTED otherwise. */
int sfb_dense_sync_step(sfb_ctx* ctx, const float* X_dev, const float* Y_dev, const int32_t* labels_dev,
                        float* scratch_dev, size_t scratch_bytes);

/* The gathered factor buffers of the last gather, for inspection.  dtype: 0 = fp32, 1 = bf16.
 * layout: 0 = pair-major (U [K x ldu], V [K x ldv]); 1 = transposed (U^T [rows x ldu], V^T [cols x ldv]).
 * DML and SC return their fp32 pair-major factors in both modes.
 * MLR in bf16 mode splits u_i = p_i - onehot(y_i) in two: the buffer holds the probabilities p_i in bf16 with a 0
 * at the label entry (i, y_i); that entry, p_iy - 1, is kept in fp32 and applied to row y_i of W separately
 * (bf16 cannot hold it when p_iy is close to 1). */
int sfb_get_factors(sfb_ctx* ctx, const void** U_dev, const void** V_dev, int32_t* dtype, int32_t* layout,
                    int64_t* ldu, int64_t* ldv);

/* The library's operand copy of W, for inspection: MLR in bf16 mode: dtype 1, the bf16 matrix [rows x ld]; the
 * tensor-core fp32 mode: dtype 2, fp32 words [rows x ld] holding tf32(w) at column c and tf32(w - tf32(w)) at column
 * ld/2 + c.  SFB_ERR_UNSUPPORTED where no persistent copy exists (the other models rebuild theirs every step; the FFMA
 * kernels read W itself). */
int sfb_get_operand_copy(sfb_ctx* ctx, const void** copy_dev, int32_t* dtype, int64_t* ld);

/* Waits for the stream, then fills the counters. */
int sfb_get_stats(sfb_ctx* ctx, sfb_stats* out);

/* Waits for the stream, returns the device status word and clears it. */
int sfb_get_status(sfb_ctx* ctx, uint32_t* status_out);

const char* sfb_strerror(int code);

/* The cudaError_t of the last failed CUDA call made through this context (0 if none). */
int sfb_last_cuda_error(sfb_ctx* ctx);

int sfb_destroy(sfb_ctx* ctx);

/* Self-test of the failure-detection path (no counterpart in the paper).  Every wait inside the tensor-core kernels
 * is bounded: after a cycle limit it gives up, the kernel sets SFB_STATUS_TIMEOUT in the status word, releases what
 * it holds and returns, so a pipeline fault surfaces as a status bit and the context stays usable.  This call
 * enqueues, on the context's stream, a one-block kernel that runs that same wait on a barrier nothing ever arrives
 * at, with a limit of max_cycles SM clock cycles (1 .. 2e9; about 1e6 = well under a millisecond).  It holds no copy
 * in flight and no tensor memory.  Afterwards sfb_get_status reports SFB_STATUS_TIMEOUT (and clears it); later steps
 * on the context are unaffected.  The limits of the product kernels are not changed by this call. */
int sfb_selftest_wait_timeout(sfb_ctx* ctx, int64_t max_cycles);

/* Largest column count sfb_prox_columns_noalloc accepts. */
#define SFB_NOALLOC_MAX_COLS 16384

/* The column prox of sparse coding on its own, for callers that may not allocate:
 *     every column b of W_dev [rows x cols] (fp32, row-major) with ||b||_2 > 1 becomes b / ||b||_2,
 * the same two kernels, in the same order, that sfb_apply_update runs for SFB_SC with sc_prox = 1.  (The paper
 * has no counterpart of this entry point: it exists for the integration cases below, not for the method.)
 *
 * Who needs it: code that runs where a device allocation is off the table -- a plug-in living inside another
 * program's fixed memory budget, a service whose device memory was carved up at start-up and is policed, or a
 * latency-bound loop that cannot afford the device-wide synchronisation an allocation can bring with it.  Those
 * callers cannot build an sfb_ctx either (it wants a workspace from them).  This call needs no context and no
 * workspace: its only scratch, the per-slab column sums (64 x SFB_NOALLOC_MAX_COLS doubles, 8 MB), is an array
 * built into the library.  Every GPU that loads the library holds those 8 MB until the process ends.
 *
 *  - It calls no allocating routine (no cudaMalloc / cudaFree, no library that allocates); the caller passes
 *    W_dev (updated in place, 16-byte aligned, cols a multiple of 4) and the stream the work is enqueued on.
 *  - cols > SFB_NOALLOC_MAX_COLS is refused with SFB_ERR_STATIC_LIMIT and nothing is launched.
 *  - The first call on each device looks up the array's device address (once per device, with that device
 *    current).  The CUDA runtime may load this library's device code on that device at that moment, the 8 MB array
 *    included: a one-off, driver-side set-up cost that is not a cudaMalloc but can synchronise the device.  Make
 *    that first call at start-up, outside any stream capture and outside latency-critical sections.
 *  - W_dev must be device memory of the CURRENT device (the array address is per device); anything else is refused
 *    with SFB_ERR_ARG.
 *  - All calls on one device share the one array.  Nothing in it has to start at zero -- each call overwrites
 *    every entry it later reads -- but two calls whose kernels overlap on the GPU (different streams, no
 *    ordering between them) race on it and both results are then undefined.  Order them on one stream or with
 *    events. */
int sfb_prox_columns_noalloc(float* W_dev, int64_t rows, int64_t cols, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SFB_H_ */
