// Tensor-core (bf16 operand) path of the SFB step: hooks called by the C ABI layer, and the host-side helpers
// the tensor-core translation units share (sfb_tc.cu: factors and forward product; sfb_update.cu: the update).
#pragma once
#include <cuda.h>

#include "sfb_internal.h"

namespace sfb {

// Appends the bf16-mode buffers to the workspace layout.
void tc_extend_layout(const sfb_config& c, Layout& L, size_t& off);
// fp32 mode on the tensor cores (MLR and its SDCA form): layout, factors, operand packing of the gathered pairs, update.
void tc32_extend_layout(const sfb_config& c, Layout& L, size_t& off);
int tc32_factors(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const int32_t* labels, const int32_t* sdca_ids,
                 float inv_lam_n);
int tc32_forward_partials(sfb_ctx* ctx, const float* X, const int32_t* labels, float* part_out);
int tc32_finish_factors(sfb_ctx* ctx, const float* parts, int shards);
int tc32_gather(sfb_ctx* ctx);
int tc32_update(sfb_ctx* ctx);
int tc_init(sfb_ctx* ctx);
void tc_destroy(sfb_ctx* ctx);
// Rebuilds the bf16 operand copy of W from the caller's fp32 W (MLR; the other models rebuild theirs every step).
int tc_refresh_operands(sfb_ctx* ctx);
// dml_norm_out (DML, row-sharded form; may be null): receives ||z_i||^2 of this context's rows and z stays unscaled.
int tc_factors(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const float* Y, const int32_t* labels,
               float* dml_norm_out = nullptr);
// Row-sharded MLR: logits and softmax partials of all K samples against this context's rows; then the factors from
// the partials of all shards.
int tc_forward_partials(sfb_ctx* ctx, const float* X, const int32_t* labels, float* part_out);
int tc_finish_factors(sfb_ctx* ctx, const float* parts, int shards);
int tc_sdca_factors(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const int32_t* labels, const int32_t* ids,
                    float inv_lam_n);
// MLR, bf16 mode: a worker's factors in fp32 as they are sent, and received fp32 factors put into the bf16 layout.
int tc_export_factors(sfb_ctx* ctx, int64_t off, int64_t n, float* U_out, float* V_out);
int tc_import_factors(sfb_ctx* ctx, int64_t off, int64_t n, const float* U_in, const float* V_in);
int tc_gather(sfb_ctx* ctx);
int tc_update(sfb_ctx* ctx);
int tc_get_factors(sfb_ctx* ctx, const void** U, const void** V, int32_t* dtype, int32_t* layout, int64_t* ldu,
                   int64_t* ldv);

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcState {
  EncodeTiledFn encode;      // cuTensorMapEncodeTiled, obtained through the runtime's driver entry point query
  int sms;                   // multiprocessors of the device
  int max_pairs;             // CTA pairs (clusters of 2) of the update kernel that can be resident at once
};

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

// 2-D row-major tensor [outer x inner] with row pitch `pitch_bytes`, box [box_outer x box_inner], 128-byte swizzle.
inline bool make_map(const TcState* st, CUtensorMap* m, CUtensorMapDataType dt, void* base, int64_t inner,
                     int64_t outer, int64_t pitch_bytes, int box_inner, int box_outer) {
  if (inner <= 0 || outer <= 0) return false;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(inner), static_cast<cuuint64_t>(outer)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(pitch_bytes)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(box_inner), static_cast<cuuint32_t>(box_outer)};
  cuuint32_t estr[2] = {1, 1};
  return st->encode(m, dt, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Fills st->max_pairs (occupancy query of the update kernel); defined beside that kernel.
int tc_update_init(sfb_ctx* ctx, TcState* st);

}  // namespace sfb
