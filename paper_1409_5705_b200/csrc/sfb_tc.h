// Tensor-core (bf16 operand) path of the SFB step: hooks called by the C ABI layer.
#pragma once
#include "sfb_internal.h"

namespace sfb {

// Appends the bf16-mode buffers to the workspace layout.
void tc_extend_layout(const sfb_config& c, Layout& L, size_t& off);
int tc_init(sfb_ctx* ctx);
void tc_destroy(sfb_ctx* ctx);
int tc_factors(sfb_ctx* ctx, int64_t off, int64_t n, const float* X, const float* Y, const int32_t* labels);
int tc_gather(sfb_ctx* ctx);
int tc_update(sfb_ctx* ctx);
int tc_after_update(sfb_ctx* ctx);
int tc_get_factors(sfb_ctx* ctx, const void** U, const void** V, int32_t* dtype, int32_t* layout, int64_t* ldu,
                   int64_t* ldv);

}  // namespace sfb
