#include "sfb_tc.h"
namespace sfb {
void tc_extend_layout(const sfb_config&, Layout&, size_t&) {}
int tc_init(sfb_ctx*) { return SFB_ERR_UNSUPPORTED; }
void tc_destroy(sfb_ctx*) {}
int tc_factors(sfb_ctx*, int64_t, int64_t, const float*, const float*, const int32_t*) { return SFB_ERR_UNSUPPORTED; }
int tc_gather(sfb_ctx*) { return SFB_ERR_UNSUPPORTED; }
int tc_update(sfb_ctx*) { return SFB_ERR_UNSUPPORTED; }
int tc_after_update(sfb_ctx*) { return SFB_ERR_UNSUPPORTED; }
int tc_get_factors(sfb_ctx*, const void**, const void**, int32_t*, int32_t*, int64_t*, int64_t*) { return SFB_ERR_UNSUPPORTED; }
}
