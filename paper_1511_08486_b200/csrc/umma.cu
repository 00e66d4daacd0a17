#include "umma_api.cuh"
namespace sfb {
struct UmmaPlan { int dummy; };
int umma_plan_create(const sfb_desc&, const Layout&, float*, int, __nv_bfloat16*, UmmaPlan**) { return SFB_ERR_UNSUPPORTED; }
void umma_plan_destroy(UmmaPlan*) {}
int umma_forward(UmmaPlan*, cudaStream_t, const void*, const __nv_bfloat16*, const void*, const sfb_aux*, RowMap, RowMap, RowMap, int*) { return SFB_ERR_UNSUPPORTED; }
int umma_apply(UmmaPlan*, cudaStream_t, void*, __nv_bfloat16*, const void*, float, int, const int*) { return SFB_ERR_UNSUPPORTED; }
}
