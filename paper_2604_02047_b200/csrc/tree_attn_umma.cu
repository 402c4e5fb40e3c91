// placeholder until the tcgen05 kernel lands
#include "goose_internal.cuh"
namespace goose {
cudaError_t init_umma_kernel() { return cudaSuccess; }
int auto_attn_impl(const goose_ctx*, int, int, int) { return GOOSE_ATTN_MMA; }
cudaError_t launch_tree_attn_umma(goose_ctx*, const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*, int64_t,
                                  const int64_t*, const int32_t*, const int32_t*, int, int, int, float,
                                  __nv_bfloat16*, float*, cudaStream_t) { return cudaErrorNotSupported; }
}
