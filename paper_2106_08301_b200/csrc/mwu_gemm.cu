// placeholder until the tensor-core kernel lands
#include "mwu_common.cuh"
extern "C" int mwu_gemm(const mwu_proj_desc *, const void *, const void *, int64_t, int64_t, void *,
                        int64_t, int32_t, uint32_t *, void *) { return MWU_ERR_CUDA; }
extern "C" int mwu_conv_implicit(const mwu_proj_desc *, const void *, const void *, int32_t, int32_t,
                                 int32_t, int32_t, int32_t, int32_t, int32_t, int32_t, void *, int32_t,
                                 uint32_t *, void *) { return MWU_ERR_CUDA; }
