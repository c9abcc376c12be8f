// placeholder until the tcgen05 engine lands
#include "common.cuh"
namespace rad {
bool tc_shape_ok(int64_t, int64_t, int64_t, const void*, int64_t, const void*, int64_t) { return false; }
int tc_forward(int, int64_t, int64_t, int64_t, const void*, int64_t, const void*, int64_t, const float*, void*,
               int64_t, float*, int64_t, void*, int64_t, uint32_t*, int32_t*, cudaStream_t) { return RAD_EUNSUPPORTED; }
int tc_input_grad(int64_t, int64_t, int64_t, const void*, int64_t, const void*, int64_t, const uint32_t*,
                  const void*, int64_t, void*, int64_t, int32_t*, cudaStream_t) { return RAD_EUNSUPPORTED; }
int tc_weight_grad(const rad_store*, const void*, int64_t, int64_t, float*, int64_t, void*, int64_t, int32_t*,
                   cudaStream_t) { return RAD_EUNSUPPORTED; }
int64_t tc_weight_grad_workspace(const rad_store*, int64_t) { return 0; }
}
