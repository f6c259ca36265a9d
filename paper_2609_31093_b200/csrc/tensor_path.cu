#include "pisa_tensor.cuh"

namespace pisa {

bool tensor_path_supported(const Geometry&, int) { return false; }
size_t tensor_route_workspace_bytes(const Geometry&) { return 0; }
size_t tensor_bsa_workspace_bytes(const Geometry&) { return 0; }
int tensor_route(const Geometry&, int, const void*, const void*, const void*, int32_t*, float*, void*, int32_t*,
                 cudaStream_t) { return PISA_ERR_UNSUPPORTED; }
int tensor_bsa(const Geometry&, int, const void*, const void*, const void*, const int32_t*, void*, float*, void*,
               int32_t*, cudaStream_t) { return PISA_ERR_UNSUPPORTED; }

}  // namespace pisa
