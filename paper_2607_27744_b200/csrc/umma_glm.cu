#include "rocs_internal.h"
namespace rocs {
bool umma_glm_supported(int32_t, int32_t, int32_t, int32_t, int32_t) { return false; }
rocs_status_t umma_glm(const rocs_plan*, int32_t, int32_t, int32_t, const void*, const void*, const void*, int32_t, int32_t, void*, void*, const float*, cudaStream_t) { return ROCS_ERR_UNSUPPORTED; }
}
