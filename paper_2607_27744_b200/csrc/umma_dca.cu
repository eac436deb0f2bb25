#include "rocs_internal.h"
namespace rocs {
bool umma_dca_supported(int32_t, int32_t, int32_t) { return false; }
rocs_status_t umma_dca(const rocs_plan*, int32_t, int32_t, int32_t, float, const void*, const void*, const void*, const int32_t*, int64_t, void*, cudaStream_t) { return ROCS_ERR_UNSUPPORTED; }
}
