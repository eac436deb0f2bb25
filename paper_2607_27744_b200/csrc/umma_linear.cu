#include "rocs_internal.h"
namespace rocs {
bool umma_linear_supported(int64_t, int32_t, int32_t, int64_t, int64_t, int64_t, bool) { return false; }
rocs_status_t umma_linear(int64_t, int32_t, int32_t, const void*, int64_t, const void*, int64_t, const float*, const float*, int64_t, const int32_t*, int, void*, int64_t, bool, cudaStream_t) { return ROCS_ERR_UNSUPPORTED; }
}
