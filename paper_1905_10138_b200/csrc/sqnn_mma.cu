// Fused decode + tcgen05 product for batch >= 16 (placeholder until the kernel lands).
#include "sqnn_launch.h"
namespace sqnn {
size_t mma_workspace_bytes(const sqnn_desc *, uint32_t) { return 0; }
int mma_dispatch(const sqnn_desc *, const DecodeArgs &, const uint64_t *, const float *, const void *, int64_t,
                 uint32_t, float *, int64_t, void *, cudaStream_t) { return SQNN_E_UNSUPPORTED; }
}
