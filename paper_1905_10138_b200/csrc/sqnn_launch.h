// Internal: launch helpers shared by the kernel translation units.
#pragma once
#include "sqnn.h"
#include "sqnn_decode.cuh"

namespace sqnn {
int fill_decode_args(const sqnn_desc *d, const void *d_blob, uint32_t *d_status, DecodeArgs *A);
int sm_count();
// Raises a kernel's dynamic shared-memory limit when `smem` needs it; remembered per kernel and
// device so that repeated launches cost nothing on the host.
int ensure_dynamic_smem(const void *kernel, size_t smem);
// Queues the packed-bits decode of every plane into `d_out` (n_q * ceil(mn/64) uint64).
int decode_bits_dispatch(const DecodeArgs &A, void *d_out, cudaStream_t st);
size_t mma_workspace_bytes(const sqnn_desc *desc, uint32_t batch);
int mma_dispatch(const sqnn_desc *desc, const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha,
                 const void *d_x, int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, void *d_workspace,
                 cudaStream_t st);

// A device entry point: an NVTX range for its duration on the host, and in checked mode
// (SQNN_DEBUG_CHECKS=1) the wait for the stream and the translation of what it left behind.
class ApiScope {
  public:
    explicit ApiScope(const char *name);
    ~ApiScope();
    ApiScope(const ApiScope &) = delete;
    ApiScope &operator=(const ApiScope &) = delete;
    // rc of the queueing code -> what the entry point returns
    int finish(int rc, const uint32_t *d_status, cudaStream_t st) const;
};
}  // namespace sqnn
