// C entry points of the device side: argument checks and dispatch on the network shape.
#include "sqnn.h"
#include "sqnn_decode.cuh"
#include <cstdlib>
#include <nvtx3/nvToolsExt.h>
#include "sqnn_launch.h"
#include "sqnn_shapes.h"

#include <cuda_runtime.h>

#include <map>
#include <mutex>
#include <utility>

namespace sqnn {

template <int N_OUT, int N_IN>
int decode_shape(const DecodeArgs &A, sqnn_out_mode mode, const uint64_t *d_mask, const float *d_alpha,
                 uint64_t n, void *d_out, cudaStream_t st);
template <int N_OUT, int N_IN>
int gemv_shape(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x, int x_dtype,
               int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t m, uint64_t n, cudaStream_t st);
#define SQNN_DECLARE(NO, NI)                                                                                  \
    template <> int decode_shape<NO, NI>(const DecodeArgs &, sqnn_out_mode, const uint64_t *, const float *,  \
                                         uint64_t, void *, cudaStream_t);                                     \
    template <> int gemv_shape<NO, NI>(const DecodeArgs &, const uint64_t *, const float *, const void *, int, \
                                       int64_t, uint32_t, float *, int64_t, uint64_t, uint64_t, cudaStream_t);
SQNN_FOR_SHAPES(SQNN_DECLARE)
SQNN_DECLARE(0, 0)
#undef SQNN_DECLARE

int fill_decode_args(const sqnn_desc *d, const void *d_blob, uint32_t *d_status, DecodeArgs *A)
{
    if (!d || !d_blob) return SQNN_E_INVALID_ARG;
    if (((uintptr_t)d_blob & 15) != 0) return SQNN_E_INVALID_ARG;
    if (d->n_out < 1 || d->n_out > SQNN_MAX_N_OUT || d->n_in < 1 || d->n_in > SQNN_MAX_N_IN ||
        d->n_q < 1 || d->n_q > SQNN_MAX_PLANES || d->m == 0 || d->n == 0 ||
        d->tile_slices != SQNN_TILE_SLICES || d->slices_padded % SQNN_PAD_SLICES != 0)
        return SQNN_E_INVALID_ARG;
    const uint8_t *b = (const uint8_t *)d_blob;
    A->mn = d->m * d->n;
    A->words64 = (A->mn + 63) / 64;
    A->n_out = d->n_out; A->n_in = d->n_in; A->n_q = d->n_q;
    A->KT = format_tiles_per_kernel_tile(d->n_out);
    A->G = 8 * A->KT;
    A->W = A->G * d->n_out / 32;
    A->ktiles = d->slices_padded / (32ull * A->G);
    A->nw = entry_words(d->n_out);
    A->nwp = entry_words_padded(d->n_out);
    A->nchunks = table_chunks(d->n_in, A->nwp);
    A->cb = chunk_bits(d->n_in, A->nwp);
    A->tab_words = table_words(d->n_out, d->n_in);
    // the table geometry is a fixed function of the shape; a descriptor that says otherwise is not ours
    if (d->tab_entry_words != A->nwp || d->tab_chunks != A->nchunks || d->tab_chunk_bits != A->cb ||
        d->tables_bytes != (uint64_t)A->tab_words * 4 || d->off_tables % 16 != 0)
        return SQNN_E_INVALID_ARG;
    A->tab = (const uint32_t *)(b + d->off_tables);
    A->status = d_status;
    for (uint32_t i = 0; i < d->n_q; ++i) {
        if (d->off_wc[i] % 16 || d->off_idx[i] % 16 || d->off_pp[i] % 16 || d->n_pp[i] > 0xffffffffull)
            return SQNN_E_INVALID_ARG;
        A->pl[i].wc = (const uint32_t *)(b + d->off_wc[i]);
        A->pl[i].idx = (const uint32_t *)(b + d->off_idx[i]);
        A->pl[i].pp = (const uint16_t *)(b + d->off_pp[i]);
        A->pl[i].n_pp = (uint32_t)d->n_pp[i];
    }
    for (uint32_t i = d->n_q; i < 8; ++i) A->pl[i] = A->pl[0];
    return SQNN_OK;
}

int ensure_dynamic_smem(const void *kernel, size_t smem)
{
    if (smem <= 48 * 1024) return SQNN_OK;
    static std::mutex mu;
    static std::map<std::pair<const void *, int>, size_t> granted;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SQNN_E_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    size_t &have = granted[std::make_pair(kernel, dev)];
    if (have >= smem) return SQNN_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SQNN_E_CUDA;
    have = smem;
    return SQNN_OK;
}

int sm_count()
{
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        cached[dev] = v;
    }
    return cached[dev];
}


static int gemv_dispatch(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x,
                         int x_dtype, int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t m, uint64_t n,
                         cudaStream_t st)
{
#define SQNN_GEMV_CASE(NO, NI) \
    if (A.n_out == NO && A.n_in == NI) return gemv_shape<NO, NI>(A, d_mask, d_alpha, d_x, x_dtype, ldx, batch, d_y, ldy, m, n, st);
    SQNN_FOR_SHAPES(SQNN_GEMV_CASE)
#undef SQNN_GEMV_CASE
    return gemv_shape<0, 0>(A, d_mask, d_alpha, d_x, x_dtype, ldx, batch, d_y, ldy, m, n, st);
}

int decode_bits_dispatch(const DecodeArgs &A, void *d_out, cudaStream_t st)
{
#define SQNN_BITS_CASE(NO, NI) \
    if (A.n_out == NO && A.n_in == NI) return decode_shape<NO, NI>(A, SQNN_OUT_BITS, nullptr, nullptr, 0, d_out, st);
    SQNN_FOR_SHAPES(SQNN_BITS_CASE)
#undef SQNN_BITS_CASE
    return decode_shape<0, 0>(A, SQNN_OUT_BITS, nullptr, nullptr, 0, d_out, st);
}

namespace {
bool checked_mode()
{
    static const bool on = [] {
        const char *v = std::getenv("SQNN_DEBUG_CHECKS");
        return v && v[0] == '1';
    }();
    return on;
}
nvtxDomainHandle_t nvtx_domain()
{
    static nvtxDomainHandle_t d = nvtxDomainCreateA("sqnn");
    return d;
}
}  // namespace

ApiScope::ApiScope(const char *name)
{
    nvtxEventAttributes_t a = {};
    a.version = NVTX_VERSION;
    a.size = NVTX_EVENT_ATTRIB_STRUCT_SIZE;
    a.messageType = NVTX_MESSAGE_TYPE_ASCII;
    a.message.ascii = name;
    nvtxDomainRangePushEx(nvtx_domain(), &a);
}
ApiScope::~ApiScope() { nvtxDomainRangePop(nvtx_domain()); }

int ApiScope::finish(int rc, const uint32_t *d_status, cudaStream_t st) const
{
    if (rc != SQNN_OK || !checked_mode()) return rc;
    if (cudaStreamSynchronize(st) != cudaSuccess || cudaGetLastError() != cudaSuccess) return SQNN_E_CUDA;
    if (d_status) {
        uint32_t word = 0;
        if (cudaMemcpy(&word, d_status, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) return SQNN_E_CUDA;
        if (word == (uint32_t)(-SQNN_E_TIMEOUT)) return SQNN_E_TIMEOUT;
        if (word != 0) return SQNN_E_BAD_BLOB;
    }
    return SQNN_OK;
}

}  // namespace sqnn

using namespace sqnn;


static int decode_queue(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
                        const float *d_alpha, sqnn_out_mode mode, void *d_out, size_t out_bytes,
                        uint32_t *d_status, void *cuda_stream)
{
    DecodeArgs A;
    int rc = fill_decode_args(desc, d_blob, d_status, &A);
    if (rc != SQNN_OK) return rc;
    if (!d_out || ((uintptr_t)d_out & 15) != 0) return SQNN_E_INVALID_ARG;
    size_t need = 0;
    switch (mode) {
        case SQNN_OUT_BITS: need = (size_t)A.n_q * A.words64 * 8; break;
        case SQNN_OUT_BF16: need = (size_t)A.mn * 2; break;
        case SQNN_OUT_SINK: need = 8; break;
        default: return SQNN_E_INVALID_ARG;
    }
    if (out_bytes < need) return SQNN_E_INVALID_ARG;
    if (mode == SQNN_OUT_BF16 && (!d_mask || !d_alpha)) return SQNN_E_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
#define SQNN_DECODE_CASE(NO, NI) \
    if (A.n_out == NO && A.n_in == NI) return decode_shape<NO, NI>(A, mode, d_mask, d_alpha, desc->n, d_out, st);
    SQNN_FOR_SHAPES(SQNN_DECODE_CASE)
#undef SQNN_DECODE_CASE
    return decode_shape<0, 0>(A, mode, d_mask, d_alpha, desc->n, d_out, st);
}

extern "C" int sqnn_decode(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
                           const float *d_alpha, sqnn_out_mode mode, void *d_out, size_t out_bytes,
                           uint32_t *d_status, void *cuda_stream)
{
    ApiScope scope("sqnn_decode");
    return scope.finish(decode_queue(desc, d_blob, d_mask, d_alpha, mode, d_out, out_bytes, d_status, cuda_stream),
                        d_status, (cudaStream_t)cuda_stream);
}

namespace sqnn {
// Store-only counterpart of k_decode_bits: same block shape, same bulk copies, nothing read.
__global__ void __launch_bounds__(768, 1) k_store_probe(uint8_t *__restrict__ out, uint64_t chunks, uint32_t chunk_bytes, uint64_t tail_at, uint32_t tail_bytes)
{
    extern __shared__ __align__(16) uint32_t smem[];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    uint32_t *region = smem + warp * (chunk_bytes / 4);
    for (uint32_t i = lane; i < chunk_bytes / 4; i += 32) region[i] = i * 0x9e3779b9u + warp;
    fence_async_smem();
    __syncwarp();
    if (lane == 0) {
        for (uint64_t c = (uint64_t)blockIdx.x * nwarps + warp; c < chunks; c += (uint64_t)gridDim.x * nwarps) {
            const uint32_t nb = c == tail_at ? tail_bytes : chunk_bytes;
            bulk_store(out + c * chunk_bytes, region, nb);
        }
        bulk_wait_read<0>();
    }
}
}  // namespace sqnn

extern "C" int sqnn_store_probe(void *d_out, size_t bytes, uint32_t chunk_bytes, void *cuda_stream)
{
    if (!d_out || ((uintptr_t)d_out & 15) || bytes == 0 || (bytes & 15) || chunk_bytes == 0 || (chunk_bytes & 15) ||
        chunk_bytes > 8192)
        return SQNN_E_INVALID_ARG;
    const uint64_t chunks = (bytes + chunk_bytes - 1) / chunk_bytes;
    const uint32_t tail_bytes = (uint32_t)(bytes - (chunks - 1) * chunk_bytes);
    const uint32_t warps = 24;
    const size_t smem = (size_t)warps * chunk_bytes;
    if (ensure_dynamic_smem(reinterpret_cast<const void *>(k_store_probe), smem) != SQNN_OK) return SQNN_E_CUDA;
    uint64_t grid = (chunks + warps - 1) / warps;
    if (grid > (uint64_t)sm_count()) grid = (uint64_t)sm_count();
    k_store_probe<<<(uint32_t)grid, warps * 32, smem, (cudaStream_t)cuda_stream>>>((uint8_t *)d_out, chunks, chunk_bytes,
                                                                                 chunks - 1, tail_bytes);
    return cudaGetLastError() == cudaSuccess ? SQNN_OK : SQNN_E_CUDA;
}

extern "C" size_t sqnn_workspace_bytes(const sqnn_desc *desc, uint32_t batch)
{
    if (!desc || batch < 16) return 0;
    return mma_workspace_bytes(desc, batch);
}

static int decode_matmul_queue(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
                               const float *d_alpha, const void *d_x, int x_dtype, uint32_t batch,
                               int64_t ldx, float *d_y, int64_t ldy, void *d_workspace,
                               size_t workspace_bytes, uint32_t *d_status, void *cuda_stream)
{
    DecodeArgs A;
    int rc = fill_decode_args(desc, d_blob, d_status, &A);
    if (rc != SQNN_OK) return rc;
    if (!d_mask || !d_alpha || !d_x || !d_y || batch == 0) return SQNN_E_INVALID_ARG;
    if (x_dtype != SQNN_X_F32 && x_dtype != SQNN_X_BF16) return SQNN_E_INVALID_ARG;
    if (ldx < (int64_t)desc->n || ldy < (int64_t)desc->m) return SQNN_E_INVALID_ARG;
    if (((uintptr_t)d_mask & 7) || ((uintptr_t)d_alpha & 3) || ((uintptr_t)d_y & 3)) return SQNN_E_INVALID_ARG;
    if (batch > SQNN_MAX_BATCH || desc->n > (1ull << 30)) return SQNN_E_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (batch <= 15)
        return gemv_dispatch(A, d_mask, d_alpha, d_x, x_dtype, ldx, batch, d_y, ldy, desc->m, desc->n, st);
    if (x_dtype != SQNN_X_BF16) return SQNN_E_UNSUPPORTED;
    // The planes are decoded to packed bits in the workspace first; the tensor-core kernel reads
    // them from there.
    if (!d_workspace || workspace_bytes < mma_workspace_bytes(desc, batch) || ((uintptr_t)d_workspace & 255))
        return SQNN_E_WORKSPACE;
    return mma_dispatch(desc, A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, d_workspace, st);
}

extern "C" int sqnn_decode_matmul(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
                                  const float *d_alpha, const void *d_x, int x_dtype, uint32_t batch,
                                  int64_t ldx, float *d_y, int64_t ldy, void *d_workspace,
                                  size_t workspace_bytes, uint32_t *d_status, void *cuda_stream)
{
    ApiScope scope("sqnn_decode_matmul");
    return scope.finish(decode_matmul_queue(desc, d_blob, d_mask, d_alpha, d_x, x_dtype, batch, ldx, d_y, ldy,
                                            d_workspace, workspace_bytes, d_status, cuda_stream),
                        d_status, (cudaStream_t)cuda_stream);
}
