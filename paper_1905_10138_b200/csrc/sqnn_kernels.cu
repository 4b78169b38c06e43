// Decode kernels (packed bits, bf16 weights, checksum sink) and the fused decode-GEMV kernel,
// with the C entry points that launch them.
#include "sqnn.h"
#include "sqnn_decode.cuh"
#include "sqnn_launch.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace sqnn {

// ------------------------------------------------------------------------------------------
// shared-memory layout of the warp-tile kernels: [tables][warp 0 regions][warp 1 regions]...
// a warp's regions: `planes` runs of 32 * W words
// ------------------------------------------------------------------------------------------
SQNN_DEV uint64_t tile_word64(const uint32_t *region, uint32_t q)
{
    const uint2 v = *reinterpret_cast<const uint2 *>(region + 2 * q);
    return (uint64_t)v.x | ((uint64_t)v.y << 32);
}

// K1: decoded planes as packed bits.  One warp tile = 16 * W consecutive uint64 of one plane.
// SINK = true: XOR of all those words instead of storing them.
template <int N_OUT, int N_IN, bool SINK>
__global__ void __launch_bounds__(256)
k_decode_bits(DecodeArgs A, uint64_t *__restrict__ out)
{
    extern __shared__ __align__(16) uint32_t smem[];
    build_tables(A, smem);
    const uint32_t W = N_OUT ? slices_per_lane(N_OUT ? N_OUT : 1) * (N_OUT ? N_OUT : 0) / 32 : A.W;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    uint32_t *region = smem + table_words(A.n_in, A.nwp, A.nchunks, A.cb) + warp * 32 * W;
    const uint64_t total = A.tiles * A.n_q;
    const uint64_t tail_bits = A.mn & 63;
    uint64_t sink = 0;
    for (uint64_t t = (uint64_t)blockIdx.x * nwarps + warp; t < total; t += (uint64_t)gridDim.x * nwarps) {
        const uint32_t plane = (uint32_t)(t / A.tiles);
        const uint64_t tile = t - (uint64_t)plane * A.tiles;
        const uint64_t q0 = tile * 16 * W;               // first uint64 of the tile inside the plane
        if (q0 >= A.words64) continue;                   // tile made of padding slices only
        decode_warp_tile<N_OUT, N_IN>(A, plane, tile, region, smem, lane);
        __syncwarp();
        uint64_t *dst = out + (uint64_t)plane * A.words64;
        for (uint32_t q = lane; q < 16 * W; q += 32) {
            const uint64_t gq = q0 + q;
            if (gq >= A.words64) break;
            uint64_t v = tile_word64(region, q);
            if (gq == A.words64 - 1 && tail_bits) v &= (1ull << tail_bits) - 1ull;
            if constexpr (SINK) sink ^= v; else dst[gq] = v;
        }
        __syncwarp();
    }
    if constexpr (SINK) {
#pragma unroll
        for (uint32_t d = 16; d >= 1; d >>= 1) sink ^= __shfl_xor_sync(0xffffffffu, sink, d);
        if (lane == 0 && sink) atomicXor(reinterpret_cast<unsigned long long *>(out), (unsigned long long)sink);
    }
}

// K2: decoded, masked, rescaled weights as bf16.  Lane j of an iteration writes the 8 weights
// of byte j of a 32-byte group of the tile's bit run, so a warp stores 512 contiguous bytes.
template <int N_OUT, int N_IN>
__global__ void __launch_bounds__(256)
k_decode_bf16(DecodeArgs A, const uint8_t *__restrict__ mask8, const float *__restrict__ alpha,
              uint64_t n, __nv_bfloat16 *__restrict__ out)
{
    extern __shared__ __align__(16) uint32_t smem[];
    build_tables(A, smem);
    const uint32_t W = N_OUT ? slices_per_lane(N_OUT ? N_OUT : 1) * (N_OUT ? N_OUT : 0) / 32 : A.W;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t n_q = A.n_q;
    uint32_t *region = smem + table_words(A.n_in, A.nwp, A.nchunks, A.cb) + warp * n_q * 32 * W;
    const uint32_t tile_bytes = 128 * W;                 // bytes of bits per tile and plane
    for (uint64_t tile = (uint64_t)blockIdx.x * nwarps + warp; tile < A.tiles; tile += (uint64_t)gridDim.x * nwarps) {
        const uint64_t p_tile = tile * (uint64_t)tile_bytes * 8;
        if (p_tile >= A.mn) continue;
        for (uint32_t i = 0; i < n_q; ++i)
            decode_warp_tile<N_OUT, N_IN>(A, i, tile, region + i * 32 * W, smem, lane);
        __syncwarp();
        uint64_t p = p_tile + 8ull * lane;               // first weight of this lane's group
        uint64_t r = p / n;
        uint64_t c = p - r * n;
        for (uint32_t t = lane; t < tile_bytes; t += 32, p += 256, c += 256) {
            if (p >= A.mn) break;
            while (c >= n) { c -= n; ++r; }
            const uint32_t mk = mask8[p >> 3];
            uint32_t bits[8];
#pragma unroll
            for (uint32_t i = 0; i < 8; ++i)
                bits[i] = i < n_q ? reinterpret_cast<const uint8_t *>(region + i * 32 * W)[t] : 0u;
            __align__(16) __nv_bfloat16 v[8];
            uint64_t rr = r, cc = c;
#pragma unroll
            for (uint32_t k = 0; k < 8; ++k) {
                if (cc >= n) { cc -= n; ++rr; }
                float s = 0.0f;
                if ((mk >> k) & 1u) {
#pragma unroll
                    for (uint32_t i = 0; i < 8; ++i) {
                        if (i < n_q) {
                            const float a = __ldg(alpha + rr * n_q + i);
                            s = __fadd_rn(s, ((bits[i] >> k) & 1u) ? a : -a);
                        }
                    }
                }
                v[k] = __float2bfloat16_rn(s);
                ++cc;
            }
            if (p + 8 <= A.mn) {
                *reinterpret_cast<uint4 *>(out + p) = *reinterpret_cast<const uint4 *>(v);
            } else {
                for (uint32_t k = 0; k < 8 && p + k < A.mn; ++k) out[p + k] = v[k];
            }
        }
        __syncwarp();
    }
}

SQNN_DEV float to_float(float v) { return v; }
SQNN_DEV float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// K3: decryption fused with Y[b][r] = sum_c W[r][c] X[b][c] for small batch, fp32 accumulate.
// A warp decodes its tile of every plane into shared memory, then walks the row segments the
// tile covers: lanes take the tile's 32-bit words in turn, visit the set bits of the mask word,
// rebuild the weight value (+-alpha_1) + (+-alpha_2) + ... and accumulate value * x.  Partial
// sums of a row segment are reduced over the warp and added to Y with one atomic per (row, b).
template <int N_OUT, int N_IN, int BT, typename XT>
__global__ void __launch_bounds__(256)
k_decode_gemv(DecodeArgs A, const uint32_t *__restrict__ mask32, const float *__restrict__ alpha,
              const XT *__restrict__ x, int64_t ldx, uint32_t batch, float *__restrict__ y,
              int64_t ldy, uint64_t n)
{
    extern __shared__ __align__(16) uint32_t smem[];
    build_tables(A, smem);
    const uint32_t W = N_OUT ? slices_per_lane(N_OUT ? N_OUT : 1) * (N_OUT ? N_OUT : 0) / 32 : A.W;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t n_q = A.n_q;
    uint32_t *region = smem + table_words(A.n_in, A.nwp, A.nchunks, A.cb) + warp * n_q * 32 * W;
    for (uint64_t tile = (uint64_t)blockIdx.x * nwarps + warp; tile < A.tiles; tile += (uint64_t)gridDim.x * nwarps) {
        const uint64_t gw0 = tile * 32 * W;              // first 32-bit word of the tile
        const uint64_t P0 = gw0 * 32;
        if (P0 >= A.mn) continue;
        const uint64_t P1 = (P0 + 1024ull * W < A.mn) ? P0 + 1024ull * W : A.mn;
        for (uint32_t i = 0; i < n_q; ++i)
            decode_warp_tile<N_OUT, N_IN>(A, i, tile, region + i * 32 * W, smem, lane);
        __syncwarp();
        for (uint64_t r = P0 / n; r * n < P1; ++r) {
            const uint64_t a = r * n > P0 ? r * n : P0;
            const uint64_t b = (r + 1) * n < P1 ? (r + 1) * n : P1;
            float al[8];
#pragma unroll
            for (uint32_t i = 0; i < 8; ++i) al[i] = i < n_q ? __ldg(alpha + r * n_q + i) : 0.0f;
            const uint64_t w_lo = a >> 5, w_hi = (b - 1) >> 5;
            for (uint32_t bc = 0; bc < batch; bc += BT) {
                float acc[BT];
#pragma unroll
                for (int q = 0; q < BT; ++q) acc[q] = 0.0f;
                for (uint64_t gw = w_lo + lane; gw <= w_hi; gw += 32) {
                    const uint32_t lw = (uint32_t)(gw - gw0);
                    uint32_t mk = __ldg(mask32 + gw);
                    const uint64_t lo = gw * 32;
                    if (lo < a) mk &= 0xffffffffu << (uint32_t)(a - lo);
                    if (lo + 32 > b) mk &= 0xffffffffu >> (uint32_t)(lo + 32 - b);
                    uint32_t wb[8];
#pragma unroll
                    for (uint32_t i = 0; i < 8; ++i) wb[i] = i < n_q ? region[i * 32 * W + lw] : 0u;
                    const int64_t cbase = (int64_t)lo - (int64_t)(r * n);
                    while (mk) {
                        const uint32_t k = (uint32_t)__ffs((int)mk) - 1u;
                        mk &= mk - 1u;
                        float v = 0.0f;
#pragma unroll
                        for (uint32_t i = 0; i < 8; ++i)
                            if (i < n_q) v += ((wb[i] >> k) & 1u) ? al[i] : -al[i];
                        const int64_t c = cbase + (int64_t)k;
#pragma unroll
                        for (int q = 0; q < BT; ++q)
                            if (bc + q < batch) acc[q] = fmaf(v, to_float(x[(int64_t)(bc + q) * ldx + c]), acc[q]);
                    }
                }
#pragma unroll
                for (int q = 0; q < BT; ++q) {
                    float s = acc[q];
#pragma unroll
                    for (uint32_t d = 16; d >= 1; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
                    if (lane == 0 && bc + q < batch) atomicAdd(y + (int64_t)(bc + q) * ldy + r, s);
                }
            }
        }
        __syncwarp();
    }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
static uint32_t gcd_host(uint32_t a, uint32_t b) { return b ? gcd_host(b, a % b) : a; }

int fill_decode_args(const sqnn_desc *d, const void *d_blob, uint32_t *d_status, DecodeArgs *A)
{
    if (!d || !d_blob) return SQNN_E_INVALID_ARG;
    if (((uintptr_t)d_blob & 15) != 0) return SQNN_E_INVALID_ARG;
    if (d->n_out < 1 || d->n_out > SQNN_MAX_N_OUT || d->n_in < 1 || d->n_in > SQNN_MAX_N_IN ||
        d->n_q < 1 || d->n_q > SQNN_MAX_PLANES || d->m == 0 || d->n == 0 ||
        d->block_slices != SQNN_BLOCK_SLICES || d->slices_padded % SQNN_PAD_SLICES != 0)
        return SQNN_E_INVALID_ARG;
    const uint8_t *b = (const uint8_t *)d_blob;
    A->mn = d->m * d->n;
    A->words64 = (A->mn + 63) / 64;
    A->n_out = d->n_out; A->n_in = d->n_in; A->n_q = d->n_q;
    const uint32_t g = 32 / gcd_host(d->n_out, 32);
    A->G = g < 4 ? 4 : g;
    A->W = A->G * d->n_out / 32;
    A->tiles = d->slices_padded / (32ull * A->G);
    A->nw = entry_words(d->n_out);
    A->nwp = entry_words_padded(d->n_out);
    A->nchunks = table_chunks(d->n_in, A->nwp);
    A->cb = chunk_bits(d->n_in, A->nwp);
    A->rows = (const uint32_t *)(b + d->off_xornet);
    A->status = d_status;
    for (uint32_t i = 0; i < d->n_q; ++i) {
        if (d->off_wc[i] % 16 || d->off_np[i] % 16 || d->off_idx[i] % 16 || d->off_dp[i] % 16 ||
            d->n_dp[i] > 0xffffffffull || d->w_np[i] > 9)
            return SQNN_E_INVALID_ARG;
        A->pl[i].wc = (const uint32_t *)(b + d->off_wc[i]);
        A->pl[i].np = (const uint32_t *)(b + d->off_np[i]);
        A->pl[i].idx = (const uint32_t *)(b + d->off_idx[i]);
        A->pl[i].dp = b + d->off_dp[i];
        A->pl[i].n_dp = (uint32_t)d->n_dp[i];
        A->pl[i].w_np = d->w_np[i];
    }
    for (uint32_t i = d->n_q; i < 8; ++i) A->pl[i] = A->pl[0];
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

// Picks warps per block so the dynamic shared memory fits; returns 0 if not even one warp fits.
static uint32_t pick_warps(const DecodeArgs &A, uint32_t planes, size_t *smem_bytes)
{
    const size_t tab = (size_t)table_words(A.n_in, A.nwp, A.nchunks, A.cb) * 4;
    const size_t per_warp = (size_t)planes * 32 * A.W * 4;
    const size_t limit = 200 * 1024;
    if (tab + per_warp > limit) return 0;
    uint32_t warps = (uint32_t)((limit - tab) / per_warp);
    if (warps > 8) warps = 8;
    *smem_bytes = tab + warps * per_warp;
    return warps;
}

template <typename K>
static int prepare(K kernel, size_t smem)
{
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SQNN_E_CUDA;
    return SQNN_OK;
}

static uint32_t grid_for(uint64_t warp_tiles, uint32_t warps, uint32_t blocks_per_sm)
{
    uint64_t need = (warp_tiles + warps - 1) / warps;
    uint64_t cap = (uint64_t)sm_count() * blocks_per_sm;
    if (need < 1) need = 1;
    return (uint32_t)(need < cap ? need : cap);
}

#define SQNN_FOR_SHAPES(X) X(40, 12) X(40, 16) X(60, 12) X(80, 8) X(80, 16) X(100, 10) X(200, 10)

template <int N_OUT, int N_IN>
static int launch_decode(const DecodeArgs &A, sqnn_out_mode mode, const uint64_t *d_mask,
                         const float *d_alpha, uint64_t n, void *d_out, cudaStream_t st)
{
    size_t smem = 0;
    if (mode == SQNN_OUT_BITS || mode == SQNN_OUT_SINK) {
        const uint32_t warps = pick_warps(A, 1, &smem);
        if (!warps) return SQNN_E_UNSUPPORTED;
        const uint32_t grid = grid_for(A.tiles * A.n_q, warps, 4);
        if (mode == SQNN_OUT_BITS) {
            auto k = k_decode_bits<N_OUT, N_IN, false>;
            if (prepare(k, smem)) return SQNN_E_CUDA;
            k<<<grid, warps * 32, smem, st>>>(A, (uint64_t *)d_out);
        } else {
            if (cudaMemsetAsync(d_out, 0, 8, st) != cudaSuccess) return SQNN_E_CUDA;
            auto k = k_decode_bits<N_OUT, N_IN, true>;
            if (prepare(k, smem)) return SQNN_E_CUDA;
            k<<<grid, warps * 32, smem, st>>>(A, (uint64_t *)d_out);
        }
    } else {
        const uint32_t warps = pick_warps(A, A.n_q, &smem);
        if (!warps) return SQNN_E_UNSUPPORTED;
        const uint32_t grid = grid_for(A.tiles, warps, 4);
        auto k = k_decode_bf16<N_OUT, N_IN>;
        if (prepare(k, smem)) return SQNN_E_CUDA;
        k<<<grid, warps * 32, smem, st>>>(A, (const uint8_t *)d_mask, d_alpha, n, (__nv_bfloat16 *)d_out);
    }
    return cudaGetLastError() == cudaSuccess ? SQNN_OK : SQNN_E_CUDA;
}

template <int N_OUT, int N_IN, int BT, typename XT>
static int launch_gemv_bt(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x,
                          int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t n, cudaStream_t st)
{
    size_t smem = 0;
    const uint32_t warps = pick_warps(A, A.n_q, &smem);
    if (!warps) return SQNN_E_UNSUPPORTED;
    const uint32_t grid = grid_for(A.tiles, warps, 2);
    auto k = k_decode_gemv<N_OUT, N_IN, BT, XT>;
    if (prepare(k, smem)) return SQNN_E_CUDA;
    k<<<grid, warps * 32, smem, st>>>(A, (const uint32_t *)d_mask, d_alpha, (const XT *)d_x, ldx, batch, d_y, ldy, n);
    return cudaGetLastError() == cudaSuccess ? SQNN_OK : SQNN_E_CUDA;
}

template <int N_OUT, int N_IN, typename XT>
static int launch_gemv(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x,
                       int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t n, cudaStream_t st)
{
    if (batch == 1) return launch_gemv_bt<N_OUT, N_IN, 1, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st);
    if (batch == 2) return launch_gemv_bt<N_OUT, N_IN, 2, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st);
    if (batch <= 4) return launch_gemv_bt<N_OUT, N_IN, 4, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st);
    return launch_gemv_bt<N_OUT, N_IN, 8, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st);
}

int gemv_dispatch(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x,
                  int x_dtype, int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t m, uint64_t n,
                  cudaStream_t st)
{
    // Y is accumulated with atomics: clear it first.
    cudaError_t e = (ldy == (int64_t)m)
        ? cudaMemsetAsync(d_y, 0, (size_t)batch * m * sizeof(float), st)
        : cudaMemset2DAsync(d_y, (size_t)ldy * sizeof(float), 0, (size_t)m * sizeof(float), batch, st);
    if (e != cudaSuccess) return SQNN_E_CUDA;
#define SQNN_GEMV_CASE(NO, NI)                                                                         \
    if (A.n_out == NO && A.n_in == NI) {                                                               \
        return x_dtype == SQNN_X_BF16                                                                  \
            ? launch_gemv<NO, NI, __nv_bfloat16>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st) \
            : launch_gemv<NO, NI, float>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st);        \
    }
    SQNN_FOR_SHAPES(SQNN_GEMV_CASE)
#undef SQNN_GEMV_CASE
    return x_dtype == SQNN_X_BF16
        ? launch_gemv<0, 0, __nv_bfloat16>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st)
        : launch_gemv<0, 0, float>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st);
}

}  // namespace sqnn

using namespace sqnn;

extern "C" int sqnn_decode(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
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
    if (A.n_out == NO && A.n_in == NI) return launch_decode<NO, NI>(A, mode, d_mask, d_alpha, desc->n, d_out, st);
    SQNN_FOR_SHAPES(SQNN_DECODE_CASE)
#undef SQNN_DECODE_CASE
    return launch_decode<0, 0>(A, mode, d_mask, d_alpha, desc->n, d_out, st);
}

extern "C" size_t sqnn_workspace_bytes(const sqnn_desc *desc, uint32_t batch)
{
    if (!desc || batch < 16) return 0;
    return mma_workspace_bytes(desc, batch);
}

extern "C" int sqnn_decode_matmul(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
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
    if (batch > SQNN_MAX_BATCH) return SQNN_E_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (batch <= 15)
        return gemv_dispatch(A, d_mask, d_alpha, d_x, x_dtype, ldx, batch, d_y, ldy, desc->m, desc->n, st);
    if (x_dtype != SQNN_X_BF16) return SQNN_E_UNSUPPORTED;
    const size_t need = mma_workspace_bytes(desc, batch);
    if (need && (!d_workspace || workspace_bytes < need || ((uintptr_t)d_workspace & 255))) return SQNN_E_WORKSPACE;
    return mma_dispatch(desc, A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, d_workspace, st);
}
