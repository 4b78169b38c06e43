// Decode kernels (packed bits, bf16 weights, checksum sink) and the fused decode-GEMV kernel,
// as templates over the network shape, with their launchers.
#pragma once
#include "sqnn.h"
#include "sqnn_decode.cuh"
#include "sqnn_launch.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace sqnn {

// ------------------------------------------------------------------------------------------
// shared-memory layout of the warp-tile kernels:
//   [tables][warp 0: regions, d_patch stage][warp 1: ...]...[activations (GEMV only)]
// a region is a run of 32 * W words (one warp tile of one plane)
// ------------------------------------------------------------------------------------------
SQNN_DEV uint64_t tile_word64(const uint32_t *region, uint32_t q)
{
    const uint2 v = *reinterpret_cast<const uint2 *>(region + 2 * q);
    return (uint64_t)v.x | ((uint64_t)v.y << 32);
}

template <int N_OUT>
SQNN_DEV uint32_t words_per_lane(const DecodeArgs &A)
{
    if constexpr (N_OUT != 0) return slices_per_lane(N_OUT) * N_OUT / 32;
    else return A.W;
}

// K1: decoded planes as packed bits.  One warp tile = 16 * W consecutive uint64 of one plane,
// built in the warp's shared-memory region and written out by a bulk copy while the warp
// already fetches and expands its next tile (it waits for the copy only when it is about to
// overwrite the region); the global loads of the next tile are issued before the current tile
// is expanded.  SINK = true: XOR of all those words instead of
// storing them.
template <int N_OUT, int N_IN, bool SINK>
__global__ void __launch_bounds__(512, 2)
k_decode_bits(DecodeArgs A, uint64_t *__restrict__ out)
{
    extern __shared__ __align__(16) uint32_t smem[];
    build_tables(A, smem);
    const uint32_t W = words_per_lane<N_OUT>(A);
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t per_warp = 32 * W + STAGE_WORDS;
    uint32_t *mybase = smem + table_words(A.n_in, A.nwp, A.nchunks, A.cb) + warp * per_warp;
    uint32_t *stage = mybase + 32 * W;
    const uint64_t tail_bits = A.mn & 63;
    // tiles that hold at least one real word, per plane (the launcher keeps the count below 2^31);
    // (plane, tile) advance without division
    const uint32_t live = (uint32_t)((A.words64 + 16 * W - 1) / (16 * W));
    // tiles before this one lie wholly inside the plane and end on a whole word
    const uint32_t full_tiles = (uint32_t)(A.words64 / (16 * W)) -
                                ((tail_bits != 0 && A.words64 % (16 * W) == 0) ? 1u : 0u);
    const uint32_t stride = gridDim.x * nwarps;
    uint32_t tile = blockIdx.x * nwarps + warp;
    uint32_t plane = 0;
    while (plane < A.n_q && tile >= live) { tile -= live; ++plane; }
    uint64_t sink = 0;
    if constexpr (N_OUT != 0) {
        TileIn<N_OUT, N_IN> cur, nxt;
        if (plane < A.n_q) tile_fetch<N_OUT, N_IN>(A.pl[plane], tile, lane, cur);
        while (plane < A.n_q) {
            uint32_t ntile = tile + stride;
            uint32_t nplane = plane;
            while (nplane < A.n_q && ntile >= live) { ntile -= live; ++nplane; }
            if (nplane < A.n_q) tile_fetch<N_OUT, N_IN>(A.pl[nplane], ntile, lane, nxt);
            uint32_t st[4];
            stage_fetch<N_OUT, N_IN>(A, A.pl[plane], cur, lane, st);
            uint32_t *region = mybase;
            tile_decode<N_OUT, N_IN, !SINK>(A, A.pl[plane], cur, st, region, smem, stage, lane);
            uint64_t *pbase = out + (uint64_t)plane * A.words64;
            const uint64_t q0 = (uint64_t)tile * (16 * W);   // first uint64 of the tile inside the plane
            uint64_t *dst = pbase + q0;
            if (!SINK && tile < full_tiles && (reinterpret_cast<uintptr_t>(pbase) & 15) == 0) {
                fence_async_smem();
                __syncwarp();
                if (lane == 0) bulk_store(dst, region, 128 * W);
            } else {
                for (uint32_t q = lane; q < 16 * W; q += 32) {
                    if (q0 + q >= A.words64) break;
                    uint64_t v = tile_word64(region, q);
                    if (q0 + q == A.words64 - 1 && tail_bits) v &= (1ull << tail_bits) - 1ull;
                    if constexpr (SINK) sink ^= v; else dst[q] = v;
                }
                __syncwarp();
            }
            cur = nxt;
            tile = ntile;
            plane = nplane;
        }
    } else {
        while (plane < A.n_q) {
            uint32_t *region = mybase;
            decode_warp_tile<0, 0>(A, plane, tile, region, smem, stage, lane);
            const uint64_t q0 = (uint64_t)tile * (16 * W);
            uint64_t *dst = out + (uint64_t)plane * A.words64 + q0;
            for (uint32_t q = lane; q < 16 * W; q += 32) {
                if (q0 + q >= A.words64) break;
                uint64_t v = tile_word64(region, q);
                if (q0 + q == A.words64 - 1 && tail_bits) v &= (1ull << tail_bits) - 1ull;
                if constexpr (SINK) sink ^= v; else dst[q] = v;
            }
            __syncwarp();
            tile += stride;
            while (plane < A.n_q && tile >= live) { tile -= live; ++plane; }
        }
    }
    if constexpr (SINK) {
#pragma unroll
        for (uint32_t d = 16; d >= 1; d >>= 1) sink ^= __shfl_xor_sync(0xffffffffu, sink, d);
        if (lane == 0 && sink) atomicXor(reinterpret_cast<unsigned long long *>(out), (unsigned long long)sink);
    } else {
        if (lane == 0) bulk_wait_read<0>();              // shared memory must outlive the copies
    }
}

SQNN_DEV void cp_async16(void *sdst, const void *gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" :: "r"(smem_addr(sdst)), "l"(gsrc) : "memory");
}
SQNN_DEV void cp_async4(void *sdst, const void *gsrc)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" :: "r"(smem_addr(sdst)), "l"(gsrc) : "memory");
}
SQNN_DEV void cp_async_wait_all() { asm volatile("cp.async.wait_all;\n" ::: "memory"); }

// Starts the copy of a tile's 32 * W mask words (first word gw0) into shared memory: 16-byte
// asynchronous copies where a whole vector is in range, plain loads (zero past the end) otherwise.
// Finish with cp_async_wait_all() and a warp barrier.
SQNN_DEV void stage_mask_tile(uint32_t *mask_s, const uint32_t *__restrict__ mask32, uint64_t gw0,
                              uint64_t mask_words, uint32_t W, uint32_t lane, bool vec_ok)
{
    for (uint32_t v = lane; v < 8 * W; v += 32) {
        if (vec_ok && gw0 + 4 * v + 4 <= mask_words) {
            cp_async16(mask_s + 4 * v, mask32 + gw0 + 4 * v);
        } else {
#pragma unroll
            for (uint32_t e = 0; e < 4; ++e)
                mask_s[4 * v + e] = gw0 + 4 * v + e < mask_words ? __ldg(mask32 + gw0 + 4 * v + e) : 0u;
        }
    }
}

// K2: decoded, masked, rescaled weights as bf16.  Lane j of an iteration writes the 8 weights
// of byte j of a 32-byte group of the tile's bit run, so a warp stores 512 contiguous bytes.
// The tile's mask words arrive by cp.async while the tile is decoded; a lane keeps the scales
// of the row it is in.  NQ = number of planes when it is 1, 2 or 3, 0 = any.
template <int N_OUT, int N_IN, int NQ>
__global__ void __launch_bounds__(256)
k_decode_bf16(DecodeArgs A, const uint32_t *__restrict__ mask32, const float *__restrict__ alpha,
              uint64_t n, __nv_bfloat16 *__restrict__ out)
{
    extern __shared__ __align__(16) uint32_t smem[];
    build_tables(A, smem);
    const uint32_t W = words_per_lane<N_OUT>(A);
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t n_q = A.n_q;
    const uint32_t per_warp = (n_q + 1) * 32 * W + STAGE_WORDS;
    uint32_t *region = smem + table_words(A.n_in, A.nwp, A.nchunks, A.cb) + warp * per_warp;
    uint32_t *mask_s = region + n_q * 32 * W;
    uint32_t *stage = mask_s + 32 * W;
    const uint8_t *mask_s8 = reinterpret_cast<const uint8_t *>(mask_s);
    const uint32_t tile_bytes = 128 * W;                 // bytes of bits per tile and plane
    const uint64_t mask_words = A.words64 * 2;
    const bool mask_vec = (reinterpret_cast<uintptr_t>(mask32) & 15) == 0;
    constexpr int NR = NQ > 0 ? NQ : 1;
    for (uint64_t tile = (uint64_t)blockIdx.x * nwarps + warp; tile < A.tiles; tile += (uint64_t)gridDim.x * nwarps) {
        const uint64_t p_tile = tile * (uint64_t)tile_bytes * 8;
        if (p_tile >= A.mn) continue;
        stage_mask_tile(mask_s, mask32, tile * 32 * W, mask_words, W, lane, mask_vec);
        for (uint32_t i = 0; i < n_q; ++i)
            decode_warp_tile<N_OUT, N_IN>(A, i, tile, region + i * 32 * W, smem, stage, lane);
        cp_async_wait_all();
        __syncwarp();
        uint64_t p = p_tile + 8ull * lane;               // first weight of this lane's group
        uint64_t r = p / n;
        uint64_t c = p - r * n;
        float al[NR];
        uint64_t r_al = ~0ull;
        for (uint32_t t = lane; t < tile_bytes; t += 32, p += 256, c += 256) {
            if (p >= A.mn) break;
            while (c >= n) { c -= n; ++r; }
            const uint32_t mk = mask_s8[t];
            if (NQ > 0 && c + 8 <= n && p + 8 <= A.mn) {
                if (r != r_al) {
#pragma unroll
                    for (int i = 0; i < NR; ++i) al[i] = __ldg(alpha + r * n_q + i);
                    r_al = r;
                }
                uint32_t bits[NR];
#pragma unroll
                for (int i = 0; i < NR; ++i) bits[i] = reinterpret_cast<const uint8_t *>(region + i * 32 * W)[t];
                uint32_t w[4];
#pragma unroll
                for (uint32_t h = 0; h < 4; ++h) {
                    float two[2];
#pragma unroll
                    for (uint32_t e = 0; e < 2; ++e) {
                        const uint32_t k = 2 * h + e;
                        float s = 0.0f;
#pragma unroll
                        for (int i = 0; i < NR; ++i) {
                            const float term = ((bits[i] >> k) & 1u) ? al[i] : -al[i];
                            s = i == 0 ? term : __fadd_rn(s, term);
                        }
                        two[e] = ((mk >> k) & 1u) ? s : 0.0f;
                    }
                    const __nv_bfloat162 pk = __floats2bfloat162_rn(two[0], two[1]);
                    w[h] = *reinterpret_cast<const uint32_t *>(&pk);
                }
                *reinterpret_cast<uint4 *>(out + p) = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
                uint64_t rr = r, cc = c;
                for (uint32_t k = 0; k < 8 && p + k < A.mn; ++k) {
                    if (cc >= n) { cc -= n; ++rr; }
                    float s = 0.0f;
                    if ((mk >> k) & 1u) {
                        for (uint32_t i = 0; i < n_q; ++i) {
                            const float a = __ldg(alpha + rr * n_q + i);
                            const uint32_t bi = reinterpret_cast<const uint8_t *>(region + i * 32 * W)[t];
                            s = __fadd_rn(s, ((bi >> k) & 1u) ? a : -a);
                        }
                    }
                    out[p + k] = __float2bfloat16_rn(s);
                    ++cc;
                }
            }
        }
        __syncwarp();
    }
}

SQNN_DEV float to_float(float v) { return v; }
SQNN_DEV float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// BT activations of one column, stored contiguously in shared memory.
template <int BT, typename XT>
SQNN_DEV void load_x(const XT *p, float (&v)[BT])
{
    struct __align__(sizeof(XT) * BT > 16 ? 16 : sizeof(XT) * BT) Pack { XT e[BT]; };
    const Pack pk = *reinterpret_cast<const Pack *>(p);
#pragma unroll
    for (int q = 0; q < BT; ++q) v[q] = to_float(pk.e[q]);
}

// Words of a row segment a lane works on at the same time in the GEMV kernel (build-time tunable).
#ifndef SQNN_GEMV_WORDS_PER_ROUND
#define SQNN_GEMV_WORDS_PER_ROUND 2
#endif

// Words of per-warp scratch the GEMV kernel keeps for the scales of the rows a tile touches.
constexpr uint32_t GEMV_ALPHA_WORDS = 64;

// K3: decryption fused with Y[b][r] = sum_c W[r][c] X[b][c] for small batch, fp32 accumulate.
// A warp decodes its tile of every plane into shared memory, then walks the row segments the
// tile covers: lanes take the tile's 32-bit words in turn, visit the set bits of the mask word,
// rebuild the weight value (+-alpha_1) + (+-alpha_2) + ... and accumulate value * x.  Partial
// sums of a row segment are reduced over the warp and added to Y with one atomic per (row, b).
// Everything the walk reads is on chip by then: the tile's mask words arrive by cp.async while
// the tile is decoded, the scales of its rows are fetched up front, and (XS = true) the
// activations of the current batch chunk sit in shared memory as xs[c][BT].
// NQ = number of planes when it is 1, 2 or 3 (scales and plane words stay in registers), 0 = any.
template <int N_OUT, int N_IN, int BT, typename XT, bool XS, int NQ>
__global__ void __launch_bounds__(640)
k_decode_gemv(DecodeArgs A, const uint32_t *__restrict__ mask32, const float *__restrict__ alpha,
              const XT *__restrict__ x, int64_t ldx, uint32_t batch, float *__restrict__ y,
              int64_t ldy, uint32_t n, uint32_t wpt)
{
    extern __shared__ __align__(16) uint32_t smem[];
    const uint32_t W = words_per_lane<N_OUT>(A);
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t n_q = A.n_q;
    // `wpt` warps form a group that shares one tile: the planes (and the mask / scale staging)
    // are dealt out over the group's warps, then all of them walk the tile's words
    const uint32_t group = warp / wpt, sub = warp - group * wpt, ngroups = nwarps / wpt;
    const uint32_t per_group = (n_q + 1) * 32 * W + GEMV_ALPHA_WORDS;
    uint32_t *warp0 = smem + table_words(A.n_in, A.nwp, A.nchunks, A.cb);
    uint32_t *region = warp0 + group * per_group;
    uint32_t *mask_s = region + n_q * 32 * W;
    float *alpha_s = reinterpret_cast<float *>(mask_s + 32 * W);
    uint32_t *stage = warp0 + ngroups * per_group + warp * STAGE_WORDS;
    XT *xs = reinterpret_cast<XT *>(warp0 + ngroups * per_group + nwarps * STAGE_WORDS);
    const uint64_t mask_words = A.words64 * 2;
    const uint64_t alpha_count = (A.mn / n) * n_q;
    const bool mask_vec = (reinterpret_cast<uintptr_t>(mask32) & 15) == 0;
    const uint64_t tile_first = (uint64_t)blockIdx.x * ngroups + group, tile_step = (uint64_t)gridDim.x * ngroups;

    // Whatever the first tile needs from global memory is requested up front with nothing waiting
    // on it -- the rows of M and this warp's seeds / patch offsets into registers, the tile's mask
    // words, the scales of its first rows and the activations by asynchronous copies -- so that
    // one memory latency covers them all; the d_patch words follow once the offsets are here.
    const RowsAhead rows_ahead = fetch_rows(A);
    auto request = [&](uint64_t tile) {
        const uint64_t gw0 = tile * 32 * W;
        if (gw0 * 32 >= A.mn) return;
        if (sub == n_q % wpt) {
            stage_mask_tile(mask_s, mask32, gw0, mask_words, W, lane, mask_vec);
            const uint64_t r_first = gw0 * 32 / n;
            for (uint32_t i = lane; i < GEMV_ALPHA_WORDS; i += 32) {
                const uint64_t at = r_first * n_q + i;
                if (at < alpha_count) cp_async4(alpha_s + i, alpha + at);
                else alpha_s[i] = 0.0f;
            }
        }
    };
    TileIn<N_OUT ? N_OUT : 40, N_OUT ? N_IN : 12> pre;      // seeds of plane `sub` of the next tile
    if constexpr (N_OUT != 0) {
        if (tile_first < A.tiles && sub < n_q) tile_fetch<N_OUT, N_IN>(A.pl[sub], tile_first, lane, pre);
    }
    if (tile_first < A.tiles) request(tile_first);
    uint32_t st_pre[4] = {0u, 0u, 0u, 0u};

    for (uint32_t bc = 0; bc < batch; bc += BT) {
        if constexpr (XS) {
            if (bc != 0) __syncthreads();
            if (BT == 1 && (reinterpret_cast<uintptr_t>(x + (int64_t)bc * ldx) & 15) == 0) {
                constexpr uint32_t PER = 16 / sizeof(XT);
                const uint4 *src = reinterpret_cast<const uint4 *>(x + (int64_t)bc * ldx);
                uint4 *dst = reinterpret_cast<uint4 *>(xs);
                for (uint32_t v = threadIdx.x; v < n / PER; v += blockDim.x) cp_async16(dst + v, src + v);
                for (uint32_t c = (n / PER) * PER + threadIdx.x; c < n; c += blockDim.x) xs[c] = x[(int64_t)bc * ldx + c];
            } else {
#pragma unroll 4
                for (uint32_t c = threadIdx.x; c < n; c += blockDim.x) {
                    XT v[BT];
#pragma unroll
                    for (int q = 0; q < BT; ++q) v[q] = bc + q < batch ? x[(int64_t)(bc + q) * ldx + c] : XT(0.0f);
#pragma unroll
                    for (int q = 0; q < BT; ++q) xs[c * BT + q] = v[q];
                }
            }
        }
        if (bc == 0) {
            build_tables_begin(A, rows_ahead);           // block barrier: the first requests are back
            if constexpr (N_OUT != 0) {
                if (tile_first < A.tiles && sub < n_q) stage_fetch<N_OUT, N_IN>(A, A.pl[sub], pre, lane, st_pre);
            }
            cp_async_wait_all();
            build_tables_finish(A, smem);                // ends with a block barrier
        } else {
            cp_async_wait_all();
            __syncthreads();
        }
        for (uint64_t tile = tile_first; tile < A.tiles; tile += tile_step) {
            const uint64_t gw0 = tile * 32 * W;          // first 32-bit word of the tile
            const uint64_t P0 = gw0 * 32;
            if (P0 >= A.mn) continue;
            const uint64_t P1 = (P0 + 1024ull * W < A.mn) ? P0 + 1024ull * W : A.mn;
            const uint64_t r_first = P0 / n;
            if (bc != 0 || tile != tile_first) request(tile);       // not requested ahead of time
            if constexpr (N_OUT != 0) {
                for (uint32_t i = sub; i < n_q; i += wpt) {
                    TileIn<N_OUT, N_IN> in;
                    uint32_t st[4];
                    if (i == sub && bc == 0 && tile == tile_first) {
                        in = pre;
#pragma unroll
                        for (int q = 0; q < 4; ++q) st[q] = st_pre[q];
                    } else {
                        tile_fetch<N_OUT, N_IN>(A.pl[i], tile, lane, in);
                        stage_fetch<N_OUT, N_IN>(A, A.pl[i], in, lane, st);
                    }
                    tile_decode<N_OUT, N_IN>(A, A.pl[i], in, st, region + i * 32 * W, smem, stage, lane);
                }
            } else {
                for (uint32_t i = sub; i < n_q; i += wpt)
                    decode_warp_tile<N_OUT, N_IN>(A, i, tile, region + i * 32 * W, smem, stage, lane);
            }
            cp_async_wait_all();
            if (wpt == 1) __syncwarp();
            else asm volatile("bar.sync %0, %1;\n" :: "r"(1 + group), "r"(32 * wpt) : "memory");
            // Y is cleared by the kernel before this one in the stream; under a programmatic dependent
            // launch this is where its results are awaited (a no-op otherwise)
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (uint64_t r = r_first; r * n < P1; ++r) {
                const uint64_t a = r * n > P0 ? r * n : P0;
                const uint64_t b = (r + 1) * n < P1 ? (r + 1) * n : P1;
                constexpr int NR = NQ > 0 ? NQ : 1;
                float al[NR];
                const uint32_t ai = (uint32_t)(r - r_first) * n_q;
                if constexpr (NQ > 0) {
#pragma unroll
                    for (int i = 0; i < NQ; ++i)
                        al[i] = ai + i < GEMV_ALPHA_WORDS ? alpha_s[ai + i] : __ldg(alpha + r * n_q + i);
                }
                const uint32_t lw_lo = (uint32_t)((a >> 5) - gw0), lw_hi = (uint32_t)(((b - 1) >> 5) - gw0);
                const int32_t c_tile = (int32_t)((int64_t)P0 - (int64_t)(r * n));   // column of tile bit 0
                const uint32_t a_loc = (uint32_t)(a - P0), b_loc = (uint32_t)(b - P0);
                float acc[BT];
#pragma unroll
                for (int q = 0; q < BT; ++q) acc[q] = 0.0f;
                // a lane takes up to four of the segment's words at a time and visits one set mask
                // bit of each per round: four independent chains of shared-memory reads
                constexpr uint32_t K = SQNN_GEMV_WORDS_PER_ROUND;
                const uint32_t wstep = 32 * wpt;
                for (uint32_t lw0 = lw_lo + sub * 32 + lane; lw0 <= lw_hi; lw0 += wstep * K) {
                    uint32_t mk[K], wb[K][NR], k_idle[K];
                    int32_t cb[K];
                    uint32_t any = 0;
#pragma unroll
                    for (uint32_t j = 0; j < K; ++j) {
                        const uint32_t lw = lw0 + j * wstep;
                        mk[j] = 0;
                        cb[j] = c_tile + (int32_t)a_loc;    // a valid column for the idle slots
                        k_idle[j] = 0;
#pragma unroll
                        for (int i = 0; i < NR; ++i) wb[j][i] = 0;
                        if (lw <= lw_hi) {
                            uint32_t m = mask_s[lw];
                            const uint32_t lo = lw * 32;
                            if (lo < a_loc) {
                                m &= 0xffffffffu << (a_loc - lo);
                                k_idle[j] = a_loc - lo;     // bit 0 of this word belongs to the row before
                            }
                            if (lo + 32 > b_loc) m &= 0xffffffffu >> (lo + 32 - b_loc);
                            mk[j] = m;
                            cb[j] = c_tile + (int32_t)lo;
                            if constexpr (NQ > 0) {
#pragma unroll
                                for (int i = 0; i < NQ; ++i) wb[j][i] = region[i * 32 * W + lw];
                            } else {
                                wb[j][0] = lw;
                            }
                        }
                        any |= mk[j];
                    }
                    while (any) {
                        any = 0;
                        // branch-free: an exhausted word contributes value 0 at a column of this row
                        // (0 * x must not meet an x read from outside the row: it could be Inf or NaN)
#pragma unroll
                        for (uint32_t j = 0; j < K; ++j) {
                            const bool live = mk[j] != 0;
                            const uint32_t k = live ? 31u - (uint32_t)__clz((int)mk[j]) : k_idle[j];
                            mk[j] &= ~(1u << k);
                            float v = 0.0f;
                            if constexpr (NQ > 0) {
#pragma unroll
                                for (int i = 0; i < NQ; ++i) {
                                    const float t = ((wb[j][i] >> k) & 1u) ? al[i] : -al[i];
                                    v = i == 0 ? t : v + t;
                                }
                            } else {
                                for (uint32_t i = 0; i < n_q; ++i) {
                                    const float a1 = __ldg(alpha + r * n_q + i);
                                    v += ((region[i * 32 * W + wb[j][0]] >> k) & 1u) ? a1 : -a1;
                                }
                            }
                            v = live ? v : 0.0f;
                            const int32_t c = cb[j] + (int32_t)k;
                            if constexpr (XS) {
                                float xv[BT];
                                load_x<BT, XT>(xs + (uint32_t)c * BT, xv);
#pragma unroll
                                for (int q = 0; q < BT; ++q) acc[q] = fmaf(v, xv[q], acc[q]);
                            } else {
#pragma unroll
                                for (int q = 0; q < BT; ++q)
                                    if (bc + q < batch) acc[q] = fmaf(v, to_float(x[(int64_t)(bc + q) * ldx + c]), acc[q]);
                            }
                            any |= mk[j];
                        }
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
            if (wpt == 1) __syncwarp();                  // the group is done with its regions
            else asm volatile("bar.sync %0, %1;\n" :: "r"(1 + group), "r"(32 * wpt) : "memory");
        }
    }
}

// ------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------
// Picks warps per block so the dynamic shared memory fits; returns 0 if not even one warp fits.
inline uint32_t pick_warps(const DecodeArgs &A, uint32_t regions, size_t extra, size_t *smem_bytes,
                           uint32_t extra_warp_words = 0, uint32_t max_warps = 8, size_t limit = 200 * 1024)
{
    const size_t tab = (size_t)table_words(A.n_in, A.nwp, A.nchunks, A.cb) * 4;
    const size_t per_warp = ((size_t)regions * 32 * A.W + STAGE_WORDS + extra_warp_words) * 4;
    if (tab + per_warp + extra > limit) return 0;
    uint32_t warps = (uint32_t)((limit - tab - extra) / per_warp);
    if (warps > max_warps) warps = max_warps;
    *smem_bytes = tab + warps * per_warp + extra;
    return warps;
}

template <typename K>
inline int prepare(K kernel, size_t smem)
{
    return ensure_dynamic_smem(reinterpret_cast<const void *>(kernel), smem);
}

inline uint32_t grid_for(uint64_t warp_tiles, uint32_t warps, uint32_t blocks_per_sm)
{
    uint64_t need = (warp_tiles + warps - 1) / warps;
    uint64_t cap = (uint64_t)sm_count() * blocks_per_sm;
    if (need < 1) need = 1;
    return (uint32_t)(need < cap ? need : cap);
}

template <int N_OUT, int N_IN>
inline int launch_decode(const DecodeArgs &A, sqnn_out_mode mode, const uint64_t *d_mask,
                         const float *d_alpha, uint64_t n, void *d_out, cudaStream_t st)
{
    size_t smem = 0;
    if (mode == SQNN_OUT_BITS || mode == SQNN_OUT_SINK) {
        // half of the shared memory per block, so that two blocks of up to 16 warps share an SM
        const uint32_t warps = pick_warps(A, 1, 0, &smem, 0, 16, 100 * 1024);
        if (!warps) return SQNN_E_UNSUPPORTED;
        const uint64_t live = (A.words64 + 16ull * A.W - 1) / (16ull * A.W);
        if (live * A.n_q >= (1ull << 31)) return SQNN_E_UNSUPPORTED;
        const uint32_t grid = grid_for(live * A.n_q, warps, 2);
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
        const uint32_t warps = pick_warps(A, A.n_q + 1, 0, &smem);
        if (!warps) return SQNN_E_UNSUPPORTED;
        const uint64_t live = (A.words64 * 2 + 32ull * A.W - 1) / (32ull * A.W);
        const uint32_t grid = grid_for(live, warps, 4);
#define SQNN_BF16_LAUNCH(NQV)                                                                            \
    do {                                                                                                 \
        auto k = k_decode_bf16<N_OUT, N_IN, NQV>;                                                        \
        if (prepare(k, smem)) return SQNN_E_CUDA;                                                        \
        k<<<grid, warps * 32, smem, st>>>(A, (const uint32_t *)d_mask, d_alpha, n, (__nv_bfloat16 *)d_out); \
    } while (0)
        if (A.n_q == 1) SQNN_BF16_LAUNCH(1);
        else if (A.n_q == 2) SQNN_BF16_LAUNCH(2);
        else if (A.n_q == 3) SQNN_BF16_LAUNCH(3);
        else SQNN_BF16_LAUNCH(0);
#undef SQNN_BF16_LAUNCH
    }
    return cudaGetLastError() == cudaSuccess ? SQNN_OK : SQNN_E_CUDA;
}

template <int N_OUT, int N_IN, int BT, typename XT>
inline int launch_gemv_bt(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x,
                          int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t n, cudaStream_t st)
{
    // Aim at ~32 warps per SM: with few tiles, up to 4 warps share a tile; a block holds up to
    // 15 tile groups (named barriers) and 20 warps.
    const uint64_t live = (A.words64 * 2 + 32ull * A.W - 1) / (32ull * A.W);
    const uint32_t sms = (uint32_t)sm_count();
    uint32_t wpt = 1;
    // (only while a row still gives every lane of the group at least two words)
    while (wpt < 4 && live * wpt * 2 <= 32ull * sms && n >= 2048ull * wpt * 2) wpt *= 2;
    uint32_t groups = (uint32_t)((live + sms - 1) / sms);
    const uint32_t max_groups = 20 / wpt < 15 ? 20 / wpt : 15;
    groups = groups < 1 ? 1 : groups > max_groups ? max_groups : groups;
    if (wpt == 1 && groups < 4) groups = 4;
    const size_t tab = (size_t)table_words(A.n_in, A.nwp, A.nchunks, A.cb) * 4;
    const size_t per_group = ((size_t)(A.n_q + 1) * 32 * A.W + GEMV_ALPHA_WORDS + (size_t)wpt * STAGE_WORDS) * 4;
    const size_t limit = 200 * 1024;
    const size_t xbytes = (size_t)n * BT * sizeof(XT);
    bool xs = xbytes <= 160 * 1024 && tab + per_group + xbytes <= limit;
    const size_t extra = xs ? xbytes : 0;
    if (tab + per_group + extra > limit) return SQNN_E_UNSUPPORTED;
    while (groups > 1 && tab + groups * per_group + extra > limit) --groups;
    size_t smem = tab + groups * per_group + extra;
    const uint32_t warps = groups * wpt;
    const uint32_t grid = grid_for(live, groups, 2);
    // A grid that fits one block per SM asks for more than half of an SM's shared memory, so that
    // no two of its blocks are placed on the same SM while other SMs stay empty.
    if (grid <= sms && smem < 116 * 1024) smem = 116 * 1024;
    // The kernel may start while the kernel before it in the stream (the one clearing Y) still
    // runs; it waits for that kernel's results before its first atomic on Y.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(warps * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
#define SQNN_GEMV_LAUNCH(XSV, NQV)                                                                           \
    do {                                                                                                     \
        auto k = k_decode_gemv<N_OUT, N_IN, BT, XT, XSV, NQV>;                                               \
        if (prepare(k, smem)) return SQNN_E_CUDA;                                                            \
        if (cudaLaunchKernelEx(&cfg, k, A, (const uint32_t *)d_mask, d_alpha, (const XT *)d_x, ldx, batch,   \
                               d_y, ldy, (uint32_t)n, wpt) != cudaSuccess) return SQNN_E_CUDA;               \
    } while (0)
    if (!xs) SQNN_GEMV_LAUNCH(false, 0);
    else if (A.n_q == 1) SQNN_GEMV_LAUNCH(true, 1);
    else if (A.n_q == 2) SQNN_GEMV_LAUNCH(true, 2);
    else if (A.n_q == 3) SQNN_GEMV_LAUNCH(true, 3);
    else SQNN_GEMV_LAUNCH(true, 0);
#undef SQNN_GEMV_LAUNCH
    return cudaGetLastError() == cudaSuccess ? SQNN_OK : SQNN_E_CUDA;
}

template <int N_OUT, int N_IN, typename XT>
inline int launch_gemv(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x,
                       int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t n, cudaStream_t st)
{
    if (batch == 1) return launch_gemv_bt<N_OUT, N_IN, 1, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st);
    if (batch == 2) return launch_gemv_bt<N_OUT, N_IN, 2, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st);
    if (batch <= 4) return launch_gemv_bt<N_OUT, N_IN, 4, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st);
    return launch_gemv_bt<N_OUT, N_IN, 8, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, n, st);
}


// One network shape = one translation unit (sqnn_shape.cu compiled with -DSQNN_NO / -DSQNN_NI).
template <int N_OUT, int N_IN>
int decode_shape(const DecodeArgs &A, sqnn_out_mode mode, const uint64_t *d_mask, const float *d_alpha,
                 uint64_t n, void *d_out, cudaStream_t st);
template <int N_OUT, int N_IN>
int gemv_shape(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x, int x_dtype,
               int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t n, cudaStream_t st);

}  // namespace sqnn
