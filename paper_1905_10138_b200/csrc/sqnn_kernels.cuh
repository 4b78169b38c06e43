// Decode kernels (packed bits, bf16 weights, checksum sink) as templates over the network
// shape, with their launchers.
#pragma once
#include "sqnn.h"
#include "sqnn_decode.cuh"
#include "sqnn_launch.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace sqnn {

// ------------------------------------------------------------------------------------------
// shared-memory layout of the warp-tile kernels:  [tables][warp 0: regions][warp 1: ...]...
// a region is a run of 32 * W words (one kernel tile of one plane)
// ------------------------------------------------------------------------------------------
SQNN_DEV uint64_t tile_word64(const uint32_t *region, uint32_t q)
{
    const uint2 v = *reinterpret_cast<const uint2 *>(region + 2 * q);
    return (uint64_t)v.x | ((uint64_t)v.y << 32);
}

template <int N_OUT>
SQNN_DEV uint32_t words_per_lane(const DecodeArgs &A)
{
    if constexpr (N_OUT != 0) return N_OUT / 4;
    else return A.W;
}

// Position of a warp in the list of (plane, tile) items, advanced without division.
struct TilePos {
    uint32_t plane, tile;
};
SQNN_DEV TilePos advance(TilePos p, uint32_t by, uint32_t live, uint32_t n_q)
{
    p.tile += by;
    while (p.plane < n_q && p.tile >= live) { p.tile -= live; ++p.plane; }
    return p;
}

// K1: decoded planes as packed bits.  One kernel tile = 16 * W consecutive uint64 of one plane,
// built in the warp's shared-memory region and written out by a bulk copy while the warp already
// works on its next tile (it waits for the copy only when it is about to overwrite the region).
// Global loads run two tiles ahead: while tile t is expanded, the seeds and the patch offsets of
// tile t + 2 and the patch entries of tile t + 1 (whose offsets arrived an iteration ago) are in
// flight.  REP: the lookup tables sit in shared memory in replicated form (every lane of a load
// wavefront reads its own copy in its own banks); filling them takes a few microseconds, which pays
// once a warp has several tiles to decode.  One block per SM.
// SINK = true: XOR of all those words instead of storing them.
constexpr uint32_t DECODE_BITS_THREADS = 768;
template <int N_OUT, int N_IN>
inline uint32_t decode_bits_table_words(const DecodeArgs &A, bool rep)
{
    if constexpr (N_OUT != 0) return rep ? table_words_replicated(N_OUT, N_IN) : A.tab_words;
    else return A.tab_words;
}
// ONE_PLANE: the layer has a single plane (its stream pointers are then kernel constants instead of
// being looked up by a plane index in every step).
template <int N_OUT, int N_IN, bool SINK, bool ONE_PLANE, bool REP>
__global__ void __launch_bounds__(DECODE_BITS_THREADS, 1)
k_decode_bits(DecodeArgs A, uint64_t *__restrict__ out)
{
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t tab_words_s;
    if constexpr (N_OUT != 0 && REP) {
        tab_words_s = table_words_replicated(N_OUT, N_IN);       // filled below, after the first fetches are out
    } else {
        tables_request(A, smem);
        tab_words_s = A.tab_words;
    }
    const uint32_t W = words_per_lane<N_OUT>(A);
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    uint32_t *region = smem + tab_words_s + warp * 32 * W;
    const uint64_t tail_bits = A.mn & 63;
    // tiles that hold at least one real word, per plane (the launcher keeps the count below 2^31)
    const uint32_t live = (uint32_t)((A.words64 + 16 * W - 1) / (16 * W));
    // tiles before this one lie wholly inside the plane and end on a whole word
    const uint32_t full_tiles = (uint32_t)(A.words64 / (16 * W)) -
                                ((tail_bits != 0 && A.words64 % (16 * W) == 0) ? 1u : 0u);
    const uint32_t stride = gridDim.x * nwarps;
    const TilePos p_first = advance(TilePos{0u, 0u}, blockIdx.x * nwarps + warp, live, A.n_q);
    uint64_t sink = 0;

    auto write_out = [&](TilePos p) {
        uint64_t *pbase = out + (uint64_t)p.plane * A.words64;
        const uint64_t q0 = (uint64_t)p.tile * (16 * W);     // first uint64 of the tile inside the plane
        uint64_t *dst = pbase + q0;
        if (!SINK && p.tile < full_tiles && (reinterpret_cast<uintptr_t>(pbase) & 15) == 0) {
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
    };

    auto plane_of = [&](const TilePos &p) -> const PlanePtrs & { return ONE_PLANE ? A.pl[0] : A.pl[p.plane]; };
    if constexpr (N_OUT != 0) {
        using S = Shape<N_OUT, N_IN>;
        // Three sets of registers take turns as "current", "next" and "the one after": a step works on
        // the current tile while it requests the patch entries of the next (its offsets arrived a step
        // ago) and the seeds and offsets of the one after.  Nothing in flight is ever copied.
        TilePos pa = p_first, pb = advance(pa, stride, live, A.n_q), pc{A.n_q, 0u};
        TileSeeds<N_OUT, N_IN> sa, sb, sc;
        TileRun ra{0u, 0u}, rb{0u, 0u}, rc{0u, 0u};
        uint32_t wa[PATCH_AHEAD], wb[PATCH_AHEAD], wc[PATCH_AHEAD];
        if (pa.plane < A.n_q) { fetch_seeds<N_OUT, N_IN>(plane_of(pa), pa.tile, lane, sa); ra = fetch_run(plane_of(pa), pa.tile); }
        if (pb.plane < A.n_q) { fetch_seeds<N_OUT, N_IN>(plane_of(pb), pb.tile, lane, sb); rb = fetch_run(plane_of(pb), pb.tile); }
        if constexpr (REP) tables_replicate<entry_words_padded(N_OUT)>(A, smem);
        if (pa.plane < A.n_q) fetch_patches(A, plane_of(pa), ra, lane, wa);
        if constexpr (!REP) cp_async_wait_all();
        __syncthreads();                                 // the tables are in place
        auto step = [&](TilePos &p0, TileSeeds<N_OUT, N_IN> &s0, TileRun &r0, uint32_t (&w0)[PATCH_AHEAD],
                        TilePos &p1, TileRun &r1, uint32_t (&w1)[PATCH_AHEAD],
                        TilePos &p2, TileSeeds<N_OUT, N_IN> &s2, TileRun &r2) {
            // everything this step consumes was requested at least a step ago: take delivery of it now,
            // before the loads of this step are issued
#pragma unroll
            for (uint32_t k = 0; k < S::NRAW; ++k) s0.raw[k] = settle(s0.raw[k]);
#pragma unroll
            for (uint32_t k = 0; k < PATCH_AHEAD; ++k) w0[k] = settle(w0[k]);
            r0.base = settle(r0.base); r0.end = settle(r0.end);
            r1.base = settle(r1.base); r1.end = settle(r1.end);
            p2 = advance(p1, stride, live, A.n_q);
            if (p1.plane < A.n_q) fetch_patches(A, plane_of(p1), r1, lane, w1);
            if (p2.plane < A.n_q) { fetch_seeds<N_OUT, N_IN>(plane_of(p2), p2.tile, lane, s2); r2 = fetch_run(plane_of(p2), p2.tile); }
            tile_expand<N_OUT, N_IN, !SINK, REP>(s0, region, smem, lane);
            __syncwarp();
            tile_patch(A, plane_of(p0), r0, w0, region, 0u, S::TILE_BITS, lane);
            __syncwarp();
            write_out(p0);
            return p1.plane < A.n_q;
        };
        if (pa.plane < A.n_q) {
            for (;;) {
                if (!step(pa, sa, ra, wa, pb, rb, wb, pc, sc, rc)) break;
                if (!step(pb, sb, rb, wb, pc, rc, wc, pa, sa, ra)) break;
                if (!step(pc, sc, rc, wc, pa, ra, wa, pb, sb, rb)) break;
            }
        }
    } else {
        cp_async_wait_all();
        __syncthreads();
        for (TilePos p = p_first; p.plane < A.n_q; p = advance(p, stride, live, A.n_q)) {
            decode_ktile_generic(A, p.plane, p.tile, region, smem, lane);
            write_out(p);
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

// Starts the copy of `words` mask words (first word gw0) into shared memory: 16-byte
// asynchronous copies where a whole vector is in range, plain loads (zero past the end) otherwise.
// `words` is a multiple of 4 and gw0 a multiple of 4.  The calling threads are `nthreads` threads
// numbered `t`.  Finish with a cp.async wait and a barrier over those threads.
SQNN_DEV void stage_mask(uint32_t *mask_s, const uint32_t *__restrict__ mask32, uint64_t gw0, uint64_t mask_words,
                         uint32_t words, uint32_t t, uint32_t nthreads, bool vec_ok)
{
    for (uint32_t v = t; v < words / 4; v += nthreads) {
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
// With one plane a weight is +-bf16(alpha) or 0, so four weights at a time come from a table indexed
// by (mask nibble, bit nibble): a keep-mask and a sign-flip per weight, applied to the row's scale
// with one logic operation per pair of weights (exact for any alpha; a pruned weight is +0).  The
// table is kept in 8 copies, lane l reads copy l % 8, so that lookups of different entries do not
// share banks.
constexpr uint32_t BF16_LUT_COPIES = 8;
constexpr uint32_t BF16_LUT_WORDS = 256 * BF16_LUT_COPIES * 4;
constexpr uint32_t BF16_THREADS = 768;                   // one block per SM, as many warps as shared memory holds
template <int N_OUT, int N_IN, int NQ>
__global__ void __launch_bounds__(BF16_THREADS, 1)
k_decode_bf16(DecodeArgs A, const uint32_t *__restrict__ mask32, const float *__restrict__ alpha,
              uint64_t n, __nv_bfloat16 *__restrict__ out)
{
    extern __shared__ __align__(16) uint32_t smem[];
    tables_request(A, smem);
    uint4 *lut = reinterpret_cast<uint4 *>(smem + A.tab_words);          // [256][copies]: keep masks (x, y), sign flips (z, w)
    if constexpr (NQ == 1) {
        for (uint32_t e = threadIdx.x; e < 256; e += blockDim.x) {
            uint32_t keep[4], flip[4];
#pragma unroll
            for (uint32_t k = 0; k < 4; ++k) {
                const uint32_t m = (e >> (4 + k)) & 1u, b = (e >> k) & 1u;
                keep[k] = m ? 0xffffu : 0u;
                flip[k] = (m && !b) ? 0x8000u : 0u;
            }
            const uint4 v = make_uint4(keep[0] | (keep[1] << 16), keep[2] | (keep[3] << 16),
                                       flip[0] | (flip[1] << 16), flip[2] | (flip[3] << 16));
#pragma unroll
            for (uint32_t c = 0; c < BF16_LUT_COPIES; ++c) lut[e * BF16_LUT_COPIES + c] = v;
        }
    }
    cp_async_wait_all();
    __syncthreads();
    const uint32_t W = words_per_lane<N_OUT>(A);
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t n_q = A.n_q;
    const uint32_t per_warp = (n_q + 1) * 32 * W;
    uint32_t *region = smem + A.tab_words + (NQ == 1 ? BF16_LUT_WORDS : 0u) + warp * per_warp;
    uint32_t *mask_s = region + n_q * 32 * W;
    const uint8_t *mask_s8 = reinterpret_cast<const uint8_t *>(mask_s);
    const uint32_t tile_bytes = 128 * W;                 // bytes of bits per tile and plane
    const uint64_t mask_words = A.words64 * 2;
    const bool mask_vec = (reinterpret_cast<uintptr_t>(mask32) & 15) == 0;
    constexpr int NR = NQ > 0 ? NQ : 1;
    for (uint64_t tile = (uint64_t)blockIdx.x * nwarps + warp; tile < A.ktiles; tile += (uint64_t)gridDim.x * nwarps) {
        const uint64_t p_tile = tile * (uint64_t)tile_bytes * 8;
        if (p_tile >= A.mn) continue;
        stage_mask(mask_s, mask32, tile * 32 * W, mask_words, 32 * W, lane, 32, mask_vec);
        for (uint32_t i = 0; i < n_q; ++i)
            decode_warp_tile<N_OUT, N_IN>(A, i, tile, region + i * 32 * W, smem, lane);
        cp_async_wait_all();
        __syncwarp();
        // byte t of the tile's bit run holds the weights p_tile + 8 t ..; bytes below nfull lie wholly inside
        // the plane, bytes below nbytes hold at least one of its weights
        const uint64_t left = A.mn - p_tile;
        const uint32_t nbytes = left >= 8ull * tile_bytes ? tile_bytes : (uint32_t)((left + 7) / 8);
        const uint32_t nfull = left >= 8ull * tile_bytes ? tile_bytes : (uint32_t)(left / 8);
        __nv_bfloat16 *out_t = out + p_tile;
        const uint8_t *bits_s8 = reinterpret_cast<const uint8_t *>(region);
        const uint32_t lut_lane = lane & (BF16_LUT_COPIES - 1);
        uint64_t r = (p_tile + 8ull * lane) / n;         // row and column of the lane's first weight
        uint64_t c = (p_tile + 8ull * lane) - r * n;
        float al[NR];
        uint32_t ab2 = 0;                                // bf16(alpha) of the row, twice (one plane)
        uint64_t r_al = ~0ull;
        for (uint32_t t = lane; t < nbytes; t += 32, c += 256) {
            while (c >= n) { c -= n; ++r; }
            const uint32_t mk = mask_s8[t];
            const uint64_t p = p_tile + 8ull * t;        // (the slow path's)
            if (NQ == 1 && c + 8 <= n && t < nfull) {
                if (r != r_al) {
                    al[0] = __ldg(alpha + r);
                    r_al = r;
                    const uint32_t ab = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(al[0]));
                    ab2 = ab | (ab << 16);
                }
                const uint32_t bt = bits_s8[t];
                const uint4 e0 = lut[((((mk & 15u) << 4) | (bt & 15u))) * BF16_LUT_COPIES + lut_lane];
                const uint4 e1 = lut[((mk & 0xf0u) | (bt >> 4)) * BF16_LUT_COPIES + lut_lane];
                *reinterpret_cast<uint4 *>(out_t + 8 * t) = make_uint4((ab2 & e0.x) ^ e0.z, (ab2 & e0.y) ^ e0.w,
                                                                       (ab2 & e1.x) ^ e1.z, (ab2 & e1.y) ^ e1.w);
            } else if (NQ > 0 && c + 8 <= n && t < nfull) {
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
                *reinterpret_cast<uint4 *>(out_t + 8 * t) = make_uint4(w[0], w[1], w[2], w[3]);
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

// ------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------
// Picks warps per block so the dynamic shared memory fits; returns 0 if not even one warp fits.
inline uint32_t pick_warps(const DecodeArgs &A, uint32_t regions, size_t *smem_bytes, uint32_t max_warps, size_t limit)
{
    const size_t tab = (size_t)A.tab_words * 4;
    const size_t per_warp = (size_t)regions * 32 * A.W * 4;
    if (tab + per_warp > limit) return 0;
    uint32_t warps = (uint32_t)((limit - tab) / per_warp);
    if (warps > max_warps) warps = max_warps;
    *smem_bytes = tab + warps * per_warp;
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
        // one block per SM: the tables and one region per warp.  The replicated tables are worth their
        // fill only when a warp gets several tiles.
        const uint64_t live = (A.words64 + 16ull * A.W - 1) / (16ull * A.W);
        if (live * A.n_q >= (1ull << 31)) return SQNN_E_UNSUPPORTED;
        const bool rep = N_OUT != 0 && live * A.n_q >= 3ull * (DECODE_BITS_THREADS / 32) * (uint64_t)sm_count();
        const size_t tab = (size_t)decode_bits_table_words<N_OUT, N_IN>(A, rep) * 4, per_warp = (size_t)32 * A.W * 4;
        const size_t limit = 224 * 1024;
        if (tab + per_warp > limit) return SQNN_E_UNSUPPORTED;
        uint32_t warps = (uint32_t)((limit - tab) / per_warp);
        if (warps > DECODE_BITS_THREADS / 32) warps = DECODE_BITS_THREADS / 32;
        smem = tab + warps * per_warp;
        const uint32_t grid = grid_for(live * A.n_q, warps, 1);
#define SQNN_BITS_LAUNCH2(SINKV, ONEV, REPV)                                                             \
    do {                                                                                                 \
        auto k = k_decode_bits<N_OUT, N_IN, SINKV, ONEV, REPV>;                                          \
        if (prepare(k, smem)) return SQNN_E_CUDA;                                                        \
        k<<<grid, warps * 32, smem, st>>>(A, (uint64_t *)d_out);                                         \
    } while (0)
#define SQNN_BITS_LAUNCH(SINKV, ONEV)                                                                    \
    do {                                                                                                 \
        if (rep) SQNN_BITS_LAUNCH2(SINKV, ONEV, true); else SQNN_BITS_LAUNCH2(SINKV, ONEV, false);       \
    } while (0)
        if (mode == SQNN_OUT_BITS) {
            if (A.n_q == 1) SQNN_BITS_LAUNCH(false, true); else SQNN_BITS_LAUNCH(false, false);
        } else {
            if (cudaMemsetAsync(d_out, 0, 8, st) != cudaSuccess) return SQNN_E_CUDA;
            if (A.n_q == 1) SQNN_BITS_LAUNCH(true, true); else SQNN_BITS_LAUNCH(true, false);
        }
#undef SQNN_BITS_LAUNCH2
#undef SQNN_BITS_LAUNCH
    } else {
        const size_t lut_bytes = A.n_q == 1 ? (size_t)BF16_LUT_WORDS * 4 : 0;
        const uint32_t warps = pick_warps(A, A.n_q + 1, &smem, BF16_THREADS / 32, 224 * 1024 - lut_bytes);
        if (!warps) return SQNN_E_UNSUPPORTED;
        smem += lut_bytes;
        const uint64_t live = (A.words64 * 2 + 32ull * A.W - 1) / (32ull * A.W);
        const uint32_t grid = grid_for(live, warps, 1);
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

// One network shape = one translation unit (sqnn_shape.cu compiled with -DSQNN_NO / -DSQNN_NI).
template <int N_OUT, int N_IN>
int decode_shape(const DecodeArgs &A, sqnn_out_mode mode, const uint64_t *d_mask, const float *d_alpha,
                 uint64_t n, void *d_out, cudaStream_t st);
template <int N_OUT, int N_IN>
int gemv_shape(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x, int x_dtype,
               int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t m, uint64_t n, cudaStream_t st);

}  // namespace sqnn
