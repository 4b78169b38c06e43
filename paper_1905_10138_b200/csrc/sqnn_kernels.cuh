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
    build_tables<N_OUT, N_IN>(A, smem);
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
    build_tables<N_OUT, N_IN>(A, smem);
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

// a / b with the short 32-bit division whenever a fits 32 bits (it does for layers below 2^32 weights).
SQNN_DEV uint64_t div_u64_u32(uint64_t a, uint32_t b)
{
    return (a >> 32) == 0 ? (uint64_t)((uint32_t)a / b) : a / b;
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

// Shared-memory accesses by 32-bit shared address (no generic-address arithmetic in the hot loop).
SQNN_DEV uint32_t lds_u32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
// v = [a] if `take` is non-zero, otherwise v keeps its value.
SQNN_DEV void lds_u32_if(uint32_t &v, uint32_t a, uint32_t take)
{
    asm volatile("{ .reg .pred q; setp.ne.u32 q, %2, 0; @q ld.shared.u32 %0, [%1]; }" : "+r"(v) : "r"(a), "r"(take));
}
// acc = v * x + acc if `live` is non-zero (a skipped lane must not touch acc: its x may be anything).
SQNN_DEV void fma_if(float &acc, float v, float x, uint32_t live)
{
    asm("{ .reg .pred q; setp.ne.u32 q, %3, 0; @q fma.rn.f32 %0, %1, %2, %0; }" : "+f"(acc) : "f"(v), "f"(x), "r"(live));
}
// BT activations of one column from shared address a (xs[c][BT]).
template <int BT, typename XT>
SQNN_DEV void lds_x(uint32_t a, float (&v)[BT])
{
    if constexpr (sizeof(XT) == 2) {
        if constexpr (BT == 1) {
            unsigned short h;
            asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(a));
            v[0] = __uint_as_float((uint32_t)h << 16);
        } else if constexpr (BT == 2) {
            const uint32_t w = lds_u32(a);
            v[0] = __uint_as_float(w << 16); v[1] = __uint_as_float(w & 0xffff0000u);
        } else if constexpr (BT == 4) {
            uint32_t w0, w1;
            asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(w0), "=r"(w1) : "r"(a));
            v[0] = __uint_as_float(w0 << 16); v[1] = __uint_as_float(w0 & 0xffff0000u);
            v[2] = __uint_as_float(w1 << 16); v[3] = __uint_as_float(w1 & 0xffff0000u);
        } else {
            static_assert(BT == 8, "batch chunk of 1, 2, 4 or 8");
            uint32_t w[4];
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(a));
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                v[2 * q] = __uint_as_float(w[q] << 16);
                v[2 * q + 1] = __uint_as_float(w[q] & 0xffff0000u);
            }
        }
    } else {
        if constexpr (BT == 1) {
            v[0] = __uint_as_float(lds_u32(a));
        } else if constexpr (BT == 2) {
            asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v[0]), "=f"(v[1]) : "r"(a));
        } else {
#pragma unroll
            for (int q = 0; q < BT; q += 4)
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(v[q]), "=f"(v[q + 1]), "=f"(v[q + 2]), "=f"(v[q + 3]) : "r"(a + 4 * q));
        }
    }
}

// Head of one step of the walk below, written out instruction by instruction: takes the highest care bit
// k1 and then the lowest care bit k2 out of `mk` (k = 0 where there is none), reports in live1 / live2
// whether there was one, and forms the weight values (+-alpha_1) + (+-alpha_2) + ... from bits k1 and k2
// of the plane words.
SQNN_DEV void walk_head(uint32_t &mk, uint32_t &k1, uint32_t &live1, float &v1, uint32_t &k2, uint32_t &live2,
                        float &v2, const uint32_t (&wb)[1], const float (&al)[1], const float (&ng)[1])
{
    asm("{\n .reg .pred pl, ps;\n .reg .b32 t, u;\n .reg .f32 w;\n"
        " mov.u32 %2, %6;\n setp.ne.u32 pl, %6, 0;\n bfind.u32 %0, %6;\n selp.u32 %0, %0, 0, pl;\n"
        " shl.b32 t, 1, %0;\n @pl xor.b32 %6, %6, t;\n"
        " and.b32 u, %7, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 %1, %8, %9, ps;\n"
        " neg.s32 t, %6;\n and.b32 t, t, %6;\n mov.u32 %5, t;\n bfind.u32 %3, t;\n setp.ne.u32 pl, t, 0;\n"
        " selp.u32 %3, %3, 0, pl;\n xor.b32 %6, %6, t;\n"
        " and.b32 u, %7, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 %4, %8, %9, ps;\n}"
        : "=&r"(k1), "=&f"(v1), "=&r"(live1), "=&r"(k2), "=&f"(v2), "=&r"(live2), "+r"(mk)
        : "r"(wb[0]), "f"(al[0]), "f"(ng[0]));
}
SQNN_DEV void walk_head(uint32_t &mk, uint32_t &k1, uint32_t &live1, float &v1, uint32_t &k2, uint32_t &live2,
                        float &v2, const uint32_t (&wb)[2], const float (&al)[2], const float (&ng)[2])
{
    asm("{\n .reg .pred pl, ps;\n .reg .b32 t, u;\n .reg .f32 w;\n"
        " mov.u32 %2, %6;\n setp.ne.u32 pl, %6, 0;\n bfind.u32 %0, %6;\n selp.u32 %0, %0, 0, pl;\n"
        " shl.b32 t, 1, %0;\n @pl xor.b32 %6, %6, t;\n"
        " and.b32 u, %7, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 %1, %9, %11, ps;\n and.b32 u, %8, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 w, %10, %12, ps;\n add.rn.f32 %1, %1, w;\n"
        " neg.s32 t, %6;\n and.b32 t, t, %6;\n mov.u32 %5, t;\n bfind.u32 %3, t;\n setp.ne.u32 pl, t, 0;\n"
        " selp.u32 %3, %3, 0, pl;\n xor.b32 %6, %6, t;\n"
        " and.b32 u, %7, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 %4, %9, %11, ps;\n and.b32 u, %8, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 w, %10, %12, ps;\n add.rn.f32 %4, %4, w;\n}"
        : "=&r"(k1), "=&f"(v1), "=&r"(live1), "=&r"(k2), "=&f"(v2), "=&r"(live2), "+r"(mk)
        : "r"(wb[0]), "r"(wb[1]), "f"(al[0]), "f"(al[1]), "f"(ng[0]), "f"(ng[1]));
}
SQNN_DEV void walk_head(uint32_t &mk, uint32_t &k1, uint32_t &live1, float &v1, uint32_t &k2, uint32_t &live2,
                        float &v2, const uint32_t (&wb)[3], const float (&al)[3], const float (&ng)[3])
{
    asm("{\n .reg .pred pl, ps;\n .reg .b32 t, u;\n .reg .f32 w;\n"
        " mov.u32 %2, %6;\n setp.ne.u32 pl, %6, 0;\n bfind.u32 %0, %6;\n selp.u32 %0, %0, 0, pl;\n"
        " shl.b32 t, 1, %0;\n @pl xor.b32 %6, %6, t;\n"
        " and.b32 u, %7, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 %1, %10, %13, ps;\n and.b32 u, %8, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 w, %11, %14, ps;\n add.rn.f32 %1, %1, w;\n and.b32 u, %9, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 w, %12, %15, ps;\n add.rn.f32 %1, %1, w;\n"
        " neg.s32 t, %6;\n and.b32 t, t, %6;\n mov.u32 %5, t;\n bfind.u32 %3, t;\n setp.ne.u32 pl, t, 0;\n"
        " selp.u32 %3, %3, 0, pl;\n xor.b32 %6, %6, t;\n"
        " and.b32 u, %7, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 %4, %10, %13, ps;\n and.b32 u, %8, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 w, %11, %14, ps;\n add.rn.f32 %4, %4, w;\n and.b32 u, %9, t;\n setp.ne.u32 ps, u, 0;\n selp.f32 w, %12, %15, ps;\n add.rn.f32 %4, %4, w;\n}"
        : "=&r"(k1), "=&f"(v1), "=&r"(live1), "=&r"(k2), "=&f"(v2), "=&r"(live2), "+r"(mk)
        : "r"(wb[0]), "r"(wb[1]), "r"(wb[2]), "f"(al[0]), "f"(al[1]), "f"(al[2]), "f"(ng[0]), "f"(ng[1]), "f"(ng[2]));
}

// Tail of one step of the walk: when the lane's word is used up (mk == 0) it moves to its next word at
// shared address wa + step_a if that is still inside the segment (<= hi_a) -- mask word into mk (the
// segment's last word trimmed by last_mask), plane words into wb, xa advanced by step_x -- and is done
// otherwise (it then stays where it is).  Returns, the same in every lane, whether any lane is not done.
// Plane i's word lies (NQ - i) * plane_bytes below the mask word.
SQNN_DEV uint32_t walk_tail(uint32_t &mk, uint32_t &wa, uint32_t &xa, uint32_t (&wb)[1], uint32_t step_a,
                            uint32_t hi_a, uint32_t step_x, uint32_t plane_bytes, uint32_t last_mask)
{
    uint32_t cont;
    asm volatile("{\n .reg .pred pz, pt, pd, pa, pq;\n .reg .b32 na, a0;\n"
        " setp.eq.u32 pz, %1, 0;\n add.u32 na, %2, %5;\n setp.le.and.u32 pt, na, %6, pz;\n"
        " setp.gt.and.u32 pd, na, %6, pz;\n vote.sync.any.pred pa, !pd, 0xffffffff;\n selp.u32 %0, 1, 0, pa;\n"
        " sub.u32 a0, na, %8;\n"
        " @pt ld.shared.u32 %1, [na];\n @pt ld.shared.u32 %4, [a0];\n"
        " @pt mov.u32 %2, na;\n @pt add.u32 %3, %3, %7;\n"
        " setp.eq.and.u32 pq, na, %6, pt;\n @pq and.b32 %1, %1, %9;\n}"
        : "=&r"(cont), "+r"(mk), "+r"(wa), "+r"(xa), "+r"(wb[0])
        : "r"(step_a), "r"(hi_a), "r"(step_x), "r"(plane_bytes), "r"(last_mask));
    return cont;
}
SQNN_DEV uint32_t walk_tail(uint32_t &mk, uint32_t &wa, uint32_t &xa, uint32_t (&wb)[2], uint32_t step_a,
                            uint32_t hi_a, uint32_t step_x, uint32_t plane_bytes, uint32_t last_mask)
{
    uint32_t cont;
    asm volatile("{\n .reg .pred pz, pt, pd, pa, pq;\n .reg .b32 na, a0, a1;\n"
        " setp.eq.u32 pz, %1, 0;\n add.u32 na, %2, %6;\n setp.le.and.u32 pt, na, %7, pz;\n"
        " setp.gt.and.u32 pd, na, %7, pz;\n vote.sync.any.pred pa, !pd, 0xffffffff;\n selp.u32 %0, 1, 0, pa;\n"
        " sub.u32 a1, na, %9;\n sub.u32 a0, a1, %9;\n"
        " @pt ld.shared.u32 %1, [na];\n @pt ld.shared.u32 %4, [a0];\n @pt ld.shared.u32 %5, [a1];\n"
        " @pt mov.u32 %2, na;\n @pt add.u32 %3, %3, %8;\n"
        " setp.eq.and.u32 pq, na, %7, pt;\n @pq and.b32 %1, %1, %10;\n}"
        : "=&r"(cont), "+r"(mk), "+r"(wa), "+r"(xa), "+r"(wb[0]), "+r"(wb[1])
        : "r"(step_a), "r"(hi_a), "r"(step_x), "r"(plane_bytes), "r"(last_mask));
    return cont;
}
SQNN_DEV uint32_t walk_tail(uint32_t &mk, uint32_t &wa, uint32_t &xa, uint32_t (&wb)[3], uint32_t step_a,
                            uint32_t hi_a, uint32_t step_x, uint32_t plane_bytes, uint32_t last_mask)
{
    uint32_t cont;
    asm volatile("{\n .reg .pred pz, pt, pd, pa, pq;\n .reg .b32 na, a0, a1, a2;\n"
        " setp.eq.u32 pz, %1, 0;\n add.u32 na, %2, %7;\n setp.le.and.u32 pt, na, %8, pz;\n"
        " setp.gt.and.u32 pd, na, %8, pz;\n vote.sync.any.pred pa, !pd, 0xffffffff;\n selp.u32 %0, 1, 0, pa;\n"
        " sub.u32 a2, na, %10;\n sub.u32 a1, a2, %10;\n sub.u32 a0, a1, %10;\n"
        " @pt ld.shared.u32 %1, [na];\n @pt ld.shared.u32 %4, [a0];\n @pt ld.shared.u32 %5, [a1];\n @pt ld.shared.u32 %6, [a2];\n"
        " @pt mov.u32 %2, na;\n @pt add.u32 %3, %3, %9;\n"
        " setp.eq.and.u32 pq, na, %8, pt;\n @pq and.b32 %1, %1, %11;\n}"
        : "=&r"(cont), "+r"(mk), "+r"(wa), "+r"(xa), "+r"(wb[0]), "+r"(wb[1]), "+r"(wb[2])
        : "r"(step_a), "r"(hi_a), "r"(step_x), "r"(plane_bytes), "r"(last_mask));
    return cont;
}

// The walk of one row segment of a decoded tile (GEMV kernel), activations in shared memory as xs[c][BT].
// Each lane walks its own words of the segment -- word `lw`, then every `wstep`-th up to `lw_hi` -- from
// both ends (two care bits a step), and moves on to its next word as soon as the current one is used up: lanes
// do not wait for one another between words, so the warp runs for as long as its busiest lane has care
// bits.  The body is free of branches under a warp-uniform loop condition, so the lanes stay converged.
// Only care positions contribute; an idle lane's load stays inside shared memory and its result is dropped.
//   mask_sa      shared address of the tile's mask words; plane i's words lie (NQ - i) * plane_bytes below
//   xs_sa        shared address of xs[0]
//   c_tile       column (in this row) of bit 0 of the tile; may be negative
template <int BT, typename XT, int NQ>
SQNN_DEV void walk_segment(uint32_t mask_sa, uint32_t plane_bytes, uint32_t xs_sa, uint32_t lw, uint32_t lw_lo,
                           uint32_t lw_hi, uint32_t wstep, uint32_t first_mask, uint32_t last_mask, int32_t c_tile,
                           const float (&al)[NQ], float (&acc)[BT])
{
    constexpr uint32_t XB = BT * sizeof(XT);                 // bytes of one column of xs
    const uint32_t hi_a = mask_sa + 4 * lw_hi;
    const uint32_t step_a = 4 * wstep, step_x = 32 * XB * wstep;
    uint32_t wa = mask_sa + 4 * lw;                          // shared address of the lane's current mask word
    uint32_t xa = xs_sa + (uint32_t)(c_tile + (int32_t)(32 * lw)) * XB;    // ... of the column of its bit 0
    const uint32_t more = lw <= lw_hi ? 1u : 0u;
    uint32_t mk = 0, wb[NQ];
#pragma unroll
    for (int i = 0; i < NQ; ++i) wb[i] = 0;
    lds_u32_if(mk, wa, more);
#pragma unroll
    for (int i = 0; i < NQ; ++i) lds_u32_if(wb[i], wa - (NQ - i) * plane_bytes, more);
    if (lw == lw_lo) mk &= first_mask;
    if (lw == lw_hi) mk &= last_mask;
    // a lane without a word in this segment parks on the segment's last word with nothing to do
    if (!more) { wa = hi_a; xa = xs_sa + (uint32_t)(c_tile + (int32_t)(32 * lw_hi)) * XB; }
    float ng[NQ];
#pragma unroll
    for (int i = 0; i < NQ; ++i) ng[i] = -al[i];
    uint32_t cont = __any_sync(0xffffffffu, more != 0) ? 1u : 0u;
    while (cont) {
        uint32_t k1, k2, live1, live2;
        float v1, v2, xv1[BT], xv2[BT];
        walk_head(mk, k1, live1, v1, k2, live2, v2, wb, al, ng);
        lds_x<BT, XT>(xa + k1 * XB, xv1);
        lds_x<BT, XT>(xa + k2 * XB, xv2);
#pragma unroll
        for (int q = 0; q < BT; ++q) fma_if(acc[q], v1, xv1[q], live1);
#pragma unroll
        for (int q = 0; q < BT; ++q) fma_if(acc[q], v2, xv2[q], live2);
        cont = walk_tail(mk, wa, xa, wb, step_a, hi_a, step_x, plane_bytes, last_mask);
    }
}

// Words of per-warp scratch the GEMV kernel keeps for the scales of the rows a tile touches.
constexpr uint32_t GEMV_ALPHA_WORDS = 64;

// K3: decryption fused with Y[b][r] = sum_c W[r][c] X[b][c] for small batch, fp32 accumulate.
// A group of 1 to 4 warps shares a tile: its warps decode the tile's planes into shared memory (one
// plane per warp), then all of them walk the row segments the tile covers.  In a segment each lane
// owns every (32 * warps)-th 32-bit word (with short rows every 32nd word of the segments that are its
// warp's turn); it takes two care bits of its word a step, rebuilds the weight values
// (+-alpha_1) + (+-alpha_2) + ... from the plane words and accumulates value * x, and moves to its next
// word as soon as this one is used up (walk_segment).  Partial sums of a row segment are reduced over
// the warp and added to Y with one atomic per (row, b).
// Everything the walk reads is on chip by then: the tile's mask words arrive by cp.async while
// the tile is decoded, the scales of its rows are fetched up front, and (XS = true) the
// activations of the current batch chunk sit in shared memory as xs[c][BT].
// NQ = number of planes when it is 1, 2 or 3 (scales and plane words stay in registers), 0 = any.
template <int N_OUT, int N_IN, int BT, typename XT, bool XS, int NQ>
__global__ void __launch_bounds__(640)
k_decode_gemv(DecodeArgs A, const uint32_t *__restrict__ mask32, const float *__restrict__ alpha,
              const XT *__restrict__ x, int64_t ldx, uint32_t batch, float *__restrict__ y,
              int64_t ldy, uint32_t n, uint32_t wpt, uint32_t seg_par)
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
    const uint64_t alpha_count = div_u64_u32(A.mn, n) * n_q;
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
            const uint64_t r_first = div_u64_u32(gw0 * 32, n);
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
            // the asynchronous copies (activations, mask, scales) are awaited inside, before the closing barrier
            build_tables_finish<N_OUT, N_IN, true>(A, smem);
        } else {
            cp_async_wait_all();
            __syncthreads();
        }
        for (uint64_t tile = tile_first; tile < A.tiles; tile += tile_step) {
            const uint64_t gw0 = tile * 32 * W;          // first 32-bit word of the tile
            const uint64_t P0 = gw0 * 32;
            if (P0 >= A.mn) continue;
            const uint64_t P1 = (P0 + 1024ull * W < A.mn) ? P0 + 1024ull * W : A.mn;
            const uint64_t r_first = div_u64_u32(P0, n);
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
            // row segments of the tile, in tile-local bit coordinates [a_loc, b_loc); c_tile is the column
            // (in the segment's row) of tile bit 0 and goes negative from the second row on
            const uint32_t T = (uint32_t)(P1 - P0);
            // seg_par: the group's warps take whole segments instead of sharing the words of each, so that a
            // lane gets more words of a row.  Each segment goes to the warp that has been given the fewest
            // weights so far (every warp keeps the same books, so they agree without talking).
            // (With many short segments per tile, seg_par == 1, they simply take turns.)
            uint32_t a_loc = 0, b_loc = 0, ai = 0, turn = 0;
            uint32_t g0 = 0, g1 = 0, g2 = 0, g3 = 0;     // weights given to each warp of the group so far
            int32_t c_tile = (int32_t)(P0 - r_first * n);
            for (uint64_t r = r_first; a_loc < T;
                 ++r, ai += n_q, c_tile -= (int32_t)n, a_loc = b_loc, turn = turn + 1 == wpt ? 0 : turn + 1) {
                b_loc = (uint32_t)((int32_t)n - c_tile);
                b_loc = b_loc < T ? b_loc : T;
                if (seg_par == 1) {
                    if (turn != sub) continue;
                } else if (seg_par == 2) {
                    uint32_t pick = 0, least = g0;
                    if (wpt > 1 && g1 < least) { pick = 1; least = g1; }
                    if (wpt > 2 && g2 < least) { pick = 2; least = g2; }
                    if (wpt > 3 && g3 < least) { pick = 3; least = g3; }
                    const uint32_t len = b_loc - a_loc;
                    g0 += pick == 0 ? len : 0u;
                    g1 += pick == 1 ? len : 0u;
                    g2 += pick == 2 ? len : 0u;
                    g3 += pick == 3 ? len : 0u;
                    if (pick != sub) continue;
                }
                constexpr int NR = NQ > 0 ? NQ : 1;
                float al[NR];
                if constexpr (NQ > 0) {
#pragma unroll
                    for (int i = 0; i < NQ; ++i)
                        al[i] = ai + i < GEMV_ALPHA_WORDS ? alpha_s[ai + i] : __ldg(alpha + r * n_q + i);
                }
                const uint32_t lw_lo = a_loc >> 5, lw_hi = (b_loc - 1) >> 5;
                float acc[BT];
#pragma unroll
                for (int q = 0; q < BT; ++q) acc[q] = 0.0f;
                const uint32_t wstep = seg_par ? 32 : 32 * wpt;
                const uint32_t first_mask = 0xffffffffu << (a_loc & 31u);
                const uint32_t last_mask = 0xffffffffu >> (31u - ((b_loc - 1u) & 31u));
                uint32_t lw = lw_lo + (seg_par ? 0 : sub * 32) + lane;
                if constexpr (XS && NQ > 0) {
                    walk_segment<BT, XT, NQ>(smem_addr(mask_s), 128 * W, smem_addr(xs), lw, lw_lo, lw_hi, wstep,
                                             first_mask, last_mask, c_tile, al, acc);
                } else {
                // the same walk in plain C++ for any number of planes and for activations left in global memory
                uint32_t mk = 0, wb[NR];
                int32_t cbase = 0;
#pragma unroll
                for (int i = 0; i < NR; ++i) wb[i] = 0;
                auto take_word = [&]() {
                    uint32_t m = mask_s[lw];
                    if (lw == lw_lo) m &= first_mask;
                    if (lw == lw_hi) m &= last_mask;
                    mk = m;
                    cbase = c_tile + (int32_t)(lw * 32);
                    if constexpr (NQ > 0) {
#pragma unroll
                        for (int i = 0; i < NQ; ++i) wb[i] = region[i * 32 * W + lw];
                    } else {
                        wb[0] = lw;
                    }
                };
                bool more = lw <= lw_hi;
                if (more) take_word();
                const int32_t c_safe = c_tile + (int32_t)a_loc;     // a column of this row, for idle lanes
                // branch-free body under a warp-uniform loop condition: the lanes stay converged
                while (__any_sync(0xffffffffu, more)) {
                    const bool live = mk != 0;
                    const uint32_t k = live ? 31u - (uint32_t)__clz((int)mk) : 0u;
                    const uint32_t bit = live ? 1u << k : 0u;
                    mk ^= bit;
                    float v = 0.0f;
                    if constexpr (NQ > 0) {
#pragma unroll
                        for (int i = 0; i < NQ; ++i) {
                            const float t = (wb[i] & bit) ? al[i] : -al[i];
                            v = i == 0 ? t : v + t;
                        }
                    } else {
                        for (uint32_t i = 0; i < n_q; ++i) {
                            const float a1 = __ldg(alpha + r * n_q + i);
                            v += (region[i * 32 * W + wb[0]] & bit) ? a1 : -a1;
                        }
                    }
                    v = live ? v : 0.0f;
                    const int32_t c = live ? cbase + (int32_t)k : c_safe;
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
                    if (mk == 0 && more) {
                        lw += wstep;
                        more = lw <= lw_hi;
                        if (more) take_word();
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
    // One tile group per tile an SM gets (up to 15, the named barriers), and as many warps per group
    // (up to 4) as fit a block of 20 warps.
    // (More warps per block at fewer registers were slower: every warp repeats the per-tile bookkeeping.)
    const uint64_t live = (A.words64 * 2 + 32ull * A.W - 1) / (32ull * A.W);
    const uint32_t sms = (uint32_t)sm_count();
    constexpr uint32_t max_warps = 20;
    uint32_t groups = (uint32_t)((live + sms - 1) / sms);
    groups = groups < 1 ? 1 : groups > 15 ? 15 : groups;
    uint32_t wpt = max_warps / groups;
    wpt = wpt < 1 ? 1 : wpt > 4 ? 4 : wpt;
    // a tile that spans more rows than the group has warps: the warps take whole row segments in turn, which
    // gives a lane more words of a row (a steadier load per lane) than sharing the words of every segment
    // (2 = by load, for tiles of fewer than 8 rows; 1 = in turn)
    const uint32_t seg_par = (wpt > 1 && 4ull * 1024 * A.W >= 5ull * n * wpt) ? (1024ull * A.W < 8ull * n ? 2u : 1u) : 0u;
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
                               d_y, ldy, (uint32_t)n, wpt, seg_par) != cudaSuccess) return SQNN_E_CUDA;               \
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
