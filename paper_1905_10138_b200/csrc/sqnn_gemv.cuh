// K3: decryption fused with Y[b][r] = sum_c W[r][c] X[b][c] for small batch (<= 15), fp32
// accumulation on the plain ALUs, as a template over the network shape, with its launcher.
//
// Work split.  A block owns a run of whole rows of W.  The bits of those rows are one contiguous
// range of every flattened plane, so the block decodes the kernel tiles that cover that range
// (the first and the last one may be shared with a neighbouring block, which decodes them too)
// into shared memory, next to the same range of the pruning mask, and then walks its rows: a warp
// takes a row (or one of `parts` equal runs of a row's words), each lane visits the care bits of
// its words, rebuilds the weight (+-alpha_1) + (+-alpha_2) + ... from the plane bits and
// accumulates weight * x.  Row sums are reduced over the warp (and over the parts through shared
// memory) and stored: every Y[b][r] has one owner and a fixed summation order, no atomics and no
// clearing of Y.  Everything the walk reads is on chip: tables, decoded bits, mask words, the
// scales of the block's rows and (XS = true) the activations of the current batch chunk as
// xs[c][BT].  Rows that do not fit shared memory at once are taken in chunks.
// With one activation vector and 16-byte aligned operands the tables, the activations and the mask
// range of a block's first chunk are fetched by three bulk copies (cp.async.bulk, completion on an
// mbarrier, bounded wait) that thread 0 issues at kernel entry; otherwise by cp.async from every
// thread.
#pragma once
#include "sqnn_kernels.cuh"

namespace sqnn {

struct GemvArgs {
    DecodeArgs A;
    const uint32_t *mask32;
    uint64_t mask_words;
    const float *alpha;
    const void *x;
    int64_t ldx;
    float *y;
    int64_t ldy;
    uint64_t m;
    uint32_t n, batch;
    uint32_t rows_per_block, rows_per_chunk, parts;
    uint32_t region_words;        // words of one bit vector of a chunk in shared memory (whole kernel tiles)
    uint32_t alpha_words, part_words, xs_words;
    uint32_t bulk_stage;          // tables, activations and mask may be staged by bulk copies (sizes and alignment allow it)
};

// One-dimensional bulk copy global -> shared by the copy engine, completion counted in bytes on an
// mbarrier; both addresses 16-byte aligned, size a multiple of 16.
SQNN_DEV void stage_bar_init(uint64_t *bar)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" :: "r"(smem_addr(bar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
}
SQNN_DEV void stage_bar_expect(uint64_t *bar, uint32_t bytes)
{
    asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}\n"
                 :: "r"(smem_addr(bar)), "r"(bytes) : "memory");
}
SQNN_DEV void bulk_load(void *sdst, const void *gsrc, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 :: "r"(smem_addr(sdst)), "l"(gsrc), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
// Waits for phase 0 of the barrier, for about a second at most; false if it gave up.
SQNN_DEV bool stage_bar_wait(uint64_t *bar)
{
    const long long t0 = clock64();
    for (;;) {
        uint32_t ok;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0, %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                     : "=r"(ok) : "r"(smem_addr(bar)), "r"(1000000u) : "memory");
        if (ok) return true;
        if (clock64() - t0 > 2000000000ll) return false;
    }
}

SQNN_DEV float to_float(float v) { return v; }
SQNN_DEV float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

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
            uint32_t w;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(a));
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
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v[0]) : "r"(a));
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

template <int N_OUT, int N_IN, int BT, typename XT, bool XS, int NQ>
__global__ void __launch_bounds__(1024, 1)
k_decode_gemv(const GemvArgs g)
{
    extern __shared__ __align__(16) uint32_t smem[];
    const DecodeArgs &A = g.A;
    const uint32_t W = words_per_lane<N_OUT>(A);
    const uint32_t TW = 32 * W;                                  // words per kernel tile
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t n = g.n, n_q = A.n_q, P = g.parts;
    uint32_t *tab_s = smem;
    uint32_t *bits_s = tab_s + A.tab_words;                      // [plane][region_words]
    uint32_t *mask_s = bits_s + n_q * g.region_words;
    float *alpha_s = reinterpret_cast<float *>(mask_s + g.region_words);
    float *part_s = alpha_s + g.alpha_words;                     // [row][part][BT]
    XT *xs = reinterpret_cast<XT *>(part_s + g.part_words);      // [c][BT]
    const XT *x = reinterpret_cast<const XT *>(g.x);
    const bool mask_vec = (reinterpret_cast<uintptr_t>(g.mask32) & 15) == 0;
    const uint64_t row0 = (uint64_t)blockIdx.x * g.rows_per_block;
    const uint64_t row_end = row0 + g.rows_per_block < g.m ? row0 + g.rows_per_block : g.m;

    // Stages the activations of batch rows [bc, bc + BT) as xs[c][BT]; ends with a commit.
    auto stage_x = [&](uint32_t bc) {
        if constexpr (XS) {
            if (BT == 1 && (reinterpret_cast<uintptr_t>(x + (int64_t)bc * g.ldx) & 15) == 0) {
                constexpr uint32_t PER = 16 / sizeof(XT);
                const uint4 *src = reinterpret_cast<const uint4 *>(x + (int64_t)bc * g.ldx);
                uint4 *dst = reinterpret_cast<uint4 *>(xs);
                for (uint32_t v = threadIdx.x; v < n / PER; v += blockDim.x) cp_async16(dst + v, src + v);
                for (uint32_t c = (n / PER) * PER + threadIdx.x; c < n; c += blockDim.x) xs[c] = x[(int64_t)bc * g.ldx + c];
            } else {
#pragma unroll 4
                for (uint32_t c = threadIdx.x; c < n; c += blockDim.x) {
                    XT v[BT];
#pragma unroll
                    for (int q = 0; q < BT; ++q) v[q] = bc + q < g.batch ? x[(int64_t)(bc + q) * g.ldx + c] : XT(0.0f);
#pragma unroll
                    for (int q = 0; q < BT; ++q) xs[c * BT + q] = v[q];
                }
            }
        }
        cp_async_commit();
    };

    // With one activation vector and everything 16-byte aligned, thread 0 hands the three big transfers of the
    // block's first chunk -- tables, activations, mask -- to the copy engine at once, before anything else
    // runs; otherwise every thread requests its share by cp.async (three commit groups, as below).
    __shared__ uint64_t stage_bar;
    bool bulk = false;
    if constexpr (XS && BT == 1) {
        const uint64_t tile_bits = 32ull * TW;
        const uint64_t rb0 = row0 + g.rows_per_chunk < row_end ? row0 + g.rows_per_chunk : row_end;
        const uint64_t k0 = (row0 * n) / tile_bits, k1 = (rb0 * n + tile_bits - 1) / tile_bits;
        bulk = g.bulk_stage && row0 < row_end && k1 * TW <= g.mask_words;      // the mask range lies inside the array
        if (bulk && threadIdx.x == 0) {
            const uint32_t tab_bytes = A.tab_words * 4, x_bytes = n * (uint32_t)sizeof(XT), mask_bytes = (uint32_t)(k1 - k0) * TW * 4;
            stage_bar_init(&stage_bar);
            stage_bar_expect(&stage_bar, tab_bytes + x_bytes + mask_bytes);
            bulk_load(tab_s, A.tab, tab_bytes, &stage_bar);
            bulk_load(xs, x, x_bytes, &stage_bar);
            bulk_load(mask_s, g.mask32 + k0 * TW, mask_bytes, &stage_bar);
        }
    }
    if (!bulk) {
        tables_request(A, tab_s);                                // commit group: tables
        stage_x(0);                                              // commit group: activations
    }
    uint32_t xs_holds = 0;                                       // batch chunk in xs

    for (uint64_t ra = row0; ra < row_end; ra += g.rows_per_chunk) {
        const uint64_t rb = ra + g.rows_per_chunk < row_end ? ra + g.rows_per_chunk : row_end;
        const uint32_t nrows = (uint32_t)(rb - ra);
        // kernel tiles that cover the bits [ra * n, rb * n)
        const uint64_t tile_bits = 32ull * TW;
        const uint64_t kt0 = (ra * n) / tile_bits, kt1 = (rb * n + tile_bits - 1) / tile_bits;
        const uint32_t nt = (uint32_t)(kt1 - kt0);
        const uint64_t gw0 = kt0 * TW;                           // first word of the chunk's regions
        if (ra != row0) __syncthreads();                         // the walk of the previous chunk is over
        if (!(bulk && ra == row0))
            stage_mask(mask_s, g.mask32, gw0, g.mask_words, nt * TW, threadIdx.x, blockDim.x, mask_vec);
        for (uint32_t i = threadIdx.x; i < nrows * n_q; i += blockDim.x) cp_async4(alpha_s + i, g.alpha + ra * n_q + i);
        cp_async_commit();                                       // commit group: mask and scales

        // decode: item = (tile, plane), dealt out over the warps; a warp's first item is fetched
        // before anybody waits for the tables
        const uint32_t items = nt * n_q;
        uint32_t item = warp;
        if constexpr (N_OUT != 0) {
            using S = Shape<N_OUT, N_IN>;
            TileSeeds<N_OUT, N_IN> s;
            TileRun run{0u, 0u};
            uint32_t pw[PATCH_AHEAD];
            auto fetch = [&](uint32_t it) {
                const uint32_t t = it / n_q, pl = it - t * n_q;
                fetch_seeds<N_OUT, N_IN>(A.pl[pl], kt0 + t, lane, s);
                run = fetch_run(A.pl[pl], kt0 + t);
                fetch_patches(A, A.pl[pl], run, lane, pw);
            };
            if (item < items) fetch(item);
            if (ra == row0) {
                if (bulk) {
                    __syncthreads();                             // the barrier's initialisation is visible to all
                    if (!stage_bar_wait(&stage_bar)) flag(A.status, (uint32_t)(-SQNN_E_TIMEOUT));
                } else {
                    cp_async_wait_group<2>();                    // tables (the two younger groups may be pending)
                    __syncthreads();
                }
            }
            while (item < items) {
                const uint32_t t = item / n_q, pl = item - t * n_q;
                uint32_t *region = bits_s + pl * g.region_words + t * TW;
                tile_expand<N_OUT, N_IN>(s, region, tab_s, lane);
                __syncwarp();
                tile_patch(A, A.pl[pl], run, pw, region, 0u, S::TILE_BITS, lane);
                item += nwarps;
                if (item < items) fetch(item);
            }
        } else {
            if (ra == row0) {
                if (bulk) {
                    __syncthreads();
                    if (!stage_bar_wait(&stage_bar)) flag(A.status, (uint32_t)(-SQNN_E_TIMEOUT));
                } else {
                    cp_async_wait_group<2>();
                    __syncthreads();
                }
            }
            for (; item < items; item += nwarps) {
                const uint32_t t = item / n_q, pl = item - t * n_q;
                decode_ktile_generic(A, pl, kt0 + t, bits_s + pl * g.region_words + t * TW, tab_s, lane);
            }
        }
        cp_async_wait_all();
        __syncthreads();                                         // bits, mask, scales, activations in place

        const uint32_t nitems = nrows * P;
        for (uint32_t bc = 0; bc < g.batch; bc += BT) {
            if (XS && xs_holds != bc) {
                __syncthreads();                                 // nobody reads xs any more
                stage_x(bc);
                cp_async_wait_all();
                __syncthreads();
                xs_holds = bc;
            } else if (P > 1 && bc != 0) {
                __syncthreads();                                 // the partial sums of the previous chunk are consumed
            }
            for (uint32_t it = warp; it < nitems; it += nwarps) {
                const uint32_t rl = it / P, part = it - rl * P;
                const uint64_t r = ra + rl;
                const uint32_t o = (uint32_t)(r * n - gw0 * 32);             // bit of the region where the row starts
                const uint32_t first = o >> 5, last = (o + n - 1) >> 5;
                const uint32_t per = (last - first + P) / P;                 // words per part
                const uint32_t wb = first + part * per;
                const uint32_t we = wb + per < last + 1 ? wb + per : last + 1;
                const uint32_t first_mask = 0xffffffffu << (o & 31u);
                const uint32_t last_mask = 0xffffffffu >> (31u - ((o + n - 1) & 31u));
                constexpr int NR = NQ > 0 ? NQ : 8;
                uint32_t al[NR];                                             // scales as bit patterns
#pragma unroll
                for (int i = 0; i < NR; ++i) al[i] = (uint32_t)i < n_q ? __float_as_uint(alpha_s[rl * n_q + i]) : 0u;
                float acc[BT];
#pragma unroll
                for (int q = 0; q < BT; ++q) acc[q] = 0.0f;
                const uint32_t xs_sa = smem_addr(xs);
                constexpr uint32_t XB = BT * sizeof(XT);
                // A lane takes the words wb + lane, wb + lane + 32, ... and visits the care bits of each,
                // highest first.  (Letting lanes run ahead to their next word inside one flat loop was
                // measured slower: the refill code then runs in nearly every step.)
                for (uint32_t w = wb + lane; w < we; w += 32) {
                    uint32_t mk = mask_s[w];
                    if (w == first) mk &= first_mask;
                    if (w == last) mk &= last_mask;
                    uint32_t nb[NR];                                         // complemented plane words
#pragma unroll
                    for (int i = 0; i < NR; ++i) nb[i] = (uint32_t)i < n_q ? ~bits_s[i * g.region_words + w] : 0u;
                    const int32_t c31 = (int32_t)(w * 32 + 31) - (int32_t)o; // column of bit 31 of this word
                    while (mk) {
                        const uint32_t z = (uint32_t)__clz((int)mk);         // bit 31 - z is the highest care bit left
                        mk &= ~(0x80000000u >> z);
                        const int32_t c = c31 - (int32_t)z;
                        // weight = (+-alpha_1) + (+-alpha_2) + ... in plane order; with one plane the scale is
                        // applied to the row sum instead and the weight is +-1
                        float v;
                        if constexpr (NQ == 1) {
                            v = __uint_as_float(0x3f800000u | ((nb[0] << z) & 0x80000000u));
                        } else {
                            v = __uint_as_float(al[0] ^ ((nb[0] << z) & 0x80000000u));
#pragma unroll
                            for (int i = 1; i < NR; ++i)
                                if ((uint32_t)i < n_q) v = __fadd_rn(v, __uint_as_float(al[i] ^ ((nb[i] << z) & 0x80000000u)));
                        }
                        float xv[BT];
                        if constexpr (XS) {
                            lds_x<BT, XT>(xs_sa + (uint32_t)c * XB, xv);
                        } else {
#pragma unroll
                            for (int q = 0; q < BT; ++q)
                                xv[q] = bc + q < g.batch ? to_float(x[(int64_t)(bc + q) * g.ldx + c]) : 0.0f;
                        }
#pragma unroll
                        for (int q = 0; q < BT; ++q) acc[q] = fmaf(v, xv[q], acc[q]);
                    }
                }
#pragma unroll
                for (int q = 0; q < BT; ++q) {
                    float sum = acc[q];
#pragma unroll
                    for (uint32_t d = 16; d >= 1; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
                    if (lane == 0) {
                        if (P > 1) {
                            part_s[(rl * P + part) * BT + q] = sum;
                        } else if (bc + q < g.batch) {
                            if constexpr (NQ == 1) sum *= __uint_as_float(al[0]);
                            g.y[(int64_t)(bc + q) * g.ldy + (int64_t)r] = sum;
                        }
                    }
                }
            }
            if (P > 1) {
                __syncthreads();
                for (uint32_t i = threadIdx.x; i < nrows * BT; i += blockDim.x) {
                    const uint32_t rl = i / BT, q = i - rl * BT;
                    float sum = 0.0f;
                    for (uint32_t part = 0; part < P; ++part) sum += part_s[(rl * P + part) * BT + q];
                    if (NQ == 1) sum *= alpha_s[rl];
                    if (bc + q < g.batch) g.y[(int64_t)(bc + q) * g.ldy + (int64_t)(ra + rl)] = sum;
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// launcher
// ------------------------------------------------------------------------------------------
template <int N_OUT, int N_IN, int BT, typename XT>
inline int launch_gemv_bt(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x,
                          int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t m, uint64_t n, cudaStream_t st)
{
    uint32_t nwarps = 32;
    const size_t limit = 220 * 1024;
    const uint32_t sms = (uint32_t)sm_count();
    GemvArgs g;
    g.A = A;
    g.mask32 = (const uint32_t *)d_mask;
    g.mask_words = A.words64 * 2;
    g.alpha = d_alpha;
    g.x = d_x; g.ldx = ldx; g.y = d_y; g.ldy = ldy;
    g.m = m; g.n = (uint32_t)n; g.batch = batch;
    const uint64_t R = (m + sms - 1) / sms;
    const uint64_t grid = (m + R - 1) / R;
    if (R > 0xffffffffull) return SQNN_E_UNSUPPORTED;
    g.rows_per_block = (uint32_t)R;
    {
        // a block with a few rows and a few tiles to decode gets a few warps: a thread block is cheaper to start
        // and to synchronise the smaller it is (tiny layers are all launch and latency)
        const uint64_t tb = 32ull * 32ull * A.W;
        const uint64_t items = ((R * n + tb - 1) / tb + 1) * A.n_q;
        const uint64_t want = R > items ? R : items;
        if (want <= 4) nwarps = 4;
        else if (want <= 8) nwarps = 8;
        else if (want <= 16) nwarps = 16;
    }
    const uint64_t TW = 32ull * A.W, tile_bits = 32 * TW;
    const size_t tab = (size_t)A.tab_words * 4;
    const size_t xbytes = ((size_t)n * BT * sizeof(XT) + 15) & ~(size_t)15;
    bool xs = xbytes <= 128 * 1024;
    // Warps sharing a row.  A warp walks its run of a row's words 32 at a time, and every item (a row, or one
    // of `parts` runs of it) costs about one such step more for its set-up and reduction, so the walk of a chunk
    // takes (rounds of items over the warps) x (steps per item + 1); the cheapest split wins, the smaller one on
    // a tie.  (Measured on 41 rows of 94 words: 1 part 13.5 us, 2 parts 15.2, 3 parts 13.8, 4 parts 16.5.)
    auto pick_parts = [&](uint64_t rows) {
        const uint64_t row_words = (n + 31) / 32 + 1;
        uint32_t best = 1;
        uint64_t best_cost = ~0ull;
        for (uint32_t p = 1; p <= 32 && p <= row_words; ++p) {
            const uint64_t per = (row_words + p - 1) / p;
            const uint64_t cost = ((rows * p + nwarps - 1) / nwarps) * ((per + 31) / 32 + 1);
            if (cost < best_cost) { best = p; best_cost = cost; }
        }
        return best;
    };
    uint64_t RC = R;
    size_t smem = 0;
    for (;;) {
        g.parts = pick_parts(RC);
        const uint64_t tiles = (RC * n + tile_bits - 1) / tile_bits + 1;
        const uint64_t region_words = tiles * TW;
        g.alpha_words = (uint32_t)((RC * A.n_q + 3) & ~3ull);
        g.part_words = (uint32_t)((RC * g.parts * BT + 3) & ~3ull);
        g.xs_words = xs ? (uint32_t)(xbytes / 4) : 0u;
        const uint64_t need = tab + (uint64_t)(A.n_q + 1) * region_words * 4 +
                              4ull * (g.alpha_words + g.part_words + g.xs_words);
        if (need <= limit) {
            g.region_words = (uint32_t)region_words;
            g.rows_per_chunk = (uint32_t)RC;
            smem = (size_t)need;
            break;
        }
        if (RC > 1) { RC = (RC + 1) / 2; continue; }
        if (xs) { xs = false; RC = R; continue; }               // leave the activations in global memory
        return SQNN_E_UNSUPPORTED;                               // one row of bits does not fit
    }
    // bulk staging of the first chunk: one activation vector in shared memory, 16-byte aligned sources and sizes
    g.bulk_stage = (BT == 1 && xs && ((uintptr_t)d_x & 15) == 0 && (n * sizeof(XT)) % 16 == 0 &&
                    ((uintptr_t)d_mask & 15) == 0 && ((uintptr_t)A.tab & 15) == 0 && (tab + 0) % 16 == 0 &&
                    (size_t)g.region_words * 4 < (1u << 20)) ? 1u : 0u;
#define SQNN_GEMV_LAUNCH(XSV, NQV)                                                                       \
    do {                                                                                                 \
        auto k = k_decode_gemv<N_OUT, N_IN, BT, XT, XSV, NQV>;                                           \
        if (prepare(k, smem)) return SQNN_E_CUDA;                                                        \
        k<<<(uint32_t)grid, nwarps * 32, smem, st>>>(g);                                                 \
    } while (0)
    if (xs) {
        if (A.n_q == 1) SQNN_GEMV_LAUNCH(true, 1);
        else if (A.n_q == 2) SQNN_GEMV_LAUNCH(true, 2);
        else if (A.n_q == 3) SQNN_GEMV_LAUNCH(true, 3);
        else SQNN_GEMV_LAUNCH(true, 0);
    } else {
        if (A.n_q == 1) SQNN_GEMV_LAUNCH(false, 1);
        else SQNN_GEMV_LAUNCH(false, 0);
    }
#undef SQNN_GEMV_LAUNCH
    return cudaGetLastError() == cudaSuccess ? SQNN_OK : SQNN_E_CUDA;
}

template <int N_OUT, int N_IN, typename XT>
inline int launch_gemv(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha, const void *d_x,
                       int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, uint64_t m, uint64_t n, cudaStream_t st)
{
    if (batch == 1) return launch_gemv_bt<N_OUT, N_IN, 1, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, m, n, st);
    if (batch == 2) return launch_gemv_bt<N_OUT, N_IN, 2, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, m, n, st);
    if (batch <= 4) return launch_gemv_bt<N_OUT, N_IN, 4, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, m, n, st);
    return launch_gemv_bt<N_OUT, N_IN, 8, XT>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, m, n, st);
}

}  // namespace sqnn
