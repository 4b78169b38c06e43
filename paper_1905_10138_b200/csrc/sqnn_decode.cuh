// Device-side decryption of one warp tile: seeds -> XOR-gate network (table lookup) ->
// patch flips, producing a run of consecutive output words in shared memory.
//
// Work split.  A lane owns G consecutive slices, G chosen so that G * n_out is a multiple of
// 32 bits and 32 * G is a multiple of 128 slices; its W = G * n_out / 32 output words are
// private to it while it expands and patches.  A warp tile is therefore 32 * G consecutive
// slices = 32 * W consecutive 32-bit words of the flattened plane, starting on a boundary of
// the per-128-slice d_patch offsets.
//
// The network (Section 3.1, w~ = M . w^c) is evaluated with tables: the seed is cut into
// chunks of cb bits and table[chunk][value] holds the XOR of the columns of M selected by
// the value, as an n_out-bit word padded to nwp 32-bit words.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#define SQNN_DEV __device__ __forceinline__

namespace sqnn {

struct PlanePtrs {
    const uint32_t *wc;    // seed stream
    const uint32_t *np;    // n_patch stream (unused when w_np == 0)
    const uint32_t *idx;   // d_patch entries before each block of 128 slices
    const uint8_t *dp;     // d_patch entries
    uint32_t n_dp;
    uint32_t w_np;
};

struct DecodeArgs {
    uint64_t mn;           // weights per plane
    uint64_t words64;      // ceil(mn / 64)
    uint64_t tiles;        // warp tiles per plane
    uint32_t n_out, n_in, n_q;
    uint32_t G, W;         // slices and words per lane
    uint32_t nw, nwp;      // words per table entry: used, padded (1, 2, 4, 8)
    uint32_t nchunks, cb;  // table chunks, bits per chunk
    const uint32_t *rows;  // rows of M
    uint32_t *status;      // sticky error word or NULL
    PlanePtrs pl[8];
};

__host__ __device__ constexpr uint32_t gcd_u32(uint32_t a, uint32_t b) { return b == 0 ? a : gcd_u32(b, a % b); }
__host__ __device__ constexpr uint32_t slices_per_lane(uint32_t n_out)
{
    return (32 / gcd_u32(n_out, 32)) < 4 ? 4 : (32 / gcd_u32(n_out, 32));
}
__host__ __device__ constexpr uint32_t entry_words(uint32_t n_out) { return (n_out + 31) / 32; }
__host__ __device__ constexpr uint32_t entry_words_padded(uint32_t n_out)
{
    return entry_words(n_out) <= 1 ? 1 : entry_words(n_out) <= 2 ? 2 : entry_words(n_out) <= 4 ? 4 : 8;
}
// Fewest chunks whose tables stay within 48 KB.
__host__ __device__ constexpr uint32_t table_chunks(uint32_t n_in, uint32_t nwp)
{
    for (uint32_t c = 1; c <= 8; ++c) {
        uint32_t cb = (n_in + c - 1) / c;
        if (cb <= 14 && (uint64_t)c * (1ull << cb) * nwp * 4 <= 48 * 1024) return c;
    }
    return 8;
}
__host__ __device__ constexpr uint32_t chunk_bits(uint32_t n_in, uint32_t nwp)
{
    return (n_in + table_chunks(n_in, nwp) - 1) / table_chunks(n_in, nwp);
}

SQNN_DEV uint32_t extract_bits(const uint32_t *__restrict__ base, uint64_t bitpos, uint32_t width)
{
    const uint64_t w = bitpos >> 5;
    const uint32_t sh = (uint32_t)(bitpos & 31);
    const uint32_t lo = __ldg(base + w), hi = __ldg(base + w + 1);   // sections end with slack
    const uint32_t v = __funnelshift_r(lo, hi, sh);
    return width >= 32 ? v : (v & ((1u << width) - 1u));
}

SQNN_DEV void flag(uint32_t *status, uint32_t code)
{
    if (status) atomicMax(status, code);
}

// Shared-memory words the tables need, rounded so that what follows stays 16-byte aligned.
inline __host__ __device__ uint32_t table_words(uint32_t n_in, uint32_t nwp, uint32_t nchunks, uint32_t cb)
{
    return (nchunks * (1u << cb) * nwp + n_in * nwp + 3u) & ~3u;
}

// Builds the column words of M and the chunk tables.  All threads of the block take part.
SQNN_DEV void build_tables(const DecodeArgs &A, uint32_t *tab)
{
    const uint32_t nwp = A.nwp, n_in = A.n_in, n_out = A.n_out, cb = A.cb;
    uint32_t *cols = tab + A.nchunks * (1u << cb) * nwp;
    for (uint32_t i = threadIdx.x; i < n_in * nwp; i += blockDim.x) {
        const uint32_t t = i / nwp, k = i % nwp;
        uint32_t w = 0;
        for (uint32_t j = 32 * k; j < n_out && j < 32 * k + 32; ++j)
            w |= ((__ldg(A.rows + j) >> t) & 1u) << (j - 32 * k);
        cols[i] = w;
    }
    __syncthreads();
    const uint32_t total = A.nchunks * (1u << cb) * nwp;
    for (uint32_t i = threadIdx.x; i < total; i += blockDim.x) {
        const uint32_t k = i % nwp, e = i / nwp;
        const uint32_t v = e & ((1u << cb) - 1u), ch = e >> cb;
        uint32_t x = 0;
        for (uint32_t b = 0; b < cb; ++b) {
            const uint32_t t = ch * cb + b;
            if (t < n_in && ((v >> b) & 1u)) x ^= cols[t * nwp + k];
        }
        tab[i] = x;
    }
    __syncthreads();
}

template <int NWP>
SQNN_DEV void load_entry(const uint32_t *tab, uint32_t e, uint32_t (&x)[NWP])
{
    if constexpr (NWP == 1) {
        x[0] = tab[e];
    } else if constexpr (NWP == 2) {
        const uint2 v = *reinterpret_cast<const uint2 *>(tab + 2 * e);
        x[0] = v.x; x[1] = v.y;
    } else if constexpr (NWP == 4) {
        const uint4 v = *reinterpret_cast<const uint4 *>(tab + 4 * e);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    } else {
        const uint4 v = *reinterpret_cast<const uint4 *>(tab + 8 * e);
        const uint4 u = *reinterpret_cast<const uint4 *>(tab + 8 * e + 4);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
        x[4] = u.x; x[5] = u.y; x[6] = u.z; x[7] = u.w;
    }
}

// Expands and patches the lane's G slices of warp tile `tile` of `plane` into
// region[lane * W .. lane * W + W).  N_OUT / N_IN = 0 selects the run-time shape.
template <int N_OUT, int N_IN>
SQNN_DEV void decode_warp_tile(const DecodeArgs &A, uint32_t plane, uint64_t tile,
                               uint32_t *region, const uint32_t *tab, uint32_t lane)
{
    const PlanePtrs &P = A.pl[plane];
    if constexpr (N_OUT != 0) {
        constexpr uint32_t n_out = N_OUT, n_in = N_IN;
        constexpr uint32_t G = slices_per_lane(n_out), W = G * n_out / 32;
        constexpr uint32_t NW = entry_words(n_out), NWP = entry_words_padded(n_out);
        constexpr uint32_t NCH = table_chunks(n_in, NWP), CB = chunk_bits(n_in, NWP);
        const uint64_t s0 = (tile * 32 + lane) * G;
        uint32_t *mine = region + lane * W;
        uint32_t seeds[G];
#pragma unroll
        for (uint32_t i = 0; i < G; ++i) seeds[i] = extract_bits(P.wc, (s0 + i) * n_in, n_in);
        uint64_t acc = 0;
        uint32_t have = 0, wp = 0;
#pragma unroll
        for (uint32_t i = 0; i < G; ++i) {
            uint32_t x[NWP];
            load_entry<NWP>(tab, seeds[i] & ((1u << CB) - 1u), x);
#pragma unroll
            for (uint32_t ch = 1; ch < NCH; ++ch) {
                uint32_t y[NWP];
                load_entry<NWP>(tab, (ch << CB) | ((seeds[i] >> (ch * CB)) & ((1u << CB) - 1u)), y);
#pragma unroll
                for (uint32_t k = 0; k < NW; ++k) x[k] ^= y[k];
            }
#pragma unroll
            for (uint32_t k = 0; k < NW; ++k) {
                const uint32_t bits = (k == NW - 1) ? n_out - 32 * k : 32;
                acc |= (uint64_t)x[k] << have;
                have += bits;
                if (have >= 32) { mine[wp++] = (uint32_t)acc; acc >>= 32; have -= 32; }
            }
        }
    } else {
        const uint32_t n_out = A.n_out, n_in = A.n_in, G = A.G, W = A.W;
        const uint32_t nw = A.nw, nwp = A.nwp, nch = A.nchunks, cb = A.cb;
        const uint32_t cmask = (1u << cb) - 1u;
        const uint64_t s0 = (tile * 32 + lane) * G;
        uint32_t *mine = region + lane * W;
        uint64_t acc = 0;
        uint32_t have = 0, wp = 0;
        for (uint32_t i = 0; i < G; ++i) {
            const uint32_t seed = extract_bits(P.wc, (s0 + i) * n_in, n_in);
            for (uint32_t k = 0; k < nw; ++k) {
                uint32_t x = 0;
                for (uint32_t ch = 0; ch < nch; ++ch)
                    x ^= tab[((ch << cb) | ((seed >> (ch * cb)) & cmask)) * nwp + k];
                const uint32_t bits = (k == nw - 1) ? n_out - 32 * k : 32;
                acc |= (uint64_t)x << have;
                have += bits;
                if (have >= 32) { mine[wp++] = (uint32_t)acc; acc >>= 32; have -= 32; }
            }
        }
    }
    // Patches (Section 3.2): the lane's first entry sits at the block offset of the tile plus
    // the n_patch counts of the lanes before it.
    if (P.w_np != 0) {
        const uint32_t n_out = N_OUT ? (uint32_t)N_OUT : A.n_out;
        const uint32_t G = N_OUT ? slices_per_lane(N_OUT ? N_OUT : 1) : A.G;
        const uint32_t W = N_OUT ? G * n_out / 32 : A.W;
        const uint64_t s0 = (tile * 32 + lane) * G;
        uint32_t *mine = region + lane * W;
        uint32_t cnt = 0;
        for (uint32_t i = 0; i < G; ++i) cnt += extract_bits(P.np, (s0 + i) * P.w_np, P.w_np);
        uint32_t incl = cnt;
#pragma unroll
        for (uint32_t d = 1; d < 32; d <<= 1) {
            const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        if (__any_sync(0xffffffffu, cnt != 0)) {
            uint32_t at = __ldg(P.idx + tile * (G / 4)) + incl - cnt;
            if (cnt != 0) {
                for (uint32_t i = 0; i < G; ++i) {
                    const uint32_t npi = extract_bits(P.np, (s0 + i) * P.w_np, P.w_np);
                    for (uint32_t k = 0; k < npi; ++k, ++at) {
                        if (at >= P.n_dp) { flag(A.status, 2u); continue; }
                        const uint32_t pos = P.dp[at];
                        if (pos >= n_out) { flag(A.status, 1u); continue; }
                        const uint32_t bit = i * n_out + pos;
                        mine[bit >> 5] ^= 1u << (bit & 31);
                    }
                }
            }
        }
    }
}

}  // namespace sqnn
