// Device-side decryption of one warp tile: seeds -> XOR-gate network (table lookup) ->
// patch flips, producing a run of consecutive output words in shared memory.
//
// Work split.  A lane owns G consecutive slices, G a multiple of 4 chosen so that G * n_out is
// a multiple of 32 bits; its W = G * n_out / 32 output words are private to it while it expands
// and patches.  A warp tile is therefore 32 * G consecutive slices = 32 * W consecutive 32-bit
// words of the flattened plane, and it starts on a boundary of the per-128-slice d_patch
// offsets.  In the packed streams a tile is G * n_in words of seeds and G * w_np words of
// n_patch counts.
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
// Smallest multiple of 4 slices whose bits fill whole words, doubled (up to 8) while the lane
// would own fewer than 16 words, so that small networks still get tiles worth their overhead.
__host__ __device__ constexpr uint32_t slices_per_lane(uint32_t n_out)
{
    uint32_t g = 32 / gcd_u32(n_out, 32);
    if (g < 4) g = 4;
    while (g < 8 && g * n_out / 32 < 16) g *= 2;
    return g;
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

SQNN_DEV uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Asynchronous copy shared -> global by the bulk-copy engine; 16-byte aligned, size % 16 == 0.
SQNN_DEV void bulk_store(void *gdst, const void *ssrc, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n"
                 :: "l"(gdst), "r"(smem_addr(ssrc)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;\n" ::: "memory");
}
// Waits until at most PENDING of this thread's bulk copies still read their shared source.
template <int PENDING>
SQNN_DEV void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;\n" :: "n"(PENDING) : "memory");
}
SQNN_DEV void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

// Shared-memory words the tables need, rounded so that what follows stays 16-byte aligned.
inline __host__ __device__ uint32_t table_words(uint32_t n_in, uint32_t nwp, uint32_t nchunks, uint32_t cb)
{
    return (nchunks * (1u << cb) * nwp + n_in * nwp + 3u) & ~3u;
}

// Builds the column words of M and the chunk tables.  All threads of the block take part.
// An entry's value splits as (high << lo_bits) | low: entries with only low or only high bits
// are XORed together from the columns directly, every other entry is the XOR of those two.
// The build comes in two calls so that a kernel can request the rows of M first, start its other
// fetches, and only then wait: build_tables_begin stores the rows in shared memory (block
// barrier), build_tables_finish does the rest (ends with a block barrier).
struct RowsAhead { uint32_t r0, r1; };              // rows threadIdx.x and threadIdx.x + blockDim.x

SQNN_DEV uint32_t *rows_scratch()
{
    __shared__ uint32_t rows_s[256];
    return rows_s;
}

SQNN_DEV RowsAhead fetch_rows(const DecodeArgs &A)
{
    RowsAhead p{0u, 0u};
    if (threadIdx.x < A.n_out) p.r0 = __ldg(A.rows + threadIdx.x);
    if (threadIdx.x + blockDim.x < A.n_out) p.r1 = __ldg(A.rows + threadIdx.x + blockDim.x);
    return p;
}

SQNN_DEV void build_tables_begin(const DecodeArgs &A, RowsAhead ahead)
{
    uint32_t *rows_s = rows_scratch();
    const uint32_t n_out = A.n_out;
    if (threadIdx.x < n_out) rows_s[threadIdx.x] = ahead.r0;
    if (threadIdx.x + blockDim.x < n_out) rows_s[threadIdx.x + blockDim.x] = ahead.r1;
    for (uint32_t j = threadIdx.x + 2 * blockDim.x; j < n_out; j += blockDim.x) rows_s[j] = __ldg(A.rows + j);
    __syncthreads();
}

// N_OUT, N_IN: the network shape when it is known at compile time (the index arithmetic then folds), 0 = read it from A.
// WAIT_ASYNC: the thread's pending cp.async copies are awaited just before the closing barrier, so that what they
// bring in is visible to the whole block after it while the build itself runs under their latency.
template <int N_OUT = 0, int N_IN = 0, bool WAIT_ASYNC = false>
SQNN_DEV void build_tables_finish(const DecodeArgs &A, uint32_t *tab)
{
    const uint32_t *rows_s = rows_scratch();
    constexpr bool CT = N_OUT != 0;
    constexpr uint32_t NWP_C = entry_words_padded(CT ? N_OUT : 32);
    const uint32_t nwp = CT ? NWP_C : A.nwp, n_in = CT ? (uint32_t)N_IN : A.n_in, n_out = CT ? (uint32_t)N_OUT : A.n_out;
    const uint32_t cb = CT ? chunk_bits(CT ? N_IN : 8, NWP_C) : A.cb;
    const uint32_t nchunks = CT ? table_chunks(CT ? N_IN : 8, NWP_C) : A.nchunks;
    const uint32_t kshift = nwp == 1 ? 0 : nwp == 2 ? 1 : nwp == 4 ? 2 : 3;
    uint32_t *cols = tab + nchunks * (1u << cb) * nwp;
    // word k of column t: bit j of it is bit t of row 32 k + j -- one ballot over 32 rows
    const uint32_t lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    for (uint32_t i = threadIdx.x >> 5; i < n_in * nwp; i += nwarps) {
        const uint32_t t = i >> kshift, k = i & (nwp - 1);
        const uint32_t j = 32 * k + lane;
        const uint32_t r = j < n_out ? rows_s[j] : 0u;
        const uint32_t w = __ballot_sync(0xffffffffu, (r >> t) & 1u);
        if (lane == 0) cols[i] = w;
    }
    __syncthreads();
    const uint32_t lo_bits = cb / 2, hi_bits = cb - lo_bits;
    const uint32_t n_lo = 1u << lo_bits, n_hi = 1u << hi_bits;
    const uint32_t direct = (n_lo + n_hi - 1) * nwp;          // per chunk: low-only and high-only entries
    for (uint32_t i = threadIdx.x; i < nchunks * direct; i += blockDim.x) {
        const uint32_t ch = i / direct, r = i - ch * direct;
        const uint32_t k = r & (nwp - 1), e = r >> kshift;
        const uint32_t v = e < n_lo ? e : (e - n_lo + 1) << lo_bits;
        uint32_t x = 0;
#pragma unroll 4
        for (uint32_t b = 0; b < cb; ++b) {
            const uint32_t t = ch * cb + b;
            if (t < n_in && ((v >> b) & 1u)) x ^= cols[(t << kshift) + k];
        }
        tab[((((ch << cb) | v)) << kshift) + k] = x;
    }
    __syncthreads();
    const uint32_t total = nchunks * (1u << cb) * nwp;
    for (uint32_t i = threadIdx.x; i < total; i += blockDim.x) {
        const uint32_t k = i & (nwp - 1), e = i >> kshift;
        const uint32_t v = e & ((1u << cb) - 1u);
        const uint32_t l = v & (n_lo - 1), h = v & ~(n_lo - 1);
        if (l != 0 && h != 0) {
            const uint32_t chbase = e - v;
            tab[i] = tab[((chbase | l) << kshift) + k] ^ tab[((chbase | h) << kshift) + k];
        }
    }
    if constexpr (WAIT_ASYNC) asm volatile("cp.async.wait_all;\n" ::: "memory");
    __syncthreads();
}

template <int N_OUT = 0, int N_IN = 0>
SQNN_DEV void build_tables(const DecodeArgs &A, uint32_t *tab)
{
    build_tables_begin(A, fetch_rows(A));
    build_tables_finish<N_OUT, N_IN>(A, tab);
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

// Per-warp scratch of the patch step: 128 words of staged d_patch bytes (one window of up to
// PATCH_WIN entries, after up to 3 bytes of alignment) and one 16-bit mark per entry of the window.
constexpr uint32_t PATCH_WIN = 508;
constexpr uint32_t STAGE_DP_WORDS = 128;
constexpr uint32_t STAGE_WORDS = STAGE_DP_WORDS + 256;

// Compile-time facts of a network shape.
template <int N_OUT, int N_IN>
struct Shape {
    static constexpr uint32_t n_out = N_OUT, n_in = N_IN;
    static constexpr uint32_t G = slices_per_lane(N_OUT), W = G * N_OUT / 32;
    static constexpr uint32_t NW = entry_words(N_OUT), NWP = entry_words_padded(N_OUT);
    static constexpr uint32_t NCH = table_chunks(N_IN, NWP), CB = chunk_bits(N_IN, NWP);
    static constexpr uint32_t SPAN = G * N_IN, NSW = (SPAN + 31) / 32;
    static_assert(G <= 8, "compile-time shapes keep at most 8 slices per lane");
};

// What one lane reads from global memory for one tile of one plane.
template <int N_OUT, int N_IN>
struct TileIn {
    uint32_t raw[Shape<N_OUT, N_IN>::NSW + 1];   // words holding the lane's G seeds
    uint32_t np0, np1, np2;                      // words holding the lane's G n_patch fields
    uint32_t base, total;                        // the tile's run of d_patch entries
};

template <int N_OUT, int N_IN>
SQNN_DEV void tile_fetch(const PlanePtrs &P, uint64_t tile, uint32_t lane, TileIn<N_OUT, N_IN> &in)
{
    using S = Shape<N_OUT, N_IN>;
    const uint32_t *w = P.wc + tile * (S::G * S::n_in) + ((lane * S::SPAN) >> 5);
#pragma unroll
    for (uint32_t k = 0; k <= S::NSW; ++k) in.raw[k] = __ldg(w + k);
    in.base = in.total = in.np0 = in.np1 = in.np2 = 0;
    if (P.w_np != 0) {
        const uint32_t *ix = P.idx + tile * (S::G / 4);
        in.base = __ldg(ix);
        in.total = __ldg(ix + S::G / 4) - in.base;
        const uint32_t *q = P.np + tile * (S::G * P.w_np) + ((lane * S::G * P.w_np) >> 5);
        in.np0 = __ldg(q);
        in.np1 = __ldg(q + 1);
        in.np2 = __ldg(q + 2);
    }
}

// The tile's staged d_patch words: lane l fetches words l, l + 32, l + 64, l + 96 of the run.
template <int N_OUT, int N_IN>
SQNN_DEV void stage_fetch(const DecodeArgs &A, const PlanePtrs &P, TileIn<N_OUT, N_IN> &in, uint32_t lane,
                          uint32_t (&st)[4])
{
    st[0] = st[1] = st[2] = st[3] = 0;
    if (in.total == 0) return;
    if (in.base > P.n_dp || in.total > P.n_dp - in.base) {       // offsets point outside the section
        flag(A.status, 2u);
        in.total = 0;
        return;
    }
    const uint32_t nbytes = in.total < PATCH_WIN ? in.total : PATCH_WIN;
    const uint32_t nwords = ((in.base & 3u) + nbytes + 3) >> 2;
    const uint32_t *src = reinterpret_cast<const uint32_t *>(P.dp) + (in.base >> 2);
#pragma unroll
    for (uint32_t j = 0; j < 4; ++j)
        if (lane + 32 * j < nwords) st[j] = __ldg(src + lane + 32 * j);
}

// Flips the patched positions of a tile (Section 3.2), the warp working through the tile's run of
// d_patch entries 32 at a time.  An entry does not say which slice it belongs to; that follows
// from the n_patch counts.  Each lane knows where the entries of its own G slices start (a warp
// scan of the per-lane counts), so it drops a mark (the slice's first bit + 1) at the index of each of its
// slices' first entry; every entry then takes the nearest mark at or before it (a ballot and one
// shuffle per 32 entries), and the lane holding the entry flips bit slice * n_out + position of
// the tile with a shared-memory atomic.  Runs longer than PATCH_WIN entries are handled in
// windows, the last mark carrying over.  `win` holds the lane's n_patch fields (G fields of w_np bits, lowest first),
// `st` the first window's d_patch words fetched ahead of time.
template <uint32_t G, uint32_t N_OUT, typename WT>
SQNN_DEV void patch_tile(const DecodeArgs &A, const PlanePtrs &P, uint32_t *region, uint32_t *stage,
                         const uint32_t (&st)[4], uint32_t base, uint32_t total, WT win, uint32_t lane)
{
    const uint32_t w_np = P.w_np;
    const uint32_t fm = (1u << w_np) - 1u;
    uint32_t f[G];
    uint32_t cnt = 0;
#pragma unroll
    for (uint32_t i = 0; i < G; ++i) {
        f[i] = (uint32_t)(win >> (i * w_np)) & fm;
        cnt += f[i];
    }
    uint32_t incl = cnt;
#pragma unroll
    for (uint32_t d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
    }
    const uint32_t first = incl - cnt;
    if (__shfl_sync(0xffffffffu, incl, 31) != total) {      // counts disagree with the offsets
        flag(A.status, 2u);
        return;
    }
    uint32_t *marks32 = stage + STAGE_DP_WORDS;
    uint16_t *marks = reinterpret_cast<uint16_t *>(marks32);
    const uint32_t below_me = 0xffffffffu >> (31 - lane);   // lanes 0 .. lane
    uint32_t carry = 0, bad = 0;
    for (uint32_t w0 = 0; w0 < total; w0 += PATCH_WIN) {
        const uint32_t wn = total - w0 < PATCH_WIN ? total - w0 : PATCH_WIN;
        const uint32_t ob = (base + w0) & 3u;
        if (w0 == 0) {
#pragma unroll
            for (uint32_t j = 0; j < 4; ++j) stage[lane + 32 * j] = st[j];
        } else {
            const uint32_t nwords = (ob + wn + 3) >> 2;
            const uint32_t *src = reinterpret_cast<const uint32_t *>(P.dp) + ((base + w0) >> 2);
#pragma unroll
            for (uint32_t j = 0; j < 4; ++j)
                if (lane + 32 * j < nwords) stage[lane + 32 * j] = __ldg(src + lane + 32 * j);
        }
        // marks of whole 64-entry groups are cleared, so the last group reads zeros past wn
        for (uint32_t q = lane; q < ((wn + 63) >> 6) * 32; q += 32) marks32[q] = 0;
        __syncwarp();
        // mark = first tile bit of the slice + 1, dropped at the slice's first entry
        uint32_t run = first - w0;
#pragma unroll
        for (uint32_t i = 0; i < G; ++i) {
            if (f[i] != 0 && run < wn) marks[run] = (uint16_t)((lane * G + i) * N_OUT + 1);
            run += f[i];
        }
        __syncwarp();
        const uint8_t *bytes = reinterpret_cast<const uint8_t *>(stage) + ob;
        // two groups of 32 entries per round (two independent chains of shared-memory reads and
        // shuffles); every entry takes the nearest mark at or before it, else the carry
        for (uint32_t e0 = 0; e0 < wn; e0 += 64) {
            const uint32_t ea = e0 + lane, eb = ea + 32;
            uint32_t va = marks[ea], vb = marks[eb];
            const uint32_t pa = bytes[ea], pb = bytes[eb];
            const uint32_t sa = __ballot_sync(0xffffffffu, va != 0) & below_me;
            const uint32_t sb = __ballot_sync(0xffffffffu, vb != 0) & below_me;
            const uint32_t ga = __shfl_sync(0xffffffffu, va, (31 - __clz((int)sa)) & 31);
            const uint32_t gb = __shfl_sync(0xffffffffu, vb, (31 - __clz((int)sb)) & 31);
            va = sa ? ga : carry;
            const uint32_t ca = __shfl_sync(0xffffffffu, va, 31);
            vb = sb ? gb : ca;
            carry = __shfl_sync(0xffffffffu, vb, 31);
            const bool la = ea < wn, lb = eb < wn;
            const bool oka = la && va != 0 && pa < N_OUT, okb = lb && vb != 0 && pb < N_OUT;
            bad |= (uint32_t)((la && !oka) || (lb && !okb));
            if (oka) {
                const uint32_t bit = va - 1 + pa;
                atomicXor(region + (bit >> 5), 1u << (bit & 31));
            }
            if (okb) {
                const uint32_t bit = vb - 1 + pb;
                atomicXor(region + (bit >> 5), 1u << (bit & 31));
            }
        }
        __syncwarp();
    }
    if (bad) flag(A.status, 1u);
}

// The same patch step for runs that fit one window (at most PATCH_WIN entries), which is nearly
// every tile at the patch densities the format is meant for.  Differences from patch_tile: a lane handles
// the four entries of one staged d_patch word a round, straight from the register it was fetched into
// (nothing but the marks goes through shared memory); marks are indexed by byte position in the staged
// words and, since they grow along the run, "nearest mark at or before" is a running maximum -- three
// maxima inside the lane, one ballot and one shuffle across lanes, one shuffle to carry it into the next
// round.
template <uint32_t G, uint32_t N_OUT, typename WT>
SQNN_DEV void patch_tile_fast(const DecodeArgs &A, const PlanePtrs &P, uint32_t *region, uint32_t *stage,
                              const uint32_t (&st)[4], uint32_t base, uint32_t total, WT win, uint32_t lane)
{
    const uint32_t w_np = P.w_np;
    const uint32_t fm = (1u << w_np) - 1u;
    uint32_t f[G];
    uint32_t cnt = 0;
#pragma unroll
    for (uint32_t i = 0; i < G; ++i) {
        f[i] = (uint32_t)win & fm;
        win >>= w_np;
        cnt += f[i];
    }
    uint32_t incl = cnt;
#pragma unroll
    for (uint32_t d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
    }
    if (__shfl_sync(0xffffffffu, incl, 31) != total) {      // counts disagree with the offsets
        flag(A.status, 2u);
        return;
    }
    const uint32_t ob = base & 3u;                           // entry 0 sits at byte `ob` of the staged words
    const uint32_t rounds = (ob + total + 127u) >> 7;        // 128 byte positions a round, at most 4 rounds
    uint32_t *marks32 = stage + STAGE_DP_WORDS;
    uint2 *marks64 = reinterpret_cast<uint2 *>(marks32);
    uint16_t *marks = reinterpret_cast<uint16_t *>(marks32);
    for (uint32_t j = 0; j < rounds; ++j) marks64[32 * j + lane] = make_uint2(0u, 0u);
    __syncwarp();
    // mark = first tile bit of the slice + 1, dropped at the byte position of the slice's first entry
    uint32_t run = ob + incl - cnt, mark = lane * G * N_OUT + 1u;
#pragma unroll
    for (uint32_t i = 0; i < G; ++i) {
        if (f[i] != 0) marks[run] = (uint16_t)mark;
        run += f[i];
        mark += N_OUT;
    }
    __syncwarp();
    const uint32_t lower = (1u << lane) - 1u;                // lanes below this one
    uint32_t carry = 0, bad = 0;
#pragma unroll
    for (uint32_t j = 0; j < 4; ++j) {
        if (j < rounds) {                                    // the same in every lane
            const uint2 mm = marks64[32 * j + lane];
            const uint32_t m0 = mm.x & 0xffffu, m1 = mm.x >> 16, m2 = mm.y & 0xffffu, m3 = mm.y >> 16;
            const uint32_t last = max(max(m0, m1), max(m2, m3));
            const uint32_t have = __ballot_sync(0xffffffffu, last != 0) & lower;
            const uint32_t got = __shfl_sync(0xffffffffu, last, (31 - __clz((int)have)) & 31);
            const uint32_t prev = have ? got : carry;
            uint32_t v[4];
            v[0] = max(m0, prev);
            v[1] = max(m1, v[0]);
            v[2] = max(m2, v[1]);
            v[3] = max(m3, v[2]);
            carry = __shfl_sync(0xffffffffu, v[3], 31);
            const uint32_t w = st[j];
            // byte q of this word is entry 4 * (32 j + lane) + q - ob: inside the run iff lo <= q < hi
            const int32_t lo = (int32_t)ob - (int32_t)(4u * (32u * j + lane));
            const int32_t hi = lo + (int32_t)total;
#pragma unroll
            for (int32_t q = 0; q < 4; ++q) {
                if (q >= lo && q < hi) {
                    const uint32_t pos = (w >> (8 * q)) & 0xffu;
                    if (v[q] != 0 && pos < N_OUT) {
                        const uint32_t bit = v[q] - 1u + pos;
                        atomicXor(region + (bit >> 5), 1u << (bit & 31u));
                    } else {
                        bad = 1u;
                    }
                }
            }
        }
    }
    __syncwarp();
    if (bad) flag(A.status, 1u);
}

// Expands and patches the lane's G slices of one tile (already fetched into `in`, staged d_patch
// words in `st`) into region[lane * W .. lane * W + W); the patch step then works on the whole
// tile.  `stage` is the warp's STAGE_WORDS words of shared scratch.  WAIT_BULK: lane 0 first waits for its pending bulk copy out of
// `region`, just before the region is overwritten.  Ends with the warp synchronised.
template <int N_OUT, int N_IN, bool WAIT_BULK = false>
SQNN_DEV void tile_decode(const DecodeArgs &A, const PlanePtrs &P, const TileIn<N_OUT, N_IN> &in,
                          const uint32_t (&st)[4], uint32_t *region, const uint32_t *tab, uint32_t *stage,
                          uint32_t lane)
{
    using S = Shape<N_OUT, N_IN>;
    constexpr uint32_t G = S::G, W = S::W, NW = S::NW, NWP = S::NWP, NCH = S::NCH, CB = S::CB;
    constexpr uint32_t n_out = S::n_out, n_in = S::n_in, NSW = S::NSW;
    uint32_t *mine = region + lane * W;

    // seeds -> table entries
    const uint32_t sh0 = (lane * S::SPAN) & 31u;
    uint32_t al[NSW];
#pragma unroll
    for (uint32_t k = 0; k < NSW; ++k) al[k] = __funnelshift_r(in.raw[k], in.raw[k + 1], sh0);
    uint32_t x[G][NWP];
#pragma unroll
    for (uint32_t i = 0; i < G; ++i) {
        constexpr uint32_t smask = n_in >= 32 ? 0xffffffffu : ((1u << n_in) - 1u);
        const uint32_t o = i * n_in, w = o >> 5, s = o & 31;
        uint32_t seed;
        if (s + n_in <= 32) seed = (al[w] >> s) & smask;
        else seed = __funnelshift_r(al[w], al[w + 1 < NSW ? w + 1 : w], s) & smask;
        load_entry<NWP>(tab, seed & ((1u << CB) - 1u), x[i]);
#pragma unroll
        for (uint32_t ch = 1; ch < NCH; ++ch) {
            uint32_t y[NWP];
            load_entry<NWP>(tab, (ch << CB) | ((seed >> (ch * CB)) & ((1u << CB) - 1u)), y);
#pragma unroll
            for (uint32_t k = 0; k < NW; ++k) x[i][k] ^= y[k];
        }
    }
    if constexpr (WAIT_BULK) {                       // the bulk copy of the previous tile still reads `region`
        if (lane == 0) bulk_wait_read<0>();
        __syncwarp();
    }
    // output word k = bits [32k, 32k + 32) of the concatenated entries (entry bits >= n_out are 0)
#pragma unroll
    for (uint32_t k = 0; k < W; ++k) {
        const uint32_t i0 = (32 * k) / n_out, o = 32 * k - i0 * n_out;
        const uint32_t lo = x[i0][o >> 5];
        const uint32_t hi = ((o >> 5) + 1 < NW) ? x[i0][((o >> 5) + 1 < NW) ? (o >> 5) + 1 : 0] : 0u;
        uint32_t word = (o & 31) ? __funnelshift_r(lo, hi, o & 31) : lo;
        uint32_t filled = n_out - o;
#pragma unroll
        for (uint32_t i = i0 + 1; i < G; ++i) {
            if (filled < 32) { word |= x[i][0] << filled; filled += n_out; }
        }
        mine[k] = word;
    }

    // patches (warp-uniform branch: `total` is the same in every lane)
    if (in.total != 0) {
        __syncwarp();                                   // every lane's words are in place
        const uint32_t nb = lane * G * P.w_np, sh = nb & 31u;
        // the words fetched ahead hold at most PATCH_WIN entries (then alignment bytes + entries <= 511)
        const bool one_window = in.total <= PATCH_WIN;                   // the same in every lane
        if (G * P.w_np <= 32) {
            const uint32_t win = __funnelshift_r(in.np0, in.np1, sh) &
                                 (G * P.w_np == 32 ? 0xffffffffu : (1u << (G * P.w_np)) - 1u);
            if (one_window) patch_tile_fast<G, n_out, uint32_t>(A, P, region, stage, st, in.base, in.total, win, lane);
            else patch_tile<G, n_out, uint32_t>(A, P, region, stage, st, in.base, in.total, win, lane);
        } else {
            uint64_t win = (uint64_t)__funnelshift_r(in.np0, in.np1, sh) |
                           ((uint64_t)__funnelshift_r(in.np1, in.np2, sh) << 32);
            if (G * P.w_np < 64) win &= (1ull << (G * P.w_np)) - 1ull;
            if (one_window) patch_tile_fast<G, n_out, uint64_t>(A, P, region, stage, st, in.base, in.total, win, lane);
            else patch_tile<G, n_out, uint64_t>(A, P, region, stage, st, in.base, in.total, win, lane);
        }
    }
    __syncwarp();
}

// Fetch + decode of one tile without overlap (for the kernels that do more work per tile).
template <int N_OUT, int N_IN>
SQNN_DEV void decode_warp_tile(const DecodeArgs &A, uint32_t plane, uint64_t tile,
                               uint32_t *region, const uint32_t *tab, uint32_t *stage, uint32_t lane);

// Run-time shape: plain loops, every read through extract_bits.
SQNN_DEV void decode_warp_tile_generic(const DecodeArgs &A, uint32_t plane, uint64_t tile,
                                       uint32_t *region, const uint32_t *tab, uint32_t lane)
{
    const PlanePtrs &P = A.pl[plane];
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
    // Patches (Section 3.2): the lane's first entry sits at the block offset of the tile plus
    // the n_patch counts of the lanes before it.
    if (P.w_np != 0) {
        uint32_t cnt = 0;
        for (uint32_t i = 0; i < G; ++i) cnt += extract_bits(P.np, (s0 + i) * P.w_np, P.w_np);
        uint32_t incl = cnt;
#pragma unroll
        for (uint32_t d = 1; d < 32; d <<= 1) {
            const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        if (cnt != 0) {
            uint32_t at = __ldg(P.idx + tile * (G / 4)) + incl - cnt;
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
    __syncwarp();
}

template <int N_OUT, int N_IN>
SQNN_DEV void decode_warp_tile(const DecodeArgs &A, uint32_t plane, uint64_t tile,
                               uint32_t *region, const uint32_t *tab, uint32_t *stage, uint32_t lane)
{
    if constexpr (N_OUT != 0) {
        const PlanePtrs &P = A.pl[plane];
        TileIn<N_OUT, N_IN> in;
        uint32_t st[4];
        tile_fetch<N_OUT, N_IN>(P, tile, lane, in);
        stage_fetch<N_OUT, N_IN>(A, P, in, lane, st);
        tile_decode<N_OUT, N_IN>(A, P, in, st, region, tab, stage, lane);
    } else {
        decode_warp_tile_generic(A, plane, tile, region, tab, lane);
    }
}

}  // namespace sqnn
