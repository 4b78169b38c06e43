// Host side of the library: encryption of slices (Algorithm 1 / exhaustive search), the
// packed blob format, its validation and size accounting.  No CUDA in this file.
#include "sqnn.h"
#include "sqnn_blob.h"
#include "sqnn_layout.h"

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

namespace {

inline int popc64(uint64_t v) { return __builtin_popcountll(v); }
inline int ctz32(uint32_t v) { return __builtin_ctz(v); }

// `count` (<= 64) bits of a packed vector starting at flat position p; positions >= limit read 0.
inline uint64_t window(const uint64_t *words, uint64_t p, uint32_t count, uint64_t limit)
{
    if (p >= limit) return 0;
    if (p + count > limit) count = (uint32_t)(limit - p);
    const uint64_t w = p >> 6;
    const uint32_t sh = (uint32_t)(p & 63);
    uint64_t v = words[w] >> sh;
    if (sh && sh + count > 64) v |= words[w + 1] << (64 - sh);
    if (count < 64) v &= ((uint64_t)1 << count) - 1;
    return v;
}

inline uint32_t ceil_lg_u64(uint64_t v)   // smallest e with 2^e >= v (0 for v <= 1)
{
    uint32_t e = 0;
    while (((uint64_t)1 << e) < v) ++e;
    return e;
}

struct SliceBits {            // wanted bits and care flags of one slice, n_out <= 256
    uint64_t want[4];
    uint64_t care[4];
};

inline void load_slice(const uint64_t *plane, const uint64_t *mask, uint64_t mn, uint32_t n_out,
                       uint64_t s, SliceBits &sb)
{
    const uint64_t p0 = s * (uint64_t)n_out;
    for (uint32_t k = 0; k < 4; ++k) {
        const uint32_t lo = k * 64;
        if (lo >= n_out) { sb.want[k] = sb.care[k] = 0; continue; }
        const uint32_t cnt = std::min<uint32_t>(64, n_out - lo);
        sb.care[k] = window(mask, p0 + lo, cnt, mn);
        sb.want[k] = window(plane, p0 + lo, cnt, mn);
    }
}

// w~ = M . w^c over GF(2): bit j = parity(rows[j] AND seed)
inline void expand(const uint32_t *rows, uint32_t n_out, uint32_t seed, uint64_t out[4])
{
    out[0] = out[1] = out[2] = out[3] = 0;
    for (uint32_t j = 0; j < n_out; ++j)
        out[j >> 6] |= (uint64_t)(__builtin_popcount(rows[j] & seed) & 1) << (j & 63);
}

// Algorithm 1 on one slice.  The augmented matrix is kept in reduced row-echelon form while
// care rows are appended in ascending position: a new row is first reduced against the pivots;
// if it reduces to 0 = 1 it is the unsolvable case and is dropped (it will show up as a patch),
// if it reduces to 0 = 0 it is redundant, otherwise its lowest set column becomes a new pivot
// and is eliminated from the older rows.  Free variables are 0, so a pivot variable equals the
// right-hand side of its row.
inline uint32_t encode_alg1(const uint32_t *rows, uint32_t n_out, const SliceBits &sb)
{
    uint32_t prow[SQNN_MAX_N_IN], pcol[SQNN_MAX_N_IN];
    uint8_t prhs[SQNN_MAX_N_IN];
    uint32_t npiv = 0;
    for (uint32_t k = 0; k * 64 < n_out; ++k) {
        uint64_t c = sb.care[k];
        while (c) {
            const uint32_t j = k * 64 + (uint32_t)__builtin_ctzll(c);
            c &= c - 1;
            uint32_t a = rows[j];
            uint8_t b = (uint8_t)((sb.want[k] >> (j & 63)) & 1);
            for (uint32_t q = 0; q < npiv; ++q)
                if ((a >> pcol[q]) & 1) { a ^= prow[q]; b ^= prhs[q]; }
            if (a == 0) continue;                 // redundant or contradictory: nothing to keep
            const uint32_t col = (uint32_t)ctz32(a);
            for (uint32_t q = 0; q < npiv; ++q)
                if ((prow[q] >> col) & 1) { prow[q] ^= a; prhs[q] ^= b; }
            prow[npiv] = a; prhs[npiv] = b; pcol[npiv] = col;
            ++npiv;
        }
    }
    uint32_t seed = 0;
    for (uint32_t q = 0; q < npiv; ++q)
        if (prhs[q]) seed |= 1u << pcol[q];
    return seed;
}

// All 2^n_in outputs of the network, 4 words each.
void build_outputs(const uint32_t *rows, uint32_t n_out, uint32_t n_in, std::vector<uint64_t> &tab)
{
    const uint64_t cnt = (uint64_t)1 << n_in;
    tab.assign(cnt * 4, 0);
    for (uint64_t v = 0; v < cnt; ++v) expand(rows, n_out, (uint32_t)v, &tab[v * 4]);
}

inline uint32_t encode_exhaustive(const std::vector<uint64_t> &tab, uint32_t n_in, const SliceBits &sb)
{
    const uint64_t cnt = (uint64_t)1 << n_in;
    uint32_t best = 0;
    int best_wrong = 1 << 30;
    for (uint64_t v = 0; v < cnt; ++v) {
        const uint64_t *o = &tab[v * 4];
        int wrong = 0;
        for (int k = 0; k < 4; ++k) wrong += popc64((o[k] ^ sb.want[k]) & sb.care[k]);
        if (wrong < best_wrong) { best_wrong = wrong; best = (uint32_t)v; }
    }
    return best;
}

struct PlaneArrays {
    std::vector<uint32_t> wc;
    std::vector<uint16_t> np;
    std::vector<uint8_t> dp;
};

uint64_t round_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

// Packs bit fields of `width` bits (value i at bits [i*width, (i+1)*width)) into uint32 words.
// Groups of 32 values fill whole words, so groups can be written independently.
template <typename T>
void pack_fields(const T *vals, uint64_t count, uint32_t width, uint32_t *dst)
{
    if (width == 0) return;
    const int64_t groups = (int64_t)((count + 31) / 32);
#pragma omp parallel for schedule(static)
    for (int64_t g = 0; g < groups; ++g) {
        uint32_t *w = dst + (uint64_t)g * width;
        uint64_t acc = 0;
        uint32_t have = 0, wi = 0;
        const uint64_t lo = (uint64_t)g * 32, hi = std::min<uint64_t>(count, lo + 32);
        for (uint64_t i = lo; i < hi; ++i) {
            acc |= (uint64_t)vals[i] << have;
            have += width;
            while (have >= 32) { w[wi++] = (uint32_t)acc; acc >>= 32; have -= 32; }
        }
        if (have) w[wi] = (uint32_t)acc;
    }
}

inline uint32_t read_field(const uint32_t *src, uint64_t index, uint32_t width)
{
    if (width == 0) return 0;
    const uint64_t bit = index * width;
    const uint64_t w = bit >> 5;
    const uint32_t sh = (uint32_t)(bit & 31);
    uint64_t v = (uint64_t)src[w] | ((uint64_t)src[w + 1] << 32);   // sections end with slack
    return (uint32_t)((v >> sh) & (((uint64_t)1 << width) - 1));
}

// The lookup tables of the network in the layout the kernels index (sqnn_layout.h).
void build_tables(const uint32_t *rows, uint32_t n_out, uint32_t n_in, uint32_t *tab)
{
    const uint32_t nwp = sqnn::entry_words_padded(n_out);
    const uint32_t nch = sqnn::table_chunks(n_in, nwp), cb = sqnn::chunk_bits(n_in, nwp);
    std::memset(tab, 0, (size_t)sqnn::table_words(n_out, n_in) * 4);
    for (uint32_t ch = 0; ch < nch; ++ch)
        for (uint32_t v = 0; v < (1u << cb); ++v) {
            // chunk bits that lie past n_in select no column
            const uint64_t sel64 = (uint64_t)v << (ch * cb);
            const uint32_t sel = (uint32_t)(sel64 & (n_in >= 32 ? 0xffffffffull : ((1ull << n_in) - 1ull)));
            uint32_t *e = tab + (size_t)(((ch << cb) | v)) * nwp;
            for (uint32_t j = 0; j < n_out; ++j)
                e[j >> 5] |= (uint32_t)(__builtin_popcount(rows[j] & sel) & 1) << (j & 31);
        }
}

struct BlobPlan {
    sqnn_desc d;
};

// Section offsets of a device blob for the given patch totals.
void plan_blob(uint64_t m, uint64_t n, uint32_t n_q, uint32_t n_out, uint32_t n_in, const uint64_t *n_pp, sqnn_desc *out)
{
    sqnn_desc d;
    std::memset(&d, 0, sizeof d);
    const uint64_t mn = m * n;
    const uint64_t l = (mn + n_out - 1) / n_out;
    const uint64_t lp = round_up(l, SQNN_PAD_SLICES);
    d.m = m; d.n = n; d.slices = l; d.slices_padded = lp;
    d.n_q = n_q; d.n_out = n_out; d.n_in = n_in; d.tile_slices = SQNN_TILE_SLICES;
    d.tab_entry_words = sqnn::entry_words_padded(n_out);
    d.tab_chunks = sqnn::table_chunks(n_in, d.tab_entry_words);
    d.tab_chunk_bits = sqnn::chunk_bits(n_in, d.tab_entry_words);
    uint64_t off = SQNN_BLOB_HEADER_BYTES;
    d.off_xornet = off;
    off += round_up((uint64_t)n_out * 4, 16) + 16;
    d.off_tables = off;
    d.tables_bytes = (uint64_t)sqnn::table_words(n_out, n_in) * 4;
    off += round_up(d.tables_bytes, 16) + 16;
    for (uint32_t i = 0; i < n_q; ++i) {
        d.n_pp[i] = n_pp[i];
        d.off_wc[i] = off;  off += round_up(lp * n_in / 8, 16) + 16;
        d.off_idx[i] = off; off += round_up((lp / SQNN_TILE_SLICES + 1) * 4, 16) + 16;
        d.off_pp[i] = off;  off += round_up(n_pp[i] * 2, 16) + 16;
    }
    d.total_bytes = off;
    *out = d;
}

int build_blob(const sqnn_xornet *net, uint64_t m, uint64_t n, uint32_t n_q,
               const uint32_t *const *wc, const uint16_t *const *np, const uint8_t *const *dp8,
               const uint16_t *const *dp16, void **blob, size_t *blob_bytes)
{
    const uint64_t mn = m * n;
    const uint32_t n_out = net->n_out, n_in = net->n_in;
    const uint64_t l = (mn + n_out - 1) / n_out;
    uint64_t n_pp[SQNN_MAX_PLANES] = {0};
    for (uint32_t i = 0; i < n_q; ++i) {
        uint64_t sum = 0;
        for (uint64_t s = 0; s < l; ++s) {
            if (np[i][s] > n_out) return SQNN_E_INVALID_ARG;
            sum += np[i][s];
        }
        if (sum > 0xffffffffull) return SQNN_E_INVALID_ARG;
        n_pp[i] = sum;
    }
    sqnn_desc d;
    plan_blob(m, n, n_q, n_out, n_in, n_pp, &d);
    const uint64_t lp = d.slices_padded;
    uint8_t *b = (uint8_t *)std::calloc(d.total_bytes, 1);
    if (!b) return SQNN_E_NOMEM;
    sqnn_blob_header *h = (sqnn_blob_header *)b;
    std::memcpy(h->magic, SQNN_BLOB_MAGIC, 8);
    h->version = SQNN_BLOB_VERSION;
    h->header_bytes = SQNN_BLOB_HEADER_BYTES;
    h->desc = d;
    std::memcpy(b + d.off_xornet, net->rows, (size_t)n_out * 4);
    build_tables(net->rows, n_out, n_in, (uint32_t *)(b + d.off_tables));
    for (uint32_t i = 0; i < n_q; ++i) {
        if (n_in < 32)
            for (uint64_t s = 0; s < l; ++s)
                if (wc[i][s] >> n_in) { std::free(b); return SQNN_E_INVALID_ARG; }
        pack_fields(wc[i], l, n_in, (uint32_t *)(b + d.off_wc[i]));
        uint32_t *idx = (uint32_t *)(b + d.off_idx[i]);
        uint16_t *dst = (uint16_t *)(b + d.off_pp[i]);
        uint64_t run = 0;
        const uint64_t tiles = lp / SQNN_TILE_SLICES;
        for (uint64_t t = 0; t <= tiles; ++t) {
            idx[t] = (uint32_t)run;
            if (t == tiles) break;
            const uint64_t lo = t * SQNN_TILE_SLICES, hi = std::min<uint64_t>(l, lo + SQNN_TILE_SLICES);
            for (uint64_t s = lo; s < hi; ++s) {
                int64_t prev = -1;
                for (uint32_t k = 0; k < np[i][s]; ++k, ++run) {
                    const uint32_t pos = dp8 ? dp8[i][run] : dp16[i][run];
                    // positions inside a slice ascend strictly; the last slice holds real positions only
                    if (pos >= n_out || (int64_t)pos <= prev || s * n_out + pos >= mn) { std::free(b); return SQNN_E_INVALID_ARG; }
                    prev = pos;
                    dst[run] = (uint16_t)((s - lo) * n_out + pos);
                }
            }
        }
        if (run != n_pp[i]) { std::free(b); return SQNN_E_INVALID_ARG; }
    }
    *blob = b;
    *blob_bytes = d.total_bytes;
    return SQNN_OK;
}

bool net_ok(const sqnn_xornet *net)
{
    return net && net->rows && net->n_out >= 1 && net->n_out <= SQNN_MAX_N_OUT &&
           net->n_in >= 1 && net->n_in <= SQNN_MAX_N_IN;
}

}  // namespace

extern "C" {

void sqnn_free(void *p) { std::free(p); }

const char *sqnn_status_string(int status)
{
    switch (status) {
        case SQNN_OK: return "ok";
        case SQNN_E_INVALID_ARG: return "invalid argument";
        case SQNN_E_BAD_BLOB: return "malformed blob";
        case SQNN_E_UNSUPPORTED: return "unsupported";
        case SQNN_E_NOMEM: return "out of host memory";
        case SQNN_E_CUDA: return "CUDA runtime error";
        case SQNN_E_TIMEOUT: return "device-side wait timed out";
        case SQNN_E_WORKSPACE: return "workspace missing or too small";
        default: return "unknown status";
    }
}

// Shared by sqnn_encode_host and sqnn_encode_seeds_host: seeds come from Algorithm 1, from the
// exhaustive search, or from the caller (given != NULL); patch counts and positions follow by
// expanding each seed and comparing on the care bits.
static int encode_impl(const sqnn_xornet *net, const sqnn_planes *layer, bool exhaustive,
                       const uint32_t *const *given, void **blob, size_t *blob_bytes, sqnn_stats *stats)
{
    try {
        const uint64_t mn = layer->m * layer->n;
        const uint32_t n_out = net->n_out, n_in = net->n_in, n_q = layer->n_q;
        const uint64_t l = (mn + n_out - 1) / n_out;
        const uint64_t words = (mn + 63) / 64;
        std::vector<uint64_t> tab;
        if (exhaustive && !given) build_outputs(net->rows, n_out, n_in, tab);
        std::vector<PlaneArrays> pa(n_q);
        for (uint32_t i = 0; i < n_q; ++i) {
            const uint64_t *plane = layer->planes + (uint64_t)i * words;
            pa[i].wc.assign(l, 0);
            pa[i].np.assign(l, 0);
            int bad_seed = 0;
            // pass 1: seed and patch count of every slice (slices are independent)
#pragma omp parallel for schedule(dynamic, 4096)
            for (int64_t s = 0; s < (int64_t)l; ++s) {
                SliceBits sb;
                load_slice(plane, layer->mask, mn, n_out, (uint64_t)s, sb);
                uint32_t seed;
                if (given) {
                    seed = given[i][s];
                    if (n_in < 32 && (seed >> n_in)) {
#pragma omp atomic write
                        bad_seed = 1;
                        seed = 0;
                    }
                } else {
                    seed = exhaustive ? encode_exhaustive(tab, n_in, sb) : encode_alg1(net->rows, n_out, sb);
                }
                uint64_t out[4];
                expand(net->rows, n_out, seed, out);
                int wrong = 0;
                for (int k = 0; k < 4; ++k) wrong += popc64((out[k] ^ sb.want[k]) & sb.care[k]);
                pa[i].wc[s] = seed;
                pa[i].np[s] = (uint16_t)wrong;
            }
            if (bad_seed) return SQNN_E_INVALID_ARG;
            // pass 2: positions of the wrong care bits, written at the running offset
            std::vector<uint64_t> start(l + 1, 0);
            for (uint64_t s = 0; s < l; ++s) start[s + 1] = start[s] + pa[i].np[s];
            pa[i].dp.assign(start[l] + 1, 0);
#pragma omp parallel for schedule(dynamic, 4096)
            for (int64_t s = 0; s < (int64_t)l; ++s) {
                if (!pa[i].np[s]) continue;
                SliceBits sb;
                load_slice(plane, layer->mask, mn, n_out, (uint64_t)s, sb);
                uint64_t out[4];
                expand(net->rows, n_out, pa[i].wc[s], out);
                uint64_t at = start[s];
                for (uint32_t k = 0; k * 64 < n_out; ++k) {
                    uint64_t bad = (out[k] ^ sb.want[k]) & sb.care[k];
                    while (bad) {
                        pa[i].dp[at++] = (uint8_t)(k * 64 + (uint32_t)__builtin_ctzll(bad));
                        bad &= bad - 1;
                    }
                }
            }
        }
        std::vector<const uint32_t *> wcp(n_q);
        std::vector<const uint16_t *> npp(n_q);
        std::vector<const uint8_t *> dpp(n_q);
        for (uint32_t i = 0; i < n_q; ++i) { wcp[i] = pa[i].wc.data(); npp[i] = pa[i].np.data(); dpp[i] = pa[i].dp.data(); }
        int rc = build_blob(net, layer->m, layer->n, n_q, wcp.data(), npp.data(), dpp.data(), nullptr, blob, blob_bytes);
        if (rc != SQNN_OK) return rc;
        if (stats) {
            rc = sqnn_stats_host(*blob, *blob_bytes, stats);
            if (rc != SQNN_OK) { std::free(*blob); *blob = nullptr; return rc; }
        }
        return SQNN_OK;
    } catch (const std::bad_alloc &) {
        return SQNN_E_NOMEM;
    }
}

static bool layer_ok(const sqnn_planes *layer)
{
    return layer && layer->planes && layer->mask && layer->n_q >= 1 && layer->n_q <= SQNN_MAX_PLANES &&
           layer->m != 0 && layer->n != 0 && layer->m <= ((uint64_t)1 << 40) / layer->n;
}

int sqnn_encode_host(const sqnn_xornet *net, const sqnn_planes *layer, uint32_t flags,
                     void **blob, size_t *blob_bytes, sqnn_stats *stats)
{
    if (!net_ok(net) || !layer_ok(layer) || !blob || !blob_bytes) return SQNN_E_INVALID_ARG;
    const bool exhaustive = (flags & SQNN_ENCODE_EXHAUSTIVE) != 0;
    if (exhaustive && net->n_in > 20) return SQNN_E_INVALID_ARG;
    return encode_impl(net, layer, exhaustive, nullptr, blob, blob_bytes, stats);
}

int sqnn_encode_seeds_host(const sqnn_xornet *net, const sqnn_planes *layer, const uint32_t *const *wc,
                           void **blob, size_t *blob_bytes, sqnn_stats *stats)
{
    if (!net_ok(net) || !layer_ok(layer) || !wc || !blob || !blob_bytes) return SQNN_E_INVALID_ARG;
    for (uint32_t i = 0; i < layer->n_q; ++i)
        if (!wc[i]) return SQNN_E_INVALID_ARG;
    return encode_impl(net, layer, false, wc, blob, blob_bytes, stats);
}

int sqnn_pack_host(const sqnn_xornet *net, uint64_t m, uint64_t n, uint32_t n_q,
                   const uint32_t *const *wc, const uint16_t *const *np, const uint16_t *const *dp,
                   void **blob, size_t *blob_bytes)
{
    if (!net_ok(net) || !wc || !np || !dp || !blob || !blob_bytes) return SQNN_E_INVALID_ARG;
    if (n_q < 1 || n_q > SQNN_MAX_PLANES || m == 0 || n == 0 || m > ((uint64_t)1 << 40) / n)
        return SQNN_E_INVALID_ARG;
    for (uint32_t i = 0; i < n_q; ++i)
        if (!wc[i] || !np[i] || !dp[i]) return SQNN_E_INVALID_ARG;
    try {
        return build_blob(net, m, n, n_q, wc, np, nullptr, dp, blob, blob_bytes);
    } catch (const std::bad_alloc &) {
        return SQNN_E_NOMEM;
    }
}

int sqnn_describe_host(const void *blob, size_t blob_bytes, sqnn_desc *desc)
{
    if (!blob || !desc) return SQNN_E_INVALID_ARG;
    if (blob_bytes < SQNN_BLOB_HEADER_BYTES) return SQNN_E_BAD_BLOB;
    const uint8_t *b = (const uint8_t *)blob;
    sqnn_blob_header h;
    std::memcpy(&h, b, sizeof h);
    if (std::memcmp(h.magic, SQNN_BLOB_MAGIC, 8) != 0 || h.version != SQNN_BLOB_VERSION ||
        h.header_bytes != SQNN_BLOB_HEADER_BYTES)
        return SQNN_E_BAD_BLOB;
    const sqnn_desc &d = h.desc;
    if (d.n_out < 1 || d.n_out > SQNN_MAX_N_OUT || d.n_in < 1 || d.n_in > SQNN_MAX_N_IN ||
        d.n_q < 1 || d.n_q > SQNN_MAX_PLANES || d.tile_slices != SQNN_TILE_SLICES)
        return SQNN_E_BAD_BLOB;
    if (d.m == 0 || d.n == 0 || d.m > ((uint64_t)1 << 40) / d.n) return SQNN_E_BAD_BLOB;
    for (uint32_t i = 0; i < d.n_q; ++i)
        if (d.n_pp[i] > 0xffffffffull) return SQNN_E_BAD_BLOB;
    // every offset and size is a fixed function of the shape and the patch totals
    sqnn_desc want;
    plan_blob(d.m, d.n, d.n_q, d.n_out, d.n_in, d.n_pp, &want);
    if (std::memcmp(&want, &d, sizeof d) != 0 || d.total_bytes != blob_bytes) return SQNN_E_BAD_BLOB;
    const uint64_t mn = d.m * d.n, l = d.slices, lp = d.slices_padded;
    const uint32_t *rows = (const uint32_t *)(b + d.off_xornet);
    if (d.n_in < 32)
        for (uint32_t j = 0; j < d.n_out; ++j)
            if (rows[j] >> d.n_in) return SQNN_E_BAD_BLOB;
    try {
        std::vector<uint32_t> tab(sqnn::table_words(d.n_out, d.n_in));
        build_tables(rows, d.n_out, d.n_in, tab.data());
        if (std::memcmp(tab.data(), b + d.off_tables, (size_t)d.tables_bytes) != 0) return SQNN_E_BAD_BLOB;
    } catch (const std::bad_alloc &) {
        return SQNN_E_NOMEM;
    }
    const uint64_t tiles = lp / SQNN_TILE_SLICES;
    const uint64_t tile_bits = (uint64_t)SQNN_TILE_SLICES * d.n_out;
    for (uint32_t i = 0; i < d.n_q; ++i) {
        const uint32_t *wcs = (const uint32_t *)(b + d.off_wc[i]);
        const uint32_t *idx = (const uint32_t *)(b + d.off_idx[i]);
        const uint16_t *pp = (const uint16_t *)(b + d.off_pp[i]);
        for (uint64_t s = l; s < lp; ++s)
            if (read_field(wcs, s, d.n_in) != 0) return SQNN_E_BAD_BLOB;
        if (idx[0] != 0 || idx[tiles] != d.n_pp[i]) return SQNN_E_BAD_BLOB;
        for (uint64_t t = 0; t < tiles; ++t) {
            if (idx[t + 1] < idx[t] || idx[t + 1] > d.n_pp[i]) return SQNN_E_BAD_BLOB;
            int64_t prev = -1;
            for (uint64_t k = idx[t]; k < idx[t + 1]; ++k) {
                const uint64_t pos = pp[k];
                if (pos >= tile_bits || (int64_t)pos <= prev || t * tile_bits + pos >= mn) return SQNN_E_BAD_BLOB;
                prev = (int64_t)pos;
            }
        }
    }
    *desc = d;
    return SQNN_OK;
}

// n_patch of every slice of one plane, from the patch positions of a validated blob.
static void count_patches(const uint8_t *b, const sqnn_desc &d, uint32_t plane, uint16_t *np)
{
    const uint32_t *idx = (const uint32_t *)(b + d.off_idx[plane]);
    const uint16_t *pp = (const uint16_t *)(b + d.off_pp[plane]);
    std::memset(np, 0, sizeof(uint16_t) * (size_t)d.slices);
    const uint64_t tiles = d.slices_padded / SQNN_TILE_SLICES;
    for (uint64_t t = 0; t < tiles; ++t)
        for (uint64_t k = idx[t]; k < idx[t + 1]; ++k)
            ++np[t * SQNN_TILE_SLICES + pp[k] / d.n_out];
}

int sqnn_unpack_host(const void *blob, size_t blob_bytes, uint32_t plane,
                     uint32_t **wc, uint16_t **np, uint16_t **dp, uint64_t *n_dp)
{
    if (!wc || !np || !dp || !n_dp) return SQNN_E_INVALID_ARG;
    sqnn_desc d;
    int rc = sqnn_describe_host(blob, blob_bytes, &d);
    if (rc != SQNN_OK) return rc;
    if (plane >= d.n_q) return SQNN_E_INVALID_ARG;
    const uint8_t *b = (const uint8_t *)blob;
    const uint64_t l = d.slices;
    uint32_t *w = (uint32_t *)std::malloc(sizeof(uint32_t) * (l ? l : 1));
    uint16_t *p = (uint16_t *)std::malloc(sizeof(uint16_t) * (l ? l : 1));
    uint16_t *q = (uint16_t *)std::malloc(sizeof(uint16_t) * (d.n_pp[plane] ? d.n_pp[plane] : 1));
    if (!w || !p || !q) { std::free(w); std::free(p); std::free(q); return SQNN_E_NOMEM; }
    const uint32_t *wcs = (const uint32_t *)(b + d.off_wc[plane]);
    for (uint64_t s = 0; s < l; ++s) w[s] = read_field(wcs, s, d.n_in);
    count_patches(b, d, plane, p);
    // positions ascend inside a tile, so they already stand in slice order, ascending inside a slice
    const uint16_t *pp = (const uint16_t *)(b + d.off_pp[plane]);
    for (uint64_t k = 0; k < d.n_pp[plane]; ++k) q[k] = (uint16_t)(pp[k] % d.n_out);
    *wc = w; *np = p; *dp = q; *n_dp = d.n_pp[plane];
    return SQNN_OK;
}

int sqnn_stats_host(const void *blob, size_t blob_bytes, sqnn_stats *stats)
{
    if (!stats) return SQNN_E_INVALID_ARG;
    sqnn_desc d;
    int rc = sqnn_describe_host(blob, blob_bytes, &d);
    if (rc != SQNN_OK) return rc;
    std::memset(stats, 0, sizeof *stats);
    const uint8_t *b = (const uint8_t *)blob;
    const uint64_t mn = d.m * d.n, l = d.slices, lp = d.slices_padded;
    stats->slices = l;
    double eq1_bits = 0.0;
    try {
        std::vector<uint16_t> np(l ? l : 1);
        for (uint32_t i = 0; i < d.n_q; ++i) {
            count_patches(b, d, i, np.data());
            uint32_t maxp = 0;
            uint64_t sum = 0;
            for (uint64_t s = 0; s < l; ++s) {
                const uint32_t p = np[s];
                maxp = std::max(maxp, p);
                sum += p;
                ++stats->patch_hist[p < SQNN_PATCH_HIST_BINS - 1 ? p : SQNN_PATCH_HIST_BINS - 1];
            }
            stats->patches[i] = sum;
            stats->max_patch[i] = maxp;
            // Eq. 1, literally: n_in/n_out * mn + l * ceil(lg max p) + sum p * ceil(lg n_out)
            eq1_bits += (double)d.n_in / (double)d.n_out * (double)mn +
                        (double)l * ceil_lg_u64(maxp) + (double)sum * ceil_lg_u64(d.n_out);
            stats->bits_wc += (round_up(lp * d.n_in / 8, 16) + 16) * 8;
            stats->bits_index += (round_up((lp / SQNN_TILE_SLICES + 1) * 4, 16) + 16) * 8;
            stats->bits_dpatch += (round_up(sum * 2, 16) + 16) * 8;
        }
    } catch (const std::bad_alloc &) {
        return SQNN_E_NOMEM;
    }
    stats->bits_tables = (round_up(d.tables_bytes, 16) + 16) * 8;
    stats->bits_index += stats->bits_tables;
    stats->bpw_eq1 = eq1_bits / (double)mn;
    stats->bpw_actual = (double)(stats->bits_wc + stats->bits_npatch + stats->bits_index + stats->bits_dpatch) / (double)mn;
    return SQNN_OK;
}

int sqnn_stats_blocked_host(const void *blob, size_t blob_bytes, uint64_t block_slices,
                            double *bpw_eq1, uint64_t *bits_npatch)
{
    if (block_slices == 0) return SQNN_E_INVALID_ARG;
    sqnn_desc d;
    int rc = sqnn_describe_host(blob, blob_bytes, &d);
    if (rc != SQNN_OK) return rc;
    const uint8_t *b = (const uint8_t *)blob;
    const uint64_t mn = d.m * d.n, l = d.slices;
    uint64_t np_bits = 0, dp_entries = 0;
    try {
        std::vector<uint16_t> np(l ? l : 1);
        for (uint32_t i = 0; i < d.n_q; ++i) {
            count_patches(b, d, i, np.data());
            for (uint64_t s0 = 0; s0 < l; s0 += block_slices) {
                const uint64_t s1 = std::min(l, s0 + block_slices);
                uint32_t maxp = 0;
                for (uint64_t s = s0; s < s1; ++s) maxp = std::max<uint32_t>(maxp, np[s]);
                np_bits += (s1 - s0) * ceil_lg_u64(maxp);
            }
            dp_entries += d.n_pp[i];
        }
    } catch (const std::bad_alloc &) {
        return SQNN_E_NOMEM;
    }
    if (bits_npatch) *bits_npatch = np_bits;
    if (bpw_eq1)
        *bpw_eq1 = ((double)d.n_q * (double)d.n_in / (double)d.n_out * (double)mn + (double)np_bits +
                    (double)dp_entries * ceil_lg_u64(d.n_out)) / (double)mn;
    return SQNN_OK;
}

// ---------------------------------------------------------------------------------------------
// Algorithm 1 with 64-bit rows of M (host only)
// ---------------------------------------------------------------------------------------------
namespace {

inline uint32_t bit_at(const uint64_t *words, uint64_t p) { return (uint32_t)((words[p >> 6] >> (p & 63)) & 1); }

// Seed of one slice (positions [p0, p1) of the plane) by the same incremental elimination as
// encode_alg1, and the list of care positions the seed does not reproduce.
inline uint64_t encode_alg1_wide(const uint64_t *rows, const uint64_t *plane, const uint64_t *mask,
                                 uint64_t p0, uint64_t p1, std::vector<uint16_t> &wrong)
{
    uint64_t prow[64];
    uint32_t pcol[64];
    uint8_t prhs[64];
    uint32_t npiv = 0;
    for (uint64_t p = p0; p < p1; ++p) {
        if (!bit_at(mask, p)) continue;
        uint64_t a = rows[p - p0];
        uint8_t b = (uint8_t)bit_at(plane, p);
        for (uint32_t q = 0; q < npiv; ++q)
            if ((a >> pcol[q]) & 1) { a ^= prow[q]; b ^= prhs[q]; }
        if (a == 0) continue;
        const uint32_t col = (uint32_t)__builtin_ctzll(a);
        for (uint32_t q = 0; q < npiv; ++q)
            if ((prow[q] >> col) & 1) { prow[q] ^= a; prhs[q] ^= b; }
        prow[npiv] = a; prhs[npiv] = b; pcol[npiv] = col;
        ++npiv;
    }
    uint64_t seed = 0;
    for (uint32_t q = 0; q < npiv; ++q)
        if (prhs[q]) seed |= (uint64_t)1 << pcol[q];
    wrong.clear();
    for (uint64_t p = p0; p < p1; ++p)
        if (bit_at(mask, p) && (uint32_t)(__builtin_popcountll(rows[p - p0] & seed) & 1) != bit_at(plane, p))
            wrong.push_back((uint16_t)(p - p0));
    return seed;
}

}  // namespace

int sqnn_encode_wide_host(uint32_t n_out, uint32_t n_in, const uint64_t *rows, uint64_t mn,
                          const uint64_t *plane, const uint64_t *mask,
                          uint64_t **wc, uint16_t **np, uint16_t **dp, uint64_t *n_dp, double *bpw_eq1)
{
    if (!rows || !plane || !mask || !wc || !np || !dp || !n_dp || n_out < 1 || n_out > 4096 || n_in < 1 || n_in > 64 ||
        mn == 0 || mn > ((uint64_t)1 << 40))
        return SQNN_E_INVALID_ARG;
    if (n_in < 64)
        for (uint32_t j = 0; j < n_out; ++j)
            if (rows[j] >> n_in) return SQNN_E_INVALID_ARG;
    try {
        const uint64_t l = (mn + n_out - 1) / n_out;
        std::vector<uint64_t> seeds(l);
        std::vector<std::vector<uint16_t>> lists(l);
#pragma omp parallel
        {
            std::vector<uint16_t> wrong;
#pragma omp for schedule(dynamic, 256)
            for (int64_t s = 0; s < (int64_t)l; ++s) {
                const uint64_t p0 = (uint64_t)s * n_out, p1 = std::min(mn, p0 + n_out);
                seeds[s] = encode_alg1_wide(rows, plane, mask, p0, p1, wrong);
                lists[s] = wrong;
            }
        }
        uint64_t total = 0, maxp = 0;
        for (uint64_t s = 0; s < l; ++s) { total += lists[s].size(); maxp = std::max<uint64_t>(maxp, lists[s].size()); }
        uint64_t *w = (uint64_t *)std::malloc(sizeof(uint64_t) * l);
        uint16_t *c = (uint16_t *)std::malloc(sizeof(uint16_t) * l);
        uint16_t *q = (uint16_t *)std::malloc(sizeof(uint16_t) * (total ? total : 1));
        if (!w || !c || !q) { std::free(w); std::free(c); std::free(q); return SQNN_E_NOMEM; }
        uint64_t at = 0;
        for (uint64_t s = 0; s < l; ++s) {
            w[s] = seeds[s];
            c[s] = (uint16_t)lists[s].size();
            for (uint16_t v : lists[s]) q[at++] = v;
        }
        *wc = w; *np = c; *dp = q; *n_dp = total;
        if (bpw_eq1)
            *bpw_eq1 = ((double)n_in / (double)n_out * (double)mn + (double)l * ceil_lg_u64(maxp) +
                        (double)total * ceil_lg_u64(n_out)) / (double)mn;
        return SQNN_OK;
    } catch (const std::bad_alloc &) {
        return SQNN_E_NOMEM;
    }
}

// ---------------------------------------------------------------------------------------------
// storage form
// ---------------------------------------------------------------------------------------------
namespace {

const char STORE_MAGIC[8] = {'S', 'Q', 'N', 'N', 'S', 'T', 'R', '1'};

struct StoreHeader {
    char magic[8];
    uint64_t m, n, block_slices, total_bytes;
    uint32_t n_q, n_out, n_in, reserved;
    uint64_t n_dp[SQNN_MAX_PLANES];
    uint64_t reserved2;
};
static_assert(sizeof(StoreHeader) == 128, "storage header is 128 bytes");

struct BitWriter {
    std::vector<uint8_t> &buf;
    uint64_t acc = 0;
    uint32_t have = 0;
    explicit BitWriter(std::vector<uint8_t> &b) : buf(b) {}
    void put(uint32_t v, uint32_t width)
    {
        if (width == 0) return;
        acc |= (uint64_t)v << have;
        have += width;
        while (have >= 8) { buf.push_back((uint8_t)acc); acc >>= 8; have -= 8; }
    }
    void flush() { if (have) { buf.push_back((uint8_t)acc); acc = 0; have = 0; } }     // streams start on a byte
};

struct BitReader {
    const uint8_t *p, *end;
    uint64_t acc = 0;
    uint32_t have = 0;
    bool ok = true;
    BitReader(const uint8_t *b, const uint8_t *e) : p(b), end(e) {}
    uint32_t get(uint32_t width)
    {
        if (width == 0) return 0;
        while (have < width) {
            if (p >= end) { ok = false; return 0; }
            acc |= (uint64_t)*p++ << have;
            have += 8;
        }
        const uint32_t v = (uint32_t)(acc & (((uint64_t)1 << width) - 1));
        acc >>= width;
        have -= width;
        return v;
    }
    void align() { acc = 0; have = 0; }
};

}  // namespace

int sqnn_store_host(const void *blob, size_t blob_bytes, uint64_t block_slices,
                    void **stored, size_t *stored_bytes, sqnn_store_info *info)
{
    if (!stored || !stored_bytes || block_slices == 0) return SQNN_E_INVALID_ARG;
    sqnn_desc d;
    int rc = sqnn_describe_host(blob, blob_bytes, &d);
    if (rc != SQNN_OK) return rc;
    try {
        const uint8_t *b = (const uint8_t *)blob;
        const uint64_t l = d.slices;
        const uint32_t w_dp = ceil_lg_u64(d.n_out);
        StoreHeader h;
        std::memset(&h, 0, sizeof h);
        std::memcpy(h.magic, STORE_MAGIC, 8);
        h.m = d.m; h.n = d.n; h.block_slices = block_slices;
        h.n_q = d.n_q; h.n_out = d.n_out; h.n_in = d.n_in;
        std::vector<uint8_t> out(sizeof h, 0);
        out.insert(out.end(), b + d.off_xornet, b + d.off_xornet + (size_t)d.n_out * 4);
        sqnn_store_info si;
        std::memset(&si, 0, sizeof si);
        std::vector<uint16_t> np(l ? l : 1);
        for (uint32_t i = 0; i < d.n_q; ++i) {
            h.n_dp[i] = d.n_pp[i];
            const uint32_t *wcs = (const uint32_t *)(b + d.off_wc[i]);
            const uint16_t *pp = (const uint16_t *)(b + d.off_pp[i]);
            count_patches(b, d, i, np.data());
            BitWriter bw(out);
            for (uint64_t s = 0; s < l; ++s) bw.put(read_field(wcs, s, d.n_in), d.n_in);
            bw.flush();
            si.bits_wc += l * d.n_in;
            const uint64_t blocks = (l + block_slices - 1) / block_slices;
            std::vector<uint8_t> widths(blocks);
            for (uint64_t k = 0; k < blocks; ++k) {
                uint32_t maxp = 0;
                for (uint64_t s = k * block_slices; s < std::min(l, (k + 1) * block_slices); ++s) maxp = std::max<uint32_t>(maxp, np[s]);
                widths[k] = (uint8_t)ceil_lg_u64((uint64_t)maxp + 1);
            }
            out.insert(out.end(), widths.begin(), widths.end());
            si.bits_widths += blocks * 8;
            for (uint64_t s = 0; s < l; ++s) {
                bw.put(np[s], widths[s / block_slices]);
                si.bits_npatch += widths[s / block_slices];
            }
            bw.flush();
            for (uint64_t k = 0; k < d.n_pp[i]; ++k) bw.put(pp[k] % d.n_out, w_dp);
            bw.flush();
            si.bits_dpatch += d.n_pp[i] * w_dp;
        }
        h.total_bytes = out.size();
        std::memcpy(out.data(), &h, sizeof h);
        uint8_t *res = (uint8_t *)std::malloc(out.size());
        if (!res) return SQNN_E_NOMEM;
        std::memcpy(res, out.data(), out.size());
        *stored = res;
        *stored_bytes = out.size();
        si.total_bytes = out.size();
        si.bpw = (double)(si.bits_wc + si.bits_widths + si.bits_npatch + si.bits_dpatch) / (double)(d.m * d.n);
        if (info) *info = si;
        return SQNN_OK;
    } catch (const std::bad_alloc &) {
        return SQNN_E_NOMEM;
    }
}

int sqnn_load_host(const void *stored, size_t stored_bytes, void **blob, size_t *blob_bytes)
{
    if (!stored || !blob || !blob_bytes) return SQNN_E_INVALID_ARG;
    if (stored_bytes < sizeof(StoreHeader)) return SQNN_E_BAD_BLOB;
    const uint8_t *b = (const uint8_t *)stored, *end = b + stored_bytes;
    StoreHeader h;
    std::memcpy(&h, b, sizeof h);
    if (std::memcmp(h.magic, STORE_MAGIC, 8) != 0 || h.total_bytes != stored_bytes) return SQNN_E_BAD_BLOB;
    if (h.n_out < 1 || h.n_out > SQNN_MAX_N_OUT || h.n_in < 1 || h.n_in > SQNN_MAX_N_IN || h.n_q < 1 ||
        h.n_q > SQNN_MAX_PLANES || h.m == 0 || h.n == 0 || h.m > ((uint64_t)1 << 40) / h.n || h.block_slices == 0)
        return SQNN_E_BAD_BLOB;
    try {
        const uint64_t mn = h.m * h.n, l = (mn + h.n_out - 1) / h.n_out;
        const uint32_t w_dp = ceil_lg_u64(h.n_out);
        const uint8_t *p = b + sizeof h;
        if ((uint64_t)(end - p) < (uint64_t)h.n_out * 4) return SQNN_E_BAD_BLOB;
        std::vector<uint32_t> rows(h.n_out);
        std::memcpy(rows.data(), p, (size_t)h.n_out * 4);
        p += (size_t)h.n_out * 4;
        std::vector<PlaneArrays> pa(h.n_q);
        std::vector<std::vector<uint16_t>> dp16(h.n_q);
        for (uint32_t i = 0; i < h.n_q; ++i) {
            if (h.n_dp[i] > 0xffffffffull) return SQNN_E_BAD_BLOB;
            // nothing is allocated for more slices than the rest of the buffer could hold seeds for
            if (l > (uint64_t)(end - p) * 8 / h.n_in) return SQNN_E_BAD_BLOB;
            BitReader br(p, end);
            pa[i].wc.resize(l);
            pa[i].np.resize(l);
            for (uint64_t s = 0; s < l; ++s) pa[i].wc[s] = br.get(h.n_in);
            if (!br.ok) return SQNN_E_BAD_BLOB;
            br.align();
            const uint64_t blocks = (l + h.block_slices - 1) / h.block_slices;
            if ((uint64_t)(end - br.p) < blocks) return SQNN_E_BAD_BLOB;
            const uint8_t *widths = br.p;
            br.p += blocks;
            uint64_t sum = 0;
            for (uint64_t s = 0; s < l; ++s) {
                const uint32_t w = widths[s / h.block_slices];
                if (w > 9) return SQNN_E_BAD_BLOB;
                const uint32_t v = br.get(w);
                if (v > h.n_out) return SQNN_E_BAD_BLOB;
                pa[i].np[s] = (uint16_t)v;
                sum += v;
            }
            if (!br.ok || sum != h.n_dp[i]) return SQNN_E_BAD_BLOB;
            br.align();
            if (w_dp && sum > (uint64_t)(end - br.p) * 8 / w_dp) return SQNN_E_BAD_BLOB;
            dp16[i].resize(sum ? sum : 1);
            for (uint64_t k = 0; k < sum; ++k) dp16[i][k] = (uint16_t)br.get(w_dp);
            if (!br.ok) return SQNN_E_BAD_BLOB;
            br.align();
            p = br.p;
        }
        if (p != end) return SQNN_E_BAD_BLOB;
        sqnn_xornet net{h.n_out, h.n_in, rows.data()};
        if (h.n_in < 32)
            for (uint32_t j = 0; j < h.n_out; ++j)
                if (rows[j] >> h.n_in) return SQNN_E_BAD_BLOB;
        std::vector<const uint32_t *> wcp(h.n_q);
        std::vector<const uint16_t *> npp(h.n_q), dpp(h.n_q);
        for (uint32_t i = 0; i < h.n_q; ++i) { wcp[i] = pa[i].wc.data(); npp[i] = pa[i].np.data(); dpp[i] = dp16[i].data(); }
        const int rc = build_blob(&net, h.m, h.n, h.n_q, wcp.data(), npp.data(), nullptr, dpp.data(), blob, blob_bytes);
        return rc == SQNN_E_INVALID_ARG ? SQNN_E_BAD_BLOB : rc;     // bad contents, not a bad call
    } catch (const std::bad_alloc &) {
        return SQNN_E_NOMEM;
    }
}

int sqnn_fifo_model_host(const uint16_t *np, uint64_t l, uint32_t n_fifo, uint32_t rate, uint32_t depth,
                         sqnn_fifo_result *result)
{
    if (!result || (!np && l) || n_fifo == 0 || rate == 0 || depth == 0) return SQNN_E_INVALID_ARG;
    std::memset(result, 0, sizeof *result);
    uint64_t left = 0;                                   // entries the stream has not delivered yet
    for (uint64_t s = 0; s < l; ++s) left += np[s];
    uint64_t held = 0;                                   // entries in the FIFO
    for (uint64_t s = 0; s < l; ++s) {
        uint64_t due = np[s];
        for (;;) {                                       // one pass = one cycle spent on slice s
            ++result->cycles;
            uint64_t in = std::min<uint64_t>(rate, left);
            if (in > depth - held) { in = depth - held; ++result->stall_full; }
            held += in;
            left -= in;
            result->peak = std::max(result->peak, held);
            const uint64_t out = std::min(std::min<uint64_t>(due, n_fifo), held);
            held -= out;
            due -= out;
            if (due == 0) break;
            if (out == n_fifo) ++result->stall_bandwidth; else ++result->stall_empty;
        }
    }
    return SQNN_OK;
}

}  // extern "C"
