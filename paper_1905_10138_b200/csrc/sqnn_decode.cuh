// Device-side decryption of one warp tile: seeds -> XOR-gate network (table lookup) ->
// patch flips, producing a run of consecutive output words in shared memory.
//
// Work split.  A lane owns G consecutive slices, G = 8 * KT with KT the number of format tiles
// (256 slices) per kernel tile, chosen so that G * n_out is a multiple of 32 bits; its
// W = G * n_out / 32 output words are private to it while it expands.  A kernel tile is therefore
// 32 * G consecutive slices = 32 * W consecutive 32-bit words of the flattened plane.  In the
// seed stream a lane's 8 slices of one format tile are n_in consecutive bytes.
//
// The network (Section 3.1, w~ = M . w^c) is evaluated with the lookup tables stored in the
// blob (geometry in sqnn_layout.h), copied to shared memory once per block.
//
// Patches (Section 3.2) come per format tile as 16-bit bit positions inside the tile; the warp
// flips them in the shared-memory copy of the tile with one shared-memory reduction each, lanes
// taking entries in turn -- no counts, no prefix sum.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "sqnn.h"
#include "sqnn_layout.h"

#define SQNN_DEV __device__ __forceinline__

namespace sqnn {

struct PlanePtrs {
    const uint32_t *wc;    // seed stream
    const uint32_t *idx;   // patch entries before each format tile (+ closing entry)
    const uint16_t *pp;    // patch entries: bit position inside the format tile
    uint32_t n_pp;
};

struct DecodeArgs {
    uint64_t mn;           // weights per plane
    uint64_t words64;      // ceil(mn / 64)
    uint64_t ktiles;       // kernel tiles per plane (padded stream)
    uint32_t n_out, n_in, n_q;
    uint32_t KT, G, W;     // format tiles per kernel tile, slices and words per lane
    uint32_t nw, nwp;      // words per table entry: used, padded (1, 2, 4, 8)
    uint32_t nchunks, cb;  // table chunks, bits per chunk
    uint32_t tab_words;    // words of all tables (multiple of 4)
    const uint32_t *tab;   // tables in the blob
    uint32_t *status;      // sticky error word or NULL
    PlanePtrs pl[8];
};

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

SQNN_DEV void cp_async16(void *sdst, const void *gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" :: "r"(smem_addr(sdst)), "l"(gsrc) : "memory");
}
SQNN_DEV void cp_async4(void *sdst, const void *gsrc)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" :: "r"(smem_addr(sdst)), "l"(gsrc) : "memory");
}
SQNN_DEV void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int PENDING>
SQNN_DEV void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;\n" :: "n"(PENDING) : "memory"); }
SQNN_DEV void cp_async_wait_all() { asm volatile("cp.async.wait_all;\n" ::: "memory"); }

// Read-only global loads that stay where they are written: the compiler may not move a volatile asm
// statement past another one, so a load issued ahead of time is not sunk down to its first use.
SQNN_DEV uint32_t ldg_ahead(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
SQNN_DEV uint2 ldg_ahead(const uint2 *p)
{
    uint2 v;
    asm volatile("ld.global.nc.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
SQNN_DEV uint4 ldg_ahead(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Makes the warp wait here for a value loaded earlier (a volatile register move reads it).  Used before
// new loads are issued: the few scoreboards a warp has are shared between loads, so a register whose
// load finished long ago can otherwise end up waiting for loads issued just before its first use.
SQNN_DEV uint32_t settle(uint32_t v)
{
    uint32_t r;
    asm volatile("mov.u32 %0, %1;" : "=r"(r) : "r"(v));
    return r;
}

// Flips one bit of a shared-memory word (address given as a 32-bit shared address).
SQNN_DEV void smem_flip(uint32_t region_sa, uint32_t bit)
{
    asm volatile("red.shared.xor.b32 [%0], %1;\n" :: "r"(region_sa + ((bit >> 5) << 2)), "r"(1u << (bit & 31u)) : "memory");
}

// Starts the copy of the lookup tables from the blob into shared memory (all threads of the
// block; one commit group).  Wait for the group and pass a block barrier before the first lookup.
SQNN_DEV void tables_request(const DecodeArgs &A, uint32_t *tab_s)
{
    for (uint32_t v = threadIdx.x; v < A.tab_words / 4; v += blockDim.x) cp_async16(tab_s + 4 * v, A.tab + 4 * v);
    cp_async_commit();
}

// The same tables, replicated for conflict-free lookups (sqnn_layout.h): element (entry e, copy j)
// -- for 32-byte entries (entry e, half h, copy j) -- is stored at consecutive 16-byte (or smaller)
// slots in the order of its linear index, so the fill is a coalesced copy in which 32 / NWP
// consecutive threads store the same entry.  All threads of the block; ends without a barrier.
template <int NWP>
SQNN_DEV void tables_replicate(const DecodeArgs &A, uint32_t *tab_s)
{
    constexpr uint32_t R = table_copies(NWP);
    constexpr uint32_t VW = NWP >= 4 ? 4 : NWP;                  // words per stored element (16, 8 or 4 bytes)
    constexpr uint32_t PER = 32 / R;                             // source elements one warp store covers
    const uint32_t elems = (A.nchunks << A.cb) * (NWP / VW);     // source elements (halves count separately)
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    // a warp takes 32 source elements at a time: one coalesced load, then R stores of 32 consecutive
    // replicated elements each, the values handed round by shuffles
    for (uint32_t e0 = warp * 32; e0 < elems; e0 += nwarps * 32) {
        uint32_t v[VW];
#pragma unroll
        for (uint32_t k = 0; k < VW; ++k) v[k] = 0;
        if (e0 + lane < elems) {
            if constexpr (VW == 4) {
                const uint4 t = __ldg(reinterpret_cast<const uint4 *>(A.tab + 4 * (e0 + lane)));
                v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
            } else if constexpr (VW == 2) {
                const uint2 t = __ldg(reinterpret_cast<const uint2 *>(A.tab + 2 * (e0 + lane)));
                v[0] = t.x; v[1] = t.y;
            } else {
                v[0] = __ldg(A.tab + e0 + lane);
            }
        }
#pragma unroll
        for (uint32_t j = 0; j < R; ++j) {
            const uint32_t src = j * PER + lane / R;             // source element (within the 32) of this lane's store
            uint32_t o[VW];
#pragma unroll
            for (uint32_t k = 0; k < VW; ++k) o[k] = __shfl_sync(0xffffffffu, v[k], src);
            const uint32_t i = (e0 + j * PER) * R + lane;        // replicated element index
            if (e0 + src < elems) {
                if constexpr (VW == 4) *reinterpret_cast<uint4 *>(tab_s + 4 * i) = make_uint4(o[0], o[1], o[2], o[3]);
                else if constexpr (VW == 2) *reinterpret_cast<uint2 *>(tab_s + 2 * i) = make_uint2(o[0], o[1]);
                else tab_s[i] = o[0];
            }
        }
    }
}

// Entry e of the tables in shared memory.  REP: from the replicated tables, through the copy of this lane.
template <int NWP, bool REP>
SQNN_DEV void load_entry(const uint32_t *tab, uint32_t e, uint32_t lane, uint32_t (&x)[NWP])
{
    constexpr uint32_t R = table_copies(NWP);
    if constexpr (NWP == 1) {
        x[0] = REP ? tab[e * R + lane] : tab[e];
    } else if constexpr (NWP == 2) {
        const uint2 v = *reinterpret_cast<const uint2 *>(tab + 2 * (REP ? e * R + (lane & (R - 1)) : e));
        x[0] = v.x; x[1] = v.y;
    } else if constexpr (NWP == 4) {
        const uint4 v = *reinterpret_cast<const uint4 *>(tab + 4 * (REP ? e * R + (lane & (R - 1)) : e));
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    } else {
        const uint32_t i0 = REP ? (2 * e) * R + (lane & (R - 1)) : 2 * e;
        const uint32_t i1 = REP ? (2 * e + 1) * R + (lane & (R - 1)) : 2 * e + 1;
        const uint4 v = *reinterpret_cast<const uint4 *>(tab + 4 * i0);
        const uint4 u = *reinterpret_cast<const uint4 *>(tab + 4 * i1);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
        x[4] = u.x; x[5] = u.y; x[6] = u.z; x[7] = u.w;
    }
}

// Compile-time facts of a network shape (n_out a multiple of 4: one format tile per kernel tile).
template <int N_OUT, int N_IN>
struct Shape {
    static_assert(N_OUT % 4 == 0, "compile-time shapes have n_out a multiple of 4");
    static constexpr uint32_t n_out = N_OUT, n_in = N_IN;
    static constexpr uint32_t G = 8, W = N_OUT / 4;
    static constexpr uint32_t NW = entry_words(N_OUT), NWP = entry_words_padded(N_OUT);
    static constexpr uint32_t NCH = table_chunks(N_IN, NWP), CB = chunk_bits(N_IN, NWP);
    static constexpr uint32_t SPAN = 8 * N_IN;                       // seed bits of one lane
    static constexpr bool ALIGNED = SPAN % 32 == 0;                   // a lane's seeds start on a word
    static constexpr uint32_t NSW = (SPAN + 31) / 32;                 // words holding them
    static constexpr uint32_t NRAW = ALIGNED ? NSW : NSW + 1;
    static constexpr uint32_t TILE_BITS = SQNN_TILE_SLICES * N_OUT;
};

// The words holding a lane's 8 seeds of one tile.
template <int N_OUT, int N_IN>
struct TileSeeds {
    uint32_t raw[Shape<N_OUT, N_IN>::NRAW];
};
// A tile's run of patch entries [base, end) and the first words of it, fetched ahead of time:
// lane l holds 32-bit words (base >> 1) + l + 32 k, k < 4, of the entry array (two entries each).
struct TileRun {
    uint32_t base, end;
};
constexpr uint32_t PATCH_AHEAD = 4;

template <int N_OUT, int N_IN>
SQNN_DEV void fetch_seeds(const PlanePtrs &P, uint64_t tile, uint32_t lane, TileSeeds<N_OUT, N_IN> &s)
{
    using S = Shape<N_OUT, N_IN>;
    const uint32_t *w = P.wc + tile * (8 * S::n_in) + ((lane * S::SPAN) >> 5);
    if constexpr (S::ALIGNED && S::NSW == 4) {
        const uint4 v = ldg_ahead(reinterpret_cast<const uint4 *>(w));
        s.raw[0] = v.x; s.raw[1] = v.y; s.raw[2] = v.z; s.raw[3] = v.w;
    } else if constexpr (S::ALIGNED && S::NSW == 2) {
        const uint2 v = ldg_ahead(reinterpret_cast<const uint2 *>(w));
        s.raw[0] = v.x; s.raw[1] = v.y;
    } else {
#pragma unroll
        for (uint32_t k = 0; k < S::NRAW; ++k) s.raw[k] = ldg_ahead(w + k);     // sections end with slack
    }
}

SQNN_DEV TileRun fetch_run(const PlanePtrs &P, uint64_t tile)
{
    TileRun r;
    r.base = ldg_ahead(P.idx + tile);
    r.end = ldg_ahead(P.idx + tile + 1);
    return r;
}

// Checks the run against the section and requests its first words.
SQNN_DEV void fetch_patches(const DecodeArgs &A, const PlanePtrs &P, TileRun &run, uint32_t lane,
                            uint32_t (&pw)[PATCH_AHEAD])
{
    if (run.end < run.base || run.end > P.n_pp) {                // offsets point outside the section
        flag(A.status, 2u);
        run.end = run.base = 0;
    }
    const uint32_t *pp32 = reinterpret_cast<const uint32_t *>(P.pp);
    const uint32_t w0 = run.base >> 1, wend = (run.end + 1) >> 1;
#pragma unroll
    for (uint32_t k = 0; k < PATCH_AHEAD; ++k) {
        const uint32_t aw = w0 + lane + 32 * k;
        pw[k] = 0u;
        if (aw < wend) pw[k] = ldg_ahead(pp32 + aw);
    }
}

// One patch entry: flips bit bit0 + pos of the region if the entry belongs to the run (t < total,
// t = its index minus the run's base, as unsigned) and pos lies inside the tile.  Branch-free: the
// reduction is predicated.  Returns pos if the entry belongs to the run, else 0 (for the range check).
SQNN_DEV uint32_t flip_entry(uint32_t region_sa, uint32_t bit0, uint32_t tile_bits, uint32_t pos, uint32_t t, uint32_t total)
{
    uint32_t seen;
    asm volatile("{\n .reg .pred p, q;\n .reg .b32 a, v, s, b;\n"
                 " setp.lt.u32 q, %3, %4;\n"                    // the entry belongs to the run
                 " setp.lt.and.u32 p, %2, %5, q;\n"             // ... and its position lies inside the tile
                 " selp.u32 %0, %2, 0, q;\n"
                 " add.u32 b, %2, %6;\n"
                 " shr.u32 a, b, 5;\n shl.b32 a, a, 2;\n add.u32 a, a, %1;\n"
                 " and.b32 s, b, 31;\n shl.b32 v, 1, s;\n"
                 " @p red.shared.xor.b32 [a], v;\n}"
                 : "=r"(seen) : "r"(region_sa), "r"(pos), "r"(t), "r"(total), "r"(tile_bits), "r"(bit0) : "memory");
    return seen;
}

// Flips the patched positions of one format tile (Section 3.2) whose first bit is bit `bit0` of
// the region.  Every lane's words of the tile must be in place (warp barrier before), and the
// region is complete after the warp barrier that follows.  `pw`: words fetched by fetch_patches.
SQNN_DEV void tile_patch(const DecodeArgs &A, const PlanePtrs &P, const TileRun &run, const uint32_t (&pw)[PATCH_AHEAD],
                         uint32_t *region, uint32_t bit0, uint32_t tile_bits, uint32_t lane)
{
    if (run.end == run.base) return;                             // the same in every lane
    const uint32_t region_sa = smem_addr(region);
    const uint32_t total = run.end - run.base;
    const uint32_t w0 = run.base >> 1, wend = (run.end + 1) >> 1;
    // index, relative to the run, of the low entry of this lane's first word: -1 when the run starts
    // in the high half of its first word (the unsigned compare in flip_entry then rejects it)
    const uint32_t t0 = 2 * (w0 + lane) - run.base;
    uint32_t top = 0;                                            // largest position seen
#pragma unroll
    for (uint32_t k = 0; k < PATCH_AHEAD; ++k) {
        top = max(top, flip_entry(region_sa, bit0, tile_bits, pw[k] & 0xffffu, t0 + 64 * k, total));
        top = max(top, flip_entry(region_sa, bit0, tile_bits, pw[k] >> 16, t0 + 64 * k + 1, total));
    }
    // longer runs: eight words (sixteen entries) per lane and round; the words of the next round are
    // requested before this round's are used
    constexpr uint32_t RB = 8;
    const uint32_t *pp32 = reinterpret_cast<const uint32_t *>(P.pp);
    uint32_t a0 = w0 + 32 * PATCH_AHEAD;
    if (a0 < wend) {
        uint32_t cur[RB], nxt[RB];
        auto request = [&](uint32_t at, uint32_t (&w)[RB]) {
#pragma unroll
            for (uint32_t k = 0; k < RB; ++k) {
                const uint32_t aw = at + lane + 32 * k;
                w[k] = 0u;
                if (aw < wend) w[k] = ldg_ahead(pp32 + aw);
            }
        };
        request(a0, cur);
        for (; a0 < wend; a0 += 32 * RB) {
            request(a0 + 32 * RB, nxt);
            const uint32_t t = 2 * (a0 + lane) - run.base;
#pragma unroll
            for (uint32_t k = 0; k < RB; ++k) {
                top = max(top, flip_entry(region_sa, bit0, tile_bits, cur[k] & 0xffffu, t + 64 * k, total));
                top = max(top, flip_entry(region_sa, bit0, tile_bits, cur[k] >> 16, t + 64 * k + 1, total));
            }
#pragma unroll
            for (uint32_t k = 0; k < RB; ++k) cur[k] = nxt[k];
        }
    }
    if (top >= tile_bits) flag(A.status, 1u);
}

// Expands the lane's 8 slices of one tile into region[lane * W .. lane * W + W).  WAIT_BULK: lane 0
// first waits for its pending bulk copy out of `region`, just before the region is overwritten.
// REP: `tab` holds the replicated tables.
template <int N_OUT, int N_IN, bool WAIT_BULK = false, bool REP = false>
SQNN_DEV void tile_expand(const TileSeeds<N_OUT, N_IN> &in, uint32_t *region, const uint32_t *tab, uint32_t lane)
{
    using S = Shape<N_OUT, N_IN>;
    constexpr uint32_t G = S::G, W = S::W, NW = S::NW, NWP = S::NWP, NCH = S::NCH, CB = S::CB;
    constexpr uint32_t n_out = S::n_out, n_in = S::n_in, NSW = S::NSW;
    uint32_t *mine = region + lane * W;

    // seeds -> table entries
    uint32_t al[NSW];
    if constexpr (S::ALIGNED) {
#pragma unroll
        for (uint32_t k = 0; k < NSW; ++k) al[k] = in.raw[k];
    } else {
        const uint32_t sh0 = (lane * S::SPAN) & 31u;
#pragma unroll
        for (uint32_t k = 0; k < NSW; ++k) al[k] = __funnelshift_r(in.raw[k], in.raw[k + 1], sh0);
    }
    uint32_t x[G][NWP];
#pragma unroll
    for (uint32_t i = 0; i < G; ++i) {
        constexpr uint32_t smask = n_in >= 32 ? 0xffffffffu : ((1u << n_in) - 1u);
        const uint32_t o = i * n_in, w = o >> 5, s = o & 31;
        uint32_t seed;
        if (s + n_in <= 32) seed = (al[w] >> s) & smask;
        else seed = __funnelshift_r(al[w], al[w + 1 < NSW ? w + 1 : w], s) & smask;
        load_entry<NWP, REP>(tab, seed & ((1u << CB) - 1u), lane, x[i]);
#pragma unroll
        for (uint32_t ch = 1; ch < NCH; ++ch) {
            uint32_t y[NWP];
            load_entry<NWP, REP>(tab, (ch << CB) | ((seed >> (ch * CB)) & ((1u << CB) - 1u)), lane, y);
#pragma unroll
            for (uint32_t k = 0; k < NW; ++k) x[i][k] ^= y[k];
        }
    }
    // output word k = bits [32k, 32k + 32) of the concatenated entries (entry bits >= n_out are 0)
    uint32_t out[W];
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
        out[k] = word;
    }
    if constexpr (WAIT_BULK) {                       // the bulk copy of the previous tile still reads `region`
        if (lane == 0) bulk_wait_read<0>();
        __syncwarp();
    }
    // the widest stores the lane's base allows (lane stride W words): conflict-free for every W
    if constexpr (W % 4 == 0) {
#pragma unroll
        for (uint32_t k = 0; k < W; k += 4)
            *reinterpret_cast<uint4 *>(mine + k) = make_uint4(out[k], out[k + 1], out[k + 2], out[k + 3]);
    } else if constexpr (W % 2 == 0) {
#pragma unroll
        for (uint32_t k = 0; k < W; k += 2) *reinterpret_cast<uint2 *>(mine + k) = make_uint2(out[k], out[k + 1]);
    } else {
#pragma unroll
        for (uint32_t k = 0; k < W; ++k) mine[k] = out[k];
    }
}

// Run-time shape: plain loops, every read through extract_bits.  Ends with the warp synchronised.
SQNN_DEV void decode_ktile_generic(const DecodeArgs &A, uint32_t plane, uint64_t ktile,
                                   uint32_t *region, const uint32_t *tab, uint32_t lane)
{
    const PlanePtrs &P = A.pl[plane];
    const uint32_t n_out = A.n_out, n_in = A.n_in, G = A.G, W = A.W;
    const uint32_t nw = A.nw, nwp = A.nwp, nch = A.nchunks, cb = A.cb;
    const uint32_t cmask = (1u << cb) - 1u;
    const uint64_t s0 = (ktile * 32 + lane) * G;
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
    __syncwarp();
    // patches (Section 3.2), one format tile after the other
    const uint32_t tile_bits = SQNN_TILE_SLICES * n_out;
    const uint32_t region_sa = smem_addr(region);
    uint32_t bad = 0;
    for (uint32_t f = 0; f < A.KT; ++f) {
        const uint64_t ft = ktile * A.KT + f;
        uint32_t base = __ldg(P.idx + ft), end = __ldg(P.idx + ft + 1);
        if (end < base || end > P.n_pp) { flag(A.status, 2u); continue; }
        for (uint32_t e = base + lane; e < end; e += 32) {
            const uint32_t pos = P.pp[e];
            if (pos < tile_bits) smem_flip(region_sa, f * tile_bits + pos); else bad = 1;
        }
    }
    if (bad) flag(A.status, 1u);
    __syncwarp();
}

// Fetch + expand + patch of one kernel tile without overlap (for the kernels that do more work per
// tile).  `tab`: the tables in shared memory.  Ends with the warp synchronised.
template <int N_OUT, int N_IN>
SQNN_DEV void decode_warp_tile(const DecodeArgs &A, uint32_t plane, uint64_t tile,
                               uint32_t *region, const uint32_t *tab, uint32_t lane)
{
    if constexpr (N_OUT != 0) {
        using S = Shape<N_OUT, N_IN>;
        const PlanePtrs &P = A.pl[plane];
        TileSeeds<N_OUT, N_IN> in;
        uint32_t pw[PATCH_AHEAD];
        fetch_seeds<N_OUT, N_IN>(P, tile, lane, in);
        TileRun run = fetch_run(P, tile);
        fetch_patches(A, P, run, lane, pw);
        tile_expand<N_OUT, N_IN>(in, region, tab, lane);
        __syncwarp();
        tile_patch(A, P, run, pw, region, 0u, S::TILE_BITS, lane);
        __syncwarp();
    } else {
        decode_ktile_generic(A, plane, tile, region, tab, lane);
    }
}

}  // namespace sqnn
