// Geometry of the device blob that the host packer and the kernels must agree on: how the
// XOR-gate network's lookup tables are cut into chunks and how slices are grouped into tiles.
// Plain functions, usable from host C++ and from device code.
#ifndef SQNN_LAYOUT_H_
#define SQNN_LAYOUT_H_
#include <stdint.h>

#if defined(__CUDACC__)
#define SQNN_HD __host__ __device__
#else
#define SQNN_HD
#endif

namespace sqnn {

// The network (Section 3.1, w~ = M . w^c) is evaluated with tables: the seed is cut into chunks
// of cb bits and table[chunk][value] holds the XOR of the columns of M selected by the value, as
// an n_out-bit word padded to nwp 32-bit words (bits >= n_out are 0).  Entry (chunk, value)
// starts at word ((chunk << cb) | value) * nwp.
SQNN_HD constexpr uint32_t entry_words(uint32_t n_out) { return (n_out + 31) / 32; }
SQNN_HD constexpr uint32_t entry_words_padded(uint32_t n_out)
{
    return entry_words(n_out) <= 1 ? 1 : entry_words(n_out) <= 2 ? 2 : entry_words(n_out) <= 4 ? 4 : 8;
}
// A kernel may keep several copies of the tables in shared memory, copy j holding all its entries
// in the banks that lane j of a load wavefront owns, so that lookups at unrelated indices never
// collide: 32 / nwp lanes share a wavefront for entries of up to 16 bytes (8 lanes for 32-byte
// entries, read as two halves).  One replicated entry therefore takes 128 bytes (256 for 32-byte
// entries).  The chunking is the coarsest whose replicated tables stay within 128 KB, i.e. at
// most 1024 entries (512 of 32 bytes) over all chunks.
SQNN_HD constexpr uint32_t table_copies(uint32_t nwp) { return nwp >= 4 ? 8 : 32 / nwp; }
SQNN_HD constexpr uint32_t table_chunks(uint32_t n_in, uint32_t nwp)
{
    for (uint32_t c = 1; c <= 8; ++c) {
        uint32_t cb = (n_in + c - 1) / c;
        if (cb <= 10 && c * (1u << cb) <= (nwp == 8 ? 512u : 1024u)) return c;
    }
    return 8;
}
SQNN_HD constexpr uint32_t chunk_bits(uint32_t n_in, uint32_t nwp)
{
    return (n_in + table_chunks(n_in, nwp) - 1) / table_chunks(n_in, nwp);
}
// Words of all tables, rounded to a multiple of 4 (16 bytes).
SQNN_HD constexpr uint32_t table_words(uint32_t n_out, uint32_t n_in)
{
    return (table_chunks(n_in, entry_words_padded(n_out)) * (1u << chunk_bits(n_in, entry_words_padded(n_out))) *
            entry_words_padded(n_out) + 3u) & ~3u;
}

// A format tile is SQNN_TILE_SLICES = 256 consecutive slices: 32 * n_in bytes of seeds, 32 * n_out
// bytes of output, so every tile starts on a 32-byte boundary in both.  Kernels work on kernel
// tiles of 32 lanes x G slices with G * n_out a multiple of 32 bits: G = 8 * kt format tiles,
// kt = 1 when n_out is a multiple of 4, 2 when it is even, 4 otherwise.
SQNN_HD constexpr uint32_t format_tiles_per_kernel_tile(uint32_t n_out)
{
    return (n_out % 4 == 0) ? 1u : (n_out % 2 == 0) ? 2u : 4u;
}

// Words of the replicated tables in shared memory.
SQNN_HD constexpr uint32_t table_words_replicated(uint32_t n_out, uint32_t n_in)
{
    return table_chunks(n_in, entry_words_padded(n_out)) * (1u << chunk_bits(n_in, entry_words_padded(n_out))) *
           entry_words_padded(n_out) * table_copies(entry_words_padded(n_out));
}

}  // namespace sqnn
#endif
