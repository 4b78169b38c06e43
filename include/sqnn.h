/*
 * sqnn.h -- C interface of the B200 (sm_100a) library that decodes XOR-gate-network
 * encrypted weight bit-planes and multiplies the decoded sparse quantized weights with
 * activations ("Structured Compression by Weight Encryption for Unstructured Pruning and
 * Quantization", Kwon et al.).
 *
 * Notation (the paper's): a layer has m x n weights, pruned by a mask and quantized to n_q
 * binary-code bit-planes W^q_i (Section 3.1).  Each plane is flattened row-major (flat
 * position p = r*n + c) and cut into l = ceil(mn / n_out) slices of n_out positions
 * (Section 3.1; l in Section 3.2).  A slice w^q is stored as its encrypted seed w^c of n_in
 * bits; the fixed network M (n_out x n_in over GF(2)) expands it: w~ = M . w^c.  Care bits
 * the network could not produce are listed as n_patch (count, same width for every slice of
 * a plane) and d_patch (positions inside the slice) and are flipped after the expansion
 * (Section 3.2).  Positions past mn in the last slice are don't-cares.
 *
 * Two byte layouts carry the same three parts (w^c, n_patch, d_patch).  The *device blob* is what
 * the kernels read: the seed stream, the network's lookup tables, and the patches regrouped per
 * tile of 256 slices as 16-bit bit positions inside the tile (position = slice-in-tile * n_out +
 * d_patch), so that the decoder needs no n_patch stream and no prefix sum to find a slice's
 * patches.  The *storage form* (sqnn_store_host / sqnn_load_host) is the compact layout of
 * Section 3.2 for files: n_patch fields whose width is chosen per block of slices (Section 5.2)
 * and d_patch entries of ceil(lg n_out) bits.  sqnn_unpack_host returns the same logical arrays
 * from a device blob whichever way it was made.
 *
 * General rules
 *  - Plain C.  Every function returns an int status (SQNN_OK = 0, negative = error) unless
 *    noted; nothing aborts, throws or prints.
 *  - "host" pointers are ordinary process memory, "device" pointers are CUDA global memory
 *    of the current device.  All pointers are borrowed for the call; device pointers must
 *    stay valid until the work queued on the stream has run.
 *  - Device entry points only queue work on the given CUDA stream (a cudaStream_t passed as
 *    void*, NULL = the legacy default stream) and do not synchronise.  They allocate no
 *    device memory and create no streams.
 *  - Host buffers the library returns (blob, unpacked arrays) are released with sqnn_free.
 *  - d_status (device, one uint32, may be NULL) receives a sticky non-zero code when a
 *    kernel had to skip a malformed patch entry (1: position outside its tile, 2: a tile's
 *    offsets point past the end of the patch section) or gave up a bounded wait
 *    (6 = -SQNN_E_TIMEOUT); the caller zeroes it.  Kernels never trap.
 *  - Checked mode: with the environment variable SQNN_DEBUG_CHECKS=1 (read once, at the first
 *    device call) every device entry point, after queueing its work, waits for the stream,
 *    and returns SQNN_E_CUDA if a CUDA error surfaced, SQNN_E_TIMEOUT if *d_status is 6 and
 *    SQNN_E_BAD_BLOB if it is any other non-zero code, instead of SQNN_OK.  Meant for
 *    debugging; it serialises the stream.
 *  - Every device entry point is an NVTX range named after the function (domain "sqnn"), visible
 *    in profiler timelines; without a profiler attached the ranges cost nothing measurable.
 */
#ifndef SQNN_H_
#define SQNN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SQNN_MAX_PLANES   8      /* n_q <= 8                                            */
#define SQNN_MAX_N_OUT    256    /* n_out <= 256: a d_patch position fits one byte      */
#define SQNN_MAX_N_IN     32     /* n_in <= 32: a seed fits one uint32                  */
#define SQNN_TILE_SLICES  256    /* patches are indexed per tile of 256 slices          */
#define SQNN_PAD_SLICES   1024   /* streams are zero-padded to a multiple of 1024 slices*/
#define SQNN_MAX_BATCH    1024
#define SQNN_PATCH_HIST_BINS 16  /* n_patch = 0 .. 14, last bin: 15 and more            */
#define SQNN_STATIC_SCRATCH_BYTES (8u << 20)   /* built-in scratch of sqnn_decode_matmul_static */

enum {
    SQNN_OK            =  0,
    SQNN_E_INVALID_ARG = -1,   /* NULL where data is required, size / range out of bounds */
    SQNN_E_BAD_BLOB    = -2,   /* blob fails validation                                   */
    SQNN_E_UNSUPPORTED = -3,   /* valid request the library has no path for               */
    SQNN_E_NOMEM       = -4,   /* host allocation failed                                  */
    SQNN_E_CUDA        = -5,   /* a CUDA runtime call failed (launch configuration, ...)  */
    SQNN_E_TIMEOUT     = -6,   /* a bounded device-side wait gave up (status word only)   */
    SQNN_E_WORKSPACE   = -7    /* workspace missing or smaller than sqnn_workspace_bytes  */
};

/* encode flags */
#define SQNN_ENCODE_ALG1        0u   /* Algorithm 1 (patch searching), the default           */
#define SQNN_ENCODE_EXHAUSTIVE  1u   /* all 2^n_in seeds, fewest patches (Section 5.2); n_in <= 20 */

/* activation element types of sqnn_decode_matmul */
#define SQNN_X_F32   0
#define SQNN_X_BF16  1

/* The XOR-gate network M (Section 3.1): rows[j] bit t = M[j][t], j < n_out, t < n_in. host */
typedef struct sqnn_xornet {
    uint32_t n_out, n_in;
    const uint32_t *rows;
} sqnn_xornet;

/* Quantized, pruned layer as packed bits (host).  Bit p of a vector = (word[p >> 6] >> (p & 63)) & 1.
 * planes: n_q consecutive vectors of ceil(mn / 64) words, bit 1 <-> +1.  mask: 1 = care (unpruned). */
typedef struct sqnn_planes {
    uint64_t m, n;
    uint32_t n_q;
    const uint64_t *planes;
    const uint64_t *mask;
} sqnn_planes;

/* Size accounting.  bpw_eq1 = sum over planes of 1 / r with r from Eq. 1 taken literally
 * (ceil(lg max p) bits per n_patch, ceil(lg n_out) bits per d_patch entry).  bpw_actual counts
 * the bytes of the device blob's sections as stored (padding included; header and the rows of M
 * excluded), per weight: bits_wc the seed streams, bits_dpatch the 16-bit patch positions,
 * bits_index the per-tile patch offsets plus the lookup tables (bits_tables of it), bits_npatch 0
 * (the device blob has no n_patch stream; counts follow from the positions).  The pruning mask
 * (1 bit / weight, kept outside the blob) is not part of either.  patch_hist[k] = number of
 * slices (all planes) with n_patch = k, the last bin collecting 15 and more (Section 5.2 looks
 * at this distribution). */
typedef struct sqnn_stats {
    uint64_t slices;                          /* l per plane                              */
    uint64_t patches[SQNN_MAX_PLANES];        /* sum of n_patch per plane                 */
    uint32_t max_patch[SQNN_MAX_PLANES];      /* max n_patch per plane                    */
    uint64_t bits_wc, bits_npatch, bits_dpatch, bits_index;   /* stored sizes, all planes */
    uint64_t bits_tables;                     /* part of bits_index                       */
    uint64_t patch_hist[SQNN_PATCH_HIST_BINS];
    double   bpw_eq1, bpw_actual;
} sqnn_stats;

/* Parsed header of a device blob.  Offsets are bytes from the start of the blob, each a multiple
 * of 16.  Tables: the lookup tables of the network -- the seed is cut into tab_chunks chunks of
 * tab_chunk_bits bits, entry (chunk, value) = XOR of the columns of M the value selects, as
 * tab_entry_words 32-bit words (bits >= n_out zero) at word ((chunk << tab_chunk_bits) | value) *
 * tab_entry_words; the geometry is a fixed function of (n_out, n_in).  Per plane i: the w^c
 * stream (slice s occupies bits [s*n_in, (s+1)*n_in), least significant bit first inside
 * little-endian 32-bit words); the tile index (uint32 per tile of 256 slices: number of patch
 * entries before the tile, plus one closing entry = n_pp[i]); the patch entries (uint16 each:
 * bit position inside the tile, ascending inside a tile).  Streams cover slices_padded slices
 * (padding slices have seed 0 and no patch) and every section ends with >= 16 zero bytes. */
typedef struct sqnn_desc {
    uint64_t m, n, slices, slices_padded;
    uint32_t n_q, n_out, n_in, tile_slices;
    uint32_t tab_chunks, tab_chunk_bits, tab_entry_words, reserved;
    uint64_t off_xornet;                      /* n_out uint32 rows                        */
    uint64_t off_tables, tables_bytes;
    uint64_t off_wc[SQNN_MAX_PLANES], off_idx[SQNN_MAX_PLANES], off_pp[SQNN_MAX_PLANES];
    uint64_t n_pp[SQNN_MAX_PLANES];           /* patch entries per plane = sum of n_patch */
    uint64_t total_bytes;
} sqnn_desc;

/* Encryption of every slice of every plane (Section 3.1, Algorithm 1 of Section 3.3; with
 * SQNN_ENCODE_EXHAUSTIVE the search of Section 5.2) and packing into one blob.  Host only.
 * Readings fixed here: care positions are tried in ascending order; the kept system is solved
 * with all free variables 0 (pivot columns of the reduced row-echelon form, lowest column
 * first), a slice without care bits gets seed 0; d_patch lists the care positions whose
 * expanded bit is wrong.  *blob is allocated by the library (sqnn_free).  stats may be NULL.
 * Errors: INVALID_ARG (NULL, n_out/n_in/n_q out of range, m*n = 0), NOMEM. */
int sqnn_encode_host(const sqnn_xornet *net, const sqnn_planes *layer, uint32_t flags,
                     void **blob, size_t *blob_bytes, sqnn_stats *stats);

/* As sqnn_encode_host, but the seeds are given: wc[i][s] is the seed of slice s of plane i (for
 * instance from sqnn_search_seeds).  n_patch and d_patch follow by expanding each seed and
 * comparing on the care bits (Algorithm 1, its last three steps).  Any seed gives a lossless blob;
 * better seeds give fewer patches.  Errors: INVALID_ARG (also a seed >= 2^n_in), NOMEM. */
int sqnn_encode_seeds_host(const sqnn_xornet *net, const sqnn_planes *layer, const uint32_t *const *wc,
                           void **blob, size_t *blob_bytes, sqnn_stats *stats);

/* Algorithm 1 (Section 3.3) on one flattened plane for networks the device format does not take:
 * up to 64 inputs and up to 4096 outputs (the sweeps of Section 3.3 run n_in up to 60 with the best
 * n_out in the hundreds).  Host only; no blob is built.  rows[j] bit t = M[j][t] (64-bit rows);
 * plane / mask: packed bits of mn positions as in sqnn_planes.  Outputs, allocated by the library
 * (sqnn_free): wc[l] seeds, np[l] patch counts, dp[*n_dp] positions in slice order, ascending inside
 * a slice, l = ceil(mn / n_out); *bpw_eq1 (may be NULL) = Eq. 1's bits per weight, taken literally.
 * Same readings as sqnn_encode_host.  Errors: INVALID_ARG, NOMEM. */
int sqnn_encode_wide_host(uint32_t n_out, uint32_t n_in, const uint64_t *rows, uint64_t mn,
                          const uint64_t *plane, const uint64_t *mask,
                          uint64_t **wc, uint16_t **np, uint16_t **dp, uint64_t *n_dp, double *bpw_eq1);

/* Packs logical per-plane arrays (the three parts of the format, Section 3.2) into a blob:
 * wc[i][s] seed of slice s (bit t = w^c[t]), np[i][s] = n_patch, dp[i] = all d_patch entries of
 * plane i in slice order.  Arrays are host, length l, l and sum(np[i]).  Errors: INVALID_ARG
 * (also for a seed >= 2^n_in or a position >= n_out), NOMEM. */
int sqnn_pack_host(const sqnn_xornet *net, uint64_t m, uint64_t n, uint32_t n_q,
                   const uint32_t *const *wc, const uint16_t *const *np, const uint16_t *const *dp,
                   void **blob, size_t *blob_bytes);

/* Inverse of sqnn_pack_host for one plane.  wc / np get l entries, dp gets *n_dp entries; each
 * array is allocated by the library (sqnn_free).  Validates the blob first (BAD_BLOB). */
int sqnn_unpack_host(const void *blob, size_t blob_bytes, uint32_t plane,
                     uint32_t **wc, uint16_t **np, uint16_t **dp, uint64_t *n_dp);

/* Validates a host blob and fills *desc: magic / version, section bounds and alignment, the table
 * geometry and the tables themselves (recomputed from the rows of M), tile offsets non-decreasing
 * and closing at n_pp, every patch position inside its tile and not past the last real slice,
 * positions strictly ascending inside a tile, padding slices empty.  BAD_BLOB on any violation. */
int sqnn_describe_host(const void *blob, size_t blob_bytes, sqnn_desc *desc);

/* Size accounting of a host blob (Eq. 1, Section 3.2, and stored bytes). */
int sqnn_stats_host(const void *blob, size_t blob_bytes, sqnn_stats *stats);

/* Blocked n_patch assignment (Section 5.2): what Eq. 1 gives when the n_patch field width is
 * chosen per block of `block_slices` consecutive slices (from that block's own largest count)
 * instead of once per plane, Eq. 1 taken literally (sqnn_store_host builds the format itself).
 * *bits_npatch = sum over planes and blocks of (slices in the block) * ceil(lg max p of the block),
 * *bpw_eq1 = Eq. 1's bits per weight with that middle term (the block widths themselves, which the
 * paper does not count, are not counted).  Either output may be NULL.  Errors: INVALID_ARG
 * (block_slices = 0), BAD_BLOB. */
int sqnn_stats_blocked_host(const void *blob, size_t blob_bytes, uint64_t block_slices,
                            double *bpw_eq1, uint64_t *bits_npatch);

/* Sizes of a storage-form buffer (sqnn_store_host): bits of the seed streams, of the per-block width
 * bytes, of the n_patch fields and of the d_patch entries over all planes, the whole buffer in
 * bytes (header, rows of M and byte padding of each stream included) and bits per weight of the
 * four streams together. */
typedef struct sqnn_store_info {
    uint64_t bits_wc, bits_widths, bits_npatch, bits_dpatch;
    uint64_t total_bytes;
    double bpw;
} sqnn_store_info;

/* Storage form of a layer: the three parts of Section 3.2 packed for files, with the blocked n_patch
 * assignment of Section 5.2 made real.  Per plane: the w^c stream (n_in bits per slice, l slices, no
 * padding slices); one width byte per block of `block_slices` consecutive slices, w = ceil(lg(max
 * n_patch of the block + 1)) -- the narrowest field that can hold every count of the block, 0 for a
 * block without patches (Eq. 1 writes ceil(lg max p), which cannot hold the value max p when it is a
 * power of two; sqnn_stats_blocked_host reports that literal figure); the n_patch fields, w bits each,
 * block after block; the d_patch entries, ceil(lg n_out) bits each, slice order.  How a block's width
 * reaches the decoder is not stated in the paper; the width bytes are this library's answer and are
 * counted.  blob: a device blob (validated first).  *stored is allocated by the library (sqnn_free).
 * info may be NULL.  Errors: INVALID_ARG (NULL, block_slices = 0), BAD_BLOB, NOMEM. */
int sqnn_store_host(const void *blob, size_t blob_bytes, uint64_t block_slices,
                    void **stored, size_t *stored_bytes, sqnn_store_info *info);

/* Inverse of sqnn_store_host: validates a storage-form buffer (magic, sizes, every count <= n_out and
 * within its block's width, every position < n_out and ascending inside a slice) and rebuilds the
 * device blob, byte for byte the one sqnn_store_host was given.  *blob is allocated by the library
 * (sqnn_free).  Errors: INVALID_ARG, BAD_BLOB, NOMEM. */
int sqnn_load_host(const void *stored, size_t stored_bytes, void **blob, size_t *blob_bytes);

/* Result of sqnn_fifo_model_host. */
typedef struct sqnn_fifo_result {
    uint64_t cycles;            /* cycles to pass all slices; relative execution time = cycles / l */
    uint64_t stall_bandwidth;   /* cycles a slice was held because more than n_fifo entries were due */
    uint64_t stall_empty;       /* cycles a slice was held because the FIFO had run dry              */
    uint64_t stall_full;        /* cycles the d_patch stream waited on a full FIFO                   */
    uint64_t peak;              /* largest occupancy reached                                          */
} sqnn_fifo_result;

/* Cycle model of the patch-data FIFO that Section 5.1 puts beside each XOR-gate network, run over
 * the n_patch counts of one plane (np[l], host): the network passes one slice per cycle unless it
 * has to wait for patch data; d_patch arrives as a stream of `rate` entries per cycle into a FIFO
 * of `depth` entries (the stream waits while it is full; it writes before the patch logic reads in
 * the same cycle); the FIFO's n_fifo banks hand over at most n_fifo entries per cycle, and a slice
 * leaves in the cycle its last entry is handed over.  The section gives no equations; these are
 * the readings taken.  Errors: INVALID_ARG (NULL, or a zero parameter). */
int sqnn_fifo_model_host(const uint16_t *np, uint64_t l, uint32_t n_fifo, uint32_t rate, uint32_t depth,
                         sqnn_fifo_result *result);

/* Releases memory returned by the functions above.  NULL is allowed. */
void sqnn_free(void *p);

typedef enum sqnn_out_mode {
    SQNN_OUT_BITS = 0,   /* decoded planes as packed bits: n_q vectors of ceil(mn/64) uint64 words,
                            bit layout as sqnn_planes.planes; bits past mn in the last word are 0.
                            All positions are written, don't-care positions included.            */
    SQNN_OUT_BF16 = 1,   /* dense m x n bf16 (row-major): 0 where mask = 0, else the fp32 sum
                            (+-alpha[r][0]) + (+-alpha[r][1]) + ... in plane order, rounded to
                            bf16 nearest-even; bit 1 <-> +alpha.  Needs d_mask and d_alpha.       */
    SQNN_OUT_SINK = 2    /* one uint64: XOR of all words of the BITS output (measures the pure
                            compressed-stream rate; nothing but 8 bytes is written).             */
} sqnn_out_mode;

/* Decryption of a whole layer on the device (Section 3.1: w~ = M . w^c; Section 3.2: flip the
 * d_patch positions).  desc: host, from sqnn_describe_host.  d_blob: device copy of the same
 * blob, 16-byte aligned.  d_mask: device, ceil(mn/64) uint64 (BF16 mode only, else may be NULL).
 * d_alpha: device, m x n_q floats row-major (BF16 mode only).  d_out: device, out_bytes bytes:
 * BITS n_q*ceil(mn/64)*8, BF16 mn*2, SINK 8; 16-byte aligned.  Errors: INVALID_ARG (NULL,
 * misaligned, out_bytes too small), UNSUPPORTED, CUDA. */
int sqnn_decode(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
                const float *d_alpha, sqnn_out_mode mode, void *d_out, size_t out_bytes,
                uint32_t *d_status, void *cuda_stream);

/* Decryption fused with the product the layer exists for: Y[b][r] = sum_c W[r][c] * X[b][c],
 * W[r][c] = mask[r][c] * sum_i alpha[r][i] * (2 b_i[r][c] - 1) with b_i the decoded planes
 * (Sections 3.1, 3.2; the sparse quantized product of Section 1).  The rescaled weights never
 * reach global memory.  d_x: device, batch rows of n elements (x_dtype SQNN_X_F32 or
 * SQNN_X_BF16), row stride ldx elements.  d_y: device fp32, batch rows of m, row stride ldy;
 * fully overwritten.
 *  - batch <= 15: one kernel; every block decodes the slices that cover its own rows into shared
 *    memory and accumulates in fp32 on the plain ALUs (weights exact).  Each Y[b][r] is summed in
 *    a fixed order, so results are bit-identical from run to run.  No workspace is used.  A row
 *    must fit shared memory as bits: n * (n_q + 1) <= 1 400 000, else UNSUPPORTED.
 *  - batch >= 16: two kernels.  The decode kernel writes the planes as packed bits (1 bit per
 *    weight and plane) into d_workspace; the tcgen05 kernel reads boxes of them, expands them to
 *    bf16 tiles in shared memory and multiplies with fp32 accumulation in tensor memory.
 *    Activations must be BF16 with a 16-byte aligned base and a row pitch that is a multiple of
 *    16 bytes.  d_workspace: device scratch of at least sqnn_workspace_bytes(desc, batch) bytes,
 *    256-byte aligned, contents undefined before and after; required.  Column ranges handled by
 *    different blocks are combined with fp32 atomics on Y, so results can differ from run to run
 *    in the last bits (well inside the 1e-2 tolerance of this path).
 * Errors: INVALID_ARG, UNSUPPORTED (F32 activations with batch >= 16, unaligned activations with
 * batch >= 16, batch > SQNN_MAX_BATCH, rows too long for batch <= 15), WORKSPACE (batch >= 16 and
 * the workspace is missing, too small or misaligned), CUDA. */
int sqnn_decode_matmul(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
                       const float *d_alpha, const void *d_x, int x_dtype, uint32_t batch,
                       int64_t ldx, float *d_y, int64_t ldy, void *d_workspace,
                       size_t workspace_bytes, uint32_t *d_status, void *cuda_stream);

/* The tensor-core product (batch >= 16, BF16 activations) of sqnn_decode_matmul for callers that
 * can neither allocate device memory nor hand over a workspace: code running under a stream
 * capture, plug-ins inside a framework that owns the device heap, serving loops with a frozen
 * memory plan.  (The paper has no counterpart; this is a packaging variant of the call above.)
 * Arguments and results as for sqnn_decode_matmul, minus the workspace: the decoded planes
 * (packed bits) go to an array of SQNN_STATIC_SCRATCH_BYTES bytes built into the library, which
 * every GPU that loads the library holds until the process exits.  The call itself makes no
 * cudaMalloc / cudaFree and calls no allocating routine.
 *  - Size limit: sqnn_workspace_bytes(desc, batch) must not exceed SQNN_STATIC_SCRATCH_BYTES
 *    (8 MiB: about 67 million weight bits over all planes); larger layers get SQNN_E_WORKSPACE.
 *  - batch < 16 or F32 activations: SQNN_E_UNSUPPORTED (those paths need no scratch; use
 *    sqnn_decode_matmul).
 *  - The first call on each device looks up the array's device address (with that device
 *    current) and remembers it for the life of the process; make that first call before any
 *    stream capture begins.  After a cudaDeviceReset the remembered address is stale: do not
 *    reset a device this entry point has been used on.
 *  - All calls share the one array and it keeps whatever the last call left.  Nothing in it needs
 *    clearing (each call overwrites all it reads), but two calls whose kernels may run at the
 *    same time on one GPU -- different streams, or different threads -- race on it: serialise them.
 * Errors otherwise as sqnn_decode_matmul. */
int sqnn_decode_matmul_static(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
                              const float *d_alpha, const void *d_x, int x_dtype, uint32_t batch,
                              int64_t ldx, float *d_y, int64_t ldy, uint32_t *d_status,
                              void *cuda_stream);

/* Exhaustive seed search on the device (Section 5.2, "minimizing n_patch for small n_in"): for every
 * slice of every plane all 2^n_in seeds are expanded and the one with the fewest wrong care bits is
 * kept, the smallest seed among equals.  net: host.  d_planes / d_mask: device, packed as in
 * sqnn_planes.  d_wc / d_np: device outputs, n_q * l entries each (plane-major, l = ceil(mn/n_out)):
 * the seed and its number of wrong care bits (= n_patch).  Queues on the stream, allocates nothing.
 * Cost grows as 2^n_in per slice.  Errors: INVALID_ARG, UNSUPPORTED (n_in > 20), CUDA. */
int sqnn_search_seeds(const sqnn_xornet *net, uint64_t m, uint64_t n, uint32_t n_q,
                      const uint64_t *d_planes, const uint64_t *d_mask, uint32_t *d_wc, uint16_t *d_np,
                      void *cuda_stream);

/* Measurement aid (the paper has no counterpart): writes `bytes` bytes (a multiple of 16) to d_out
 * (device, 16-byte aligned) the way the packed-bit decode writes its output -- every warp fills a
 * shared-memory region of chunk_bytes bytes (a multiple of 16, at most 8192) once and sends it out
 * with bulk copies -- but reads no compressed stream and expands nothing.  Its rate is the ceiling
 * the decode kernel's output path allows on this GPU.  Errors: INVALID_ARG, CUDA. */
int sqnn_store_probe(void *d_out, size_t bytes, uint32_t chunk_bytes, void *cuda_stream);

/* For the library's own tests (the paper has no counterpart; not meant for applications).  Bit 0 of
 * `flags` makes the loader role of the tensor-core kernel issue no loads, so that the bounded waits of
 * the roles that consume its data run out: the kernel then reports 6 (= -SQNN_E_TIMEOUT) through
 * d_status, frees its tensor memory and returns; Y is left incomplete.  wait_limit_cycles is the number
 * of SM clock cycles such a wait may take (0 = the default, about two seconds).  Applies to calls made
 * after it, process-wide. */
void sqnn_set_debug_flags(uint32_t flags, uint64_t wait_limit_cycles);

/* Scratch bytes sqnn_decode_matmul needs for this layer and batch (0 for batch <= 15). */
size_t sqnn_workspace_bytes(const sqnn_desc *desc, uint32_t batch);

/* Human-readable name of a status code; never NULL. */
const char *sqnn_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* SQNN_H_ */
