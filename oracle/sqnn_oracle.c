/*
 * CPU oracle for the XOR-gate-network weight representation of
 * "Structured Compression by Weight Encryption for Unstructured Pruning and
 * Quantization" (Kwon et al.).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * method computes.  It is called by the tests, by the smoke check and by the
 * benchmark's CPU-baseline leg, and by nothing else.  It shares no code, header,
 * table or helper with the CUDA library, and neither side includes the other.
 *
 * Style: one byte per bit, one loop per index of the paper's formulas, no bit
 * tricks, no blocking.  Matrices over GF(2) are arrays of 0/1 bytes.
 *
 *   M        : the XOR-gate network, n_out x n_in, row-major (Section 3.1)
 *   w^q      : one slice of n_out weight bits, with a care flag per position
 *   w^c      : the encrypted slice, n_in bits (Section 3.1)
 *   n_patch  : number of care bits the network could not produce (Section 3.2)
 *   d_patch  : their positions inside the slice, ascending (Section 3.2)
 *
 * Parity status: every function below is pinned by tests that do not use this
 * file to produce their expectation (brute force, closed forms, numpy / torch
 * library routines, hand-computed vectors), except where a header says
 * "parity unpinned".  Real-model bits/weight figures of Section 4 need trained
 * weights that are not available: parity unpinned for those (no function here
 * claims them).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Number of threads the parallel loops below will use (1 without OpenMP). */
int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_set_num_threads(int t)
{
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* ------------------------------------------------------------------------- */
/* Decryption, Section 3.1: w~ = M . w^c over GF(2).                          */
/* out[j] = XOR over t of M[j][t] AND wc[t].                                  */
/* ------------------------------------------------------------------------- */
void orc_xor_network(int n_out, int n_in, const uint8_t *M, const uint8_t *wc, uint8_t *out)
{
    for (int j = 0; j < n_out; ++j) {
        int acc = 0;
        for (int t = 0; t < n_in; ++t)
            acc ^= (M[j * n_in + t] & wc[t]);
        out[j] = (uint8_t)acc;
    }
}

/* ------------------------------------------------------------------------- */
/* Reduced row-echelon form over GF(2) of an augmented matrix                  */
/* a[rows][n_in + 1] (last column = right-hand side), in place.               */
/* Textbook Gauss-Jordan: columns left to right, first row at or below the    */
/* current rank that has a 1 becomes the pivot row, every other row with a 1  */
/* in that column gets the pivot row added.  pivot_col[i] receives the pivot  */
/* column of row i for i < rank.  Returns the rank of the coefficient part.   */
/* ------------------------------------------------------------------------- */
static int gauss_jordan_gf2(uint8_t *a, int rows, int n_in, int *pivot_col)
{
    const int w = n_in + 1;
    int rank = 0;
    for (int col = 0; col < n_in && rank < rows; ++col) {
        int pr = -1;
        for (int i = rank; i < rows; ++i)
            if (a[i * w + col]) { pr = i; break; }
        if (pr < 0) continue;
        if (pr != rank) {
            for (int c = 0; c < w; ++c) {
                uint8_t tmp = a[pr * w + c];
                a[pr * w + c] = a[rank * w + c];
                a[rank * w + c] = tmp;
            }
        }
        for (int i = 0; i < rows; ++i) {
            if (i != rank && a[i * w + col])
                for (int c = 0; c < w; ++c)
                    a[i * w + c] ^= a[rank * w + c];
        }
        pivot_col[rank] = col;
        ++rank;
    }
    return rank;
}

/* A reduced system is solvable iff no row reads 0 ... 0 | 1. */
static int is_consistent(const uint8_t *a, int rows, int n_in)
{
    const int w = n_in + 1;
    for (int i = 0; i < rows; ++i) {
        int any = 0;
        for (int c = 0; c < n_in; ++c) any |= a[i * w + c];
        if (!any && a[i * w + n_in]) return 0;
    }
    return 1;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1 (patch searching) on one slice.                                */
/*                                                                            */
/* Care positions are tried in ascending order.  The equation of a care bit   */
/* joins the kept equations; a fresh copy of all kept equations is brought to */
/* reduced row-echelon form; if the system turned inconsistent the equation   */
/* is dropped again (that care bit will be a patch).  After the loop the kept */
/* system is solved with every free variable set to 0 (the reading that makes */
/* w^c unique), the network is evaluated on w^c, and the care positions whose */
/* produced bit differs from the wanted bit form d_patch.                     */
/*                                                                            */
/* wq[j], care[j] in {0,1};  wc gets n_in bits;  dpatch needs room for n_out  */
/* entries.  Returns n_patch, or -1 if memory ran out.                        */
/* ------------------------------------------------------------------------- */
int orc_encode_slice(int n_out, int n_in, const uint8_t *M, const uint8_t *wq,
                     const uint8_t *care, uint8_t *wc, uint16_t *dpatch)
{
    const int w = n_in + 1;
    uint8_t *kept = (uint8_t *)malloc((size_t)(n_out > 0 ? n_out : 1) * w);
    uint8_t *work = (uint8_t *)malloc((size_t)(n_out > 0 ? n_out : 1) * w);
    int *pivot_col = (int *)malloc(sizeof(int) * (size_t)(n_in > 0 ? n_in : 1));
    uint8_t *decoded = (uint8_t *)malloc((size_t)(n_out > 0 ? n_out : 1));
    if (!kept || !work || !pivot_col || !decoded) {
        free(kept); free(work); free(pivot_col); free(decoded);
        return -1;
    }
    int rows = 0;
    for (int i = 0; i < n_out; ++i) {
        if (!care[i]) continue;                     /* only not-pruned bits */
        for (int t = 0; t < n_in; ++t) kept[rows * w + t] = M[i * n_in + t];
        kept[rows * w + n_in] = wq[i];
        ++rows;
        memcpy(work, kept, (size_t)rows * w);
        gauss_jordan_gf2(work, rows, n_in, pivot_col);
        if (!is_consistent(work, rows, n_in)) --rows;   /* this care bit cannot be met: drop its equation */
    }
    /* Solve the kept equations: pivot variables take the right-hand side of   */
    /* their row, free variables are 0.                                        */
    for (int t = 0; t < n_in; ++t) wc[t] = 0;
    if (rows > 0) {
        memcpy(work, kept, (size_t)rows * w);
        int rank = gauss_jordan_gf2(work, rows, n_in, pivot_col);
        for (int i = 0; i < rank; ++i) wc[pivot_col[i]] = work[i * w + n_in];
    }
    orc_xor_network(n_out, n_in, M, wc, decoded);
    int n_patch = 0;
    for (int i = 0; i < n_out; ++i)
        if (care[i] && decoded[i] != wq[i]) dpatch[n_patch++] = (uint16_t)i;
    free(kept); free(work); free(pivot_col); free(decoded);
    return n_patch;
}

/* ------------------------------------------------------------------------- */
/* Exhaustive search of Section 5.2: list all 2^n_in seeds, keep the one with */
/* the fewest wrong care bits (the smallest seed value among equals, seed     */
/* value = sum of wc[t] << t).  n_in <= 24.                                   */
/* ------------------------------------------------------------------------- */
int orc_encode_slice_exhaustive(int n_out, int n_in, const uint8_t *M, const uint8_t *wq,
                                const uint8_t *care, uint8_t *wc, uint16_t *dpatch)
{
    if (n_in > 24) return -1;
    uint8_t seed[32], decoded[4096];
    if (n_out > 4096) return -1;
    long best_v = 0;
    int best = n_out + 1;
    for (long v = 0; v < (1L << n_in); ++v) {
        for (int t = 0; t < n_in; ++t) seed[t] = (uint8_t)((v >> t) & 1);
        orc_xor_network(n_out, n_in, M, seed, decoded);
        int wrong = 0;
        for (int i = 0; i < n_out; ++i)
            if (care[i] && decoded[i] != wq[i]) ++wrong;
        if (wrong < best) { best = wrong; best_v = v; }
    }
    for (int t = 0; t < n_in; ++t) wc[t] = (uint8_t)((best_v >> t) & 1);
    orc_xor_network(n_out, n_in, M, wc, decoded);
    int n_patch = 0;
    for (int i = 0; i < n_out; ++i)
        if (care[i] && decoded[i] != wq[i]) dpatch[n_patch++] = (uint16_t)i;
    return n_patch;
}

/* ------------------------------------------------------------------------- */
/* Decode of one slice, Sections 3.1 and 3.2: run the network, then flip the  */
/* positions listed in d_patch.  All n_out bits are produced, don't-care      */
/* positions included.                                                        */
/* ------------------------------------------------------------------------- */
void orc_decode_slice(int n_out, int n_in, const uint8_t *M, const uint8_t *wc,
                      int n_patch, const uint16_t *dpatch, uint8_t *out)
{
    orc_xor_network(n_out, n_in, M, wc, out);
    for (int k = 0; k < n_patch; ++k)
        out[dpatch[k]] ^= 1;
}

/* ------------------------------------------------------------------------- */
/* One bit-plane, flattened row-major into mn positions and cut into          */
/* l = ceil(mn / n_out) slices (Section 3.2, the format paragraph).           */
/* Positions past mn in the last slice are don't-cares.                       */
/*                                                                            */
/* bits[p], care[p] : one byte per position, p < mn                           */
/* wc_out[s]        : seed of slice s as an integer, bit t = w^c[t]           */
/* np_out[s]        : n_patch of slice s                                      */
/* dp_out           : all d_patch entries in slice order; caller provides     */
/*                    room for dp_cap entries                                 */
/* Returns the number of d_patch entries, or -1 on overflow / no memory.      */
/* Slices are independent; the first pass runs them in parallel and the       */
/* second pass concatenates their patch lists in slice order.                 */
/* ------------------------------------------------------------------------- */
int64_t orc_encode_plane(int64_t mn, int n_out, int n_in, const uint8_t *M,
                         const uint8_t *bits, const uint8_t *care, int exhaustive,
                         uint64_t *wc_out, uint16_t *np_out, uint16_t *dp_out, int64_t dp_cap)
{
    const int64_t l = (mn + n_out - 1) / n_out;
    if (n_in > 64) return -1;
    uint16_t *all_dp = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)(l > 0 ? l : 1) * (size_t)n_out);
    if (!all_dp) return -1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t s = 0; s < l; ++s) {
        uint8_t *wq = (uint8_t *)calloc((size_t)n_out, 1);
        uint8_t *cr = (uint8_t *)calloc((size_t)n_out, 1);
        uint8_t wc[64];
        if (!wq || !cr) {
#pragma omp atomic write
            failed = 1;
            free(wq); free(cr);
            continue;
        }
        for (int j = 0; j < n_out; ++j) {
            int64_t p = s * n_out + j;
            if (p < mn) { wq[j] = bits[p]; cr[j] = care[p]; }
        }
        int np = exhaustive
            ? orc_encode_slice_exhaustive(n_out, n_in, M, wq, cr, wc, all_dp + s * n_out)
            : orc_encode_slice(n_out, n_in, M, wq, cr, wc, all_dp + s * n_out);
        if (np < 0) {
#pragma omp atomic write
            failed = 1;
            np = 0;
        }
        uint64_t v = 0;
        for (int t = 0; t < n_in; ++t) v |= ((uint64_t)wc[t]) << t;
        wc_out[s] = v;
        np_out[s] = (uint16_t)np;
        free(wq); free(cr);
    }
    int64_t total = 0;
    if (!failed) {
        for (int64_t s = 0; s < l; ++s) {
            for (int k = 0; k < np_out[s]; ++k) {
                if (total >= dp_cap) { failed = 1; break; }
                dp_out[total++] = all_dp[s * n_out + k];
            }
            if (failed) break;
        }
    }
    free(all_dp);
    return failed ? -1 : total;
}

/* ------------------------------------------------------------------------- */
/* Decode slices [s_begin, s_end) of one plane.  dp_start[s] is the index of  */
/* slice s's first entry in dp (the running sum of n_patch, which the caller  */
/* may pass as NULL to have it computed here).  bits_out[p] is written for    */
/* every p < mn that falls in those slices.                                   */
/* ------------------------------------------------------------------------- */
int orc_decode_plane(int64_t mn, int n_out, int n_in, const uint8_t *M,
                     const uint64_t *wc, const uint16_t *np, const uint16_t *dp,
                     int64_t s_begin, int64_t s_end, uint8_t *bits_out)
{
    const int64_t l = (mn + n_out - 1) / n_out;
    if (s_begin < 0 || s_end > l || n_in > 64) return -1;
    int64_t *start = (int64_t *)malloc(sizeof(int64_t) * (size_t)(l + 1));
    if (!start) return -1;
    start[0] = 0;
    for (int64_t s = 0; s < l; ++s) start[s + 1] = start[s] + np[s];
    int failed = 0;
#pragma omp parallel for schedule(static)
    for (int64_t s = s_begin; s < s_end; ++s) {
        uint8_t seed[64];
        uint8_t *out = (uint8_t *)malloc((size_t)n_out);
        if (!out) { failed = 1; continue; }
        for (int t = 0; t < n_in; ++t) seed[t] = (uint8_t)((wc[s] >> t) & 1);
        orc_decode_slice(n_out, n_in, M, seed, np[s], dp + start[s], out);
        for (int j = 0; j < n_out; ++j) {
            int64_t p = s * n_out + j;
            if (p < mn) bits_out[p] = out[j];
        }
        free(out);
    }
    free(start);
    return failed ? -1 : 0;
}

/* ------------------------------------------------------------------------- */
/* fp32 -> bf16 by the format's definition: keep sign, 8 exponent bits and    */
/* the top 7 fraction bits, round to nearest, ties to even; NaN stays NaN.    */
/* ------------------------------------------------------------------------- */
uint16_t orc_bf16_from_f32(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u && (u & 0x007fffffu) != 0)
        return (uint16_t)((u >> 16) | 0x0040u);       /* quiet NaN */
    uint32_t kept = u >> 16;
    uint32_t dropped = u & 0xffffu;
    if (dropped > 0x8000u || (dropped == 0x8000u && (kept & 1u)))
        kept += 1;
    return (uint16_t)kept;
}

/* ------------------------------------------------------------------------- */
/* Reconstruction of the weight values from decoded planes (the binary-code   */
/* form sum_i alpha_i * b_i with b_i in {-1,+1}; bit 1 <-> +1):               */
/*   W[r][c] = 0                         if mask[r][c] = 0 (pruned)           */
/*           = (+-a_1) + (+-a_2) + ...   otherwise, added in plane order in   */
/*             fp32 (each term exact, so the sum has one defined rounding     */
/*             sequence).                                                     */
/* planes: n_q x m x n bytes.  alpha: m x n_q floats.                         */
/* w32 (m x n floats) and wbf16 (m x n uint16) may each be NULL.              */
/* ------------------------------------------------------------------------- */
void orc_reconstruct(int64_t m, int64_t n, int n_q, const uint8_t *planes, const uint8_t *mask,
                     const float *alpha, float *w32, uint16_t *wbf16)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < m; ++r) {
        for (int64_t c = 0; c < n; ++c) {
            int64_t p = r * n + c;
            volatile float acc = 0.0f;    /* volatile: one fp32 rounding per add */
            if (mask[p]) {
                for (int i = 0; i < n_q; ++i) {
                    float a = alpha[r * n_q + i];
                    float term = planes[(int64_t)i * m * n + p] ? a : -a;
                    if (i == 0) acc = term; else acc = acc + term;
                }
            }
            if (w32) w32[p] = acc;
            if (wbf16) wbf16[p] = orc_bf16_from_f32(acc);
        }
    }
}

/* ------------------------------------------------------------------------- */
/* The product the decoded layer feeds: Y[b][r] = sum_c W[r][c] * X[b][c] in  */
/* fp64, with W[r][c] the exact (fp64) sum of the fp32 scales, not a rounded  */
/* value.  X: batch x n doubles.  Y: batch x m doubles.                       */
/* ------------------------------------------------------------------------- */
void orc_matmul(int64_t m, int64_t n, int n_q, const uint8_t *planes, const uint8_t *mask,
                const float *alpha, const double *X, int64_t batch, double *Y)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < m; ++r) {
        for (int64_t b = 0; b < batch; ++b) {
            double acc = 0.0;
            for (int64_t c = 0; c < n; ++c) {
                int64_t p = r * n + c;
                if (!mask[p]) continue;
                double wv = 0.0;
                for (int i = 0; i < n_q; ++i) {
                    double a = (double)alpha[r * n_q + i];
                    wv += planes[(int64_t)i * m * n + p] ? a : -a;
                }
                acc += wv * X[b * n + c];
            }
            Y[b * m + r] = acc;
        }
    }
}

/* smallest e with 2^e >= v, for v >= 1; 0 for v <= 1 */
static int ceil_lg(int64_t v)
{
    int e = 0;
    while (((int64_t)1 << e) < v) ++e;
    return e;
}

/* ------------------------------------------------------------------------- */
/* Eq. 1, the compression ratio of one plane, taken literally:                */
/*   r = mn / ( n_in/n_out * mn + l * ceil(lg max p) + sum p * ceil(lg n_out))*/
/* with ceil(lg 0) and ceil(lg 1) read as 0.  out[0] = r, out[1] = bits of    */
/* w^c (first term), out[2] = bits of n_patch, out[3] = bits of d_patch,      */
/* out[4] = max p, out[5] = sum p.                                            */
/* ------------------------------------------------------------------------- */
void orc_eq1(int64_t mn, int n_out, int n_in, const uint16_t *np, double *out)
{
    const int64_t l = (mn + n_out - 1) / n_out;
    int64_t maxp = 0, sump = 0;
    for (int64_t s = 0; s < l; ++s) {
        if (np[s] > maxp) maxp = np[s];
        sump += np[s];
    }
    double b_wc = (double)n_in / (double)n_out * (double)mn;
    double b_np = (double)l * (double)ceil_lg(maxp);
    double b_dp = (double)sump * (double)ceil_lg(n_out);
    out[0] = (double)mn / (b_wc + b_np + b_dp);
    out[1] = b_wc;
    out[2] = b_np;
    out[3] = b_dp;
    out[4] = (double)maxp;
    out[5] = (double)sump;
}

/* ------------------------------------------------------------------------- */
/* Blocked n_patch assignment (Section 5.2): the plane's l slices are cut     */
/* into blocks of `block` consecutive slices and the width of the n_patch     */
/* field is chosen per block from that block's own max p, so Eq. 1's middle   */
/* term l * ceil(lg max p) becomes  sum over blocks of                        */
/*   (slices in the block) * ceil(lg max p of the block).                     */
/* The paper does not say how a block's width is made known to the decoder;   */
/* out[3] reports one byte per block for it, separately.                      */
/* out[0] = r with blocked widths (width bytes not counted), out[1] = bits of */
/* n_patch with blocked widths, out[2] = number of blocks, out[3] = bits of   */
/* the per-block width bytes.                                                 */
/* ------------------------------------------------------------------------- */
void orc_eq1_blocked(int64_t mn, int n_out, int n_in, const uint16_t *np, int64_t block, double *out)
{
    const int64_t l = (mn + n_out - 1) / n_out;
    int64_t sump = 0, blocks = 0;
    double b_np = 0.0;
    for (int64_t s0 = 0; s0 < l; s0 += block) {
        int64_t s1 = s0 + block < l ? s0 + block : l;
        int64_t maxp = 0;
        for (int64_t s = s0; s < s1; ++s) {
            if (np[s] > maxp) maxp = np[s];
            sump += np[s];
        }
        b_np += (double)(s1 - s0) * (double)ceil_lg(maxp);
        blocks += 1;
    }
    double b_wc = (double)n_in / (double)n_out * (double)mn;
    double b_dp = (double)sump * (double)ceil_lg(n_out);
    out[0] = (double)mn / (b_wc + b_np + b_dp);
    out[1] = b_np;
    out[2] = (double)blocks;
    out[3] = 8.0 * (double)blocks;
}

/* ------------------------------------------------------------------------- */
/* Blocked n_patch assignment (Section 5.2) as a stored format: a field must  */
/* be able to hold every count of its block, the largest included, so its     */
/* width is ceil(lg(max p of the block + 1)) bits (Eq. 1's ceil(lg max p)     */
/* cannot hold max p when that is a power of two; same reading as for the     */
/* per-plane width).  out[0] = sum over blocks of (slices in the block) *     */
/* width, out[1] = number of blocks.                                          */
/* ------------------------------------------------------------------------- */
void orc_blocked_field_bits(int64_t l, const uint16_t *np, int64_t block, double *out)
{
    double bits = 0.0;
    int64_t blocks = 0;
    for (int64_t s0 = 0; s0 < l; s0 += block) {
        int64_t s1 = s0 + block < l ? s0 + block : l;
        int64_t maxp = 0;
        for (int64_t s = s0; s < s1; ++s)
            if (np[s] > maxp) maxp = np[s];
        bits += (double)(s1 - s0) * (double)ceil_lg(maxp + 1);
        blocks += 1;
    }
    out[0] = bits;
    out[1] = (double)blocks;
}

/* ------------------------------------------------------------------------- */
/* Patch-data FIFO of one XOR-gate network (Section 5.1), cycle by cycle.     */
/* Reading of the section (it gives no equations):                            */
/*  - the network decrypts one slice per cycle when nothing holds it up;      */
/*  - d_patch arrives as its own stream, `rate` entries per cycle, into a     */
/*    FIFO of `depth` entries; the stream waits while the FIFO is full;       */
/*  - the FIFO has n_fifo banks and hands at most n_fifo entries per cycle to */
/*    the patch logic; a slice leaves the decoder in the cycle in which the   */
/*    last of its n_patch entries has been handed over (a slice without       */
/*    patches takes one cycle);                                               */
/*  - within a cycle the stream writes first, then the patch logic reads.     */
/* out[0] = cycles, out[1] = cycles in which the decoder held a slice over    */
/* because more than n_fifo entries were still due (bandwidth stall),         */
/* out[2] = cycles in which it held a slice over because the FIFO ran empty,  */
/* out[3] = cycles in which the stream waited on a full FIFO, out[4] = peak   */
/* occupancy after the write phase.  Relative execution time = cycles / l.    */
/* ------------------------------------------------------------------------- */
void orc_fifo_model(int64_t l, const uint16_t *np, int n_fifo, int rate, int depth, double *out)
{
    int64_t total = 0;
    for (int64_t s = 0; s < l; ++s) total += np[s];
    int64_t cycles = 0, stall_bw = 0, stall_empty = 0, stall_full = 0, peak = 0;
    int64_t fifo = 0, produced = 0;
    int64_t s = 0;
    int64_t need = l > 0 ? np[0] : 0;
    while (s < l) {
        cycles += 1;
        /* the stream writes */
        int64_t w = rate;
        if (w > total - produced) w = total - produced;
        if (w > depth - fifo) {
            w = depth - fifo;
            stall_full += 1;
        }
        fifo += w;
        produced += w;
        if (fifo > peak) peak = fifo;
        /* the patch logic reads */
        int64_t r = need;
        if (r > n_fifo) r = n_fifo;
        if (r > fifo) r = fifo;
        fifo -= r;
        need -= r;
        if (need == 0) {
            s += 1;
            if (s < l) need = np[s];
        } else if (r == n_fifo) {
            stall_bw += 1;
        } else {
            stall_empty += 1;
        }
    }
    out[0] = (double)cycles;
    out[1] = (double)stall_bw;
    out[2] = (double)stall_empty;
    out[3] = (double)stall_full;
    out[4] = (double)peak;
}

/* ------------------------------------------------------------------------- */
/* The CSR side of the same comparison (Section 5.1, Section 1): `lanes` rows */
/* are worked on side by side, one non-zero per lane and cycle, and a group   */
/* of rows is done when its longest row is, so a group costs max nnz cycles.  */
/* Returns cycles / (sum nnz / lanes): 1.0 when every row has the same count. */
/* ------------------------------------------------------------------------- */
double orc_csr_relative_time(int64_t rows, const int64_t *nnz, int lanes)
{
    int64_t cycles = 0, sum = 0;
    for (int64_t r0 = 0; r0 < rows; r0 += lanes) {
        int64_t mx = 0;
        for (int64_t r = r0; r < rows && r < r0 + lanes; ++r) {
            if (nnz[r] > mx) mx = nnz[r];
            sum += nnz[r];
        }
        cycles += mx;
    }
    if (sum == 0) return 1.0;
    return (double)cycles / ((double)sum / (double)lanes);
}
