/* Drives the CPU oracle on small seeded cases; built with -fsanitize=address,undefined by
 * tests/test_sanitizers.py.  Exit code 0 = every care bit came back and no call failed. */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

int orc_encode_slice(int n_out, int n_in, const uint8_t *M, const uint8_t *wq, const uint8_t *care, uint8_t *wc, uint16_t *dp);
int64_t orc_encode_plane(int64_t mn, int n_out, int n_in, const uint8_t *M, const uint8_t *bits, const uint8_t *care,
                         int exhaustive, uint64_t *wc_out, uint16_t *np_out, uint16_t *dp_out, int64_t dp_cap);
int orc_decode_plane(int64_t mn, int n_out, int n_in, const uint8_t *M, const uint64_t *wc, const uint16_t *np,
                     const uint16_t *dp, int64_t s_begin, int64_t s_end, uint8_t *bits_out);
void orc_blocked_field_bits(int64_t l, const uint16_t *np, int64_t block, double *out);
void orc_fifo_model(int64_t l, const uint16_t *np, int n_fifo, int rate, int depth, double *out);

static uint64_t state = 12345;
static uint64_t next(void)
{
    uint64_t z = (state += 0x9e3779b97f4a7c15ull);
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ull;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebull;
    return z ^ (z >> 31);
}

static int one_case(int n_out, int n_in, int64_t mn, int keep_percent, int exhaustive)
{
    const int64_t l = (mn + n_out - 1) / n_out;
    uint8_t *M = malloc((size_t)n_out * n_in), *bits = malloc((size_t)mn), *care = malloc((size_t)mn), *out = malloc((size_t)mn);
    uint64_t *wc = malloc(sizeof(uint64_t) * (size_t)l);
    uint16_t *np = malloc(sizeof(uint16_t) * (size_t)l), *dp = malloc(sizeof(uint16_t) * (size_t)mn);
    if (!M || !bits || !care || !out || !wc || !np || !dp) return 1;
    for (int i = 0; i < n_out * n_in; ++i) M[i] = (uint8_t)(next() & 1);
    for (int64_t p = 0; p < mn; ++p) { bits[p] = (uint8_t)(next() & 1); care[p] = (uint8_t)((int)(next() % 100) < keep_percent); }
    const int64_t total = orc_encode_plane(mn, n_out, n_in, M, bits, care, exhaustive, wc, np, dp, mn);
    int bad = total < 0;
    if (!bad) bad = orc_decode_plane(mn, n_out, n_in, M, wc, np, dp, 0, l, out) != 0;
    for (int64_t p = 0; !bad && p < mn; ++p) bad = care[p] && out[p] != bits[p];
    double acc[4] = {0, 0, 0, 0}, fifo[8] = {0};
    orc_blocked_field_bits(l, np, 16, acc);
    orc_fifo_model(l, np, 2, 1, 8, fifo);
    if (bad) fprintf(stderr, "oracle_san: case %d x %d failed\n", n_out, n_in);
    free(M); free(bits); free(care); free(out); free(wc); free(np); free(dp);
    return bad;
}

int main(void)
{
    if (one_case(20, 6, 1003, 30, 0)) return 1;
    if (one_case(20, 6, 1003, 30, 1)) return 1;
    if (one_case(100, 10, 5021, 9, 0)) return 1;
    if (one_case(300, 40, 9000, 10, 0)) return 1;
    if (one_case(7, 3, 50, 100, 1)) return 1;
    puts("oracle_san ok");
    return 0;
}
