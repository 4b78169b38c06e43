// Drives the host half of the library (encoder, validator, unpack, statistics, storage form, FIFO
// model) on small seeded layers; built with -fsanitize=address,undefined by tests/test_sanitizers.py.
// Exit code 0 = every call behaved and every layer survived the round trips.
#include "sqnn.h"

#include <cstdint>
#include <cstdio>
#include <cstring>
#include <vector>

namespace {
uint64_t state = 0x9e3779b97f4a7c15ull;
uint64_t next()                       // splitmix64
{
    uint64_t z = (state += 0x9e3779b97f4a7c15ull);
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ull;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebull;
    return z ^ (z >> 31);
}
int fail(const char *what, int rc)
{
    std::fprintf(stderr, "host_san: %s (rc %d)\n", what, rc);
    return 1;
}
}  // namespace

static int one_layer(uint32_t n_out, uint32_t n_in, uint64_t m, uint64_t n, uint32_t n_q, double keep, uint32_t flags)
{
    std::vector<uint32_t> rows(n_out);
    for (auto &r : rows) r = (uint32_t)next() & (n_in >= 32 ? 0xffffffffu : ((1u << n_in) - 1u));
    const uint64_t mn = m * n, words = (mn + 63) / 64;
    std::vector<uint64_t> planes(n_q * words), mask(words, 0);
    for (auto &w : planes) w = next();
    for (uint64_t p = 0; p < mn; ++p)
        if ((double)(next() >> 11) / 9007199254740992.0 < keep) mask[p >> 6] |= 1ull << (p & 63);
    for (uint32_t i = 0; i < n_q; ++i)
        if (mn & 63) planes[i * words + words - 1] &= (1ull << (mn & 63)) - 1ull;
    sqnn_xornet net{n_out, n_in, rows.data()};
    sqnn_planes layer{m, n, n_q, planes.data(), mask.data()};
    void *blob = nullptr;
    size_t bytes = 0;
    sqnn_stats st;
    int rc = sqnn_encode_host(&net, &layer, flags, &blob, &bytes, &st);
    if (rc != SQNN_OK) return fail("sqnn_encode_host", rc);
    sqnn_desc d;
    if ((rc = sqnn_describe_host(blob, bytes, &d)) != SQNN_OK) return fail("sqnn_describe_host", rc);
    if (d.m != m || d.n != n || d.n_q != n_q || d.total_bytes != bytes) return fail("descriptor fields", 0);
    sqnn_stats st2;
    if ((rc = sqnn_stats_host(blob, bytes, &st2)) != SQNN_OK) return fail("sqnn_stats_host", rc);
    if (st2.slices != st.slices || st2.patches[0] != st.patches[0]) return fail("statistics differ", 0);
    double bpw = 0;
    uint64_t bnp = 0;
    if ((rc = sqnn_stats_blocked_host(blob, bytes, 64, &bpw, &bnp)) != SQNN_OK) return fail("sqnn_stats_blocked_host", rc);
    // unpack -> pack gives the same blob
    std::vector<uint32_t *> wc(n_q);
    std::vector<uint16_t *> np(n_q), dp(n_q);
    for (uint32_t i = 0; i < n_q; ++i) {
        uint64_t n_dp = 0;
        if ((rc = sqnn_unpack_host(blob, bytes, i, &wc[i], &np[i], &dp[i], &n_dp)) != SQNN_OK) return fail("sqnn_unpack_host", rc);
        if (n_dp != d.n_pp[i]) return fail("patch count", 0);
        sqnn_fifo_result fr;
        if ((rc = sqnn_fifo_model_host(np[i], d.slices, 2, 1, 8, &fr)) != SQNN_OK) return fail("sqnn_fifo_model_host", rc);
        if (fr.cycles < d.slices) return fail("fifo cycles", 0);
    }
    void *blob2 = nullptr;
    size_t bytes2 = 0;
    rc = sqnn_pack_host(&net, m, n, n_q, wc.data(), np.data(), dp.data(), &blob2, &bytes2);
    if (rc != SQNN_OK) return fail("sqnn_pack_host", rc);
    if (bytes2 != bytes || std::memcmp(blob, blob2, bytes) != 0) return fail("pack(unpack(blob)) differs", 0);
    // seeds given -> same blob again
    void *blob3 = nullptr;
    size_t bytes3 = 0;
    rc = sqnn_encode_seeds_host(&net, &layer, wc.data(), &blob3, &bytes3, nullptr);
    if (rc != SQNN_OK) return fail("sqnn_encode_seeds_host", rc);
    if (bytes3 != bytes || std::memcmp(blob, blob3, bytes) != 0) return fail("encode_seeds differs", 0);
    // storage form and back
    void *stored = nullptr, *blob4 = nullptr;
    size_t sbytes = 0, bytes4 = 0;
    sqnn_store_info info;
    if ((rc = sqnn_store_host(blob, bytes, 32, &stored, &sbytes, &info)) != SQNN_OK) return fail("sqnn_store_host", rc);
    if ((rc = sqnn_load_host(stored, sbytes, &blob4, &bytes4)) != SQNN_OK) return fail("sqnn_load_host", rc);
    if (bytes4 != bytes || std::memcmp(blob, blob4, bytes) != 0) return fail("load(store(blob)) differs", 0);
    // damaged inputs are refused, not read out of bounds
    std::vector<unsigned char> bad((unsigned char *)blob, (unsigned char *)blob + bytes);
    for (size_t cut : {size_t(0), size_t(8), bytes / 2, bytes - 1})
        if (sqnn_describe_host(bad.data(), cut, &d) == SQNN_OK) return fail("truncated blob accepted", 0);
    for (int k = 0; k < 64; ++k) {
        std::vector<unsigned char> b2 = bad;
        b2[next() % bytes] ^= (unsigned char)(1u << (next() & 7));
        sqnn_desc dd;
        (void)sqnn_describe_host(b2.data(), b2.size(), &dd);       // either verdict is fine; no bad access
        std::vector<unsigned char> s2((unsigned char *)stored, (unsigned char *)stored + sbytes);
        s2[next() % sbytes] ^= (unsigned char)(1u << (next() & 7));
        void *o = nullptr;
        size_t ob = 0;
        if (sqnn_load_host(s2.data(), s2.size(), &o, &ob) == SQNN_OK) sqnn_free(o);
    }
    for (uint32_t i = 0; i < n_q; ++i) { sqnn_free(wc[i]); sqnn_free(np[i]); sqnn_free(dp[i]); }
    sqnn_free(blob); sqnn_free(blob2); sqnn_free(blob3); sqnn_free(blob4); sqnn_free(stored);
    return 0;
}

int main()
{
    if (one_layer(80, 8, 37, 53, 1, 0.10, SQNN_ENCODE_ALG1)) return 1;
    if (one_layer(60, 12, 64, 90, 2, 0.20, SQNN_ENCODE_ALG1)) return 1;
    if (one_layer(40, 12, 31, 77, 3, 0.40, SQNN_ENCODE_ALG1)) return 1;
    if (one_layer(13, 5, 9, 41, 1, 0.50, SQNN_ENCODE_EXHAUSTIVE)) return 1;
    if (one_layer(200, 10, 16, 300, 1, 0.10, SQNN_ENCODE_ALG1)) return 1;
    // the wide encoder (64-bit rows)
    {
        const uint32_t n_out = 300, n_in = 40;
        const uint64_t mn = 3000, words = (mn + 63) / 64;
        std::vector<uint64_t> rows(n_out), plane(words), mask(words);
        for (auto &r : rows) r = next() & ((1ull << n_in) - 1ull);
        for (auto &w : plane) w = next();
        for (auto &w : mask) w = next() & next() & next();
        uint64_t *wc = nullptr, n_dp = 0;
        uint16_t *np = nullptr, *dp = nullptr;
        double bpw = 0;
        int rc = sqnn_encode_wide_host(n_out, n_in, rows.data(), mn, plane.data(), mask.data(), &wc, &np, &dp, &n_dp, &bpw);
        if (rc != SQNN_OK) return fail("sqnn_encode_wide_host", rc);
        sqnn_free(wc); sqnn_free(np); sqnn_free(dp);
    }
    std::puts("host_san ok");
    return 0;
}
