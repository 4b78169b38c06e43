// Exhaustive seed search on the device (Section 5.2): for every slice of every plane all 2^n_in
// seeds are expanded through the network and the seed with the fewest wrong care bits is kept
// (the smallest seed among equals).
//
// One warp per slice.  The 32 lanes split the seeds by their top five bits; inside its range a
// lane walks the low bits in Gray-code order, so that going from one seed to the next is one
// XOR with a column of M (w~ = M . w^c is linear over GF(2)) -- the columns sit in shared memory
// and all lanes read the same one.  The count of wrong care bits is popc((w~ ^ w^q) & care).
#include "sqnn_launch.h"

#include <cuda_runtime.h>

namespace sqnn {

namespace {

struct SearchArgs {
    uint32_t rows[SQNN_MAX_N_OUT];   // rows of M (the library holds no device memory: passed by value)
    uint32_t n_out, n_in, n_q;
    uint64_t mn, words64, slices;
    const uint64_t *planes, *mask;
    uint32_t *wc;
    uint16_t *np;
};

// 32 bits of a packed vector starting at position p; positions >= limit (<= vector length) read 0
SQNN_DEV uint32_t bits32_at(const uint64_t *__restrict__ v, uint64_t p, uint64_t limit)
{
    if (p >= limit) return 0u;
    const uint64_t w = p >> 6;
    const uint32_t sh = (uint32_t)(p & 63);
    uint64_t x = __ldg(v + w) >> sh;
    if (sh > 32 && limit > ((w + 1) << 6)) x |= __ldg(v + w + 1) << (64 - sh);   // next word holds wanted positions
    uint32_t r = (uint32_t)x;
    if (p + 32 > limit) r &= (1u << (uint32_t)(limit - p)) - 1u;
    return r;
}

template <int NW>
__global__ void __launch_bounds__(256)
k_search_seeds(const __grid_constant__ SearchArgs S)
{
    __shared__ uint32_t cols[SQNN_MAX_N_IN][NW];          // column t of M as an n_out-bit word
    __shared__ uint32_t want_s[8][NW], care_s[8][NW];     // per warp: the slice
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (uint32_t i = threadIdx.x; i < S.n_in * NW; i += blockDim.x) {
        const uint32_t t = i / NW, k = i % NW;
        uint32_t w = 0;
        for (uint32_t j = 32 * k; j < S.n_out && j < 32 * k + 32; ++j) w |= ((S.rows[j] >> t) & 1u) << (j - 32 * k);
        cols[t][k] = w;
    }
    __syncthreads();
    const uint32_t low_bits = S.n_in > 5 ? S.n_in - 5 : 0;
    const uint32_t lanes_used = S.n_in >= 5 ? 32u : (1u << S.n_in);
    const uint64_t total = S.slices * S.n_q;
    for (uint64_t job = (uint64_t)blockIdx.x * nwarps + warp; job < total; job += (uint64_t)gridDim.x * nwarps) {
        const uint32_t plane = (uint32_t)(job / S.slices);
        const uint64_t s = job - (uint64_t)plane * S.slices;
        const uint64_t p0 = s * S.n_out;
        __syncwarp();
        if (lane < NW) {
            const uint32_t lo = 32 * lane;
            uint32_t c = 0, w = 0;
            if (lo < S.n_out) {
                const uint64_t limit = p0 + S.n_out < S.mn ? p0 + S.n_out : S.mn;   // slice end (ragged tail)
                c = bits32_at(S.mask, p0 + lo, limit);
                w = bits32_at(S.planes + (uint64_t)plane * S.words64, p0 + lo, limit);
            }
            care_s[warp][lane] = c;
            want_s[warp][lane] = w;
        }
        __syncwarp();
        uint32_t want[NW], care[NW], out[NW];
#pragma unroll
        for (int k = 0; k < NW; ++k) { want[k] = want_s[warp][k]; care[k] = care_s[warp][k]; out[k] = 0; }
        uint32_t best = 0xffffffffu;
        if (lane < lanes_used) {
            const uint32_t top = lane << low_bits;
            for (uint32_t t = low_bits; t < S.n_in; ++t)
                if ((top >> t) & 1u) {
#pragma unroll
                    for (int k = 0; k < NW; ++k) out[k] ^= cols[t][k];
                }
            const uint32_t count = 1u << low_bits;
            for (uint32_t i = 0; i < count; ++i) {
                if (i != 0) {
                    const uint32_t t = (uint32_t)__ffs((int)i) - 1u;      // bit that changes in the Gray code
#pragma unroll
                    for (int k = 0; k < NW; ++k) out[k] ^= cols[t][k];
                }
                uint32_t wrong = 0;
#pragma unroll
                for (int k = 0; k < NW; ++k) wrong += (uint32_t)__popc((out[k] ^ want[k]) & care[k]);
                const uint32_t seed = top | (i ^ (i >> 1));
                const uint32_t key = (wrong << 20) | seed;                  // n_in <= 20, wrong <= 256
                best = key < best ? key : best;
            }
        }
#pragma unroll
        for (uint32_t d = 16; d >= 1; d >>= 1) {
            const uint32_t o = __shfl_xor_sync(0xffffffffu, best, d);
            best = o < best ? o : best;
        }
        if (lane == 0) {
            S.wc[job] = best & 0xfffffu;
            S.np[job] = (uint16_t)(best >> 20);
        }
    }
}

}  // namespace

}  // namespace sqnn

static int search_seeds_queue(const sqnn_xornet *net, uint64_t m, uint64_t n, uint32_t n_q,
                              const uint64_t *d_planes, const uint64_t *d_mask, uint32_t *d_wc,
                              uint16_t *d_np, void *cuda_stream)
{
    using namespace sqnn;
    if (!net || !net->rows || !d_planes || !d_mask || !d_wc || !d_np) return SQNN_E_INVALID_ARG;
    if (net->n_out < 1 || net->n_out > SQNN_MAX_N_OUT || net->n_in < 1 || net->n_in > SQNN_MAX_N_IN ||
        n_q < 1 || n_q > SQNN_MAX_PLANES || m == 0 || n == 0 || m > ((uint64_t)1 << 40) / n)
        return SQNN_E_INVALID_ARG;
    if (net->n_in > 20) return SQNN_E_UNSUPPORTED;          // 2^n_in seeds per slice
    SearchArgs S;
    for (uint32_t j = 0; j < SQNN_MAX_N_OUT; ++j) S.rows[j] = j < net->n_out ? net->rows[j] : 0u;
    S.n_out = net->n_out; S.n_in = net->n_in; S.n_q = n_q;
    S.mn = m * n;
    S.words64 = (S.mn + 63) / 64;
    S.slices = (S.mn + net->n_out - 1) / net->n_out;
    S.planes = d_planes; S.mask = d_mask; S.wc = d_wc; S.np = d_np;
    const uint64_t jobs = S.slices * n_q;
    uint64_t blocks = (jobs + 7) / 8;
    const uint64_t cap = (uint64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const uint32_t nw = (net->n_out + 31) / 32;
    if (nw <= 1) k_search_seeds<1><<<(uint32_t)blocks, 256, 0, st>>>(S);
    else if (nw <= 2) k_search_seeds<2><<<(uint32_t)blocks, 256, 0, st>>>(S);
    else if (nw <= 4) k_search_seeds<4><<<(uint32_t)blocks, 256, 0, st>>>(S);
    else k_search_seeds<8><<<(uint32_t)blocks, 256, 0, st>>>(S);
    return cudaGetLastError() == cudaSuccess ? SQNN_OK : SQNN_E_CUDA;
}

extern "C" int sqnn_search_seeds(const sqnn_xornet *net, uint64_t m, uint64_t n, uint32_t n_q,
                                 const uint64_t *d_planes, const uint64_t *d_mask, uint32_t *d_wc,
                                 uint16_t *d_np, void *cuda_stream)
{
    sqnn::ApiScope scope("sqnn_search_seeds");
    return scope.finish(search_seeds_queue(net, m, n, n_q, d_planes, d_mask, d_wc, d_np, cuda_stream), nullptr,
                        (cudaStream_t)cuda_stream);
}
