// K4: decryption fused with the product for batch >= 16 on the 5th-generation tensor cores.
//
//   Y[b][r] = sum_c W[r][c] X[b][c],   D (TMEM, fp32) [128 rows of W x N batch columns]
//                                      += A (shared, bf16, K-major) [128 x 64] . B (shared) [N x 64]^T
//
// One CTA owns 128 rows of W and a range of columns.  Per 64-column step
//   - the decode warps expand the weights of the step into the A stage (bf16, 128-byte rows,
//     128-byte swizzle) -- the expanded weights exist only in shared memory;
//   - one thread fetches the matching activations X[bc .. bc+N) x [64 columns] with TMA
//     (every CTA fetches its own tile);
//   - one thread issues tcgen05.mma (K = 16 each) that accumulate in tensor memory.
// Column ranges of different CTAs are summed with fp32 atomics on Y (cleared beforehand).
//
// The A stage.  Every plane gets its own tile of -1 / 0 / +1 (mask and sign only, four weights per
// table read) and its own accumulator, and the epilogue forms sum_i alpha[r][i] * D_i: the weights
// stay exact and the expansion is a few instructions per weight.  The batch is taken in passes whose
// n_q accumulators fit the 512 columns of tensor memory.  (Only when the sign tiles of all planes do
// not fit two pipeline stages of shared memory -- six planes and more -- one tile holds the rescaled
// weights (+-alpha_1) + (+-alpha_2) + ... rounded to bf16 instead.)
//
// Where the bits come from.  The planes have been decoded to packed bits in the workspace by the
// tiled decode kernel (queued just before this one); 128 x 512-bit boxes of them (and of the mask)
// are brought in by TMA when rows start on 16-byte boundaries, by coalesced loads otherwise.
//
// Every wait on an mbarrier is bounded; a wait that gives up sets SQNN_E_TIMEOUT in the status
// word and makes all roles leave their loops, so the kernel always returns.
#include "sqnn_launch.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

namespace sqnn {

namespace {

constexpr uint32_t ROWS = 128;            // rows of W per CTA = MMA M
constexpr uint32_t KC = 64;               // columns per pipeline step
constexpr uint32_t MACRO = 512;           // columns decoded to bits at a time
constexpr uint32_t STEPS_PER_MACRO = MACRO / KC;
constexpr uint32_t RB_WORDS = MACRO / 32 + 1;   // words per row of the bit buffer (odd stride)
// Copies of the 256-entry sign table, interleaved entry by entry: lane l reads copy l % LUT_COPIES, so two lanes
// can only collide on a bank when they agree in l % LUT_COPIES.
constexpr uint32_t LUT_COPIES = 8;
constexpr uint32_t DEC_WARPS = 16;
constexpr uint32_t DEC_THREADS = DEC_WARPS * 32;
constexpr uint32_t THREADS = DEC_THREADS + 64;  // + TMA warp + MMA warp
constexpr uint32_t A_STAGE_BYTES = ROWS * KC * 2;
constexpr uint32_t MAX_STAGES = 4;
constexpr uint64_t WAIT_LIMIT_CYCLES = 4000000000ull;   // about 2 s at 2 GHz

struct MmaArgs {
    DecodeArgs A;
    const uint32_t *mask32;
    uint64_t mask_words32;        // number of valid 32-bit mask words
    const float *alpha;
    float *y;
    int64_t ldy;
    uint64_t m, n;
    uint32_t batch;               // total batch
    uint32_t nbt;                 // batch columns per pass (multiple of 16, <= 512)
    uint32_t tmem_cols;           // power of two >= nbt, >= 32
    uint32_t stages;
    uint32_t splits;              // CTAs per row tile
    uint32_t macros_per_split;
    uint32_t b_stage_bytes;
    const uint32_t *bits32;       // decoded planes in the workspace
    uint64_t plane_words32;       // 32-bit words per plane in the workspace
    uint32_t per_plane;           // 1: one sign tile and one accumulator per plane, scales in the epilogue
    uint32_t tma_bits;            // 1: the bit buffer is filled by TMA (rows of the packed planes 16-byte aligned)
    uint32_t rbp;                 // words per row of the bit buffer
    uint32_t rb_bufs;             // bit buffers (2 with TMA)
};

// ---------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------
SQNN_DEV void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" :: "r"(smem_addr(bar)), "r"(count) : "memory");
}
SQNN_DEV void mbar_arrive(uint64_t *bar)
{
    asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.shared::cta.b64 st, [%0];\n}\n" :: "r"(smem_addr(bar)) : "memory");
}
SQNN_DEV void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}\n"
                 :: "r"(smem_addr(bar)), "r"(bytes) : "memory");
}
SQNN_DEV bool mbar_try(uint64_t *bar, uint32_t parity)
{
    // The last operand lets the hardware park the thread for up to ~1 ms while the phase is
    // pending (it wakes as soon as the phase completes), so that waiting threads do not take
    // issue slots from working ones; the caller's loop still bounds the total wait.
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity), "r"(1000000u) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the wait was abandoned (limit reached or another role gave up).
SQNN_DEV bool mbar_wait(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status)
{
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((uint64_t)(clock64() - t0) > WAIT_LIMIT_CYCLES) {
            *abort_flag = 1u;
            if (status) atomicMax(status, (uint32_t)(-SQNN_E_TIMEOUT));
            return false;
        }
    }
}
SQNN_DEV void tma_load_2d(void *sdst, const CUtensorMap *map, uint64_t *bar, int32_t x, int32_t y)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];\n"
                 :: "r"(smem_addr(sdst)), "l"(map), "r"(smem_addr(bar)), "r"(x), "r"(y) : "memory");
}
SQNN_DEV void tmem_alloc(uint32_t *slot, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n"
                 :: "r"(smem_addr(slot)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
}
SQNN_DEV void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" :: "r"(taddr), "r"(cols) : "memory");
}
SQNN_DEV void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
SQNN_DEV void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
SQNN_DEV void mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                 :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Makes the mbarrier track completion of all MMAs this thread issued so far.
SQNN_DEV void mma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n"
                 :: "r"(smem_addr(bar)) : "memory");
}
SQNN_DEV void tmem_ld8(uint32_t taddr, uint32_t (&v)[8])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile with 128-byte rows and 128-byte
// swizzle: rows 128 B apart, groups of 8 rows 1024 B apart (stride byte offset), descriptor
// version 1, layout type 2.  `addr` is the shared address of the first row, advanced by 32 B
// per K = 16 step inside the swizzled row.
SQNN_DEV uint64_t smem_desc_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3fffu);
    d |= (uint64_t)1u << 16;                       // leading byte offset (unused for this layout)
    d |= (uint64_t)(1024u >> 4) << 32;             // stride byte offset
    d |= (uint64_t)1u << 46;                       // version
    d |= (uint64_t)2u << 61;                       // 128-byte swizzle
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n.
SQNN_DEV uint32_t instr_desc_bf16(uint32_t n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((ROWS >> 4) << 24);
}

// Barrier over the decode threads that also ORs a flag, so that all of them take the same exit.
SQNN_DEV bool decode_barrier_any(uint32_t flagged)
{
    uint32_t any;
    asm volatile("{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, 1, %2, q;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(any) : "r"(flagged), "n"(DEC_THREADS) : "memory");
    return any != 0;
}

SQNN_DEV void tma_load_3d(void *sdst, const CUtensorMap *map, uint64_t *bar, int32_t x, int32_t y, int32_t z)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];\n"
                 :: "r"(smem_addr(sdst)), "l"(map), "r"(smem_addr(bar)), "r"(x), "r"(y), "r"(z) : "memory");
}

__global__ void __launch_bounds__(THREADS, 1)
k_decode_mma(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap pmap,
             const __grid_constant__ CUtensorMap kmap, const MmaArgs M)
{
    extern __shared__ __align__(16) uint8_t smem_raw[];
    const DecodeArgs &A = M.A;
    const uint32_t n_items = A.n_q + 1;                                  // planes + mask
    const uint32_t a_tiles = M.per_plane ? A.n_q : 1;                    // A tiles per stage
    const uint32_t rbp = M.rbp;                                          // words per row of the bit buffer
    // carve shared memory (A / B stages need 1024-byte alignment for the 128-byte swizzle)
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *a_stages = base;
    const uint32_t a_stage_bytes = a_tiles * A_STAGE_BYTES;
    uint8_t *b_stages = a_stages + M.stages * a_stage_bytes;
    uint32_t *rb = reinterpret_cast<uint32_t *>(b_stages + (size_t)M.stages * M.b_stage_bytes);   // [buf][item][row][rbp]
    const uint32_t rb_buf_words = n_items * ROWS * rbp;
    uint2 *lut256 = reinterpret_cast<uint2 *>(rb + M.rb_bufs * rb_buf_words);                          // [256][LUT_COPIES]
    __nv_bfloat16 *lut = reinterpret_cast<__nv_bfloat16 *>(lut256 + 256 * LUT_COPIES);                             // [row][16]
    float *alpha_s = reinterpret_cast<float *>(lut + ROWS * 16);         // [row][8]
    uint64_t *bars = reinterpret_cast<uint64_t *>(alpha_s + ROWS * 8);
    uint64_t *full_a = bars, *full_b = bars + MAX_STAGES, *empty = bars + 2 * MAX_STAGES;
    uint64_t *accum = bars + 3 * MAX_STAGES;
    uint64_t *bits_full = accum + 1, *bits_empty = accum + 3;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(accum + 5);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t row_tile = blockIdx.x / M.splits, split = blockIdx.x % M.splits;
    const uint64_t r0 = (uint64_t)row_tile * ROWS;
    const uint32_t total_macros = (uint32_t)((M.n + MACRO - 1) / MACRO);
    const uint32_t macro_begin = split * M.macros_per_split;
    const uint32_t macro_end = macro_begin + M.macros_per_split < total_macros ? macro_begin + M.macros_per_split : total_macros;
    const uint32_t total_steps = (uint32_t)((M.n + KC - 1) / KC);

    if (tid == 0) {
        for (uint32_t s = 0; s < MAX_STAGES; ++s) {
            mbar_init(full_a + s, DEC_WARPS);        // one arrival per decode warp
            mbar_init(full_b + s, 1);
            mbar_init(empty + s, 1);
        }
        mbar_init(accum, 1);
        for (uint32_t s = 0; s < 2; ++s) {
            mbar_init(bits_full + s, 1);
            mbar_init(bits_empty + s, DEC_WARPS);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == DEC_WARPS + 1) tmem_alloc(tmem_slot, M.tmem_cols);
    if (tid < 256) {
        // 4 weights of one plane at a time: index = mask nibble << 4 | bit nibble -> 4 bf16 of -1, 0, +1
        uint32_t h[4];
#pragma unroll
        for (uint32_t k = 0; k < 4; ++k)
            h[k] = ((tid >> (4 + k)) & 1u) ? (((tid >> k) & 1u) ? 0x3f80u : 0xbf80u) : 0u;
#pragma unroll
        for (uint32_t c = 0; c < LUT_COPIES; ++c)
            lut256[tid * LUT_COPIES + c] = make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
    }
    if (tid < ROWS) {
        // per-row scales and the table of all 2^n_q weight values (index bit i = plane i, bit 3 = mask)
        const uint64_t r = r0 + tid;
        float al[8];
#pragma unroll
        for (uint32_t i = 0; i < 8; ++i) {
            al[i] = (i < A.n_q && r < M.m) ? __ldg(M.alpha + r * A.n_q + i) : 0.0f;
            alpha_s[tid * 8 + i] = al[i];
        }
        for (uint32_t e = 0; e < 16; ++e) {
            float s = 0.0f;
            if (e & 8u) {
#pragma unroll
                for (uint32_t i = 0; i < 3; ++i)
                    if (i < A.n_q) s = __fadd_rn(s, ((e >> i) & 1u) ? al[i] : -al[i]);
            }
            lut[tid * 16 + e] = __float2bfloat16_rn(s);
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    uint32_t step_count = 0;                    // pipeline steps issued so far (all roles count alike)
    uint32_t macro_count = 0;                   // bit-buffer fills so far
    uint32_t accum_parity = 0;
    for (uint32_t bc = 0; bc < M.batch; bc += M.nbt) {
        const uint32_t step_begin = macro_begin * STEPS_PER_MACRO;
        uint32_t step_end = macro_end * STEPS_PER_MACRO;
        if (step_end > total_steps) step_end = total_steps;
        const uint32_t nsteps = step_end > step_begin ? step_end - step_begin : 0;
        const uint32_t nmacros = macro_end > macro_begin ? macro_end - macro_begin : 0;

        if (warp < DEC_WARPS) {
            // ------------------------------ decode warps ------------------------------
            uint32_t it = step_count, mi = macro_count;
            for (uint32_t mc = macro_begin; mc < macro_end; ++mc, ++mi) {
                const uint64_t c0 = (uint64_t)mc * MACRO;
                const uint32_t cnt = (uint32_t)(M.n - c0 < MACRO ? M.n - c0 : MACRO);
                const uint32_t buf = M.tma_bits ? (mi & 1u) : 0u;
                const uint32_t *rbb = rb + buf * rb_buf_words;
                bool stop = false;
                // phase 1: the bit vectors of the 128 rows x MACRO columns into the bit buffer
                if (M.tma_bits) {
                    // the TMA thread fetches them as 128 x 64-byte boxes; wait for this buffer
                    stop = !mbar_wait(bits_full + buf, (mi >> 1) & 1u, abort_flag, A.status);
                } else {
                    // planes exist as packed bits but rows are not 16-byte aligned: 16 consecutive
                    // lanes copy the 16 words of one row segment, 32 rows per pass
                    const uint32_t j = tid & 15;
#pragma unroll
                    for (uint32_t pass = 0; pass < ROWS / 32; ++pass) {
                        const uint32_t rl = pass * 32 + (tid >> 4);
                        const uint64_t rr = r0 + rl;
                        const uint64_t p0 = rr * M.n + c0;
                        const uint64_t w = (p0 >> 5) + j;
                        const uint32_t sh = (uint32_t)(p0 & 31);
                        const uint32_t lo = 32 * j;
                        uint32_t keep = 0;                        // bits of this word that lie in [0, cnt)
                        if (rr < M.m && lo < cnt) keep = lo + 32 > cnt ? (1u << (cnt - lo)) - 1u : 0xffffffffu;
                        for (uint32_t item = 0; item <= A.n_q; ++item) {
                            const uint32_t *src = item < A.n_q ? M.bits32 + (uint64_t)item * M.plane_words32 : M.mask32;
                            const uint64_t valid = item < A.n_q ? M.plane_words32 : M.mask_words32;
                            uint32_t v = 0;
                            if (keep) {
                                const uint32_t lo_w = w < valid ? __ldg(src + w) : 0u;
                                const uint32_t hi_w = w + 1 < valid ? __ldg(src + w + 1) : 0u;
                                v = __funnelshift_r(lo_w, hi_w, sh) & keep;
                            }
                            rb[(item * ROWS + rl) * rbp + j] = v;
                        }
                    }
                }
                if (!M.tma_bits) asm volatile("bar.sync 1, %0;\n" :: "n"(DEC_THREADS) : "memory");
                // phase 2: steps of 64 columns; one thread per (row, 16 columns)
                const uint32_t steps_here = stop ? 0u : (cnt + KC - 1) / KC;
                const uint32_t row = tid >> 2, quarter = tid & 3, sw = row & 7;
                const uint2 *lut_mine = lut256 + (lane & (LUT_COPIES - 1));
                for (uint32_t ks = 0; ks < steps_here; ++ks, ++it) {
                    const uint32_t stage = it % M.stages, use = it / M.stages;
                    // one lane per warp watches the barrier that frees the stage; the warp follows it
                    if (use > 0) {
                        uint32_t freed = 1;
                        if (lane == 0) freed = mbar_wait(empty + stage, (use - 1) & 1u, abort_flag, A.status) ? 1u : 0u;
                        if (!__shfl_sync(0xffffffffu, freed, 0)) break;
                    }
                    uint8_t *a_stage = a_stages + stage * a_stage_bytes;
                    const uint32_t wi = ks * 2 + (quarter >> 1), sh16 = (quarter & 1) * 16;
                    uint32_t mw = (rbb[(A.n_q * ROWS + row) * rbp + wi] >> sh16) & 0xffffu;
                    if (M.per_plane) {
                        // sign tiles, one per plane: -1 / 0 / +1 in bf16 (the scales are applied to
                        // the accumulators afterwards), four weights per table read
                        for (uint32_t i = 0; i < A.n_q; ++i) {
                            const uint32_t bw = (rbb[(i * ROWS + row) * rbp + wi] >> sh16) & 0xffffu;
                            uint2 e[4];
#pragma unroll
                            for (uint32_t q = 0; q < 4; ++q)
                                e[q] = lut_mine[((((mw >> (4 * q)) & 15u) << 4) | ((bw >> (4 * q)) & 15u)) * LUT_COPIES];
                            uint8_t *arow = a_stage + i * A_STAGE_BYTES + row * 128;
                            *reinterpret_cast<uint4 *>(arow + (((quarter * 2) ^ sw) << 4)) = make_uint4(e[0].x, e[0].y, e[1].x, e[1].y);
                            *reinterpret_cast<uint4 *>(arow + (((quarter * 2 + 1) ^ sw) << 4)) = make_uint4(e[2].x, e[2].y, e[3].x, e[3].y);
                        }
                    } else {
                        // one tile of rescaled weights: clear the thread's 32 bytes, then write only
                        // the unpruned positions (most are zero)
                        uint8_t *arow = a_stage + row * 128;
#pragma unroll
                        for (uint32_t q = 0; q < 2; ++q)
                            *reinterpret_cast<uint4 *>(arow + (((quarter * 2 + q) ^ sw) << 4)) = make_uint4(0, 0, 0, 0);
                        if (A.n_q <= 3) {
                            uint32_t bw[3];
#pragma unroll
                            for (uint32_t i = 0; i < 3; ++i)
                                bw[i] = i < A.n_q ? rbb[(i * ROWS + row) * rbp + wi] >> sh16 : 0u;
                            const uint16_t *lr = reinterpret_cast<const uint16_t *>(lut) + row * 16;
                            while (mw) {
                                const uint32_t k = 31u - (uint32_t)__clz((int)mw);
                                mw ^= 1u << k;
                                const uint32_t e = 8u | ((bw[0] >> k) & 1u) | (((bw[1] >> k) & 1u) << 1) |
                                                   (((bw[2] >> k) & 1u) << 2);
                                *reinterpret_cast<uint16_t *>(arow + (((quarter * 2 + (k >> 3)) ^ sw) << 4) + (k & 7) * 2) = lr[e];
                            }
                        } else {
                            while (mw) {
                                const uint32_t k = 31u - (uint32_t)__clz((int)mw);
                                mw ^= 1u << k;
                                float sum = 0.0f;
                                for (uint32_t i = 0; i < A.n_q; ++i) {
                                    const float a = alpha_s[row * 8 + i];
                                    sum = __fadd_rn(sum, ((rbb[(i * ROWS + row) * rbp + wi] >> (sh16 + k)) & 1u) ? a : -a);
                                }
                                *reinterpret_cast<uint16_t *>(arow + (((quarter * 2 + (k >> 3)) ^ sw) << 4) + (k & 7) * 2) =
                                    __bfloat16_as_ushort(__float2bfloat16_rn(sum));
                            }
                        }
                    }
                    fence_async_smem();                 // generic-proxy writes -> visible to the tensor core
                    __syncwarp();
                    if (lane == 0) mbar_arrive(full_a + stage);     // the warp's 32 row segments are in place
                }
                __syncwarp();
                if (M.tma_bits && lane == 0) mbar_arrive(bits_empty + buf);   // this warp is done with the buffer
                if (decode_barrier_any(*abort_flag)) break;       // same decision in every decode thread
            }
        } else if (warp == DEC_WARPS) {
            // ------------------------------ TMA producer ------------------------------
            if (lane == 0) {
                uint32_t it = step_count, mi = macro_count;
                bool ok = true;
                auto fetch_bits = [&](uint32_t mc, uint32_t mix) {
                    const uint32_t buf = mix & 1u, useb = mix >> 1;
                    if (useb > 0 && !mbar_wait(bits_empty + buf, (useb - 1) & 1u, abort_flag, A.status)) return false;
                    uint8_t *dst = reinterpret_cast<uint8_t *>(rb + buf * rb_buf_words);
                    mbar_expect_tx(bits_full + buf, n_items * ROWS * 64);
                    for (uint32_t i = 0; i < A.n_q; ++i)
                        tma_load_3d(dst + i * ROWS * 64, &pmap, bits_full + buf, (int32_t)(mc * (MACRO / 8)), (int32_t)r0, (int32_t)i);
                    tma_load_2d(dst + A.n_q * ROWS * 64, &kmap, bits_full + buf, (int32_t)(mc * (MACRO / 8)), (int32_t)r0);
                    return true;
                };
                if (M.tma_bits && nmacros) ok = fetch_bits(macro_begin, mi);
                for (uint32_t mc = macro_begin; mc < macro_end && ok; ++mc, ++mi) {
                    if (M.tma_bits && mc + 1 < macro_end) ok = fetch_bits(mc + 1, mi + 1);
                    uint32_t st_lo = mc * STEPS_PER_MACRO, st_hi = st_lo + STEPS_PER_MACRO;
                    if (st_hi > step_end) st_hi = step_end;
                    for (uint32_t st = st_lo; st < st_hi && ok; ++st, ++it) {
                        const uint32_t stage = it % M.stages, use = it / M.stages;
                        if (use > 0 && !mbar_wait(empty + stage, (use - 1) & 1u, abort_flag, A.status)) { ok = false; break; }
                        uint8_t *b_stage = b_stages + (size_t)stage * M.b_stage_bytes;
                        mbar_expect_tx(full_b + stage, M.b_stage_bytes);
                        for (uint32_t h = 0; h * 256 < M.nbt; ++h)
                            tma_load_2d(b_stage + h * 256 * 128, &xmap, full_b + stage, (int32_t)(st * KC),
                                        (int32_t)(bc + h * 256));
                    }
                }
            }
        } else {
            // ------------------------------ MMA issuer ------------------------------
            if (lane == 0) {
                uint32_t it = step_count;
                const uint32_t nmma = M.nbt > 256 ? 2 : 1;
                const uint32_t ncols = M.nbt > 256 ? 256 : M.nbt;
                const uint32_t idesc = instr_desc_bf16(ncols);
                // descriptors differ only in the start-address field (units of 16 bytes): keep the
                // constant part and add offsets, so that issuing an MMA costs a few instructions
                const uint64_t a_desc0 = smem_desc_sw128(smem_addr(a_stages));
                const uint64_t b_desc0 = smem_desc_sw128(smem_addr(b_stages));
                const uint32_t a_stage16 = a_stage_bytes >> 4, b_stage16 = M.b_stage_bytes >> 4;
                bool ok = true;
                uint32_t acc = 0;                       // 0 for the very first MMA of every accumulator
                for (uint32_t st = step_begin; st < step_end && ok; ++st, ++it) {
                    const uint32_t stage = it % M.stages, use = it / M.stages;
                    ok = mbar_wait(full_a + stage, use & 1u, abort_flag, A.status) &&
                         mbar_wait(full_b + stage, use & 1u, abort_flag, A.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t a_desc = a_desc0 + (uint64_t)(stage * a_stage16);
                    const uint64_t b_desc = b_desc0 + (uint64_t)(stage * b_stage16);
                    for (uint32_t t = 0; t < a_tiles; ++t) {
                        for (uint32_t h = 0; h < nmma; ++h) {
                            const uint32_t d = tmem_base + t * M.nbt + h * 256;
                            const uint64_t ad = a_desc + (uint64_t)(t * (A_STAGE_BYTES >> 4));
                            const uint64_t bd = b_desc + (uint64_t)(h * (256 * 128 >> 4));
                            mma_bf16(d, ad, bd, idesc, acc);
#pragma unroll
                            for (uint32_t k16 = 1; k16 < KC / 16; ++k16)
                                mma_bf16(d, ad + 2 * k16, bd + 2 * k16, idesc, 1u);
                        }
                    }
                    acc = 1;
                    mma_commit(empty + stage);          // frees the stage when these MMAs are done
                }
                if (ok && nsteps) mma_commit(accum);
            }
        }
        step_count += nsteps;
        macro_count += nmacros;

        // ------------------------------ epilogue ------------------------------
        if (warp < DEC_WARPS && nsteps) {
            const bool ready = mbar_wait(accum, accum_parity, abort_flag, A.status);
            if (__all_sync(0xffffffffu, ready)) {                  // tcgen05.ld needs the whole warp
                tc_fence_after();
                const uint32_t quad = warp & 3, part = warp >> 2;       // TMEM lane quarter, column class
                const uint32_t rl = quad * 32 + lane;
                const uint64_t r = r0 + rl;
                for (uint32_t c = part * 8; c < M.nbt; c += 8 * (DEC_WARPS / 4)) {
                    float out[8];
                    if (M.per_plane) {
                        // Y = sum over planes of alpha[r][i] * (sign tile i . X)
#pragma unroll
                        for (uint32_t e = 0; e < 8; ++e) out[e] = 0.0f;
                        for (uint32_t i = 0; i < A.n_q; ++i) {
                            uint32_t v[8];
                            tmem_ld8(tmem_base + ((quad * 32) << 16) + i * M.nbt + c, v);
                            const float a = alpha_s[rl * 8 + i];
#pragma unroll
                            for (uint32_t e = 0; e < 8; ++e) out[e] = fmaf(a, __uint_as_float(v[e]), out[e]);
                        }
                    } else {
                        uint32_t v[8];
                        tmem_ld8(tmem_base + ((quad * 32) << 16) + c, v);
#pragma unroll
                        for (uint32_t e = 0; e < 8; ++e) out[e] = __uint_as_float(v[e]);
                    }
                    if (r < M.m) {
#pragma unroll
                        for (uint32_t e = 0; e < 8; ++e)
                            if (bc + c + e < M.batch)
                                atomicAdd(M.y + (int64_t)(bc + c + e) * M.ldy + r, out[e]);
                    }
                }
            }
        }
        if (nsteps) accum_parity ^= 1;
        tc_fence_before();
        __syncthreads();                       // accumulators are read before the next pass overwrites them
        tc_fence_after();
    }
    if (warp == DEC_WARPS + 1) tmem_dealloc(tmem_base, M.tmem_cols);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

}  // namespace

// Workspace of the two-stage form: the decoded planes as packed bits (1 bit per weight and plane).
size_t mma_workspace_bytes(const sqnn_desc *desc, uint32_t)
{
    const uint64_t words64 = (desc->m * desc->n + 63) / 64;
    return (size_t)((desc->n_q * words64 * 8 + 255) / 256 * 256);
}

int mma_dispatch(const sqnn_desc *desc, const DecodeArgs &A0, const uint64_t *d_mask, const float *d_alpha,
                 const void *d_x, int64_t ldx, uint32_t batch, float *d_y, int64_t ldy, void *d_workspace,
                 cudaStream_t st)
{
    if (((uintptr_t)d_x & 15) != 0 || (ldx % 8) != 0) return SQNN_E_UNSUPPORTED;   // TMA: 16-byte base and pitch
    if (desc->n > 0x7fffffffull || batch > 0x7fffffffu) return SQNN_E_UNSUPPORTED;
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return SQNN_E_CUDA;

    MmaArgs M;
    M.A = A0;
    M.mask32 = (const uint32_t *)d_mask;
    M.mask_words32 = M.A.words64 * 2;
    M.alpha = d_alpha;
    M.y = d_y;
    M.ldy = ldy;
    M.m = desc->m;
    M.n = desc->n;
    M.batch = batch;
    // One sign tile and one accumulator per plane, scales applied to the accumulators: the weights stay
    // exact.  (One tile of rescaled weights rounded to bf16 is not an option: a row holds only 2^n_q
    // distinct values, their rounding errors add up coherently, and the result misses the 1e-2 tolerance
    // on wide layers.)  The n_q accumulators of a pass must fit the 512 columns of tensor memory, so the
    // batch is taken in passes of at most 512 / n_q columns.
    const uint32_t b16 = (batch + 15) / 16 * 16;
    const uint32_t cap = (512u / M.A.n_q) / 16 * 16;
    M.nbt = b16 < cap ? b16 : cap;
    if (M.nbt > 256) M.nbt = 512;                       // one plane: two full 256-column MMAs per step
    M.b_stage_bytes = M.nbt * 128;
    M.bits32 = (const uint32_t *)d_workspace;
    M.plane_words32 = M.A.words64 * 2;
    M.per_plane = 1u;
    // The bit buffer is filled by TMA when the rows of the packed planes start on 16-byte boundaries.
    M.tma_bits = (desc->n % 128 == 0 && ((uintptr_t)d_mask & 15) == 0) ? 1u : 0u;
    const size_t budget = 225 * 1024;        // + 1 KB of static shared memory stays within the 227 KB a block may have
    size_t fixed = 0, per_stage = 0;
    for (;;) {
        M.rbp = M.tma_bits ? 16 : RB_WORDS;
        M.rb_bufs = M.tma_bits ? 2 : 1;
        const uint32_t a_tiles = M.per_plane ? M.A.n_q : 1;
        M.tmem_cols = 32;
        while (M.tmem_cols < a_tiles * M.nbt) M.tmem_cols *= 2;
        fixed = (size_t)M.rb_bufs * (M.A.n_q + 1) * ROWS * M.rbp * 4 +
                256 * 8 * LUT_COPIES + ROWS * 16 * 2 +
                ROWS * 8 * 4 + (3 * MAX_STAGES + 5) * 8 + 16 + 1024;
        per_stage = (size_t)a_tiles * A_STAGE_BYTES + M.b_stage_bytes;
        if (fixed + 2 * per_stage <= budget) break;
        if (M.tma_bits) { M.tma_bits = 0; continue; }          // single bit buffer
        if (M.per_plane) { M.per_plane = 0; continue; }        // too many planes for two stages
        break;
    }
    M.stages = MAX_STAGES;
    while (M.stages > 1 && fixed + (size_t)M.stages * per_stage > budget) --M.stages;
    const size_t smem = fixed + (size_t)M.stages * per_stage;
    if (smem > budget) return SQNN_E_UNSUPPORTED;

    const uint32_t row_tiles = (uint32_t)((desc->m + ROWS - 1) / ROWS);
    const uint32_t total_macros = (uint32_t)((desc->n + MACRO - 1) / MACRO);
    uint32_t splits = (uint32_t)sm_count() / row_tiles;
    if (splits < 1) splits = 1;
    if (splits > total_macros) splits = total_macros;
    M.macros_per_split = (total_macros + splits - 1) / splits;
    M.splits = (total_macros + M.macros_per_split - 1) / M.macros_per_split;

    CUtensorMap xmap, pmap, kmap;
    const cuuint64_t gdim[2] = {(cuuint64_t)desc->n, (cuuint64_t)batch};
    const cuuint64_t gstride[1] = {(cuuint64_t)ldx * 2};
    const cuuint32_t box[2] = {KC, M.nbt > 256 ? 256u : M.nbt};
    const cuuint32_t estride[3] = {1, 1, 1};
    if (encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(d_x), gdim, gstride, box, estride,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return SQNN_E_CUDA;
    pmap = xmap;
    kmap = xmap;
    if (M.tma_bits) {
        // packed planes as bytes: [plane][row][n / 8], and the mask [row][n / 8]; boxes of 128 rows x 64 bytes
        const cuuint64_t pdim[3] = {(cuuint64_t)(desc->n / 8), (cuuint64_t)desc->m, (cuuint64_t)M.A.n_q};
        const cuuint64_t pstride[2] = {(cuuint64_t)(desc->n / 8), (cuuint64_t)(M.A.words64 * 8)};
        const cuuint32_t pbox[3] = {MACRO / 8, ROWS, 1};
        if (encode(&pmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, d_workspace, pdim, pstride, pbox, estride,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            encode(&kmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint64_t *>(d_mask), pdim, pstride, pbox, estride,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return SQNN_E_CUDA;
    }

    cudaError_t e = (ldy == (int64_t)desc->m)
        ? cudaMemsetAsync(d_y, 0, (size_t)batch * desc->m * sizeof(float), st)
        : cudaMemset2DAsync(d_y, (size_t)ldy * sizeof(float), 0, (size_t)desc->m * sizeof(float), batch, st);
    if (e != cudaSuccess) return SQNN_E_CUDA;
    if (ensure_dynamic_smem(reinterpret_cast<const void *>(k_decode_mma), smem) != SQNN_OK) return SQNN_E_CUDA;
    // stage 1: the decode kernel writes the planes as packed bits into the workspace
    const int rc = decode_bits_dispatch(A0, d_workspace, st);
    if (rc != SQNN_OK) return rc;
    k_decode_mma<<<row_tiles * M.splits, THREADS, smem, st>>>(xmap, pmap, kmap, M);
    return cudaGetLastError() == cudaSuccess ? SQNN_OK : SQNN_E_CUDA;
}

}  // namespace sqnn

// ---------------------------------------------------------------------------------------------
// Tensor-core product for callers that must not allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a stream capture, inside
// a framework that owns the whole device heap through its own pool, or in a serving loop whose
// memory plan is frozen at start-up.  For them the scratch that sqnn_decode_matmul takes from
// the caller (the decoded planes as packed bits) lives in the array below, which is part of the
// loaded library image on every GPU that loads it, for as long as the process lives.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char sqnn_static_scratch[SQNN_STATIC_SCRATCH_BYTES];

namespace {

// In host code `sqnn_static_scratch` is only a handle for the runtime, not a device address, so
// the address is asked for once per device (with that device current) and remembered.
int static_scratch_address(void **out)
{
    static std::mutex mu;
    static void *addr[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SQNN_E_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, sqnn_static_scratch) != cudaSuccess || !p) return SQNN_E_CUDA;
        addr[dev] = p;
    }
    *out = addr[dev];
    return SQNN_OK;
}

}  // namespace

extern "C" int sqnn_decode_matmul_static(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
                                         const float *d_alpha, const void *d_x, int x_dtype, uint32_t batch,
                                         int64_t ldx, float *d_y, int64_t ldy, uint32_t *d_status,
                                         void *cuda_stream)
{
    sqnn::DecodeArgs A;
    int rc = sqnn::fill_decode_args(desc, d_blob, d_status, &A);
    if (rc != SQNN_OK) return rc;
    if (!d_mask || !d_alpha || !d_x || !d_y || batch == 0) return SQNN_E_INVALID_ARG;
    if (ldx < (int64_t)desc->n || ldy < (int64_t)desc->m) return SQNN_E_INVALID_ARG;
    if (((uintptr_t)d_mask & 7) || ((uintptr_t)d_alpha & 3) || ((uintptr_t)d_y & 3)) return SQNN_E_INVALID_ARG;
    if (x_dtype != SQNN_X_BF16 || batch < 16 || batch > SQNN_MAX_BATCH || desc->n > (1ull << 30))
        return SQNN_E_UNSUPPORTED;
    if (sqnn::mma_workspace_bytes(desc, batch) > SQNN_STATIC_SCRATCH_BYTES) return SQNN_E_WORKSPACE;
    void *scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != SQNN_OK) return rc;
    // Nothing in the scratch has to start at zero: the decode stage overwrites every word the
    // product stage reads.  Y is cleared by the product path itself.
    return sqnn::mma_dispatch(desc, A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, scratch,
                              (cudaStream_t)cuda_stream);
}
