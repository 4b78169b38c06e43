// K4: decryption fused with the product for batch >= 16 on the 5th-generation tensor cores.
//
//   Y[b][r] = sum_i alpha[r][i] * sum_c s_i[r][c] X[b][c],      s_i = mask * (2 b_i - 1) in {-1, 0, +1}
//
//   D (TMEM, fp32) [128 batch rows x 256 weight rows] += A (shared, bf16, K-major) [128 x 64] . B (shared) [256 x 64]^T
//
// One CTA owns 256 rows of W of ONE plane and a range of columns.  Per 64-column step
//   - one thread fetches the activations X[bc .. bc+128) x [64 columns] with TMA into the A stage (every CTA
//     fetches its own tile; rows past the batch are filled with zeros by the copy engine);
//   - the decode warps expand the plane's sign tile -1 / 0 / +1 (mask and sign only, four weights per table
//     read) into the B stage (bf16, 128-byte rows, 128-byte swizzle) -- the expanded weights exist only in
//     shared memory;
//   - one thread issues tcgen05.mma (M = 128, N = 256, K = 16 each) that accumulate in tensor memory, never
//     twice in a row into the same accumulator.
// A tcgen05.mma of M = 128 takes about as long whatever its N, so the weight rows sit on the N side at the
// full N = 256.  The scale alpha[r][i] is applied to the accumulator in the epilogue, so the weights stay
// exact (one tile of rescaled weights rounded to bf16 would not meet the tolerance: a row has only 2^n_q
// distinct values and their rounding errors add up coherently).  Planes and column ranges of different CTAs
// are summed with fp32 vector reductions on Y (cleared beforehand).  Batches beyond 128 are taken 128 rows
// at a time, two accumulators (256 batch rows) per pass over the columns.
//
// Where the bits come from.  The planes have been decoded to packed bits in the workspace by the tiled
// decode kernel (queued just before this one) and sit in L2.  A decode thread owns (row, half of a 64-column
// step); when rows start on 16-byte boundaries it takes the bits of 256 columns with one 16-byte load per
// vector (plane, mask) and trades words with its neighbour by shuffle, otherwise it reads word by word.
//
// Every wait on an mbarrier is bounded; a wait that gives up sets SQNN_E_TIMEOUT in the status word and
// makes all roles leave their loops, so the kernel always frees its tensor memory and returns.
#include "sqnn_launch.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <mutex>

namespace sqnn {

namespace {

constexpr uint32_t NROWS = 256;           // rows of W per CTA = MMA N
constexpr uint32_t MB = 128;              // batch rows per accumulator = MMA M
constexpr uint32_t KC = 64;               // columns per pipeline step
constexpr uint32_t MACRO = 256;           // columns whose bits a decode thread takes at a time
constexpr uint32_t STEPS_PER_MACRO = MACRO / KC;
constexpr uint32_t LUT_COPIES = 16;       // copies of the 256-entry sign table: lane l of a half-warp reads copy l
constexpr uint32_t DEC_WARPS = 16;
constexpr uint32_t DEC_THREADS = DEC_WARPS * 32;
constexpr uint32_t THREADS = DEC_THREADS + 64;  // + TMA warp + MMA warp
constexpr uint32_t B_STAGE_BYTES = NROWS * KC * 2;
constexpr uint32_t A_TILE_BYTES = MB * KC * 2;
constexpr uint32_t MAX_STAGES = 4;
constexpr uint64_t WAIT_LIMIT_CYCLES = 4000000000ull;   // about 2 s at 2 GHz

// Set by sqnn_set_debug_flags (for the library's own tests).
std::atomic<uint32_t> g_debug_flags{0};
std::atomic<uint64_t> g_debug_wait_cycles{0};

struct MmaArgs {
    const uint32_t *bits32;       // decoded planes in the workspace
    uint64_t plane_words32;       // 32-bit words per plane in the workspace
    const uint32_t *mask32;
    uint64_t mask_words32;        // number of valid 32-bit mask words
    const float *alpha;
    float *y;
    int64_t ldy;
    uint64_t m, n;
    uint32_t n_q;
    uint32_t batch;
    uint32_t nchunks;             // accumulators (128 batch rows each) per pass: 1 or 2
    uint32_t stages;
    uint32_t splits;              // CTAs per (row tile, plane)
    uint32_t macros_per_split;
    uint32_t aligned;             // 1: rows of the packed vectors start on 16-byte boundaries
    uint32_t vec_y;               // 1: Y rows allow 16-byte vector reductions
    uint32_t skip_loads;          // test only: the TMA role issues no loads
    uint64_t wait_limit;          // cycles a bounded wait may take
    uint32_t *status;
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
SQNN_DEV bool mbar_wait(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status, uint64_t limit)
{
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((uint64_t)(clock64() - t0) > limit) {
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
// 32 consecutive accumulator columns of this thread's lane (one wait for the whole load).
SQNN_DEV void tmem_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}
SQNN_DEV void red_add_v4(float *gdst, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};\n" :: "l"(gdst), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
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
    return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((MB >> 4) << 24);
}

// Barrier over the decode threads that also ORs a flag, so that all of them take the same exit.
SQNN_DEV bool decode_barrier_any(uint32_t flagged)
{
    uint32_t any;
    asm volatile("{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, 1, %2, q;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(any) : "r"(flagged), "n"(DEC_THREADS) : "memory");
    return any != 0;
}

// 32 bits of a packed vector starting at bit position p (words past `valid` read as zero).
SQNN_DEV uint32_t bits_at(const uint32_t *__restrict__ src, uint64_t valid, uint64_t p)
{
    const uint64_t w = p >> 5;
    const uint32_t sh = (uint32_t)(p & 31);
    const uint32_t lo = w < valid ? __ldg(src + w) : 0u;
    const uint32_t hi = (sh != 0 && w + 1 < valid) ? __ldg(src + w + 1) : 0u;
    return __funnelshift_r(lo, hi, sh);
}

__global__ void __launch_bounds__(THREADS, 1)
k_decode_mma(const __grid_constant__ CUtensorMap xmap, const MmaArgs M)
{
    extern __shared__ __align__(16) uint8_t smem_raw[];
    // carve shared memory (A / B stages need 1024-byte alignment for the 128-byte swizzle)
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *b_stages = base;                                               // [stage][256 rows][128 B]
    const uint32_t a_stage_bytes = M.nchunks * A_TILE_BYTES;
    uint8_t *a_stages = b_stages + M.stages * B_STAGE_BYTES;                 // [stage][chunk][128 rows][128 B]
    uint2 *lut256 = reinterpret_cast<uint2 *>(a_stages + M.stages * a_stage_bytes);   // [256][LUT_COPIES]
    float *alpha_s = reinterpret_cast<float *>(lut256 + 256 * LUT_COPIES);  // [256]
    uint64_t *bars = reinterpret_cast<uint64_t *>(alpha_s + NROWS);
    uint64_t *full_a = bars, *full_b = bars + MAX_STAGES, *empty = bars + 2 * MAX_STAGES;
    uint64_t *accum = bars + 3 * MAX_STAGES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(accum + 1);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // work item: (row tile, plane, column range)
    const uint32_t split = blockIdx.x % M.splits;
    const uint32_t plane = (blockIdx.x / M.splits) % M.n_q;
    const uint32_t row_tile = blockIdx.x / (M.splits * M.n_q);
    const uint64_t r0 = (uint64_t)row_tile * NROWS;
    const uint32_t total_macros = (uint32_t)((M.n + MACRO - 1) / MACRO);
    const uint32_t macro_begin = split * M.macros_per_split;
    const uint32_t macro_end = macro_begin + M.macros_per_split < total_macros ? macro_begin + M.macros_per_split : total_macros;
    const uint32_t total_steps = (uint32_t)((M.n + KC - 1) / KC);
    const uint32_t step_begin = macro_begin * STEPS_PER_MACRO;
    const uint32_t step_end = macro_end * STEPS_PER_MACRO < total_steps ? macro_end * STEPS_PER_MACRO : total_steps;
    const uint32_t nsteps = step_end > step_begin ? step_end - step_begin : 0;
    // Two accumulators always: with two batch chunks one per chunk; with one chunk the K = 16 slices
    // alternate between them and the epilogue adds them up.  (Measured: a tcgen05.mma that accumulates
    // into the accumulator of the one before it is issued about 300 cycles after it at N = 256; when
    // consecutive ones go to different accumulators the spacing is about 160 cycles.)
    const uint32_t tmem_cols = 2 * NROWS;

    if (tid == 0) {
        for (uint32_t s = 0; s < MAX_STAGES; ++s) {
            mbar_init(full_b + s, DEC_WARPS);        // one arrival per decode warp
            mbar_init(full_a + s, 1);
            mbar_init(empty + s, 1);
        }
        mbar_init(accum, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == DEC_WARPS + 1) tmem_alloc(tmem_slot, tmem_cols);
    if (tid < 256) {
        // 4 weights at a time: index = mask nibble << 4 | bit nibble -> 4 bf16 of -1, 0, +1
        uint32_t h[4];
#pragma unroll
        for (uint32_t k = 0; k < 4; ++k)
            h[k] = ((tid >> (4 + k)) & 1u) ? (((tid >> k) & 1u) ? 0x3f80u : 0xbf80u) : 0u;
#pragma unroll
        for (uint32_t c = 0; c < LUT_COPIES; ++c)
            lut256[tid * LUT_COPIES + c] = make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
    } else if (tid < 256 + NROWS) {
        const uint64_t r = r0 + (tid - 256);
        alpha_s[tid - 256] = r < M.m ? __ldg(M.alpha + r * M.n_q + plane) : 0.0f;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    uint32_t step_count = 0;                    // pipeline steps issued so far (all roles count alike)
    uint32_t accum_parity = 0;
    for (uint32_t bc = 0; bc < M.batch; bc += MB * M.nchunks) {
        if (warp < DEC_WARPS) {
            // ------------------------------ decode warps ------------------------------
            // thread = (row, half): 32 columns of a 64-column step; two threads of a row are neighbours
            const uint32_t row = tid >> 1, half = tid & 1, sw = row & 7;
            const uint64_t r = r0 + row;
            const bool live = r < M.m;
            const uint32_t *src_b = M.bits32 + (uint64_t)plane * M.plane_words32;
            const uint2 *lut_mine = lut256 + (lane & (LUT_COPIES - 1));
            // shared addresses: this row inside stage 0, its four 16-byte chunks (swizzled), this lane's table copy
            const uint32_t brow0 = smem_addr(b_stages) + (row >> 3) * 1024 + sw * 128;
            uint32_t chunk_off[4];
#pragma unroll
            for (uint32_t j = 0; j < 4; ++j) chunk_off[j] = ((half * 4 + j) ^ sw) << 4;
            const uint32_t lut_sa = smem_addr(lut_mine);
            uint32_t stage = step_count % M.stages, use = step_count / M.stages;       // advanced step by step below
            bool stop = false;
            // bits of the current macro: aligned rows -> 4 words of this thread's 128 columns per vector
            uint4 cur_m = make_uint4(0, 0, 0, 0), cur_b = make_uint4(0, 0, 0, 0);
            auto fetch_macro = [&](uint32_t mc, uint4 &vm, uint4 &vb) {
                vm = vb = make_uint4(0, 0, 0, 0);
                const uint64_t c = (uint64_t)mc * MACRO + 128 * half;       // first column of this thread's 128
                if (live && c < M.n) {
                    const uint64_t w = (r * M.n + c) >> 5;                  // a multiple of 4
                    if (w + 4 <= M.mask_words32) vm = ldg_ahead(reinterpret_cast<const uint4 *>(M.mask32 + w));
                    else {
                        vm.x = w < M.mask_words32 ? __ldg(M.mask32 + w) : 0u;
                        vm.y = w + 1 < M.mask_words32 ? __ldg(M.mask32 + w + 1) : 0u;
                        vm.z = w + 2 < M.mask_words32 ? __ldg(M.mask32 + w + 2) : 0u;
                    }
                    if (w + 4 <= M.plane_words32) vb = ldg_ahead(reinterpret_cast<const uint4 *>(src_b + w));
                    else {
                        vb.x = w < M.plane_words32 ? __ldg(src_b + w) : 0u;
                        vb.y = w + 1 < M.plane_words32 ? __ldg(src_b + w + 1) : 0u;
                        vb.z = w + 2 < M.plane_words32 ? __ldg(src_b + w + 2) : 0u;
                    }
                }
            };
            if (M.aligned && macro_begin < macro_end) fetch_macro(macro_begin, cur_m, cur_b);
            for (uint32_t mc = macro_begin; mc < macro_end && !stop; ++mc) {
                // take delivery of this macro's bits before the next macro's are requested (a warp's few
                // scoreboards are shared between loads: a first use after the new request would wait for it)
                cur_m.x = settle(cur_m.x); cur_m.y = settle(cur_m.y); cur_m.z = settle(cur_m.z); cur_m.w = settle(cur_m.w);
                cur_b.x = settle(cur_b.x); cur_b.y = settle(cur_b.y); cur_b.z = settle(cur_b.z); cur_b.w = settle(cur_b.w);
                uint4 nxt_m = make_uint4(0, 0, 0, 0), nxt_b = make_uint4(0, 0, 0, 0);
                if (M.aligned && mc + 1 < macro_end) fetch_macro(mc + 1, nxt_m, nxt_b);
                const uint32_t st_lo = mc * STEPS_PER_MACRO;
#pragma unroll
                for (uint32_t ks = 0; ks < STEPS_PER_MACRO; ++ks) {
                    if (st_lo + ks >= step_end || stop) continue;           // the same in every thread
                    // mask and sign word of this thread's 32 columns
                    uint32_t mw, bw;
                    if (M.aligned) {
                        // words 2 ks and 2 ks + 1 of the macro: the lower four live in the half-0 thread,
                        // the upper four in the half-1 thread; the neighbour hands over the one this thread lacks
                        const uint32_t am[4] = {cur_m.x, cur_m.y, cur_m.z, cur_m.w};
                        const uint32_t ab[4] = {cur_b.x, cur_b.y, cur_b.z, cur_b.w};
                        const uint32_t m0 = am[(2 * ks) & 3u], m1 = am[(2 * ks + 1) & 3u];      // compile-time picks
                        const uint32_t b0 = ab[(2 * ks) & 3u], b1 = ab[(2 * ks + 1) & 3u];
                        const uint32_t gm = __shfl_xor_sync(0xffffffffu, half ? m0 : m1, 1);
                        const uint32_t gb = __shfl_xor_sync(0xffffffffu, half ? b0 : b1, 1);
                        const bool mine = half == (ks >> 1);                // the owner of words 2 ks, 2 ks + 1
                        mw = mine ? (half ? m1 : m0) : gm;
                        bw = mine ? (half ? b1 : b0) : gb;
                    } else {
                        const uint64_t c = (uint64_t)(st_lo + ks) * KC + 32 * half;
                        mw = bw = 0;
                        if (live && c < M.n) {
                            mw = bits_at(M.mask32, M.mask_words32, r * M.n + c);
                            bw = bits_at(src_b, M.plane_words32, r * M.n + c);
                        }
                    }
                    // table indices (mask nibble << 4 | sign nibble) of the eight groups of four weights, one per
                    // byte: byte j of `lo` for weights 8j .. 8j+3, byte j of `hi` for weights 8j+4 .. 8j+7
                    const uint32_t lo = ((mw & 0x0f0f0f0fu) << 4) | (bw & 0x0f0f0f0fu);
                    const uint32_t hi = (mw & 0xf0f0f0f0u) | ((bw >> 4) & 0x0f0f0f0fu);
                    uint2 e[8];
#pragma unroll
                    for (uint32_t j = 0; j < 4; ++j) {
                        const uint32_t a0 = lut_sa + ((lo >> (8 * j)) & 0xffu) * (LUT_COPIES * 8);
                        const uint32_t a1 = lut_sa + ((hi >> (8 * j)) & 0xffu) * (LUT_COPIES * 8);
                        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(e[2 * j].x), "=r"(e[2 * j].y) : "r"(a0));
                        asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(e[2 * j + 1].x), "=r"(e[2 * j + 1].y) : "r"(a1));
                    }
                    // one lane per warp watches the barrier that frees the stage; the warp follows it
                    if (use > 0) {
                        uint32_t freed = 1;
                        if (lane == 0) freed = mbar_wait(empty + stage, (use - 1) & 1u, abort_flag, M.status, M.wait_limit) ? 1u : 0u;
                        if (!__shfl_sync(0xffffffffu, freed, 0)) { stop = true; continue; }
                    }
                    const uint32_t brow = brow0 + stage * B_STAGE_BYTES;
#pragma unroll
                    for (uint32_t j = 0; j < 4; ++j)                        // 8 weights = one 16-byte chunk
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};"
                                     :: "r"(brow + chunk_off[j]), "r"(e[2 * j].x), "r"(e[2 * j].y), "r"(e[2 * j + 1].x), "r"(e[2 * j + 1].y) : "memory");
                    fence_async_smem();                 // generic-proxy writes -> visible to the tensor core
                    __syncwarp();
                    if (lane == 0) mbar_arrive(full_b + stage);     // the warp's 16 rows are in place
                    if (++stage == M.stages) { stage = 0; ++use; }
                }
                cur_m = nxt_m;
                cur_b = nxt_b;
                // a warp that gave up makes every decode thread leave at the same macro
                if (decode_barrier_any(stop || *abort_flag)) stop = true;
            }
        } else if (warp == DEC_WARPS) {
            // ------------------------------ TMA producer ------------------------------
            if (lane == 0 && !M.skip_loads) {
                uint32_t it = step_count;
                for (uint32_t st = step_begin; st < step_end; ++st, ++it) {
                    const uint32_t stage = it % M.stages, use = it / M.stages;
                    if (use > 0 && !mbar_wait(empty + stage, (use - 1) & 1u, abort_flag, M.status, M.wait_limit)) break;
                    uint8_t *a_stage = a_stages + (size_t)stage * a_stage_bytes;
                    mbar_expect_tx(full_a + stage, a_stage_bytes);
                    for (uint32_t c = 0; c < M.nchunks; ++c)
                        tma_load_2d(a_stage + c * A_TILE_BYTES, &xmap, full_a + stage, (int32_t)(st * KC), (int32_t)(bc + c * MB));
                }
            }
        } else {
            // ------------------------------ MMA issuer ------------------------------
            if (lane == 0) {
                uint32_t it = step_count;
                const uint32_t idesc = instr_desc_bf16(NROWS);
                // descriptors differ only in the start-address field (units of 16 bytes): keep the
                // constant part and add offsets, so that issuing an MMA costs a few instructions
                const uint64_t a_desc0 = smem_desc_sw128(smem_addr(a_stages));
                const uint64_t b_desc0 = smem_desc_sw128(smem_addr(b_stages));
                bool ok = true;
                uint32_t acc = 0;                       // 0 for the very first MMA of every accumulator
                for (uint32_t st = step_begin; st < step_end && ok; ++st, ++it) {
                    const uint32_t stage = it % M.stages, use = it / M.stages;
                    ok = mbar_wait(full_b + stage, use & 1u, abort_flag, M.status, M.wait_limit) &&
                         mbar_wait(full_a + stage, use & 1u, abort_flag, M.status, M.wait_limit);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t a_desc = a_desc0 + (uint64_t)(stage * (a_stage_bytes >> 4));
                    const uint64_t b_desc = b_desc0 + (uint64_t)(stage * (B_STAGE_BYTES >> 4));
                    if (M.nchunks == 2) {
#pragma unroll
                        for (uint32_t k16 = 0; k16 < KC / 16; ++k16)
#pragma unroll
                            for (uint32_t c = 0; c < 2; ++c)
                                mma_bf16(tmem_base + c * NROWS, a_desc + (uint64_t)(c * (A_TILE_BYTES >> 4)) + 2 * k16,
                                         b_desc + 2 * k16, idesc, (acc | k16) ? 1u : 0u);
                    } else {
#pragma unroll
                        for (uint32_t k16 = 0; k16 < KC / 16; ++k16)
                            mma_bf16(tmem_base + (k16 & 1u) * NROWS, a_desc + 2 * k16, b_desc + 2 * k16, idesc,
                                     (acc | (k16 >> 1)) ? 1u : 0u);
                    }
                    acc = 1;
                    mma_commit(empty + stage);          // frees the stage when these MMAs are done
                }
                if (ok && nsteps) mma_commit(accum);
            }
        }
        step_count += nsteps;

        // ------------------------------ epilogue ------------------------------
        if (warp < DEC_WARPS && nsteps) {
            const bool ready = mbar_wait(accum, accum_parity, abort_flag, M.status, M.wait_limit);
            if (__all_sync(0xffffffffu, ready)) {                  // tcgen05.ld needs the whole warp
                tc_fence_after();
                const uint32_t quad = warp & 3, part = warp >> 2;       // TMEM lane quarter (batch rows), column quarter
                for (uint32_t c = 0; c < M.nchunks; ++c) {
                    const uint32_t b = bc + c * MB + quad * 32 + lane;  // batch row of this thread
                    if (bc + c * MB + quad * 32 >= M.batch) continue;   // the same in the whole warp
#pragma unroll 1
                    for (uint32_t q = 0; q < 2; ++q) {
                        const uint32_t col = part * 64 + q * 32;        // first of 32 weight rows
                        uint32_t v[32];
                        tmem_ld32(tmem_base + ((quad * 32) << 16) + c * NROWS + col, v);
                        if (M.nchunks == 1) {                           // the second accumulator of the only chunk
                            uint32_t u[32];
                            tmem_ld32(tmem_base + ((quad * 32) << 16) + NROWS + col, u);
#pragma unroll
                            for (uint32_t e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) + __uint_as_float(u[e]));
                        }
                        if (b < M.batch) {
                            float *dst = M.y + (int64_t)b * M.ldy + (int64_t)(r0 + col);
#pragma unroll
                            for (uint32_t e = 0; e < 32; e += 4) {
                                const float o0 = alpha_s[col + e] * __uint_as_float(v[e]);
                                const float o1 = alpha_s[col + e + 1] * __uint_as_float(v[e + 1]);
                                const float o2 = alpha_s[col + e + 2] * __uint_as_float(v[e + 2]);
                                const float o3 = alpha_s[col + e + 3] * __uint_as_float(v[e + 3]);
                                if (M.vec_y && r0 + col + e + 4 <= M.m) {
                                    red_add_v4(dst + e, o0, o1, o2, o3);
                                } else {
                                    if (r0 + col + e < M.m) atomicAdd(dst + e, o0);
                                    if (r0 + col + e + 1 < M.m) atomicAdd(dst + e + 1, o1);
                                    if (r0 + col + e + 2 < M.m) atomicAdd(dst + e + 2, o2);
                                    if (r0 + col + e + 3 < M.m) atomicAdd(dst + e + 3, o3);
                                }
                            }
                        }
                    }
                }
            }
        }
        if (nsteps) accum_parity ^= 1;
        tc_fence_before();
        __syncthreads();                       // accumulators are read before the next pass overwrites them
        tc_fence_after();
    }
    if (warp == DEC_WARPS + 1) tmem_dealloc(tmem_base, tmem_cols);
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
    M.bits32 = (const uint32_t *)d_workspace;
    M.plane_words32 = A0.words64 * 2;
    M.mask32 = (const uint32_t *)d_mask;
    M.mask_words32 = A0.words64 * 2;
    M.alpha = d_alpha;
    M.y = d_y;
    M.ldy = ldy;
    M.m = desc->m;
    M.n = desc->n;
    M.n_q = desc->n_q;
    M.batch = batch;
    M.nchunks = batch > MB ? 2u : 1u;
    M.status = A0.status;
    // rows of the packed vectors start on 16-byte boundaries when n is a multiple of 128 (the workspace is
    // 256-byte aligned and every plane in it starts on a multiple of 8 bytes: check that too)
    M.aligned = (desc->n % 128 == 0 && ((uintptr_t)d_mask & 15) == 0 && (M.plane_words32 % 4 == 0 || desc->n_q == 1)) ? 1u : 0u;
    M.vec_y = (((uintptr_t)d_y & 15) == 0 && ldy % 4 == 0) ? 1u : 0u;
    const uint32_t dbg = g_debug_flags.load();
    M.skip_loads = (dbg & 1u) ? 1u : 0u;
    M.wait_limit = g_debug_wait_cycles.load() ? g_debug_wait_cycles.load() : WAIT_LIMIT_CYCLES;

    const size_t budget = 225 * 1024;        // + 1 KB of static shared memory stays within the 227 KB a block may have
    const size_t fixed = 256 * 8 * LUT_COPIES + NROWS * 4 + (3 * MAX_STAGES + 1) * 8 + 16 + 1024;
    const size_t per_stage = B_STAGE_BYTES + (size_t)M.nchunks * A_TILE_BYTES;
    M.stages = MAX_STAGES;
    while (M.stages > 1 && fixed + (size_t)M.stages * per_stage > budget) --M.stages;
    const size_t smem = fixed + (size_t)M.stages * per_stage;
    if (smem > budget) return SQNN_E_UNSUPPORTED;

    const uint64_t row_tiles = (desc->m + NROWS - 1) / NROWS;
    const uint32_t total_macros = (uint32_t)((desc->n + MACRO - 1) / MACRO);
    const uint64_t items = row_tiles * desc->n_q;
    uint32_t splits = items >= (uint64_t)sm_count() ? 1u : (uint32_t)((uint64_t)sm_count() / items);
    if (splits < 1) splits = 1;
    if (splits > total_macros) splits = total_macros;
    M.macros_per_split = (total_macros + splits - 1) / splits;
    M.splits = (total_macros + M.macros_per_split - 1) / M.macros_per_split;
    if (items * M.splits > 0x7fffffffull) return SQNN_E_UNSUPPORTED;

    CUtensorMap xmap;
    const cuuint64_t gdim[2] = {(cuuint64_t)desc->n, (cuuint64_t)batch};
    const cuuint64_t gstride[1] = {(cuuint64_t)ldx * 2};
    const cuuint32_t box[2] = {KC, MB};
    const cuuint32_t estride[2] = {1, 1};
    if (encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(d_x), gdim, gstride, box, estride,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return SQNN_E_CUDA;

    cudaError_t e = (ldy == (int64_t)desc->m)
        ? cudaMemsetAsync(d_y, 0, (size_t)batch * desc->m * sizeof(float), st)
        : cudaMemset2DAsync(d_y, (size_t)ldy * sizeof(float), 0, (size_t)desc->m * sizeof(float), batch, st);
    if (e != cudaSuccess) return SQNN_E_CUDA;
    if (ensure_dynamic_smem(reinterpret_cast<const void *>(k_decode_mma), smem) != SQNN_OK) return SQNN_E_CUDA;
    // stage 1: the decode kernel writes the planes as packed bits into the workspace
    const int rc = decode_bits_dispatch(A0, d_workspace, st);
    if (rc != SQNN_OK) return rc;
    k_decode_mma<<<(uint32_t)(items * M.splits), THREADS, smem, st>>>(xmap, M);
    return cudaGetLastError() == cudaSuccess ? SQNN_OK : SQNN_E_CUDA;
}

}  // namespace sqnn

// For the library's own tests: bit 0 of `flags` makes the tensor-core kernel's loader issue no loads, so that
// the bounded waits of its consumers run out; wait_limit_cycles (0 = default, about 2 s) is the number of
// clock cycles such a wait may take.  Affects calls made after it; not meant for applications.
extern "C" void sqnn_set_debug_flags(uint32_t flags, uint64_t wait_limit_cycles)
{
    sqnn::g_debug_flags.store(flags);
    sqnn::g_debug_wait_cycles.store(wait_limit_cycles);
}

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

static int decode_matmul_static_queue(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
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
    if (x_dtype != SQNN_X_F32 && x_dtype != SQNN_X_BF16) return SQNN_E_INVALID_ARG;
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

extern "C" int sqnn_decode_matmul_static(const sqnn_desc *desc, const void *d_blob, const uint64_t *d_mask,
                                         const float *d_alpha, const void *d_x, int x_dtype, uint32_t batch,
                                         int64_t ldx, float *d_y, int64_t ldy, uint32_t *d_status,
                                         void *cuda_stream)
{
    sqnn::ApiScope scope("sqnn_decode_matmul_static");
    return scope.finish(decode_matmul_static_queue(desc, d_blob, d_mask, d_alpha, d_x, x_dtype, batch, ldx, d_y, ldy,
                                                   d_status, cuda_stream),
                        d_status, (cudaStream_t)cuda_stream);
}
