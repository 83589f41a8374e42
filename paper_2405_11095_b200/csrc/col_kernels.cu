// Strided pass: A butterfly stages on the index bits [lo, lo + A) of the coordinate, lo >= 10,
// i.e. the Kronecker factor (H_A (x) I_S) with S = 2^lo.  The vector is read as a matrix with
// rows S apart; a warp always covers 32 consecutive columns, so global accesses are 128-byte
// coalesced and a row segment of a packed source is exactly one word.  Sources: gradients
// (pad + flip), packed bits, or the fp32 intermediate; the sink is the fp32 intermediate
// (in place when source and sink coincide: a block reads its whole tile before writing it).
//
//   A <= 5: a thread holds the 2^A rows of one column in registers; no shared memory.
//   A >  5: a block of 2^A threads owns 2^A rows x 32 columns: round F transforms the top
//           five row bits straight from global memory, round L the remaining low row bits
//           after one exchange through shared memory.
#include <cuda.h>   // CUtensorMap and the encode entry point type; the driver is reached through the runtime

#include "common.cuh"

namespace fosgd {

// Coordinates inside one worker's vector are below 2^31, so all per-element index arithmetic is
// done on 32-bit offsets from the worker's base pointer (one widening multiply-add per access
// instead of 64-bit shifts, adds and compares).
template <int SRC>
__device__ __forceinline__ float col_load(const PassParams& p, const void* worker_src, uint32_t i, uint32_t d32,
                                          uint32_t bit)
{
    if (SRC == SRC_G32) {
        return (i < d32) ? __ldcs(static_cast<const float*>(worker_src) + i) : 0.f;
    } else if (SRC == SRC_G16) {
        return (i < d32) ? __uint_as_float((uint32_t)__ldcs(static_cast<const uint16_t*>(worker_src) + i) << 16) : 0.f;
    } else if (SRC == SRC_WS) {
        return static_cast<const float*>(worker_src)[i];
    } else {
        return plane_value(static_cast<const uint32_t*>(worker_src) + (i >> 5), p.dp >> 5, p.P, p.K, bit);
    }
}

template <int SRC>
__device__ __forceinline__ const void* worker_source(const PassParams& p, int n)
{
    const size_t es = (SRC == SRC_G16) ? 2 : 4;
    return static_cast<const char*>(p.src) + (size_t)n * (size_t)p.src_stride * es;
}

// x with its sign flipped iff bit (31 - sh) of word is set
__device__ __forceinline__ float flip_shifted(float x, uint32_t word, uint32_t sh)
{
    return __uint_as_float(__float_as_uint(x) ^ ((word << sh) & 0x80000000u));
}

// One-plane packed source: the 32 columns of a row segment are one word.  Lane r fetches the
// word of the r-th row this warp handles (one gather per warp instead of 32 broadcast loads).
__device__ __forceinline__ uint32_t bits_row_word(const void* worker_src, uint32_t irow)
{
    return __ldg(static_cast<const uint32_t*>(worker_src) + (irow >> 5));
}

// ---- A <= 5 -----------------------------------------------------------------------------
template <int A, int SRC>
__global__ void __launch_bounds__(256) col_small_kernel(const PassParams p)
{
    constexpr int R = 1 << A;
    const int n = blockIdx.y;
    const uint32_t lane = threadIdx.x & 31;
    const int64_t col = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const uint32_t lo = (uint32_t)(col & (((int64_t)1 << p.lo_log) - 1));
    const uint32_t hi = (uint32_t)(col >> p.lo_log);
    const uint32_t i_first = (hi << (p.lo_log + A)) + lo;  // row 0 of this column
    const uint32_t step = 1u << p.lo_log;
    const uint32_t d32 = (uint32_t)p.d;
    const void* const wsrc = worker_source<SRC>(p, n);

    float v[32];
    uint32_t myword = 0;  // flip word (gradient sources) or packed signs (one-plane bit source) of row `lane`
    const bool one_plane = (SRC == SRC_BITS) && p.P == 1;
    if ((int)lane < R) {
        const uint32_t irow = (i_first - lane) + lane * step;
        if (SRC == SRC_G32 || SRC == SRC_G16) myword = eps_word(p.rng, p.id0 + (uint32_t)n, irow >> 5);
        if (one_plane) myword = bits_row_word(wsrc, irow);
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const uint32_t i = i_first + r * step;
        float x;
        if (one_plane) {
            x = ((__shfl_sync(0xFFFFFFFFu, myword, r) >> lane) & 1u) ? 1.f : -1.f;
        } else {
            x = col_load<SRC>(p, wsrc, i, d32, lane);
            if (SRC == SRC_G32 || SRC == SRC_G16) x = flip_shifted(x, __shfl_sync(0xFFFFFFFFu, myword, r), 31u - lane);
        }
        v[r] = x;
    }
#pragma unroll
    for (int r = R; r < 32; ++r) v[r] = 0.f;
    butterflies32<R - 1>(v);
    float* dst = static_cast<float*>(p.dst) + (int64_t)n * p.dst_stride;
#pragma unroll
    for (int r = 0; r < R; ++r) dst[i_first + r * step] = v[r];
}

// ---- A > 5 ------------------------------------------------------------------------------
template <int A, int SRC>
__global__ void __launch_bounds__(1 << A) col_tile_kernel(const PassParams p)
{
    extern __shared__ __align__(16) float smem[];  // 2^A rows x 32 columns
    constexpr int WARPS = 1 << (A - 5);
    const int n = blockIdx.y;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t w = threadIdx.x >> 5;
    const int64_t seg = blockIdx.x;                               // 32-column segment id
    const uint32_t lo0 = (uint32_t)((seg << 5) & (((int64_t)1 << p.lo_log) - 1));
    const uint32_t hi = (uint32_t)((seg << 5) >> p.lo_log);
    const uint32_t i_tile = (hi << (p.lo_log + A)) + lo0;        // row 0, column 0 of the tile
    const uint32_t step = 1u << p.lo_log;                         // one row
    const uint32_t d32 = (uint32_t)p.d;
    const void* const wsrc = worker_source<SRC>(p, n);

    float v[32];
    uint32_t myword = 0;  // flip word (gradient sources) or packed signs (one-plane bit source) of row lane*WARPS+w
    const bool one_plane = (SRC == SRC_BITS) && p.P == 1;
    {
        const uint32_t irow = i_tile + (lane * WARPS + w) * step;
        if (SRC == SRC_G32 || SRC == SRC_G16) myword = eps_word(p.rng, p.id0 + (uint32_t)n, irow >> 5);
        if (one_plane) myword = bits_row_word(wsrc, irow);
    }
    // round F: rows k = r * WARPS + w  (register bits = top five row bits)
    const uint32_t i_f = i_tile + w * step + lane;
    const uint32_t step_f = step * WARPS;
#pragma unroll
    for (int r = 0; r < 32; ++r) {
        float x;
        if (one_plane) {
            x = ((__shfl_sync(0xFFFFFFFFu, myword, r) >> lane) & 1u) ? 1.f : -1.f;
        } else {
            x = col_load<SRC>(p, wsrc, i_f + r * step_f, d32, lane);
            if (SRC == SRC_G32 || SRC == SRC_G16) x = flip_shifted(x, __shfl_sync(0xFFFFFFFFu, myword, r), 31u - lane);
        }
        v[r] = x;
    }
    butterflies32<31>(v);
#pragma unroll
    for (int r = 0; r < 32; ++r) smem[((r * WARPS + w) << 5) + lane] = v[r];
    __syncthreads();
    // round L: rows k = w * 32 + r  (register bits = low five row bits; those below A-5 are new)
#pragma unroll
    for (int r = 0; r < 32; ++r) v[r] = smem[((w * 32 + r) << 5) + lane];
    butterflies32<(A >= 10) ? 31 : ((1 << (A - 5)) - 1)>(v);
    float* const dst = static_cast<float*>(p.dst) + (int64_t)n * p.dst_stride;
    const uint32_t i_l = i_tile + (w * 32) * step + lane;
#pragma unroll
    for (int r = 0; r < 32; ++r) __stcg(dst + i_l + r * step, v[r]);   // L2 only: read next by another kernel
}

// ---- A > 5, 16-column tiles ----------------------------------------------------------------
// Same two rounds on a tile of 2^A rows x 16 columns (half the shared memory, so two blocks fit
// on an SM and one block's loads overlap the other's arithmetic and stores).  A lane is a
// (column, row-bit) pair: in round F the row bit is bit 0 of the row, in round L bit 5, so a warp
// instruction always touches two rows x 64 contiguous bytes.  Shared memory holds element
// (row k, column c) at word k*16 + c, plus 16 words of padding per 512 (keeps round L, whose two
// half-warps sit 512 words apart, off the same banks).
__host__ __device__ constexpr int phys16(int e) { return e + ((e >> 9) << 4); }

template <int A, int SRC>
__global__ void __launch_bounds__(1 << (A - 1), 2) col_tile16_kernel(const PassParams p)
{
    extern __shared__ __align__(16) float smem[];
    const int n = blockIdx.y;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t c = lane & 15, h = lane >> 4;
    const uint32_t w = threadIdx.x >> 5;
    const int64_t seg = blockIdx.x;                               // 16-column segment id
    const uint32_t lo0 = (uint32_t)((seg << 4) & (((int64_t)1 << p.lo_log) - 1));
    const uint32_t hi = (uint32_t)((seg << 4) >> p.lo_log);
    const uint32_t i_tile = (hi << (p.lo_log + A)) + lo0;        // row 0, column 0 of the tile
    const uint32_t step = 1u << p.lo_log;                         // one row
    const uint32_t d32 = (uint32_t)p.d;
    const uint32_t bitpos = (lo0 & 31u) + c;                      // this lane's bit inside a packed/flip word
    const void* const wsrc = worker_source<SRC>(p, n);

    float v[32];
    // Per-row words (flip word of a gradient row, or the packed signs of a one-plane source row):
    // lane j fetches them for rows (r = j & 15, h = j >> 4) and (r = 16 + (j & 15), h = j >> 4).
    uint32_t word_lo = 0, word_hi = 0;
    const bool one_plane = (SRC == SRC_BITS) && p.P == 1;
    {
        const uint32_t row_a = ((lane & 15u) << (A - 5)) | (w << 1) | h;
        const uint32_t ia = i_tile + row_a * step, ib = ia + (step << (A - 1));
        if (SRC == SRC_G32 || SRC == SRC_G16) {
            word_lo = eps_word(p.rng, p.id0 + (uint32_t)n, ia >> 5);
            word_hi = eps_word(p.rng, p.id0 + (uint32_t)n, ib >> 5);
        }
        if (one_plane) {
            word_lo = bits_row_word(wsrc, ia);
            word_hi = bits_row_word(wsrc, ib);
        }
    }
    // round F: rows k = (r << (A-5)) | (w << 1) | h
    const uint32_t i_f = i_tile + ((w << 1) | h) * step + c;
    const uint32_t step_f = step << (A - 5);
    const uint32_t shamt = 31u - bitpos;
    // a block whose last coordinate is inside the gradient needs no per-element bound check
    const bool inside = i_tile + (((1u << A) - 1u) * step) + 15u < d32;
    auto load_rows = [&](const uint32_t bound) {
#pragma unroll
        for (int r = 0; r < 32; ++r) {
            // lanes of a half-warp (same h) read the word from lane r & 15 of their own half
            const uint32_t roww = __shfl_sync(0xFFFFFFFFu, r < 16 ? word_lo : word_hi, r & 15, 16);
            float x;
            if (one_plane) {
                x = ((roww >> bitpos) & 1u) ? 1.f : -1.f;
            } else {
                x = col_load<SRC>(p, wsrc, i_f + r * step_f, bound, bitpos);
                if (SRC == SRC_G32 || SRC == SRC_G16) x = flip_shifted(x, roww, shamt);
            }
            v[r] = x;
        }
    };
    if (inside) load_rows(0xFFFFFFFFu); else load_rows(d32);   // the constant bound folds the checks away
    butterflies32<31>(v);
    {
        float* const pf = smem + phys16((int)((((w << 1) | h) << 4) + c));
#pragma unroll
        for (int r = 0; r < 32; ++r) pf[phys16(r << (A - 1))] = v[r];
    }
    __syncthreads();
    // round L: rows k = (w << 6) | (h << 5) | r
    {
        const float* const pl = smem + phys16((int)((((w << 6) | (h << 5)) << 4) + c));
#pragma unroll
        for (int r = 0; r < 32; ++r) v[r] = pl[r << 4];
    }
    butterflies32<(A >= 10) ? 31 : ((1 << (A - 5)) - 1)>(v);
    float* const dst = static_cast<float*>(p.dst) + (int64_t)n * p.dst_stride;
    const uint32_t i_l = i_tile + ((w << 6) | (h << 5)) * step + c;
#pragma unroll
    for (int r = 0; r < 32; ++r) __stcg(dst + i_l + r * step, v[r]);   // L2 only: read next by another kernel
}

// ---- A = 10, fp32 sources, TMA-staged persistent pipeline ------------------------------------------
// The 16-column tile once more, with the tile fetched by the tensor copy engine.  The source is
// described by a 3-D tensor map (columns S, rows, workers); a tile is four box copies of 256 rows x
// 16 columns landing densely in a 64 KiB buffer and completing on one mbarrier.  Rows past the end
// of the gradient are zero-filled by the copy engine (the map only covers whole rows; a last,
// partial row is patched in by ordinary loads).  A dense buffer admits no padding, so both rounds
// keep row bit 0 in the lane (a warp always touches two adjacent rows = 32 consecutive words) and
// the butterfly on row bit 0 is one shuffle stage: round F transforms row bits 5..9, round L bits
// 1..4, the shuffle bit 0.  Blocks are persistent: two groups of 512 threads take tiles in turn over
// three buffers, and the group that has pulled its tile into registers for round L starts the
// copies of the tile three positions ahead into the buffer it has just freed, so loads stay in
// flight while both groups compute and store.
static __device__ int g_col_wait_timeouts;   // groups that abandoned a bounded wait

// bar.sync / bar.red are the warp-aligned forms: every lane of a warp must arrive together.  The
// code before them has lane-dependent paths (one lane issues the copies, sixteen patch a row, the
// polling loop of a bounded wait ends per lane), and nothing obliges the compiler to have rejoined
// them in front of an opaque asm statement, so the warp is converged explicitly first.
__device__ __forceinline__ void group_sync(int id, int nthreads)
{
    __syncwarp();
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// barrier + AND over the group: every thread learns whether all of them saw `ok`
__device__ __forceinline__ bool group_all(int id, int nthreads, bool ok)
{
    uint32_t all;
    __syncwarp();
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\tbar.red.and.pred q, %2, %3, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                 : "=r"(all) : "r"((uint32_t)ok), "r"(id), "r"(nthreads) : "memory");
    return all != 0;
}

template <int SRC>
__global__ void __launch_bounds__(1024, 1) col_tma16_kernel(const PassParams p, const __grid_constant__ CUtensorMap tmap,
                                                            const int64_t nsegs, const uint32_t full_rows)
{
    static_assert(SRC == SRC_G32 || SRC == SRC_WS, "4-byte elements only");
    constexpr int A = 10;
    constexpr int GT = 512;                                 // threads per group
    constexpr int BUF_WORDS = (1 << A) * 16;
    extern __shared__ __align__(128) float smem[];
    uint64_t* const full = reinterpret_cast<uint64_t*>(smem + 3 * BUF_WORDS);
    // Copies issued into / tiles taken out of each buffer (written by one thread of the issuing resp.
    // consuming group), and the flag that stops all issuing once a bounded wait has given up: the
    // block then drains what is still in flight before any of its threads exits.
    __shared__ int s_issued[3], s_taken[3], s_stop;

    const int tid = threadIdx.x;
    const int g = tid >> 9;
    const int gt = tid & (GT - 1);
    const uint32_t lane = gt & 31, c = lane & 15, h = lane >> 4, w = gt >> 5;
    const uint32_t step = 1u << p.lo_log;
    const uint32_t d32 = (uint32_t)p.d;
    const int64_t total = nsegs * p.nworkers;
    const int64_t nitems = (total - (int64_t)blockIdx.x + gridDim.x - 1) / gridDim.x;

    if (tid == 0) {
        for (int b = 0; b < 3; ++b) {
            mbar_init(full + b, 1);
            s_issued[b] = 0;
            s_taken[b] = 0;
        }
        s_stop = 0;
    }
    __syncthreads();

    auto item_coords = [&](int64_t j, int& n, uint32_t& lo0, uint32_t& hi) {
        const int64_t q = blockIdx.x + j * gridDim.x;
        n = (int)(q / nsegs);
        const int64_t seg = q % nsegs;
        lo0 = (uint32_t)((seg << 4) & (((int64_t)1 << p.lo_log) - 1));
        hi = (uint32_t)((seg << 4) >> p.lo_log);
    };
    // one thread: four box copies (256 rows x 16 columns each) into buffer j % 3
    auto issue = [&](int64_t j) {
        if (*(volatile int*)&s_stop) return;
        int n;
        uint32_t lo0, hi;
        item_coords(j, n, lo0, hi);
        uint64_t* const bar = full + (j % 3);
        const uint32_t dst0 = smem_u32(smem + (j % 3) * BUF_WORDS);
        s_issued[j % 3] += 1;
        fence_generic_before_async();
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(65536u) : "memory");
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                         ::"r"(dst0 + 16384u * q), "l"(&tmap), "r"((int)lo0), "r"((int)((hi << A) + 256 * q)),
                           "r"(n), "r"(smem_u32(bar)) : "memory");
        }
    };

    if (gt == 0) {
        if (g == 0) {
            if (nitems > 0) issue(0);
            if (nitems > 2) issue(2);
        } else {
            if (nitems > 1) issue(1);
        }
    }

    const int slot_f = (int)((w << 5) | (h << 4) | c);     // round F: row = (r << 5) | (w << 1) | h, + (r << 9)
    const int slot_l = (int)((w << 10) | (h << 4) | c);    // round L: row = (w << 6) | (r << 1) | h, + (r << 5)

    for (int64_t j = g; j < nitems; j += 2) {
        float* const buf = smem + (j % 3) * BUF_WORDS;
        int n;
        uint32_t lo0, hi;
        item_coords(j, n, lo0, hi);
        const uint32_t i_tile = (hi << (p.lo_log + A)) + lo0;
        const uint32_t bitpos = (lo0 & 31u) + c;

        uint32_t word_lo = 0, word_hi = 0;   // flip words of rows (r = lane & 15, h) and (16 + (lane & 15), h)
        if (SRC == SRC_G32) {
            const uint32_t row_a = ((lane & 15u) << 5) | (w << 1) | h;
            const uint32_t ia = i_tile + row_a * step, ib = ia + (step << 9);
            word_lo = eps_word(p.rng, p.id0 + (uint32_t)n, ia >> 5);
            word_hi = eps_word(p.rng, p.id0 + (uint32_t)n, ib >> 5);
        }
        // bounded wait; the group then agrees on the outcome, so that it stops as a whole
        if (!group_all(1 + g, GT, mbar_wait(full + (j % 3), (uint32_t)((j / 3) & 1)))) {
            if (gt == 0) {
                atomicAdd(&g_col_wait_timeouts, 1);
                *(volatile int*)&s_stop = 1;
            }
            break;
        }
        if (gt == 0) s_taken[j % 3] += 1;
        if (SRC == SRC_G32) {
            // the map covers whole rows only: a last partial row of the gradient is patched in
            const uint32_t row_p = full_rows - (hi << A);                  // tile-local index of that row
            if (row_p < (1u << A) && gt < 16) {
                const uint32_t i = full_rows * step + lo0 + (uint32_t)gt;
                if (i < d32)
                    buf[(row_p << 4) + gt] = (static_cast<const float*>(p.src) + (int64_t)n * p.src_stride)[i];
            }
            if (row_p < (1u << A)) group_sync(1 + g, GT);
        }
        float v[32];
        const uint32_t shamt = 31u - bitpos;
#pragma unroll
        for (int r = 0; r < 32; ++r) {
            float x = buf[slot_f + (r << 9)];
            if (SRC == SRC_G32) {
                const uint32_t roww = __shfl_sync(0xFFFFFFFFu, r < 16 ? word_lo : word_hi, r & 15, 16);
                x = flip_shifted(x, roww, shamt);
            }
            v[r] = x;
        }
        butterflies32<31>(v);                      // row bits 5..9
#pragma unroll
        for (int r = 0; r < 32; ++r) buf[slot_f + (r << 9)] = v[r];
        group_sync(1 + g, GT);
#pragma unroll
        for (int r = 0; r < 32; ++r) v[r] = buf[slot_l + (r << 5)];
        fence_generic_before_async();              // this thread's stores into the buffer, before the copy engine reuses it
        group_sync(1 + g, GT);                     // the buffer is free: refill it for the tile three ahead
        if (gt == 0 && j + 3 < nitems) issue(j + 3);
        butterflies32<15>(v);                      // row bits 1..4 (register bit 4 = row bit 5 is done)
        const float sgn = h ? -1.f : 1.f;          // row bit 0 lives in the lane: one shuffle stage
#pragma unroll
        for (int r = 0; r < 32; ++r) v[r] = fmaf(sgn, v[r], __shfl_xor_sync(0xFFFFFFFFu, v[r], 16));
        float* const dst = static_cast<float*>(p.dst) + (int64_t)n * p.dst_stride;
        const uint32_t i_l = i_tile + ((w << 6) | h) * step + c;
#pragma unroll
        for (int r = 0; r < 32; ++r) __stcg(dst + i_l + (r << 1) * step, v[r]);
    }
    // Both groups meet here, whether they finished or gave up.  In a healthy run every issued copy has
    // been taken; after a timeout the copies still in flight get one more bounded wait, so that the
    // engine is not left writing into shared memory that the next block of this SM may own.
    __syncthreads();
    if (tid == 0) {
        for (int b = 0; b < 3; ++b) {
            if (s_issued[b] > s_taken[b]) mbar_wait(full + b, (uint32_t)((s_issued[b] - 1) & 1));
            mbar_inval(full + b);
        }
    }
}

cudaError_t col_timeouts(int* out) { return cudaMemcpyFromSymbol(out, g_col_wait_timeouts, sizeof(int)); }

// Tensor map over the source of a strided pass: (S columns, rows, workers).  False if the driver
// entry point is missing or refuses the geometry; the caller then uses the plain kernel.
static bool make_col_tensor_map(CUtensorMap* map, const void* base, uint64_t S, uint64_t rows, uint64_t workers,
                                uint64_t worker_stride_elems)
{
    using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = []() -> EncodeFn {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeFn>(fn);
    }();
    if (encode == nullptr || rows == 0) return false;
    const cuuint64_t dims[3] = {S, rows, workers};
    const cuuint64_t strides[2] = {S * 4, worker_stride_elems * 4};
    const cuuint32_t box[3] = {16, 256, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int SRC>
static cudaError_t launch_col_tma(const PassParams& p, cudaStream_t s, bool* launched)
{
    constexpr int A = 10;
    *launched = false;
    const uint64_t S = (uint64_t)1 << p.lo_log;
    const uint64_t rows = (SRC == SRC_WS) ? (uint64_t)(p.dp >> p.lo_log) : (uint64_t)(p.d >> p.lo_log);   // whole rows
    CUtensorMap map;
    if (!make_col_tensor_map(&map, p.src, S, rows, (uint64_t)p.nworkers, (uint64_t)p.src_stride)) return cudaSuccess;
    auto kern = col_tma16_kernel<SRC>;
    constexpr size_t smem = (size_t)3 * (1 << A) * 16 * 4 + 32;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const int64_t nsegs = (p.dp >> A) / 16;
    int64_t blocks = sms;
    if (blocks > nsegs * p.nworkers) blocks = nsegs * p.nworkers;
    kern<<<(unsigned)blocks, 1024, smem, s>>>(p, map, nsegs, (uint32_t)rows);
    *launched = true;
    return cudaGetLastError();
}

// ---- packed one-plane source, fp16 arithmetic ------------------------------------------------
// The server's first pass starts from +-1, and after A <= 10 stages every value is an integer of
// magnitude <= 1024, which fp16 holds exactly.  So this variant keeps two adjacent columns per
// lane as a half2: a block owns 2^A rows x 64 columns, butterflies are HADD2 (two coordinates
// per instruction), and the intermediate is written as fp16 (half the bytes, still full
// 128-byte lines per warp).  Rows of the packed source are two words; they are staged once in
// shared memory.
template <int A>
__global__ void __launch_bounds__(1 << A) colh_tile_kernel(const PassParams p)
{
    extern __shared__ __align__(16) uint32_t smemh[];   // [2^A][32] half2 tile, then [2^A] word pairs
    constexpr int ROWS = 1 << A;
    constexpr int WARPS = 1 << (A - 5);
    uint2* const wtab = reinterpret_cast<uint2*>(smemh + ROWS * 32);
    const int n = blockIdx.y;
    const int tid = threadIdx.x;
    const uint32_t lane = tid & 31;
    const int w = tid >> 5;
    const int64_t seg = blockIdx.x;                               // 64-column segment id
    const int64_t lo0 = (seg << 6) & (((int64_t)1 << p.lo_log) - 1);
    const int64_t hi = (seg << 6) >> p.lo_log;
    const int64_t i_tile = (hi << (p.lo_log + A)) + lo0;

    {
        const uint32_t* bits = static_cast<const uint32_t*>(p.src) + (int64_t)n * p.src_stride;
        wtab[tid] = __ldg(reinterpret_cast<const uint2*>(bits + ((i_tile + ((int64_t)tid << p.lo_log)) >> 5)));
    }
    __syncthreads();

    __half2 v[32];
    const uint32_t sh = (2u * lane) & 31u;
    const uint32_t* const wsel = reinterpret_cast<const uint32_t*>(wtab) + (lane >> 4);
#pragma unroll
    for (int r = 0; r < 32; ++r) {
        const uint32_t x = (wsel[2 * (r * WARPS + w)] >> sh) & 3u;
        // bit 0 -> sign of the low half, bit 1 -> sign of the high half; set bit = +1
        const uint32_t hb = 0xBC00BC00u ^ ((x * 0x40008000u) & 0x80008000u);
        v[r] = *reinterpret_cast<const __half2*>(&hb);
    }
    butterflies32<31, __half2>(v);
    __half2* const tile = reinterpret_cast<__half2*>(smemh);
#pragma unroll
    for (int r = 0; r < 32; ++r) tile[((r * WARPS + w) << 5) + lane] = v[r];
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 32; ++r) v[r] = tile[((w * 32 + r) << 5) + lane];
    butterflies32<(A >= 10) ? 31 : ((1 << (A - 5)) - 1), __half2>(v);
    __half2* dst = reinterpret_cast<__half2*>(static_cast<__half*>(p.dst) + (int64_t)n * p.dst_stride + i_tile) + lane;
#pragma unroll
    for (int r = 0; r < 32; ++r) dst[((int64_t)(w * 32 + r) << p.lo_log) >> 1] = v[r];
}

// The same pass on 2^A rows x 32 columns (16 half2 lanes x one row bit per lane, like the
// 16-column fp32 variant): half the shared memory and half the threads per block, so two blocks
// share an SM and one block's stores overlap the other's arithmetic.  A row of the packed source
// is one word; lane j fetches the words of rows (r = j & 15, h = j >> 4) and (16 + (j & 15), h).
template <int A>
__global__ void __launch_bounds__(1 << (A - 1), 2) colh_tile32_kernel(const PassParams p)
{
    extern __shared__ __align__(16) uint32_t smemh[];
    const int n = blockIdx.y;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t c2 = lane & 15, h = lane >> 4;
    const uint32_t w = threadIdx.x >> 5;
    const int64_t seg = blockIdx.x;                               // 32-column segment id
    const uint32_t lo0 = (uint32_t)((seg << 5) & (((int64_t)1 << p.lo_log) - 1));
    const uint32_t hi = (uint32_t)((seg << 5) >> p.lo_log);
    const uint32_t i_tile = (hi << (p.lo_log + A)) + lo0;
    const uint32_t step = 1u << p.lo_log;
    const uint32_t* const bits = static_cast<const uint32_t*>(p.src) + (int64_t)n * p.src_stride;

    uint32_t word_lo, word_hi;
    {
        const uint32_t row_a = ((lane & 15u) << (A - 5)) | (w << 1) | h;
        const uint32_t ia = i_tile + row_a * step;
        word_lo = __ldg(bits + (ia >> 5));
        word_hi = __ldg(bits + ((ia + (step << (A - 1))) >> 5));
    }
    __half2 v[32];
    const uint32_t sh = 2u * c2;
#pragma unroll
    for (int r = 0; r < 32; ++r) {
        const uint32_t roww = __shfl_sync(0xFFFFFFFFu, r < 16 ? word_lo : word_hi, r & 15, 16);
        const uint32_t x = (roww >> sh) & 3u;
        const uint32_t hb = 0xBC00BC00u ^ ((x * 0x40008000u) & 0x80008000u);
        v[r] = *reinterpret_cast<const __half2*>(&hb);
    }
    butterflies32<31, __half2>(v);
    __half2* const tile = reinterpret_cast<__half2*>(smemh);
    {
        __half2* const pf = tile + phys16((int)((((w << 1) | h) << 4) + c2));
#pragma unroll
        for (int r = 0; r < 32; ++r) pf[phys16(r << (A - 1))] = v[r];
    }
    __syncthreads();
    {
        const __half2* const pl = tile + phys16((int)((((w << 6) | (h << 5)) << 4) + c2));
#pragma unroll
        for (int r = 0; r < 32; ++r) v[r] = pl[r << 4];
    }
    butterflies32<(A >= 10) ? 31 : ((1 << (A - 5)) - 1), __half2>(v);
    __half2* const dst = reinterpret_cast<__half2*>(static_cast<__half*>(p.dst) + (int64_t)n * p.dst_stride);
    const uint32_t i_l = ((i_tile + ((w << 6) | (h << 5)) * step) >> 1) + c2;
    const uint32_t step2 = step >> 1;
#pragma unroll
    for (int r = 0; r < 32; ++r)
        __stcg(reinterpret_cast<unsigned int*>(dst) + i_l + r * step2, *reinterpret_cast<const unsigned int*>(&v[r]));
}

template <int A>
static cudaError_t launch_colh_one(const PassParams& p, cudaStream_t s)
{
    if constexpr (A >= 8) {
        auto kern = colh_tile32_kernel<A>;
        constexpr size_t smem = (size_t)phys16((1 << A) * 16) * 4;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        const dim3 grid((unsigned)((p.dp >> A) / 32), (unsigned)p.nworkers);
        kern<<<grid, 1 << (A - 1), smem, s>>>(p);
    } else {
        auto kern = colh_tile_kernel<A>;
        constexpr size_t smem = (size_t)(1 << A) * (32 * 4 + 8);
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        const dim3 grid((unsigned)((p.dp >> A) / 64), (unsigned)p.nworkers);
        kern<<<grid, 1 << A, smem, s>>>(p);
    }
    return cudaGetLastError();
}

cudaError_t launch_colh(int A, const PassParams& p, cudaStream_t s)
{
    switch (A) {
        case 6: return launch_colh_one<6>(p, s);
        case 7: return launch_colh_one<7>(p, s);
        case 8: return launch_colh_one<8>(p, s);
        case 9: return launch_colh_one<9>(p, s);
        case 10: return launch_colh_one<10>(p, s);
    }
    return cudaErrorInvalidValue;
}

template <int A, int SRC>
static cudaError_t launch_col_one(const PassParams& p, cudaStream_t s)
{
    if constexpr (A <= 5) {
        const dim3 grid((unsigned)((p.dp >> A) / 256), (unsigned)p.nworkers);
        col_small_kernel<A, SRC><<<grid, 256, 0, s>>>(p);
    } else if constexpr (A >= 8) {
        // The TMA-staged kernel is used where it has been validated against the oracle: as the single
        // strided pass of a transform (lengths 2^24 and 2^25), reading the caller's gradients out of
        // place.  As the in-place second strided pass of the 2^31 transform a launch failed
        // (unspecified launch failure) and the cause was not found by inspection, so transforms with
        // two strided passes keep the plain kernel for both.
        if constexpr (A == 10 && SRC == SRC_G32) {
            if (p.dp == ((int64_t)1 << (p.lo_log + A)) && p.src != p.dst) {
                bool launched = false;
                const cudaError_t e = launch_col_tma<SRC>(p, s, &launched);
                if (e != cudaSuccess || launched) return e;
            }
        }
        auto kern = col_tile16_kernel<A, SRC>;
        constexpr size_t smem = (size_t)phys16((1 << A) * 16) * 4;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        const dim3 grid((unsigned)((p.dp >> A) / 16), (unsigned)p.nworkers);
        kern<<<grid, 1 << (A - 1), smem, s>>>(p);
    } else {
        auto kern = col_tile_kernel<A, SRC>;
        constexpr size_t smem = (size_t)(1 << A) * 32 * 4;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        const dim3 grid((unsigned)((p.dp >> A) / 32), (unsigned)p.nworkers);
        kern<<<grid, 1 << A, smem, s>>>(p);
    }
    return cudaGetLastError();
}

template <int A>
static cudaError_t launch_col_A(int src, const PassParams& p, cudaStream_t s)
{
    switch (src) {
        case SRC_G32: return launch_col_one<A, SRC_G32>(p, s);
        case SRC_G16: return launch_col_one<A, SRC_G16>(p, s);
        case SRC_BITS: return launch_col_one<A, SRC_BITS>(p, s);
        case SRC_WS: return launch_col_one<A, SRC_WS>(p, s);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_col(int A, int src, const PassParams& p, cudaStream_t s)
{
    switch (A) {
        case 1: return launch_col_A<1>(src, p, s);
        case 2: return launch_col_A<2>(src, p, s);
        case 3: return launch_col_A<3>(src, p, s);
        case 4: return launch_col_A<4>(src, p, s);
        case 5: return launch_col_A<5>(src, p, s);
        case 6: return launch_col_A<6>(src, p, s);
        case 7: return launch_col_A<7>(src, p, s);
        case 8: return launch_col_A<8>(src, p, s);
        case 9: return launch_col_A<9>(src, p, s);
        case 10: return launch_col_A<10>(src, p, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace fosgd
