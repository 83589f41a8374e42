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

#include "col4.cuh"
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
    } else if (SRC == SRC_WS16) {
        return __half2float(static_cast<const __half*>(worker_src)[i]);
    } else {
        return plane_value(static_cast<const uint32_t*>(worker_src) + (i >> 5), p.dp >> 5, p.P, p.K, bit);
    }
}

template <int SRC>
__device__ __forceinline__ const void* worker_source(const PassParams& p, int n)
{
    const size_t es = (SRC == SRC_G16 || SRC == SRC_WS16) ? 2 : 4;
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

// ---- A = 10, gradients or the fp32 intermediate: tiles staged by the tensor copy engine (col4.cuh) ----
static __device__ int g_col_wait_timeouts;   // groups that abandoned a bounded wait

__global__ void __launch_bounds__(512, 2) col4_kernel(const PassParams p, const __grid_constant__ CUtensorMap tmap,
                                                      const int nruns, const uint32_t full_rows)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    col4_run<BlockSync>(p, &tmap, full_rows, (int)(blockIdx.x / (unsigned)nruns), (blockIdx.x % (unsigned)nruns) * 8u, smem_raw,
                        (int)threadIdx.x, &g_col_wait_timeouts);
}

// the same, also leaving the sum of squares of every run's gradient entries in partial[worker * nruns + run]
__global__ void __launch_bounds__(512, 2) col4_norm_kernel(const PassParams p, const __grid_constant__ CUtensorMap tmap,
                                                           const int nruns, const uint32_t full_rows, double* const partial)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    col4_run<BlockSync, true>(p, &tmap, full_rows, (int)(blockIdx.x / (unsigned)nruns), (blockIdx.x % (unsigned)nruns) * 8u, smem_raw,
                              (int)threadIdx.x, &g_col_wait_timeouts, partial + blockIdx.x);
}

__global__ void __launch_bounds__(1024, 1) col4_duo_kernel(const PassParams p, const __grid_constant__ CUtensorMap tmap,
                                                           const int nruns, const uint32_t full_rows)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    col4_duo(p, &tmap, (uint32_t)nruns, full_rows, (uint32_t)nruns * (uint32_t)p.nworkers, smem_raw, &g_col_wait_timeouts);
}

cudaError_t col_timeouts(int* out) { return cudaMemcpyFromSymbol(out, g_col_wait_timeouts, sizeof(int)); }

// Tensor map over the gradients as the strided pass sees them: (S columns, whole rows, workers).
// False if the driver entry point is missing or refuses the geometry; the caller then uses the plain kernel.
bool make_col_tensor_map(CUtensorMap* map, const void* base, uint64_t S, uint64_t rows, uint64_t workers,
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

// Ten stages on fp32 gradients through the copy engine.  *launched stays false where it does not apply
// (rows shorter than a run of 128 columns, or the driver refuses the map).
static cudaError_t launch_col4(const PassParams& p, cudaStream_t s, bool* launched)
{
    constexpr int A = 10;
    *launched = false;
    const uint64_t S = (uint64_t)1 << p.lo_log;
    const uint64_t rows = (uint64_t)(p.d >> p.lo_log);   // whole rows
    const int64_t nsegs = (p.dp >> A) / 16;
    const int64_t nruns = nsegs / 8;
    if (S < 128 || nsegs % 8 != 0 || nruns * p.nworkers > 0x7FFFFFFF) return cudaSuccess;
    CUtensorMap map;
    if (!make_col_tensor_map(&map, p.src, S, rows, (uint64_t)p.nworkers, (uint64_t)p.src_stride)) return cudaSuccess;
    cudaError_t e;
    if (p.lo_log >= 15) {
        // rows 128 KiB apart or more: the two-group persistent form (0.44 against 0.48 ms on 8 workers of 2^25)
        if ((e = cudaFuncSetAttribute(col4_duo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Col4Duo::SMEM_BYTES)) != cudaSuccess) return e;
        int dev = 0, sms = 0;
        if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        int64_t blocks = nruns * p.nworkers;
        if (blocks > sms) blocks = sms;
        col4_duo_kernel<<<(unsigned)blocks, 1024, Col4Duo::SMEM_BYTES, s>>>(p, map, (int)nruns, (uint32_t)rows);
    } else {
        // one block per run (0.83 against 0.91 ms on 32 workers of 2^24; blocks that start at different times
        // keep the memory system evenly loaded)
        if ((e = cudaFuncSetAttribute(col4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Col4::SMEM_BYTES)) != cudaSuccess) return e;
        col4_kernel<<<(unsigned)(nruns * p.nworkers), 512, Col4::SMEM_BYTES, s>>>(p, map, (int)nruns, (uint32_t)rows);
    }
    *launched = true;
    return cudaGetLastError();
}

// Ten stages on fp32 gradients with the squared norm of every worker's gradient gathered on the way: run sums
// in partial[worker][run] (*nruns_out of them per worker).  One-block-per-run form only; *launched stays false
// where it does not apply (rows 128 KiB apart or more, rows shorter than a run, map refused).
cudaError_t launch_col4_norm(const PassParams& p, double* partial, cudaStream_t s, bool* launched, int* nruns_out)
{
    constexpr int A = 10;
    *launched = false;
    const uint64_t S = (uint64_t)1 << p.lo_log;
    const uint64_t rows = (uint64_t)(p.d >> p.lo_log);
    const int64_t nsegs = (p.dp >> A) / 16;
    const int64_t nruns = nsegs / 8;
    if (p.lo_log >= 15 || S < 128 || nsegs % 8 != 0 || nruns * p.nworkers > 0x7FFFFFFF) return cudaSuccess;
    CUtensorMap map;
    if (!make_col_tensor_map(&map, p.src, S, rows, (uint64_t)p.nworkers, (uint64_t)p.src_stride)) return cudaSuccess;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(col4_norm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Col4::SMEM_BYTES)) != cudaSuccess) return e;
    col4_norm_kernel<<<(unsigned)(nruns * p.nworkers), 512, Col4::SMEM_BYTES, s>>>(p, map, (int)nruns, (uint32_t)rows, partial);
    *launched = true;
    *nruns_out = (int)nruns;
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
        // ten stages on fp32 gradients: the copy-engine kernels, unless the driver refuses the tensor map
        if constexpr (A == 10 && SRC == SRC_G32) {
            bool launched = false;
            const cudaError_t e = launch_col4(p, s, &launched);
            if (e != cudaSuccess || launched) return e;
        }
        if constexpr (A == 10 && SRC == SRC_G16) {
            // bf16 gradients with rows megabytes apart (the top pass of a transform longer than 2^30): 32-column
            // tiles, so that a row visit moves 64 bytes in and 128 bytes out instead of half of that (31.2 against
            // 35.4 ms on 8 workers of 2^31; the same tiles from packed bits were slower, 30.7 against 28.0 ms)
            if (p.lo_log >= 20) {
                auto wide = col_tile_kernel<A, SRC>;
                constexpr size_t wsmem = (size_t)(1 << A) * 32 * 4;
                cudaError_t e = cudaFuncSetAttribute(wide, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)wsmem);
                if (e != cudaSuccess) return e;
                const dim3 grid((unsigned)((p.dp >> A) / 32), (unsigned)p.nworkers);
                wide<<<grid, 1 << A, wsmem, s>>>(p);
                return cudaGetLastError();
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
        case SRC_WS16:
            if constexpr (A >= 6) return launch_col_one<A, SRC_WS16>(p, s);   // (second strided pass of a long decoder)
            break;
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
