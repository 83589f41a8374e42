// Contiguous-tile pass: all T = log2(tile) butterfly stages of the index bits [0, T) on tiles of
// 2^T consecutive coordinates, fused with its source (gradient load + pad + flip, packed bits,
// or an intermediate of an earlier pass) and its sink (dither + sign + pack, fp32 store, or
// flip + sum over workers).  One thread block works on one tile at a time; every thread keeps
// 32 values in registers and the block runs three register rounds of up to five stages each,
// exchanging through shared memory (row pitch 36 words: no bank conflicts in any round).
//
//   round F: register bits {0, 1, T-3, T-2, T-1}   128-bit loads, 128-bit shared stores
//   round M: register bits {2, 3, 4, m1, m2}       (m1, m2) = (10, 11), or (T-2, T-1) if T < 12
//   round L: register bits {5, 6, 7, 8, 9}         lane = bits 0..4, so lane r can own packed word r
//
// A bit that two rounds hold is transformed by the first and rides along in the second.
//
// Two kernels share these rounds:
//   row_kernel        source read by the threads themselves: gradients and packed bits (the
//                     single-pass case, transform length <= 2^15), and fp32 intermediates whose
//                     tile is too large for a separate landing buffer.
//   row_stream_kernel source = intermediate of the strided passes, fetched tile by tile with
//                     the bulk async copy engine (cp.async.bulk + mbarrier) into a landing
//                     buffer beside the work tile: the copy of tile k+1 starts as soon as
//                     round F has read tile k, and runs underneath the other rounds and the sink.
#pragma once
#include "common.cuh"

namespace fosgd {

__host__ __device__ constexpr int nth_set_bit(uint32_t mask, int n)
{
    for (int b = 0; b < 32; ++b)
        if ((mask >> b) & 1u) {
            if (n == 0) return b;
            --n;
        }
    return -1;
}

// tile offset addressed by register r when the register bits are the set bits of `mask`
__host__ __device__ constexpr int reg_offset(uint32_t mask, int r)
{
    int e = 0;
    for (int rb = 0; rb < 5; ++rb)
        if ((r >> rb) & 1) e |= 1 << nth_set_bit(mask, rb);
    return e;
}

// register-level stage mask: register bit rb is active iff its tile bit is not done yet
__host__ __device__ constexpr int active_mask(uint32_t mask, uint32_t done)
{
    int a = 0;
    for (int rb = 0; rb < 5; ++rb)
        if (!((done >> nth_set_bit(mask, rb)) & 1u)) a |= 1 << rb;
    return a;
}

__host__ __device__ constexpr int phys(int e) { return e + ((e >> 5) << 2); }

// spread the thread index over the tile bits that are not register bits (lowest first)
template <uint32_t MASK, int T>
__device__ __forceinline__ int deposit(int tid)
{
    int e = 0, k = 0;
#pragma unroll
    for (int b = 0; b < T; ++b)
        if (!((MASK >> b) & 1u)) {
            e |= ((tid >> k) & 1) << b;
            ++k;
        }
    return e;
}

template <int T>
struct RowCfg {
    static constexpr int NT = 1 << (T - 5);
    static constexpr uint32_t FMASK = 0x3u | (0x7u << (T - 3));
    static constexpr int M1 = (T >= 12) ? 10 : T - 2;
    static constexpr uint32_t MMASK = 0x1Cu | (0x3u << M1);
    static constexpr uint32_t LMASK = 0x3E0u;
    static constexpr int ACT_M = active_mask(MMASK, FMASK);
    static constexpr int ACT_L = active_mask(LMASK, FMASK | MMASK);
    static constexpr int TILE_WORDS = phys(1 << T);
    static constexpr int FLIP_WORDS = (1 << T) / 32;
    static constexpr size_t SMEM_BYTES = (size_t)(TILE_WORDS + FLIP_WORDS) * 4 + 16;  // + mbarrier
    static_assert(((FMASK | MMASK | LMASK) & ((1u << T) - 1)) == ((1u << T) - 1), "bits uncovered");
};

// parameter block of a kernel by its sink: the dither sinks carry the generator's round keys
template <int SINK> struct KernelParams { using type = PassParams; };
template <> struct KernelParams<SINK_PACK1> { using type = PassParamsRK; };
template <> struct KernelParams<SINK_PACKK> { using type = PassParamsRK; };
template <int SINK>
inline typename KernelParams<SINK>::type kernel_params(const PassParams& p)
{
    if constexpr (SINK == SINK_PACK1 || SINK == SINK_PACKK) return with_round_keys(p);
    else return p;
}

// Registers are capped at 64 per thread (2048 resident threads per SM).  The store and dither
// sinks need no more by themselves.  The flip + accumulate sink holds 32 values and 32 sums per
// thread and would take ~95: capped, it spills a few words but runs twice the warps, which is
// worth 5 % on the 2^24 workload.
// (Three blocks of the one-dither sink at 40 registers were measured slower, 0.96 against 0.80 ms.)
template <int T, int SINK>
__host__ __device__ constexpr int min_blocks()
{
    return 1 << (15 - T);
}

// ---- the three rounds on the padded tile ---------------------------------------------------
template <int T>
__device__ __forceinline__ void store_round_F(float* smem, int baseF, const float (&v)[32])
{
#pragma unroll
    for (int g = 0; g < 8; ++g)
        *reinterpret_cast<float4*>(smem + phys(baseF | (g << (T - 3)))) =
            make_float4(v[4 * g + 0], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
}

template <int T>
__device__ __forceinline__ void round_M(float* smem, int baseM, float (&v)[32])
{
    using C = RowCfg<T>;
    float* const pm = smem + phys(baseM);
#pragma unroll
    for (int r = 0; r < 32; ++r) v[r] = pm[phys(reg_offset(C::MMASK, r))];
    butterflies32<C::ACT_M>(v);
#pragma unroll
    for (int r = 0; r < 32; ++r) pm[phys(reg_offset(C::MMASK, r))] = v[r];
}

__device__ __forceinline__ void load_round_L(const float* smem, int baseL, float (&v)[32])
{
    const float* const pl = smem + phys(baseL);
#pragma unroll
    for (int r = 0; r < 32; ++r) v[r] = pl[phys(r << 5)];
}

// ---- sinks: register r holds coordinate i0 + 32 r, lane = coordinate & 31 --------------------
__device__ __forceinline__ void sink_ws(const PassParams& p, int n, int64_t i0, const float (&v)[32])
{
    float* dst = static_cast<float*>(p.dst) + (int64_t)n * p.dst_stride + i0;
#pragma unroll
    for (int r = 0; r < 32; ++r) dst[r << 5] = v[r] * p.scale;
}

// Sign bits are shifted into a per-lane mask (bit r = sign of register r), then the 32 x 32 bit
// matrix is transposed across the warp so that lane r owns packed word r.
__device__ __forceinline__ void sink_pack1(const PassParamsRK& p, int n, uint32_t id, int64_t i0, uint32_t lane,
                                           const float (&v)[32], float amp)
{
    const uint32_t cbase = ((uint32_t)(i0 >> 7) << 5) + lane;
    const float dc = p.dither_c * amp;
    const float c2 = 2.f * dc, c0 = -16777215.f * dc;
    uint32_t neg = 0;
#pragma unroll
    for (int m = 7; m >= 0; --m) {
        const uint4 w = rng_words_dither(p, id, 1u, cbase + 32u * m);
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int q = 3; q >= 0; --q) {
            // z = (2 k24 + 1 - 2^24) c + y, k24 = top 24 bits of the word (two roundings: the two operations
            // are independent of each other's latency, 4 % faster than the single-rounding form of the
            // K-dither sink, and with one dither per coordinate the ties stay far inside the allowance)
            const float z = fmaf((float)(ww[q] >> 8), c2, v[4 * m + q] + c0);
            neg = __funnelshift_l(__float_as_uint(z), neg, 1);  // neg = neg << 1 | sign(z)
        }
    }
    const uint32_t mine = warp_transpose_bits(~neg, lane);
    uint32_t* dst = static_cast<uint32_t*>(p.dst) + (int64_t)n * p.dst_stride;
    dst[((i0 - lane) >> 5) + lane] = mine;
}

// K dithers: the count c_r of non-negative signs of register r is kept bit-sliced, plane b being a
// per-lane word whose bit r is bit b of c_r.  Each dither yields the sign mask of the 32 registers
// (funnel shifts, as above), which a ripple of AND/XOR adds to the planes; at the end every plane
// goes through the same warp transpose as the one-dither sink.  No per-register counters.
__device__ __forceinline__ void sink_packK(const PassParamsRK& p, int n, uint32_t id, int64_t i0, uint32_t lane,
                                           const float (&v)[32], float amp)
{
    const uint32_t cbase = ((uint32_t)(i0 >> 7) << 5) + lane;
    const float dc = p.dither_c * amp;
    uint32_t plane[8];
#pragma unroll
    for (int b = 0; b < 8; ++b) plane[b] = 0u;
    for (int k = 0; k < p.K; ++k) {
        uint32_t neg = 0;
#pragma unroll
        for (int m = 7; m >= 0; --m) {
            const uint4 w = rng_words_dither(p, id, 1u + (uint32_t)k, cbase + 32u * m);
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int q = 3; q >= 0; --q) {
                const float z = fmaf(fmaf((float)(ww[q] >> 8), 2.f, -16777215.f), dc, v[4 * m + q]);
                neg = __funnelshift_l(__float_as_uint(z), neg, 1);
            }
        }
        uint32_t carry = ~neg;   // bit r: register r counts one more
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            if (b < p.P) {
                const uint32_t t = plane[b] & carry;
                plane[b] ^= carry;
                carry = t;
            }
        }
    }
    uint32_t* dst = static_cast<uint32_t*>(p.dst) + (int64_t)n * p.dst_stride + ((i0 - lane) >> 5) + lane;
#pragma unroll
    for (int b = 0; b < 8; ++b)
        if (b < p.P) dst[(int64_t)b * (p.dp >> 5)] = warp_transpose_bits(plane[b], lane);
}

__device__ __forceinline__ void sink_final_store(const PassParams& p, int64_t i0, const float (&accv)[32], float amp)
{
    float* dst = static_cast<float*>(p.dst);
    const float sc = p.scale * amp;
#pragma unroll
    for (int r = 0; r < 32; ++r) {
        const int64_t i = i0 + (r << 5);
        if (i < p.d_out) {
            float o = accv[r];
            if (p.overwrite == 2) {
                dst[i] = fmaf(o, sc, dst[i]);   // dst += scale * sum (the descent step on top of the decoder)
            } else {
                if (!p.overwrite) o += dst[i];
                dst[i] = o * sc;
            }
        }
    }
}

// =============================================================================================
// row_kernel: sources read by the threads themselves (single-pass transforms)
// =============================================================================================
template <int T, int SRC, int SINK>
__global__ void __launch_bounds__(1 << (T - 5), min_blocks<T, SINK>()) row_kernel(const typename KernelParams<SINK>::type p)
{
    using C = RowCfg<T>;
    extern __shared__ __align__(16) float smem[];
    uint32_t* const fw = reinterpret_cast<uint32_t*>(smem + C::TILE_WORDS);

    const int tid = threadIdx.x;
    const uint32_t lane = tid & 31;
    const int64_t tile_base = (int64_t)blockIdx.x << T;
    constexpr bool kLoopWorkers = (SINK == SINK_FINAL);
    constexpr bool kFlips = (SRC == SRC_G32 || SRC == SRC_G16 || SINK == SINK_FINAL);
    const int n_begin = kLoopWorkers ? 0 : (int)blockIdx.y;
    const int n_end = kLoopWorkers ? p.nworkers : n_begin + 1;
    // one amplitude per tile (a block of the blocked mode is at least a tile): thread 0 reads it
    // first, so that its latency hides behind the tile load, and parks it in shared memory until
    // the sink (the barriers of the exchange rounds order the two)
    __shared__ float s_amp;
    if (tid == 0) s_amp = (!kLoopWorkers || p.amp_mode == AMP_SCALE) ? amplitude_at(p, n_begin, tile_base) : 1.f;

    const int baseF = deposit<C::FMASK, T>(tid);
    const int baseM = deposit<C::MMASK, T>(tid);
    const int baseL = deposit<C::LMASK, T>(tid);
    const int64_t i0 = tile_base + baseL;  // coordinate held in register 0 of round L

    float accv[32];
    if (kLoopWorkers) {
#pragma unroll
        for (int r = 0; r < 32; ++r) accv[r] = 0.f;
    }

    for (int n = n_begin; n < n_end; ++n) {
        const uint32_t id = p.id0 + (uint32_t)n;
        const float wamp = (kLoopWorkers && p.amp_mode == AMP_WEIGHT) ? amplitude_at(p, n, tile_base) : 1.f;
        if (kFlips) {
            if (kLoopWorkers) __syncthreads();  // previous worker's readers of fw and of the tile
            if (tid < C::FLIP_WORDS / 4) {
                const uint4 w = rng_words(p.rng, id, 0u, (uint32_t)(tile_base >> 7) + (uint32_t)tid);
                reinterpret_cast<uint4*>(fw)[tid] = w;
            }
            __syncthreads();
        }

        float v[32];
        // ---------------- round F: load ----------------
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const int e0 = baseF | (g << (T - 3));
            const int64_t i = tile_base + e0;
            float x0, x1, x2, x3;
            if (SRC == SRC_G32) {
                const float* src = static_cast<const float*>(p.src) + (int64_t)n * p.src_stride;
                if (i + 3 < p.d) {
                    const float4 q = __ldcs(reinterpret_cast<const float4*>(src + i));
                    x0 = q.x; x1 = q.y; x2 = q.z; x3 = q.w;
                } else {
                    x0 = (i + 0 < p.d) ? src[i + 0] : 0.f;
                    x1 = (i + 1 < p.d) ? src[i + 1] : 0.f;
                    x2 = (i + 2 < p.d) ? src[i + 2] : 0.f;
                    x3 = 0.f;
                }
            } else if (SRC == SRC_G16) {
                const uint16_t* src = static_cast<const uint16_t*>(p.src) + (int64_t)n * p.src_stride;
                uint32_t lo, hi;
                if (i + 3 < p.d) {
                    const uint2 q = __ldcs(reinterpret_cast<const uint2*>(src + i));
                    lo = q.x; hi = q.y;
                } else {
                    const uint32_t h0 = (i + 0 < p.d) ? src[i + 0] : 0u;
                    const uint32_t h1 = (i + 1 < p.d) ? src[i + 1] : 0u;
                    const uint32_t h2 = (i + 2 < p.d) ? src[i + 2] : 0u;
                    lo = h0 | (h1 << 16); hi = h2;
                }
                x0 = __uint_as_float(lo << 16); x1 = __uint_as_float(lo & 0xFFFF0000u);
                x2 = __uint_as_float(hi << 16); x3 = __uint_as_float(hi & 0xFFFF0000u);
            } else if (SRC == SRC_WS) {
                const float* src = static_cast<const float*>(p.src) + (int64_t)n * p.src_stride;
                const float4 q = __ldcs(reinterpret_cast<const float4*>(src + i));
                x0 = q.x; x1 = q.y; x2 = q.z; x3 = q.w;
            } else {  // SRC_BITS
                const uint32_t* src = static_cast<const uint32_t*>(p.src) + (int64_t)n * p.src_stride + (i >> 5);
                const uint32_t pos = (uint32_t)i & 31u;
                if (p.P == 1) {
                    const uint32_t w = __ldg(src) >> pos;
                    x0 = (w & 1u) ? 1.f : -1.f; x1 = (w & 2u) ? 1.f : -1.f;
                    x2 = (w & 4u) ? 1.f : -1.f; x3 = (w & 8u) ? 1.f : -1.f;
                } else {
                    const int64_t pw = p.dp >> 5;
                    x0 = plane_value(src, pw, p.P, p.K, pos + 0); x1 = plane_value(src, pw, p.P, p.K, pos + 1);
                    x2 = plane_value(src, pw, p.P, p.K, pos + 2); x3 = plane_value(src, pw, p.P, p.K, pos + 3);
                }
            }
            if (SRC == SRC_G32 || SRC == SRC_G16) {
                const uint32_t w = fw[e0 >> 5];
                const uint32_t pos = (uint32_t)e0 & 31u;
                x0 = flip_by_bit(x0, w, pos + 0); x1 = flip_by_bit(x1, w, pos + 1);
                x2 = flip_by_bit(x2, w, pos + 2); x3 = flip_by_bit(x3, w, pos + 3);
            }
            v[4 * g + 0] = x0; v[4 * g + 1] = x1; v[4 * g + 2] = x2; v[4 * g + 3] = x3;
        }
        butterflies32<31>(v);
        store_round_F<T>(smem, baseF, v);
        __syncthreads();
        round_M<T>(smem, baseM, v);
        __syncthreads();
        load_round_L(smem, baseL, v);
        butterflies32<C::ACT_L>(v);

        if constexpr (SINK == SINK_WS) {
            sink_ws(p, n, i0, v);
        } else if constexpr (SINK == SINK_PACK1) {
            sink_pack1(p, n, id, i0, lane, v, s_amp);
        } else if constexpr (SINK == SINK_PACKK) {
            sink_packK(p, n, id, i0, lane, v, s_amp);
        } else {
            const uint32_t* const fwl = fw + ((baseL - (int)lane) >> 5);
#pragma unroll
            for (int r = 0; r < 32; ++r) accv[r] = fmaf(flip_by_bit(v[r], fwl[r], lane), wamp, accv[r]);
        }
    }
    if (SINK == SINK_FINAL) sink_final_store(p, i0, accv, s_amp);
}

// =============================================================================================
// row_stream_kernel: tiles of an intermediate (fp32 or fp16) fetched by bulk async copies
// =============================================================================================
// bumped when a bounded wait on a bulk copy gave up (one counter per translation unit that includes this file)
static __device__ int g_async_wait_timeouts;

// one elected thread: announce `bytes` on the barrier and start the copy global -> shared
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar)
{
    // order this block's earlier generic-proxy accesses to the buffer before the async-proxy write
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// A streamed tile lands in a buffer of its own beside the padded work tile, so the copy of tile
// k+1 starts as soon as round F has read tile k out of it and runs underneath rounds M and L
// and the sink.  That needs the landing buffer to fit: fp16 tiles, or fp32 tiles up to 2^13.
template <int T, int SRC>
struct StreamCfg {
    using C = RowCfg<T>;
    static constexpr uint32_t kElem = (SRC == SRC_WS16) ? 2u : 4u;
    static constexpr uint32_t kTileBytes = kElem << T;
    static constexpr bool kFits = (SRC == SRC_WS16) || (T <= 13);
    static constexpr size_t SMEM_BYTES = C::SMEM_BYTES + kTileBytes;
};

template <int T, int SRC, int SINK>
__global__ void __launch_bounds__(1 << (T - 5), min_blocks<T, SINK>()) row_stream_kernel(const typename KernelParams<SINK>::type p, const int64_t ntiles)
{
    using C = RowCfg<T>;
    using S = StreamCfg<T, SRC>;
    static_assert(SRC == SRC_WS || SRC == SRC_WS16, "streamed sources only");
    extern __shared__ __align__(16) float smem[];
    uint32_t* const fw = reinterpret_cast<uint32_t*>(smem + C::TILE_WORDS);
    uint64_t* const bar = reinterpret_cast<uint64_t*>(fw + C::FLIP_WORDS);
    float* const landing = reinterpret_cast<float*>(bar + 2);
    constexpr uint32_t kElem = S::kElem;
    constexpr uint32_t kTileBytes = S::kTileBytes;

    const int tid = threadIdx.x;
    const uint32_t lane = tid & 31;
    constexpr bool kFinal = (SINK == SINK_FINAL);
    // SINK_FINAL: this block's tile is fixed, one amplitude scales the sum (AMP_SCALE) or every
    // worker brings its own weight (AMP_WEIGHT); pack sinks read the amplitude of each item
    // (parked in shared memory until the store; the barriers of the worker loop order the two)
    __shared__ float s_amp_final;
    if (tid == 0) s_amp_final = (kFinal && p.amp_mode == AMP_SCALE) ? amplitude_at(p, 0, (int64_t)blockIdx.x << T) : 1.f;
    // work items: SINK_FINAL -> this block's tile for every worker in turn;
    //             otherwise  -> (worker, tile) pairs strided over the grid
    const int64_t nitems = kFinal ? (int64_t)p.nworkers
                                  : (ntiles * p.nworkers - (int64_t)blockIdx.x + gridDim.x - 1) / gridDim.x;

    const int baseF = deposit<C::FMASK, T>(tid);
    const int baseM = deposit<C::MMASK, T>(tid);
    const int baseL = deposit<C::LMASK, T>(tid);

    auto item_worker = [&](int64_t j) -> int { return kFinal ? (int)j : (int)((blockIdx.x + j * gridDim.x) / ntiles); };
    auto item_tile = [&](int64_t j) -> int64_t { return kFinal ? (int64_t)blockIdx.x : (int64_t)((blockIdx.x + j * gridDim.x) % ntiles); };
    auto item_src = [&](int64_t j) -> const char* {
        return static_cast<const char*>(p.src) + ((int64_t)item_worker(j) * p.src_stride + (item_tile(j) << T)) * kElem;
    };

    if (tid == 0) {
        mbar_init(bar, 1);
        if (nitems > 0) bulk_load(landing, item_src(0), kTileBytes, bar);
    }
    __syncthreads();

    float accv[32];
    if (kFinal) {
#pragma unroll
        for (int r = 0; r < 32; ++r) accv[r] = 0.f;
    }
    uint32_t parity = 0;

    for (int64_t j = 0; j < nitems; ++j) {
        const int n = item_worker(j);
        const int64_t tile_base = item_tile(j) << T;
        const int64_t i0 = tile_base + baseL;
        const uint32_t id = p.id0 + (uint32_t)n;
        const float amp = (!kFinal || p.amp_mode == AMP_WEIGHT) ? amplitude_at(p, n, tile_base) : 1.f;

        // bounded wait; the block then agrees on the outcome, so that it stops as a whole
        if (!__syncthreads_and(mbar_wait(bar, parity) ? 1 : 0)) {
            // the one copy in flight is the one that did not arrive: a second bounded wait, so that the
            // engine is not left writing into shared memory that the next block of this SM may own
            if (tid == 0) {
                atomicAdd(&g_async_wait_timeouts, 1);
                mbar_wait(bar, parity);
                mbar_inval(bar);
            }
            __syncthreads();
            return;
        }
        parity ^= 1u;

        float v[32];
        // round F reads the tile as it arrived (linear) and writes the padded exchange layout
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const int e0 = baseF | (g << (T - 3));
            if (SRC == SRC_WS) {
                const float4 q = *reinterpret_cast<const float4*>(landing + e0);
                v[4 * g + 0] = q.x; v[4 * g + 1] = q.y; v[4 * g + 2] = q.z; v[4 * g + 3] = q.w;
            } else {
                const uint2 q = *reinterpret_cast<const uint2*>(reinterpret_cast<const __half*>(landing) + e0);
                const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&q.x));
                const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&q.y));
                v[4 * g + 0] = a.x; v[4 * g + 1] = a.y; v[4 * g + 2] = b.x; v[4 * g + 3] = b.y;
            }
        }
        butterflies32<31>(v);
        store_round_F<T>(smem, baseF, v);
        fence_generic_before_async();   // (the landing buffer is only read by the threads, never written)
        __syncthreads();   // round F complete: the landing buffer is free, nobody is in the previous item
        if (tid == 0 && j + 1 < nitems) bulk_load(landing, item_src(j + 1), kTileBytes, bar);
        if (kFinal && tid < C::FLIP_WORDS / 4) {
            const uint4 w = rng_words(p.rng, id, 0u, (uint32_t)(tile_base >> 7) + (uint32_t)tid);
            reinterpret_cast<uint4*>(fw)[tid] = w;
        }
        round_M<T>(smem, baseM, v);
        __syncthreads();
        load_round_L(smem, baseL, v);
        __syncthreads();   // the tile lives in registers: the work tile may be overwritten by the next round F
        butterflies32<C::ACT_L>(v);

        if constexpr (SINK == SINK_WS) {
            sink_ws(p, n, i0, v);
        } else if constexpr (SINK == SINK_PACK1) {
            sink_pack1(p, n, id, i0, lane, v, amp);
        } else if constexpr (SINK == SINK_PACKK) {
            sink_packK(p, n, id, i0, lane, v, amp);
        } else {
            const uint32_t* const fwl = fw + ((baseL - (int)lane) >> 5);
#pragma unroll
            for (int r = 0; r < 32; ++r) accv[r] = fmaf(flip_by_bit(v[r], fwl[r], lane), amp, accv[r]);
        }
    }
    if (kFinal) sink_final_store(p, ((int64_t)blockIdx.x << T) + baseL, accv, s_amp_final);
}

// ---- launchers ---------------------------------------------------------------------------------
template <int T, int SRC, int SINK>
cudaError_t launch_row_one(const PassParams& p, cudaStream_t s)
{
    using C = RowCfg<T>;
    const int64_t ntiles = p.dp >> T;
    if constexpr ((SRC == SRC_WS || SRC == SRC_WS16) && StreamCfg<T, SRC>::kFits) {
        auto kern = row_stream_kernel<T, SRC, SINK>;
        constexpr size_t kSmem = StreamCfg<T, SRC>::SMEM_BYTES;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        if (e != cudaSuccess) return e;
        int64_t blocks = ntiles;
        if (SINK != SINK_FINAL) {
            int dev = 0, sms = 0, per_sm = 0;
            if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
            if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
            if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, C::NT, kSmem)) != cudaSuccess) return e;
            blocks = (int64_t)sms * (per_sm > 0 ? per_sm : 1);
            if (blocks > ntiles * p.nworkers) blocks = ntiles * p.nworkers;
        }
        kern<<<(unsigned)blocks, C::NT, kSmem, s>>>(kernel_params<SINK>(p), ntiles);
    } else {
        auto kern = row_kernel<T, SRC, SINK>;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        const dim3 grid((unsigned)ntiles, SINK == SINK_FINAL ? 1u : (unsigned)p.nworkers);
        kern<<<grid, C::NT, C::SMEM_BYTES, s>>>(kernel_params<SINK>(p));
    }
    return cudaGetLastError();
}

template <int T>
cudaError_t launch_row_T(int src, int sink, const PassParams& p, cudaStream_t s)
{
#define FOSGD_ROW_CASE(SRC_, SINK_) \
    if (src == SRC_ && sink == SINK_) return launch_row_one<T, SRC_, SINK_>(p, s);
    FOSGD_ROW_CASE(SRC_G32, SINK_WS)
    FOSGD_ROW_CASE(SRC_G16, SINK_WS)
    FOSGD_ROW_CASE(SRC_WS, SINK_WS)
    FOSGD_ROW_CASE(SRC_G32, SINK_PACK1)
    FOSGD_ROW_CASE(SRC_G16, SINK_PACK1)
    FOSGD_ROW_CASE(SRC_WS, SINK_PACK1)
    FOSGD_ROW_CASE(SRC_G32, SINK_PACKK)
    FOSGD_ROW_CASE(SRC_WS, SINK_PACKK)
    FOSGD_ROW_CASE(SRC_BITS, SINK_FINAL)
    FOSGD_ROW_CASE(SRC_WS, SINK_FINAL)
    FOSGD_ROW_CASE(SRC_WS16, SINK_FINAL)
#undef FOSGD_ROW_CASE
    return cudaErrorInvalidValue;
}

}  // namespace fosgd
