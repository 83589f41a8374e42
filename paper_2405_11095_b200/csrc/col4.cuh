// Strided pass of ten stages (A = 10) on fp32 gradients, tiles staged by the tensor copy engine, four
// columns per thread.  A tile is 1024 rows x 16 columns, delivered densely (64-byte rows) by four
// cp.async.bulk.tensor box copies.  A thread owns four adjacent columns of eight rows (32
// registers); the ten row bits are covered by three register rounds of three bits each (7..9,
// 4..6, 1..3) and one shuffle stage for row bit 0, which stays in the lane so that a quarter-warp
// (4 column quads x 2 adjacent rows) always touches 128 contiguous bytes of the dense tile: every
// 128-bit shared-memory access is conflict free without padding.
//
// Work comes in runs of eight adjacent tiles (128 columns of the same 1024 rows) of one worker.
// The 128 flips of a row segment of a run are exactly one generator call, so no flip word is
// generated eight times over.  Two kernels share the rounds:
//   col4_run  one block of 512 threads per run, two landing buffers (the copy of the tile two
//             positions ahead is issued as soon as the current tile sits in registers for its
//             last round).  Fastest when rows are up to 64 KiB apart (transform length 2^24).
//   col4_duo  one persistent block of 1024 threads per SM, two groups of 512 taking tiles in turn
//             over three landing buffers.  Fastest when rows are further apart (2^25).
// Every wait on a copy is bounded; a block or group whose wait runs out stops as a whole, gives the
// copies still in flight one more bounded wait and reports through the counter it was given.
// (The same rounds on bf16 gradients and on the fp32 intermediate in place, as the strided passes of
// a 2^31 transform, were built and measured too: 302 and 410 ms against 279 and 393 ms of the plain
// kernels on 64 workers, so those passes keep the plain kernels.)
#pragma once
#include <cuda.h>   // CUtensorMap

#include "common.cuh"

namespace fosgd {

// x with its sign flipped iff bit (31 - sh) of word is set
__device__ __forceinline__ float flip_at(float x, uint32_t word, uint32_t sh)
{
    return __uint_as_float(__float_as_uint(x) ^ ((word << sh) & 0x80000000u));
}

// How the 512 threads of a run meet: the whole block (the stand-alone kernel), or one group of a larger
// block on a named barrier (the fused encoder, where another group works beside this one).
struct BlockSync {
    static __device__ __forceinline__ void sync() { __syncthreads(); }
    static __device__ __forceinline__ bool all(bool ok) { return __syncthreads_and(ok ? 1 : 0) != 0; }
};
template <int ID, int NTHREADS>
struct GroupSync {
    static __device__ __forceinline__ void sync() { group_sync(ID, NTHREADS); }
    static __device__ __forceinline__ bool all(bool ok) { return group_all(ID, NTHREADS, ok); }
};

// Tensor map over fp32 gradients as a strided pass of ten stages sees them: (S columns, whole rows, workers),
// boxes of 16 columns x 256 rows.  False if the driver entry point is missing or refuses the geometry.
bool make_col_tensor_map(CUtensorMap* map, const void* base, uint64_t S, uint64_t rows, uint64_t workers,
                         uint64_t worker_stride_elems);

struct Col4 {
    static constexpr int A = 10, ROWS = 1 << A, RUN = 8, THREADS = 512;
    static constexpr int NBUF = 2;   // landing buffers (copies in flight ahead of the tile being transformed)
    static constexpr uint32_t LAND_BYTES = ROWS * 16 * 4;
    // landing buffers, the flips of a run, one barrier per buffer
    static constexpr size_t SMEM_BYTES = (size_t)NBUF * LAND_BYTES + 16384 + 32;
};

// One run: tiles seg0 .. seg0 + 7 (16-column segments of the matrix view) of worker n, by the 512 threads
// of a block or group (tid = 0 .. 511).  timeouts: device counter bumped when a bounded wait gave up;
// the return value says whether the run completed (the same for all threads).
// NORM: also add up the squares of the run's gradient entries (fp32 within a tile, fp64 across tiles and threads,
// fixed order) and leave the sum in *run_sumsq, so that a norm needs no second pass over the gradients.
template <typename S, bool NORM = false>
__device__ __forceinline__ bool col4_run(const PassParams& p, const CUtensorMap* tmap, const uint32_t full_rows, const int n,
                                         const uint32_t seg0, unsigned char* smem_raw, const int tid, int* timeouts,
                                         double* run_sumsq = nullptr)
{
    using C = Col4;
    constexpr int A = C::A, ROWS = C::ROWS, RUN = C::RUN, NBUF = C::NBUF;
    constexpr uint32_t LAND_BYTES = C::LAND_BYTES;
    unsigned char* const land0 = smem_raw;
    uint32_t* const flips = reinterpret_cast<uint32_t*>(smem_raw + NBUF * LAND_BYTES);
    uint64_t* const full = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(flips) + 16384);

    const uint32_t kq = tid & 3, r0 = (tid >> 2) & 1, u = tid >> 3;     // column quad, row bit 0, six more row bits
    const uint32_t step = 1u << p.lo_log;
    const uint32_t d32 = (uint32_t)p.d;
    const uint32_t lo_run = (seg0 << 4) & (step - 1u);
    const uint32_t hi = (seg0 << 4) >> p.lo_log;
    const uint32_t i_run = (hi << (p.lo_log + A)) + lo_run;            // row 0, column 0 of the run

    if (tid == 0) {
#pragma unroll
        for (int b = 0; b < NBUF; ++b) mbar_init(full + b, 1);
    }
    S::sync();

    int issued = 0, taken = 0;   // thread 0 only
    bool completed = true;
    double sumsq = 0.0;
    auto issue = [&](int t) {
        uint64_t* const bar_full = full + (t % NBUF);
        const uint32_t dst0 = smem_u32(land0 + (t % NBUF) * LAND_BYTES);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar_full)), "r"(LAND_BYTES) : "memory");
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                         ::"r"(dst0 + (LAND_BYTES / 4) * q), "l"(tmap), "r"((int)(lo_run + 16u * t)),
                           "r"((int)((hi << A) + 256 * q)), "r"(n), "r"(smem_u32(bar_full)) : "memory");
        }
        ++issued;
    };
    if (tid == 0) {
#pragma unroll
        for (int b = 0; b < NBUF; ++b) issue(b);
    }
    {
        // the run's flips: rows tid and tid + 512, four words (128 columns) each = one generator call
        const uint32_t id = p.id0 + (uint32_t)n;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const uint32_t row = (uint32_t)tid + 512u * k;
            reinterpret_cast<uint4*>(flips)[row] = rng_words(p.rng, id, 0u, (i_run + row * step) >> 7);
        }
    }
    S::sync();

    for (int t = 0; t < RUN; ++t) {
        float* const buf = reinterpret_cast<float*>(land0 + (t % NBUF) * LAND_BYTES);
        // bounded wait; the block then agrees on the outcome, so that it stops as a whole
        if (!S::all(mbar_wait(full + (t % NBUF), (uint32_t)((t / NBUF) & 1)))) {
            if (tid == 0) atomicAdd(timeouts, 1);
            completed = false;
            break;
        }
        if (tid == 0) ++taken;
        {
            // the map covers whole rows only: a last partial row of the gradient is patched in
            const uint32_t row_p = full_rows - (hi << A);                  // tile-local index of that row
            if (row_p < (uint32_t)ROWS) {
                if (tid < 16) {
                    const uint32_t i = full_rows * step + lo_run + 16u * t + (uint32_t)tid;
                    if (i < d32) buf[(row_p << 4) + tid] = (static_cast<const float*>(p.src) + (int64_t)n * p.src_stride)[i];
                }
                S::sync();
            }
        }
        float v[32];
        // ---- round 1: row bits 7..9 in registers; source read, flips applied ----
        {
            const uint32_t sh = 31u - ((uint32_t)(t & 1) * 16u + 4u * kq);
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const uint32_t row = ((uint32_t)g << 7) | (u << 1) | r0;
                const float4 q = *reinterpret_cast<const float4*>(buf + (row << 4) + 4u * kq);
                const uint32_t w = flips[(row << 2) + (t >> 1)];
                v[4 * g + 0] = flip_at(q.x, w, sh); v[4 * g + 1] = flip_at(q.y, w, sh - 1u);
                v[4 * g + 2] = flip_at(q.z, w, sh - 2u); v[4 * g + 3] = flip_at(q.w, w, sh - 3u);
            }
            if (NORM) {
                float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    s0 = fmaf(v[4 * g + 0], v[4 * g + 0], s0); s1 = fmaf(v[4 * g + 1], v[4 * g + 1], s1);
                    s2 = fmaf(v[4 * g + 2], v[4 * g + 2], s2); s3 = fmaf(v[4 * g + 3], v[4 * g + 3], s3);
                }
                sumsq += (double)((s0 + s1) + (s2 + s3));
            }
            butterflies32<28>(v);
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const uint32_t row = ((uint32_t)g << 7) | (u << 1) | r0;
                *reinterpret_cast<float4*>(buf + (row << 4) + 4u * kq) =
                    make_float4(v[4 * g + 0], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
            }
        }
        S::sync();
        // ---- round 2: row bits 4..6 ----
        {
            float* const p2 = buf + ((((u >> 3) << 7) | ((u & 7u) << 1) | r0) << 4) + 4u * kq;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const float4 q = *reinterpret_cast<const float4*>(p2 + (g << 8));
                v[4 * g + 0] = q.x; v[4 * g + 1] = q.y; v[4 * g + 2] = q.z; v[4 * g + 3] = q.w;
            }
            butterflies32<28>(v);
#pragma unroll
            for (int g = 0; g < 8; ++g)
                *reinterpret_cast<float4*>(p2 + (g << 8)) = make_float4(v[4 * g + 0], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
        }
        S::sync();
        // ---- round 3: row bits 1..3, then row bit 0 across lanes ----
        {
            const float* const p3 = buf + (((u << 4) | r0) << 4) + 4u * kq;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const float4 q = *reinterpret_cast<const float4*>(p3 + (g << 5));
                v[4 * g + 0] = q.x; v[4 * g + 1] = q.y; v[4 * g + 2] = q.z; v[4 * g + 3] = q.w;
            }
        }
        fence_generic_before_async();   // this thread's stores into the buffer, before the copy engine reuses it
        S::sync();                // the tile lives in registers
        if (tid == 0 && t + NBUF < RUN) issue(t + NBUF);
        butterflies32<28>(v);
        const float sgn = r0 ? -1.f : 1.f;
#pragma unroll
        for (int r = 0; r < 32; ++r) v[r] = fmaf(sgn, v[r], __shfl_xor_sync(0xFFFFFFFFu, v[r], 4));
        float* const o = static_cast<float*>(p.dst) + (int64_t)n * p.dst_stride + i_run + 16u * t + 4u * kq + ((u << 4) | r0) * step;
#pragma unroll
        for (int g = 0; g < 8; ++g)
            __stcg(reinterpret_cast<float4*>(o + (uint32_t)(g << 1) * step),
                   make_float4(v[4 * g + 0], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]));   // L2 only: read next by another pass
    }
    // In a healthy run every issued copy has been taken; after a timeout the copies still in flight get
    // one more bounded wait, so that the engine is not left writing into shared memory that the next
    // block of this SM may own.
    S::sync();
    if (tid == 0) {
        for (int k = taken; k < issued; ++k) mbar_wait(full + (k % NBUF), (uint32_t)((k / NBUF) & 1));
#pragma unroll
        for (int b = 0; b < NBUF; ++b) mbar_inval(full + b);
    }
    if (NORM) {
        // lanes, then warps, in a fixed order (the flips are no longer needed: their space holds the warps' sums)
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) sumsq += __shfl_xor_sync(0xFFFFFFFFu, sumsq, s);
        double* const wsum = reinterpret_cast<double*>(flips);
        if ((tid & 31) == 0) wsum[tid >> 5] = sumsq;
        S::sync();
        if (tid == 0) {
            double total = 0.0;
            for (int w = 0; w < C::THREADS / 32; ++w) total += wsum[w];
            *run_sumsq = total;
        }
    }
    return completed;
}

// ---- the same transform by two groups of 512 threads that take tiles in turn --------------------
// One persistent block per SM (1024 threads) walks a flat list of tiles (its runs, eight tiles each)
// over three landing buffers: tile tt belongs to group tt % 2 and lands in buffer tt % 3, and the
// group that has pulled a tile into registers for its last round issues the copies of the tile three
// positions ahead into the buffer it just freed, so loads stay in flight while one group computes and
// the other stores.  The groups share nothing but the buffers' barriers: each keeps the flips of its
// own four tiles of the current run (16 bits per row and tile, 8 KiB), made at its first tile of the
// run.
struct Col4Duo {
    static constexpr uint32_t LAND_BYTES = 1024 * 16 * 4;
    static constexpr size_t SMEM_BYTES = (size_t)3 * LAND_BYTES + 2 * 8192 + 64;
};

__device__ __forceinline__ void col4_duo(const PassParams& p, const CUtensorMap* tmap, const uint32_t nruns,
                                         const uint32_t full_rows, const uint32_t total, unsigned char* smem_raw, int* timeouts)
{
    using C = Col4Duo;
    constexpr int A = 10, ROWS = 1 << A, GT = 512;
    constexpr uint32_t LAND_BYTES = C::LAND_BYTES;
    const int tid = threadIdx.x;
    const int g = tid >> 9, gt = tid & (GT - 1);
    uint2* const flips = reinterpret_cast<uint2*>(smem_raw + 3 * LAND_BYTES + g * 8192);   // this group's: [1024 rows] x 4 tiles x 16 bits
    uint64_t* const full = reinterpret_cast<uint64_t*>(smem_raw + 3 * LAND_BYTES + 2 * 8192);
    int* const s_stop = reinterpret_cast<int*>(full + 4);                  // set when a bounded wait gave up: nothing more is issued
    int* const s_issued = s_stop + 1;                                      // [3] copies issued into each buffer
    int* const s_taken = s_stop + 4;                                       // [3] tiles taken out of each buffer

    const uint32_t kq = gt & 3, r0 = (gt >> 2) & 1, u = gt >> 3;
    const uint32_t step = 1u << p.lo_log;
    const uint32_t d32 = (uint32_t)p.d;
    const uint32_t first = blockIdx.x, stride = gridDim.x;
    const uint32_t nitems = first < total ? (total - first + stride - 1u) / stride : 0u;
    const uint32_t ntiles = nitems * 8u;

    struct Item { int n; uint32_t lo_run, hi; };
    auto item_at = [&](uint32_t j) {
        const uint32_t q = first + j * stride;
        const uint32_t n = q / nruns, seg0 = (q - n * nruns) * 8u;
        return Item{(int)n, (seg0 << 4) & (step - 1u), (seg0 << 4) >> p.lo_log};
    };
    auto issue = [&](uint32_t tt, const Item& it) {
        if (*(volatile int*)s_stop) return;
        const uint32_t t = tt & 7u, b = tt % 3u;
        const uint32_t dst0 = smem_u32(smem_raw + b * LAND_BYTES);
        atomicAdd(s_issued + b, 1);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(full + b)), "r"(LAND_BYTES) : "memory");
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                         ::"r"(dst0 + (LAND_BYTES / 4) * q), "l"(tmap), "r"((int)(it.lo_run + 16u * t)),
                           "r"((int)((it.hi << A) + 256 * q)), "r"(it.n), "r"(smem_u32(full + b)) : "memory");
        }
    };

    if (tid == 0) {
        for (int b = 0; b < 3; ++b) {
            mbar_init(full + b, 1);
            s_issued[b] = 0;
            s_taken[b] = 0;
        }
        *s_stop = 0;
    }
    __syncthreads();
    Item cur = item_at(0), nxt = cur;
    if (tid == 0 && ntiles > 0) {
        issue(0, cur); issue(1, cur); issue(2, cur);
    }

    for (uint32_t tt = (uint32_t)g; tt < ntiles; tt += 2u) {
        const uint32_t t = tt & 7u, j = tt >> 3;
        if (t < 2u) {
            // this group's first tile of a run: coordinates, and the flips of its four tiles (rows gt and
            // gt + 512: one generator call gives the 128 flips of a row segment of the run; the group keeps
            // the 16 of each of its tiles).  The previous run's last reader is behind this group's barriers.
            if (j > 0) cur = nxt;
            if (j + 1u < nitems) nxt = item_at(j + 1u);
            {
                const uint32_t i_run = (cur.hi << (p.lo_log + A)) + cur.lo_run;
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const uint32_t row = (uint32_t)gt + 512u * k;
                    const uint4 w = rng_words(p.rng, p.id0 + (uint32_t)cur.n, 0u, (i_run + row * step) >> 7);
                    const uint32_t sh = 16u * (uint32_t)g;
                    flips[row] = make_uint2(((w.x >> sh) & 0xFFFFu) | (((w.y >> sh) & 0xFFFFu) << 16),
                                            ((w.z >> sh) & 0xFFFFu) | (((w.w >> sh) & 0xFFFFu) << 16));
                }
            }
        }
        const int n = cur.n;
        const uint32_t lo_run = cur.lo_run, hi = cur.hi;
        const uint32_t i_run = (hi << (p.lo_log + A)) + lo_run;
        float* const buf = reinterpret_cast<float*>(smem_raw + (tt % 3u) * LAND_BYTES);
        // Bounded wait for phase k = tt / 3 of the buffer's barrier.  A parity wait only tells two
        // consecutive phases apart, and the two groups share the barriers: phase k - 1 of this barrier
        // belongs to the other group's tile tt - 3, and this group can get here before that tile's copy
        // has even landed (the barrier is then still in phase k - 1, and a wait for parity k & 1 would
        // take the completed phase k - 2 for phase k and let the group loose on a buffer the copy engine
        // is writing).  So the group first waits until this tile's copy has been issued (a counter the
        // issuing thread bumps before it arms the barrier): from then on the barrier is in phase k and
        // the parity wait means what it should.  The group agrees on the outcome, so that it stops as a
        // whole (the barrier also publishes the flips written above).
        const uint32_t k = tt / 3u;
        bool arrived = false;
        for (int it = 0; it < (1 << 22); ++it) {
            if (*(volatile int*)(s_issued + (tt % 3u)) > (int)k) {
                arrived = true;
                break;
            }
        }
        arrived = arrived && mbar_wait(full + (tt % 3u), k & 1u);
        if (!group_all(1 + g, GT, arrived)) {
            if (gt == 0) {
                atomicAdd(timeouts, 1);
                *(volatile int*)s_stop = 1;
            }
            break;
        }
        if (gt == 0) atomicAdd(s_taken + (tt % 3u), 1);
        {
            // the map covers whole rows only: a last partial row of the gradient is patched in
            const uint32_t row_p = full_rows - (hi << A);
            if (row_p < (uint32_t)ROWS) {
                if (gt < 16) {
                    const uint32_t i = full_rows * step + lo_run + 16u * t + (uint32_t)gt;
                    if (i < d32) buf[(row_p << 4) + gt] = (static_cast<const float*>(p.src) + (int64_t)n * p.src_stride)[i];
                }
                group_sync(1 + g, GT);
            }
        }
        float v[32];
        {
            const uint32_t tq = t >> 1;                                   // which of this group's four tiles of the run
            const uint32_t sh = 31u - ((tq & 1u) * 16u + 4u * kq);
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const uint32_t row = ((uint32_t)r << 7) | (u << 1) | r0;
                const float4 q = *reinterpret_cast<const float4*>(buf + (row << 4) + 4u * kq);
                const uint32_t w = reinterpret_cast<const uint32_t*>(flips)[(row << 1) + (tq >> 1)];
                v[4 * r + 0] = flip_at(q.x, w, sh); v[4 * r + 1] = flip_at(q.y, w, sh - 1u);
                v[4 * r + 2] = flip_at(q.z, w, sh - 2u); v[4 * r + 3] = flip_at(q.w, w, sh - 3u);
            }
            butterflies32<28>(v);
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const uint32_t row = ((uint32_t)r << 7) | (u << 1) | r0;
                *reinterpret_cast<float4*>(buf + (row << 4) + 4u * kq) = make_float4(v[4 * r + 0], v[4 * r + 1], v[4 * r + 2], v[4 * r + 3]);
            }
        }
        group_sync(1 + g, GT);
        {
            float* const p2 = buf + ((((u >> 3) << 7) | ((u & 7u) << 1) | r0) << 4) + 4u * kq;
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const float4 q = *reinterpret_cast<const float4*>(p2 + (r << 8));
                v[4 * r + 0] = q.x; v[4 * r + 1] = q.y; v[4 * r + 2] = q.z; v[4 * r + 3] = q.w;
            }
            butterflies32<28>(v);
#pragma unroll
            for (int r = 0; r < 8; ++r)
                *reinterpret_cast<float4*>(p2 + (r << 8)) = make_float4(v[4 * r + 0], v[4 * r + 1], v[4 * r + 2], v[4 * r + 3]);
        }
        group_sync(1 + g, GT);
        {
            const float* const p3 = buf + (((u << 4) | r0) << 4) + 4u * kq;
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const float4 q = *reinterpret_cast<const float4*>(p3 + (r << 5));
                v[4 * r + 0] = q.x; v[4 * r + 1] = q.y; v[4 * r + 2] = q.z; v[4 * r + 3] = q.w;
            }
        }
        fence_generic_before_async();               // this thread's stores into the buffer, before the copy engine reuses it
        group_sync(1 + g, GT);                      // the tile lives in registers: refill its buffer for the tile three ahead
        if (gt == 0 && tt + 3u < ntiles) issue(tt + 3u, ((tt + 3u) >> 3) == j ? cur : nxt);
        butterflies32<28>(v);
        const float sgn = r0 ? -1.f : 1.f;
#pragma unroll
        for (int r = 0; r < 32; ++r) v[r] = fmaf(sgn, v[r], __shfl_xor_sync(0xFFFFFFFFu, v[r], 4));
        float* const o = static_cast<float*>(p.dst) + (int64_t)n * p.dst_stride + i_run + 16u * t + 4u * kq + ((u << 4) | r0) * step;
#pragma unroll
        for (int r = 0; r < 8; ++r)
            __stcg(reinterpret_cast<float4*>(o + (uint32_t)(r << 1) * step), make_float4(v[4 * r + 0], v[4 * r + 1], v[4 * r + 2], v[4 * r + 3]));
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

}  // namespace fosgd
