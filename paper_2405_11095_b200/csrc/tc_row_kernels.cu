// Contiguous pass of a decoder (14 stages on tiles of 2^14 coordinates, flip, sum over the workers)
// with seven of the stages on the tensor cores (tcgen05, sm_100a).
//
// The source is the fp16 intermediate of the strided pass: integers of magnitude <= 1024.  A tile
// of 2^14 consecutive coordinates is read as a matrix X of 128 rows (index bits 7..13) x 128 columns
// (bits 0..6).  By the recursion H_k = H_1 (x) H_{k-1}, H_{2^14} = H_128 (x) H_4 (x) H_32:
//   1. H_4 over column bits 5, 6 runs in packed fp16 on the plain ALUs while the tile is staged
//      (values <= 4096: still exact in fp16);
//   2. H_128 over the row bits is one 128 x 128 x 128 product D = H_128 Z per tile and worker:
//      fp16 operands in shared memory (A = H_128, K-major; B = Z as staged, columns contiguous, i.e.
//      MN-major), fp32 accumulators in tensor memory (exact: |D| <= 2^19), eight tcgen05.mma of K = 16
//      issued by one thread, completion through mbarriers;
//   3. H_32 over column bits 0..4 runs in fp32 registers: tcgen05.ld hands every thread 32
//      consecutive columns of one row, which is also one word of the flip vector, so the flip and
//      the sum over the workers follow in the same registers.
// All values are integers below 2^24 in magnitude, so the result equals the plain-ALU kernel's bit
// for bit.
//
// A block is 16 worker warps, one warp that issues the products and one service warp.  It keeps a tile
// position and walks the workers (sums in registers), then moves to its next tile.  The service warp
// keeps whole tiles (32 KiB, contiguous) arriving through the bulk copy engine into a ring of three
// landing slots and makes the flip words of the items.  Per item (tile, worker) a worker warp turns its
// share of a landed tile into the operand layout in one of two operand buffers, then drains the
// accumulator of the previous item while the product of this one runs.  Synchronisation is by
// mbarriers only (slot landed / read, operand full / free, accumulator full / free, flips ready);
// every wait is bounded.
#include "tc_common.cuh"

namespace fosgd {

static __device__ int g_tcrow_wait_timeouts;   // warps that abandoned a bounded wait

namespace {

constexpr int kT = 14;
constexpr int kWorkerWarps = 16;
constexpr int kIssueWarp = kWorkerWarps, kServiceWarp = kWorkerWarps + 1;
constexpr int kThreads = (kWorkerWarps + 2) * 32;
constexpr int kRing = 3;                                   // landing slots for whole tiles (bulk copies in flight)
constexpr uint32_t kTileBytes = 2u << kT;                  // one fp16 tile
constexpr uint32_t kAChunkStride = 128;                    // bytes between core matrices along K
constexpr uint32_t kAGroupStride = 16 * 128;               // bytes between groups of eight rows of A
constexpr uint32_t kBGroupStride = 16 * 128 + 32;          // bytes between groups of eight columns of B (+32: staging stores hit distinct banks)
constexpr uint32_t kOffA = 0;                              // H_128 as fp16: 32 KiB
constexpr uint32_t kOffB = 32768;                          // two operand buffers
constexpr uint32_t kBBytes = 16 * kBGroupStride;
constexpr uint32_t kOffFlips = kOffB + 2 * kBBytes;        // two buffers of 128 rows x 4 flip words
constexpr uint32_t kOffLand = kOffFlips + 2 * 2048;        // kRing landing slots
constexpr uint32_t kOffBar = kOffLand + kRing * kTileBytes;   // mbarriers, stop word, tensor-memory base
constexpr int kNumBars = 10 + 2 * kRing;
constexpr uint32_t kSmemBytes = kOffBar + kNumBars * 8 + 16;

enum { BAR_B_FULL = 0, BAR_B_FREE = 2, BAR_ACC_FULL = 4, BAR_ACC_FREE = 6, BAR_FLIPS = 8, BAR_LAND_FULL = 10, BAR_LAND_FREE = 10 + kRing };

// instruction descriptor: D = f32 (1 << 4), A = B = fp16 (0), A K-major, B MN-major (1 << 16), N = 128, M = 128
constexpr uint32_t kIdescF16 = (1u << 4) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdescF16), "r"(accumulate) : "memory");
}

// x with its sign flipped iff the top bit of w is set
__device__ __forceinline__ float flip_top(float x, uint32_t w)
{
    return __uint_as_float(__float_as_uint(x) ^ (w & 0x80000000u));
}

__device__ __forceinline__ void hbutterfly(uint4& a, uint4& b)
{
    __half2* const pa = reinterpret_cast<__half2*>(&a);
    __half2* const pb = reinterpret_cast<__half2*>(&b);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const __half2 x = pa[k], y = pb[k];
        pa[k] = __hadd2(x, y);
        pb[k] = __hsub2(x, y);
    }
}

}  // namespace

__global__ void __launch_bounds__(kThreads, 1) tc_row_final_kernel(const PassParams p, const int ntiles)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const uint32_t lane = tid & 31;
    uint64_t* const bar = reinterpret_cast<uint64_t*>(smem + kOffBar);
    volatile int* const s_stop = reinterpret_cast<volatile int*>(smem + kOffBar + kNumBars * 8);
    uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffBar + kNumBars * 8 + 4);

    // ---- once per block: the constant operand, barriers, tensor memory ----
    if (tid < 512) {
        // A[m][k] = (-1)^popcount(m & k) as fp16, K-major core matrices of 8 rows x 16 bytes: thread = (row m, 32 of its k)
        const uint32_t m = (uint32_t)tid >> 2, k0 = ((uint32_t)tid & 3u) * 32u;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t w[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t k = k0 + 8u * c + 2u * q;
                const uint32_t lo = (__popc(m & k) & 1) ? 0xBC00u : 0x3C00u;
                const uint32_t hi = (__popc(m & (k + 1u)) & 1) ? 0xBC00u : 0x3C00u;
                w[q] = lo | (hi << 16);
            }
            *reinterpret_cast<uint4*>(smem + kOffA + (m & 7u) * 16u + (m >> 3) * kAGroupStride + ((k0 >> 3) + c) * kAChunkStride) =
                make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    if (warp == kIssueWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
#pragma unroll
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar + BAR_B_FULL + b, kWorkerWarps);
            mbar_init(bar + BAR_B_FREE + b, 1);
            mbar_init(bar + BAR_ACC_FULL + b, 1);
            mbar_init(bar + BAR_ACC_FREE + b, kWorkerWarps);
            mbar_init(bar + BAR_FLIPS + b, 1);
        }
#pragma unroll
        for (int r = 0; r < kRing; ++r) {
            mbar_init(bar + BAR_LAND_FULL + r, 1);
            mbar_init(bar + BAR_LAND_FREE + r, kWorkerWarps);
        }
        *s_stop = 0;
    }
    fence_generic_before_async();   // the constant operand, for the tensor core's reads
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const int W = p.nworkers;
    const int my_tiles = ((int)blockIdx.x < ntiles) ? (ntiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int64_t nitems = (int64_t)my_tiles * W;   // item g: this block's tile number g / W, worker g % W

    // where an item sits: first coordinate of its tile and its worker; advanced item by item (worker fastest)
    struct Cursor {
        int64_t tile_base;
        int n;
    };
    const int64_t tile_step = (int64_t)gridDim.x << kT;
    auto advance = [&](Cursor& c) {
        if (++c.n == W) {
            c.n = 0;
            c.tile_base += tile_step;
        }
    };
    const Cursor c_first{(int64_t)blockIdx.x << kT, 0};

    if (warp == kIssueWarp) {
        // ================= the warp that issues the products =================
        if (lane == 0) {
            const uint64_t adesc = umma_desc(smem_u32(smem + kOffA), kAChunkStride, kAGroupStride);
            bool ok = true;
            int64_t g = 0;
            for (; g < nitems; ++g) {
                const uint32_t b = (uint32_t)g & 1u, u = (uint32_t)(g >> 1);
                ok = mbar_wait_or_stop(bar + BAR_B_FULL + b, u & 1u, s_stop);                        // operand staged
                if (ok && u > 0) ok = mbar_wait_or_stop(bar + BAR_ACC_FREE + b, (u - 1u) & 1u, s_stop);   // accumulator drained
                if (!ok) break;
                tc_fence_after_sync();
                const uint64_t bdesc = umma_desc(smem_u32(smem + kOffB + b * kBBytes), 128u, kBGroupStride);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)   // K = 16 per instruction: two 16-byte chunks of A, two groups of eight rows of B
                    umma_f16(tmem_base + b * 128u, adesc + (uint64_t)(ks * (256 >> 4)), bdesc + (uint64_t)(ks * (256 >> 4)), ks > 0 ? 1u : 0u);
                umma_commit(bar + BAR_B_FREE + b);
                umma_commit(bar + BAR_ACC_FULL + b);
            }
            if (!ok) {
                if (atomicExch((int*)s_stop, 1) == 0) atomicAdd(&g_tcrow_wait_timeouts, 1);
                // products already committed may still be running: one more bounded wait each before the tensor memory goes back
                for (int64_t h = (g >= 2 ? g - 2 : 0); h < g; ++h) mbar_wait(bar + BAR_ACC_FULL + (h & 1), (uint32_t)(h >> 1) & 1u);
            }
        }
    } else if (warp == kServiceWarp) {
        // ================= the service warp: tiles in through the copy engine, flip words =================
        // Lane 0 keeps kRing bulk copies of whole tiles (32 KiB, contiguous) in flight; all lanes make the
        // flip words of the items (four generator calls per lane: 128 rows x 128 flips).
        Cursor c_ld = c_first, c_fl = c_first;
        bool ok = true;
        int64_t issued = 0;   // lane 0: copies started
        auto issue_load = [&](int64_t g) -> bool {
            const uint32_t r = (uint32_t)(g % kRing), u = (uint32_t)(g / kRing);
            if (u > 0 && !mbar_wait_or_stop(bar + BAR_LAND_FREE + r, (u - 1u) & 1u, s_stop)) return false;   // every warp has read the slot
            const __half* const src = static_cast<const __half*>(p.src) + (int64_t)c_ld.n * p.src_stride + c_ld.tile_base;
            advance(c_ld);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar + BAR_LAND_FULL + r)), "r"(kTileBytes) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(smem + kOffLand + r * kTileBytes)), "l"(src), "r"(kTileBytes), "r"(smem_u32(bar + BAR_LAND_FULL + r)) : "memory");
            ++issued;
            return true;
        };
        if (lane == 0) {
            for (int64_t g = 0; g < kRing - 1 && g < nitems && ok; ++g) ok = issue_load(g);
        }
        for (int64_t g = 0; g < nitems; ++g) {
            if (lane == 0 && ok && g + kRing - 1 < nitems) ok = issue_load(g + kRing - 1);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            const uint32_t b = (uint32_t)g & 1u, u = (uint32_t)(g >> 1);
            // the drain of item g - 2 has read its flip words (every warp reads them before it frees the accumulator)
            if (u > 0 && !mbar_wait_or_stop(bar + BAR_ACC_FREE + b, (u - 1u) & 1u, s_stop)) { ok = false; }
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            const uint32_t id = p.id0 + (uint32_t)c_fl.n, c0 = (uint32_t)(c_fl.tile_base >> 7);
            advance(c_fl);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t row = lane + 32u * k;
                reinterpret_cast<uint4*>(smem + kOffFlips + b * 2048u)[row] = rng_words(p.rng, id, 0u, c0 + row);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar + BAR_FLIPS + b);
        }
        if (!ok && lane == 0) {
            if (atomicExch((int*)s_stop, 1) == 0) atomicAdd(&g_tcrow_wait_timeouts, 1);
        }
        // copies started but possibly not landed yet: one more bounded wait each, so that the engine is not
        // left writing into shared memory that the next block of this SM may own
        if (lane == 0) {
            for (int64_t h = (issued >= kRing ? issued - kRing : 0); h < issued; ++h)
                mbar_wait(bar + BAR_LAND_FULL + (h % kRing), (uint32_t)(h / kRing) & 1u);
        }
    } else {
        // ================= worker warps: stage, drain, flip, sum =================
        const uint32_t srow = (uint32_t)tid >> 2, sq = (uint32_t)tid & 3u;       // staging role: row of the tile, column chunks sq + 4 t
        const uint32_t lq = (uint32_t)warp & 3u, cw = (uint32_t)warp >> 2;       // drain role: lane quarter, 32 of the 128 columns
        const uint32_t jrow = lq * 32u + lane;                                  // output row (index bits 7..13)
        float accv[32];
        bool ok = true;
        Cursor c_drain = c_first;

        // stage item g: landed tile -> H_4 over column bits 5, 6 -> operand buffer
        auto stage_item = [&](int64_t g) -> bool {
            const uint32_t b = (uint32_t)g & 1u, u = (uint32_t)(g >> 1);
            const uint32_t r = (uint32_t)(g % kRing), ur = (uint32_t)(g / kRing);
            if (!mbar_wait_or_stop(bar + BAR_LAND_FULL + r, ur & 1u, s_stop)) return false;               // the tile has landed
            uint4 pre[4];
            const unsigned char* const land = smem + kOffLand + r * kTileBytes + srow * 256u + sq * 16u;
#pragma unroll
            for (int t = 0; t < 4; ++t) pre[t] = *reinterpret_cast<const uint4*>(land + 64 * t);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar + BAR_LAND_FREE + r);
            hbutterfly(pre[0], pre[1]);   // column bit 5
            hbutterfly(pre[2], pre[3]);
            hbutterfly(pre[0], pre[2]);   // column bit 6
            hbutterfly(pre[1], pre[3]);
            if (u > 0 && !mbar_wait_or_stop(bar + BAR_B_FREE + b, (u - 1u) & 1u, s_stop)) return false;   // product g - 2 has read the buffer
            unsigned char* const dst = smem + kOffB + b * kBBytes + sq * kBGroupStride + (srow >> 3) * 128u + (srow & 7u) * 16u;
#pragma unroll
            for (int t = 0; t < 4; ++t) *reinterpret_cast<uint4*>(dst + 4 * t * kBGroupStride) = pre[t];
            fence_generic_before_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar + BAR_B_FULL + b);
            return true;
        };
        // drain item g: accumulator -> registers, H_32 over the 32 columns, flip, add
        auto drain_item = [&](int64_t g) -> bool {
            const uint32_t b = (uint32_t)g & 1u, u = (uint32_t)(g >> 1);
            const int n = c_drain.n;
            const int64_t tile_base = c_drain.tile_base;
            advance(c_drain);
            if (!mbar_wait_or_stop(bar + BAR_ACC_FULL + b, u & 1u, s_stop)) return false;
            tc_fence_after_sync();
            if (!mbar_wait_or_stop(bar + BAR_FLIPS + b, u & 1u, s_stop)) return false;
            const uint32_t fw = reinterpret_cast<const uint32_t*>(smem + kOffFlips + b * 2048u)[jrow * 4u + cw];
            const float wamp = (p.amp_mode == AMP_WEIGHT) ? amplitude_at(p, n, tile_base) : 1.f;
            uint32_t raw[32];
            tmem_load32(tmem_base + ((lq * 32u) << 16) + b * 128u + cw * 32u, raw);
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar + BAR_ACC_FREE + b);
            float v[32];
#pragma unroll
            for (int r = 0; r < 32; ++r) v[r] = __uint_as_float(raw[r]);
            butterflies32<31>(v);
            if (p.amp_mode == AMP_WEIGHT) {
#pragma unroll
                for (int r = 0; r < 32; ++r) accv[r] = fmaf(flip_top(v[r], fw << (31 - r)), wamp, accv[r]);
            } else {
#pragma unroll
                for (int r = 0; r < 32; ++r) accv[r] += flip_top(v[r], fw << (31 - r));
            }
            if (n == W - 1) {
                // the tile's sum is complete: scale and store 32 consecutive coordinates
                const int64_t i0 = tile_base + jrow * 128u + cw * 32u;
                const float sc = p.scale * (p.amp_mode == AMP_SCALE ? amplitude_at(p, 0, tile_base) : 1.f);
                float* const dst = static_cast<float*>(p.dst) + i0;
                if (i0 + 32 <= p.d_out) {
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        float4 o = make_float4(accv[4 * q], accv[4 * q + 1], accv[4 * q + 2], accv[4 * q + 3]);
                        float4* const d4 = reinterpret_cast<float4*>(dst) + q;
                        if (p.overwrite == 2) {
                            const float4 c = *d4;
                            o = make_float4(fmaf(o.x, sc, c.x), fmaf(o.y, sc, c.y), fmaf(o.z, sc, c.z), fmaf(o.w, sc, c.w));
                        } else {
                            if (!p.overwrite) {
                                const float4 c = *d4;
                                o.x += c.x; o.y += c.y; o.z += c.z; o.w += c.w;
                            }
                            o.x *= sc; o.y *= sc; o.z *= sc; o.w *= sc;
                        }
                        *d4 = o;
                    }
                } else {
#pragma unroll
                    for (int r = 0; r < 32; ++r) {
                        if (i0 + r < p.d_out) {
                            float o = accv[r];
                            if (p.overwrite == 2) {
                                dst[r] = fmaf(o, sc, dst[r]);
                            } else {
                                if (!p.overwrite) o += dst[r];
                                dst[r] = o * sc;
                            }
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < 32; ++r) accv[r] = 0.f;
            }
            return true;
        };

#pragma unroll
        for (int r = 0; r < 32; ++r) accv[r] = 0.f;
        for (int64_t g = 0; g < nitems && ok; ++g) {
            ok = stage_item(g);
            if (!ok) break;
            if (g > 0) ok = drain_item(g - 1);        // underneath the product of item g
        }
        if (ok && nitems > 0) ok = drain_item(nitems - 1);
        if (!ok && lane == 0 && atomicExch((int*)s_stop, 1) == 0) atomicAdd(&g_tcrow_wait_timeouts, 1);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kIssueWarp) {
        __syncwarp();
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
    }
}

// One packed plane's fp16 intermediate in contiguous tiles of 2^14, and at least three workers to sum: with one or
// two (a single decoder, the downlink) the plain-ALU pass is the faster one (0.033 against 0.041 ms on one vector
// of 2^24, 0.051 against 0.057 on two; 0.069 against 0.068 on three, 0.156 against 0.119 on eight).
bool tc_row_applicable(const PassParams& p, int T, bool any_size)
{
    return T == kT && p.P == 1 && (any_size || p.nworkers >= 3) && (p.dp >> kT) >= 1 && (p.dp >> kT) <= 0x7FFFFFFF;
}

cudaError_t launch_tc_row(const PassParams& p, cudaStream_t s)
{
    cudaError_t e = cudaFuncSetAttribute(tc_row_final_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const int64_t ntiles = p.dp >> kT;
    const int64_t blocks = ntiles < sms ? ntiles : sms;
    tc_row_final_kernel<<<(unsigned)blocks, kThreads, kSmemBytes, s>>>(p, (int)ntiles);
    return cudaGetLastError();
}

cudaError_t tcrow_timeouts(int* out) { return cudaMemcpyFromSymbol(out, g_tcrow_wait_timeouts, sizeof(int)); }

}  // namespace fosgd
