// Strided pass of ten stages from one packed plane on the tensor cores (tcgen05, sm_100a).
//
// The Sylvester matrix factors as H_1024 = H_8 (x) H_128 (the recursion H_k = H_1 (x) H_{k-1}).  For
// a tile of 1024 rows x 128 columns of +-1 entries (rows = the ten index bits of the pass, 128
// consecutive columns = one 16-byte piece of every packed row):
//   1. H_8 over the top three row bits is done on the plain ALUs, four coordinates per 32-bit
//      operation: the bits b in {0,1} are expanded to bytes and the butterflies run on packed bytes
//      kept non-negative by a bias (a + b, a - b + c), so no carry crosses a byte.
//   2. H_128 over the low seven row bits is a 128 x 128 x 128 integer matrix product per value t'
//      of the top bits: D_t'[j][n] = sum_k H_128[j][k] Z_t'[k][n] with 8-bit operands in shared
//      memory (A = H_128, K-major; B = Z_t', the bytes as the expansion left them: n contiguous,
//      i.e. MN-major) and 32-bit accumulators in tensor memory: tcgen05.mma.kind::i8, four
//      instructions of K = 32 per product, issued by one thread, completion through an mbarrier.
//   3. The accumulators come back with tcgen05.ld (a thread = one output row j of a lane quarter,
//      32 columns per load), become fp16 (all values are even integers of magnitude <= 1024) and
//      go to global memory through a small patch of shared memory per warp, so that a store
//      instruction writes 64 contiguous bytes of eight rows (16 bytes per lane straight from the
//      registers would be 32 separate requests per instruction: measured a third slower).
// Constants: the +-1 entries are q = 2 b - 1 and the H_8 stages add byte biases 1, 2, 4, after which
// every t' != 0 carries bias 4 and t' = 0 carries 0 but owes -8 from the "- 1".  Through the product
// both become the same offset on output row j = 0 alone (the all-ones row of H_128): D = v / 2 + 512
// there and D = v / 2 elsewhere, v the wanted value.  The conversion uses the fp16 bit pattern
// 0x6400 + u = 1024 + u (exact for 0 <= u <= 1024): h = bits(0x6400 + D + 512) = 1536 + v / 2 and
// v = 2 h - 3072 in one packed fused multiply-add; row 0 simply adds 0x6400 instead of 0x6600.
//
// A block is 16 worker warps and one warp that issues the products, persistent over tiles.  Tensor
// memory holds four 128-column accumulators used in turn, so that while the worker warps drain one
// (tcgen05.ld, convert, store through the warp's patch) the products of the next ones run.  The packed rows of the next tile are fetched into registers under the current one.
// Synchronisation is by mbarriers (operands staged / all products of the tile done, accumulator full /
// drained); every wait is bounded.
#include "tc_common.cuh"

namespace fosgd {

static __device__ int g_tc_wait_timeouts;   // blocks that abandoned a bounded wait

namespace {

constexpr int kWorkerWarps = 16;
constexpr int kWorkers = kWorkerWarps * 32;
constexpr int kTcThreads = kWorkers + 32;
constexpr uint32_t kBOperandBytes = 8 * 2064;                 // eight column groups of 16, 2048 B each + 16 B so that they sit on different banks
constexpr uint32_t kOffA = 0;                                 // H_128 as int8, K-major core matrices: 16 KiB
constexpr uint32_t kOffB = 16384;                             // eight B operands
constexpr uint32_t kOffBits = kOffB + 8 * kBOperandBytes;     // the tile's packed rows: 1024 x 16 B
constexpr uint32_t kOffBar = kOffBits + 16384;                // eleven mbarriers, stop word, tensor-memory base address
constexpr uint32_t kPatchPitch = 64;                          // bytes per row of a warp's output patch: 32 fp16; the 16-byte chunks of a row are
                                                              // permuted by (row >> 1) & 3, which keeps both the row-wise writes and the
                                                              // eight-rows-by-64-bytes reads off each other's banks
constexpr uint32_t kOffPatch = kOffBar + 128;                 // one patch of 32 rows per worker warp
constexpr uint32_t kTcSmemBytes = kOffPatch + kWorkerWarps * 32 * kPatchPitch;

enum { BAR_B_FULL = 0, BAR_B_DONE = 1, BAR_ACC_FULL = 2, BAR_ACC_FREE = 6, BAR_BITS = 10 };

// instruction descriptor: D = s32 (2 << 4), A = B = signed 8-bit (1 << 7, 1 << 10), A K-major, B MN-major
// (1 << 16), N = 128 (N / 8 << 17), M = 128 (M / 16 << 24)
constexpr uint32_t kIdescI8 = (2u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (16u << 17) | (8u << 24);

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdescI8), "r"(accumulate) : "memory");
}

}  // namespace

__global__ void __launch_bounds__(kTcThreads, 1) tc_col_kernel(const PassParams p, const int64_t ntiles)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const uint32_t lane = tid & 31;
    uint64_t* const bar = reinterpret_cast<uint64_t*>(smem + kOffBar);
    volatile int* const s_stop = reinterpret_cast<volatile int*>(smem + kOffBar + 96);
    uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffBar + 100);

    // ---- once per block: the constant operand, barriers, tensor memory ----
    if (tid < kWorkers) {
        // A[m][k] = (-1)^popcount(m & k): row m, 32 of its k per thread; core matrix = 8 rows x 16 bytes
        const uint32_t m = (uint32_t)tid >> 2, kc0 = ((uint32_t)tid & 3u) * 2u;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t w[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                w[q] = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const uint32_t k = (kc0 + c) * 16u + 4u * q + b;
                    w[q] |= ((__popc(m & k) & 1) ? 0xFFu : 0x01u) << (8 * b);
                }
            }
            *reinterpret_cast<uint4*>(smem + kOffA + (m & 7u) * 16u + (m >> 3) * 1024u + (kc0 + c) * 128u) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    if (warp == kWorkerWarps) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        mbar_init(bar + BAR_B_FULL, kWorkerWarps);
        mbar_init(bar + BAR_B_DONE, 1);
        mbar_init(bar + BAR_BITS, kWorkerWarps);
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            mbar_init(bar + BAR_ACC_FULL + a, 1);
            mbar_init(bar + BAR_ACC_FREE + a, kWorkerWarps);
        }
        *s_stop = 0;
    }
    fence_generic_before_async();   // the constant operand, for the tensor core's reads
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const uint32_t step = 1u << p.lo_log;
    const int64_t total = ntiles * p.nworkers;
    const int64_t nitems = ((int64_t)blockIdx.x < total) ? (total - (int64_t)blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (warp == kWorkerWarps) {
        // ================= the warp that issues the products =================
        if (lane == 0) {
            const uint64_t adesc = umma_desc(smem_u32(smem + kOffA), 128u, 1024u);
            bool ok = true;
            int64_t issued = 0;   // products committed so far (eight per tile)
            for (int64_t g = 0; g < nitems && ok; ++g) {
                ok = mbar_wait_or_stop(bar + BAR_B_FULL, (uint32_t)g & 1u, s_stop);                 // the tile's eight operands are staged
                for (int t = 0; t < 8 && ok; ++t) {
                    const uint32_t a = (uint32_t)t & 3u, u = (uint32_t)(2 * g) + ((uint32_t)t >> 2);   // accumulator and how often it has been used
                    if (u > 0) ok = mbar_wait_or_stop(bar + BAR_ACC_FREE + a, (u - 1u) & 1u, s_stop);   // drained
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint64_t bdesc = umma_desc(smem_u32(smem + kOffB + (uint32_t)t * kBOperandBytes), 128u, 2064u);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)   // K = 32 per instruction: two core matrices of A, four k-groups of B
                        umma_i8(tmem_base + a * 128u, adesc + (uint64_t)(ks * (256 >> 4)), bdesc + (uint64_t)(ks * (512 >> 4)), ks > 0 ? 1u : 0u);
                    umma_commit(bar + BAR_ACC_FULL + a);
                    ++issued;
                }
                if (ok) umma_commit(bar + BAR_B_DONE);
            }
            if (!ok) {
                if (atomicExch((int*)s_stop, 1) == 0) atomicAdd(&g_tc_wait_timeouts, 1);
                // products already committed may still be running: one more bounded wait each before the tensor memory goes back
                for (int64_t h = (issued >= 4 ? issued - 4 : 0); h < issued; ++h)
                    mbar_wait(bar + BAR_ACC_FULL + (h & 3), (uint32_t)(h >> 2) & 1u);
            }
        }
    } else {
        // ================= worker warps: expand, H_8 on packed bytes, stage; drain and store =================
        const uint32_t cg = (uint32_t)tid & 7u, k1 = (uint32_t)tid >> 3;     // staging role: 16 columns of rows k1 and k1 + 64 (of every t)
        const uint32_t lq = (uint32_t)warp & 3u, cw = (uint32_t)warp >> 2;   // drain role: lane quarter, 32 of an accumulator's 128 columns
        const uint32_t j1 = lq * 32u + lane;                                // output row inside the 128-block
        const uint32_t half_bits = (j1 == 0) ? 0x6400u : 0x6600u;            // fp16 pattern base: 1024 (+ 512 except on the offset row)
        unsigned char* const patch = smem + kOffPatch + (uint32_t)warp * 32u * kPatchPitch;
        bool ok = true;

        auto tile_origin = [&](int64_t item, int& n, uint32_t& i_tile) {
            n = (int)(item / ntiles);
            const uint32_t tile = (uint32_t)(item % ntiles);
            const uint32_t col0 = (tile << 7) & (step - 1u);
            const uint32_t hi = (tile << 7) >> p.lo_log;
            i_tile = (hi << (p.lo_log + 10)) + col0;                        // row 0, column 0 of the tile
        };
        // this thread's two packed rows (tid and tid + 512) of an item: 16 bytes = 128 columns each
        auto load_bits = [&](int64_t item, uint4 (&w)[2]) {
            int n;
            uint32_t i_tile;
            tile_origin(item, n, i_tile);
            const uint32_t* const bits = static_cast<const uint32_t*>(p.src) + (int64_t)n * p.src_stride;
#pragma unroll
            for (int k = 0; k < 2; ++k) w[k] = __ldg(reinterpret_cast<const uint4*>(bits + ((i_tile + ((uint32_t)tid + 512u * k) * step) >> 5)));
        };

        uint4 next_bits[2] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0)};
        if (nitems > 0) load_bits(blockIdx.x, next_bits);
        for (int64_t g = 0; g < nitems && ok; ++g) {
            const int64_t item = (int64_t)blockIdx.x + g * gridDim.x;
            int n;
            uint32_t i_tile;
            tile_origin(item, n, i_tile);
            // ---- the tile's packed rows into shared memory, the next tile's into registers ----
            // (every worker has left the previous tile's rows behind: it passed that tile's first accumulator wait,
            // which follows the arrival of all sixteen warps on the operand barrier)
            reinterpret_cast<uint4*>(smem + kOffBits)[tid] = next_bits[0];
            reinterpret_cast<uint4*>(smem + kOffBits)[tid + 512] = next_bits[1];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar + BAR_BITS);
            if (!mbar_wait_or_stop(bar + BAR_BITS, (uint32_t)g & 1u, s_stop)) { ok = false; break; }   // all sixteen warps' rows are in
            if (g + 1 < nitems) load_bits(item + gridDim.x, next_bits);
            // all eight products of the previous tile have read the operands
            if (g > 0 && !mbar_wait_or_stop(bar + BAR_B_DONE, (uint32_t)(g - 1) & 1u, s_stop)) { ok = false; break; }
            // ---- expand to bytes, H_8 over t on packed bytes, store the eight B operands ----
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                const uint32_t kr = k1 + 64u * (uint32_t)h;
                uint32_t x[8][4];
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    const uint32_t hw = *reinterpret_cast<const uint16_t*>(smem + kOffBits + ((uint32_t)t * 128u + kr) * 16u + cg * 2u);
                    // four bits -> four bytes of {0, 1}: the multiplier puts bit i of the nibble at bit 8 i (its four copies of the
                    // nibble, shifted by 0, 7, 14 and 21, do not overlap, so nothing carries); a table in shared memory cost
                    // more than it saved (random addresses: bank conflicts on a path that is bound by shared-memory traffic)
#pragma unroll
                    for (int q = 0; q < 4; ++q) x[t][q] = (((hw >> (4 * q)) & 15u) * 0x00204081u) & 0x01010101u;
                }
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    const uint32_t bias = 0x01010101u << s;
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        if (!(t & (1 << s))) {
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const uint32_t a = x[t][q], b = x[t | (1 << s)][q];
                                x[t][q] = a + b;
                                x[t | (1 << s)][q] = a - b + bias;
                            }
                        }
                    }
                }
#pragma unroll
                for (int t = 0; t < 8; ++t)
                    *reinterpret_cast<uint4*>(smem + kOffB + (uint32_t)t * kBOperandBytes + cg * 2064u + (kr >> 3) * 128u + (kr & 7u) * 16u) =
                        make_uint4(x[t][0], x[t][1], x[t][2], x[t][3]);
            }
            fence_generic_before_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar + BAR_B_FULL);

            // ---- drain the eight accumulators: fp16 through the warp's patch to global memory ----
            __half* const dst = static_cast<__half*>(p.dst) + (int64_t)n * p.dst_stride + i_tile + cw * 32u;
#pragma unroll 1
            for (int t = 0; t < 8; ++t) {
                const uint32_t a = (uint32_t)t & 3u, u = (uint32_t)(2 * g) + ((uint32_t)t >> 2);
                if (!mbar_wait_or_stop(bar + BAR_ACC_FULL + a, u & 1u, s_stop)) { ok = false; break; }
                tc_fence_after_sync();
                uint32_t v[32];
                tmem_load32(tmem_base + ((lq * 32u) << 16) + a * 128u + cw * 32u, v);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar + BAR_ACC_FREE + a);
                const __half2 two = __floats2half2_rn(2.f, 2.f), off = __floats2half2_rn(-3072.f, -3072.f);
                // through the warp's patch, so that a store instruction writes 64 contiguous bytes of eight rows
                // instead of 16 bytes of thirty-two
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t w[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint32_t hb = __byte_perm(v[8 * q4 + 2 * q] + half_bits, v[8 * q4 + 2 * q + 1] + half_bits, 0x5410);
                        const __half2 hh = __hfma2(*reinterpret_cast<const __half2*>(&hb), two, off);
                        w[q] = *reinterpret_cast<const uint32_t*>(&hh);
                    }
                    *reinterpret_cast<uint4*>(patch + lane * kPatchPitch + (((uint32_t)q4 ^ ((lane >> 1) & 3u)) * 16u)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t r = 8u * i + (lane >> 2), c = lane & 3u;
                    const uint4 q = *reinterpret_cast<const uint4*>(patch + r * kPatchPitch + ((c ^ ((r >> 1) & 3u)) * 16u));
                    __stcg(reinterpret_cast<uint4*>(dst + (size_t)((uint32_t)t * 128u + lq * 32u + r) * step + c * 8u), q);   // L2 only: read next by another kernel
                }
                __syncwarp();
            }
        }
        if (!ok && lane == 0 && atomicExch((int*)s_stop, 1) == 0) atomicAdd(&g_tc_wait_timeouts, 1);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kWorkerWarps) {
        __syncwarp();
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// Rows of at least 128 columns, whole blocks of 1024 rows, and enough tiles to go round: a block sets up its
// constant operand and tensor memory before its first tile, so launches of fewer than 256 tiles (the server's
// own vector of a 2^24 transform, everything at 2^20) are left to the packed-fp16 kernel, which is as fast or
// faster there (0.009 against 0.017 ms on one vector of 2^20).
bool tc_col_applicable(const PassParams& p, bool any_size)
{
    return p.P == 1 && p.lo_log >= 7 && (p.dp >> (p.lo_log + 10)) >= 1 && (any_size || (p.dp >> 17) * p.nworkers >= 256);
}

// Ten strided stages from one packed plane into the fp16 intermediate.
cudaError_t launch_tc_col(const PassParams& p, cudaStream_t s)
{
    if (!tc_col_applicable(p, true)) return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(tc_col_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const int64_t ntiles = p.dp >> 17;                        // 1024 rows x 128 columns each
    int64_t blocks = ntiles * p.nworkers;
    if (blocks > sms) blocks = sms;
    tc_col_kernel<<<(unsigned)blocks, kTcThreads, kTcSmemBytes, s>>>(p, ntiles);
    return cudaGetLastError();
}

cudaError_t tc_timeouts(int* out) { return cudaMemcpyFromSymbol(out, g_tc_wait_timeouts, sizeof(int)); }

}  // namespace fosgd
