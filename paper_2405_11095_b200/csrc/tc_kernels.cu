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
//      go to global memory through a padded staging tile, so that every store instruction of a
//      warp writes two whole 256-byte rows.
// Constants: the +-1 entries are q = 2 b - 1 and the H_8 stages add byte biases 1, 2, 4, after which
// every t' != 0 carries bias 4 and t' = 0 carries 0 but owes -8 from the "- 1".  Through the product
// both become the same offset on output row j = 0 alone (the all-ones row of H_128): D = v / 2 + 512
// there and D = v / 2 elsewhere, v the wanted value.  The conversion uses the fp16 bit pattern
// 0x6400 + u = 1024 + u (exact for 0 <= u <= 1024): h = bits(0x6400 + D + 512) = 1536 + v / 2 and
// v = 2 h - 3072 in one packed fused multiply-add; row 0 simply adds 0x6400 instead of 0x6600.
//
// Tensor memory: 512 columns = four 128-column accumulators, used as two pairs in turn: while the
// threads drain one pair the products of the next pair run.  A block (1024 threads, one per SM,
// persistent over tiles) prefetches the packed rows of its next tile under the epilogue; every
// wait is bounded.
#include "common.cuh"

namespace fosgd {

static __device__ int g_tc_wait_timeouts;   // blocks that abandoned a bounded wait

namespace {

constexpr int kTcThreads = 1024;
constexpr uint32_t kBOperandBytes = 8 * 2064;                 // eight column groups of 16, 2048 B each + 16 B so that they sit on different banks
constexpr uint32_t kOffA = 0;                                 // H_128 as int8, K-major core matrices: 16 KiB
constexpr uint32_t kOffB = 16384;                             // eight B operands
constexpr uint32_t kOffBits = kOffB + 8 * kBOperandBytes;     // the tile's packed rows: 1024 x 16 B
constexpr uint32_t kOffLut = kOffBits + 16384;                // byte -> eight bytes of {0, 1}: 2 KiB
constexpr uint32_t kOffBar = kOffLut + 2048;                  // two mbarriers, tensor-memory base address
constexpr uint32_t kStagePitch = 272;                         // bytes per staged row: 128 fp16 + 16 (rows land on different banks)
constexpr uint32_t kOffStage = kOffBar + 32;                  // one accumulator as fp16: 128 rows
constexpr uint32_t kTcSmemBytes = kOffStage + 128 * kStagePitch;

// shared-memory matrix descriptor, no swizzle: start address, leading and stride byte offsets in
// units of 16 bytes, descriptor version 1
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(sbo_bytes >> 4) << 32) | ((uint64_t)1 << 46);
}

// instruction descriptor: D = s32 (2 << 4), A = B = signed 8-bit (1 << 7, 1 << 10), A K-major, B MN-major
// (1 << 16), N = 128 (N / 8 << 17), M = 128 (M / 16 << 24)
constexpr uint32_t kIdescI8 = (2u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (16u << 17) | (8u << 24);

__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdescI8), "r"(accumulate) : "memory");
}

// 16 consecutive accumulator columns of this thread's lane
__device__ __forceinline__ void tmem_load16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

}  // namespace

__global__ void __launch_bounds__(kTcThreads, 1) tc_col_kernel(const PassParams p, const int64_t ntiles)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const uint32_t lane = tid & 31;
    uint64_t* const bar = reinterpret_cast<uint64_t*>(smem + kOffBar);
    uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffBar + 16);
    const uint2* const lut = reinterpret_cast<const uint2*>(smem + kOffLut);

    // ---- once per block: expansion table, the constant operand, barrier, tensor memory ----
    if (tid < 256) {
        uint32_t lo = 0, hi = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            lo |= (((uint32_t)tid >> j) & 1u) << (8 * j);
            hi |= (((uint32_t)tid >> (4 + j)) & 1u) << (8 * j);
        }
        reinterpret_cast<uint2*>(smem + kOffLut)[tid] = make_uint2(lo, hi);
    }
    {
        // A[m][k] = (-1)^popcount(m & k): row m, sixteen k per thread; core matrix = 8 rows x 16 bytes
        const uint32_t m = (uint32_t)tid >> 3, kc = (uint32_t)tid & 7u;
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            w[q] = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const uint32_t k = kc * 16u + 4u * q + b;
                w[q] |= ((__popc(m & k) & 1) ? 0xFFu : 0x01u) << (8 * b);
            }
        }
        *reinterpret_cast<uint4*>(smem + kOffA + (m & 7u) * 16u + (m >> 3) * 1024u + kc * 128u) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        mbar_init(bar + 0, 1);
        mbar_init(bar + 1, 1);
    }
    fence_generic_before_async();   // the constant operand, for the tensor core's reads
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const uint32_t step = 1u << p.lo_log;
    const int64_t total = ntiles * p.nworkers;
    const uint32_t cg = (uint32_t)tid & 7u, k1 = (uint32_t)tid >> 3;   // producer role: 16 columns of row k1 (of every t)
    const uint32_t lq = (uint32_t)warp & 3u, cw = (uint32_t)warp >> 2; // epilogue role: lane quarter, 16 of an accumulator's 128 columns
    const uint32_t j1 = lq * 32u + lane;                              // output row inside the 128-block
    const uint32_t half_bits = (j1 == 0) ? 0x6400u : 0x6600u;          // fp16 pattern base: 1024 (+ 512 except on the offset row)
    uint32_t commits[2] = {0, 0};
    bool failed = false;

    auto tile_origin = [&](int64_t item, int& n, uint32_t& i_tile) {
        n = (int)(item / ntiles);
        const uint32_t tile = (uint32_t)(item % ntiles);
        const uint32_t col0 = (tile << 7) & (step - 1u);
        const uint32_t hi = (tile << 7) >> p.lo_log;
        i_tile = (hi << (p.lo_log + 10)) + col0;                      // row 0, column 0 of the tile
    };
    auto load_bits = [&](int64_t item) -> uint4 {
        int n;
        uint32_t i_tile;
        tile_origin(item, n, i_tile);
        const uint32_t* const bits = static_cast<const uint32_t*>(p.src) + (int64_t)n * p.src_stride;
        return __ldg(reinterpret_cast<const uint4*>(bits + ((i_tile + (uint32_t)tid * step) >> 5)));
    };
    // four products (two accumulators) of pair `pr` (t' = 2 pr, 2 pr + 1) into columns (pr & 1) * 256 ...
    auto issue_pair = [&](int pr) {
        tc_fence_after_sync();
        const uint64_t adesc = umma_desc(smem_u32(smem + kOffA), 128u, 1024u);
#pragma unroll
        for (int a = 0; a < 2; ++a) {
            const uint64_t bdesc = umma_desc(smem_u32(smem + kOffB + (uint32_t)(2 * pr + a) * kBOperandBytes), 128u, 2064u);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)   // K = 32 per instruction: two core matrices of A, four k-groups of B
                umma_i8(tmem_base + (uint32_t)(pr & 1) * 256u + (uint32_t)a * 128u, adesc + (uint64_t)(ks * (256 >> 4)),
                        bdesc + (uint64_t)(ks * (512 >> 4)), ks > 0 ? 1u : 0u);
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar + (pr & 1))) : "memory");
    };

    uint4 next_bits = make_uint4(0, 0, 0, 0);
    if ((int64_t)blockIdx.x < total) next_bits = load_bits(blockIdx.x);
    for (int64_t item = blockIdx.x; item < total; item += gridDim.x) {
        int n;
        uint32_t i_tile;
        tile_origin(item, n, i_tile);
        // ---- the tile's packed rows into shared memory (16 bytes per row), the next tile's into registers ----
        reinterpret_cast<uint4*>(smem + kOffBits)[tid] = next_bits;
        __syncthreads();
        if (item + gridDim.x < total) next_bits = load_bits(item + gridDim.x);
        // ---- expand to bytes, H_8 over t on packed bytes, store the eight B operands ----
        {
            uint32_t x[8][4];
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const uint32_t h = *reinterpret_cast<const uint16_t*>(smem + kOffBits + ((uint32_t)t * 128u + k1) * 16u + cg * 2u);
                const uint2 a = lut[h & 0xFFu], b = lut[h >> 8];
                x[t][0] = a.x; x[t][1] = a.y; x[t][2] = b.x; x[t][3] = b.y;
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
                *reinterpret_cast<uint4*>(smem + kOffB + (uint32_t)t * kBOperandBytes + cg * 2064u + (k1 >> 3) * 128u + (k1 & 7u) * 16u) =
                    make_uint4(x[t][0], x[t][1], x[t][2], x[t][3]);
        }
        fence_generic_before_async();
        tc_fence_before_sync();
        __syncthreads();
        if (tid == 0) {
            issue_pair(0);
            issue_pair(1);
        }

        __half* const dst = static_cast<__half*>(p.dst) + (int64_t)n * p.dst_stride;
#pragma unroll 1
        for (int pr = 0; pr < 4; ++pr) {
            // bounded wait for the pair's products; the block agrees on the outcome
            if (!__syncthreads_and(mbar_wait(bar + (pr & 1), commits[pr & 1] & 1u) ? 1 : 0)) {
                failed = true;
                break;
            }
            ++commits[pr & 1];
            tc_fence_after_sync();
#pragma unroll 1
            for (int a = 0; a < 2; ++a) {
                // ---- accumulator -> fp16 -> staging tile (row j1, 16 of its 128 columns per warp) ----
                uint32_t v[16];
                tmem_load16(tmem_base + ((lq * 32u) << 16) + (uint32_t)(pr & 1) * 256u + (uint32_t)a * 128u + cw * 16u, v);
                const __half2 two = __floats2half2_rn(2.f, 2.f), off = __floats2half2_rn(-3072.f, -3072.f);
                unsigned char* const srow = smem + kOffStage + j1 * kStagePitch + cw * 32u;
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    uint32_t w[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint32_t hb = __byte_perm(v[8 * g + 2 * q] + half_bits, v[8 * g + 2 * q + 1] + half_bits, 0x5410);
                        const __half2 h = __hfma2(*reinterpret_cast<const __half2*>(&hb), two, off);
                        w[q] = *reinterpret_cast<const uint32_t*>(&h);
                    }
                    *reinterpret_cast<uint4*>(srow + g * 16) = make_uint4(w[0], w[1], w[2], w[3]);
                }
                __syncthreads();
                // ---- staging tile -> global memory: a warp instruction writes two whole rows ----
                {
                    const uint32_t tq = (uint32_t)(2 * pr + a);                       // t' of this accumulator
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const uint32_t r = (uint32_t)warp * 4u + 2u * k + (lane >> 4);       // 32 warps x 4 rows
                        const uint4 q = *reinterpret_cast<const uint4*>(smem + kOffStage + r * kStagePitch + (lane & 15u) * 16u);
                        __stcg(reinterpret_cast<uint4*>(dst + i_tile + (tq * 128u + r) * step + (lane & 15u) * 8u), q);   // L2 only: read next by another kernel
                    }
                }
                if (a == 0) __syncthreads();   // the staging tile is free again
            }
            tc_fence_before_sync();
            __syncthreads();   // this pair of accumulators (and the staging tile) may be reused
            if (tid == 0 && pr + 2 < 4) issue_pair(pr + 2);
        }
        if (failed) break;
    }
    if (failed) {
        // products may still be running: one more bounded wait on both barriers before the tensor memory goes back
        if (tid == 0) {
            atomicAdd(&g_tc_wait_timeouts, 1);
            mbar_wait(bar + 0, commits[0] & 1u);
            mbar_wait(bar + 1, commits[1] & 1u);
        }
        __syncthreads();
    }
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

// rows of at least 128 columns, whole blocks of 1024 rows
bool tc_col_applicable(const PassParams& p) { return p.P == 1 && p.lo_log >= 7 && (p.dp >> (p.lo_log + 10)) >= 1; }

// Ten strided stages from one packed plane into the fp16 intermediate.
cudaError_t launch_tc_col(const PassParams& p, cudaStream_t s)
{
    if (!tc_col_applicable(p)) return cudaErrorInvalidValue;
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
