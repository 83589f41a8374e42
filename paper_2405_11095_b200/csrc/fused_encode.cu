// Uplink encoder of a 2^24-long transform (ten strided stages, then a contiguous tile of 2^14) as ONE
// persistent kernel.  Run one after the other, the strided pass is bound by memory traffic (gradients
// in, fp32 intermediate out) and the contiguous pass by instruction issue (butterflies, the dither
// generator, packing); here both run side by side on every SM, so that the memory system and the issue
// slots are busy together.
//
// A block has 1024 threads in two groups of 512, each with its own shared memory and named barrier:
//   group 0  takes runs of the strided pass (col4_run: eight 16-column tiles of one worker through the
//            tensor copy engine) from a ticket counter, worker by worker; when the runs are used up it
//            joins group 1's work;
//   group 1  takes contiguous tiles (worker, tile) from a second ticket counter, in the same worker
//            order, and before it touches a worker's intermediate waits until every run of that worker
//            has been stored (a counter per worker, bumped by the strided side after a fence).
// Work is handed out by tickets, not by block index, so a block that is not resident yet holds no work
// another block could be waiting for: the strided side never waits for anyone, hence every wait of the
// contiguous side ends.  Waits are bounded all the same; a group whose wait runs out raises the stop
// word, after which no group takes another ticket, and the call reports through the timeout counter.
//
// Synchronisation words (caller-zeroed device memory): [0] strided tickets, [1] contiguous tickets,
// [2] stop, [3] unused, [4 + n] finished strided runs of worker n.
#include <cuda.h>

#include "col4.cuh"
#include "row_kernels.cuh"

namespace fosgd {

static __device__ int g_fused_wait_timeouts;   // groups that abandoned a bounded wait

namespace {

constexpr int kT = 14;                                        // contiguous tile: 2^14 coordinates, 512 threads
constexpr int kGroup = 512;
constexpr size_t kRegionA = (Col4::SMEM_BYTES + 1023) & ~(size_t)1023;   // group 0: landing buffers + flips (or a contiguous tile)
constexpr size_t kRegionB = RowCfg<kT>::SMEM_BYTES;                      // group 1: one padded contiguous tile
constexpr size_t kFusedSmem = kRegionA + kRegionB;
static_assert(RowCfg<kT>::NT == kGroup, "one group per contiguous tile");
static_assert(kRegionB <= kRegionA, "group 0 reuses its region for contiguous tiles");

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Contiguous tiles until the tickets run out.  G = group index (named barrier 1 + G).
template <int G>
__device__ __forceinline__ void row_role(const PassParamsRK& p, uint32_t* const sync, float* const smem, const int gt,
                                         volatile uint32_t* const s_ticket, const uint32_t nruns)
{
    using C = RowCfg<kT>;
    using S = GroupSync<1 + G, kGroup>;
    const uint32_t lane = gt & 31;
    const int baseF = deposit<C::FMASK, kT>(gt);
    const int baseM = deposit<C::MMASK, kT>(gt);
    const int baseL = deposit<C::LMASK, kT>(gt);
    const uint32_t ntiles = (uint32_t)(p.dp >> kT);
    const uint32_t total = ntiles * (uint32_t)p.nworkers;

    // Thread 0 of the group draws the tickets, one tile ahead (the atomic's round trip hides under the tile in
    // progress), and remembers the last worker it has seen complete, so that most tiles start without a look
    // at that worker's counter.
    uint32_t q_next = 0xFFFFFFFFu;
    int n_ready = -1;
    if (gt == 0) q_next = atomicAdd(sync + 1, 1u);
    for (;;) {
        if (gt == 0) {
            uint32_t q = q_next;
            if (q < total) {
                q_next = atomicAdd(sync + 1, 1u);
                const int n = (int)(q / ntiles);
                if (n != n_ready) {
                    // every strided run of this worker stored?  (bounded; the stop word ends the wait early)
                    const uint32_t* const done = sync + 4 + n;
                    bool ready = false;
                    for (int it = 0; it < (1 << 22); ++it) {
                        if (ld_acquire(done) >= nruns) { ready = true; break; }
                        if ((it & 63) == 63 && ld_acquire(sync + 2) != 0u) break;
                        __nanosleep(64);
                    }
                    if (ready) {
                        n_ready = n;
                    } else {
                        if (atomicExch(sync + 2, 1u) == 0u) atomicAdd(&g_fused_wait_timeouts, 1);
                        q = 0xFFFFFFFFu;
                    }
                }
            }
            *s_ticket = q;
        }
        S::sync();   // publishes the ticket; also: the previous tile's last shared-memory reads are over
        const uint32_t q = *s_ticket;
        if (q >= total) break;
        const int n = (int)(q / ntiles);
        const int64_t tile_base = (int64_t)(q - (uint32_t)n * ntiles) << kT;
        const uint32_t id = p.id0 + (uint32_t)n;
        const float amp = amplitude_at(p, n, tile_base);

        float v[32];
        const float* const src = static_cast<const float*>(p.src) + (int64_t)n * p.src_stride + tile_base;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const float4 x = __ldcg(reinterpret_cast<const float4*>(src + (baseF | (g << (kT - 3)))));   // written by other SMs: L2
            v[4 * g + 0] = x.x; v[4 * g + 1] = x.y; v[4 * g + 2] = x.z; v[4 * g + 3] = x.w;
        }
        butterflies32<31>(v);
        store_round_F<kT>(smem, baseF, v);
        S::sync();
        round_M<kT>(smem, baseM, v);
        S::sync();
        load_round_L(smem, baseL, v);
        butterflies32<C::ACT_L>(v);
        sink_pack1(p, n, id, tile_base + baseL, lane, v, amp);
    }
}

__global__ void __launch_bounds__(2 * kGroup, 1)
enc_fused_kernel(const PassParams pc, const PassParamsRK pr, const __grid_constant__ CUtensorMap tmap, const uint32_t nruns,
                 const uint32_t full_rows, uint32_t* const sync)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ uint32_t s_ticket[3];   // strided runs of group 0, contiguous tiles of group 1, of group 0
    const int tid = threadIdx.x;
    const int gt = tid & (kGroup - 1);

    if (tid < kGroup) {
        using S = GroupSync<1, kGroup>;
        const uint32_t total = nruns * (uint32_t)pc.nworkers;
        uint32_t q_next = 0xFFFFFFFFu;   // thread 0: the ticket after this one, drawn while this run is in progress
        if (gt == 0) q_next = atomicAdd(sync + 0, 1u);
        for (;;) {
            if (gt == 0) {
                s_ticket[0] = (ld_acquire(sync + 2) == 0u) ? q_next : 0xFFFFFFFFu;
                if (q_next < total) q_next = atomicAdd(sync + 0, 1u);
            }
            S::sync();
            const uint32_t q = *(volatile uint32_t*)&s_ticket[0];   // (rewritten only after the barriers inside the run)
            if (q >= total) break;
            const uint32_t n = q / nruns;
            const bool ok = col4_run<S>(pc, &tmap, full_rows, (int)n, (q - n * nruns) * 8u, smem_raw, gt, &g_fused_wait_timeouts);
            __threadfence();   // this thread's stores of the intermediate, before the group's count below
            S::sync();
            if (gt == 0) {
                if (ok) atomicAdd(sync + 4 + n, 1u);
                else atomicExch(sync + 2, 1u);
            }
            if (!ok) break;
        }
        row_role<0>(pr, sync, reinterpret_cast<float*>(smem_raw), gt, &s_ticket[2], nruns);
    } else {
        row_role<1>(pr, sync, reinterpret_cast<float*>(smem_raw + kRegionA), gt, &s_ticket[1], nruns);
    }
}

}  // namespace

size_t enc_fused_sync_bytes(int nworkers) { return ((size_t)(4 + nworkers) * 4 + 15) & ~(size_t)15; }

// pc: the strided pass (gradients -> intermediate), pr: the contiguous pass (intermediate -> packed signs),
// both for the same workers.  *launched stays false where the fused form does not apply.
cudaError_t launch_enc_fused(const PassParams& pc, const PassParams& pr, int T, int A, uint32_t* sync, cudaStream_t s,
                             bool* launched)
{
    *launched = false;
    if (T != kT || A != Col4::A || pc.lo_log != kT) return cudaSuccess;
    const uint64_t S = (uint64_t)1 << pc.lo_log;
    const uint64_t rows = (uint64_t)(pc.d >> pc.lo_log);   // whole rows of the gradient
    const int64_t nruns = (pc.dp >> A) / (16 * Col4::RUN);
    if (nruns < 1 || (nruns * 16 * Col4::RUN) << A != pc.dp || nruns * pc.nworkers > 0x7FFFFFFF ||
        (pc.dp >> kT) * pc.nworkers > 0x7FFFFFFF)
        return cudaSuccess;
    CUtensorMap map;
    if (!make_col_tensor_map(&map, pc.src, S, rows, (uint64_t)pc.nworkers, (uint64_t)pc.src_stride)) return cudaSuccess;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(enc_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFusedSmem)) != cudaSuccess) return e;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(sync, 0, enc_fused_sync_bytes(pc.nworkers), s)) != cudaSuccess) return e;
    int64_t blocks = nruns * pc.nworkers;
    if (blocks > sms) blocks = sms;
    enc_fused_kernel<<<(unsigned)blocks, 2 * kGroup, kFusedSmem, s>>>(pc, with_round_keys(pr), map, (uint32_t)nruns, (uint32_t)rows, sync);
    *launched = true;
    return cudaGetLastError();
}

cudaError_t fused_timeouts(int* out) { return cudaMemcpyFromSymbol(out, g_fused_wait_timeouts, sizeof(int)); }

}  // namespace fosgd
