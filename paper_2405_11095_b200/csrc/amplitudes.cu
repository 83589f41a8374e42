// Dither amplitudes computed on the device (Theorem 5.5): B = max_n ||g_n||_2 over the workers of
// the call, lambda = alpha B sqrt(ln n / n), lambda^s = alpha^s lambda sqrt(ln n), n the transform
// length.  Two small kernels: per-block partial sums of squares in fp64, then one block that adds
// the partials of each worker in a fixed order (so the result does not depend on scheduling),
// takes the maximum and writes the two amplitudes as floats.
//
// Blocked mode, one amplitude per worker and block: the same law applied to every block x_b of
// 2^b coordinates with its own norm, lambda_{n,b} = alpha ||x_{n,b}||_2 sqrt(ln 2^b / 2^b) (the
// flattening bound, Lemma 3.6, holds for each block's transform separately), and for the server
// lambda^s_b = alpha^s max_n lambda_{n,b} sqrt(ln 2^b), since ||Z(x)||_2 <= lambda sqrt(n)
// (Remark 5.2) bounds the norm of the averaged block by max_n lambda_{n,b} 2^{b/2}.
#include "common.cuh"

namespace fosgd {

constexpr int kNormBlocks = 256;
constexpr float kMinBlockAmplitude = 1e-30f;

template <bool BF16>
__global__ void __launch_bounds__(256) sumsq_partial_kernel(const void* grads, int64_t d, int64_t worker_stride, double* partial)
{
    const int n = blockIdx.y;
    double acc = 0.0;
    // 16-byte loads over the aligned body (rows start 16-byte aligned), scalar loads over the tail
    constexpr int V = BF16 ? 8 : 4;
    const int64_t nv = d / V;
    const uint4* row = reinterpret_cast<const uint4*>(static_cast<const char*>(grads) + (int64_t)n * worker_stride * (BF16 ? 2 : 4));
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < nv; i += (int64_t)gridDim.x * 256) {
        const uint4 w = __ldg(row + i);
        const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (BF16) {
                const double lo = (double)__uint_as_float(u[k] << 16), hi = (double)__uint_as_float(u[k] & 0xFFFF0000u);
                acc += lo * lo;
                acc += hi * hi;
            } else {
                const double x = (double)__uint_as_float(u[k]);
                acc += x * x;
            }
        }
    }
    if (blockIdx.x == 0) {
        for (int64_t i = nv * V + threadIdx.x; i < d; i += 256) {
            float x;
            if (BF16) x = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(row)[i] << 16);
            else x = reinterpret_cast<const float*>(row)[i];
            acc += (double)x * (double)x;
        }
    }
    __shared__ double red[256];
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) partial[(int64_t)n * gridDim.x + blockIdx.x] = red[0];
}

__global__ void __launch_bounds__(256) amplitudes_finalize_kernel(const double* partial, int M, int nblocks, double alpha,
                                                                  double alpha_s, double n_eff, float* lam_out, float* lam_s_out)
{
    __shared__ double best[256];
    double mine = 0.0;
    for (int n = threadIdx.x; n < M; n += 256) {
        double s = 0.0;
        for (int b = 0; b < nblocks; ++b) s += partial[(int64_t)n * nblocks + b];
        mine = fmax(mine, s);
    }
    best[threadIdx.x] = mine;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) best[threadIdx.x] = fmax(best[threadIdx.x], best[threadIdx.x + s]);
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const double B = sqrt(best[0]);
        const double lam = alpha * B * sqrt(log(n_eff) / n_eff);
        lam_out[0] = (float)lam;
        if (lam_s_out) lam_s_out[0] = (float)(alpha_s * lam * sqrt(log(n_eff)));
    }
}

// ---- one amplitude per worker and block ----------------------------------------------------
// Each warp sums the squares of 1024 consecutive coordinates in 32 coalesced steps and emits the
// sum of every segment of 2^s of them, s = min(b, 10): the block sums themselves for b <= 10,
// partials of 1024 coordinates for larger blocks.
template <bool BF16>
__global__ void __launch_bounds__(128) segment_sumsq_kernel(const void* grads, int64_t d, int64_t dp, int64_t worker_stride,
                                                            int s, double* seg)
{
    const int n = blockIdx.y;
    const uint32_t lane = threadIdx.x & 31u;
    const int64_t warp_base = ((int64_t)blockIdx.x * 4 + (threadIdx.x >> 5)) << 10;
    if (warp_base >= dp) return;
    const float* g32 = static_cast<const float*>(grads) + (int64_t)n * worker_stride;
    const uint16_t* g16 = static_cast<const uint16_t*>(grads) + (int64_t)n * worker_stride;
    auto value = [&](int64_t i) -> float {
        if (i >= d) return 0.f;
        return BF16 ? __uint_as_float((uint32_t)g16[i] << 16) : g32[i];
    };
    double acc = 0.0;
    if (s == 10) {
        // one segment per warp: four consecutive coordinates per lane and step (rows start 16-byte
        // aligned, so the groups of four are aligned too)
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const int64_t i = warp_base + t * 128 + lane * 4;
            float x[4];
            if (i + 3 < d) {
                if (BF16) {
                    const uint2 w = __ldg(reinterpret_cast<const uint2*>(g16 + i));
                    x[0] = __uint_as_float(w.x << 16); x[1] = __uint_as_float(w.x & 0xFFFF0000u);
                    x[2] = __uint_as_float(w.y << 16); x[3] = __uint_as_float(w.y & 0xFFFF0000u);
                } else {
                    const float4 q = __ldg(reinterpret_cast<const float4*>(g32 + i));
                    x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w;
                }
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k) x[k] = value(i + k);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) acc += (double)x[k] * (double)x[k];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) seg[(int64_t)n * (dp >> 10) + (warp_base >> 10)] = acc;
        return;
    }
    const int steps = 1 << (s - 5);          // coalesced steps of 32 coordinates per segment
    for (int t = 0; t < 32; ++t) {
        const float x = value(warp_base + t * 32 + lane);
        acc += (double)x * (double)x;
        if (((t + 1) & (steps - 1)) == 0) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
            const int64_t k = (warp_base >> s) + (t >> (s - 5));
            if (lane == 0 && (k << s) < dp) seg[(int64_t)n * (dp >> s) + k] = acc;
            acc = 0.0;
        }
    }
}

// One warp per (worker, block): adds the block's segment sums lane-strided, then across lanes,
// always in the same order.
__global__ void __launch_bounds__(128) block_amplitudes_kernel(const double* seg, int64_t nb, int64_t segs_per_block,
                                                               int M, double alpha, double n_eff, float* lam)
{
    const int64_t w = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    const uint32_t lane = threadIdx.x & 31u;
    if (w >= nb * M) return;
    const double* row = seg + w * segs_per_block;      // (n * nb + blk) * segs_per_block
    double acc = 0.0;
    for (int64_t k = lane; k < segs_per_block; k += 32) acc += row[k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    // floor: a block of zeros keeps a positive amplitude, so that its sign bits are still
    // decided by the dither (and decode to ~0) instead of by the sign of a zero
    if (lane == 0) lam[w] = fmaxf((float)(alpha * sqrt(acc) * sqrt(log(n_eff) / n_eff)), kMinBlockAmplitude);
}

__global__ void __launch_bounds__(128) server_block_amplitudes_kernel(const float* lam, int64_t nb, int M, double alpha_s,
                                                                      double n_eff, float* lam_s)
{
    const int64_t blk = (int64_t)blockIdx.x * 128 + threadIdx.x;
    if (blk >= nb) return;
    float m = 0.f;
    for (int n = 0; n < M; ++n) m = fmaxf(m, lam[(int64_t)n * nb + blk]);
    lam_s[blk] = (float)(alpha_s * (double)m * sqrt(log(n_eff)));
}

cudaError_t launch_block_amplitudes(const void* grads, int bf16, int64_t d, int64_t dp, int64_t worker_stride, int M,
                                    int block_log2, double alpha, double alpha_s, float* lam, float* lam_s,
                                    double* seg, cudaStream_t st)
{
    const int s = block_log2 < 10 ? block_log2 : 10;
    const int64_t nb = dp >> block_log2;
    const double n_eff = (double)((int64_t)1 << block_log2);
    const dim3 grid((unsigned)((dp + 4095) >> 12), (unsigned)M);
    if (bf16) segment_sumsq_kernel<true><<<grid, 128, 0, st>>>(grads, d, dp, worker_stride, s, seg);
    else segment_sumsq_kernel<false><<<grid, 128, 0, st>>>(grads, d, dp, worker_stride, s, seg);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int64_t warps = nb * M;
    block_amplitudes_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, st>>>(seg, nb, (int64_t)1 << (block_log2 - s), M, alpha,
                                                                        n_eff, lam);
    e = cudaGetLastError();
    if (e != cudaSuccess || lam_s == nullptr) return e;
    server_block_amplitudes_kernel<<<(unsigned)((nb + 127) / 128), 128, 0, st>>>(lam, nb, M, alpha_s, n_eff, lam_s);
    return cudaGetLastError();
}

cudaError_t launch_amplitudes(const void* grads, int bf16, int64_t d, int64_t worker_stride, int M, double alpha,
                              double alpha_s, double n_eff, float* lam, float* lam_s, double* partial, cudaStream_t s)
{
    const dim3 grid(kNormBlocks, (unsigned)M);
    if (bf16) sumsq_partial_kernel<true><<<grid, 256, 0, s>>>(grads, d, worker_stride, partial);
    else sumsq_partial_kernel<false><<<grid, 256, 0, s>>>(grads, d, worker_stride, partial);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    amplitudes_finalize_kernel<<<1, 256, 0, s>>>(partial, M, kNormBlocks, alpha, alpha_s, n_eff, lam, lam_s);
    return cudaGetLastError();
}

// the second step alone: amplitudes from partial sums of squares that another kernel gathered ([M][nparts])
cudaError_t launch_amplitudes_finalize(const double* partial, int M, int nparts, double alpha, double alpha_s, double n_eff,
                                       float* lam, float* lam_s, cudaStream_t s)
{
    amplitudes_finalize_kernel<<<1, 256, 0, s>>>(partial, M, nparts, alpha, alpha_s, n_eff, lam, lam_s);
    return cudaGetLastError();
}

}  // namespace fosgd
