// Shared device helpers and launch parameter blocks of libfosgd (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace fosgd {

// ---- sources and sinks of a transform pass -------------------------------------------
enum Src : int {
    SRC_G32 = 0,   // caller gradients, fp32: zero padding beyond d, sign flip D_eps
    SRC_G16 = 1,   // caller gradients, bf16 (exact upcast), same padding and flip
    SRC_BITS = 2,  // packed signs / count planes: q_i = 2 c_i - K
    SRC_WS = 3,    // fp32 intermediate of an earlier pass
    SRC_WS16 = 4   // fp16 intermediate (exact small integers from a packed one-plane source)
};
enum Sink : int {
    SINK_WS = 0,     // fp32 intermediate (or the scaled transform output of fosgd_flatten)
    SINK_PACK1 = 1,  // dither + sign + pack, K = 1
    SINK_PACKK = 2,  // K dithers, count, P bit planes
    SINK_FINAL = 3   // flip, sum over the workers of the launch, optional read-modify-write, scale
};

struct Rng {
    uint32_t k0, k1;   // Philox key: lo32(seed), hi32(seed) ^ hi32(step)
    uint32_t step_lo;  // counter word 2
};

struct PassParams {
    const void* src;
    void* dst;
    int64_t src_stride;  // elements (grads, ws) or words (bits) between consecutive workers
    int64_t dst_stride;
    int64_t d;           // valid source elements per worker (gradient sources)
    int64_t dp;          // padded length d'
    int64_t d_out;       // SINK_FINAL: outputs written (d for a decoder, d' for the accumulator)
    float scale;         // SINK_WS and SINK_FINAL: multiplier on the stored value
    float dither_c;      // lambda * sqrt(n) * 2^-24: dither integer -> unnormalised transform units
    int P, K;            // bit planes and dithers
    int overwrite;       // SINK_FINAL: 1 = store scale * sum, 0 = store scale * (dst + sum), 2 = dst += scale * sum
    int nworkers;        // workers handled by this launch
    uint32_t id0;        // generator id of the launch's first worker
    int lo_log;          // strided pass: log2 of the stride between butterfly partners
    // Amplitudes resident on the device (null: folded into dither_c / scale on the host).  Worker n,
    // coordinate i reads amp_dev[n * amp_stride + (i >> amp_shift)]: a single entry (stride 0,
    // shift 31) or one entry per worker and block of the blocked mode.  Pack sinks multiply
    // dither_c by it; SINK_FINAL follows amp_mode.
    const float* amp_dev;
    int64_t amp_stride;
    int amp_shift;
    int amp_mode;        // AMP_DITHER, AMP_SCALE or AMP_WEIGHT
    Rng rng;
};

enum AmpMode {
    AMP_DITHER = 0,  // SINK_FINAL ignores the amplitudes
    AMP_SCALE = 1,   // SINK_FINAL multiplies its scale by worker 0's entry (one amplitude for all workers)
    AMP_WEIGHT = 2   // SINK_FINAL weights every worker's contribution by that worker's entry
};

// 1 when no table is given
__device__ __forceinline__ float amplitude_at(const PassParams& p, int n, int64_t i)
{
    return p.amp_dev ? __ldg(p.amp_dev + (int64_t)n * p.amp_stride + (i >> p.amp_shift)) : 1.f;
}

// The parameter block of the kernels with a dither sink: PassParams plus the ten round keys of the
// generator (Weyl sequence of the key), computed once on the host.  As kernel parameters they sit in
// the constant bank and feed the round's logic instruction directly, which saves the two additions
// per round that every call would otherwise repeat (4 % of the one-dither pack pass).  The other
// kernels keep the plain block: with the table in it the flip + accumulate kernels, which never use
// it, ran 8 % slower.
struct PassParamsRK : PassParams {
    uint32_t rk0[10], rk1[10];
};

inline PassParamsRK with_round_keys(const PassParams& p)
{
    PassParamsRK r;
    static_cast<PassParams&>(r) = p;
    for (int i = 0; i < 10; ++i) {
        r.rk0[i] = p.rng.k0 + (uint32_t)i * 0x9E3779B9u;
        r.rk1[i] = p.rng.k1 + (uint32_t)i * 0xBB67AE85u;
    }
    return r;
}

// ---- Philox4x32-10 (Salmon et al., SC'11), written from the published round function ----
// Two forms of the same ten rounds.  rng_words_dither takes the round keys from a table in the
// parameter bank: for the dither sinks, whose every thread makes eight calls per tile.  rng_words
// advances the key by addition inside the rounds: for the flip words, which a thread generates once
// or twice per tile.
__device__ __forceinline__ uint4 rng_words_dither(const PassParamsRK& p, uint32_t id, uint32_t domain, uint32_t c)
{
    uint32_t c0 = c, c1 = domain, c2 = p.rng.step_lo, c3 = id;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ p.rk0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ p.rk1[r];
        c0 = n0;
        c1 = (uint32_t)p1;
        c2 = n2;
        c3 = (uint32_t)p0;
    }
    return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint4 rng_words(const Rng& g, uint32_t id, uint32_t domain, uint32_t c)
{
    uint32_t c0 = c, c1 = domain, c2 = g.step_lo, c3 = id, k0 = g.k0, k1 = g.k1;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c0 = n0;
        c1 = (uint32_t)p1;
        c2 = n2;
        c3 = (uint32_t)p0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint32_t pick(const uint4& w, uint32_t j)
{
    return j == 0 ? w.x : (j == 1 ? w.y : (j == 2 ? w.z : w.w));
}

// Word j of the flip vector eps (32 flips, set bit = -1): output j&3 of counter j>>2, domain 0.
__device__ __forceinline__ uint32_t eps_word(const Rng& g, uint32_t id, uint32_t j)
{
    return pick(rng_words(g, id, 0u, j >> 2), j & 3u);
}

// Dither integer from one generator word: t = 2*k24 + 1 - 2^24 (odd, |t| < 2^24, exact in fp32).
__device__ __forceinline__ float dither_from_word(uint32_t w)
{
    return (float)((int)((w >> 8) << 1) - 16777215);
}

__device__ __forceinline__ float flip_by_bit(float x, uint32_t word, uint32_t bit)
{
    return __uint_as_float(__float_as_uint(x) ^ (((word >> bit) & 1u) << 31));
}

// value of coordinate (word, bit) read from P count planes spaced `plane_words` apart: 2c - K
__device__ __forceinline__ float plane_value(const uint32_t* w0, int64_t plane_words, int P, int K,
                                             uint32_t bit)
{
    int c = 0;
    for (int p = 0; p < P; ++p) c |= (int)((__ldg(w0 + (int64_t)p * plane_words) >> bit) & 1u) << p;
    return (float)(2 * c - K);
}

// 32 x 32 bit-matrix transpose across a warp: on entry lane l holds row l (bit r = entry (l, r));
// on return lane l holds column l (bit r = entry (r, l)).  Five exchange rounds.
__device__ __forceinline__ uint32_t warp_transpose_bits(uint32_t x, uint32_t lane)
{
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const uint32_t mask = (s == 16) ? 0x0000FFFFu : (s == 8) ? 0x00FF00FFu : (s == 4) ? 0x0F0F0F0Fu
                            : (s == 2) ? 0x33333333u : 0x55555555u;
        const uint32_t y = __shfl_xor_sync(0xFFFFFFFFu, x, s);
        // lanes with bit s clear keep their low halves and take the partner's low halves shifted up
        x = (lane & s) ? ((x & ~mask) | ((y >> s) & mask)) : ((x & mask) | ((y << s) & ~mask));
    }
    return x;
}

// In-register butterflies over the register-index bits selected by ACTIVE (5-bit mask).
template <int ACTIVE, typename V = float>
__device__ __forceinline__ void butterflies32(V (&v)[32])
{
#pragma unroll
    for (int s = 0; s < 5; ++s) {
        if ((ACTIVE >> s) & 1) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                if (!(i & (1 << s))) {
                    const V a = v[i], b = v[i | (1 << s)];
                    v[i] = a + b;
                    v[i | (1 << s)] = a - b;
                }
            }
        }
    }
}

// ---- mbarrier helpers (asynchronous copies signal completion on a shared-memory barrier) ----
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// bounded wait for the barrier phase with the given parity; false if it never completed
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity)
{
    for (int it = 0; it < (1 << 22); ++it) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

__device__ __forceinline__ void mbar_inval(uint64_t* bar)
{
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Every thread that touched a shared-memory buffer through ordinary loads and stores runs this
// before the barrier after which one thread hands the buffer to the asynchronous copy engine.
__device__ __forceinline__ void fence_generic_before_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

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

// ---- shared by the translation units of the C-ABI (not exported) -----------------------------
// thread-local last CUDA error behind fosgd_last_cuda_error()
__attribute__((visibility("hidden"))) void set_last_cuda_error(int e);
// argument checks of fosgd_decode without the scratch: FOSGD_OK, FOSGD_EINVAL, FOSGD_EALIGN or FOSGD_EUNSUPPORTED
__attribute__((visibility("hidden"))) int check_decode_args(const void* bits, int64_t d, float lambda, int block_log2,
                                                            const void* out);

// ---- host-visible launchers (one translation unit per family) --------------------------
cudaError_t launch_row(int T, int src, int sink, const PassParams& p, cudaStream_t s);
cudaError_t launch_col(int A, int src, const PassParams& p, cudaStream_t s);
cudaError_t launch_colh(int A, const PassParams& p, cudaStream_t s);   // one-plane bits -> fp16 intermediate
bool tc_col_applicable(const PassParams& p, bool any_size);                            // ten strided stages from one plane on the tensor cores
cudaError_t launch_tc_col(const PassParams& p, cudaStream_t s);          // one-plane bits -> fp16 intermediate
cudaError_t tc_timeouts(int* out);
bool tc_row_applicable(const PassParams& p, int T, bool any_size);                     // contiguous 2^14 tiles of the fp16 intermediate, seven stages on the tensor cores
cudaError_t launch_tc_row(const PassParams& p, cudaStream_t s);          // fp16 intermediate -> flip + sum sink
cudaError_t tcrow_timeouts(int* out);
// uplink encoder of a 2^24-long transform as one kernel (strided and contiguous pass side by side)
size_t enc_fused_sync_bytes(int nworkers);                               // zeroed device words the launch needs
cudaError_t launch_enc_fused(const PassParams& pc, const PassParams& pr, int T, int A, uint32_t* sync, cudaStream_t s,
                             bool* launched);
cudaError_t fused_timeouts(int* out);
cudaError_t col_timeouts(int* out);                                      // synchronising read of the strided unit's counter
cudaError_t launch_small(int L, int src, int sink, const PassParams& p, cudaStream_t s);
cudaError_t launch_amplitudes(const void* grads, int bf16, int64_t d, int64_t worker_stride, int M, double alpha,
                              double alpha_s, double n_eff, float* lam, float* lam_s, double* partial, cudaStream_t s);
cudaError_t launch_amplitudes_finalize(const double* partial, int M, int nparts, double alpha, double alpha_s, double n_eff,
                                       float* lam, float* lam_s, cudaStream_t s);
cudaError_t launch_col4_norm(const PassParams& p, double* partial, cudaStream_t s, bool* launched, int* nruns_out);
cudaError_t launch_block_amplitudes(const void* grads, int bf16, int64_t d, int64_t dp, int64_t worker_stride, int M,
                                    int block_log2, double alpha, double alpha_s, float* lam, float* lam_s,
                                    double* seg, cudaStream_t st);

}  // namespace fosgd
