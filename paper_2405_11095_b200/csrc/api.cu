// C-ABI of libfosgd: argument checks, pass planning and kernel launches (no allocation, no
// synchronisation, no state besides the thread-local last CUDA error).
#include <math.h>
#include <stdio.h>

#include <atomic>

#include "../../include/fosgd.h"
#include "common.cuh"

namespace fosgd {

cudaError_t launch_row_10(int, int, const PassParams&, cudaStream_t);
cudaError_t launch_row_11(int, int, const PassParams&, cudaStream_t);
cudaError_t launch_row_12(int, int, const PassParams&, cudaStream_t);
cudaError_t launch_row_13(int, int, const PassParams&, cudaStream_t);
cudaError_t launch_row_14(int, int, const PassParams&, cudaStream_t);
cudaError_t launch_row_15(int, int, const PassParams&, cudaStream_t);

cudaError_t row_timeouts_10(int*);
cudaError_t row_timeouts_11(int*);
cudaError_t row_timeouts_12(int*);
cudaError_t row_timeouts_13(int*);
cudaError_t row_timeouts_14(int*);
cudaError_t row_timeouts_15(int*);

cudaError_t launch_row(int T, int src, int sink, const PassParams& p, cudaStream_t s)
{
    switch (T) {
        case 10: return launch_row_10(src, sink, p, s);
        case 11: return launch_row_11(src, sink, p, s);
        case 12: return launch_row_12(src, sink, p, s);
        case 13: return launch_row_13(src, sink, p, s);
        case 14: return launch_row_14(src, sink, p, s);
        case 15: return launch_row_15(src, sink, p, s);
    }
    return cudaErrorInvalidValue;
}

namespace {

thread_local int g_last_cuda_error = 0;

// Optional per-launch timing hooks (fosgd_trace_passes): caller-owned events, recorded around
// every kernel launch issued by this thread.
struct TraceEntry { char kind; int size, src, sink, workers; bool decoder; };   // workers = 0: the server's own vector (downlink)
thread_local cudaEvent_t* g_trace_events = nullptr;
thread_local int g_trace_capacity = 0;
thread_local int g_trace_count = 0;
constexpr int kTraceMax = 256;
thread_local TraceEntry g_trace_log[kTraceMax];
thread_local char g_trace_label[48];

bool trace_begin(cudaStream_t s)
{
    const bool on = g_trace_events != nullptr && g_trace_count < g_trace_capacity && g_trace_count < kTraceMax;
    if (on) cudaEventRecord(g_trace_events[2 * g_trace_count], s);
    return on;
}

void trace_end(bool on, cudaStream_t s, const TraceEntry& entry)
{
    if (!on) return;
    cudaEventRecord(g_trace_events[2 * g_trace_count + 1], s);
    g_trace_log[g_trace_count] = entry;
    ++g_trace_count;
}

// decoder: the pass belongs to a transform that ends in the flip + sum sink (tells the intermediate passes
// of the two directions apart in the trace)
cudaError_t traced(char kind, int size, int src, int sink, const PassParams& p, cudaStream_t s, bool decoder = false)
{
    const bool on = trace_begin(s);
    cudaError_t e = kind == 'r' ? launch_row(size, src, sink, p, s)
                  : kind == 'c' ? launch_col(size, src, p, s)
                  : kind == 'h' ? launch_colh(size, p, s)
                  : kind == 't' ? launch_tc_col(p, s)
                  : kind == 'u' ? launch_tc_row(p, s)
                                : launch_small(size, src, sink, p, s);
    trace_end(on, s, TraceEntry{kind, size, src, sink, p.id0 == FOSGD_SERVER_ID ? 0 : p.nworkers, decoder});
    return e;
}

// How a transform of length 2^L is cut into passes over the index bits:
//   contiguous pass on bits [0, T), then up to two strided passes on [T, T+A0), [T+A0, L).
// The strided passes run first (they are the ones that read the source), highest bits first.
struct Plan {
    int L;       // log2 of the transform length
    int T;       // contiguous tile (10..15), or L itself when L < 10 (single small kernel)
    int ncol;    // strided passes
    int A[2];    // stages of each strided pass
    int lo[2];   // lowest index bit of each strided pass
};

Plan make_plan(int L)
{
    Plan pl{};
    pl.L = L;
    if (L <= 15) {
        pl.T = L;
        pl.ncol = 0;
        return pl;
    }
    pl.ncol = (L - 15 + 9) / 10;
    pl.T = L - 10 * pl.ncol;
    if (pl.T < 10) pl.T = 10;
    const int rest = L - pl.T;
    if (pl.ncol == 1) {
        pl.A[0] = rest;
    } else {
        pl.A[0] = rest / 2;
        pl.A[1] = rest - pl.A[0];
    }
    pl.lo[0] = pl.T;
    pl.lo[1] = pl.T + pl.A[0];
    return pl;
}

int ilog2(int64_t x)
{
    int l = 0;
    while (((int64_t)1 << l) < x) ++l;
    return l;
}

bool valid_block(int b) { return b == 0 || (b >= 5 && b <= 30); }

int64_t padded_dim(int64_t d, int block_log2)
{
    if (d < 1 || !valid_block(block_log2) || d > ((int64_t)1 << 31)) return -1;
    if (block_log2 == 0) {
        int64_t p = 32;
        while (p < d) p <<= 1;
        return p;
    }
    const int64_t blk = (int64_t)1 << block_log2;
    const int64_t dp = ((d + blk - 1) / blk) * blk;
    return dp > ((int64_t)1 << 31) ? -1 : dp;
}

int planes(int K)
{
    if (K < 1 || K > 255) return 0;
    int P = 0;
    while ((1 << P) < K + 1) ++P;
    return P;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool good_lambda(float l) { return isfinite(l) && l > 0.f; }

size_t src_elem_bytes(int src) { return (src == SRC_G16 || src == SRC_WS16) ? 2 : 4; }
size_t sink_elem_bytes(int) { return 4; }

struct Geometry {
    int64_t dp;
    int L;        // log2 transform length
    double rootn; // sqrt(transform length)
    Plan plan;
    size_t ws_per_worker;
};

bool make_geometry(int64_t d, int block_log2, Geometry* g)
{
    g->dp = padded_dim(d, block_log2);
    if (g->dp < 0) return false;
    g->L = block_log2 == 0 ? ilog2(g->dp) : block_log2;
    g->rootn = sqrt((double)((int64_t)1 << g->L));
    g->plan = make_plan(g->L);
    g->ws_per_worker = g->plan.ncol > 0 ? (size_t)g->dp * 4 : 0;
    return true;
}

Rng make_rng(uint64_t seed, uint64_t step)
{
    Rng r;
    r.k0 = (uint32_t)seed;
    r.k1 = (uint32_t)(seed >> 32) ^ (uint32_t)(step >> 32);
    r.step_lo = (uint32_t)step;
    return r;
}

// which passes of a decoder whose source is one packed plane run on the tensor cores (FOSGD_TC_* bits;
// both by default: each measured faster than its plain-ALU kernel)
std::atomic<int> g_tensor_core_pass{FOSGD_TC_STRIDED | FOSGD_TC_CONTIGUOUS};
bool tc_enabled() { return (g_tensor_core_pass.load(std::memory_order_relaxed) & FOSGD_TC_STRIDED) != 0; }
bool tc_row_enabled() { return (g_tensor_core_pass.load(std::memory_order_relaxed) & FOSGD_TC_CONTIGUOUS) != 0; }
bool tc_any_size() { return (g_tensor_core_pass.load(std::memory_order_relaxed) & FOSGD_TC_ANY_SIZE) != 0; }
// whether an encoder of ten strided stages + a 2^14 tile runs as the one-kernel form or as two kernels (default:
// measured on a B200 the two kernels are the faster form)
std::atomic<int> g_fused_encoder{0};
bool fused_encoder_enabled() { return g_fused_encoder.load(std::memory_order_relaxed) != 0; }

// Enqueue one source -> sink transform for p.nworkers workers.  Workers are processed in
// chunks of as many as the scratch buffer holds; SINK_FINAL accumulates chunk after chunk.
int run_transform(const Geometry& g, int src, int sink, PassParams p, void* ws, size_t ws_bytes,
                  cudaStream_t s)
{
    const Plan& pl = g.plan;
    cudaError_t e = cudaSuccess;
#define FOSGD_CUDA_OK(call) do { e = (call); if (e != cudaSuccess) { g_last_cuda_error = (int)e; return FOSGD_ECUDA; } } while (0)
    if (pl.ncol == 0) {
        FOSGD_CUDA_OK((pl.L < 10) ? traced('s', pl.L, src, sink, p, s) : traced('r', pl.T, src, sink, p, s));
        return FOSGD_OK;
    }
    if (ws == nullptr || ws_bytes < g.ws_per_worker) return FOSGD_EWORKSPACE;
    const size_t cap = ws_bytes / g.ws_per_worker;
    const int total = p.nworkers;
    int chunk = (int)(cap < (size_t)total ? cap : (size_t)total);
    // The one-kernel encoder (fused_encode.cu) keeps its ticket and progress words behind the chunk's
    // intermediates.  Scratch sized for exactly `chunk` workers has no room for them: the chunk then gives up
    // its last worker's slot (a caller who adds enc_fused_sync_bytes to the scratch keeps the full chunk).
    const bool fused_geometry = src == SRC_G32 && sink == SINK_PACK1 && pl.ncol == 1 && pl.A[0] == 10 && pl.T == 14 &&
                                fused_encoder_enabled();
    bool fused = false;
    if (fused_geometry) {
        if (ws_bytes - (size_t)chunk * g.ws_per_worker >= enc_fused_sync_bytes(chunk)) fused = true;
        else if (chunk >= 2) { --chunk; fused = true; }
    }
    const float final_scale = p.scale;
    const int first_overwrite = p.overwrite;
    const char* src0 = static_cast<const char*>(p.src);
    char* dst0 = static_cast<char*>(p.dst);
    const uint32_t id0 = p.id0;
    // a packed one-plane source through a single strided pass stays exact in fp16 (|value| <= 2^A)
    const bool half_path = (src == SRC_BITS && p.P == 1 && pl.ncol == 1 && pl.A[0] >= 6);
    // A packed one-plane source through two strided passes (transform length above 2^25): the first pass's output
    // is still exact in fp16, so with room for it beside the fp32 intermediate (6 instead of 4 bytes per
    // coordinate and worker) the first pass writes half the bytes in 256-byte rows and the second reads half.
    bool half_first = (src == SRC_BITS && p.P == 1 && pl.ncol == 2 && pl.A[1] >= 6 && pl.A[1] <= 10 &&
                       ws_bytes >= g.ws_per_worker + g.ws_per_worker / 2);
    if (half_first) {
        const size_t cap16 = ws_bytes / (g.ws_per_worker + g.ws_per_worker / 2);
        chunk = (int)(cap16 < (size_t)total ? cap16 : (size_t)total);
    }
    char* const ws16 = static_cast<char*>(ws) + (size_t)chunk * g.ws_per_worker;   // (used by half_first only)
    for (int n0 = 0; n0 < total; n0 += chunk) {
        const int m = (total - n0 < chunk) ? total - n0 : chunk;
        PassParams q = p;
        q.nworkers = m;
        q.id0 = id0 + (uint32_t)n0;
        if (p.amp_dev) q.amp_dev = p.amp_dev + (int64_t)n0 * p.amp_stride;
        const void* const srck = src0 + (size_t)n0 * (size_t)p.src_stride * src_elem_bytes(src);
        bool tensor_pass = false;
        if (fused) {
            PassParams pc = q, pr = q;
            pc.src = srck;
            pc.dst = ws;
            pc.dst_stride = g.dp;
            pc.lo_log = pl.lo[0];
            pr.src = ws;
            pr.src_stride = g.dp;
            pr.dst = dst0 + (size_t)n0 * (size_t)p.dst_stride * sink_elem_bytes(sink);
            bool launched = false;
            const bool on = trace_begin(s);
            e = launch_enc_fused(pc, pr, pl.T, pl.A[0], reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + (size_t)chunk * g.ws_per_worker),
                                 s, &launched);
            if (launched) trace_end(on, s, TraceEntry{'f', pl.L, src, sink, p.id0 == FOSGD_SERVER_ID ? 0 : m, false});
            if (e != cudaSuccess) { g_last_cuda_error = (int)e; return FOSGD_ECUDA; }
            if (launched) continue;
            // (not launched: nothing was recorded or enqueued besides the start event, which the next pass re-records)
        }
        if (half_path) {
            PassParams pc = q;
            pc.src = srck;
            pc.dst = ws;
            pc.dst_stride = g.dp;
            pc.lo_log = pl.lo[0];
            // ten stages: H_8 on packed bytes + H_128 on the tensor cores, same fp16 intermediate
            tensor_pass = pl.A[0] == 10 && tc_enabled() && tc_col_applicable(pc, tc_any_size());
            if (tensor_pass) FOSGD_CUDA_OK(traced('t', pl.A[0], SRC_BITS, 4, pc, s));
            else FOSGD_CUDA_OK(traced('h', pl.A[0], SRC_BITS, 4, pc, s));
        } else if (half_first) {
            PassParams pc = q;
            pc.src = srck;
            pc.dst = ws16;
            pc.dst_stride = g.dp;
            pc.lo_log = pl.lo[1];
            if (pl.A[1] == 10 && tc_enabled() && tc_col_applicable(pc, tc_any_size())) FOSGD_CUDA_OK(traced('t', pl.A[1], SRC_BITS, 4, pc, s));
            else FOSGD_CUDA_OK(traced('h', pl.A[1], SRC_BITS, 4, pc, s));
            PassParams pm = q;
            pm.src = ws16;
            pm.src_stride = g.dp;
            pm.dst = ws;
            pm.dst_stride = g.dp;
            pm.lo_log = pl.lo[0];
            FOSGD_CUDA_OK(traced('c', pl.A[0], SRC_WS16, SINK_WS, pm, s, true));
        } else {
            // strided passes, highest bits first: source -> ws, then ws -> ws in place
            for (int c = pl.ncol - 1; c >= 0; --c) {
                PassParams pc = q;
                const bool first = (c == pl.ncol - 1);
                pc.src = first ? srck : ws;
                pc.src_stride = first ? p.src_stride : g.dp;
                pc.dst = ws;
                pc.dst_stride = g.dp;
                pc.lo_log = pl.lo[c];
                FOSGD_CUDA_OK(traced('c', pl.A[c], first ? src : (int)SRC_WS, SINK_WS, pc, s, sink == SINK_FINAL));
            }
        }
        PassParams pr = q;
        pr.src = ws;
        pr.src_stride = g.dp;
        if (sink == SINK_FINAL) {
            pr.overwrite = (n0 == 0) ? first_overwrite : 0;
            pr.scale = (n0 + m == total) ? final_scale : 1.f;
            if (p.amp_mode == AMP_SCALE && n0 + m != total) pr.amp_mode = AMP_DITHER;
        } else {
            pr.dst = dst0 + (size_t)n0 * (size_t)p.dst_stride * sink_elem_bytes(sink);
        }
        if (half_path && sink == SINK_FINAL && tc_row_enabled() && tc_row_applicable(pr, pl.T, tc_any_size()))
            FOSGD_CUDA_OK(traced('u', pl.T, SRC_WS16, sink, pr, s));
        else
            FOSGD_CUDA_OK(traced('r', pl.T, half_path ? (int)SRC_WS16 : (int)SRC_WS, sink, pr, s));
    }
#undef FOSGD_CUDA_OK
    return FOSGD_OK;
}

// An amplitude given by value, or resident on the device (then `value` is 1 and the kernels
// multiply their host-computed factors by the table entry): a single float, or one per worker
// and block of the blocked mode.
struct Amp {
    float value;
    const float* dev;
    int64_t stride;   // floats between workers' rows
    int shift;        // coordinate i -> entry i >> shift
};

Amp amp_value(float v) { return Amp{v, nullptr, 0, 31}; }

// table of the device-amplitude calls: per_block = 0 -> one float; 1 -> [workers][d' >> b]
bool amp_device(const float* dev, int per_block, int block_log2, int64_t dp, bool per_worker, Amp* out)
{
    if (dev == nullptr || (per_block != 0 && per_block != 1)) return false;
    if (per_block && block_log2 == 0) return false;
    *out = per_block ? Amp{1.f, dev, per_worker ? (dp >> block_log2) : 0, block_log2} : Amp{1.f, dev, 0, 31};
    return true;
}

void set_amp(PassParams* p, const Amp& a, int mode)
{
    p->amp_dev = a.dev;
    p->amp_stride = a.stride;
    p->amp_shift = a.shift;
    p->amp_mode = a.dev ? mode : AMP_DITHER;
}

int check_grad_args(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M, int block_log2)
{
    if (grads == nullptr || d < 1 || M < 1 || M > 65535 || !valid_block(block_log2)) return FOSGD_EINVAL;
    if (dtype != FOSGD_F32 && dtype != FOSGD_BF16) return FOSGD_EUNSUPPORTED;
    if (M > 1 && worker_stride < d) return FOSGD_EINVAL;
    const size_t es = dtype == FOSGD_BF16 ? 2 : 4;
    if (!aligned16(grads) || (M > 1 && ((size_t)worker_stride * es) % 16 != 0)) return FOSGD_EALIGN;
    return FOSGD_OK;
}

}  // namespace

void set_last_cuda_error(int e) { g_last_cuda_error = e; }

int check_decode_args(const void* bits, int64_t d, float lambda, int block_log2, const void* out)
{
    if (bits == nullptr || out == nullptr || d < 1 || !valid_block(block_log2) || !good_lambda(lambda))
        return FOSGD_EINVAL;
    if (!aligned16(bits) || !aligned16(out)) return FOSGD_EALIGN;
    return padded_dim(d, block_log2) < 0 ? FOSGD_EUNSUPPORTED : FOSGD_OK;
}

}  // namespace fosgd

using namespace fosgd;

extern "C" {

int64_t fosgd_padded_dim(int64_t d, int block_log2) { return padded_dim(d, block_log2); }

int fosgd_planes(int K) { return planes(K); }

float fosgd_lambda(double B, double alpha, int64_t d_eff)
{
    return (float)(alpha * B * sqrt(log((double)d_eff) / (double)d_eff));
}

float fosgd_lambda_server(double lambda, double alpha_s, int64_t d_eff)
{
    return (float)(alpha_s * lambda * sqrt(log((double)d_eff)));
}

int fosgd_workspace_bytes(int op, int64_t d, int M, int dtype, int block_log2, int K, size_t* out)
{
    if (out == nullptr || d < 1 || M < 1 || !valid_block(block_log2)) return FOSGD_EINVAL;
    if (op < FOSGD_OP_ENCODE || op > FOSGD_OP_BLOCK_AMPLITUDES) return FOSGD_EUNSUPPORTED;
    if (op == FOSGD_OP_BLOCK_AMPLITUDES && block_log2 == 0) return FOSGD_EINVAL;
    if (dtype != FOSGD_F32 && dtype != FOSGD_BF16) return FOSGD_EUNSUPPORTED;
    if ((op == FOSGD_OP_AGGREGATE || op == FOSGD_OP_DOWNLINK_DECODE) && planes(K) == 0) return FOSGD_EINVAL;
    Geometry g;
    if (!make_geometry(d, block_log2, &g)) return FOSGD_EUNSUPPORTED;
    // amplitudes: 256 partial sums per worker, or one per segment of min(2^b, 1024) coordinates
    if (op == FOSGD_OP_AMPLITUDES) *out = (size_t)M * 256 * sizeof(double);
    else if (op == FOSGD_OP_BLOCK_AMPLITUDES) *out = (size_t)M * (size_t)(g.dp >> (block_log2 < 10 ? block_log2 : 10)) * sizeof(double);
    else *out = g.ws_per_worker;
    return FOSGD_OK;
}

static int encode_impl(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M,
                       uint32_t worker_id0, uint64_t seed, uint64_t step, Amp lam, int block_log2,
                       uint32_t* bits, void* ws, size_t ws_bytes, fosgd_stream stream)
{
    const float lambda = lam.value;
    int st = check_grad_args(grads, dtype, d, worker_stride, M, block_log2);
    if (st != FOSGD_OK) return st;
    if (bits == nullptr) return FOSGD_EINVAL;
    if (!aligned16(bits) || (ws && !aligned16(ws))) return FOSGD_EALIGN;
    Geometry g;
    if (!make_geometry(d, block_log2, &g)) return FOSGD_EUNSUPPORTED;
    PassParams p{};
    p.src = grads; p.src_stride = worker_stride; p.d = d; p.dp = g.dp;
    p.dst = bits; p.dst_stride = g.dp >> 5;
    p.dither_c = (float)((double)lambda * g.rootn / 16777216.0);
    set_amp(&p, lam, AMP_DITHER);
    p.P = 1; p.K = 1; p.nworkers = M; p.id0 = worker_id0; p.rng = make_rng(seed, step);
    return run_transform(g, dtype == FOSGD_BF16 ? SRC_G16 : SRC_G32, SINK_PACK1, p, ws, ws_bytes,
                         (cudaStream_t)stream);
}

int fosgd_encode(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M,
                 uint32_t worker_id0, uint64_t seed, uint64_t step, float lambda, int block_log2,
                 uint32_t* bits, void* ws, size_t ws_bytes, fosgd_stream stream)
{
    if (!good_lambda(lambda)) return FOSGD_EINVAL;
    return encode_impl(grads, dtype, d, worker_stride, M, worker_id0, seed, step, amp_value(lambda), block_log2,
                       bits, ws, ws_bytes, stream);
}

int fosgd_encode_dev(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M,
                     uint32_t worker_id0, uint64_t seed, uint64_t step, const float* lambda_dev, int per_block,
                     int block_log2, uint32_t* bits, void* ws, size_t ws_bytes, fosgd_stream stream)
{
    Amp lam;
    if (!amp_device(lambda_dev, per_block, block_log2, padded_dim(d, block_log2), true, &lam)) return FOSGD_EINVAL;
    return encode_impl(grads, dtype, d, worker_stride, M, worker_id0, seed, step, lam, block_log2,
                       bits, ws, ws_bytes, stream);
}

int fosgd_flatten(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M,
                  uint32_t worker_id0, uint64_t seed, uint64_t step, int block_log2,
                  float* out, void* ws, size_t ws_bytes, fosgd_stream stream)
{
    int st = check_grad_args(grads, dtype, d, worker_stride, M, block_log2);
    if (st != FOSGD_OK) return st;
    if (out == nullptr) return FOSGD_EINVAL;
    if (!aligned16(out) || (ws && !aligned16(ws))) return FOSGD_EALIGN;
    Geometry g;
    if (!make_geometry(d, block_log2, &g)) return FOSGD_EUNSUPPORTED;
    PassParams p{};
    p.src = grads; p.src_stride = worker_stride; p.d = d; p.dp = g.dp;
    p.dst = out; p.dst_stride = g.dp;
    p.scale = (float)(1.0 / g.rootn);
    p.P = 1; p.K = 1; p.nworkers = M; p.id0 = worker_id0; p.rng = make_rng(seed, step);
    return run_transform(g, dtype == FOSGD_BF16 ? SRC_G16 : SRC_G32, SINK_WS, p, ws, ws_bytes,
                         (cudaStream_t)stream);
}

int fosgd_decode(const uint32_t* bits, int64_t d, uint32_t worker_id, uint64_t seed, uint64_t step,
                 float lambda, int block_log2, float* out, void* ws, size_t ws_bytes,
                 fosgd_stream stream)
{
    const int st = check_decode_args(bits, d, lambda, block_log2, out);
    if (st != FOSGD_OK) return st;
    if (ws && !aligned16(ws)) return FOSGD_EALIGN;
    Geometry g;
    if (!make_geometry(d, block_log2, &g)) return FOSGD_EUNSUPPORTED;
    PassParams p{};
    p.src = bits; p.src_stride = g.dp >> 5; p.d = d; p.dp = g.dp;
    p.dst = out; p.d_out = d; p.overwrite = 1;
    p.scale = (float)((double)lambda / g.rootn);
    p.P = 1; p.K = 1; p.nworkers = 1; p.id0 = worker_id; p.rng = make_rng(seed, step);
    return run_transform(g, SRC_BITS, SINK_FINAL, p, ws, ws_bytes, (cudaStream_t)stream);
}

// downlink encoder on gbar: all d' accumulator entries are the input, no new padding
static int reencode_impl(const Geometry& g, const float* gbar, uint64_t seed, uint64_t step, Amp lam_s, int K,
                         uint32_t* down_bits, void* ws, size_t ws_bytes, fosgd_stream stream)
{
    PassParams e{};
    const int P = planes(K);
    e.src = gbar; e.src_stride = g.dp; e.d = g.dp; e.dp = g.dp;
    e.dst = down_bits; e.dst_stride = (int64_t)P * (g.dp >> 5);
    e.dither_c = (float)((double)lam_s.value * g.rootn / 16777216.0);
    set_amp(&e, lam_s, AMP_DITHER);
    e.P = P; e.K = K; e.nworkers = 1; e.id0 = FOSGD_SERVER_ID; e.rng = make_rng(seed, step);
    return run_transform(g, SRC_G32, K == 1 ? SINK_PACK1 : SINK_PACKK, e, ws, ws_bytes,
                         (cudaStream_t)stream);
}

static int aggregate_impl(const uint32_t* bits, int64_t d, int M, uint32_t worker_id0, int N_total,
                          uint64_t seed, uint64_t step, Amp lam, int block_log2,
                          float* acc, int flags, Amp lam_s, int K, uint32_t* down_bits,
                          void* ws, size_t ws_bytes, fosgd_stream stream)
{
    const float lambda = lam.value, lambda_s = lam_s.value;
    if (bits == nullptr || acc == nullptr || d < 1 || M < 1 || M > 65535 || N_total < M ||
        !valid_block(block_log2) || (flags & ~(FOSGD_AGG_BEGIN | FOSGD_AGG_END)) != 0)
        return FOSGD_EINVAL;
    const bool end = (flags & FOSGD_AGG_END) != 0;
    const bool reencode = end && down_bits != nullptr;
    if (reencode && planes(K) == 0) return FOSGD_EINVAL;
    if (!aligned16(bits) || !aligned16(acc) || (ws && !aligned16(ws)) || (down_bits && !aligned16(down_bits)))
        return FOSGD_EALIGN;
    Geometry g;
    if (!make_geometry(d, block_log2, &g)) return FOSGD_EUNSUPPORTED;
    if (g.plan.ncol > 0 && (ws == nullptr || ws_bytes < g.ws_per_worker)) return FOSGD_EWORKSPACE;

    PassParams p{};
    p.src = bits; p.src_stride = g.dp >> 5; p.d = d; p.dp = g.dp;
    p.dst = acc; p.d_out = g.dp; p.overwrite = (flags & FOSGD_AGG_BEGIN) ? 1 : 0;
    p.scale = end ? (float)((double)lambda / ((double)N_total * g.rootn)) : 1.f;
    // one amplitude for all workers scales the finished sum; per-worker amplitudes weight every term
    set_amp(&p, lam, lam.stride ? AMP_WEIGHT : (end ? AMP_SCALE : AMP_DITHER));
    p.P = 1; p.K = 1; p.nworkers = M; p.id0 = worker_id0; p.rng = make_rng(seed, step);
    int st = run_transform(g, SRC_BITS, SINK_FINAL, p, ws, ws_bytes, (cudaStream_t)stream);
    if (st != FOSGD_OK || !reencode) return st;

    return reencode_impl(g, acc, seed, step, lam_s, K, down_bits, ws, ws_bytes, stream);
}

int fosgd_server_aggregate(const uint32_t* bits, int64_t d, int M, uint32_t worker_id0, int N_total,
                           uint64_t seed, uint64_t step, float lambda, int block_log2,
                           float* acc, int flags, float lambda_s, int K, uint32_t* down_bits,
                           void* ws, size_t ws_bytes, fosgd_stream stream)
{
    if (!good_lambda(lambda)) return FOSGD_EINVAL;
    if ((flags & FOSGD_AGG_END) && down_bits != nullptr && !good_lambda(lambda_s)) return FOSGD_EINVAL;
    return aggregate_impl(bits, d, M, worker_id0, N_total, seed, step, amp_value(lambda), block_log2, acc, flags,
                          amp_value(lambda_s), K, down_bits, ws, ws_bytes, stream);
}

int fosgd_server_aggregate_dev(const uint32_t* bits, int64_t d, int M, uint32_t worker_id0, int N_total,
                               uint64_t seed, uint64_t step, const float* lambda_dev, const float* lambda_s_dev,
                               int per_block, int block_log2, float* acc, int flags, int K, uint32_t* down_bits,
                               void* ws, size_t ws_bytes, fosgd_stream stream)
{
    const int64_t dp = padded_dim(d, block_log2);
    Amp lam, lam_s = amp_value(1.f);
    if (!amp_device(lambda_dev, per_block, block_log2, dp, true, &lam)) return FOSGD_EINVAL;
    if ((flags & FOSGD_AGG_END) && down_bits != nullptr &&
        !amp_device(lambda_s_dev, per_block, block_log2, dp, false, &lam_s))
        return FOSGD_EINVAL;
    return aggregate_impl(bits, d, M, worker_id0, N_total, seed, step, lam, block_log2, acc, flags,
                          lam_s, K, down_bits, ws, ws_bytes, stream);
}

// out = D(q) (axpy_factor == 0), or out += axpy_factor * D(q)
static int downlink_impl(const uint32_t* down_bits, int64_t d, uint64_t seed, uint64_t step,
                         Amp lam_s, int K, int block_log2, float* out, void* ws,
                         size_t ws_bytes, fosgd_stream stream, double axpy_factor = 0.0)
{
    const float lambda_s = lam_s.value;
    if (down_bits == nullptr || out == nullptr || d < 1 || !valid_block(block_log2) || planes(K) == 0)
        return FOSGD_EINVAL;
    if (!aligned16(down_bits) || !aligned16(out) || (ws && !aligned16(ws))) return FOSGD_EALIGN;
    Geometry g;
    if (!make_geometry(d, block_log2, &g)) return FOSGD_EUNSUPPORTED;
    PassParams p{};
    const int P = planes(K);
    p.src = down_bits; p.src_stride = (int64_t)P * (g.dp >> 5); p.d = d; p.dp = g.dp;
    p.dst = out; p.d_out = d; p.overwrite = axpy_factor != 0.0 ? 2 : 1;
    p.scale = (float)((axpy_factor != 0.0 ? axpy_factor : 1.0) * (double)lambda_s / ((double)K * g.rootn));
    set_amp(&p, lam_s, AMP_SCALE);
    p.P = P; p.K = K; p.nworkers = 1; p.id0 = FOSGD_SERVER_ID; p.rng = make_rng(seed, step);
    return run_transform(g, SRC_BITS, SINK_FINAL, p, ws, ws_bytes, (cudaStream_t)stream);
}

int fosgd_downlink_decode(const uint32_t* down_bits, int64_t d, uint64_t seed, uint64_t step,
                          float lambda_s, int K, int block_log2, float* out, void* ws,
                          size_t ws_bytes, fosgd_stream stream)
{
    if (!good_lambda(lambda_s)) return FOSGD_EINVAL;
    return downlink_impl(down_bits, d, seed, step, amp_value(lambda_s), K, block_log2, out, ws, ws_bytes, stream);
}

int fosgd_downlink_decode_dev(const uint32_t* down_bits, int64_t d, uint64_t seed, uint64_t step,
                              const float* lambda_s_dev, int per_block, int K, int block_log2, float* out, void* ws,
                              size_t ws_bytes, fosgd_stream stream)
{
    Amp lam_s;
    if (!amp_device(lambda_s_dev, per_block, block_log2, padded_dim(d, block_log2), false, &lam_s)) return FOSGD_EINVAL;
    return downlink_impl(down_bits, d, seed, step, lam_s, K, block_log2, out, ws, ws_bytes, stream);
}

int fosgd_downlink_encode(const float* gbar, int64_t d, uint64_t seed, uint64_t step, float lambda_s,
                          const float* lambda_s_dev, int per_block, int K, int block_log2, uint32_t* down_bits,
                          void* ws, size_t ws_bytes, fosgd_stream stream)
{
    if (gbar == nullptr || down_bits == nullptr || d < 1 || !valid_block(block_log2) || planes(K) == 0)
        return FOSGD_EINVAL;
    if (!aligned16(gbar) || !aligned16(down_bits) || (ws && !aligned16(ws))) return FOSGD_EALIGN;
    Geometry g;
    if (!make_geometry(d, block_log2, &g)) return FOSGD_EUNSUPPORTED;
    Amp lam_s = amp_value(lambda_s);
    if (lambda_s_dev != nullptr) {
        if (!amp_device(lambda_s_dev, per_block, block_log2, g.dp, false, &lam_s)) return FOSGD_EINVAL;
    } else if (!good_lambda(lambda_s) || per_block != 0) {
        return FOSGD_EINVAL;
    }
    return reencode_impl(g, gbar, seed, step, lam_s, K, down_bits, ws, ws_bytes, stream);
}

int fosgd_downlink_apply(const uint32_t* down_bits, int64_t d, uint64_t seed, uint64_t step, float lambda_s,
                         const float* lambda_s_dev, int per_block, int K, int block_log2, float step_size,
                         float* x, void* ws, size_t ws_bytes, fosgd_stream stream)
{
    if (!isfinite(step_size) || step_size == 0.f) return FOSGD_EINVAL;
    Amp lam_s = amp_value(lambda_s);
    if (lambda_s_dev != nullptr) {
        if (!amp_device(lambda_s_dev, per_block, block_log2, padded_dim(d, block_log2), false, &lam_s)) return FOSGD_EINVAL;
    } else if (!good_lambda(lambda_s) || per_block != 0) {
        return FOSGD_EINVAL;
    }
    return downlink_impl(down_bits, d, seed, step, lam_s, K, block_log2, x, ws, ws_bytes, stream, -(double)step_size);
}

int fosgd_amplitudes(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M, double alpha,
                     double alpha_s, int block_log2, int per_block, float* lambda_dev, float* lambda_s_dev,
                     void* ws, size_t ws_bytes, fosgd_stream stream)
{
    int st = check_grad_args(grads, dtype, d, worker_stride, M, block_log2);
    if (st != FOSGD_OK) return st;
    if (lambda_dev == nullptr || !(alpha > 0.0) || !(alpha_s > 0.0) || !isfinite(alpha) || !isfinite(alpha_s) ||
        (per_block != 0 && per_block != 1) || (per_block && block_log2 == 0))
        return FOSGD_EINVAL;
    Geometry g;
    if (!make_geometry(d, block_log2, &g)) return FOSGD_EUNSUPPORTED;
    if (per_block && (g.dp >> block_log2) * (int64_t)M > ((int64_t)1 << 31)) return FOSGD_EUNSUPPORTED;
    const size_t need = per_block ? (size_t)M * (size_t)(g.dp >> (block_log2 < 10 ? block_log2 : 10)) * sizeof(double)
                                  : (size_t)M * 256 * sizeof(double);
    if (ws == nullptr || ws_bytes < need) return FOSGD_EWORKSPACE;
    if (!aligned16(ws)) return FOSGD_EALIGN;
    const bool on = g_trace_events != nullptr && g_trace_count < g_trace_capacity && g_trace_count < kTraceMax;
    if (on) cudaEventRecord(g_trace_events[2 * g_trace_count], (cudaStream_t)stream);
    const cudaError_t e =
        per_block ? launch_block_amplitudes(grads, dtype == FOSGD_BF16, d, g.dp, worker_stride, M, block_log2, alpha,
                                            alpha_s, lambda_dev, lambda_s_dev, static_cast<double*>(ws),
                                            (cudaStream_t)stream)
                  : launch_amplitudes(grads, dtype == FOSGD_BF16, d, worker_stride, M, alpha, alpha_s,
                                      (double)((int64_t)1 << g.L), lambda_dev, lambda_s_dev, static_cast<double*>(ws),
                                      (cudaStream_t)stream);
    if (on) {
        cudaEventRecord(g_trace_events[2 * g_trace_count + 1], (cudaStream_t)stream);
        g_trace_log[g_trace_count] = TraceEntry{'n', g.L, dtype == FOSGD_BF16 ? 1 : 0, 5, M, false};
        ++g_trace_count;
    }
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; return FOSGD_ECUDA; }
    return FOSGD_OK;
}

int fosgd_encode_measured(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M, uint32_t worker_id0,
                          uint64_t seed, uint64_t step, double alpha, double alpha_s, int block_log2, float* lambda_dev,
                          float* lambda_s_dev, uint32_t* bits, void* ws, size_t ws_bytes, void* amp_ws,
                          size_t amp_ws_bytes, fosgd_stream stream)
{
    int st = check_grad_args(grads, dtype, d, worker_stride, M, block_log2);
    if (st != FOSGD_OK) return st;
    if (lambda_dev == nullptr || bits == nullptr || !(alpha > 0.0) || !(alpha_s > 0.0) || !isfinite(alpha) || !isfinite(alpha_s))
        return FOSGD_EINVAL;
    if (!aligned16(bits) || (ws && !aligned16(ws)) || (amp_ws && !aligned16(amp_ws))) return FOSGD_EALIGN;
    Geometry g;
    if (!make_geometry(d, block_log2, &g)) return FOSGD_EUNSUPPORTED;
    if (amp_ws == nullptr || amp_ws_bytes < (size_t)M * 256 * sizeof(double)) return FOSGD_EWORKSPACE;
    if (g.plan.ncol > 0 && (ws == nullptr || ws_bytes < g.ws_per_worker)) return FOSGD_EWORKSPACE;
    const Plan& pl = g.plan;
    cudaStream_t s = (cudaStream_t)stream;
    // One pass over the gradients where the strided pass can carry the sums: fp32, ten strided stages through the
    // copy engine, and scratch for all M workers at once (the amplitude is a maximum over all of them, so every
    // strided pass must be over before the first dither).
    if (dtype == FOSGD_F32 && pl.ncol == 1 && pl.A[0] == 10 && ws_bytes / g.ws_per_worker >= (size_t)M) {
        PassParams pc{};
        pc.src = grads; pc.src_stride = worker_stride; pc.d = d; pc.dp = g.dp;
        pc.dst = ws; pc.dst_stride = g.dp; pc.lo_log = pl.lo[0];
        pc.P = 1; pc.K = 1; pc.nworkers = M; pc.id0 = worker_id0; pc.rng = make_rng(seed, step);
        bool launched = false;
        int nruns = 0;
        bool on = trace_begin(s);
        cudaError_t e = launch_col4_norm(pc, static_cast<double*>(amp_ws), s, &launched, &nruns);
        if (launched) trace_end(on, s, TraceEntry{'c', pl.A[0], SRC_G32, SINK_WS, M, false});
        if (e != cudaSuccess) { g_last_cuda_error = (int)e; return FOSGD_ECUDA; }
        if (launched) {
            on = trace_begin(s);
            e = launch_amplitudes_finalize(static_cast<const double*>(amp_ws), M, nruns, alpha, alpha_s,
                                           (double)((int64_t)1 << g.L), lambda_dev, lambda_s_dev, s);
            trace_end(on, s, TraceEntry{'n', g.L, 0, 5, M, false});
            if (e != cudaSuccess) { g_last_cuda_error = (int)e; return FOSGD_ECUDA; }
            PassParams pr = pc;
            pr.src = ws; pr.src_stride = g.dp;
            pr.dst = bits; pr.dst_stride = g.dp >> 5;
            pr.dither_c = (float)(g.rootn / 16777216.0);
            set_amp(&pr, Amp{1.f, lambda_dev, 0, 31}, AMP_DITHER);
            e = traced('r', pl.T, SRC_WS, SINK_PACK1, pr, s);
            if (e != cudaSuccess) { g_last_cuda_error = (int)e; return FOSGD_ECUDA; }
            return FOSGD_OK;
        }
    }
    // elsewhere: the norm pass, then the encoder
    st = fosgd_amplitudes(grads, dtype, d, worker_stride, M, alpha, alpha_s, block_log2, 0, lambda_dev, lambda_s_dev,
                          amp_ws, amp_ws_bytes, stream);
    if (st != FOSGD_OK) return st;
    return fosgd_encode_dev(grads, dtype, d, worker_stride, M, worker_id0, seed, step, lambda_dev, 0, block_log2, bits,
                            ws, ws_bytes, stream);
}

const char* fosgd_strerror(int status)
{
    switch (status) {
        case FOSGD_OK: return "ok";
        case FOSGD_EINVAL: return "invalid argument";
        case FOSGD_EALIGN: return "pointer or stride not 16-byte aligned";
        case FOSGD_EWORKSPACE: return "workspace missing or too small";
        case FOSGD_EUNSUPPORTED: return "unsupported dtype, op or size";
        case FOSGD_ECUDA: return "CUDA launch error (see fosgd_last_cuda_error)";
        case FOSGD_ELIMIT: return "scratch need exceeds the built-in array (multi-pass transforms: d' <= 2^20 coordinates)";
    }
    return "unknown status";
}

int fosgd_last_cuda_error(void) { return g_last_cuda_error; }

int fosgd_async_timeouts(int* count)
{
    if (count == nullptr) return FOSGD_EINVAL;
    cudaError_t (*const fns[])(int*) = {row_timeouts_10, row_timeouts_11, row_timeouts_12,
                                        row_timeouts_13, row_timeouts_14, row_timeouts_15};
    int total = 0;
    {
        int t = 0;
        int f = 0;
        cudaError_t e = col_timeouts(&total);
        if (e == cudaSuccess) e = tc_timeouts(&t);
        int u = 0;
        if (e == cudaSuccess) e = fused_timeouts(&f);
        if (e == cudaSuccess) e = tcrow_timeouts(&u);
        if (e != cudaSuccess) { g_last_cuda_error = (int)e; return FOSGD_ECUDA; }
        total += t + f + u;
    }
    for (auto fn : fns) {
        int c = 0;
        const cudaError_t e = fn(&c);
        if (e != cudaSuccess) { g_last_cuda_error = (int)e; return FOSGD_ECUDA; }
        total += c;
    }
    *count = total;
    return FOSGD_OK;
}

int fosgd_trace_passes(void** events, int capacity)
{
    if (events != nullptr && capacity < 1) return FOSGD_EINVAL;
    g_trace_events = reinterpret_cast<cudaEvent_t*>(events);
    g_trace_capacity = events ? capacity : 0;
    g_trace_count = 0;
    return FOSGD_OK;
}

int fosgd_trace_count(void) { return g_trace_count; }

const char* fosgd_trace_label(int k)
{
    if (k < 0 || k >= g_trace_count) return "";
    static const char* const srcs[] = {"f32", "bf16", "bits", "ws", "ws16"};
    static const char* const sinks[] = {"ws", "pack1", "packK", "final", "ws16", "amp"};
    const TraceEntry& t = g_trace_log[k];
    char who[16];
    if (t.workers > 0) snprintf(who, sizeof who, "%d", t.workers);
    else snprintf(who, sizeof who, "srv");
    snprintf(g_trace_label, sizeof g_trace_label, "%s%d:%s->%s@%s",
             t.kind == 'r' ? "row" : (t.kind == 'c' ? (t.decoder ? "dcol" : "col") : (t.kind == 'h' ? "colh" : (t.kind == 'n' ? "norm" : (t.kind == 't' ? "tc" : (t.kind == 'u' ? "tcrow" : (t.kind == 'f' ? "fused" : "small")))))),
             t.size, srcs[t.src], sinks[t.sink], who);
    return g_trace_label;
}

int fosgd_set_tensor_core_pass(int mask)
{
    return g_tensor_core_pass.exchange(mask & (FOSGD_TC_STRIDED | FOSGD_TC_CONTIGUOUS | FOSGD_TC_ANY_SIZE), std::memory_order_relaxed);
}

int fosgd_set_fused_encoder(int on)
{
    return g_fused_encoder.exchange(on ? 1 : 0, std::memory_order_relaxed);
}

const char* fosgd_version(void) { return "libfosgd 0.1 (sm_100a)"; }

}  // extern "C"
