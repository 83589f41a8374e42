"""Python binding of libfosgd (FO-SGD gradient-compression round trip on one B200).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
Tensors are torch CUDA tensors used as device buffers; the calls enqueue work on torch's
current stream and return without synchronising.  There is no CPU fallback: the first call
into the package without a built ``libfosgd.so`` raises ImportError.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libfosgd.so")

F32, BF16 = 0, 1
AGG_BEGIN, AGG_END = 1, 2
OP_ENCODE, OP_DECODE, OP_AGGREGATE, OP_DOWNLINK_DECODE, OP_FLATTEN, OP_AMPLITUDES, OP_BLOCK_AMPLITUDES = range(7)
OK, EINVAL, EALIGN, EWORKSPACE, EUNSUPPORTED, ECUDA, ELIMIT = 0, -1, -2, -3, -4, -5, -6
NOALLOC_SCRATCH_BYTES = 4 << 20
SERVER_ID = 0xFFFFFFFF

EXPORTS = ("fosgd_padded_dim", "fosgd_planes", "fosgd_lambda", "fosgd_lambda_server",
           "fosgd_workspace_bytes", "fosgd_encode", "fosgd_flatten", "fosgd_decode",
           "fosgd_server_aggregate", "fosgd_downlink_decode", "fosgd_strerror",
           "fosgd_last_cuda_error", "fosgd_version", "fosgd_trace_passes", "fosgd_trace_count",
           "fosgd_trace_label", "fosgd_decode_noalloc", "fosgd_async_timeouts", "fosgd_amplitudes",
           "fosgd_encode_dev", "fosgd_server_aggregate_dev", "fosgd_downlink_decode_dev", "fosgd_downlink_apply",
           "fosgd_downlink_encode", "fosgd_probe_issue_rate", "fosgd_set_tensor_core_pass",
           "fosgd_set_fused_encoder", "fosgd_encode_measured")


class FosgdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.fosgd_strerror(status).decode()
        if status == ECUDA:
            msg += f" [cudaError {_lib.fosgd_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({status})")


def _load() -> C.CDLL:
    if not os.path.exists(_SO):
        raise ImportError(
            f"{_SO} is missing: build it with `python -m paper_2405_11095_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    L = C.CDLL(_SO)
    i64, u64, u32, cint, vp, f32, dbl, sz = (C.c_int64, C.c_uint64, C.c_uint32, C.c_int, C.c_void_p,
                                             C.c_float, C.c_double, C.c_size_t)
    L.fosgd_padded_dim.argtypes, L.fosgd_padded_dim.restype = [i64, cint], i64
    L.fosgd_planes.argtypes, L.fosgd_planes.restype = [cint], cint
    L.fosgd_lambda.argtypes, L.fosgd_lambda.restype = [dbl, dbl, i64], f32
    L.fosgd_lambda_server.argtypes, L.fosgd_lambda_server.restype = [dbl, dbl, i64], f32
    L.fosgd_workspace_bytes.argtypes = [cint, i64, cint, cint, cint, cint, C.POINTER(sz)]
    L.fosgd_encode.argtypes = [vp, cint, i64, i64, cint, u32, u64, u64, f32, cint, vp, vp, sz, vp]
    L.fosgd_flatten.argtypes = [vp, cint, i64, i64, cint, u32, u64, u64, cint, vp, vp, sz, vp]
    L.fosgd_decode.argtypes = [vp, i64, u32, u64, u64, f32, cint, vp, vp, sz, vp]
    L.fosgd_server_aggregate.argtypes = [vp, i64, cint, u32, cint, u64, u64, f32, cint, vp, cint,
                                         f32, cint, vp, vp, sz, vp]
    L.fosgd_downlink_decode.argtypes = [vp, i64, u64, u64, f32, cint, cint, vp, vp, sz, vp]
    L.fosgd_decode_noalloc.argtypes = [vp, i64, u32, u64, u64, f32, cint, vp, vp]
    L.fosgd_async_timeouts.argtypes = [C.POINTER(cint)]
    L.fosgd_amplitudes.argtypes = [vp, cint, i64, i64, cint, dbl, dbl, cint, cint, vp, vp, vp, sz, vp]
    L.fosgd_encode_dev.argtypes = [vp, cint, i64, i64, cint, u32, u64, u64, vp, cint, cint, vp, vp, sz, vp]
    L.fosgd_server_aggregate_dev.argtypes = [vp, i64, cint, u32, cint, u64, u64, vp, vp, cint, cint, vp, cint, cint,
                                             vp, vp, sz, vp]
    L.fosgd_downlink_encode.argtypes = [vp, i64, u64, u64, C.c_float, vp, cint, cint, cint, vp, vp, sz, vp]
    L.fosgd_downlink_apply.argtypes = [vp, i64, u64, u64, C.c_float, vp, cint, cint, cint, C.c_float, vp, vp, sz, vp]
    L.fosgd_downlink_decode_dev.argtypes = [vp, i64, u64, u64, vp, cint, cint, cint, vp, vp, sz, vp]
    L.fosgd_probe_issue_rate.argtypes = [cint, cint, C.POINTER(dbl), vp, vp]
    L.fosgd_set_tensor_core_pass.argtypes, L.fosgd_set_tensor_core_pass.restype = [cint], cint
    L.fosgd_set_fused_encoder.argtypes, L.fosgd_set_fused_encoder.restype = [cint], cint
    L.fosgd_encode_measured.argtypes = [vp, cint, i64, i64, cint, u32, u64, u64, dbl, dbl, cint, vp, vp, vp, vp, sz, vp, sz, vp]
    L.fosgd_strerror.argtypes, L.fosgd_strerror.restype = [cint], C.c_char_p
    L.fosgd_last_cuda_error.restype = cint
    L.fosgd_version.restype = C.c_char_p
    L.fosgd_trace_passes.argtypes = [C.POINTER(vp), cint]
    L.fosgd_trace_count.restype = cint
    L.fosgd_trace_label.argtypes, L.fosgd_trace_label.restype = [cint], C.c_char_p
    return L


_handle = None


def lib() -> C.CDLL:
    """The raw C-ABI handle (for callers that pass plain device pointers).  Loaded on first
    use; raises ImportError if the shared library has not been built."""
    global _handle
    if _handle is None:
        _handle = _load()
    return _handle


class _Lazy:
    def __getattr__(self, name):
        return getattr(lib(), name)


_lib = _Lazy()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise FosgdError(status, where)


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise FosgdError(EUNSUPPORTED, f"dtype {t.dtype}")


def padded_dim(d: int, block_log2: int = 0) -> int:
    return _lib.fosgd_padded_dim(d, block_log2)


def planes(K: int) -> int:
    return _lib.fosgd_planes(K)


def transform_len(d: int, block_log2: int = 0) -> int:
    return padded_dim(d, 0) if block_log2 == 0 else 1 << block_log2


def lambda_(B: float, alpha: float, d_eff: int) -> float:
    return _lib.fosgd_lambda(B, alpha, d_eff)


def lambda_server(lam: float, alpha_s: float, d_eff: int) -> float:
    return _lib.fosgd_lambda_server(lam, alpha_s, d_eff)


def workspace_bytes(op: int, d: int, M: int = 1, dtype: int = F32, block_log2: int = 0, K: int = 1) -> int:
    out = C.c_size_t(0)
    _check(_lib.fosgd_workspace_bytes(op, d, M, dtype, block_log2, K, C.byref(out)), "fosgd_workspace_bytes")
    return out.value


def encode(grads, d, bits, lam, seed, step, worker_id0=0, block_log2=0, ws=None, worker_stride=None):
    """fosgd_encode: grads [M, >=d] (fp32/bf16, row stride = worker_stride) -> bits [M, d'/32] int32."""
    M = grads.shape[0] if grads.dim() == 2 else 1
    stride = worker_stride if worker_stride is not None else (grads.stride(0) if grads.dim() == 2 else d)
    _check(_lib.fosgd_encode(_ptr(grads), _dtype_code(grads), d, stride, M, worker_id0, seed, step, lam,
                             block_log2, _ptr(bits), _ptr(ws), _nbytes(ws), _stream()), "fosgd_encode")
    return bits


def flatten(grads, d, out, seed, step, worker_id0=0, block_log2=0, ws=None, worker_stride=None):
    """fosgd_flatten: out [M, d'] fp32 = H D_eps x."""
    M = grads.shape[0] if grads.dim() == 2 else 1
    stride = worker_stride if worker_stride is not None else (grads.stride(0) if grads.dim() == 2 else d)
    _check(_lib.fosgd_flatten(_ptr(grads), _dtype_code(grads), d, stride, M, worker_id0, seed, step,
                              block_log2, _ptr(out), _ptr(ws), _nbytes(ws), _stream()), "fosgd_flatten")
    return out


def decode(bits, d, out, lam, seed, step, worker_id, block_log2=0, ws=None):
    """fosgd_decode: bits [d'/32] -> out [d] fp32."""
    _check(_lib.fosgd_decode(_ptr(bits), d, worker_id, seed, step, lam, block_log2, _ptr(out), _ptr(ws),
                             _nbytes(ws), _stream()), "fosgd_decode")
    return out


def decode_noalloc(bits, d, out, lam, seed, step, worker_id, block_log2=0):
    """fosgd_decode_noalloc: fosgd_decode for callers that cannot allocate device scratch.

    The scratch is a fixed 4 MiB array inside the library (multi-pass transforms up to d' = 2^20,
    else ELIMIT; single-pass ones need none); the call allocates nothing.  Calls share that array: do not let two of them overlap on a GPU.
    The first call on a device should happen outside stream capture."""
    _check(_lib.fosgd_decode_noalloc(_ptr(bits), d, worker_id, seed, step, lam, block_log2, _ptr(out),
                                     _stream()), "fosgd_decode_noalloc")
    return out


def server_aggregate(bits, d, acc, lam, seed, step, N_total=None, worker_id0=0, flags=AGG_BEGIN | AGG_END,
                     lam_s=0.0, K=1, down_bits=None, block_log2=0, ws=None):
    """fosgd_server_aggregate: bits [M, d'/32] -> acc [d'] fp32 (and down_bits [P, d'/32] on END)."""
    M = bits.shape[0] if bits.dim() == 2 else 1
    _check(_lib.fosgd_server_aggregate(_ptr(bits), d, M, worker_id0, M if N_total is None else N_total,
                                       seed, step, lam, block_log2, _ptr(acc), flags, lam_s, K,
                                       _ptr(down_bits), _ptr(ws), _nbytes(ws), _stream()),
           "fosgd_server_aggregate")
    return acc


def downlink_decode(down_bits, d, out, lam_s, seed, step, K=1, block_log2=0, ws=None):
    """fosgd_downlink_decode: down_bits [P, d'/32] -> out [d] fp32."""
    _check(_lib.fosgd_downlink_decode(_ptr(down_bits), d, seed, step, lam_s, K, block_log2, _ptr(out),
                                      _ptr(ws), _nbytes(ws), _stream()), "fosgd_downlink_decode")
    return out


def amplitudes(grads, d, lam, lam_s=None, alpha=2.0, alpha_s=2.0, block_log2=0, per_block=False, ws=None,
               worker_stride=None):
    """fosgd_amplitudes: device tensors lam ([1], or [M, d' >> b] with per_block) and lam_s ([1] or
    [d' >> b], optional) <- the amplitudes of the gradients' own norms."""
    M = grads.shape[0] if grads.dim() == 2 else 1
    stride = worker_stride if worker_stride is not None else (grads.stride(0) if grads.dim() == 2 else d)
    _check(_lib.fosgd_amplitudes(_ptr(grads), _dtype_code(grads), d, stride, M, alpha, alpha_s, block_log2,
                                 int(per_block), _ptr(lam), _ptr(lam_s), _ptr(ws), _nbytes(ws), _stream()),
           "fosgd_amplitudes")
    return lam, lam_s


def encode_dev(grads, d, bits, lam, seed, step, worker_id0=0, block_log2=0, per_block=False, ws=None,
               worker_stride=None):
    """fosgd_encode_dev: fosgd_encode with the amplitude(s) read from the device tensor `lam`."""
    M = grads.shape[0] if grads.dim() == 2 else 1
    stride = worker_stride if worker_stride is not None else (grads.stride(0) if grads.dim() == 2 else d)
    _check(_lib.fosgd_encode_dev(_ptr(grads), _dtype_code(grads), d, stride, M, worker_id0, seed, step,
                                 _ptr(lam), int(per_block), block_log2, _ptr(bits), _ptr(ws), _nbytes(ws), _stream()),
           "fosgd_encode_dev")
    return bits


def encode_measured(grads, d, bits, lam, lam_s, seed, step, alpha=2.0, alpha_s=2.0, worker_id0=0, block_log2=0, ws=None,
                    amp_ws=None, worker_stride=None):
    """fosgd_encode_measured: amplitudes(...) and encode_dev(...) in one call (one amplitude for all workers);
    the gradients are read once where the encoder's first pass can carry the norm.  lam, lam_s: device [1]."""
    M = grads.shape[0] if grads.dim() == 2 else 1
    stride = worker_stride if worker_stride is not None else (grads.stride(0) if grads.dim() == 2 else d)
    _check(_lib.fosgd_encode_measured(_ptr(grads), _dtype_code(grads), d, stride, M, worker_id0, seed, step, alpha, alpha_s,
                                      block_log2, _ptr(lam), _ptr(lam_s), _ptr(bits), _ptr(ws), _nbytes(ws), _ptr(amp_ws),
                                      _nbytes(amp_ws), _stream()), "fosgd_encode_measured")
    return bits


def server_aggregate_dev(bits, d, acc, lam, seed, step, N_total=None, worker_id0=0, flags=AGG_BEGIN | AGG_END,
                         lam_s=None, K=1, down_bits=None, block_log2=0, per_block=False, ws=None):
    """fosgd_server_aggregate_dev: amplitudes read from the device tensors `lam` and `lam_s`."""
    M = bits.shape[0] if bits.dim() == 2 else 1
    _check(_lib.fosgd_server_aggregate_dev(_ptr(bits), d, M, worker_id0, M if N_total is None else N_total,
                                           seed, step, _ptr(lam), _ptr(lam_s), int(per_block), block_log2, _ptr(acc),
                                           flags, K, _ptr(down_bits), _ptr(ws), _nbytes(ws), _stream()),
           "fosgd_server_aggregate_dev")
    return acc


def downlink_decode_dev(down_bits, d, out, lam_s, seed, step, K=1, block_log2=0, per_block=False, ws=None):
    """fosgd_downlink_decode_dev: lambda^s read from the device tensor `lam_s`."""
    _check(_lib.fosgd_downlink_decode_dev(_ptr(down_bits), d, seed, step, _ptr(lam_s), int(per_block), K, block_log2,
                                          _ptr(out), _ptr(ws), _nbytes(ws), _stream()), "fosgd_downlink_decode_dev")
    return out


def downlink_encode(gbar, d, down_bits, lam_s, seed, step, K=1, block_log2=0, per_block=False, ws=None):
    """fosgd_downlink_encode: the server's encoder on a finished average gbar [d'] -> down_bits
    [P, d'/32].  lam_s: a float, or a device tensor in either layout of `amplitudes`."""
    dev = None if isinstance(lam_s, (int, float)) else lam_s
    _check(_lib.fosgd_downlink_encode(_ptr(gbar), d, seed, step, 0.0 if dev is not None else float(lam_s), _ptr(dev),
                                      int(per_block), K, block_log2, _ptr(down_bits), _ptr(ws), _nbytes(ws),
                                      _stream()), "fosgd_downlink_encode")
    return down_bits


def downlink_apply(down_bits, d, x, lam_s, seed, step, step_size, K=1, block_log2=0, per_block=False, ws=None):
    """fosgd_downlink_apply: x <- x - step_size * D(down_bits) (eq. (4.2) fused into the downlink
    decoder).  lam_s: a float, or a device tensor in either layout of `amplitudes`."""
    dev = None if isinstance(lam_s, (int, float)) else lam_s
    _check(_lib.fosgd_downlink_apply(_ptr(down_bits), d, seed, step, 0.0 if dev is not None else float(lam_s),
                                     _ptr(dev), int(per_block), K, block_log2, float(step_size), _ptr(x),
                                     _ptr(ws), _nbytes(ws), _stream()), "fosgd_downlink_apply")
    return x


TC_STRIDED, TC_CONTIGUOUS, TC_ANY_SIZE = 1, 2, 4


def set_tensor_core_pass(mask: int) -> int:
    """fosgd_set_tensor_core_pass: which decoder passes from one packed plane run on the tensor cores
    (TC_STRIDED | TC_CONTIGUOUS bits, TC_ANY_SIZE to skip the size thresholds); returns the
    previous mask."""
    return int(_lib.fosgd_set_tensor_core_pass(int(mask)))


def set_fused_encoder(on: bool) -> bool:
    """fosgd_set_fused_encoder: run the uplink encoder of a 2^24-long transform as one kernel (True) or as
    its two passes one after the other (False, the default and the faster form); returns the previous setting."""
    return bool(_lib.fosgd_set_fused_encoder(int(bool(on))))


def fused_sync_bytes(M: int) -> int:
    """FOSGD_FUSED_SYNC_BYTES: scratch beyond M * workspace_bytes(OP_ENCODE, ...) with which the one-kernel
    encoder takes all M workers in one launch."""
    return ((M + 4) * 4 + 15) & ~15


PROBE_FADD, PROBE_FFMA, PROBE_LOP3, PROBE_IMAD = range(4)


def probe_issue_rate(kind: int, iters: int, sink) -> float:
    """fosgd_probe_issue_rate: enqueue the probe kernel of `kind` on the current stream and return
    the lane operations it executes (time it with events around this call)."""
    ops = C.c_double(0.0)
    _check(_lib.fosgd_probe_issue_rate(kind, iters, C.byref(ops), _ptr(sink), _stream()), "fosgd_probe_issue_rate")
    return ops.value


def async_timeouts() -> int:
    """fosgd_async_timeouts: blocks that abandoned a bounded wait (0 when healthy); synchronises."""
    c = C.c_int(0)
    _check(_lib.fosgd_async_timeouts(C.byref(c)), "fosgd_async_timeouts")
    return c.value


def version() -> str:
    return _lib.fosgd_version().decode()


class PassTrace:
    """Per-kernel CUDA-event timing of the library calls made inside a ``with`` block
    (fosgd_trace_passes).  ``durations_ms()`` synchronises and returns [(label, ms), ...]."""

    def __init__(self, capacity: int = 32):
        import torch
        self.capacity = capacity
        self.events = [torch.cuda.Event(enable_timing=True) for _ in range(2 * capacity)]
        for e in self.events:           # torch creates the handle lazily, on first record
            e.record()
        self._arr = (C.c_void_p * (2 * capacity))(*[e.cuda_event for e in self.events])
        self.labels = []

    def __enter__(self):
        _check(_lib.fosgd_trace_passes(self._arr, self.capacity), "fosgd_trace_passes")
        return self

    def __exit__(self, *exc):
        n = _lib.fosgd_trace_count()
        self.labels = [_lib.fosgd_trace_label(k).decode() for k in range(n)]
        _lib.fosgd_trace_passes(None, 0)
        return False

    def durations_ms(self):
        import torch
        torch.cuda.synchronize()
        return [(lab, self.events[2 * k].elapsed_time(self.events[2 * k + 1]))
                for k, lab in enumerate(self.labels)]
