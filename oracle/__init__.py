"""ctypes front end of the CPU oracle (``fosgd_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  The library package never imports this module.  Arrays are numpy; all
floating point is float64 except the packed words (uint32) and the sign margins (float32).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fosgd_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_SO = os.path.join(_OUT_DIR, "libfosgd_oracle.so")

SERVER_ID = 0xFFFFFFFF


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, no fast-math, no threading)."""
    if (not force and os.path.exists(_SO)
            and os.path.getmtime(_SO) >= os.path.getmtime(_SRC)):
        return _SO
    os.makedirs(_OUT_DIR, exist_ok=True)
    tmp = _SO + f".tmp{os.getpid()}"
    subprocess.run(["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"],
                   check=True)
    os.replace(tmp, _SO)
    return _SO


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u32p, f64p, f32p = (C.POINTER(C.c_uint32), C.POINTER(C.c_double), C.POINTER(C.c_float))
        i64, u64, u32, dbl, cint = C.c_int64, C.c_uint64, C.c_uint32, C.c_double, C.c_int
        L.fosgd_oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.fosgd_oracle_rng_words.argtypes = [u64, u64, u32, u32, u32, u32p]
        L.fosgd_oracle_eps.argtypes = [u64, u64, u32, i64]
        L.fosgd_oracle_eps.restype = cint
        L.fosgd_oracle_dither_t.argtypes = [u64, u64, u32, u32, i64]
        L.fosgd_oracle_dither_t.restype = C.c_int32
        L.fosgd_oracle_fwht.argtypes = [f64p, i64]
        L.fosgd_oracle_padded_dim.argtypes = [i64, cint]
        L.fosgd_oracle_padded_dim.restype = i64
        L.fosgd_oracle_lambda.argtypes = [dbl, dbl, i64]
        L.fosgd_oracle_lambda.restype = dbl
        L.fosgd_oracle_lambda_server.argtypes = [dbl, dbl, i64]
        L.fosgd_oracle_lambda_server.restype = dbl
        L.fosgd_oracle_planes.argtypes = [cint]
        L.fosgd_oracle_planes.restype = cint
        L.fosgd_oracle_flatten.argtypes = [f64p, i64, cint, u64, u64, u32, f64p]
        L.fosgd_oracle_flatten_entry.argtypes = [f64p, i64, cint, u64, u64, u32, i64]
        L.fosgd_oracle_flatten_entry.restype = dbl
        L.fosgd_oracle_encode.argtypes = [f64p, i64, cint, u64, u64, u32, dbl, cint, u32p, f32p]
        i64p = C.POINTER(C.c_int64)
        L.fosgd_oracle_decode_entry.argtypes = [u32p, i64, cint, u64, u64, u32, dbl, cint, i64]
        L.fosgd_oracle_decode_entry.restype = dbl
        L.fosgd_oracle_flatten_grid.argtypes = [C.c_void_p, cint, i64, u64, u64, u32, cint, i64p, cint, i64p, cint, f64p]
        L.fosgd_oracle_decode_grid.argtypes = [u32p, i64, u64, u64, u32, dbl, cint, cint, i64p, cint, i64p, cint, f64p]
        L.fosgd_oracle_decode_full.argtypes = [u32p, i64, cint, u64, u64, u32, dbl, cint, f64p]
        L.fosgd_oracle_encode_tab.argtypes = [f64p, i64, cint, u64, u64, u32, f64p, cint, u32p, f32p]
        L.fosgd_oracle_decode_full_tab.argtypes = [u32p, i64, cint, u64, u64, u32, f64p, cint, f64p]
        L.fosgd_oracle_aggregate.argtypes = [u32p, i64, cint, u32, u64, u64, dbl, cint, f64p]
        L.fosgd_oracle_downlink_encode.argtypes = [f64p, i64, cint, u64, u64, dbl, cint, u32p, f32p]
        L.fosgd_oracle_downlink_decode.argtypes = [u32p, i64, cint, u64, u64, dbl, cint, f64p]
        _lib = L
    return _lib


def _p(a: np.ndarray, ct):
    return a.ctypes.data_as(C.POINTER(ct))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _u32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.uint32)


def philox4x32_10(ctr, key) -> np.ndarray:
    c, k, o = _u32(ctr), _u32(key), np.zeros(4, np.uint32)
    lib().fosgd_oracle_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(o, C.c_uint32))
    return o


def rng_words(seed, step, wid, domain, c) -> np.ndarray:
    o = np.zeros(4, np.uint32)
    lib().fosgd_oracle_rng_words(seed, step, wid, domain, c, _p(o, C.c_uint32))
    return o


def eps(seed, step, wid, i) -> int:
    return lib().fosgd_oracle_eps(seed, step, wid, i)


def eps_vector(seed, step, wid, n) -> np.ndarray:
    return np.array([eps(seed, step, wid, i) for i in range(n)], dtype=np.float64)


def dither_t(seed, step, wid, k, i) -> int:
    return lib().fosgd_oracle_dither_t(seed, step, wid, k, i)


def fwht(x) -> np.ndarray:
    y = _f64(x).copy()
    lib().fosgd_oracle_fwht(_p(y, C.c_double), y.size)
    return y


def padded_dim(d, block_log2=0) -> int:
    return lib().fosgd_oracle_padded_dim(d, block_log2)


def transform_len(d, block_log2=0) -> int:
    return padded_dim(d, 0) if block_log2 == 0 else 1 << block_log2


def lam(B, alpha, d_eff) -> float:
    return lib().fosgd_oracle_lambda(B, alpha, d_eff)


def lam_server(lam_, alpha_s, d_eff) -> float:
    return lib().fosgd_oracle_lambda_server(lam_, alpha_s, d_eff)


def planes(K) -> int:
    return lib().fosgd_oracle_planes(K)


def flatten(g, seed, step, wid, block_log2=0) -> np.ndarray:
    g = _f64(g)
    y = np.empty(padded_dim(g.size, block_log2), np.float64)
    lib().fosgd_oracle_flatten(_p(g, C.c_double), g.size, block_log2, seed, step, wid,
                               _p(y, C.c_double))
    return y


def flatten_entry(g, seed, step, wid, k, block_log2=0) -> float:
    g = _f64(g)
    return lib().fosgd_oracle_flatten_entry(_p(g, C.c_double), g.size, block_log2, seed, step,
                                            wid, k)


def decode_entry(pl, d, seed, step, wid, lam_, k, K=1, block_log2=0) -> float:
    """One output of the decoder (Def. 3.8) from the matrix definition."""
    pl = _u32(pl)
    return lib().fosgd_oracle_decode_entry(_p(pl, C.c_uint32), d, block_log2, seed, step, wid, lam_, K, k)


def _grid(k_hi, k_lo):
    hi, lo = np.ascontiguousarray(k_hi, dtype=np.int64), np.ascontiguousarray(k_lo, dtype=np.int64)
    return hi, lo, np.empty((hi.size, lo.size), np.float64)


def flatten_grid(g, seed, step, wid, split_log2, k_hi, k_lo) -> np.ndarray:
    """Entries k = k_hi[a] * 2^split_log2 + k_lo[b] of the global transform H D_eps x -> [n_hi, n_lo].
    g: float64, or float32 (used as is, for vectors too long to hold twice in host memory)."""
    g = np.ascontiguousarray(g)
    if g.dtype != np.float32:
        g = _f64(g)
    hi, lo, out = _grid(k_hi, k_lo)
    lib().fosgd_oracle_flatten_grid(g.ctypes.data_as(C.c_void_p), int(g.dtype == np.float32), g.size, seed, step,
                                    wid, split_log2, _p(hi, C.c_int64), hi.size, _p(lo, C.c_int64), lo.size,
                                    _p(out, C.c_double))
    return out


def decode_grid(pl, d, seed, step, wid, lam_, split_log2, k_hi, k_lo, K=1) -> np.ndarray:
    """Entries k = k_hi[a] * 2^split_log2 + k_lo[b] of the global decoder (Def. 3.8) -> [n_hi, n_lo]."""
    pl = _u32(pl)
    hi, lo, out = _grid(k_hi, k_lo)
    lib().fosgd_oracle_decode_grid(_p(pl, C.c_uint32), d, seed, step, wid, lam_, K, split_log2,
                                   _p(hi, C.c_int64), hi.size, _p(lo, C.c_int64), lo.size, _p(out, C.c_double))
    return out


def _lam_table(lam_, dp, block_log2):
    """None for a single amplitude, else the per-block table [d' >> b] as float64."""
    if np.ndim(lam_) == 0:
        return None
    tab = _f64(lam_)
    assert block_log2 > 0 and tab.shape == (dp >> block_log2,), "one amplitude per block"
    return tab


def encode(g, seed, step, wid, lam_, K=1, block_log2=0, want_margin=False):
    """-> planes [P, d'/32] uint32 (and the sign margins [d'] float32 if asked).
    lam_: one amplitude, or (blocked mode) an array with one amplitude per block."""
    g = _f64(g)
    dp = padded_dim(g.size, block_log2)
    out = np.zeros((planes(K), dp // 32), np.uint32)
    zm = np.empty(dp, np.float32) if want_margin else None
    tab = _lam_table(lam_, dp, block_log2)
    if tab is None:
        lib().fosgd_oracle_encode(_p(g, C.c_double), g.size, block_log2, seed, step, wid, lam_, K,
                                  _p(out, C.c_uint32), _p(zm, C.c_float) if want_margin else None)
    else:
        lib().fosgd_oracle_encode_tab(_p(g, C.c_double), g.size, block_log2, seed, step, wid,
                                      _p(tab, C.c_double), K, _p(out, C.c_uint32),
                                      _p(zm, C.c_float) if want_margin else None)
    return (out, zm) if want_margin else out


def decode_full(pl, d, seed, step, wid, lam_, K=1, block_log2=0) -> np.ndarray:
    pl = _u32(pl)
    dp = padded_dim(d, block_log2)
    out = np.empty(dp, np.float64)
    tab = _lam_table(lam_, dp, block_log2)
    if tab is None:
        lib().fosgd_oracle_decode_full(_p(pl, C.c_uint32), d, block_log2, seed, step, wid, lam_, K,
                                       _p(out, C.c_double))
    else:
        lib().fosgd_oracle_decode_full_tab(_p(pl, C.c_uint32), d, block_log2, seed, step, wid,
                                           _p(tab, C.c_double), K, _p(out, C.c_double))
    return out


def block_amplitudes(G, alpha, alpha_s, block_log2):
    """Per-block amplitude law: G [M, d] -> (lam [M, nb], lam_s [nb]) with
    lam[n, k] = alpha ||G[n] on block k||_2 sqrt(ln 2^b / 2^b) (Lemma 3.6 / Theorem 5.5 per block)
    and lam_s[k] = alpha_s max_n lam[n, k] sqrt(ln 2^b) (Remark 5.2 bounds the averaged block).
    lam is floored at 1e-30 (a block of zeros keeps a dither that decides its bits)."""
    G = np.atleast_2d(_f64(G))
    M, d = G.shape
    dp = padded_dim(d, block_log2)
    n = 1 << block_log2
    X = np.zeros((M, dp))
    X[:, :d] = G
    norms = np.sqrt((X.reshape(M, dp // n, n) ** 2).sum(axis=2))
    lam_ = np.maximum(alpha * norms * np.sqrt(np.log(n) / n), 1e-30)
    return lam_, alpha_s * lam_.max(axis=0) * np.sqrt(np.log(n))


def aggregate(bits, d, seed, step, lam_, worker_id0=0, block_log2=0) -> np.ndarray:
    """eq. (4.1).  lam_: one amplitude, or [M, nb] per worker and block (then every worker is
    decoded with its own table and the decoded vectors are averaged)."""
    bits = _u32(bits)
    M = bits.shape[0]
    if np.ndim(lam_) == 2:
        total = np.zeros(padded_dim(d, block_log2))
        for n in range(M):
            total += decode_full(bits[n], d, seed, step, worker_id0 + n, lam_[n], 1, block_log2)
        return total / M
    out = np.empty(padded_dim(d, block_log2), np.float64)
    lib().fosgd_oracle_aggregate(_p(bits, C.c_uint32), d, M, worker_id0, seed, step, lam_,
                                 block_log2, _p(out, C.c_double))
    return out


def downlink_encode(gbar, seed, step, lam_s, K=1, block_log2=0, want_margin=False):
    return encode(gbar, seed, step, SERVER_ID, lam_s, K, block_log2, want_margin)


def downlink_decode(pl, dp, seed, step, lam_s, K=1, block_log2=0) -> np.ndarray:
    return decode_full(pl, dp, seed, step, SERVER_ID, lam_s, K, block_log2)


def unpack(words, n=None) -> np.ndarray:
    """Packed words -> 0/1 array (bit i of the vector = bit i&31 of word i>>5)."""
    w = _u32(words).reshape(-1)
    b = ((w[:, None] >> np.arange(32, dtype=np.uint32)[None, :]) & 1).astype(np.uint8).reshape(-1)
    return b if n is None else b[:n]
