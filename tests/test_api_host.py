"""Host-side behaviour of the C-ABI that needs no GPU: exported symbols, size helpers and the
argument checks (every rejected call returns before anything is enqueued)."""
import ctypes as C
import math
import os
import re

import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def F():
    import paper_2405_11095_b200 as f
    f.lib()
    return f


def test_every_declared_symbol_is_exported(F):
    header = open(os.path.join(ROOT, "include", "fosgd.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(fosgd_[a-z_0-9]+)\s*\(", header))
    assert {"fosgd_encode", "fosgd_decode", "fosgd_server_aggregate", "fosgd_downlink_decode"} <= declared
    lib = C.CDLL(os.path.join(ROOT, "paper_2405_11095_b200", "libfosgd.so"))
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(F.EXPORTS)


def test_size_helpers_agree_with_oracle(F):
    for d in (1, 31, 32, 33, 1000, 65536, 65537, 25_557_032, 1_315_819_520, 1 << 31):
        assert F.padded_dim(d) == oracle.padded_dim(d)
        for b in (5, 10, 20, 30):
            assert F.padded_dim(d, b) == oracle.padded_dim(d, b)
    assert F.padded_dim(0) == -1 and F.padded_dim((1 << 31) + 1) == -1 and F.padded_dim(100, 3) == -1
    assert F.padded_dim(100, 31) == -1
    for K in range(1, 256):
        assert F.planes(K) == oracle.planes(K)
    assert F.planes(0) == 0 and F.planes(256) == 0
    for d in (1 << 16, 1 << 24, 1 << 31):
        lam = F.lambda_(3.0, 2.0, d)
        assert math.isclose(lam, oracle.lam(3.0, 2.0, d), rel_tol=1e-6)
        assert math.isclose(F.lambda_server(lam, 2.5, d), oracle.lam_server(lam, 2.5, d), rel_tol=1e-6)


def test_workspace_sizes(F):
    assert F.workspace_bytes(F.OP_ENCODE, 1 << 15) == 0           # one tile: no scratch
    assert F.workspace_bytes(F.OP_ENCODE, (1 << 15) + 1) == 4 << 16
    assert F.workspace_bytes(F.OP_AGGREGATE, 1 << 24, M=32) == 4 << 24
    assert F.workspace_bytes(F.OP_DECODE, 25_557_032, block_log2=20) == 4 * (25 << 20)
    assert F.workspace_bytes(F.OP_DOWNLINK_DECODE, 1_315_819_520, K=7) == 4 << 31
    with pytest.raises(F.FosgdError) as e:
        F.workspace_bytes(19, 100)
    assert e.value.status == F.EUNSUPPORTED
    with pytest.raises(F.FosgdError) as e:
        F.workspace_bytes(F.OP_AGGREGATE, 100, K=300)
    assert e.value.status == F.EINVAL


def test_argument_checks_return_before_any_launch(F):
    L = F.lib()
    a = 1 << 20          # fake, 16-byte aligned "device" addresses: rejected calls never touch them
    enc = lambda **k: L.fosgd_encode(k.get("g", a), k.get("dt", 0), k.get("d", 1 << 16), k.get("ws_", 1 << 16),
                                     k.get("M", 2), 0, 1, 2, k.get("lam", 0.1), k.get("b", 0), k.get("bits", a),
                                     k.get("ws", None), k.get("wsb", 0), None)
    assert enc(g=None) == F.EINVAL
    assert enc(bits=None) == F.EINVAL
    assert enc(d=0) == F.EINVAL
    assert enc(M=0) == F.EINVAL
    assert enc(lam=0.0) == F.EINVAL and enc(lam=float("inf")) == F.EINVAL and enc(lam=-1.0) == F.EINVAL
    assert enc(b=4) == F.EINVAL and enc(b=31) == F.EINVAL
    assert enc(dt=7) == F.EUNSUPPORTED
    assert enc(g=a + 4) == F.EALIGN
    assert enc(ws_=(1 << 16) + 1) == F.EALIGN           # stride * 4 bytes not a multiple of 16
    assert enc(ws_=100) == F.EINVAL                      # workers overlap
    assert enc(d=(1 << 31) + 1, ws_=(1 << 31) + 4) == F.EUNSUPPORTED
    assert enc() == F.EWORKSPACE                         # 2^16 needs scratch
    assert enc(ws=a, wsb=1000) == F.EWORKSPACE
    assert enc(ws=a + 8, wsb=1 << 30) == F.EALIGN

    dec = lambda **k: L.fosgd_decode(k.get("bits", a), k.get("d", 1 << 16), 0, 1, 2, k.get("lam", 0.1), 0,
                                     k.get("out", a), None, 0, None)
    assert dec(bits=None) == F.EINVAL and dec(out=None) == F.EINVAL and dec(lam=float("nan")) == F.EINVAL
    assert dec(out=a + 4) == F.EALIGN
    assert dec() == F.EWORKSPACE

    agg = lambda **k: L.fosgd_server_aggregate(k.get("bits", a), 1 << 16, k.get("M", 2), 0, k.get("N", 2), 1, 2,
                                               0.1, 0, k.get("acc", a), k.get("flags", 3), k.get("lam_s", 0.2),
                                               k.get("K", 1), k.get("down", a), None, 0, None)
    assert agg(acc=None) == F.EINVAL
    assert agg(N=1) == F.EINVAL                           # fewer workers in total than in the chunk
    assert agg(flags=4) == F.EINVAL
    assert agg(K=0) == F.EINVAL and agg(K=256) == F.EINVAL and agg(lam_s=0.0) == F.EINVAL
    assert agg(K=0, down=None) == F.EWORKSPACE            # K is not read without a downlink buffer
    assert agg(K=0, flags=1) == F.EWORKSPACE              # ... nor before END
    assert agg() == F.EWORKSPACE

    dl = lambda **k: L.fosgd_downlink_decode(k.get("bits", a), 1 << 16, 1, 2, 0.2, k.get("K", 3), 0,
                                             k.get("out", a), None, 0, None)
    assert dl(K=0) == F.EINVAL and dl(bits=None) == F.EINVAL
    assert dl() == F.EWORKSPACE

    amp = lambda **k: L.fosgd_amplitudes(k.get("g", a), 0, 1 << 16, 1 << 16, k.get("M", 2), k.get("alpha", 2.0), 2.0,
                                         k.get("b", 0), k.get("pb", 0), k.get("out", a), a, k.get("ws", a),
                                         k.get("wsb", 1 << 20), None)
    assert amp(g=None) == F.EINVAL and amp(out=None) == F.EINVAL and amp(alpha=0.0) == F.EINVAL
    assert amp(ws=None) == F.EWORKSPACE and amp(wsb=100) == F.EWORKSPACE
    assert amp(pb=1) == F.EINVAL and amp(pb=2, b=10) == F.EINVAL      # a table needs the blocked mode
    assert amp(pb=1, b=10, wsb=2 * 64 * 8 - 1) == F.EWORKSPACE
    assert L.fosgd_encode_dev(a, 0, 1 << 16, 1 << 16, 2, 0, 1, 2, None, 0, 0, a, a, 1 << 30, None) == F.EINVAL
    assert L.fosgd_encode_dev(a, 0, 1 << 16, 1 << 16, 2, 0, 1, 2, a, 1, 0, a, a, 1 << 30, None) == F.EINVAL
    assert L.fosgd_server_aggregate_dev(a, 1 << 16, 2, 0, 2, 1, 2, None, a, 0, 0, a, 3, 1, a, a, 1 << 30, None) == F.EINVAL
    assert L.fosgd_server_aggregate_dev(a, 1 << 16, 2, 0, 2, 1, 2, a, None, 0, 0, a, 3, 1, a, a, 1 << 30, None) == F.EINVAL
    assert L.fosgd_downlink_decode_dev(a, 1 << 16, 1, 2, None, 0, 1, 0, a, a, 1 << 30, None) == F.EINVAL
    enc = lambda **k: L.fosgd_downlink_encode(k.get("g", a), 1 << 16, 1, 2, k.get("lam", 0.5), k.get("dev", None),
                                              k.get("pb", 0), k.get("K", 1), 0, k.get("out", a), a, 1 << 30, None)
    assert enc(g=None) == F.EINVAL and enc(out=None) == F.EINVAL and enc(K=0) == F.EINVAL
    assert enc(lam=0.0) == F.EINVAL and enc(pb=1) == F.EINVAL and enc(dev=a, pb=1) == F.EINVAL
    app = lambda **k: L.fosgd_downlink_apply(a, 1 << 16, 1, 2, k.get("lam", 0.5), None, 0, 1, 0, k.get("delta", 0.1),
                                             k.get("x", a), a, 1 << 30, None)
    assert app(delta=0.0) == F.EINVAL and app(delta=float("nan")) == F.EINVAL and app(x=None) == F.EINVAL
    assert app(lam=-1.0) == F.EINVAL
    assert F.workspace_bytes(F.OP_AMPLITUDES, 1 << 16, M=3) == 3 * 2048
    assert F.workspace_bytes(F.OP_BLOCK_AMPLITUDES, 1 << 16, M=3, block_log2=7) == 3 * 512 * 8
    assert F.workspace_bytes(F.OP_BLOCK_AMPLITUDES, 1 << 16, M=3, block_log2=12) == 3 * 64 * 8

    em = lambda **k: L.fosgd_encode_measured(k.get("g", a), k.get("dt", 0), 1 << 16, 1 << 16, k.get("M", 2), 0, 1, 2,
                                             k.get("alpha", 2.0), 2.0, 0, k.get("lam", a), a, k.get("bits", a),
                                             k.get("ws", a), k.get("wsb", 1 << 30), k.get("aws", a), k.get("awsb", 1 << 20), None)
    assert em(g=None) == F.EINVAL and em(lam=None) == F.EINVAL and em(bits=None) == F.EINVAL and em(alpha=-1.0) == F.EINVAL
    assert em(dt=5) == F.EUNSUPPORTED and em(bits=a + 4) == F.EALIGN and em(aws=a + 8) == F.EALIGN
    assert em(aws=None) == F.EWORKSPACE and em(awsb=2 * 2048 - 1) == F.EWORKSPACE
    assert em(ws=None, wsb=0) == F.EWORKSPACE and em(wsb=100) == F.EWORKSPACE
    assert L.fosgd_set_tensor_core_pass(L.fosgd_set_tensor_core_pass(0)) == 0        # (returns the previous mask; restored)
    assert L.fosgd_set_fused_encoder(L.fosgd_set_fused_encoder(1)) == 1

    assert L.fosgd_decode_noalloc(a, (1 << 20) + 1, 0, 1, 2, 0.1, 0, a, None) == F.ELIMIT
    assert L.fosgd_decode_noalloc(a, 0, 0, 1, 2, 0.1, 0, a, None) == F.EINVAL

    for st in (0, -1, -2, -3, -4, -5, -6):
        assert L.fosgd_strerror(st) and L.fosgd_strerror(st) != b"unknown status"
    assert L.fosgd_strerror(-99) == b"unknown status"
    assert L.fosgd_trace_passes(None, 0) == F.OK and L.fosgd_trace_count() == 0


def test_missing_library_fails_loudly(monkeypatch, F):
    monkeypatch.setattr(F, "_SO", os.path.join(ROOT, "no_such_dir", "libfosgd.so"))
    monkeypatch.setattr(F, "_handle", None)
    with pytest.raises(ImportError):
        F.padded_dim(10)
