"""Parity on the five benchmark workloads at full size, in the launch configuration bench.py
times (all workers of a config in one call where they fit).  Configs 0-3: every bit and every
averaged coordinate against the oracle.  Config 4 (d = 1.3e9, d' = 2^31): for workers 0, 1, 31 and
63, sampled transform outputs, uplink bits, entries of the 4-worker average, downlink planes and
downlink decoder outputs that the oracle computes from the matrix definition, plus properties
that hold at any size (norm preservation, Remark 5.2's exact norm)."""
import numpy as np
import pytest
import torch

import oracle
from parity import assert_bits_match, assert_l2_close, assert_transform_close, pmap, to_np_words

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def F():
    import paper_2405_11095_b200 as f
    return f


def full_round_trip(F, w, block_log2=0, K=None):
    from paper_2405_11095_b200 import synthetic
    K = w.K if K is None else K
    d, M = w.d, w.M
    seed, step = 20240511, 3
    stride = (d + 7) // 8 * 8
    grads = torch.zeros(M, stride, dtype=w.dtype, device=DEV)
    for n in range(M):
        synthetic.worker_gradient(w, n, DEV, out=grads[n, :d])
    dp = F.padded_dim(d, block_log2)
    n_eff = F.transform_len(d, block_log2)
    lam = F.lambda_(synthetic.norm_bound(grads[:, :d]), w.alpha, n_eff)
    lam_s = F.lambda_server(lam, w.alpha_s, n_eff)
    P = F.planes(K)
    ws_per = F.workspace_bytes(F.OP_AGGREGATE, d, block_log2=block_log2, K=K)
    ws = torch.empty(max(16, ws_per * M), dtype=torch.uint8, device=DEV)
    bits = torch.zeros(M, dp // 32, dtype=torch.int32, device=DEV)
    acc = torch.empty(dp, dtype=torch.float32, device=DEV)
    down = torch.zeros(P, dp // 32, dtype=torch.int32, device=DEV)
    out = torch.empty(d, dtype=torch.float32, device=DEV)
    F.encode(grads, d, bits, lam, seed, step, block_log2=block_log2, ws=ws, worker_stride=stride)
    F.server_aggregate(bits, d, acc, lam, seed, step, lam_s=lam_s, K=K, down_bits=down, block_log2=block_log2, ws=ws)
    F.downlink_decode(down, d, out, lam_s, seed, step, K=K, block_log2=block_log2, ws=ws)
    torch.cuda.synchronize()

    gh = grads[:, :d].cpu().double().numpy()
    gb = to_np_words(bits)

    def check_worker(n):
        ref, margin = oracle.encode(gh[n], seed, step, n, lam, block_log2=block_log2, want_margin=True)
        return assert_bits_match(gb[n][None], ref, margin, lam)

    ties = sum(pmap(check_worker, range(M)))
    gbar = np.zeros(dp)
    for part in pmap(lambda n: oracle.decode_full(gb[n], d, seed, step, n, lam, block_log2=block_log2), range(M)):
        gbar += part
    gbar /= M
    assert_l2_close(acc.cpu().numpy(), gbar)
    ref_down, margin = oracle.downlink_encode(gbar, seed, step, lam_s, K=K, block_log2=block_log2, want_margin=True)
    ties += assert_bits_match(to_np_words(down), ref_down, margin, lam_s, K=K)
    ref_out = oracle.downlink_decode(to_np_words(down), dp, seed, step, lam_s, K=K, block_log2=block_log2)
    assert_l2_close(out.cpu().numpy(), ref_out[:d])
    return ties


@pytest.mark.parametrize("cfg", [0, 1])
def test_config_small_full_round_trip(F, cfg):
    from paper_2405_11095_b200 import synthetic
    full_round_trip(F, synthetic.WORKLOADS[cfg])
    full_round_trip(F, synthetic.WORKLOADS[cfg], K=3)


def test_config2_sparse_full_round_trip(F):
    from paper_2405_11095_b200 import synthetic
    full_round_trip(F, synthetic.WORKLOADS[2])


@pytest.mark.parametrize("block_log2", [0, 20])
def test_config3_resnet50_full_round_trip(F, block_log2):
    from paper_2405_11095_b200 import synthetic
    full_round_trip(F, synthetic.WORKLOADS[3], block_log2=block_log2)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_two_strided_passes_2p26(F, dtype):
    # L = 26 is the smallest length that needs two strided passes; every output, bit and decoded
    # coordinate against the oracle, for both input types
    d, seed, step = (1 << 26) - 12345, 5, 6
    stride = d + 1 if dtype == torch.float32 else d + 1 + 8 - (d + 1) % 8
    g = torch.randn(1, stride, generator=torch.Generator(device=DEV).manual_seed(1), device=DEV).to(dtype)
    dp = F.padded_dim(d)
    ws = torch.empty(F.workspace_bytes(F.OP_ENCODE, d), dtype=torch.uint8, device=DEV)
    y = torch.empty(1, dp, dtype=torch.float32, device=DEV)
    F.flatten(g, d, y, seed, step, ws=ws, worker_stride=stride)
    gh = g[0, :d].cpu().double().numpy()
    lam = oracle.lam(float(np.linalg.norm(gh)), 2.0, dp)
    bits = torch.zeros(1, dp // 32, dtype=torch.int32, device=DEV)
    F.encode(g, d, bits, lam, seed, step, ws=ws, worker_stride=stride)
    out = torch.empty(d, dtype=torch.float32, device=DEV)
    F.decode(bits[0], d, out, lam, seed, step, 0, ws=ws)
    torch.cuda.synchronize()
    assert_transform_close(y[0].cpu().numpy(), oracle.flatten(gh, seed, step, 0))
    ref, margin = oracle.encode(gh, seed, step, 0, lam, want_margin=True)
    assert_bits_match(to_np_words(bits), ref, margin, lam)
    assert_l2_close(out.cpu().numpy(), oracle.decode_full(to_np_words(bits)[0], d, seed, step, 0, lam)[:d])


@pytest.mark.parametrize("dtype,d,ws_workers", [(torch.float32, (1 << 24) - 12345, 3), (torch.bfloat16, (1 << 23) + 5, 2),
                                                 (torch.float32, 1 << 24, 2)])
def test_encoder_2p24_batches_and_ragged_tails(F, dtype, d, ws_workers):
    # transforms of length 2^24 on several workers take the encoder whose two passes share one kernel:
    # a ragged last row of the strided view, rows that are padding only, both input types, and a scratch
    # buffer that holds fewer workers than the call (batches), every bit against the oracle
    M, seed, step, id0 = 3, 909, 12, 40
    stride = (d + 7) // 8 * 8
    g = torch.zeros(M, stride, dtype=dtype, device=DEV)
    g[:, :d] = torch.randn(M, d, generator=torch.Generator(device=DEV).manual_seed(d % 1000), device=DEV).to(dtype)
    dp = F.padded_dim(d)
    assert dp == 1 << 24
    ws = torch.empty(F.workspace_bytes(F.OP_ENCODE, d) * ws_workers, dtype=torch.uint8, device=DEV)
    gh = g[:, :d].cpu().double().numpy()
    lam = oracle.lam(float(np.linalg.norm(gh, axis=1).max()), 2.0, dp)
    bits = torch.zeros(M, dp // 32, dtype=torch.int32, device=DEV)
    F.encode(g, d, bits, lam, seed, step, worker_id0=id0, ws=ws, worker_stride=stride)
    torch.cuda.synchronize()
    gb = to_np_words(bits)

    def check(n):
        ref, margin = oracle.encode(gh[n], seed, step, id0 + n, lam, want_margin=True)
        return assert_bits_match(gb[n][None], ref, margin, lam)

    pmap(check, range(M))
    assert F.async_timeouts() == 0


# ---- config 4 (d = 1.3e9, bf16, 64 workers): sampled coordinates at full size --------------------
CFG4_WORKERS = (0, 1, 31, 63)
GRID_SPLIT = 12          # global mode: samples k = k_hi * 2^12 + k_lo


def cfg4_sample_grid(dp, rng):
    """Global mode (d' = 2^31, passes over index bits [0,11), [11,21), [21,31)): a product grid of
    32 x 16 = 512 coordinates.  k_lo takes every value of the low five bits (the lane / packed-bit
    position) once, with bits 5..11 running through all-zero, all-one (both ends of a contiguous
    tile), single bits and random patterns; k_hi does the same for the bits of the two strided
    passes."""
    low5 = rng.permutation(32)
    mid7 = np.concatenate([[0, 127, 63, 64, 1, 2, 4, 8, 16, 32], rng.integers(0, 128, 22)])
    k_lo = (mid7 << 5) | low5
    nhi = dp >> GRID_SPLIT
    k_hi = np.concatenate([[0, nhi - 1, 1, nhi >> 1, (nhi >> 1) - 1, 1 << 9, (1 << 9) - 1, 1 << 8],
                           rng.integers(0, nhi, 8)])
    return k_hi.astype(np.int64), k_lo.astype(np.int64)


def grid_in_threads(fn, k_hi, k_lo, parts=4):
    """fn(k_hi, k_lo_part) -> [n_hi, len(part)], the k_lo set cut into parts that run side by side."""
    cols = pmap(lambda c: fn(k_hi, c), np.array_split(k_lo, parts))
    return np.concatenate(cols, axis=1)


def assert_sampled_bits(words, ks, y_ref, lam, seed, step, wid, K=1, plane_words=None):
    """Bits (K = 1) or count planes of the sampled coordinates against sign(y + tau_k), wherever the
    oracle's decision is not inside the tie band."""
    ties = 0
    for idx, (k, yr) in enumerate(zip(ks, y_ref)):
        zs = [yr + lam * oracle.dither_t(seed, step, wid, kk, int(k)) / 2.0 ** 24 for kk in range(K)]
        if min(abs(z) for z in zs) <= 1e-5 * lam:
            ties += 1
            continue
        c = sum(1 for z in zs if z >= 0)
        got = sum(((int(words[p][idx]) >> (int(k) & 31)) & 1) << p for p in range(len(words)))
        assert got == c, (int(k), got, c)
    assert ties <= max(2, len(ks) // 100)
    return ties


@pytest.mark.parametrize("block_log2", [0, 20])
def test_config4_bf16_1p3B_sampled(F, block_log2):
    """Config 4 at full size: the transform, the uplink bits, the 4-worker server average, the downlink
    planes and the downlink decoder, each on 512 coordinates per worker that the oracle computes from
    the matrix definition (global mode: on a product grid; blocked mode: entry by entry), plus the
    properties that hold at any size."""
    from paper_2405_11095_b200 import synthetic
    w = synthetic.WORKLOADS[4]
    d, seed, step, K = w.d, 77, 1, w.K
    b = block_log2
    dp = F.padded_dim(d, b)
    n_eff = F.transform_len(d, b)
    P = F.planes(K)
    ws = torch.empty(F.workspace_bytes(F.OP_AGGREGATE, d, block_log2=b), dtype=torch.uint8, device=DEV)
    g = torch.empty(1, d, dtype=torch.bfloat16, device=DEV)
    y = torch.empty(1, dp, dtype=torch.float32, device=DEV)
    bits = torch.zeros(len(CFG4_WORKERS), dp // 32, dtype=torch.int32, device=DEV)
    rng = np.random.default_rng(4 + b)
    if b == 0:
        k_hi, k_lo = cfg4_sample_grid(dp, rng)
        ks = (k_hi[:, None] * (1 << GRID_SPLIT) + k_lo[None, :]).reshape(-1)
    else:
        blk = 1 << b
        ks = np.concatenate([rng.integers(0, dp, 480), [0, 31, 32, 1023, 1024, blk - 1, blk, dp - blk, dp - 1],
                             (dp - blk) + rng.integers(0, blk, 23)]).astype(np.int64)
    ks_dev = torch.from_numpy(ks).to(DEV)
    lam = None
    for slot, n in enumerate(CFG4_WORKERS):
        synthetic.worker_gradient(w, n, DEV, out=g[0])
        norm = float(g.double().norm())
        if lam is None:
            lam = F.lambda_(1.05 * norm, w.alpha, n_eff)      # an a-priori bound, same for all workers
        F.flatten(g, d, y, seed, step, worker_id0=n, block_log2=b, ws=ws)
        F.encode(g, d, bits[slot:slot + 1], lam, seed, step, worker_id0=n, block_log2=b, ws=ws)
        torch.cuda.synchronize()
        # property at full size: H D_eps is orthonormal
        assert abs(float(y.double().norm()) / norm - 1) < 1e-5
        yv = y[0, ks_dev].cpu().double().numpy()
        wv = to_np_words(bits[slot, ks_dev >> 5])
        scale = float(y.abs().max())
        gh = g[0].float().cpu().numpy()                       # bf16 -> fp32 is exact
        if b == 0:
            ref = grid_in_threads(lambda hi, lo: oracle.flatten_grid(gh, seed, step, n, GRID_SPLIT, hi, lo),
                                  k_hi, k_lo).reshape(-1)
        else:
            gd = gh.astype(np.float64)
            ref = np.array(pmap(lambda k: oracle.flatten_entry(gd, seed, step, n, int(k), block_log2=b), ks))
            del gd
        del gh
        assert np.abs(yv - ref).max() <= 1e-5 * scale
        assert np.linalg.norm(yv - ref) <= 1e-5 * np.linalg.norm(ref)
        assert_sampled_bits([wv], ks, ref, lam, seed, step, n)
    del y, g

    # ---- server: the four workers in three chunks into one accumulator, then the downlink encoder ----
    lam_s = F.lambda_server(lam, w.alpha_s, n_eff)
    acc = torch.empty(dp, dtype=torch.float32, device=DEV)
    down = torch.zeros(P, dp // 32, dtype=torch.int32, device=DEV)
    N = len(CFG4_WORKERS)
    F.server_aggregate(bits[0:2], d, acc, lam, seed, step, N_total=N, worker_id0=0, flags=F.AGG_BEGIN,
                       block_log2=b, ws=ws)
    F.server_aggregate(bits[2:3], d, acc, lam, seed, step, N_total=N, worker_id0=31, flags=0, block_log2=b, ws=ws)
    F.server_aggregate(bits[3:4], d, acc, lam, seed, step, N_total=N, worker_id0=63, flags=F.AGG_END,
                       lam_s=lam_s, K=K, down_bits=down, block_log2=b, ws=ws)
    out = torch.empty(d, dtype=torch.float32, device=DEV)
    F.downlink_decode(down, d, out, lam_s, seed, step, K=K, block_log2=b, ws=ws)
    torch.cuda.synchronize()
    # ||gbar|| <= lambda sqrt(d') (Remark 5.2 and the triangle inequality)
    assert float(acc.double().norm()) <= lam * np.sqrt(dp) * (1 + 1e-5)
    bw = to_np_words(bits)
    if b == 0:
        parts = [grid_in_threads(lambda hi, lo, s=slot, n=n: oracle.decode_grid(bw[s], d, seed, step, n, lam,
                                                                                GRID_SPLIT, hi, lo), k_hi, k_lo, parts=2)
                 for slot, n in enumerate(CFG4_WORKERS)]
        gbar_ref = np.mean(parts, axis=0).reshape(-1)
    else:
        gbar_ref = np.mean([pmap(lambda k, s=slot, n=n: oracle.decode_entry(bw[s], d, seed, step, n, lam, int(k),
                                                                            block_log2=b), ks)
                            for slot, n in enumerate(CFG4_WORKERS)], axis=0)
    accv = acc[ks_dev].cpu().double().numpy()
    assert np.linalg.norm(accv - gbar_ref) <= 1e-5 * np.linalg.norm(gbar_ref)
    assert np.abs(accv - gbar_ref).max() <= 1e-5 * np.abs(gbar_ref).max()
    del bw

    # downlink planes: the oracle's transform of the accumulator the GPU holds (the encoder's input)
    acch = acc.cpu().numpy()
    if b == 0:
        ys = grid_in_threads(lambda hi, lo: oracle.flatten_grid(acch, seed, step, oracle.SERVER_ID, GRID_SPLIT, hi, lo),
                             k_hi, k_lo).reshape(-1)
    else:
        accd = acch.astype(np.float64)
        ys = np.array(pmap(lambda k: oracle.flatten_entry(accd, seed, step, oracle.SERVER_ID, int(k), block_log2=b), ks))
        del accd
    del acch
    dwords = [to_np_words(down[p, ks_dev >> 5]) for p in range(P)]
    assert_sampled_bits(dwords, ks, ys, lam_s, seed, step, oracle.SERVER_ID, K=K)

    # downlink decoder on the planes the GPU produced, coordinates below d
    dw = to_np_words(down)
    keep = ks < d
    if b == 0:
        ref_out = grid_in_threads(lambda hi, lo: oracle.decode_grid(dw, dp, seed, step, oracle.SERVER_ID, lam_s,
                                                                    GRID_SPLIT, hi, lo, K=K), k_hi, k_lo).reshape(-1)[keep]
    else:
        ref_out = np.array(pmap(lambda k: oracle.decode_entry(dw, dp, seed, step, oracle.SERVER_ID, lam_s, int(k),
                                                              K=K, block_log2=b), ks[keep]))
    outv = out[ks_dev[torch.from_numpy(keep).to(DEV)]].cpu().double().numpy()
    assert keep.sum() >= 200
    assert np.linalg.norm(outv - ref_out) <= 1e-5 * np.linalg.norm(ref_out)
    # the decoded average is an unbiased estimate of the mean gradient: <Z, x> / ||x||^2 ~ 1 for worker 63
    g = torch.empty(d, dtype=torch.bfloat16, device=DEV)
    synthetic.worker_gradient(w, CFG4_WORKERS[-1], DEV, out=g)
    x = g.double()
    one = torch.empty(dp, dtype=torch.float32, device=DEV)
    F.server_aggregate(bits[3:4], d, one, lam, seed, step, N_total=1, worker_id0=63, block_log2=b, ws=ws)
    torch.cuda.synchronize()
    assert abs(float(one.double().norm()) / (lam * np.sqrt(dp)) - 1) < 1e-5      # Remark 5.2: ||D(q)|| = lambda sqrt(d')
    ratio = float((one[:d].double() * x).sum() / (x * x).sum())
    assert abs(ratio - 1) < 0.05
    if b == 0:
        # the same decoder with 6 bytes of scratch per coordinate: first strided pass in fp16 (on the tensor cores),
        # second one fp16 -> fp32; all values are exact integers up to the final scale, so nothing may differ
        del x, g
        ws6 = torch.empty(ws.numel() * 3 // 2, dtype=torch.uint8, device=DEV)
        two = torch.empty(dp, dtype=torch.float32, device=DEV)
        with F.PassTrace() as tr:
            F.server_aggregate(bits[3:4], d, two, lam, seed, step, N_total=1, worker_id0=63, block_log2=b, ws=ws6)
        torch.cuda.synchronize()
        assert any("ws16->ws" in lab for lab in tr.labels), tr.labels
        assert torch.equal(one, two)


def test_no_bounded_wait_gave_up(F):
    # the streaming kernels poll their tile copies a bounded number of times; none may have run out
    assert F.async_timeouts() == 0


@pytest.mark.parametrize("cfg,block_log2", [(1, 0), (2, 0), (3, 0), (3, 20)])
def test_tensor_core_pass_matches_plain_alu_pass(F, cfg, block_log2):
    """The strided decode pass from packed bits on the tensor cores (H_8 on packed bytes + 8-bit integer
    products for H_128) against the oracle through the whole server side, and bit for bit against the
    plain-ALU kernel's accumulator."""
    from paper_2405_11095_b200 import synthetic
    w = synthetic.WORKLOADS[cfg]
    M = min(w.M, 4)
    d, seed, step = w.d, 31, 7
    dp = F.padded_dim(d, block_log2)
    n_eff = F.transform_len(d, block_log2)
    rng = np.random.default_rng(cfg)
    words = rng.integers(0, 2 ** 32, (M, dp // 32), dtype=np.uint64).astype(np.uint32)
    words[0, : dp // 64] = 0xFFFFFFFF            # long runs of equal signs: the extreme values of the small factors
    words[1, dp // 64:] = 0
    bits = torch.from_numpy(words.view(np.int32)).to(DEV)
    lam = 0.37
    ws = torch.empty(F.workspace_bytes(F.OP_AGGREGATE, d, block_log2=block_log2) * M, dtype=torch.uint8, device=DEV)
    acc = {}
    for mask in (0, F.TC_STRIDED, F.TC_CONTIGUOUS, F.TC_STRIDED | F.TC_CONTIGUOUS, F.TC_STRIDED | F.TC_CONTIGUOUS | F.TC_ANY_SIZE):
        prev = F.set_tensor_core_pass(mask)
        try:
            a = torch.empty(dp, dtype=torch.float32, device=DEV)
            with F.PassTrace() as tr:
                F.server_aggregate(bits, d, a, lam, seed, step, block_log2=block_log2, ws=ws)
            torch.cuda.synchronize()
            acc[mask] = a
            # the kernels asked for are the ones that ran (the strided one needs 256 tiles of 2^17 to be chosen,
            # the contiguous one tiles of 2^14: transform length 2^24)
            ran_strided = any(lab.startswith("tc10") for lab in tr.labels)
            ran_contiguous = any(lab.startswith("tcrow") for lab in tr.labels)
            anysz = bool(mask & F.TC_ANY_SIZE)
            assert ran_strided == (bool(mask & F.TC_STRIDED) and (anysz or (dp >> 17) * M >= 256)), tr.labels
            assert ran_contiguous == (bool(mask & F.TC_CONTIGUOUS) and n_eff == 1 << 24 and (anysz or M >= 3)), tr.labels
        finally:
            F.set_tensor_core_pass(prev)
    for mask in acc:
        assert torch.equal(acc[mask], acc[0]), mask
    gbar = np.zeros(dp)
    for part in pmap(lambda n: oracle.decode_full(words[n], d, seed, step, n, lam, block_log2=block_log2), range(M)):
        gbar += part
    assert_l2_close(acc[F.TC_CONTIGUOUS].cpu().numpy(), gbar / M)
    assert F.async_timeouts() == 0


def test_tensor_core_contiguous_pass_sinks(F):
    """The contiguous decode pass on the tensor cores (H_128 as an fp16 product, the other seven stages on the
    plain ALUs) in every form of its sink: a decoder that returns d < d' coordinates, chunked aggregation
    (begin / add / end), per-worker amplitudes read on the device, and the update x <- x - step * D(q): each bit
    for bit against the plain-ALU pass (all values are exact integers until the final scale), the first also
    against the oracle."""
    d, seed, step, M = (1 << 24) - 70_001, 17, 4, 3
    dp = F.padded_dim(d)
    rng = np.random.default_rng(3)
    words = rng.integers(0, 2 ** 32, (M, dp // 32), dtype=np.uint64).astype(np.uint32)
    bits = torch.from_numpy(words.view(np.int32)).to(DEV)
    ws = torch.empty(F.workspace_bytes(F.OP_AGGREGATE, d) * 2, dtype=torch.uint8, device=DEV)
    lam, lam_s = 0.21, 1.7
    amp = torch.tensor([[0.5], [1.25], [3.0]], dtype=torch.float32, device=DEV)   # one block of 2^24 per worker
    amp_s = torch.tensor([0.75], dtype=torch.float32, device=DEV)
    x0 = torch.randn(d, generator=torch.Generator(device=DEV).manual_seed(1), device=DEV)
    res = {}
    TC = F.TC_CONTIGUOUS | F.TC_ANY_SIZE      # also for the one- and two-worker launches below
    for mask in (0, TC):
        prev = F.set_tensor_core_pass(mask)
        try:
            one = torch.full((d + 64,), 7.0, dtype=torch.float32, device=DEV)
            F.decode(bits[1], d, one, lam, seed, step, 1, ws=ws)
            acc = torch.empty(dp, dtype=torch.float32, device=DEV)
            F.server_aggregate(bits[:2], d, acc, lam, seed, step, N_total=M, flags=F.AGG_BEGIN, ws=ws)
            F.server_aggregate(bits[2:], d, acc, lam, seed, step, N_total=M, worker_id0=2, flags=F.AGG_END, ws=ws)
            accw = torch.empty(dp, dtype=torch.float32, device=DEV)
            F.server_aggregate_dev(bits, d, accw, amp, seed, step, lam_s=amp_s, block_log2=24, per_block=True, ws=ws)
            x = x0.clone()
            F.downlink_apply(bits[0], d, x, lam_s, seed, step, 0.125, ws=ws)
            torch.cuda.synchronize()
            res[mask] = (one, acc, accw, x)
        finally:
            F.set_tensor_core_pass(prev)
    for a, b in zip(res[0], res[TC]):
        assert torch.equal(a, b)
    one = res[TC][0]
    assert bool((one[d:] == 7.0).all())                       # nothing written beyond the d outputs
    assert_l2_close(one[:d].cpu().numpy(), oracle.decode_full(words[1], d, seed, step, 1, lam)[:d])
    assert F.async_timeouts() == 0


@pytest.mark.parametrize("d,M,ws_workers,extra", [
    (1 << 24, 3, 3, True),                 # one launch, progress words behind the intermediates
    (1 << 24, 3, 3, False),                # scratch for exactly three workers: launches of two and one
    ((1 << 24) - 70_001, 5, 2, True),      # ragged length (a partial last row of the strided view), three launches
    ((1 << 23) + 5, 2, 2, True),           # mostly padding
])
def test_fused_encoder_matches_two_kernel_encoder(F, d, M, ws_workers, extra):
    """The one-kernel uplink encoder of a 2^24-long transform (strided and contiguous pass side by side in
    every block) against the oracle on one worker, and word for word against the same encoder run as two
    kernels."""
    seed, step = 5, 9
    dp = F.padded_dim(d)
    assert dp == 1 << 24
    stride = (d + 7) // 8 * 8
    g = torch.Generator(device=DEV).manual_seed(d % 1000 + M)
    grads = torch.randn(M, stride, generator=g, device=DEV) * torch.rand(M, 1, generator=g, device=DEV)
    lam = F.lambda_(float(grads[:, :d].double().norm(dim=1).max()), 2.0, dp)
    nbytes = F.workspace_bytes(F.OP_ENCODE, d) * ws_workers + (F.fused_sync_bytes(ws_workers) if extra else 0)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
    out = {}
    for on in (True, False):
        prev = F.set_fused_encoder(on)
        try:
            bits = torch.zeros(M, dp // 32, dtype=torch.int32, device=DEV)
            with F.PassTrace() as tr:
                F.encode(grads, d, bits, lam, seed, step, ws=ws, worker_stride=stride, worker_id0=2)
            torch.cuda.synchronize()
            assert any(lab.startswith("fused") for lab in tr.labels) == on, tr.labels
            out[on] = bits
        finally:
            F.set_fused_encoder(prev)
    assert torch.equal(out[True], out[False])
    assert F.async_timeouts() == 0
    n = M - 1
    ref, margin = oracle.encode(grads[n, :d].cpu().double().numpy(), seed, step, 2 + n, lam, want_margin=True)
    assert_bits_match(to_np_words(out[True][n])[None], ref, margin, lam)


@pytest.mark.parametrize("d,M,b,dtype", [
    ((1 << 24) - 70_001, 3, 0, torch.float32),     # strided pass carries the sums (one read of the gradients)
    (1 << 20, 5, 0, torch.float32),
    (3 * (1 << 20) + 5, 2, 20, torch.float32),     # blocked mode, one amplitude for all workers and blocks
    ((1 << 16) + 3, 3, 0, torch.float32),          # nine strided stages: the two calls one after the other
    (1 << 20, 2, 0, torch.bfloat16),               # bf16: likewise
])
def test_encode_measured_equals_amplitudes_then_encode(F, d, M, b, dtype):
    """fosgd_encode_measured against fosgd_amplitudes + fosgd_encode_dev: the same amplitudes (to the last bits:
    the sums are taken in another order), the same packed words for the amplitude it wrote, and those words
    against the oracle."""
    seed, step = 77, 5
    dp = F.padded_dim(d, b)
    stride = (d + 7) // 8 * 8
    g = torch.Generator(device=DEV).manual_seed(d % 997 + M)
    grads = (torch.randn(M, stride, generator=g, device=DEV) * (1 + torch.arange(M, device=DEV)[:, None])).to(dtype)
    ws = torch.empty(max(16, F.workspace_bytes(F.OP_ENCODE, d, block_log2=b) * M), dtype=torch.uint8, device=DEV)
    amp_ws = torch.empty(F.workspace_bytes(F.OP_AMPLITUDES, d, M=M, block_log2=b), dtype=torch.uint8, device=DEV)
    lam1, lam_s1 = torch.zeros(1, device=DEV), torch.zeros(1, device=DEV)
    lam2, lam_s2 = torch.zeros(1, device=DEV), torch.zeros(1, device=DEV)
    bits1 = torch.zeros(M, dp // 32, dtype=torch.int32, device=DEV)
    bits2 = torch.zeros(M, dp // 32, dtype=torch.int32, device=DEV)
    F.encode_measured(grads, d, bits1, lam1, lam_s1, seed, step, alpha=2.0, alpha_s=3.0, worker_id0=4, block_log2=b, ws=ws,
                      amp_ws=amp_ws, worker_stride=stride)
    F.amplitudes(grads, d, lam2, lam_s2, alpha=2.0, alpha_s=3.0, block_log2=b, ws=amp_ws, worker_stride=stride)
    F.encode_dev(grads, d, bits2, lam1, seed, step, worker_id0=4, block_log2=b, ws=ws, worker_stride=stride)
    torch.cuda.synchronize()
    assert abs(lam1.item() / lam2.item() - 1) < 1e-6 and abs(lam_s1.item() / lam_s2.item() - 1) < 1e-6
    n_eff = F.transform_len(d, b)
    x = grads[:, :d].double()
    lam_ref = 2.0 * float(x.norm(dim=1).max()) * np.sqrt(np.log(n_eff) / n_eff)
    assert abs(lam1.item() / lam_ref - 1) < 1e-6
    assert torch.equal(bits1, bits2)
    n = M - 1
    ref, margin = oracle.encode(x[n].cpu().numpy(), seed, step, 4 + n, lam1.item(), block_log2=b, want_margin=True)
    assert_bits_match(to_np_words(bits1[n])[None], ref, margin, lam1.item())
    assert F.async_timeouts() == 0


def test_long_decoder_with_fp16_first_pass(F):
    """A decoder with two strided passes (transform length 2^26): where the scratch holds 6 instead of 4 bytes per
    coordinate for at least one worker, its first pass keeps its (exact) output in fp16.  Bit for bit against the fp32 route,
    and against the oracle."""
    d, seed, step, M = (1 << 26) - 12_345, 3, 8, 3
    dp = F.padded_dim(d)
    rng = np.random.default_rng(26)
    words = rng.integers(0, 2 ** 32, (M, dp // 32), dtype=np.uint64).astype(np.uint32)
    words[0, : dp // 64] = 0xFFFFFFFF
    bits = torch.from_numpy(words.view(np.int32)).to(DEV)
    lam = 0.83
    per = F.workspace_bytes(F.OP_AGGREGATE, d)
    acc = {}
    # scratch for one worker in fp32 only: worker by worker on the fp32 route; 1.5 x M workers: all three at once
    for name, nbytes in (("fp32", per), ("fp16 first", per * M * 3 // 2)):
        ws = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
        a = torch.empty(dp, dtype=torch.float32, device=DEV)
        with F.PassTrace() as tr:
            F.server_aggregate(bits, d, a, lam, seed, step, ws=ws)
        torch.cuda.synchronize()
        assert any("ws16->ws" in lab for lab in tr.labels) == (name == "fp16 first"), tr.labels
        acc[name] = a
        del ws
    assert torch.equal(acc["fp32"], acc["fp16 first"])
    gbar = np.zeros(dp)
    for part in pmap(lambda n: oracle.decode_full(words[n], d, seed, step, n, lam), range(M)):
        gbar += part
    assert_l2_close(acc["fp16 first"].cpu().numpy(), gbar / M)
    assert F.async_timeouts() == 0
