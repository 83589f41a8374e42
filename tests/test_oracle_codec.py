"""Pins for the oracle's quantizer, encoder/decoder and server average: the closed forms of
the paper's appendix (Lemmas A.4-A.6, Cor. A.8), Remark 3.3 and Remark 5.2."""
import numpy as np
import pytest

import oracle


def preimage(y, seed, step, wid):
    """g with H D_eps g = y, from Def. 3.5: (H D_eps)^-1 = D_eps H^T."""
    n = y.size
    return oracle.eps_vector(seed, step, wid, n) * oracle.fwht(y) / np.sqrt(n)


def signs(bits_words, n):
    return 2.0 * oracle.unpack(bits_words, n) - 1.0


def test_sign_convention_and_saturation():
    # sgn(0) = +1: a zero vector quantizes to bit = (tau >= 0), and tau is never 0
    n, lam = 64, 0.5
    bits = oracle.encode(np.zeros(n), 1, 2, 3, lam)
    t = np.array([oracle.dither_t(1, 2, 3, 0, i) for i in range(n)])
    assert (oracle.unpack(bits, n) == (t > 0)).all()
    # entries beyond +-lambda saturate whatever the dither
    y = np.where(np.arange(n) % 2 == 0, 2.0 * lam, -2.0 * lam)
    for step in range(5):
        b = oracle.unpack(oracle.encode(preimage(y, 1, step, 3), 1, step, 3, lam), n)
        assert (b == (np.arange(n) % 2 == 0)).all()
    # y = +lambda exactly is always +1, y = -lambda exactly is always -1 (|tau| < lambda)
    y = np.where(np.arange(n) % 2 == 0, lam, -lam)
    for step in range(5):
        b, zm = oracle.encode(preimage(y, 1, step, 3), 1, step, 3, lam, want_margin=True)
        assert (oracle.unpack(b, n) == (np.arange(n) % 2 == 0)).all()
        assert (zm > 0).all()


def test_bit_layout():
    # bit i of the vector sits in word i>>5 at position i&31, 1 <=> +1
    n, lam = 128, 1.0
    y = np.full(n, -3.0)
    y[[0, 5, 31, 32, 100]] = 3.0
    w = oracle.encode(preimage(y, 4, 4, 4), 4, 4, 4, lam)[0]
    assert list(w) == [(1 << 0) | (1 << 5) | (1 << 31), 1 << 0, 0, 1 << 4]


def test_quantizer_mean_is_clip_and_mse_closed_form():
    # Lemma A.4: E Q(x) = clip(x, -lambda, lambda); for |x|_inf <= lambda,
    # E||Q(x) - x||^2 = (lambda^2 d - ||x||^2) / K.
    n, lam, T = 64, 1.0, 6000
    y = np.linspace(-1.6, 1.6, n)
    mean = np.zeros(n)
    for step in range(T):
        mean += lam * signs(oracle.encode(preimage(y, 11, step, 0), 11, step, 0, lam), n)
    mean /= T
    clip = np.clip(y, -lam, lam)
    sigma = np.sqrt(np.maximum(lam ** 2 - clip ** 2, 0) / T)
    assert (np.abs(mean - clip) <= 4.5 * sigma + 1e-12).all()
    inside = np.abs(y) > lam
    np.testing.assert_array_equal(mean[inside], clip[inside])     # saturated: no randomness
    # soft-threshold residual, statement 2
    resid = y - mean
    soft = np.sign(y) * np.maximum(np.abs(y) - lam, 0)
    assert (np.abs(resid - soft) <= 4.5 * sigma + 1e-12).all()

    yin = np.linspace(-0.9, 0.9, n)
    for K in (1, 3):
        acc = 0.0
        for step in range(T):
            pl = oracle.encode(preimage(yin, 12, step, 0), 12, step, 0, lam, K=K)
            c = sum(oracle.unpack(pl[p], n).astype(int) << p for p in range(pl.shape[0]))
            q = (lam / K) * (2 * c - K)
            acc += ((q - yin) ** 2).sum()
        expect = (lam ** 2 * n - (yin ** 2).sum()) / K
        assert abs(acc / T / expect - 1) < 0.03, (K, acc / T, expect)


def test_value_set_and_planes():
    # Remark 3.3: (K/lambda) Q in {-K, -K+2, ..., K}, log2(K+1) bits per entry
    assert [oracle.planes(K) for K in (1, 2, 3, 4, 7, 8, 15, 255)] == [1, 2, 2, 3, 3, 4, 4, 8]
    n = 256
    g = np.random.default_rng(0).standard_normal(n)
    lam = oracle.lam(np.linalg.norm(g), 2.0, n)
    for K in (1, 2, 3, 5, 7):
        pl = oracle.encode(g, 1, 1, 1, lam, K=K)
        c = sum(oracle.unpack(pl[p], n).astype(int) << p for p in range(pl.shape[0]))
        assert c.min() >= 0 and c.max() <= K
        # each dither separately reproduces the count
        y = oracle.flatten(g, 1, 1, 1)
        cc = np.zeros(n, int)
        for k in range(K):
            tau = lam * np.array([oracle.dither_t(1, 1, 1, k, i) for i in range(n)]) / 2.0 ** 24
            cc += (y + tau >= 0)
        assert (c == cc).all()


def test_inner_product_second_moment():
    # Lemma A.5: E<x, Q(y)>^2 = <x,y>^2 + ||x||^2 lambda^2 - sum x_i^2 y_i^2, |y|_inf <= lambda
    n, lam, T = 32, 1.0, 20000
    rng = np.random.default_rng(5)
    x = rng.standard_normal(n)
    y = rng.uniform(-0.9, 0.9, n)
    vals = np.empty(T)
    for step in range(T):
        q = lam * signs(oracle.encode(preimage(y, 21, step, 0), 21, step, 0, lam), n)
        vals[step] = (x @ q) ** 2
    expect = (x @ y) ** 2 + (x @ x) * lam ** 2 - (x ** 2 * y ** 2).sum()
    assert abs(vals.mean() - expect) < 4.5 * vals.std() / np.sqrt(T)


@pytest.mark.parametrize("block_log2", [0, 5])
def test_decoder_scale_exact_norm(block_log2):
    # Remark 5.2 with K = 1: ||D(q)|| = lambda sqrt(d') for ANY bit string
    d = 200
    dp = oracle.padded_dim(d, block_log2)
    rng = np.random.default_rng(2)
    bits = rng.integers(0, 2 ** 32, dp // 32, dtype=np.uint64).astype(np.uint32)
    lam = 0.37
    out = oracle.decode_full(bits, d, 1, 2, 3, lam, block_log2=block_log2)
    np.testing.assert_allclose(np.linalg.norm(out), lam * np.sqrt(dp), rtol=1e-13)
    # K > 1: bounded by lambda sqrt(d')
    pl = rng.integers(0, 2 ** 32, (2, dp // 32), dtype=np.uint64).astype(np.uint32)
    pl[1] &= ~pl[0]                                   # counts in {0,1,2} <= K = 3
    outk = oracle.decode_full(pl, d, 1, 2, 3, lam, K=3, block_log2=block_log2)
    assert np.linalg.norm(outk) <= lam * np.sqrt(dp) * (1 + 1e-13)


def test_decoder_is_inverse_basis_times_q():
    # D(q) = lambda D_eps H^T q, checked against the dense matrix
    n, lam = 64, 0.25
    rng = np.random.default_rng(3)
    bits = rng.integers(0, 2 ** 32, n // 32, dtype=np.uint64).astype(np.uint32)
    q = signs(bits, n)
    i = np.arange(n)
    H = np.where(np.array([[bin(a & b).count("1") & 1 for b in i] for a in i]), -1.0, 1.0) / 8.0
    e = oracle.eps_vector(6, 7, 8, n)
    np.testing.assert_allclose(oracle.decode_full(bits, n, 6, 7, 8, lam), lam * e * (H.T @ q),
                               atol=1e-14)


def test_composite_unbiased_and_mse():
    # Z = D o E (Def. 5.1).  In range: E Z(x) = x and E||Z(x) - x||^2 = lambda^2 d' - ||x||^2
    # (Lemma A.6 with A = (H_eps)^-1, ||A||_F^2 = d').  d is not a power of two on purpose.
    d, T = 100, 4000
    dp = oracle.padded_dim(d)
    g = np.random.default_rng(8).standard_normal(d)
    lam = oracle.lam(np.linalg.norm(g), 3.0, dp)      # alpha = 3: in range with margin
    mean = np.zeros(dp)
    mse = np.empty(T)
    for step in range(T):
        assert np.abs(oracle.flatten(g, 31, step, 0)).max() <= lam
        z = oracle.decode_full(oracle.encode(g, 31, step, 0, lam), d, 31, step, 0, lam)
        mean += z
        mse[step] = ((z[:d] - g) ** 2).sum() + (z[d:] ** 2).sum()
    mean /= T
    # each coordinate of Z is (lambda/sqrt(d')) times a sum of d' independent signs: std <= lambda
    assert np.abs(mean[:d] - g).max() < 5 * lam / np.sqrt(T)
    assert np.abs(mean[d:]).max() < 5 * lam / np.sqrt(T)
    expect = lam ** 2 * dp - (g ** 2).sum()
    assert abs(mse.mean() / expect - 1) < 5 * mse.std() / np.sqrt(T) / expect + 1e-3


def test_worker_average_variance():
    # Cor. A.8 (in-range event): E||(1/N) sum Z_n(x_n) - (1/N) sum x_n||^2
    #   = (1/N^2) sum_n (lambda^2 d' - ||x_n||^2); also ||gbar|| <= lambda sqrt(d').
    d, N, T = 64, 4, 1500
    rng = np.random.default_rng(9)
    xs = rng.standard_normal((N, d))
    lam = oracle.lam(np.linalg.norm(xs, axis=1).max(), 3.0, d)
    errs = np.empty(T)
    for step in range(T):
        bits = np.stack([oracle.encode(xs[n], 41, step, n, lam)[0] for n in range(N)])
        gbar = oracle.aggregate(bits, d, 41, step, lam)
        assert np.linalg.norm(gbar) <= lam * np.sqrt(d) * (1 + 1e-12)
        # aggregate is the plain mean of the per-worker decoders
        if step == 0:
            ref = np.mean([oracle.decode_full(bits[n], d, 41, 0, n, lam) for n in range(N)], axis=0)
            np.testing.assert_allclose(gbar, ref, atol=1e-14)
        errs[step] = ((gbar - xs.mean(0)) ** 2).sum()
    expect = sum(lam ** 2 * d - (xs[n] ** 2).sum() for n in range(N)) / N ** 2
    assert abs(errs.mean() / expect - 1) < 5 * errs.std() / np.sqrt(T) / expect


def test_downlink_roundtrip_error_scales_as_one_over_K():
    # Lemma A.4(3) through the composite: E||Z_{lambda_s,K}(p) - p||^2 = (lambda_s^2 d' - ||p||^2)/K
    d, T = 128, 1200
    p = np.random.default_rng(10).standard_normal(d) * 0.1
    lam_s = oracle.lam(np.linalg.norm(p), 3.0, d)
    for K in (1, 4):
        errs = np.empty(T)
        for step in range(T):
            pl = oracle.downlink_encode(p, 51, step, lam_s, K=K)
            out = oracle.downlink_decode(pl, d, 51, step, lam_s, K=K)
            errs[step] = ((out - p) ** 2).sum()
        expect = (lam_s ** 2 * d - (p ** 2).sum()) / K
        assert abs(errs.mean() / expect - 1) < 5 * errs.std() / np.sqrt(T) / expect + 1e-3
    # the server's flips and dithers are those of the reserved id
    pl = oracle.downlink_encode(p, 51, 0, lam_s, K=1)
    assert (pl == oracle.encode(p, 51, 0, oracle.SERVER_ID, lam_s)).all()


def test_margin_is_distance_to_decision():
    d = 96
    g = np.random.default_rng(11).standard_normal(d)
    lam = 0.5
    bits, zm = oracle.encode(g, 1, 1, 1, lam, want_margin=True)
    y = oracle.flatten(g, 1, 1, 1)
    tau = lam * np.array([oracle.dither_t(1, 1, 1, 0, i) for i in range(y.size)]) / 2.0 ** 24
    np.testing.assert_allclose(zm, np.abs(y + tau).astype(np.float32), rtol=1e-6)
    assert (oracle.unpack(bits, y.size) == (y + tau >= 0)).all()


def test_block_amplitude_tables_reduce_to_single_amplitude():
    """Per-block tables (blocked mode): a constant table is the single-amplitude codec bit for bit,
    and with distinct entries block k of the table codec equals block k of the single-amplitude
    codec run with that entry (the blocks' transforms are independent, Def. 3.7 / 3.8 per block)."""
    rng = np.random.default_rng(21)
    d, b, K, seed, step, wid = 1500, 8, 3, 11, 5, 2
    g = rng.standard_normal(d) * np.repeat(10.0 ** rng.uniform(-3, 0, 6), 256)[:d]
    dp = oracle.padded_dim(d, b)
    nb, n = dp >> b, 1 << b
    const = np.full(nb, 0.37)
    assert np.array_equal(oracle.encode(g, seed, step, wid, const, K=K, block_log2=b),
                          oracle.encode(g, seed, step, wid, 0.37, K=K, block_log2=b))
    tab = 10.0 ** rng.uniform(-2, 0, nb)
    pl, zm = oracle.encode(g, seed, step, wid, tab, K=K, block_log2=b, want_margin=True)
    dec = oracle.decode_full(pl, d, seed, step, wid, tab, K=K, block_log2=b)
    for k in range(nb):
        pk, zk = oracle.encode(g, seed, step, wid, float(tab[k]), K=K, block_log2=b, want_margin=True)
        w = slice(k * n // 32, (k + 1) * n // 32)
        assert np.array_equal(pl[:, w], pk[:, w])
        assert np.array_equal(zm[k * n:(k + 1) * n], zk[k * n:(k + 1) * n])
        dk = oracle.decode_full(pl, d, seed, step, wid, float(tab[k]), K=K, block_log2=b)
        assert np.array_equal(dec[k * n:(k + 1) * n], dk[k * n:(k + 1) * n])
    # Remark 5.2 per block (K = 1): the decoded block has norm exactly lambda_k sqrt(n)
    p1 = oracle.encode(g, seed, step, wid, tab, block_log2=b)
    d1 = oracle.decode_full(p1, d, seed, step, wid, tab, block_log2=b)
    np.testing.assert_allclose(np.linalg.norm(d1.reshape(nb, n), axis=1), tab * np.sqrt(n), rtol=1e-12)


def test_block_amplitude_law():
    """lam[n, k] is Theorem 5.5's law for the block's own norm and length; lam_s[k] follows the
    server law from the largest worker amplitude; a zero block is floored, not zero."""
    rng = np.random.default_rng(22)
    M, d, b = 3, 700, 7
    G = rng.standard_normal((M, d))
    G[:, 128:256] = 0.0
    lam, lam_s = oracle.block_amplitudes(G, 2.0, 3.0, b)
    n = 1 << b
    assert lam.shape == (M, 6) and lam_s.shape == (6,)
    for m in range(M):
        for k in (0, 2, 5):
            blk = G[m, k * n:(k + 1) * n]
            assert np.isclose(lam[m, k], oracle.lam(np.linalg.norm(blk), 2.0, n), rtol=1e-14)
    assert (lam[:, 1] == 1e-30).all()
    for k in range(6):
        assert np.isclose(lam_s[k], oracle.lam_server(lam[:, k].max(), 3.0, n), rtol=1e-14)
    # the flattening event of Lemma 3.6 per block: no transformed entry exceeds its block's lambda
    y = oracle.flatten(G[0], 1, 2, 0, block_log2=b).reshape(6, n)
    assert (np.abs(y).max(axis=1) <= lam[0] + 1e-300).all()


def _dense_h(n):
    i = np.arange(n)
    return np.where(np.array([[bin(a & b).count("1") & 1 for b in i] for a in i]), -1.0, 1.0) / np.sqrt(n)


@pytest.mark.parametrize("K", [1, 3])
def test_decode_entry_is_the_dense_matrix_row(K):
    # Def. 3.8 entry by entry: (lambda/K) eps_k sum_j H[k][j] (2 c_j - K), against the dense matrix
    # written out here and against the full decoder, in global and in blocked mode
    n, lam = 128, 0.75
    rng = np.random.default_rng(20 + K)
    P = oracle.planes(K)
    pl = rng.integers(0, 2 ** 32, (P, n // 32), dtype=np.uint64).astype(np.uint32)
    if P == 2:
        pl[1] &= ~pl[0] | rng.integers(0, 2 ** 32, n // 32, dtype=np.uint64).astype(np.uint32)   # counts 0..3
    c = sum(oracle.unpack(pl[p], n).astype(int) << p for p in range(P))
    q = 2.0 * c - K
    e = oracle.eps_vector(6, 7, 8, n)
    dense = lam / K * e * (_dense_h(n) @ q)
    full = oracle.decode_full(pl, n, 6, 7, 8, lam, K=K)
    for k in range(n):
        v = oracle.decode_entry(pl, n, 6, 7, 8, lam, k, K=K)
        assert abs(v - dense[k]) <= 1e-13
        assert abs(v - full[k]) <= 1e-13
    # blocked mode: the sum runs over the block of k only, d not a multiple of the block
    d, b = 200, 6
    dp = oracle.padded_dim(d, b)
    plb = rng.integers(0, 2 ** 32, (1, dp // 32), dtype=np.uint64).astype(np.uint32)
    fullb = oracle.decode_full(plb, d, 1, 2, 3, lam, block_log2=b)
    Hb = _dense_h(1 << b)
    eb = oracle.eps_vector(1, 2, 3, dp)
    qb = signs(plb[0], dp)
    for k in (0, 63, 64, 129, dp - 1):
        blk = k >> b
        ref = lam * eb[k] * (Hb[k & 63] @ qb[blk << b:(blk + 1) << b])
        v = oracle.decode_entry(plb, d, 1, 2, 3, lam, k, block_log2=b)
        assert abs(v - ref) <= 1e-13 and abs(v - fullb[k]) <= 1e-13


@pytest.mark.parametrize("split", [1, 4, 7, 9])
def test_grid_entries_match_full_transforms(split):
    # the product-grid functions (Kronecker split of the Sylvester matrix at `split` bits) against the
    # full transform, the single-entry functions and, for one small case, the dense matrix
    d, seed, step, wid = 700, 3, 4, 5
    dp = oracle.padded_dim(d)                         # 1024
    rng = np.random.default_rng(split)
    g = rng.standard_normal(d)
    k_hi = np.unique(np.concatenate([[0, (dp >> split) - 1], rng.integers(0, dp >> split, 5)]))
    k_lo = np.unique(np.concatenate([[0, (1 << split) - 1], rng.integers(0, 1 << split, 6)]))
    y = oracle.flatten(g, seed, step, wid)
    grid = oracle.flatten_grid(g, seed, step, wid, split, k_hi, k_lo)
    grid32 = oracle.flatten_grid(g.astype(np.float32), seed, step, wid, split, k_hi, k_lo)
    y32 = oracle.flatten(g.astype(np.float32).astype(np.float64), seed, step, wid)
    x = np.zeros(dp)
    x[:d] = g * oracle.eps_vector(seed, step, wid, d)
    dense = _dense_h(dp) @ x
    for a, kh in enumerate(k_hi):
        for b, kl in enumerate(k_lo):
            k = int(kh) * (1 << split) + int(kl)
            assert abs(grid[a, b] - y[k]) <= 1e-12
            assert abs(grid[a, b] - dense[k]) <= 1e-12
            assert abs(grid[a, b] - oracle.flatten_entry(g, seed, step, wid, k)) <= 1e-12
            assert abs(grid32[a, b] - y32[k]) <= 1e-12
    for K in (1, 7):
        P = oracle.planes(K)
        pl = rng.integers(0, 2 ** 32, (P, dp // 32), dtype=np.uint64).astype(np.uint32)
        lam = 0.3
        full = oracle.decode_full(pl, d, seed, step, wid, lam, K=K)
        gridd = oracle.decode_grid(pl, d, seed, step, wid, lam, split, k_hi, k_lo, K=K)
        for a, kh in enumerate(k_hi):
            for b, kl in enumerate(k_lo):
                k = int(kh) * (1 << split) + int(kl)
                assert abs(gridd[a, b] - full[k]) <= 1e-12
                assert abs(gridd[a, b] - oracle.decode_entry(pl, d, seed, step, wid, lam, k, K=K)) <= 1e-12


def test_k_dither_error_bound():
    # Lemma A.9: for ||x|| <= B, lambda = alpha B sqrt(log d / d), alpha >= 2,
    #   E||Z_{lambda,K}(x) - x||^2 <= alpha^2 B^2 log d / K + 8 B^2 exp(-alpha^2 log d / 8)
    # (expectation over eps and the K dithers: the step number draws both afresh)
    d, T, alpha = 256, 600, 2.0
    rng = np.random.default_rng(12)
    cases = [rng.standard_normal(d), np.eye(d)[17] * 3.0, np.where(rng.random(d) < 0.05, rng.standard_normal(d), 0.0)]
    for x in cases:
        B = np.linalg.norm(x)
        lam = oracle.lam(B, alpha, d)
        for K in (1, 3, 15):
            errs = np.empty(T)
            for step in range(T):
                pl = oracle.encode(x, 61, step, 9, lam, K=K)
                z = oracle.decode_full(pl, d, 61, step, 9, lam, K=K)
                errs[step] = ((z - x) ** 2).sum()
            bound = alpha ** 2 * B ** 2 * np.log(d) / K + 8 * B ** 2 * np.exp(-alpha ** 2 * np.log(d) / 8)
            assert errs.mean() + 5 * errs.std() / np.sqrt(T) <= bound
            # the first term is attained up to ||x||^2 / K when the flattened vector stays in range
            assert errs.mean() >= 0.5 * (lam ** 2 * d - B ** 2) / K
