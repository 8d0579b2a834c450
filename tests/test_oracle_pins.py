"""Pins for the CPU oracle: each test ties a part of it to something other than
itself -- a value the paper prints, a closed form, brute force on tiny inputs,
a library routine for a special case, or an invariant of the mathematics."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import zipcache_oracle as zo

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.RandomState(seed)


# ---------------------------------------------------------------- Eq. 8 / 9
def _brute_force_causal_attention(Q, K):
    """l x l causal softmax attention with pure Python loops (Eq. 2 + mask)."""
    l, d = K.shape
    A = [[0.0] * l for _ in range(l)]
    for i in range(l):
        logits = []
        for j in range(i + 1):
            acc = 0.0
            for c in range(d):
                acc += float(Q[i, c]) * float(K[j, c])
            logits.append(acc / math.sqrt(d))
        mx = max(logits)
        es = [math.exp(v - mx) for v in logits]
        tot = sum(es)
        for j in range(i + 1):
            A[i][j] = es[j] / tot
    return A


@pytest.mark.parametrize("l,d,seed", [(1, 4, 0), (2, 4, 1), (17, 8, 2), (24, 16, 3)])
def test_normalized_score_matches_brute_force_full_matrix(l, d, seed):
    """Eq. 8 on the explicit l x l lower-triangular matrix (all tokens probes)."""
    rs = _rng(seed)
    Q = rs.standard_normal((l, d))
    K = rs.standard_normal((l, d))
    A = _brute_force_causal_attention(Q, K)
    expect = []
    for j in range(l):
        col = [A[i][j] for i in range(l)]
        nnz = sum(1 for i in range(l) if i >= j)      # lower triangle incl. diagonal
        expect.append(sum(col) / nnz)
    got = zo.normalized_scores(Q[None], K, np.arange(l))
    np.testing.assert_allclose(got, np.asarray(expect), rtol=1e-12, atol=0)


def test_probe_subset_matches_brute_force_rows():
    """Eq. 9 substituted into Eq. 8 with a strict subset of rows."""
    l, d = 20, 8
    rs = _rng(5)
    Q = rs.standard_normal((l, d))
    K = rs.standard_normal((l, d))
    P = [3, 7, 8, 15, 19]
    A = _brute_force_causal_attention(Q, K)
    expect = np.zeros(l)
    for j in range(l):
        rows = [p for p in P if p >= j]
        expect[j] = sum(A[p][j] for p in rows) / len(rows)
    got = zo.normalized_scores(Q[None], K, P)
    np.testing.assert_allclose(got, expect, rtol=1e-12)


def test_zero_query_closed_form_harmonic():
    """Q = 0 makes row r uniform over r+1 columns, so with all rows probes
    p~_j = (H_l - H_j) / (l - j) and the accumulated score is H_l - H_j."""
    l, d = 40, 8
    K = _rng(7).standard_normal((l, d))
    Q = np.zeros((1, l, d))
    H = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, l + 1))])
    j = np.arange(l)
    expect = (H[l] - H[j]) / (l - j)
    got = zo.normalized_scores(Q, K, np.arange(l))
    np.testing.assert_allclose(got, expect, rtol=1e-13)
    acc = zo.accumulated_scores([zo.probe_attention(Q[0], K, np.arange(l))])
    np.testing.assert_allclose(acc, H[l] - H[j], rtol=1e-13)
    # the bias the paper describes (Sec. 4.2): first token's accumulated score
    # exceeds 1 and always exceeds the last token's
    assert acc[0] > 1.0 and acc[0] > acc[-1]
    assert abs(acc[-1] - 1.0 / l) < 1e-15


def test_probe_attention_invariants_and_gqa_reduction():
    l, d, G = 33, 16, 4
    rs = _rng(11)
    Q = rs.standard_normal((G, l, d))
    K = rs.standard_normal((l, d))
    P = zo.probe_positions(l, 0.2, 0.2, 99)
    assert P[-1] == l - 1
    As = [zo.probe_attention(Q[g][P], K, P) for g in range(G)]
    for A in As:
        np.testing.assert_allclose(A.sum(axis=1), 1.0, rtol=1e-13)
        for r, p in enumerate(P):
            assert np.all(A[r, p + 1:] == 0.0)
            assert np.all(A[r, : p + 1] > 0.0)
    col = zo.accumulated_scores(As)
    assert abs(col.sum() - G * len(P)) < 1e-10
    # GQA aggregate = mean over heads of the single-head Eq. 8 score
    per_head = np.stack([zo.normalized_scores(Q[g:g + 1], K, P) for g in range(G)])
    np.testing.assert_allclose(zo.normalized_scores(Q, K, P), per_head.mean(axis=0), rtol=1e-12)
    # l = 1
    assert zo.normalized_scores(np.ones((1, 1, d)), np.ones((1, d)), [0])[0] == 1.0


def test_normalized_scores_rejects_list_not_ending_at_last_token():
    with pytest.raises(ValueError):
        zo.normalized_scores(np.zeros((1, 8, 4)), np.zeros((8, 4)), [1, 2, 3])


def test_structural_nnz_counts_unmasked_rows():
    assert zo.structural_nnz([2, 5, 9], 10).tolist() == [3, 3, 3, 2, 2, 2, 1, 1, 1, 1]


# ---------------------------------------------------------------- probe sampler
@pytest.mark.parametrize("l", [1, 2, 17, 100, 512, 4096])
def test_probe_positions_structure(l):
    P = zo.probe_positions(l, 0.05, 0.05, 1234)
    n_rec, n_rnd = zo.probe_counts(l, 0.05, 0.05)
    assert n_rec == max(1, int(0.05 * l)) and n_rnd == min(l - n_rec, int(0.05 * l))
    assert len(P) == n_rec + n_rnd
    assert np.all(np.diff(P) > 0)                       # ascending, unique
    assert P[-n_rec:].tolist() == list(range(l - n_rec, l))
    assert np.all(P[:n_rnd] < l - n_rec)
    # deterministic, seed-dependent
    assert np.array_equal(P, zo.probe_positions(l, 0.05, 0.05, 1234))
    if n_rnd > 4:
        assert not np.array_equal(P, zo.probe_positions(l, 0.05, 0.05, 1235))


def test_probe_counts_at_benchmark_lengths():
    assert zo.probe_counts(512, 0.05, 0.05) == (25, 25)
    assert zo.probe_counts(4096, 0.05, 0.05) == (204, 204)
    assert zo.probe_counts(8192, 0.05, 0.05) == (409, 409)
    assert zo.probe_counts(32768, 0.05, 0.05) == (1638, 1638)


def test_probe_sampler_is_roughly_uniform():
    hits = np.zeros(50)
    for seed in range(400):
        P = zo.probe_positions(60, 1 / 6, 0.2, seed)   # 10 recent, 12 random of 50
        hits[P[:12]] += 1
    assert hits.min() > 50 and hits.max() < 150          # expectation 96 each


# ---------------------------------------------------------------- split
def test_split_salient_brute_force_and_ties():
    rs = _rng(3)
    for trial in range(30):
        n = int(rs.randint(1, 40))
        p = rs.randint(0, 6, size=n).astype(np.float64) / 4.0   # many ties
        n_s = int(rs.randint(0, n + 1))
        keyed = sorted(range(n), key=lambda j: (-p[j], j))
        sal, reg = zo.split_salient(p, n_s)
        assert sal.tolist() == sorted(keyed[:n_s])
        assert reg.tolist() == sorted(keyed[n_s:])
        assert len(set(sal) & set(reg)) == 0 and len(sal) + len(reg) == n
        if 0 < n_s < n:
            assert p[sal].min() >= p[reg].max()


def test_salient_counts_at_benchmark_lengths():
    assert zo.salient_count(0.4, 512) == 204
    assert zo.salient_count(0.4, 4096) == 1638
    assert zo.salient_count(0.3, 8192) == 2457
    assert zo.salient_count(0.4, 32768) == 13107
    assert zo.salient_count(0.4, 100) == 40
    assert zo.salient_count(0.0, 100) == 0 and zo.salient_count(1.0, 100) == 100


# ---------------------------------------------------------------- CSTQuant
def _outlier_matrix(n, d, seed, dtype=torch.float16):
    rs = _rng(seed)
    X = rs.standard_normal((n, d))
    X[:, rs.choice(d, 3, replace=False)] *= 15.0
    return torch.tensor(X).to(dtype).to(torch.float32).numpy()


@pytest.mark.parametrize("bits", [2, 4])
@pytest.mark.parametrize("n,d", [(1, 8), (5, 16), (64, 128), (201, 128)])
def test_cst_quant_half_step_bound_and_code_range(bits, n, d):
    X = _outlier_matrix(n, d, 17 + bits + n)
    q = zo.cst_quant(X, bits)
    L = (1 << bits) - 1
    c, s, z, codes = (q[k].astype(np.float64) for k in ("c", "s", "z", "codes"))
    assert codes.min() >= 0 and codes.max() <= L
    Y = X.astype(np.float64) / c[None, :]
    recon = (codes - z[:, None]) * s[:, None]
    # |y - (code - z) s| <= s/2 (tiny slack for the fp32 division that formed y)
    assert np.all(np.abs(Y - recon) <= s[:, None] * (0.5 + 1e-5))
    # each token's smallest channel maps to code 0 and its largest to L
    for t in range(n):
        if Y[t].max() > Y[t].min():
            assert codes[t, Y[t].argmin()] == 0 and codes[t, Y[t].argmax()] == L
            order = np.argsort(Y[t], kind="stable")
            assert np.all(np.diff(codes[t, order]) >= 0)        # monotone in y
    # z is an integer; dequantised values restore each channel's magnitude
    assert np.all(z == np.rint(z))
    X_hat = zo.cst_dequant(q)
    assert np.all(np.abs(X_hat - X) <= c[None, :] * s[:, None] * (0.5 + 1e-5))


def test_channel_factor_is_sqrt_of_channel_absmax_and_roundtrips():
    X = _outlier_matrix(50, 32, 23)
    q = zo.cst_quant(X, 4)
    np.testing.assert_array_equal(q["c"], np.sqrt(np.abs(X).max(axis=0)).astype(np.float32))
    c = q["c"]
    back = (X / c[None, :]).astype(np.float32) * c[None, :]
    ulp = np.spacing(np.abs(X).astype(np.float32))
    assert np.all(np.abs(back.astype(np.float64) - X) <= ulp)   # c * (x / c) = x to 1 ulp
    # after normalisation every channel's magnitude is sqrt of what it was (Eq. 6)
    Y = X / c[None, :]
    np.testing.assert_allclose(np.abs(Y).max(axis=0), c, rtol=1e-6)


def test_degenerate_rows_and_channels():
    X = np.zeros((3, 8), dtype=np.float32)
    X[1, :] = 2.5          # constant token
    X[2, :] = -0.75        # constant negative token
    q = zo.cst_quant(X, 2)
    assert np.all(q["c"] == np.sqrt(np.float32(2.5)))
    # constant rows (after normalisation) reconstruct exactly up to fp32 rounding of y
    np.testing.assert_allclose(zo.cst_dequant(q), X, rtol=1e-6, atol=0)
    assert np.all(q["codes"] == 0)
    Z = np.zeros((3, 8), dtype=np.float32)
    qz = zo.cst_quant(Z, 4)
    assert np.all(qz["c"] == 1) and np.all(qz["s"] == 1) and np.all(qz["codes"] == 0)
    assert np.all(zo.cst_dequant(qz) == 0)
    # empty subset
    qe = zo.cst_quant(np.zeros((0, 8), dtype=np.float32), 4)
    assert qe["codes"].shape == (0, 8) and np.all(qe["c"] == 1)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_unit_channel_factors_reduce_to_library_affine_quantiser(bits):
    """With every |channel| max equal to 1 the factors are 1 and CSTQuant is
    plain asymmetric per-row uniform quantisation; torch's per-channel fake
    quantiser (axis = token) is the library statement of Eq. 5."""
    rs = _rng(31)
    n, d = 37, 24
    X = rs.uniform(-1, 1, size=(n, d)).astype(np.float32)
    X[rs.randint(0, n, size=d), np.arange(d)] = np.where(rs.rand(d) < 0.5, -1.0, 1.0)
    q = zo.cst_quant(X, bits)
    assert np.all(q["c"] == 1.0)
    L = (1 << bits) - 1
    xt = torch.tensor(X)
    got = torch.fake_quantize_per_channel_affine(
        xt, torch.tensor(q["s"]), torch.tensor(q["z"]).to(torch.int32), 0, 0, L).numpy()
    np.testing.assert_allclose(zo.cst_dequant(q), got.astype(np.float64), rtol=0, atol=1e-6)
    # and the parameters are Eq. 5's: s = (max - min) / (2^k - 1), z = -round(min / s)
    for t in range(n):
        assert abs(q["s"][t] - (X[t].max() - X[t].min()) / L) <= 1e-7
        assert q["z"][t] == -round(float(np.float32(X[t].min()) / q["s"][t]))


def test_fp32_codes_agree_with_fp64_away_from_rounding_boundaries():
    X = _outlier_matrix(300, 128, 41, dtype=torch.bfloat16)
    for bits in (2, 4):
        q = zo.cst_quant(X, bits)
        L = (1 << bits) - 1
        Y = X.astype(np.float64) / q["c"].astype(np.float64)[None, :]
        real = zo.token_quant_reference_fp64(Y, bits)
        frac = np.abs(real - np.floor(real) - 0.5)
        safe = frac > 1e-4
        expect = np.clip(np.rint(real), 0, L)
        assert safe.mean() > 0.99
        assert np.array_equal(q["codes"][safe], expect[safe].astype(np.uint8))


def test_round_half_to_even_is_used():
    """A single token with x_i = y_i |y_i| has c_i = |y_i| and normalised values
    y exactly; y = (0, .5, 1.5, 2.5, 3.5, 15) at 4 bits gives s = 1, z = 0 and
    codes that sit on .5 boundaries: ties must go to the even integer."""
    Y = np.array([[0.0, 0.5, 1.5, 2.5, 3.5, 15.0]], dtype=np.float32)
    X = (Y * np.abs(Y)).astype(np.float32)
    q = zo.cst_quant(X, 4)
    assert q["s"][0] == 1.0 and q["z"][0] == 0.0
    assert q["codes"][0].tolist() == [0, 0, 2, 2, 4, 15]


def test_pack_unpack_canonical_layout():
    codes = np.arange(16, dtype=np.uint8).reshape(1, 16) % 16
    p4 = zo.pack_codes(codes, 4)
    assert p4[0, 0] == (0 | (1 << 4)) and p4[0, 7] == (14 | (15 << 4))
    c2 = (np.arange(16, dtype=np.uint8).reshape(1, 16)) % 4
    p2 = zo.pack_codes(c2, 2)
    assert p2[0, 0] == (0 | (1 << 2) | (2 << 4) | (3 << 6))
    for bits, c in ((4, codes), (2, c2)):
        assert np.array_equal(zo.unpack_codes(zo.pack_codes(c, bits), bits, 16), c)


# ---------------------------------------------------------------- Appendix A
def test_appendix_a_printed_ratios():
    rows = {}
    with open(os.path.join(GOLDEN, "appendix_a_ratios.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                rows[k] = float(v)
    got = {
        "group": zo.compression_ratio("group", "group", 8, 4096, 4096, 4, 32, 16),
        "token": zo.compression_ratio("token", "token", 8, 4096, 4096, 4, 32, 16),
        "baseline": zo.compression_ratio("channel", "cst", 8, 4096, 4096, 4, 32, 16),
    }
    for k, v in rows.items():
        assert round(got[k], 3) == v, (k, got[k], v)


def test_table1_parameter_counts():
    b, hd, l, n = 8, 4096, 4096, 32
    want = {}
    with open(os.path.join(GOLDEN, "table1_param_counts.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, _, val = line.split()
                want[name] = int(val)
    pc = zo.quant_param_count
    assert pc("token", b, hd, l, n) == want["tokenwise_one_tensor"]
    assert pc("group", b, hd, l, n) == want["groupwise_one_tensor"]
    assert pc("cst", b, hd, l, n) == want["cst_one_tensor"]
    assert pc("channel", b, hd, l, n) + pc("cst", b, hd, l, n) == want["channel_K_plus_cst_V"]
    assert 2 * pc("token", b, hd, l, n) == want["tokenwise_K_and_V"]
    assert 2 * pc("group", b, hd, l, n) == want["groupwise_K_and_V"]


# ---------------------------------------------------------------- decode (Eq. 4, Alg. 3)
def _small_unit(G=2, d=16, l=48, ratio=0.5, bits=(4, 2), window=100, seed=0):
    rs = _rng(seed)
    Q = rs.standard_normal((G, l, d))
    K = _outlier_matrix(l, d, seed + 1).astype(np.float64)
    V = rs.standard_normal((l, d)).astype(np.float32).astype(np.float64)
    P = zo.probe_positions(l, 0.1, 0.1, seed)
    u = zo.UnitCache(G, d, ratio, bits[0], bits[1], window)
    u.prefill_compress(Q, K, V, P)
    return u, Q, K, V, rs


def test_all_tokens_16_bit_equals_library_attention():
    """bits_hi = 16 with every token salient: decode must be exact attention."""
    G, d, l = 4, 32, 70
    u, Q, K, V, rs = _small_unit(G, d, l, ratio=1.0, bits=(16, 2), seed=3)
    assert u.segments[0].lo.n == 0
    ks, vs = [], []
    for step in range(5):
        k, v, q = rs.standard_normal(d), rs.standard_normal(d), rs.standard_normal((G, d))
        ks.append(k), vs.append(v)
        u.append(k, v)
        o = u.decode_attention(q, False)
        K_all = torch.tensor(np.vstack([K] + ks))
        V_all = torch.tensor(np.vstack([V] + vs))
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.tensor(q)[None, :, None, :], K_all[None, None].expand(1, G, -1, -1),
            V_all[None, None].expand(1, G, -1, -1))[0, :, 0, :].numpy()
        np.testing.assert_allclose(o, ref, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(o, zo.exact_attention(q, K_all.numpy(), V_all.numpy()),
                                   rtol=1e-12)


def test_decode_equals_exact_attention_over_dequantised_cache_and_is_order_free():
    u, Q, K, V, rs = _small_unit(seed=5)
    seg = u.segments[0]
    # rebuild the dequantised cache in ORIGINAL token order
    K_hat = np.zeros_like(K)
    V_hat = np.zeros_like(V)
    for sub in (seg.hi, seg.lo):
        K_hat[sub.idx] = sub.K_hat
        V_hat[sub.idx] = sub.V_hat
    k, v, q = rs.standard_normal(16), rs.standard_normal(16), rs.standard_normal((2, 16))
    u.append(k, v)
    o = u.decode_attention(q, False)
    ref = zo.exact_attention(q, np.vstack([K_hat, k]), np.vstack([V_hat, v]))
    np.testing.assert_allclose(o, ref, rtol=1e-11, atol=1e-13)
    # any split of the tokens merged by (max, sum, weighted acc) gives the same result
    Kc, Vc = np.vstack([K_hat, k]), np.vstack([V_hat, v])
    parts = [(0, 10), (10, 11), (11, 49)]
    m = np.full(2, -np.inf)
    ssum = np.zeros(2)
    acc = np.zeros((2, 16))
    for a, b in parts:
        lg = q @ Kc[a:b].T / math.sqrt(16)
        m_new = np.maximum(m, lg.max(axis=1))
        scale = np.exp(m - m_new)
        e = np.exp(lg - m_new[:, None])
        ssum = ssum * scale + e.sum(axis=1)
        acc = acc * scale[:, None] + e @ Vc[a:b]
        m = m_new
    np.testing.assert_allclose(acc / ssum[:, None], o, rtol=1e-11)
    # quantisation error is bounded through the half-step bound (sanity, not parity)
    exact = zo.exact_attention(q, np.vstack([K, k]), np.vstack([V, v]))
    assert np.abs(o - exact).max() < 1.0


def test_folded_dequantisation_algebra():
    """q . k_hat = s_t (q' . code - z_t sum q') with q' = q * c^K, and
    o = c^V * (sum_t w_t code_t - sum_t w_t z_t) with w_t = a_t s_t."""
    u, Q, K, V, rs = _small_unit(G=1, seed=9)
    sub = u.segments[0].lo
    q = rs.standard_normal(16)
    qK, qV = sub.qK, sub.qV
    qp = q * qK["c"].astype(np.float64)
    dots = qK["codes"].astype(np.float64) @ qp
    logits_folded = qK["s"].astype(np.float64) * (dots - qK["z"].astype(np.float64) * qp.sum())
    np.testing.assert_allclose(logits_folded, sub.K_hat @ q, rtol=1e-9, atol=1e-11)
    a = np.exp(logits_folded - logits_folded.max())
    a /= a.sum()
    w = a * qV["s"].astype(np.float64)
    o_folded = qV["c"].astype(np.float64) * (w @ qV["codes"].astype(np.float64)
                                             - (w * qV["z"].astype(np.float64)).sum())
    np.testing.assert_allclose(o_folded, a @ sub.V_hat, rtol=1e-9, atol=1e-11)


def test_streaming_flush_matches_window_submatrix():
    """With every decode step a probe step, the flushed window's score is Eq. 8
    on the window's columns of the decode-time attention rows (brute force here),
    and the window becomes a new segment with floor(r * window) salient tokens."""
    window, G, d = 8, 2, 16
    u, Q, K, V, rs = _small_unit(G=G, d=d, l=30, ratio=0.5, window=window, seed=13)
    rows = []
    toks = []
    for step in range(window):
        k, v, q = rs.standard_normal(d), rs.standard_normal(d), rs.standard_normal((G, d))
        toks.append((k, v))
        u.append(k, v)
        n_before = len(u.segments)
        u.decode_attention(q, True)
        rows.append(u.last_attention[:, -(step + 1):].copy())    # window columns so far
    assert len(u.segments) == n_before + 1 and u.tail_K.shape[0] == 0 and u.i == 0
    colsum = np.zeros(window)
    nnz = np.zeros(window)
    for step, a in enumerate(rows):
        colsum[: step + 1] += a.sum(axis=0)
        nnz[: step + 1] += 1
    expect = colsum / (G * nnz)
    seg = u.segments[-1]
    np.testing.assert_allclose(seg.p_tilde, expect, rtol=1e-12)
    assert nnz.tolist() == [window - j for j in range(window)]
    assert seg.hi.n == 4 and seg.lo.n == 4
    sal, reg = zo.split_salient(expect, 4)
    assert np.array_equal(seg.hi.idx, sal) and np.array_equal(seg.lo.idx, reg)
    Kw = np.stack([t[0] for t in toks]).astype(np.float32)
    np.testing.assert_array_equal(seg.hi.qK["codes"], zo.cst_quant(Kw[sal], 4)["codes"])


def test_probe_steps_without_flags_are_only_the_last_five():
    window, G, d = 10, 1, 8
    u, Q, K, V, rs = _small_unit(G=G, d=d, l=12, ratio=0.5, window=window, seed=17)
    seen = []
    for step in range(window - 1):
        u.append(rs.standard_normal(d), rs.standard_normal(d))
        u.decode_attention(rs.standard_normal((G, d)), False)
        seen.append(u.tail_nnz.copy())
    # steps 1..5 collect nothing; steps 6..9 (i > window-5) do
    assert seen[4].sum() == 0
    assert seen[5][:6].tolist() == [1] * 6 and seen[5][6:].sum() == 0
    assert seen[8][:6].tolist() == [4] * 6 and seen[8][8] == 1


def test_multi_unit_wrapper_keeps_units_independent():
    b, hq, hkv, d, l = 2, 4, 2, 16, 40
    rs = _rng(21)
    Q = rs.standard_normal((b, hq, l, d))
    K = rs.standard_normal((b, hkv, l, d)).astype(np.float32).astype(np.float64)
    V = rs.standard_normal((b, hkv, l, d)).astype(np.float32).astype(np.float64)
    P = zo.probe_positions(l, 0.1, 0.1, 5)
    full = zo.ZipCacheOracle(b, hq, hkv, d, 0.4)
    full.prefill_compress(Q, K, V, P)
    one = zo.ZipCacheOracle(b, hq, hkv, d, 0.4, units=[(1, 0)])
    one.prefill_compress(Q, K, V, P)
    np.testing.assert_array_equal(full.units[(1, 0)].segments[0].hi.qK["codes"],
                                  one.units[(1, 0)].segments[0].hi.qK["codes"])
    single = zo.UnitCache(2, d, 0.4)
    single.prefill_compress(Q[1, 0:2], K[1, 0], V[1, 0], P)
    np.testing.assert_array_equal(single.segments[0].p_tilde,
                                  full.units[(1, 0)].segments[0].p_tilde)


# ---------------------------------------------------------------- ChannelQuant (keys)
@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("n,d", [(1, 8), (7, 16), (64, 128), (201, 128)])
def test_channel_quant_half_step_bound_per_channel(bits, n, d):
    """Eq. 5 per channel: every element within half a step of its channel's grid, the channel's
    smallest token at code 0 and its largest at the top code, codes monotone along a channel."""
    X = _outlier_matrix(n, d, 91 + bits + n)
    X[:, 0] += 40.0                                  # an all-positive channel: negative zero point
    q = zo.channel_quant(X, bits)
    L = (1 << bits) - 1
    s, z, codes = (q[k].astype(np.float64) for k in ("s", "z", "codes"))
    assert s.shape == (d,) and z.shape == (d,) and codes.shape == (n, d)
    assert codes.min() >= 0 and codes.max() <= L and np.all(z == np.rint(z))
    recon = zo.channel_dequant(q)
    # slack: the fp32 quotient x / s carries an error of |x / s| 2^-24 steps
    slack = 1e-5 + np.abs(X / s[None, :]).max() * 2.0 ** -22
    assert np.all(np.abs(X - recon) <= s[None, :] * (0.5 + slack))
    for i in range(d):
        if X[:, i].max() > X[:, i].min():
            assert codes[X[:, i].argmin(), i] == 0 and codes[X[:, i].argmax(), i] == L
            order = np.argsort(X[:, i], kind="stable")
            assert np.all(np.diff(codes[order, i]) >= 0)
    if n > 1:
        assert z[0] < 0                              # the shifted channel lies above zero


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_channel_quant_is_the_library_per_column_affine_quantiser(bits):
    """torch's per-channel fake quantiser along the CHANNEL axis is the library statement of
    channelwise Eq. 5; parameters are Eq. 5's own formulas evaluated per column."""
    rs = _rng(77)
    n, d = 53, 24
    X = (rs.standard_normal((n, d)) * rs.uniform(0.2, 12.0, size=d)[None, :]).astype(np.float32)
    q = zo.channel_quant(X, bits)
    L = (1 << bits) - 1
    got = torch.fake_quantize_per_channel_affine(
        torch.tensor(X), torch.tensor(q["s"]), torch.tensor(q["z"]).to(torch.int32), 1, 0, L).numpy()
    np.testing.assert_allclose(zo.channel_dequant(q), got.astype(np.float64), rtol=0, atol=1e-5)
    for i in range(d):
        assert abs(q["s"][i] - (X[:, i].max() - X[:, i].min()) / L) <= 1e-6 * q["s"][i] + 1e-9
        assert q["z"][i] == -round(float(np.float32(X[:, i].min()) / q["s"][i]))


def test_channel_quant_equals_token_quant_of_the_transpose():
    """Channelwise quantisation of X is tokenwise quantisation of X^T: with unit channel
    factors cst_quant(X^T) must give the transposed codes and the same parameters."""
    rs = _rng(5)
    X = rs.uniform(-1, 1, size=(16, 40)).astype(np.float32)
    # make every column of X^T (= row of X) reach |1| so that cst_quant's factors are all 1
    X[np.arange(16), rs.randint(0, 40, size=16)] = 1.0
    qc = zo.channel_quant(X, 4)
    qt = zo.cst_quant(np.ascontiguousarray(X.T), 4)
    # cst_quant normalises the 16 channels of X^T, i.e. the tokens of X: all factors 1
    assert np.all(qt["c"] == 1.0)
    np.testing.assert_array_equal(qc["codes"], qt["codes"].T)
    np.testing.assert_array_equal(qc["s"], qt["s"])
    np.testing.assert_array_equal(qc["z"], qt["z"])


def test_channel_quant_degenerate_channels():
    X = np.zeros((4, 6), dtype=np.float32)
    X[:, 1] = 3.5                                    # constant channel
    X[:, 2] = -0.25
    q = zo.channel_quant(X, 2)
    np.testing.assert_allclose(zo.channel_dequant(q), X, rtol=1e-6, atol=0)
    assert q["s"][0] == 1 and q["z"][0] == 0 and np.all(q["codes"][:, 0] == 0)
    qe = zo.channel_quant(np.zeros((0, 6), dtype=np.float32), 4)
    assert qe["codes"].shape == (0, 6) and np.all(qe["s"] == 1)


def test_key_scheme_channel_reaches_the_cache_and_decode():
    """UnitCache with k_scheme="channel": keys dequantise by channel parameters, values by
    CSTQuant, and decode attention equals exact attention over that dequantised cache."""
    rs = _rng(12)
    l, d, G = 90, 16, 2
    Q = rs.standard_normal((G, l, d)); K = rs.standard_normal((l, d)) * 3; V = rs.standard_normal((l, d))
    P = zo.probe_positions(l, 0.1, 0.1, 3)
    u = zo.UnitCache(G, d, 0.4, 4, 2, window=100, k_scheme="channel")
    u.prefill_compress(Q, K, V, P)
    seg = u.segments[0]
    for sub in (seg.hi, seg.lo):
        assert sub.qK["scheme"] == "channel" and sub.qK["s"].shape == (d,)
        np.testing.assert_array_equal(sub.K_hat, zo.channel_dequant(zo.channel_quant(K.astype(np.float32)[sub.idx], sub.bits)))
        np.testing.assert_array_equal(sub.V_hat, zo.cst_dequant(zo.cst_quant(V.astype(np.float32)[sub.idx], sub.bits)))
    q = rs.standard_normal((G, d))
    k_new, v_new = rs.standard_normal(d), rs.standard_normal(d)
    u.append(k_new, v_new)
    o = u.decode_attention(q, False)
    K_all = np.vstack([seg.hi.K_hat, seg.lo.K_hat, k_new[None]])
    V_all = np.vstack([seg.hi.V_hat, seg.lo.V_hat, v_new[None]])
    np.testing.assert_allclose(o, zo.exact_attention(q, K_all, V_all), rtol=1e-12)


# ---------------------------------------------------------------- accounting of mixed precision
def test_table3_printed_ratios_of_the_mixed_precision_cache():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "table3_ratios.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 2
    for r, printed in rows:
        got = zo.mixed_precision_ratio(8, 4096, 840, float(r), 4, 2, "channel", "cst", 16)
        assert round(got, 2) == float(printed), (r, got)
    # one subset at 4 bits is Appendix A's own case
    assert abs(zo.mixed_precision_ratio(8, 4096, 4096, 1.0, 4, 2) -
               zo.compression_ratio("channel", "cst", 8, 4096, 4096)) < 1e-12


def test_cache_footprint_counts_every_stored_byte():
    """The footprint of the layout this repository stores (parameters per unit and subset),
    against a count written out by hand for one small shape."""
    b, h, d, n_hi, n_lo = 2, 3, 128, 10, 30
    by_hand_cst = b * h * ((2 * 10 * 128 * 4 // 8 + 10 * 16 + 2 * 128 * 4) + (2 * 30 * 128 * 2 // 8 + 30 * 16 + 2 * 128 * 4))
    assert zo.cache_footprint_bytes(b, h, d, n_hi, n_lo, 4, 2, "cst") == by_hand_cst
    by_hand_ch = b * h * ((2 * 10 * 128 * 4 // 8 + 10 * 8 + 3 * 128 * 4) + (2 * 30 * 128 * 2 // 8 + 30 * 8 + 3 * 128 * 4))
    assert zo.cache_footprint_bytes(b, h, d, n_hi, n_lo, 4, 2, "channel") == by_hand_ch
    # channelwise keys drop 8 bytes per token and add 512 bytes per (unit, subset)
    assert by_hand_cst - by_hand_ch == b * h * (40 * 8 - 2 * 512)
    # with the paper's counting (16-bit parameters) the real layout of a long cache comes close
    # to Table 3's figure: per-head token groups cost h_kv times more token parameters
    l, r = 4096, 0.6
    n_s = int(r * l)
    real = zo.cache_footprint_bytes(8, 32, 128, n_s, l - n_s, 4, 2, "channel", param_bytes=2)
    ratio = (2 * 8 * 4096 * l * 2) / real
    assert 4.75 < ratio < zo.mixed_precision_ratio(8, 4096, l, r, 4, 2)


# ---------------------------------------------------------------- 16-bit parameters
@pytest.mark.parametrize("bits", [2, 4])
def test_f16_parameters_keep_the_half_step_bound(bits):
    """Scales rounded UP to fp16: parameters are exactly representable in 16 bits, the codes
    stay in range without clipping at the top, and |y - (code - z) s| <= s/2 holds for the
    STORED scale."""
    X = _outlier_matrix(150, 128, 41)
    q = zo.cst_quant_f16_params(X, bits)
    L = (1 << bits) - 1
    for k in ("c", "s"):
        np.testing.assert_array_equal(q[k], q[k].astype(np.float16).astype(np.float32))
    assert np.all(np.abs(q["z"]) < 2 ** 15) and np.all(q["z"] == np.rint(q["z"]))
    c, s, z, codes = (q[k].astype(np.float64) for k in ("c", "s", "z", "codes"))
    Y = X.astype(np.float64) / c[None, :]
    assert np.all(np.abs(Y - (codes - z[:, None]) * s[:, None]) <= s[:, None] * (0.5 + 1e-5))
    exact = zo.cst_quant(X, bits)
    # never below the fp32 scale of the same normalised row, and within one fp16 step of it
    assert np.all(q["s"] >= (Y.max(axis=1) - Y.min(axis=1)) / L * (1 - 1e-6))
    assert np.all(q["s"] <= exact["s"] * (1 + 2.0 ** -9))
    assert np.mean(q["codes"] == exact["codes"]) > 0.9
    # a scale rounded DOWN cannot cover the row: its top code falls short of the maximum
    y_max = 1.0
    s_exact = y_max / L
    s_down = float(np.nextafter(zo.round_up_to_f16(np.array([s_exact]))[0], np.float16(0)))
    if s_down < s_exact:
        assert L * s_down < y_max <= L * float(zo.round_up_to_f16(np.array([s_exact]))[0])


def test_round_up_to_f16():
    x = np.array([0.1, 1.0, 1.0003, 65504.0, 6e-8, 0.0], dtype=np.float32)
    up = zo.round_up_to_f16(x)
    assert np.all(up.astype(np.float32) >= x)
    below = np.nextafter(up, np.float16(-np.inf)).astype(np.float32)
    assert np.all((below < x) | (up.astype(np.float32) == x))


# ---------------------------------------------------------------- token-level saliency
def test_token_scope_shares_one_split_across_heads():
    """scope="token": every KV head of a batch row gets the same salient list, chosen from the
    mean of the per-head normalised scores; with one KV head it is the per-head split."""
    rs = _rng(8)
    b, hq, hkv, l, d = 2, 4, 2, 60, 8
    Q = rs.standard_normal((b, hq, l, d)); K = rs.standard_normal((b, hkv, l, d)); V = rs.standard_normal((b, hkv, l, d))
    P = zo.probe_positions(l, 0.1, 0.1, 1)
    oc = zo.ZipCacheOracle(b, hq, hkv, d, 0.4, window=8, scope="token")
    oc.prefill_compress(Q, K, V, P)
    for bi in range(b):
        per_head = [zo.normalized_scores(Q[bi, kv * 2:(kv + 1) * 2], K[bi, kv], P) for kv in range(hkv)]
        sal, _ = zo.split_salient(sum(per_head) / hkv, zo.salient_count(0.4, l))
        for kv in range(hkv):
            np.testing.assert_array_equal(oc.units[(bi, kv)].segments[0].hi.idx, sal)
    # decode across one window: the re-compressed window's split is shared as well
    for s in range(8):
        oc.append(rs.standard_normal((b, hkv, d)), rs.standard_normal((b, hkv, d)))
        oc.decode_attention(rs.standard_normal((b, hq, d)), s % 2 == 0)
    for bi in range(b):
        a, c = oc.units[(bi, 0)].segments[1], oc.units[(bi, 1)].segments[1]
        np.testing.assert_array_equal(a.hi.idx, c.hi.idx)
        assert a.n == 8 and len(oc.units[(bi, 0)].tail_K) == 0
    one = zo.ZipCacheOracle(1, 2, 1, d, 0.4, scope="token")
    ref = zo.ZipCacheOracle(1, 2, 1, d, 0.4)
    one.prefill_compress(Q[:1, :2], K[:1, :1], V[:1, :1], P)
    ref.prefill_compress(Q[:1, :2], K[:1, :1], V[:1, :1], P)
    np.testing.assert_array_equal(one.units[(0, 0)].segments[0].hi.idx, ref.units[(0, 0)].segments[0].hi.idx)


# ---------------------------------------------------------------- token groups over all heads (Alg. 1, X in R^{l x hd})
def test_token_groups_over_all_heads():
    """group="all_heads": one (s, z) per token for the channels of every KV head of its batch row
    (Sec. 4.1: 2bl parameters per tensor beside the hd channel factors).  Pinned by pure-Python
    loops for the token statistics, the half-step bound under the shared scale, the parameter
    count, and the reduction to the per-head grouping when there is one KV head."""
    rs = _rng(21)
    b, hq, hkv, l, d = 2, 4, 2, 40, 8
    Q = rs.standard_normal((b, hq, l, d)); K = rs.standard_normal((b, hkv, l, d)) * 3; V = rs.standard_normal((b, hkv, l, d))
    K[:, 1] *= 7.0                                    # heads of unlike range: the shared scale is the wider head's
    P = zo.probe_positions(l, 0.1, 0.1, 1)
    oc = zo.ZipCacheOracle(b, hq, hkv, d, 0.4, window=8, scope="token", group="all_heads")
    oc.prefill_compress(Q, K, V, P)
    f32 = np.float32
    n_params = 0
    for bi in range(b):
        subs = [oc.units[(bi, kv)].segments[0].hi for kv in range(hkv)]
        idx = subs[0].idx
        for tensor, X in (("qK", K), ("qV", V)):
            qs = [getattr(sub, tensor) for sub in subs]
            for kv in range(1, hkv):
                np.testing.assert_array_equal(qs[kv]["s"], qs[0]["s"])      # one (s, z) per token for all heads
                np.testing.assert_array_equal(qs[kv]["z"], qs[0]["z"])
            n_params += 2 * len(idx) + hkv * d
            # the token statistics by loops: minimum and maximum of x / c over every head's channels
            for r, j in enumerate(idx):
                ys = []
                for kv in range(hkv):
                    Xs = X[bi, kv].astype(f32)[idx]
                    for ch in range(d):
                        c = f32(np.sqrt(f32(np.abs(Xs[:, ch]).max())))
                        assert c == qs[kv]["c"][ch]
                        ys.append(f32(Xs[r, ch] / c))
                mn, mx = min(ys), max(ys)
                assert qs[0]["s"][r] == f32(f32(mx - mn) / f32(15))
                assert qs[0]["z"][r] == -np.rint(f32(mn / qs[0]["s"][r]))
                # half-step bound of every head's codes under the shared scale
                k = 0
                for kv in range(hkv):
                    for ch in range(d):
                        y = ys[k]; k += 1
                        code = float(qs[kv]["codes"][r, ch])
                        assert abs(float(y) - (code - float(qs[0]["z"][r])) * float(qs[0]["s"][r])) <= 0.5 * float(qs[0]["s"][r]) * (1 + 1e-5)
    # Sec. 4.1's count for the salient subsets: (2 n_s + h d) per tensor and batch row
    n_s = zo.salient_count(0.4, l)
    assert n_params == b * 2 * (2 * n_s + hkv * d)
    # a re-compressed window is grouped the same way
    for s in range(8):
        oc.append(rs.standard_normal((b, hkv, d)), rs.standard_normal((b, hkv, d)))
        oc.decode_attention(rs.standard_normal((b, hq, d)), s % 2 == 0)
    for bi in range(b):
        a, c = oc.units[(bi, 0)].segments[1].lo, oc.units[(bi, 1)].segments[1].lo
        np.testing.assert_array_equal(a.qV["s"], c.qV["s"]); np.testing.assert_array_equal(a.qK["z"], c.qK["z"])
    # one KV head: the same as the grouping per head
    one = zo.ZipCacheOracle(1, 2, 1, d, 0.4, scope="token", group="all_heads")
    ref = zo.ZipCacheOracle(1, 2, 1, d, 0.4, scope="token")
    for o in (one, ref):
        o.prefill_compress(Q[:1, :2], K[:1, :1], V[:1, :1], P)
    for name in ("hi", "lo"):
        for t in ("qK", "qV"):
            x, y = getattr(getattr(one.units[(0, 0)].segments[0], name), t), getattr(getattr(ref.units[(0, 0)].segments[0], name), t)
            for key in ("c", "s", "z", "codes"):
                np.testing.assert_array_equal(x[key], y[key])
    with pytest.raises(ValueError):
        zo.ZipCacheOracle(1, 2, 1, d, 0.4, group="all_heads")          # needs one split per token


# ---------------------------------------------------------------- Eq. 2: causal prefill attention
@pytest.mark.parametrize("l,d", [(1, 8), (7, 8), (33, 16), (130, 32)])
def test_prefill_attention_is_library_causal_attention(l, d):
    """Eq. 2 with the causal mask against the library's scaled-dot-product attention
    (is_causal=True, fp64 on the CPU), and its row log-sum-exp against the library's logsumexp
    of the masked logits; the rows of Eq. 9's probe attention are rebuilt from that number."""
    rs = _rng(3 + l)
    Q, K, V = rs.standard_normal((l, d)), rs.standard_normal((l, d)) * 2, rs.standard_normal((l, d))
    O, lse2 = zo.prefill_attention(Q, K, V)
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(Q)[None, None], torch.tensor(K)[None, None], torch.tensor(V)[None, None], is_causal=True)
    np.testing.assert_allclose(O, want[0, 0].numpy(), rtol=1e-10, atol=1e-12)
    S = torch.tensor(Q @ K.T / math.sqrt(d))
    S = S.masked_fill(torch.triu(torch.ones(l, l, dtype=torch.bool), diagonal=1), float("-inf"))
    np.testing.assert_allclose(lse2, (torch.logsumexp(S, dim=1) / math.log(2.0)).numpy(), rtol=1e-12)
    P = list(range(0, l, 3)) + ([l - 1] if (l - 1) % 3 else [])
    A = zo.probe_attention(Q[P], K, P)
    for r, p in enumerate(P):
        rebuilt = np.exp2(S[p, : p + 1].numpy() / math.log(2.0) - lse2[p])
        np.testing.assert_allclose(A[r, : p + 1], rebuilt, rtol=1e-10)


def test_prefill_attention_brute_force_and_last_row_is_decode():
    """Pure-Python loops on a tiny case; the last row of the causal output is Eq. 4 for the
    last query over all keys."""
    rs = _rng(9)
    l, d = 9, 4
    Q, K, V = rs.standard_normal((l, d)), rs.standard_normal((l, d)), rs.standard_normal((l, d))
    A = _brute_force_causal_attention(Q, K)
    O, _ = zo.prefill_attention(Q, K, V)
    for i in range(l):
        for c in range(d):
            assert abs(O[i, c] - sum(A[i][j] * V[j, c] for j in range(i + 1))) < 1e-12
    np.testing.assert_allclose(O[-1], zo.exact_attention(Q[-1:], K, V)[0], rtol=1e-12)
