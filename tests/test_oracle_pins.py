"""Pins for the CPU checker: what the paper and the mathematics fix, independent of the checker's own code."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import bpc_oracle as O

RNG = np.random.default_rng(20260804)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_storage_facts.txt")


def _facts():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split()
            out[k] = int(v)
    return out


def _keys(n, d, rng=RNG):
    scale = np.exp(0.5 * rng.standard_normal(d))
    scale[rng.choice(d, 4, replace=False)] *= 8
    return rng.standard_normal(d) * 0.5 + scale * rng.standard_normal((n, d))


# ------------------------------------------------------------------ Algorithm 1
def test_fit_frobenius_identity_and_orthogonality():
    # For u in {+-1}^N and v = uR/N:  ||R - u v||_F^2 = ||R||_F^2 - N ||v||^2, and u (R - u v) = 0.
    N, D, b = 257, 24, 16
    K = _keys(N, D)
    vs = RNG.standard_normal((b, D))
    P, H, tr = O.fit(K, vs)
    R = K.copy()
    for i in range(b):
        lhs = tr[i + 1] ** 2
        rhs = tr[i] ** 2 - N * np.dot(P[i], P[i])
        assert abs(lhs - rhs) <= 1e-10 * tr[0] ** 2
        R = R - np.outer(H[:, i], P[i])
        assert np.max(np.abs(H[:, i] @ R)) <= 1e-9 * np.abs(K).sum()
    assert np.all(np.diff(tr) <= 1e-12)                      # residual never grows (Figure: residual norms)
    assert abs(np.linalg.norm(K - H @ P) - tr[-1]) <= 1e-9 * tr[0]   # running residual == recomputed one
    assert set(np.unique(H)) <= {-1.0, 1.0}


def test_fit_first_bit_matches_definition():
    # iteration 1 written out by hand: u = sign(K v*), v = u K / N (not K^T-transposed, not unnormalised)
    N, D = 50, 7
    K = _keys(N, D)
    vs = RNG.standard_normal((1, D))
    P, H, _ = O.fit(K, vs)
    u = np.array([1.0 if sum(K[n, c] * vs[0, c] for c in range(D)) >= 0 else -1.0 for n in range(N)])
    v = np.array([sum(u[n] * K[n, c] for n in range(N)) / N for c in range(D)])
    assert np.array_equal(H[:, 0], u)
    assert np.allclose(P[0], v, rtol=0, atol=1e-13)


def test_fit_rank_one_closed_form():
    # K = u0 v0^T with u0 in {+-1}^N: one iteration recovers (+-u0, +-v0) and leaves R = 0.
    N, D = 64, 10
    u0 = np.where(RNG.random(N) < 0.5, -1.0, 1.0)
    v0 = RNG.standard_normal(D)
    K = np.outer(u0, v0)
    vs = RNG.standard_normal((2, D))
    P, H, tr = O.fit(K, vs)
    sgn = 1.0 if np.dot(v0, vs[0]) >= 0 else -1.0
    assert np.array_equal(H[:, 0], sgn * u0)
    assert np.allclose(P[0], sgn * v0, atol=1e-13)
    assert tr[1] <= 1e-12 * tr[0]


def test_fit_v_is_least_squares_optimum():
    N, D = 40, 6
    K = _keys(N, D)
    vs = RNG.standard_normal((1, D))
    P, H, tr = O.fit(K, vs)
    base = np.linalg.norm(K - np.outer(H[:, 0], P[0]))
    for _ in range(20):
        dv = 1e-3 * RNG.standard_normal(D)
        assert np.linalg.norm(K - np.outer(H[:, 0], P[0] + dv)) > base
    # and it equals numpy's least-squares solution for the fixed u
    sol = np.linalg.lstsq(H[:, :1], K, rcond=None)[0][0]
    assert np.allclose(sol, P[0], atol=1e-12)


# ------------------------------------------------------------------ Algorithm 2
def test_encode_greedy_step_is_optimal_and_residual_matches():
    n, D, b = 33, 16, 12
    K = _keys(n, D)
    P = RNG.standard_normal((b, D)) * 0.3
    bits, rn = O.encode(K, P)
    h = 2.0 * bits - 1.0
    assert np.allclose(rn, np.linalg.norm(K - h @ P, axis=1), atol=1e-12)      # Eq. 8
    for row in range(n):
        r = K[row].copy()
        for i in range(b):
            u = h[row, i]
            assert np.linalg.norm(r - u * P[i]) <= np.linalg.norm(r + u * P[i]) + 1e-12
            r = r - u * P[i]


def test_encode_orthogonal_rows_reduce_to_sign_projection():
    n, D, b = 100, 32, 16
    Q, _ = np.linalg.qr(RNG.standard_normal((D, D)))
    P = (Q[:, :b] * RNG.uniform(0.5, 2.0, b)).T          # orthogonal rows of different length
    K = _keys(n, D)
    bits, _ = O.encode(K, P)
    assert np.array_equal(bits, (K @ P.T >= 0).astype(np.uint8))
    plain, _ = O.encode(K, P, residual_correction=False)
    assert np.array_equal(bits, plain)
    # exact recovery of a signed sum of rows
    hh = np.where(RNG.random((5, b)) < 0.5, -1.0, 1.0)
    bits2, rn2 = O.encode(hh @ P, P)
    assert np.array_equal(bits2, (hh > 0).astype(np.uint8))
    assert np.max(rn2) < 1e-12


def test_encode_matches_gram_form():
    # t_i = k.P_i - sum_{j<i} u_j (P_j.P_i): same decisions as updating the residual.
    n, D, b = 64, 20, 24
    K = _keys(n, D)
    P = RNG.standard_normal((b, D)) * 0.4
    bits, _ = O.encode(K, P)
    Gm = P @ P.T
    T = K @ P.T
    for row in range(n):
        t = T[row].copy()
        for i in range(b):
            u = 1.0 if t[i] >= 0 else -1.0
            assert int(u > 0) == bits[row, i]
            t[i + 1:] -= u * Gm[i, i + 1:]


def test_encode_nonorthogonal_differs_from_plain_sign():
    # the residual update is part of the hash function (guards against dropping it)
    K = _keys(512, 32)
    vs = RNG.standard_normal((32, 32))
    P, _, _ = O.fit(K, vs)
    a, ra = O.encode(K, P)
    c, rc = O.encode(K, P, residual_correction=False)
    assert np.mean(a != c) > 0.05
    assert np.linalg.norm(ra) < np.linalg.norm(rc)


def test_pack_layout_and_storage_facts():
    f = _facts()
    bits = np.zeros((3, 128), dtype=np.uint8)
    bits[0, 0] = 1; bits[1, 63] = 1; bits[2, 64] = 1; bits[2, 127] = 1
    w = O.pack_bits(bits)
    assert w.shape == (3, 2) and w.dtype == np.uint64
    assert int(w[0, 0]) == 1 and int(w[1, 0]) == 1 << 63 and int(w[2, 0]) == 0
    assert int(w[2, 1]) == (1 | (1 << 63))
    r = RNG.integers(0, 2, (17, 256)).astype(np.uint8)
    assert np.array_equal(O.unpack_bits(O.pack_bits(r), 256), r)
    assert O.codes_bytes(1, 64) == f["code_bytes_per_key_at_64_bits"]
    assert f["kv_bytes_per_key_bf16_d128"] // O.codes_bytes(1, 64) == f["code_to_kv_ratio_inverse"]


# ------------------------------------------------------------------ query hash
def test_query_hash_scale_invariance_and_range():
    f = _facts()
    G, D, b = 4, 32, 64
    P = RNG.standard_normal((b, D))
    q = RNG.standard_normal((G, D))
    for mode in (O.HAMMING, O.WEIGHTED7):
        _, s1, a1 = O.query_hash(q, P, mode)
        for alpha in (0.25, 2.0, 1024.0):          # powers of two: exact in floating point
            _, s2, a2 = O.query_hash(alpha * q, P, mode)
            assert np.array_equal(s1, s2) and np.array_equal(a1, a2)
        _, s3, _ = O.query_hash(3.7 * q, P, mode)
        assert np.array_equal(s1, s3)
    _, s, a = O.query_hash(q, P, O.WEIGHTED7)
    assert a.min() >= 0 and a.max() == f["query_magnitude_max"]
    assert np.all(a.max(axis=1) == 127)            # abs-max scaling puts the largest entry of each head at 127
    p = q @ P.T
    # quantised projection approximates the real one up to the per-head scale (half a step)
    for g in range(G):
        step = np.abs(p[g]).max() / 127.0
        assert np.max(np.abs(s[g] * a[g] * step - p[g])) <= 0.5 * step + 1e-12
    _, s, a = O.query_hash(q, P, O.HAMMING)
    assert np.all(a == 1)
    assert np.array_equal(s, np.where(p >= 0, 1.0, -1.0))


# ------------------------------------------------------------------ hash score
def test_hamming_identity():
    b = 128
    for _ in range(20):
        cq = RNG.integers(0, 2, b).astype(np.uint8)
        ck = RNG.integers(0, 2, (1, b)).astype(np.uint8)
        s = (2.0 * cq - 1.0)[None, :]
        sc = O.hash_scores(ck, s, np.ones((1, b), dtype=np.int64))[0]
        d = O.hamming_distance(O.pack_bits(cq[None])[0], O.pack_bits(ck)[0])
        assert d == int(np.sum(cq != ck[0]))
        assert d * 2 == b - sc                     # d_H = (b - <c_q, c_k>) / 2


def test_alg3_bitplanes_equal_integer_dot_exhaustive_8bit():
    f = _facts()
    b = 8
    a = np.array([127, 0, 1, 64, 3, 126, 85, 42], dtype=np.int64)
    planes = O.magnitude_planes(a)
    assert planes.shape[0] == f["magnitude_planes"]
    for sbits in range(0, 256, 7):
        s_neg = np.array([(sbits >> j) & 1 for j in range(b)], dtype=np.uint8)
        s = 1 - 2 * s_neg.astype(np.int64)
        for hb in range(256):
            h_bits = np.array([(hb >> j) & 1 for j in range(b)], dtype=np.uint8)
            h = 2 * h_bits.astype(np.int64) - 1
            want = int(np.sum(h * s * a))
            # key bit 1 means +1, query sign bit 1 means negative (sign-magnitude): XOR is 1 exactly
            # where the product h*s is +1.
            got = O.hash_score_alg3(h_bits, s_neg, planes)
            assert got == want
            assert O.hash_scores(h_bits[None], s[None].astype(np.float64), a[None])[0] == want


def test_alg3_random_wide_and_group_collapse():
    for b in (64, 128, 256):
        G, n = 4, 50
        bits = RNG.integers(0, 2, (n, b)).astype(np.uint8)
        P = RNG.standard_normal((b, 16))
        q = RNG.standard_normal((G, 16))
        for mode in (O.HAMMING, O.WEIGHTED7):
            _, s, a = O.query_hash(q, P, mode)
            sc = O.hash_scores(bits, s, a)
            A = O.collapsed_weights(s, a)
            h = 2 * bits.astype(np.int64) - 1
            assert np.array_equal(sc, h @ A)                         # sum of head scores == <A, h>
            for i in range(0, n, 7):
                tot = 0
                for g in range(G):
                    pos = (s[g] > 0).astype(np.uint8)                # sign word in "1 = positive" polarity
                    agree = 1 - np.bitwise_xor(bits[i], pos)         # product h*s is +1
                    planes = O.magnitude_planes(a[g])
                    c = sum((int(np.count_nonzero(agree & planes[j])) -
                             int(np.count_nonzero((1 - agree) & planes[j]))) << j for j in range(7))
                    tot += c
                assert tot == sc[i]
            if mode == O.HAMMING:
                assert np.all((sc - G * b) % 2 == 0)                 # S = G*b (mod 2)


# ------------------------------------------------------------------ top-k
def test_topk_matches_bruteforce_with_ties():
    for n, k in ((1, 1), (10, 3), (64, 64), (200, 17), (200, 1)):
        sc = RNG.integers(-5, 6, n)
        want = sorted(sorted(range(n), key=lambda i: (-int(sc[i]), i))[:k])
        assert list(O.topk(sc, k)) == want
    sc = np.array([3, 9, 9, 1, 9])
    assert list(O.topk(sc, 1)) == [1]
    assert list(O.topk(sc, 2)) == [1, 2]
    assert list(O.topk(sc, 5)) == [0, 1, 2, 3, 4]


def test_budget_rounding():
    assert O.budget(4096, 20000) == 82          # 2 % of 4096 keys, rounded up
    assert O.budget(32768, 20000) == 656
    assert O.budget(131072, 20000) == 2622
    assert O.budget(100, 20000, count=2048) == 100
    assert O.budget(5000, 20000, count=1024) == 1024
    assert O.budget(0, 20000) == 0


# ------------------------------------------------------------------ attention
def test_attend_full_budget_is_dense_softmax_attention():
    torch = pytest.importorskip("torch")
    G, D, n = 4, 32, 77
    q = RNG.standard_normal((G, D)); K = _keys(n, D); V = RNG.standard_normal((n, D))
    out = O.attend(q, K, V, np.arange(n))
    ref = torch.softmax(torch.from_numpy(q) @ torch.from_numpy(K).T / math.sqrt(D), dim=-1) @ torch.from_numpy(V)
    assert np.allclose(out, ref.numpy(), atol=1e-12)
    # k = 1 returns the value row; permutation and logit-shift invariance; explicit scale
    assert np.allclose(O.attend(q, K, V, np.array([5])), np.tile(V[5], (G, 1)))
    idx = RNG.choice(n, 20, replace=False)
    a = O.attend(q, K, V, np.sort(idx)); bb = O.attend(q, K, V, idx)
    assert np.allclose(a, bb, atol=1e-13)
    Kshift = K + 0.0
    qn = q / np.linalg.norm(q, axis=1, keepdims=True)
    assert np.allclose(O.attend(q, K, V, idx, sm_scale=0.5),
                       O.attend(2 * q, K, V, idx, sm_scale=0.25), atol=1e-12)


def test_decode_unit_budget_n_equals_dense():
    G, D, n, b = 2, 16, 40, 64
    K = _keys(n, D); V = RNG.standard_normal((n, D)); q = RNG.standard_normal((G, D))
    P, _, _ = O.fit(K, RNG.standard_normal((b, D)))
    bits, _ = O.encode(K, P)
    r = O.decode_unit(q, K, V, bits, P, ppm=1000000)
    assert list(r["idx"]) == list(range(n))
    assert np.allclose(r["out"], O.attend(q, K, V, np.arange(n)), atol=1e-13)
    r2 = O.decode_unit(q, K, V, bits, P, ppm=20000)
    assert len(r2["idx"]) == 1 and r2["scores"][r2["idx"][0]] == r2["scores"].max()


def test_bf16_rounding_matches_torch():
    torch = pytest.importorskip("torch")
    x = RNG.standard_normal(10000).astype(np.float32) * np.float32(37.0)
    x[:4] = np.array([1.00390625, 1.01171875, 0.0, -1.00390625], dtype=np.float32)   # ties
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_bf16(x), want)


def test_replay_with_adoption_flags_only_real_mismatches():
    n, D, b = 50, 16, 32
    K = _keys(n, D); P = RNG.standard_normal((b, D)) * 0.3
    bits, _ = O.encode(K, P)
    hard, amb = O.replay_encode_with_adoption(K, P, bits)
    assert not hard.any() and not amb.any()
    bad = bits.copy(); bad[3, 5] ^= 1
    hard, amb = O.replay_encode_with_adoption(K, P, bad)
    assert hard[3, 5] and hard.sum() >= 1 and not hard[:3].any()


# ------------------------------------------------------------------ error-aware safeguard
def test_eas_set_bruteforce_and_union():
    err = np.array([0.5, 2.0, 2.0, 0.1, 3.0, 2.0])
    assert list(O.eas_set(err, 1)) == [4]
    assert list(O.eas_set(err, 3)) == [1, 2, 4]          # ties at 2.0 go to the lowest indices
    assert list(O.eas_set(err, 10)) == [0, 1, 2, 3, 4, 5]
    assert list(O.eas_set(err, 0)) == []
    r = RNG.random(300)
    for m in (1, 7, 299):
        want = sorted(sorted(range(300), key=lambda i: (-r[i], i))[:m])
        assert list(O.eas_set(r, m)) == want
    assert list(O.eas_union([1, 5, 9], [5, 2])) == [1, 2, 5, 9]


def test_reconstruction_error_identity_from_decision_values():
    # ||k - h P||^2 = ||k||^2 - 2 sum_i |t_i| + trace(P P^T), t_i = decision value of bit i in Algorithm 2:
    # (the by-product a sweep-based encoder can use instead of forming the residual)
    n, D, b = 40, 24, 16
    K = _keys(n, D); P = RNG.standard_normal((b, D)) * 0.4
    bits, rn = O.encode(K, P)
    for row in range(n):
        r = K[row].copy(); tsum = 0.0
        for i in range(b):
            t = float(r @ P[i]); tsum += abs(t)
            r = r - (1.0 if t >= 0 else -1.0) * P[i]
        rhs = float(K[row] @ K[row]) - 2.0 * tsum + float(np.trace(P @ P.T))
        assert abs(rn[row] ** 2 - rhs) <= 1e-9 * max(1.0, float(K[row] @ K[row]))


def test_decode_unit_with_safeguard_set():
    G, D, n, b = 2, 16, 200, 64
    K = _keys(n, D); V = RNG.standard_normal((n, D)); q = RNG.standard_normal((G, D))
    P, _, _ = O.fit(K, RNG.standard_normal((b, D)))
    bits, err = O.encode(K, P)
    s_err = O.eas_set(err, 4)
    plain = O.decode_unit(q, K, V, bits, P, ppm=100000)                 # k = 20
    r = O.decode_unit(q, K, V, bits, P, ppm=100000, s_err=s_err)
    assert len(r["hash_idx"]) == 16 and set(r["hash_idx"]) <= set(plain["idx"])   # top-16 is a prefix of top-20
    assert set(s_err) <= set(r["idx"]) and 16 <= len(r["idx"]) <= 20
    assert np.allclose(r["out"], O.attend(q, K, V, r["idx"]), atol=1e-13)
    tiny = O.decode_unit(q, K, V, bits, P, ppm=0, count=3, s_err=s_err)   # budget below the safeguard size
    assert list(tiny["idx"]) == list(s_err[:3]) and len(tiny["hash_idx"]) == 0


def test_fit_power_iteration_finds_the_sign_of_the_top_singular_vector():
    """Section "Binary Principal Components Finding": u = sign((R R^T)^n R v*^T) tends to the sign pattern of R's largest
    left singular vector as n grows (library SVD as the outside reference), even from a start that is nearly
    orthogonal to the top right singular vector, where the printed n = 0 rule picks up other directions."""
    rng = np.random.default_rng(77)
    N, D = 400, 16
    a = rng.standard_normal(N); a /= np.linalg.norm(a)
    bvec = rng.standard_normal(D); bvec /= np.linalg.norm(bvec)
    K = 40.0 * np.outer(a, bvec) + 0.5 * rng.standard_normal((N, D))
    U, S, Vt = np.linalg.svd(K, full_matrices=False)
    assert S[0] > 3 * S[1]
    top = np.sign(U[:, 0])
    # a start direction with only a small component along the top right singular vector
    g = rng.standard_normal(D)
    g -= (g @ Vt[0]) * Vt[0]
    v0 = (g / np.linalg.norm(g) + 0.02 * Vt[0])[None, :]
    _, H0, _ = O.fit(K, v0, power_iters=0)
    _, H8, _ = O.fit(K, v0, power_iters=8)
    agree0 = max(np.mean(H0[:, 0] == top), np.mean(H0[:, 0] == -top))
    agree8 = max(np.mean(H8[:, 0] == top), np.mean(H8[:, 0] == -top))
    assert agree8 == 1.0
    assert agree0 < 0.9
    # and the first binary component then removes more of the matrix
    _, _, tr0 = O.fit(K, v0, power_iters=0)
    _, _, tr8 = O.fit(K, v0, power_iters=8)
    assert tr8[1] < tr0[1]


def test_fit_power_iteration_zero_is_algorithm_1_and_residual_gram_downdate():
    """n = 0 reproduces Algorithm 1 exactly; and one greedy step changes the residual's Gram matrix by a rank-one term,
    (R - u^T v)^T (R - u^T v) = R^T R - N v^T v (because u R = N v and u u^T = N), the closed form that lets
    (R R^T)^n R v*^T = R (R^T R)^n v*^T be evaluated without extra passes over R."""
    rng = np.random.default_rng(5)
    K = rng.standard_normal((300, 12)) * np.linspace(0.2, 3.0, 12)
    vs = rng.standard_normal((6, 12))
    Pa, Ha, _ = O.fit(K, vs)
    Pb, Hb, _ = O.fit(K, vs, power_iters=0)
    assert np.array_equal(Pa, Pb) and np.array_equal(Ha, Hb)
    R = K.copy()
    N = R.shape[0]
    C = R.T @ R
    for i in range(3):
        z = np.linalg.matrix_power(C, 2) @ vs[i]
        u = O.sign_pm1(R @ z)
        w = R @ vs[i]
        for _ in range(2):
            w = R @ (R.T @ w)
        assert np.array_equal(u, O.sign_pm1(w))                     # R (R^T R)^n v = (R R^T)^n R v
        v = (u @ R) / N
        R = R - np.outer(u, v)
        C = C - N * np.outer(v, v)
        assert np.allclose(C, R.T @ R, rtol=1e-10, atol=1e-9)


def test_quality_yardsticks_against_brute_force_and_closed_forms():
    """TOPK (Oracle) baseline and the output-similarity measure (appendix "Baseline Methods" and the cosine table):
    exact_topk against a brute-force rank count, dense attention against attention over the full index set and the
    uniform-logit closed form, recall and cosine on hand-made cases."""
    rng = np.random.default_rng(11)
    K = rng.standard_normal((57, 6)); K[9] = K[3]; K[20] = K[3]          # exact ties
    q = rng.standard_normal(6)
    k = 10
    got = O.exact_topk(q, K, k)
    s = K @ q
    # brute force: key i is selected iff fewer than k keys beat it (larger score, or equal score and lower index)
    beats = [(np.sum(s > s[i]) + np.sum((s == s[i]) & (np.arange(57) < i))) < k for i in range(57)]
    assert np.array_equal(got, np.nonzero(beats)[0])
    assert O.exact_topk(q, K, 0).size == 0 and np.array_equal(O.exact_topk(q, K, 99), np.arange(57))
    # dense attention: all-zero query -> uniform weights -> the mean of V
    V = rng.standard_normal((57, 6))
    out = O.dense_attend(np.zeros((2, 6)), K, V)
    assert np.allclose(out, np.tile(V.mean(0), (2, 1)))
    qg = rng.standard_normal((3, 6))
    assert np.allclose(O.dense_attend(qg, K, V), O.attend(qg, K, V, np.arange(57)))
    # selecting every key makes sparse = dense; recall and cosine on small cases
    assert O.selection_recall([1, 2, 3, 4], [2, 4, 6, 8]) == 0.5
    assert O.selection_recall([], []) == 1.0
    assert abs(O.cosine_similarity([1, 0], [1, 1]) - 2 ** -0.5) < 1e-15
    assert O.cosine_similarity([1, 2, 3], [-2, -4, -6]) == -1.0
