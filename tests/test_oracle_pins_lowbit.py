"""Pins of the oracle's Appendix C functions (1-bit weights and activations, ternary gradients, XNOR + popcount
products, Algorithm 1) against what the mathematics fixes: hand-written values, plain integer products, exact
cases, and the binomial bound on the stochastic ternarisation.  CPU only."""
import numpy as np

from oracle import qbp_oracle as O


def _pm1(shape, seed):
    return (np.random.Generator(np.random.PCG64(seed)).integers(0, 2, shape) * 2 - 1).astype(np.int8)


def test_binarize_sign_convention_and_bit_order():
    x = np.array([0.0, -0.0, 1e-30, -1e-30, 3.0, -3.0], dtype=np.float32)
    assert O.binarize(x).tolist() == [1, 1, 1, -1, 1, -1]           # x >= 0 -> +1 (so does -0.0)
    # 35 columns: bits 0, 3 and 34 set -> word 0 = 1 + 8, word 1 = bit 2; the spare bits stay 0
    row = -np.ones((1, 35), dtype=np.int8); row[0, [0, 3, 34]] = 1
    assert O.pack_bits(row).tolist() == [[9, 4]]
    tern = np.zeros((1, 35), dtype=np.int8); tern[0, 1] = -1; tern[0, 33] = 1
    assert O.pack_bits(tern, mask=True).tolist() == [[2, 2]] and O.pack_bits(tern).tolist() == [[0, 2]]


def test_binarised_gaussian_vector_keeps_the_papers_angle():
    """The paper's supplement prints the angle between a Gaussian vector and its sign binarisation: arccos sqrt(2 / pi),
    about 37 degrees (tests/golden/paper_constants.txt)."""
    import math
    from pathlib import Path
    val = tol = None
    for line in (Path(__file__).parent / "golden" / "paper_constants.txt").read_text().splitlines():
        f = line.split("#")[0].split()
        if len(f) == 3 and f[0] == "binary_quantization_angle_degrees":
            val, tol = float(f[1]), float(f[2])
    x = np.random.Generator(np.random.PCG64(3)).normal(0, 1, 200000).astype(np.float32)
    b = O.binarize(x).astype(np.float64)
    cos = float(x.astype(np.float64) @ b) / (np.linalg.norm(x.astype(np.float64)) * np.linalg.norm(b))
    angle = math.degrees(math.acos(cos))
    assert abs(angle - val) <= tol and abs(angle - math.degrees(math.acos(math.sqrt(2 / math.pi)))) < 0.2


def test_xnor_popcount_product_is_the_plus_minus_one_dot_product():
    for M, N, K in ((5, 7, 70), (3, 4, 32), (2, 2, 1), (6, 5, 257)):
        A = _pm1((M, K), 1 + K); B = _pm1((N, K), 2 + K)
        want = A.astype(np.int64) @ B.astype(np.int64).T
        assert np.array_equal(O.xnor_gemm(O.pack_bits(A), O.pack_bits(B), K), want)
    a = _pm1((1, 100), 9)
    assert O.xnor_gemm(O.pack_bits(a), O.pack_bits(a), 100)[0, 0] == 100          # a . a = K
    assert O.xnor_gemm(O.pack_bits(a), O.pack_bits(-a), 100)[0, 0] == -100        # a . (-a) = -K


def test_sample_index_sits_in_the_last_counter_word():
    seed, tid = 0x1234567890ABCDEF, 77
    for i in (0, 1, 5, 4 * (1 << 32) + 2):
        assert O.random_word_sample(seed, tid, i, 0) == O.random_word(seed, tid, i)
        for k in (1, 19):
            j = i >> 2
            want = O.philox4x32_10([j & 0xFFFFFFFF, j >> 32, tid, k], [seed & 0xFFFFFFFF, seed >> 32])[i & 3]
            assert O.random_word_sample(seed, tid, i, k) == int(want)


def test_stochastic_ternarisation_exact_cases():
    g = np.array([2.0, -2.0, 0.0, 0.5, -1.0, 1e-9], dtype=np.float32)
    for k in range(50):
        t, s = O.stc_tern(g, seed=3, tensor_id=4, sample=k)
        assert s == np.float32(2.0)                                   # the scale is max |g|
        assert t[0] == 1 and t[1] == -1 and t[2] == 0                 # |g| = s: always kept; g = 0: never
        assert set(t.tolist()) <= {-1, 0, 1}
        assert np.all((t == 0) | (np.sign(t) == np.sign(g)))          # a kept element carries the sign of g
    t, s = O.stc_tern(np.zeros(9, dtype=np.float32))
    assert s == 0 and not t.any()
    a, _ = O.stc_tern(g, 3, 4, 7); b, _ = O.stc_tern(g, 3, 4, 7)
    assert np.array_equal(a, b)                                       # a function of (seed, id, sample, position)


def test_stochastic_ternarisation_is_unbiased_within_the_binomial_bound():
    rng = np.random.Generator(np.random.PCG64(11))
    g = rng.normal(0, 1, 64).astype(np.float32)
    S = 4000
    tot = np.zeros(64)
    for k in range(S):
        t, s = O.stc_tern(g, seed=5, tensor_id=6, sample=k)
        tot += t
    p = np.abs(g.astype(np.float64)) / float(s)
    sigma = float(s) * np.sqrt(p * (1 - p) / S)
    assert np.all(np.abs(float(s) * tot / S - g) <= 4.5 * sigma + 1e-6)          # E[s t] = g
    # the kept fraction is |g| / s, not its square or its root: a coarse check on an element well inside (0, 1)
    i = int(np.argmin(np.abs(p - 0.5)))
    assert abs(abs(tot[i]) / S - p[i]) < 0.05


def test_gated_xnor_product_is_the_ternary_times_binary_dot_product():
    rng = np.random.Generator(np.random.PCG64(12))
    for M, N, K in ((4, 6, 70), (3, 3, 32), (5, 2, 129)):
        T = rng.integers(-1, 2, (M, K)).astype(np.int8); B = _pm1((N, K), 13 + K)
        want = T.astype(np.int64) @ B.astype(np.int64).T
        got = O.gated_xnor_gemm(O.pack_bits(T, mask=True), O.pack_bits(T), O.pack_bits(B), K)
        assert np.array_equal(got, want)


def test_algorithm_1_one_sample_is_one_product_and_many_samples_approach_the_exact_gradient():
    rng = np.random.Generator(np.random.PCG64(14))
    rows, N, K = 8, 3, 4
    g = rng.normal(0, 1, (rows, N)).astype(np.float32); a = _pm1((rows, K), 15)
    t0, s = O.stc_tern(g, seed=8, tensor_id=9, sample=0)
    one = O.tbp_update(g, a, 1, seed=8, tensor_id=9)
    assert np.array_equal(one, float(s) * (a.astype(np.float64).T @ t0.astype(np.float64)))
    three = O.tbp_update(g, a, 3, seed=8, tensor_id=9)
    acc = sum(a.astype(np.int64).T @ O.stc_tern(g, 8, 9, k)[0].astype(np.int64) for k in range(3))
    assert np.array_equal(three, float(s) * acc / 3.0)                # the mean of the samples' products
    S = 3000
    many = O.tbp_update(g, a, S, seed=8, tensor_id=9)
    exact = a.astype(np.float64).T @ g.astype(np.float64)
    assert np.all(np.abs(many - exact) <= 5.0 * float(s) * np.sqrt(rows / S))
