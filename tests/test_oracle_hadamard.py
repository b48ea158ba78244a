"""Pins for the oracle's Hadamard matrices and rotation (no GPU).

Each check compares the oracle with something it does not compute itself: the
defining identity H H^T = n I in exact integers, a library construction, field
arithmetic redone here by brute force, closed forms of the transform."""
import numpy as np
import pytest
import scipy.linalg

from oracle import smoothrot_oracle as orc


@pytest.mark.parametrize("n", [1, 2, 128, 512, 4096])
def test_sylvester_is_hadamard_and_matches_library(n):
    H = orc.sylvester(n).astype(np.int64)
    assert set(np.unique(H)) <= {-1, 1}
    if n <= 512:
        assert np.array_equal(H @ H.T, n * np.eye(n, dtype=np.int64))
    else:  # exact in float32: every partial sum is an integer below 2^24
        Hf = H.astype(np.float32)
        assert np.array_equal(Hf @ Hf.T, n * np.eye(n, dtype=np.float32))
    assert np.array_equal(H, scipy.linalg.hadamard(n).astype(np.int64))


def test_sylvester_recursion_block_form():
    H = orc.sylvester(64).astype(int)
    h = orc.sylvester(32).astype(int)
    assert np.array_equal(H, np.block([[h, h], [h, -h]]))


# --- GF(27) redone here, independently: polynomials over GF(3) as tuples -------
def _polymulmod(a, b):
    """(a0,a1,a2)*(b0,b1,b2) mod (x^3 + 2x + 1) over GF(3), by long division."""
    p = [0] * 5
    for i, ai in enumerate(a):
        for j, bj in enumerate(b):
            p[i + j] = (p[i + j] + ai * bj) % 3
    mod = [1, 2, 0, 1]  # 1 + 2x + 0x^2 + x^3
    for deg in (4, 3):
        c = p[deg]
        if c:
            for t in range(4):
                p[deg - 3 + t] = (p[deg - 3 + t] - c * mod[t]) % 3
    return tuple(p[:3])


def _elem(e):
    return (e % 3, (e // 3) % 3, e // 9)


def _idx(c):
    return c[0] + 3 * c[1] + 9 * c[2]


def test_gf27_polynomial_is_irreducible_and_field_ops_match():
    # a cubic over GF(3) is irreducible iff it has no root in GF(3)
    assert all((t ** 3 + 2 * t + 1) % 3 != 0 for t in range(3))
    for a in range(27):
        for b in range(27):
            assert orc.gf27_mul(a, b) == _idx(_polymulmod(_elem(a), _elem(b)))
            d = tuple((x - y) % 3 for x, y in zip(_elem(a), _elem(b)))
            assert orc.gf27_sub(a, b) == _idx(d)
    # x (index 3) generates the 26 non-zero elements
    seen, cur = set(), (1, 0, 0)
    for _ in range(26):
        seen.add(cur)
        cur = _polymulmod(cur, (0, 1, 0))
    assert len(seen) == 26 and cur == (1, 0, 0)


def test_quadratic_character():
    squares = {_idx(_polymulmod(_elem(y), _elem(y))) for y in range(1, 27)}
    assert len(squares) == 13
    assert sorted(squares) == [1, 6, 7, 8, 9, 11, 12, 13, 15, 16, 20, 22, 25]
    for e in range(27):
        want = 0 if e == 0 else (1 if e in squares else -1)
        assert orc.gf27_chi(e) == want
    # q = 27 = 3 mod 4  =>  -1 is a non-square, so chi is odd and Q is skew
    assert orc.gf27_chi(2) == -1  # the element -1 = 2


def test_paley28_structure():
    H = orc.paley28().astype(np.int64)
    assert H.shape == (28, 28) and set(np.unique(H)) == {-1, 1}
    assert np.array_equal(H @ H.T, 28 * np.eye(28, dtype=np.int64))
    assert np.array_equal(H.T @ H, 28 * np.eye(28, dtype=np.int64))
    S = H - np.eye(28, dtype=np.int64)
    assert np.array_equal(S, -S.T)                    # skew part
    Q = S[1:, 1:]
    assert np.all(Q.sum(axis=1) == 0) and np.all(Q.sum(axis=0) == 0)
    assert np.all(np.diag(Q) == 0)
    assert np.all((Q == 1).sum(axis=1) == 13) and np.all((Q == -1).sum(axis=1) == 13)
    assert np.array_equal(Q @ Q.T, 27 * np.eye(27, dtype=np.int64) - np.ones((27, 27), np.int64))
    assert np.all(H[0] == 1) and H[0, 0] == 1 and np.all(H[1:, 0] == -1)
    # Q[a, b] depends on a - b only: Q[a, b] = Q[a - b, 0]
    for a in range(27):
        for b in range(27):
            d = _idx(tuple((x - y) % 3 for x, y in zip(_elem(a), _elem(b))))
            assert Q[a, b] == Q[d, 0]


def test_kronecker_index_order_and_orthogonality_small():
    K = 28 * 8
    H = orc.hadamard_matrix(K).astype(np.int64)
    assert np.array_equal(H @ H.T, K * np.eye(K, dtype=np.int64))
    P, Wn = orc.paley28().astype(int), orc.sylvester(8).astype(int)
    for (a, b, a2, b2) in [(0, 0, 0, 0), (3, 5, 17, 2), (27, 7, 1, 6), (12, 1, 12, 1)]:
        assert H[a * 8 + b, a2 * 8 + b2] == P[a, a2] * Wn[b, b2]


def test_order_14336_rows_are_orthogonal():
    """H H^T = 14336 I, checked exactly on a seeded sample of rows against all
    rows (float32 sums of +-1 are exact up to 2^24), and in full through the
    factors: (A x B)(A x B)^T = (A A^T) x (B B^T)."""
    K = 14336
    H = orc.hadamard_matrix(K)
    assert H.shape == (K, K) and H.dtype == np.int8
    rng = np.random.default_rng(5)
    rows = np.sort(rng.choice(K, size=48, replace=False))
    G = H[rows].astype(np.float32) @ H.astype(np.float32).T
    want = np.zeros_like(G)
    want[np.arange(len(rows)), rows] = K
    assert np.array_equal(G, want)
    A = orc.paley28().astype(np.int64)
    B = orc.sylvester(512).astype(np.int64)
    # (A x B)(A x B)^T = (A A^T) x (B B^T) = (28 I) x (512 I) = 14336 I
    assert np.array_equal(A @ A.T, 28 * np.eye(28, dtype=np.int64))
    assert np.array_equal(B @ B.T, 512 * np.eye(512, dtype=np.int64))


def test_split_order():
    assert orc.split_order(4096) == (1, 4096)
    assert orc.split_order(14336) == (28, 512)
    assert orc.split_order(28) == (28, 1)
    assert orc.split_order(12) == (12, 1)
    assert orc.split_order(5120) == (20, 256)
    assert orc.split_order(3072) == (12, 256)
    for bad in (0, 3, 11008, 28 * 3, 36, 60, 44):
        with pytest.raises(ValueError):
            orc.split_order(bad)


@pytest.mark.parametrize("q", [11, 19])
def test_paley_prime_structure(q):
    """Orders 12 and 20: the same structure facts as for order 28, and the character checked
    against Euler's criterion e^((q-1)/2) mod q (another route to it than listing squares)."""
    n = q + 1
    H = orc.paley_prime(q).astype(np.int64)
    assert H.shape == (n, n) and set(np.unique(H)) == {-1, 1}
    assert np.array_equal(H @ H.T, n * np.eye(n, dtype=np.int64))
    assert np.array_equal(H.T @ H, n * np.eye(n, dtype=np.int64))
    S = H - np.eye(n, dtype=np.int64)
    assert np.array_equal(S, -S.T)
    Q = S[1:, 1:]
    assert np.all(np.diag(Q) == 0) and np.all(Q.sum(axis=1) == 0) and np.all(Q.sum(axis=0) == 0)
    assert np.array_equal(Q @ Q.T, q * np.eye(q, dtype=np.int64) - np.ones((q, q), np.int64))
    assert np.all(H[0] == 1) and np.all(H[1:, 0] == -1)
    for e in range(q):
        euler = pow(e, (q - 1) // 2, q)
        assert orc.legendre(e, q) == {0: 0, 1: 1, q - 1: -1}[euler]
    for a in range(q):                      # circulant: Q[a, b] = chi(a - b)
        for b in range(q):
            assert Q[a, b] == Q[(a - b) % q, 0]
    assert orc.legendre(-1, q) == -1        # q = 3 mod 4: -1 is a non-square, Q is skew


@pytest.mark.parametrize("K", [12 * 8, 20 * 16])
def test_kronecker_with_orders_12_and_20(K):
    base, n = orc.split_order(K)
    H = orc.hadamard_matrix(K).astype(np.int64)
    assert np.array_equal(H @ H.T, K * np.eye(K, dtype=np.int64))
    P, Wn = orc.base_matrix(base).astype(int), orc.sylvester(n).astype(int)
    rng = np.random.default_rng(K)
    for _ in range(16):
        a, a2 = rng.integers(base, size=2)
        b, b2 = rng.integers(n, size=2)
        assert H[a * n + b, a2 * n + b2] == P[a, a2] * Wn[b, b2]


@pytest.mark.parametrize("K", [128, 512, 28 * 4, 28 * 16, 1024, 12 * 32, 20 * 8])
def test_fast_rotation_equals_dense_definition(K):
    rng = np.random.default_rng(K)
    x = rng.standard_normal((5, K))
    pre = rng.standard_normal(K)
    for p in (None, pre):
        a, b = orc.rotate(x, p, K), orc.rotate_dense(x, p, K)
        assert np.abs(a - b).max() <= 1e-12 * np.abs(b).max()


@pytest.mark.parametrize("K", [4096, 14336])
def test_fast_rotation_equals_dense_on_full_width_rows(K):
    rng = np.random.default_rng(K)
    x = rng.standard_normal((2, K))
    pre = rng.uniform(0.5, 2.0, K)
    H = orc.hadamard_matrix(K)
    want = np.zeros((2, K))
    for c0 in range(0, K, 2048):            # dense product, a column block at a time
        want[:, c0:c0 + 2048] = (x * pre) @ H[:, c0:c0 + 2048].astype(np.float64)
    want /= np.sqrt(K)
    got = orc.rotate(x, pre, K)
    assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()


@pytest.mark.parametrize("K", [128, 4096, 28 * 32, 14336, 3072, 5120])
def test_rotation_closed_forms(K):
    rng = np.random.default_rng(K + 1)
    base, n = orc.split_order(K)
    # unit vector: every output has magnitude c / sqrt(K), signs = row j of H
    j, c = int(rng.integers(K)), 3.75
    e = np.zeros((1, K)); e[0, j] = c
    y = orc.rotate(e, None, K)
    assert np.allclose(np.abs(y), c / np.sqrt(K), rtol=1e-14, atol=0)
    if base == 1:
        signs = np.array([1 - 2 * (bin(j & k).count("1") & 1) for k in range(K)])
        assert np.array_equal(np.sign(y[0]).astype(int), signs)
        # constant vector -> sqrt(K) * c * e_0 (first column of a Sylvester matrix is all ones)
        y1 = orc.rotate(np.full((1, K), c), None, K)
        want = np.zeros(K); want[0] = c * np.sqrt(K)
        assert np.allclose(y1[0], want, rtol=1e-13, atol=1e-9)
    else:
        # first row of H28 x Hn is all +1: e_0 -> constant c / sqrt(K)
        e0 = np.zeros((1, K)); e0[0, 0] = c
        assert np.allclose(orc.rotate(e0, None, K), c / np.sqrt(K), rtol=1e-14)
    # Parseval and linearity
    x = rng.standard_normal((3, K)); pre = rng.standard_normal(K)
    y = orc.rotate(x, pre, K)
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x * pre, axis=1), rtol=1e-12)
    z = rng.standard_normal((3, K))
    assert np.allclose(orc.rotate(2.5 * x - z, pre, K), 2.5 * y - orc.rotate(z, pre, K),
                       rtol=1e-10, atol=1e-10)
    # the rotation is orthogonal: applying H^T / sqrt(K) brings x * pre back
    H = None
    if K <= 4096:
        H = orc.hadamard_matrix(K).astype(np.float64)
        assert np.allclose((y @ H.T) / np.sqrt(K), x * pre, rtol=1e-10, atol=1e-10)


@pytest.mark.parametrize("K", [128, 28 * 16])
def test_function_preservation_eq2(K):
    """Eq. 2:  X W^T == (X diag(s)^-1 diag(d) H_n)(H_n^T diag(d) diag(s) W^T), fp64, 1e-10."""
    rng = np.random.default_rng(11)
    X = rng.standard_normal((9, K)); X[:2, 5] *= 800.0
    W = rng.standard_normal((13, K)) * 0.02
    s = rng.uniform(0.05, 40.0, K)
    d = rng.integers(0, 2, K) * 2.0 - 1.0
    xr = orc.rotate(X, d / s, K)
    wr = orc.rotate(W, s * d, K)
    Y0, Y1 = X @ W.T, xr @ wr.T
    assert np.abs(Y0 - Y1).max() <= 1e-10 * np.abs(Y0).max()
