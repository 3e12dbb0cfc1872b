"""Pins for the float64 CPU oracle: it is checked against what the paper and the
mathematics fix, never against itself or against the CUDA path.

Citations are to the paper's sections / equations / algorithms.
"""
import itertools
import os

import numpy as np
import pytest
import scipy.linalg

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
PALEY_ORDERS = [4, 8, 12, 20, 24, 28, 32, 44, 48, 60, 68, 72, 80, 84, 104, 108]


# ----------------------------------------------------------------------------
# independent restatements used only here (second route, pure Python)
# ----------------------------------------------------------------------------
def _chi_prime(a, p):
    a %= p
    if a == 0:
        return 0
    return 1 if a in {(x * x) % p for x in range(1, p)} else -1


def _gf27_mul_py(e, f):
    """Polynomial product in GF(3)[x] reduced by x^3 + 2x + 1 via long division."""
    a = [e % 3, (e // 3) % 3, e // 9]
    b = [f % 3, (f // 3) % 3, f // 9]
    prod = [0] * 5
    for i, j in itertools.product(range(3), range(3)):
        prod[i + j] = (prod[i + j] + a[i] * b[j]) % 3
    mod = [1, 2, 0, 1]  # 1 + 2x + 0x^2 + x^3
    for deg in (4, 3):
        c = prod[deg]
        if c:
            for t in range(4):
                prod[deg - 3 + t] = (prod[deg - 3 + t] - c * mod[t]) % 3
    return prod[0] + 3 * prod[1] + 9 * prod[2]


def _paley_py(m):
    """Algorithm 2 written out again in Python (prime p, or GF(27) for m = 28)."""
    H = np.ones((m, m), dtype=np.int64)
    if m == 28:
        squares = {_gf27_mul_py(x, x) for x in range(1, 27)}

        def chi(i, j):
            a = [i % 3, (i // 3) % 3, i // 9]
            b = [j % 3, (j // 3) % 3, j // 9]
            e = sum(((a[t] - b[t]) % 3) * 3 ** t for t in range(3))
            return 0 if e == 0 else (1 if e in squares else -1)
    else:
        p = m - 1

        def chi(i, j):
            return _chi_prime(i - j, p)
    for i in range(1, m):
        H[i, 0] = -1
        H[0, i] = -1
        for j in range(1, m):
            H[i, j] = -1 if i == j else chi(i - 1, j - 1)
    return H


def _signs(s):
    return [{"+": 1, "-": -1, "0": 0}[c] for c in s]


def _fingerprints():
    out = {}
    for line in open(os.path.join(GOLDEN, "paley_fingerprints.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        out[k] = _signs(v)
    return out


# ----------------------------------------------------------------------------
# Sylvester matrices, Eq. (1)
# ----------------------------------------------------------------------------
def test_sylvester_printed_matrices():
    """H_2 and H_4 exactly as printed in Eq. (1)."""
    blocks, cur = {}, None
    for line in open(os.path.join(GOLDEN, "eq1_sylvester.txt")):
        if line.startswith("#") or not line.strip():
            continue
        if line.startswith("H"):
            cur = int(line.split()[1])
            blocks[cur] = []
        else:
            blocks[cur].append([int(v) for v in line.split()])
    for n, rows in blocks.items():
        assert np.array_equal(oracle.sylvester(n), np.array(rows))


@pytest.mark.parametrize("n", [1, 2, 4, 8, 16, 64, 256])
def test_sylvester_recursion_library_and_closed_form(n):
    H = oracle.sylvester(n).astype(np.int64)
    # Eq. (1) recursion: H_{2n} = [[H, H], [H, -H]]
    if n >= 2:
        h = oracle.sylvester(n // 2).astype(np.int64)
        assert np.array_equal(H, np.block([[h, h], [h, -h]]))
    # library routine with the same natural order
    assert np.array_equal(H, scipy.linalg.hadamard(n) if n > 1 else np.array([[1]]))
    # closed form (-1)^popcount(i & j)
    i, j = np.meshgrid(np.arange(n), np.arange(n), indexing="ij")
    pc = np.vectorize(lambda v: bin(v).count("1"))(i & j)
    assert np.array_equal(H, 1 - 2 * (pc & 1))
    # Appendix A: H H^T = n I
    assert np.array_equal(H @ H.T, n * np.eye(n, dtype=np.int64))


# ----------------------------------------------------------------------------
# Legendre symbol (Section 2.3.3) and Paley construction (Algorithm 2)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("p", [3, 7, 11, 19, 23, 43])
def test_legendre_definition(p):
    for a in range(-2 * p, 2 * p + 1):
        assert oracle.legendre(a, p) == _chi_prime(a, p)
    # Euler's criterion, a textbook identity: (a/p) = a^((p-1)/2) mod p
    for a in range(1, p):
        e = pow(a, (p - 1) // 2, p)
        assert oracle.legendre(a, p) == (1 if e == 1 else -1)
    # exactly (p-1)/2 residues and (p-1)/2 non-residues
    vals = [oracle.legendre(a, p) for a in range(1, p)]
    assert vals.count(1) == vals.count(-1) == (p - 1) // 2


def test_gf27_field():
    """GF(27) = GF(3)[x]/(x^3+2x+1): the modulus has no root in GF(3); x has order 26."""
    for r in range(3):
        assert (r ** 3 + 2 * r + 1) % 3 != 0
    for e, f in itertools.product(range(27), range(27)):
        assert oracle.gf27_mul(e, f) == _gf27_mul_py(e, f)
        assert oracle.gf27_mul(e, f) == oracle.gf27_mul(f, e)
    # x (index 3) is primitive: its powers visit all 26 non-zero elements
    seen, cur = [], 1
    for _ in range(26):
        seen.append(cur)
        cur = oracle.gf27_mul(cur, 3)
    assert cur == 1 and sorted(seen) == list(range(1, 27))
    # quadratic character: squares are the even powers of a primitive element
    for t, e in enumerate(seen):
        assert oracle.gf27_chi(e) == (1 if t % 2 == 0 else -1)
    assert oracle.gf27_chi(0) == 0
    # subtraction is coefficient-wise mod 3
    for e, f in itertools.product(range(27), range(27)):
        g = oracle.gf27_sub(e, f)
        for t in range(3):
            assert ((e // 3 ** t) % 3 - (f // 3 ** t) % 3 - (g // 3 ** t) % 3) % 3 == 0


@pytest.mark.parametrize("m", PALEY_ORDERS)
def test_paley_is_hadamard_and_follows_algorithm2(m):
    H = oracle.hadamard_m(m).astype(np.int64)
    assert set(np.unique(H)) == {-1, 1}
    assert np.array_equal(H @ H.T, m * np.eye(m, dtype=np.int64))      # Appendix A
    # Algorithm 2 structure: H[0,0] = +1; first row, first column, diagonal = -1
    assert H[0, 0] == 1
    assert np.all(H[0, 1:] == -1) and np.all(H[1:, 0] == -1)
    assert np.all(np.diag(H)[1:] == -1)
    assert np.array_equal(H, _paley_py(m))
    # the core is skew: for i != j >= 1, H[i,j] = -H[j,i]  (p = 3 mod 4), so H != H^T
    core = H[1:, 1:] + np.eye(m - 1, dtype=np.int64)
    assert np.array_equal(core, -core.T)


@pytest.mark.parametrize("m", [2, 3, 6, 10, 14, 16, 18, 26, 36])
def test_paley_rejects_orders_without_construction(m):
    # p = m-1 must be a prime = 3 (mod 4) (Section 2.3.3); e.g. p = 5, 13 are = 1 (mod 4)
    with pytest.raises(ValueError):
        oracle.hadamard_m(m)


def test_paley_fingerprints():
    fp = _fingerprints()
    assert [oracle.gf27_chi(e) for e in range(27)] == fp["chi27"]
    assert [oracle.legendre(a, 19) for a in range(19)] == fp["chi19"]
    assert list(oracle.hadamard_m(28)[1]) == fp["h28row1"]
    assert list(oracle.hadamard_m(20)[1]) == fp["h20row1"]


# ----------------------------------------------------------------------------
# Kronecker composition, padding, rotation
# ----------------------------------------------------------------------------
SMALL = [(1, 3), (1, 4), (12, 3), (20, 3), (28, 3), (12, 4), (1, 7), (28, 4)]


@pytest.mark.parametrize("m,k", SMALL)
def test_rotation_equals_dense_matmul(m, k):
    """y = (H_m (x) H_{2^k}) x_pad / sqrt(d'), against an explicit numpy matrix product
    built from this file's own Paley code and scipy's Sylvester matrix."""
    rng = np.random.default_rng(100 * m + k)
    n2 = 1 << k
    dp = m * n2
    Hm = _paley_py(m) if m > 1 else np.array([[1]])
    Hs = scipy.linalg.hadamard(n2)
    Hfull = np.kron(Hm, Hs)
    assert np.array_equal(Hfull @ Hfull.T, dp * np.eye(dp, dtype=np.int64))
    assert np.array_equal(oracle.hadamard_full(m, k), Hfull)
    for d in (dp, dp - 1, dp - n2 // 2, max(1, dp // 3)):
        x = rng.standard_normal(d)
        xp = np.concatenate([x, np.zeros(dp - d)])
        want = Hfull @ xp / np.sqrt(dp)
        for dense in (True, False):
            got = oracle.rotate(x, dp, m, dense=dense)
            np.testing.assert_allclose(got, want, rtol=0, atol=1e-12 * np.abs(want).max())
        # Eq. (2): rotating the zero-padded operand uses only the first d columns of H
        np.testing.assert_allclose(oracle.rotate(x, dp, m), Hfull[:, :d] @ x / np.sqrt(dp),
                                   rtol=0, atol=1e-12 * np.abs(want).max())
        # y = H x, not x H: for the non-symmetric Paley factor the two differ
        if m > 1 and d == dp:
            other = Hfull.T @ xp / np.sqrt(dp)
            assert np.abs(other - want).max() > 1e-3
            np.testing.assert_allclose(oracle.rotate(x, dp, m, transpose=True), other,
                                       rtol=0, atol=1e-12 * np.abs(want).max())


@pytest.mark.parametrize("m,k,d", [(1, 12, 4096), (28, 7, 3584), (20, 10, 18944), (1, 7, 128),
                                   (12, 5, 300), (24, 6, 1536)])
def test_fast_rotation_matches_definition_at_workload_sizes(m, k, d):
    rng = np.random.default_rng(7)
    dp = m << k
    x = rng.standard_t(3, size=d)
    x[rng.integers(0, d, 4)] *= 50
    yd = oracle.rotate(x, dp, m, dense=True)
    yf = oracle.rotate(x, dp, m, dense=False)
    assert np.abs(yd - yf).max() <= 1e-12 * np.abs(yd).max()
    # rotations preserve length (Section 2.3.1)
    assert abs(np.linalg.norm(yd) - np.linalg.norm(x)) <= 1e-12 * np.linalg.norm(x)
    # inverse by the transpose recovers the padded input, zeros in the tail included
    back = oracle.rotate(yf, dp, m, dense=False, transpose=True)
    assert np.abs(back[:d] - x).max() <= 1e-11 * np.abs(x).max()
    assert np.abs(back[d:]).max() <= 1e-11 * np.abs(x).max() if d < dp else True


@pytest.mark.parametrize("m,k", [(1, 6), (1, 12), (20, 4), (28, 7)])
def test_lemma1_and_theorem2(m, k):
    """Lemma 1: x = c e_0 gives |y_i| = c / sqrt(n) for every i.  Theorem 2: the largest
    entry of the normalised matrix is exactly 1/sqrt(n)."""
    dp = m << k
    c = 200.0
    for pos in (0, 1, dp // 2 + 3, dp - 1):
        x = np.zeros(dp)
        x[pos] = c
        y = oracle.rotate(x, dp, m, dense=False)
        np.testing.assert_allclose(np.abs(y), c / np.sqrt(dp), rtol=1e-13)


def test_absmax_experiment():
    """Appendix A.1.2: N(0, 0.1^2) plus a peak of 200 -> max|Hx| close to 200/sqrt(n)."""
    rng = np.random.default_rng(11)
    for n in (256, 1024, 4096):
        x = 0.1 * rng.standard_normal(n)
        x[17] += 200.0
        y = oracle.rotate(x, n, 1, dense=False)
        peak = 200.0 / np.sqrt(n)
        # the noise adds a N(0, 0.1^2) term to every coordinate; its max over n is < 0.5
        assert abs(np.abs(y).max() - peak) < 0.5
        assert np.abs(y).max() < 0.1 * np.abs(x).max()


# ----------------------------------------------------------------------------
# Quantizer (Section 2.1, Section 3.1)
# ----------------------------------------------------------------------------
def _examples():
    for line in open(os.path.join(GOLDEN, "quantizer_examples.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = [s.strip() for s in line.split("|")]
        yield (int(f[0]), f[1] == "literal", float(f[2]), np.array(f[3].split(), dtype=np.float64),
               float(f[4]), np.array(f[5].split(), dtype=np.int32), float(f[6]))


def test_quantizer_hand_worked_examples():
    n = 0
    for bits, literal, alpha, y, delta, codes, err in _examples():
        q, dl = oracle.quantize(y, bits, 0, alpha, literal)
        assert dl[0] == delta
        assert np.array_equal(q, codes)
        assert oracle.clip_error(y, bits, 0, alpha, literal) == err
        n += 1
    assert n == 5


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("group", [0, 8, 32])
@pytest.mark.parametrize("alpha", [1.0, 0.9, 0.5, 0.3])
def test_quantizer_properties(bits, group, alpha):
    rng = np.random.default_rng(bits * 100 + group)
    y = rng.standard_t(3, size=256)
    q, dl = oracle.quantize(y, bits, group, alpha)
    D = 2 ** (bits - 1) - 1
    assert oracle.levels(bits) == D and oracle.levels(bits, True) == 2 ** bits - 1
    assert q.min() >= -D and q.max() <= D
    g = group or 256
    for s in range(256 // g):
        v, c, d_ = y[s * g:(s + 1) * g], q[s * g:(s + 1) * g], dl[s]
        M = np.abs(v).max()
        assert d_ == alpha * M / D
        yh = c * d_
        inside = np.abs(v) <= alpha * M
        assert np.all(np.abs(v - yh)[inside] <= d_ / 2 * (1 + 1e-12))
        # clipped elements sit on the edge of the range: |yhat| = alpha M (Section 3.1)
        np.testing.assert_allclose(np.abs(yh[~inside]), alpha * M, rtol=1e-14)
        assert np.all(np.sign(yh[~inside]) == np.sign(v[~inside]))
        if alpha == 1.0:
            # Section 2.1: the extreme value is preserved
            i = np.argmax(np.abs(v))
            np.testing.assert_allclose(yh[i], v[i], rtol=1e-14)
            assert abs(c[i]) == D
        # the error at alpha = 1 is bounded by n Delta^2 / 4
        if alpha == 1.0:
            assert np.sum((v - yh) ** 2) <= g * d_ ** 2 / 4


def test_quantizer_zero_group_and_ties():
    q, dl = oracle.quantize(np.zeros(16), 3, 8, 0.9)
    assert np.all(q == 0) and np.all(dl == 0)
    assert oracle.clip_error(np.zeros(16), 3, 8, 0.9) == 0.0
    # ties go to the even code: with Delta = 1, 0.5 -> 0, 1.5 -> 2, 2.5 -> 2, -0.5 -> 0
    q, dl = oracle.quantize(np.array([0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.0, 0.0]), 3, 0, 1.0)
    assert dl[0] == 1.0 and list(q) == [0, 2, 2, 0, -2, -2, 3, 0]


def test_literal_mode_is_default_mode_one_bit_wider():
    """Delta = max|X| / (2^b - 1) as printed in Section 2.1 equals the default reading at b+1."""
    rng = np.random.default_rng(3)
    y = rng.standard_normal(512) * 3
    for b in (2, 3, 4):
        for alpha in (1.0, 0.8):
            q1, d1 = oracle.quantize(y, b, 64, alpha, literal=True)
            q2, d2 = oracle.quantize(y, b + 1, 64, alpha, literal=False)
            assert np.array_equal(q1, q2) and np.array_equal(d1, d2)


# ----------------------------------------------------------------------------
# Packing (paper silent: pinned by a hand-packed example and the round trip)
# ----------------------------------------------------------------------------
def test_packing_hand_example_and_round_trip():
    # b = 4: element 2j -> low nibble, 2j+1 -> high nibble; -1 = 0xF, -7 = 0x9
    assert list(oracle.pack([1, -1, 7, -7], 4)) == [0xF1, 0x97]
    # b = 3: codes [1,-1,3,-3,0,2,-2,1] -> fields 1,7,3,5,0,2,6,1, little-endian bit stream
    fields = [1, 7, 3, 5, 0, 2, 6, 1]
    word = sum(f << (3 * j) for j, f in enumerate(fields))
    want = [word & 0xFF, (word >> 8) & 0xFF, (word >> 16) & 0xFF]
    assert list(oracle.pack([1, -1, 3, -3, 0, 2, -2, 1], 3)) == want
    rng = np.random.default_rng(5)
    for bits in (3, 4):
        D = 2 ** (bits - 1) - 1
        q = rng.integers(-D, D + 1, size=4096).astype(np.int32)
        buf = oracle.pack(q, bits)
        assert buf.shape[0] == 4096 * bits // 8
        assert np.array_equal(oracle.unpack(buf, 4096, bits), q)


# ----------------------------------------------------------------------------
# Batched drivers, clip error, dequantize
# ----------------------------------------------------------------------------
def _bf16_bits(x64):
    import torch
    t = torch.from_numpy(x64.astype(np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16), t.to(torch.float64).numpy()


@pytest.mark.parametrize("m,k,d,group,bits", [(1, 7, 128, 0, 4), (28, 3, 224, 8, 3), (20, 4, 300, 0, 4),
                                              (12, 5, 384, 32, 3)])
def test_rows_driver_matches_single_row_functions(m, k, d, group, bits):
    rng = np.random.default_rng(17)
    dp = m << k
    stride = d + 8
    xb, xf = _bf16_bits(rng.standard_t(3, size=(9, stride)))
    res = oracle.rotate_quantize_rows(xb, d, dp, m, bits, group, 0.9, dense=True)
    res_fast = oracle.rotate_quantize_rows(xb, d, dp, m, bits, group, 0.9, dense=False, nthreads=2)
    for r in range(9):
        y = oracle.rotate(xf[r, :d], dp, m, dense=True)
        q, dl = oracle.quantize(y, bits, group, 0.9)
        assert np.array_equal(res["y"][r], y)
        assert np.array_equal(res["q"][r], q)
        assert np.array_equal(res["delta"][r], dl)
        assert np.array_equal(res["packed"][r], oracle.pack(q, bits))
        np.testing.assert_allclose(res_fast["y"][r], y, rtol=0, atol=1e-12 * np.abs(y).max())
    # fp32 input path gives the same numbers for bf16-representable data
    res32 = oracle.rotate_quantize_rows(xf.astype(np.float32), d, dp, m, bits, group, 0.9, dense=True)
    assert np.array_equal(res32["y"], res["y"]) and np.array_equal(res32["packed"], res["packed"])


@pytest.mark.parametrize("m,k,d,group", [(1, 8, 256, 0), (28, 3, 224, 8), (20, 4, 300, 0)])
def test_clip_error_is_reconstruction_error_in_input_space(m, k, d, group):
    """Orthogonality (Section 2.3.1): sum (y - yhat)^2 = || x_pad - H^T yhat / sqrt(d') ||^2,
    and with K = 1 it equals the error of rotate_quantize followed by dequantize."""
    rng = np.random.default_rng(23)
    dp = m << k
    x32 = rng.standard_t(3, size=(6, d)).astype(np.float32)
    alphas = np.array([1.0, 0.85, 0.6, 0.3])
    bits = 3
    err, rows = oracle.clip_error_rows(x32, d, dp, m, bits, group, alphas, want_rows=True)
    np.testing.assert_allclose(err, rows.sum(axis=0), rtol=1e-14)
    for kk, a in enumerate(alphas):
        res = oracle.rotate_quantize_rows(x32, d, dp, m, bits, group, a, dense=True)
        yhat = oracle.dequantize_rows(res["packed"], res["delta"], d, dp, m, bits, group, inverse=False)
        e_rot = ((res["y"] - yhat) ** 2).sum(axis=1)
        np.testing.assert_allclose(rows[:, kk], e_rot, rtol=1e-11)
        # through the inverse rotation, in the padded input space
        xpad = np.concatenate([x32.astype(np.float64), np.zeros((6, dp - d))], axis=1)
        xhat_pad = np.stack([oracle.rotate(yhat[r], dp, m, dense=True, transpose=True) for r in range(6)])
        e_in = ((xpad - xhat_pad) ** 2).sum(axis=1)
        np.testing.assert_allclose(rows[:, kk], e_in, rtol=1e-9)
        xhat = oracle.dequantize_rows(res["packed"], res["delta"], d, dp, m, bits, group, inverse=True)
        np.testing.assert_allclose(xhat, xhat_pad[:, :d], rtol=0, atol=1e-12 * np.abs(xpad).max())
    # at alpha = 1 the error is bounded by d' Delta^2 / 4 per scale group
    res = oracle.rotate_quantize_rows(x32, d, dp, m, bits, group, 1.0)
    g = group or dp
    bound = (res["delta"] ** 2 * g / 4).sum(axis=1)
    assert np.all(rows[:, 0] <= bound * (1 + 1e-12))


def test_rows_driver_rejects_bad_arguments():
    x = np.zeros((2, 16), dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.rotate_quantize_rows(x, 16, 24, 3, 3, 0, 1.0)       # no H_3
    with pytest.raises(ValueError):
        oracle.rotate_quantize_rows(x, 16, 16, 1, 3, 5, 1.0)       # group does not divide d'
    with pytest.raises(ValueError):
        oracle.rotate_quantize_rows(x, 32, 16, 1, 3, 0, 1.0)       # d > d'
    with pytest.raises(ValueError):
        oracle.rotate_quantize_rows(x.astype(np.float64), 16, 16, 1, 3, 0, 1.0)
