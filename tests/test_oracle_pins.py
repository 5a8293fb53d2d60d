"""Pins for the CPU oracle: closed forms, invariants, hand-worked cases, brute force.

Each test checks the oracle against something other than itself: a value the
paper fixes, a mathematical identity, a library routine, or exhaustive
enumeration on tiny inputs.
"""
import itertools
import os

import numpy as np
import pytest

from paper_2502_20586_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
GRID = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def _lines(name):
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                yield line.split()


# --------------------------------------------------------------------------- Philox

def test_philox_known_answers(ref):
    n = 0
    for tok in _lines("philox4x32_10_kat.txt"):
        v = [int(t, 16) for t in tok if t != "->"]
        out = ref.philox4x32_10(v[0:4], v[4:6])
        assert [int(o) for o in out] == v[6:10]
        n += 1
    assert n == 3


def test_sign_vector_and_draw_indexing(ref):
    """S_j and the 8-bit SR draws sit where the counter layout says (seed = key, index = counter)."""
    seed = 0x0123456789ABCDEF
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for g in (32, 64, 128, 256):
        S = ref.sign_vector(seed, g)
        assert set(np.unique(S)) <= {-1, 1}
        for j in (0, 1, 31, g // 2, g - 1):
            out = ref.philox4x32_10([j >> 7, 0, 0, 0], key)
            bit = (int(out[(j >> 5) & 3]) >> (j & 31)) & 1
            assert S[j] == 1 - 2 * bit
    # a 256-long vector is an extension of the shorter ones, and is not constant
    assert np.array_equal(ref.sign_vector(seed, 256)[:64], ref.sign_vector(seed, 64))
    assert abs(int(ref.sign_vector(seed, 256).sum())) < 64
    for tag, i in ((1, 0), (2, 5), (3, 16), (4, 2**33 + 7)):
        out = ref.philox4x32_10([(i >> 4) & 0xFFFFFFFF, (i >> 4) >> 32, tag, 1], key)
        f = i & 15
        assert ref.sr_draw(seed, tag, i) == (int(out[f >> 2]) >> (8 * (f & 3))) & 0xFF
    # different stream tags give different (independent) streams
    a = [ref.sr_draw(seed, 1, i) for i in range(256)]
    b = [ref.sr_draw(seed, 2, i) for i in range(256)]
    assert a != b and len(set(a)) > 100


def test_sr_draws_are_uniform(ref):
    n = 1 << 16
    d = np.array([ref.sr_draw(7, 1, i) for i in range(n)])
    counts = np.bincount(d, minlength=256)
    chi2 = ((counts - n / 256.0) ** 2 / (n / 256.0)).sum()
    assert chi2 < 255 + 6 * np.sqrt(2 * 255)          # 6 sigma of a chi-square with 255 dof


# --------------------------------------------------------------------------- Hadamard (Eq. 4)

@pytest.mark.parametrize("g", [2, 4, 32, 64, 128, 256])
def test_hadamard_closed_forms(ref, g):
    H = ref.hadamard(g).astype(np.int64)
    assert np.array_equal(H @ H.T, g * np.eye(g, dtype=np.int64))          # H H^T = g I
    assert np.array_equal(H, H.T)
    assert np.all(H[0] == 1) and np.all(H[:, 0] == 1)
    i, j = np.meshgrid(np.arange(g), np.arange(g), indexing="ij")
    pop = np.vectorize(lambda v: bin(v).count("1"))(i & j)
    assert np.array_equal(H, 1 - 2 * (pop & 1))                            # (-1)^popcount(i & j)
    scipy_linalg = pytest.importorskip("scipy.linalg")
    assert np.array_equal(H, scipy_linalg.hadamard(g))                     # library routine


def test_rht_one_hot_and_norm(ref):
    """A one-hot chunk maps to S_i H[i, :] / sqrt(g); every chunk keeps its 2-norm (orthogonality)."""
    g, seed = 64, 11
    H = ref.hadamard(g).astype(np.float64)
    S = ref.sign_vector(seed, g).astype(np.float64)
    x = np.zeros((3, 2 * g), np.float32)
    x[0, 5] = 2.0
    x[1, g + 17] = -3.0
    x[2, :] = np.random.default_rng(0).standard_normal(2 * g)
    y = ref.rht(wl.to_bf16_bits(x), g, seed).astype(np.float64)
    assert np.allclose(y[0, :g], 2.0 * S[5] * H[5] / 8.0, rtol=0, atol=1e-7)
    assert np.all(y[0, g:] == 0)
    assert np.allclose(y[1, g:], -3.0 * S[17] * H[17] / 8.0, rtol=0, atol=1e-7)
    xb = wl.bf16_bits_to_f64(wl.to_bf16_bits(x))
    for c in range(2):
        assert np.isclose(np.linalg.norm(y[2, c * g:(c + 1) * g]), np.linalg.norm(xb[2, c * g:(c + 1) * g]), rtol=1e-6)
    # g = 0: identity
    assert np.array_equal(ref.rht(wl.to_bf16_bits(x), 0, seed), wl.bf16_bits_to_f32(wl.to_bf16_bits(x)))


@pytest.mark.parametrize("g", [32, 64, 128, 256])
def test_gemm_invariant_under_shared_rht(ref, g):
    """(A B_d)(B B_d)^T = A B^T for the dgrad (contiguous) and wgrad (transposed) chunkings."""
    rng = np.random.default_rng(g)
    b, m, n = 2 * g, 512, 96
    dY = wl.to_bf16_bits(rng.standard_normal((b, m)))
    W = wl.to_bf16_bits(rng.standard_normal((m, n)))
    X = wl.to_bf16_bits(rng.standard_normal((b, n)))
    dYf, Wf, Xf = (wl.bf16_bits_to_f64(t) for t in (dY, W, X))
    seed = 3
    # dgrad: reduce over m.  dY is [b, m] (contiguous chunks), W^T is [n, m] (transposed view)
    q1 = ref.rht(dY, g, seed).astype(np.float64)
    q2 = ref.rht(W, g, seed, transpose=True).astype(np.float64)
    exact = dYf @ Wf
    assert np.linalg.norm(q1 @ q2.T - exact) / np.linalg.norm(exact) < 5e-7     # fp32 rounding of y only
    # wgrad: reduce over b
    q3 = ref.rht(dY, g, seed, transpose=True).astype(np.float64)
    q4 = ref.rht(X, g, seed, transpose=True).astype(np.float64)
    exact = dYf.T @ Xf
    assert np.linalg.norm(q3 @ q4.T - exact) / np.linalg.norm(exact) < 5e-7
    # exact fp64 statement of the identity with the oracle's own H and S (rel <= 1e-12)
    H = ref.hadamard(g).astype(np.float64)
    S = ref.sign_vector(seed, g).astype(np.float64)
    Bd = np.kron(np.eye(m // g), np.diag(S) @ H / np.sqrt(g))
    lhs = (dYf @ Bd) @ (Wf.T @ Bd).T
    assert np.linalg.norm(lhs - dYf @ Wf) / np.linalg.norm(dYf @ Wf) < 1e-12
    assert np.linalg.norm(q1 - dYf @ Bd) / np.linalg.norm(q1) < 1e-7
    # different seeds give different transforms, the product is unchanged
    assert not np.array_equal(ref.sign_vector(seed, g), ref.sign_vector(seed + 1, g))


def test_hadamard_tail_bound_brute_force(ref):
    """Eq. 5: P(|e_i H S x| >= a) <= 2 exp(-a^2 k / (2 |x|^2)) over ALL 2^k sign vectors, H orthonormal."""
    rng = np.random.default_rng(5)
    for k, xs in ((8, [rng.standard_normal(8), np.eye(8)[3]]), (16, [rng.standard_normal(16)])):
        H = ref.hadamard(k).astype(np.float64) / np.sqrt(k)
        signs = np.array(list(itertools.product((1.0, -1.0), repeat=k)))      # [2^k, k]
        for x in xs:
            z = np.abs((signs * x) @ H)                                       # [2^k, k]: |e_i H S x|
            worst = 0.0
            for a in np.linspace(0.05, 1.2 * np.linalg.norm(x), 60):
                p = (z >= a).mean(axis=0)                                     # per output index i
                bound = 2 * np.exp(-a * a * k / (2 * np.dot(x, x)))
                worst = max(worst, float((p / bound).max()))
            assert worst <= 1.0


# --------------------------------------------------------------------------- element format, scale, rounding

def test_e2m1_code_table(ref):
    # 1 sign, 2 exponent (bias 1), 1 mantissa: subnormal M * 0.5; normal (1 + M/2) 2^(E-1)
    for code in range(16):
        s, e, mbit = code >> 3, (code >> 1) & 3, code & 1
        mag = 0.5 * mbit if e == 0 else (1 + 0.5 * mbit) * 2.0 ** (e - 1)
        assert ref.e2m1_value(code) == (-mag if s else mag)
    assert [ref.e2m1_value(c) for c in range(8)] == GRID
    assert max(GRID) / min(v for v in GRID if v > 0) == 12.0                  # dynamic range 6 / 0.5


def test_worked_blocks(ref):
    n = 0
    for tok in _lines("worked_blocks.txt"):
        kind = tok[0]
        if kind == "scale":
            assert ref.e8m0_from_amax(float(tok[1])) == int(tok[2]), tok
        elif kind == "rn":
            assert ref.e2m1_value(ref.rn_round(float(tok[1]))) == float(tok[2]), tok
        elif kind == "sr":
            w, lo, hi, p_up = (float(t) for t in tok[1:5])
            vals = [ref.e2m1_value(ref.sr_round(w, r)) for r in range(256)]
            assert set(vals) <= {lo, hi}, tok
            assert abs(vals.count(hi) / 256.0 - p_up) <= 2.0 ** -9 + 1e-12, tok
            assert abs(np.mean(vals) - w) <= abs(hi - lo) * 2.0 ** -9 + 1e-12, tok     # unbiased
        n += 1
    assert n >= 30


def test_scale_rule_against_log2(ref):
    """byte - 127 = floor(log2 amax) - 2 on exact powers of two and their neighbours; clamps."""
    for e in range(-126, 128):
        p = np.float32(2.0) ** np.float32(e)
        assert ref.e8m0_from_amax(p) == max(e - 2, -127) + 127
        below = np.nextafter(p, np.float32(0))
        if below > 0 and e > -126:
            assert ref.e8m0_from_amax(below) == max(e - 3, -127) + 127
    assert ref.e8m0_from_amax(np.float32(1e-45)) == 0                         # fp32 subnormal
    assert ref.e8m0_from_amax(np.finfo(np.float32).max) == 127 + 125
    assert ref.e8m0_from_amax(float("inf")) == 255
    # after dividing by X the block maximum lies in [4, 8) (Section 3.1)
    rng = np.random.default_rng(1)
    for amax in np.abs(rng.standard_normal(200)).astype(np.float32) * 10 + 1e-3:
        e = ref.e8m0_from_amax(amax) - 127
        assert 4.0 <= float(amax) / 2.0 ** e < 8.0


def test_sr_is_unbiased_by_enumeration(ref):
    """E over all 256 draws of SR(w) equals w up to gap / 512; exactly when 256 frac is an integer."""
    for w in np.linspace(0, 5.999, 1201):
        for sgn in (1.0, -1.0):
            vals = np.array([ref.e2m1_value(ref.sr_round(sgn * w, r)) for r in range(0, 256)])
            lo = max(v for v in GRID if v <= w)
            hi = min(v for v in GRID if v > w)
            assert set(np.abs(vals)) <= {lo, hi}
            assert abs(vals.mean() - sgn * w) <= (hi - lo) / 512 + 1e-12
            frac256 = (w - lo) / (hi - lo) * 256
            if frac256 == int(frac256):
                assert vals.mean() == sgn * w
            # variance of the two-point law: (c - a)(a - f) up to the discretisation of P(up)
            assert abs(vals.var() - (hi - w) * (w - lo)) <= (hi - lo) ** 2 / 256 + 1e-12
    assert np.var([ref.e2m1_value(ref.sr_round(5.25, r)) for r in range(256)]) == pytest.approx(0.9375)
    # grid points are fixed points; the sign of zero is kept
    for c in range(16):
        v = ref.e2m1_value(c)
        assert all(ref.sr_round(v, r) == c for r in (0, 127, 255)) or c == 8
    assert ref.sr_round(-0.0, 0) == 8 and ref.sr_round(0.0, 255) == 0


def test_sr_matches_dither_form_on_uniform_grid(ref):
    """Eq. 1-2 on the uniform part of the grid (spacing 1/2 on [0, 2]): delta = 1/2 - (r + 1/2)/256."""
    rng = np.random.default_rng(2)
    ties = [(k + 0.5) / 512 for k in (0, 1, 77, 128, 200, 255, 256, 300, 511, 767, 1023)]   # frac * 256 = r + 1/2 exactly
    for w in list(rng.uniform(0, 2, 400)) + ties:
        x = 2 * w                                              # grid-index units: integers are grid points
        for r in (0, 1, 77, 128, 200, 255):
            delta = 0.5 - (r + 0.5) / 256.0
            expect = np.ceil(x) if (x - np.floor(x)) + delta >= 0.5 else np.floor(x)
            if x == np.floor(x):
                expect = x
            assert ref.e2m1_value(ref.sr_round(w, r)) == expect / 2


def test_quantize_blocks_sr_and_rn(ref):
    """Algorithm 2 end to end on a block: scale from the un-prescaled amax, |w| < 6, Philox draws by index."""
    seed, tag = 99, 3
    rng = np.random.default_rng(4)
    y = (rng.standard_normal((4, 96)) * np.array([[1e-3], [1.0], [37.0], [1e4]])).astype(np.float32)
    y[1, 32:64] = 0.0                                          # all-zero block
    codes, scales = ref.quantize(y, ref.ROUND_SR, seed, tag)
    for r in range(4):
        for b in range(3):
            V = y[r, 32 * b:32 * b + 32].astype(np.float64)
            amax = np.abs(V).max()
            byte = int(scales[r, b])
            if amax == 0:
                assert byte == 0 and np.all(codes[r, 32 * b:32 * b + 32] == 0)
                continue
            assert byte - 127 == int(np.floor(np.log2(amax))) - 2
            w = 0.75 * V / 2.0 ** (byte - 127)
            assert np.abs(w).max() < 6.0 and np.abs(w).max() >= 3.0            # never clips
            for i in range(32):
                idx = r * 96 + 32 * b + i
                assert codes[r, 32 * b + i] == ref.sr_round(w[i], ref.sr_draw(seed, tag, idx))
    codes_rn, scales_rn = ref.quantize(y, ref.ROUND_RN, seed, tag)
    assert np.array_equal(scales, scales_rn)
    deq = ref.dequantize(codes_rn, scales_rn)
    X = 2.0 ** (scales_rn.astype(np.float64) - 127).repeat(32, axis=1)
    # nearest rounding: error at most half the local gap unless the value clipped above 6 X
    clipped = np.abs(y) > 6 * X
    gap = np.where(np.abs(y) / X >= 4, 2.0, np.where(np.abs(y) / X >= 2, 1.0, 0.5)) * X
    assert np.all(np.abs(deq - y)[~clipped] <= gap[~clipped] / 2 + 1e-30)
    assert np.all(np.abs(deq)[clipped] == (6 * X)[clipped])
    # packing: even element in the low nibble
    p = ref.pack(codes)
    assert p.shape == (4, 48) and p[0, 0] == (codes[0, 0] | (codes[0, 1] << 4))


def test_clip_fraction_alg1_vs_alg2(ref):
    """Section 3.1: Algorithm 1 clips a few percent of N(0,1) entries ("roughly 3%"); Algorithm 2 none."""
    y = np.random.default_rng(6).standard_normal((512, 1024)).astype(np.float32)
    _, scales = ref.quantize(y, ref.ROUND_RN, 0, 0)
    X = 2.0 ** (scales.astype(np.float64) - 127).repeat(32, axis=1)
    frac = float((np.abs(y) / X > 6).mean())
    assert 0.01 < frac < 0.05
    assert float((0.75 * np.abs(y) / X >= 6).mean()) == 0.0


def test_sr_monte_carlo_through_philox(ref):
    """E[X * SR(3/4 v / X)] = 3/4 v with the real generator: mean over many stream tags, 5 sigma."""
    rng = np.random.default_rng(8)
    y = rng.standard_normal((8, 64)).astype(np.float32)
    T = 4000
    acc = np.zeros(y.shape)
    for t in range(T):
        codes, scales = ref.quantize(y, ref.ROUND_SR, 1234, t)
        acc += ref.dequantize(codes, scales)
    X = 2.0 ** (scales.astype(np.float64) - 127).repeat(32, axis=1)
    sigma = X / np.sqrt(T)                                   # per-draw std <= gap/2 <= X
    assert np.all(np.abs(acc / T - 0.75 * y) <= 5 * sigma + X / 512)


def test_transform_with_a_given_matrix(ref):
    """Section 3.2: any orthogonal matrix may stand in for the RHT.  With T = diag(S) H_g / sqrt(g) (exact in bf16 for
    g = 64) the given-matrix transform is the RHT; with the identity it is the input; with a random orthogonal Q (QR of
    a Gaussian matrix, fp64) norms and products are preserved; bf16 rounding of Q costs about 2^-9."""
    rng = np.random.default_rng(17)
    x = wl.grad_like(rng, (64, 256), 1.0)
    seed, g = 77, 64
    S = ref.sign_vector(seed, g).astype(np.float64)
    T = (S[:, None] * ref.hadamard(g).astype(np.float64)) / 8.0
    Tb = wl.to_bf16_bits(T.astype(np.float32))
    assert np.array_equal(wl.bf16_bits_to_f64(Tb), T)                      # +-1/8: exact
    for tr in (False, True):
        assert np.array_equal(ref.transform(x, Tb, transpose=tr), ref.rht(x, g, seed, transpose=tr))
    eye = wl.to_bf16_bits(np.eye(32, dtype=np.float32))
    assert np.array_equal(ref.transform(x, eye), wl.bf16_bits_to_f64(x).astype(np.float32))
    Q, _ = np.linalg.qr(rng.standard_normal((32, 32)))
    Qb = wl.to_bf16_bits(Q.astype(np.float32))
    y = ref.transform(x, Qb).astype(np.float64)
    xv = wl.bf16_bits_to_f64(x)
    want = (xv.reshape(64, 8, 32) @ wl.bf16_bits_to_f64(Qb)).reshape(64, 256)       # numpy's own product with the same bf16 matrix
    assert np.abs(y - want).max() <= 2.0 ** -23 * np.abs(want).max()
    nx, ny = np.linalg.norm(xv.reshape(64, 8, 32), axis=2), np.linalg.norm(y.reshape(64, 8, 32), axis=2)
    assert np.abs(ny / nx - 1).max() < 2.0 ** -6                           # orthogonal up to the bf16 rounding of Q
    b = wl.weight_like(rng, (16, 256))
    yb = ref.transform(b, Qb).astype(np.float64)
    exact = xv @ wl.bf16_bits_to_f64(b).T
    assert np.linalg.norm(y @ yb.T - exact) / np.linalg.norm(exact) < 2.0 ** -6


# --------------------------------------------------------------------------- second SR reading (16-bit dither)

def _rev(v, bits):
    return int(format(v, "0%db" % bits)[::-1], 2)


def test_sr16_draw_layout(ref):
    """The 16-bit dithers of four consecutive elements come from one Philox word: bytes (b2, b0) and (b3, b1),
    odd elements bit-reversed, so the leading eight bits of the four dithers are four different bytes."""
    seed = 0x0123456789ABCDEF
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for tag, h in ((1, 0), (2, 3), (3, 4), (4, (2**33 + 8) // 4)):
        i = 4 * h
        out = ref.philox4x32_10([(i >> 4) & 0xFFFFFFFF, (i >> 4) >> 32, tag, 1], key)
        word = int(out[(i >> 2) & 3])
        b = [(word >> (8 * k)) & 0xFF for k in range(4)]
        d = [ref.sr16_draw(seed, tag, i + j) for j in range(4)]
        assert d[0] == 256 * b[2] + b[0] and d[2] == 256 * b[3] + b[1]
        assert d[1] == _rev(d[0], 16) and d[3] == _rev(d[2], 16)
        assert [x >> 8 for x in d] == [b[2], _rev(b[0], 8), b[3], _rev(b[1], 8)]
        # the same bytes the 8-bit reading draws for these four elements
        assert [ref.sr_draw(seed, tag, i + j) for j in range(4)] == b
    n = 1 << 15
    d = np.array([ref.sr16_draw(7, 1, i) for i in range(n)])
    for top in (d >> 8, d & 0xFF, (d >> 4) & 0xFF):
        counts = np.bincount(top, minlength=256)
        chi2 = ((counts - n / 256.0) ** 2 / (n / 256.0)).sum()
        assert chi2 < 255 + 6 * np.sqrt(2 * 255)
    # leading bytes of paired elements are uncorrelated
    a, b2 = (d[0::4] >> 8).astype(float), (d[1::4] >> 8).astype(float)
    assert abs(np.corrcoef(a, b2)[0, 1]) < 5 / np.sqrt(len(a))


def test_sr16_law_by_enumeration(ref):
    """P(up) = floor(65536 frac) / 65536: the smallest dither that rounds up is 65536 - floor(65536 frac);
    E[SR16(w)] lies in (w - gap / 65536, w]; the hand-worked cases of the 8-bit reading hold to 2^-16."""
    def first_up(w):                                           # monotone in R: bisection over [0, 65536]
        lo = max(i for i, v in enumerate(GRID) if v <= abs(w))
        a, b = 0, 65536                                        # invariant: R < a rounds down, R >= b rounds up
        while a < b:
            mid = (a + b) // 2
            if (ref.sr16_round(w, mid) & 7) == lo + 1: b = mid
            else: a = mid + 1
        return a
    rng = np.random.default_rng(21)
    ws = list(rng.uniform(0, 5.9999, 300)) + [5.25, 0.75, 0.225, 1.65, 5.4, 3.0 + 2.0 ** -16, 4 + 2.0 ** -14, 0.5 - 2.0 ** -18, 1e-12]
    for w in ws:
        lo = max(v for v in GRID if v <= w)
        hi = min(v for v in GRID if v > w)
        F = int(np.floor((w - lo) / (hi - lo) * 65536))
        for sgn in (1.0, -1.0):
            t = first_up(sgn * w)
            assert t == 65536 - F or (F == 0 and t == 65536)
            if 0 < t < 65536:                                   # both sides of the threshold, and monotone beyond
                assert ref.e2m1_value(ref.sr16_round(sgn * w, t - 1)) == sgn * lo
                assert ref.e2m1_value(ref.sr16_round(sgn * w, t)) == sgn * hi
                assert ref.e2m1_value(ref.sr16_round(sgn * w, 65535)) == sgn * hi
            assert ref.e2m1_value(ref.sr16_round(sgn * w, 0)) == sgn * lo
        mean = lo + (hi - lo) * F / 65536.0
        assert w - (hi - lo) / 65536.0 < mean <= w
    # full enumeration for the worked SR cases: two outcomes, probability and mean as printed, variance (c - a)(a - f)
    for tok in _lines("worked_blocks.txt"):
        if tok[0] != "sr":
            continue
        w, lo, hi, p_up = (float(t) for t in tok[1:5])
        vals = np.array([ref.e2m1_value(ref.sr16_round(w, R)) for R in range(65536)])
        assert set(vals) <= {lo, hi}
        assert abs((vals == hi).mean() - p_up) <= 2.0 ** -16 + 1e-12
        assert abs(vals.mean() - w) <= abs(hi - lo) * 2.0 ** -16 + 1e-12
        assert abs(vals.var() - abs(hi - w) * abs(w - lo)) <= (hi - lo) ** 2 * 2.0 ** -15
    # grid points are fixed points, the sign of zero is kept, |w| >= 6 saturates
    for c in range(16):
        v = ref.e2m1_value(c)
        assert all(ref.sr16_round(v, R) == c for R in (0, 1, 32768, 65535)) or c == 8
    assert ref.sr16_round(-0.0, 65535) == 8 and ref.sr16_round(0.0, 65535) == 0
    assert ref.sr16_round(6.5, 0) == 7 and ref.sr16_round(-7.0, 0) == 15


def test_quantize_blocks_sr16(ref):
    """Algorithm 2 with the 16-bit reading: same scales as the 8-bit reading, codes from (w, dither by index);
    unbiased through the real generator, and paired elements round independently."""
    seed, tag = 99, 3
    rng = np.random.default_rng(4)
    y = (rng.standard_normal((4, 96)) * np.array([[1e-3], [1.0], [37.0], [1e4]])).astype(np.float32)
    y[1, 32:64] = 0.0
    codes, scales = ref.quantize(y, ref.ROUND_SR16, seed, tag)
    assert np.array_equal(scales, ref.quantize(y, ref.ROUND_SR, seed, tag)[1])
    for r in range(4):
        for b in range(3):
            V = y[r, 32 * b:32 * b + 32].astype(np.float64)
            w = 0.75 * V / 2.0 ** (int(scales[r, b]) - 127)
            for i in range(32):
                idx = r * 96 + 32 * b + i
                assert codes[r, 32 * b + i] == ref.sr16_round(w[i], ref.sr16_draw(seed, tag, idx))
    # row_ids shift the element index that keys the dither
    sub = ref.quantize(y[2:3], ref.ROUND_SR16, seed, tag, row_ids=np.array([2]))[0]
    assert np.array_equal(sub[0], codes[2])
    y = rng.standard_normal((8, 64)).astype(np.float32)
    T = 3000
    acc = np.zeros(y.shape)
    err = np.zeros((T,) + y.shape)
    for t in range(T):
        c, sc = ref.quantize(y, ref.ROUND_SR16, 1234, t)
        dq = ref.dequantize(c, sc)
        acc += dq
        err[t] = dq - 0.75 * y
    X = 2.0 ** (sc.astype(np.float64) - 127).repeat(32, axis=1)
    assert np.all(np.abs(acc / T - 0.75 * y) <= 5 * X / np.sqrt(T) + X * 2.0 ** -15)
    e = err / X
    for j in (0, 2):                                           # elements (4h, 4h+1) and (4h+2, 4h+3) share 16 bits
        a, b2 = e[:, :, j::4], e[:, :, j + 1::4]
        corr = ((a - a.mean(0)) * (b2 - b2.mean(0))).mean(0) / (a.std(0) * b2.std(0) + 1e-30)
        assert np.abs(corr).max() < 6 / np.sqrt(T)
    # Algorithm 3 carries the 16/9 in this reading too
    dY = wl.grad_like(rng, (32, 32), 1e-3)
    Xa = wl.activation_like(rng, (32, 32))
    W = wl.weight_like(rng, (32, 32))
    ex = wl.bf16_bits_to_f64(dY) @ wl.bf16_bits_to_f64(W)
    sx = sum(ref.linear_backward(dY, Xa, W, 32, ref.ROUND_SR16, 500 + t)[0] for t in range(48)) / 48
    assert abs(np.vdot(sx, ex) / np.vdot(ex, ex) - 1.0) < 0.05


# --------------------------------------------------------------------------- GEMM and Algorithm 3

def test_gemm_special_cases(ref):
    M, N, K = 5, 7, 96
    ones = np.full((M, K), 2, np.uint8)                                          # code 2 = 1.0
    s127 = np.full((M, K // 32), 127, np.uint8)
    C = ref.gemm(ones, s127, np.full((N, K), 2, np.uint8), np.full((N, K // 32), 127, np.uint8))
    assert np.all(C == K)
    # one nonzero block: X_A X_B sum of code products, exactly
    A = np.zeros((M, K), np.uint8); B = np.zeros((N, K), np.uint8)
    sa = np.full((M, 3), 127, np.uint8); sb = np.full((N, 3), 127, np.uint8)
    A[2, 32:64] = 7; B[4, 32:64] = 0xD                                          # 6 and -3
    sa[2, 1] = 127 + 5; sb[4, 1] = 127 - 9
    C = ref.gemm(A, sa, B, sb)
    expect = np.zeros((M, N)); expect[2, 4] = 2.0 ** 5 * 2.0 ** -9 * 32 * 6 * -3
    assert np.array_equal(C, expect)
    # alpha, row/col sampling, and agreement with numpy on dequantised operands
    rng = np.random.default_rng(9)
    A = rng.integers(0, 16, (M, K)).astype(np.uint8); B = rng.integers(0, 16, (N, K)).astype(np.uint8)
    sa = rng.integers(120, 135, (M, 3)).astype(np.uint8); sb = rng.integers(120, 135, (N, 3)).astype(np.uint8)
    full = ref.gemm(A, sa, B, sb, alpha=16 / 9)
    assert np.allclose(full, 16 / 9 * ref.dequantize(A, sa) @ ref.dequantize(B, sb).T, rtol=1e-14)
    sub = ref.gemm(A, sa, B, sb, alpha=16 / 9, rows=[4, 0], cols=[6, 1, 3])
    assert np.array_equal(sub, full[np.ix_([4, 0], [6, 1, 3])])
    # the oracle's bf16 product is numpy's
    a = wl.to_bf16_bits(rng.standard_normal((6, 40))); b = wl.to_bf16_bits(rng.standard_normal((40, 9)))
    assert np.allclose(ref.gemm_bf16(a, b, b_transpose=True), wl.bf16_bits_to_f64(a) @ wl.bf16_bits_to_f64(b), rtol=1e-13)


def test_linear_backward_exact_on_representable_inputs(ref):
    """Algorithm 3 with nearest rounding and no RHT is exact when every operand already is MXFP4.

    Entries are E2M1 grid values times a per-32-block power of two, along BOTH dimensions, so each of the
    four operand views quantises without error and dX = dY W, dW = dY^T X exactly.  A transposed operand,
    a wrong stride or swapped output fails this."""
    rng = np.random.default_rng(10)
    b, m, n = 64, 96, 128

    def mx_like(shape):
        mag = rng.choice(GRID, size=shape) * rng.choice([-1.0, 1.0], size=shape)
        mag[::32, :] = 6.0                      # every column block of 32 rows holds a 6 ...
        mag[:, ::32] = 6.0                      # ... and every row block of 32 columns too
        return wl.to_bf16_bits(mag * 2.0 ** rng.integers(-3, 4))

    dY, X, W = mx_like((b, m)), mx_like((b, n)), mx_like((m, n))
    dX, dW = ref.linear_backward(dY, X, W, 0, ref.ROUND_RN, 0)
    assert np.array_equal(dX, wl.bf16_bits_to_f64(dY) @ wl.bf16_bits_to_f64(W))
    assert np.array_equal(dW, wl.bf16_bits_to_f64(dY).T @ wl.bf16_bits_to_f64(X))
    sub_dx, sub_dw = ref.linear_backward(dY, X, W, 0, ref.ROUND_RN, 0, dx_rows=[3, 60], dx_cols=[0, 127],
                                         dw_rows=[95], dw_cols=[1, 2, 3])
    assert np.array_equal(sub_dx, dX[np.ix_([3, 60], [0, 127])])
    assert np.array_equal(sub_dw, dW[np.ix_([95], [1, 2, 3])])


def test_linear_backward_is_unbiased(ref):
    """Lemma 3.1: with SR (and the shared RHT) the mean over seeds tends to dY W and dY^T X like T^-1/2,
    while nearest rounding plateaus at its bias."""
    rng = np.random.default_rng(12)
    b, m, n, g = 64, 64, 64, 32
    dY = wl.grad_like(rng, (b, m), 1e-3, outlier_rate=0.01)
    X = wl.activation_like(rng, (b, n))
    W = wl.weight_like(rng, (m, n))
    ex_dx = wl.bf16_bits_to_f64(dY) @ wl.bf16_bits_to_f64(W)
    ex_dw = wl.bf16_bits_to_f64(dY).T @ wl.bf16_bits_to_f64(X)
    err = {}
    for T in (4, 64):
        sx = np.zeros_like(ex_dx); sw = np.zeros_like(ex_dw)
        for t in range(T):
            dx, dw = ref.linear_backward(dY, X, W, g, ref.ROUND_SR, 1000 + t)
            sx += dx; sw += dw
        err[T] = (np.linalg.norm(sx / T - ex_dx) / np.linalg.norm(ex_dx),
                  np.linalg.norm(sw / T - ex_dw) / np.linalg.norm(ex_dw))
    # 16x more samples -> about 4x less error (allow 2.5x)
    assert err[64][0] < err[4][0] / 2.5 and err[64][1] < err[4][1] / 2.5
    one_dx, one_dw = ref.linear_backward(dY, X, W, g, ref.ROUND_SR, 1000)
    assert np.linalg.norm(one_dx - ex_dx) / np.linalg.norm(ex_dx) < 0.5      # a sane single-shot error
    # without the 16/9 the SR estimate would be 9/16 of the product: check the factor is in
    assert abs(np.vdot(sx / 64, ex_dx) / np.vdot(ex_dx, ex_dx) - 1.0) < 0.05
    # RN: averaging over seeds changes only S; the bias does not average out as fast
    sx = np.zeros_like(ex_dx)
    for t in range(64):
        sx += ref.linear_backward(dY, X, W, 0, ref.ROUND_RN, 1000 + t)[0]
    assert np.linalg.norm(sx / 64 - ex_dx) / np.linalg.norm(ex_dx) > err[64][0]


def test_sr_gemm_variance_formula_and_rht_trend(ref):
    """Variance proof: Var(C) = sum_i X_A^2 X_B^2 [v_A v_B + v_A mu_B^2 + v_B mu_A^2] with the per-element
    two-point variance v = (c - a)(a - f); sampled over seeds.  Fig. 2 trend: with outliers the variance
    after the RHT is lower."""
    rng = np.random.default_rng(13)
    b = 128

    def var_terms(y):
        """mu = w, v = (c - w)(w - f), X per element for the Algorithm-2 quantisation of an fp32 row."""
        _, scales = ref.quantize(y, ref.ROUND_SR, 0, 0)
        X = 2.0 ** (scales.astype(np.float64) - 127).repeat(32, axis=1)
        w = np.abs(0.75 * y.astype(np.float64) / X)
        lo = np.array([[max(v for v in GRID if v <= t) for t in row] for row in w])
        hi = np.array([[min(v for v in GRID if v > t) for t in row] for row in w])
        return X, 0.75 * y.astype(np.float64) / X, (hi - w) * (w - lo)

    A = rng.standard_normal((1, b)).astype(np.float32)
    B = rng.standard_normal((1, b)).astype(np.float32)
    XA, muA, vA = var_terms(A); XB, muB, vB = var_terms(B)
    predicted = float((XA ** 2 * XB ** 2 * (vA * vB + vA * muB ** 2 + vB * muA ** 2)).sum())
    T = 6000
    samples = np.empty(T)
    for t in range(T):
        ca, sa = ref.quantize(A, ref.ROUND_SR, t, 1)
        cb, sb = ref.quantize(B, ref.ROUND_SR, t, 2)
        samples[t] = ref.gemm(ca, sa, cb, sb)[0, 0]
    assert abs(samples.mean() - 9 / 16 * float(np.vdot(A.astype(np.float64), B.astype(np.float64)))) < 5 * np.sqrt(predicted / T)
    assert abs(samples.var() / predicted - 1.0) < 0.12
    # Fig. 2 trend (closed form, averaged over draws): A, B ~ N(0, I) + Bernoulli(p) N(0, 5 I)
    def mean_var(p, use_rht, trials=48):
        tot = 0.0
        for t in range(trials):
            r = np.random.default_rng(1000 + t)
            a = r.standard_normal((1, b)) + (r.random((1, b)) < p) * r.standard_normal((1, b)) * np.sqrt(5.0)
            c = r.standard_normal((1, b)) + (r.random((1, b)) < p) * r.standard_normal((1, b)) * np.sqrt(5.0)
            ab, cb_ = wl.to_bf16_bits(a), wl.to_bf16_bits(c)
            ya = ref.rht(ab, 64 if use_rht else 0, t)
            yc = ref.rht(cb_, 64 if use_rht else 0, t)
            xa, ma, va = var_terms(ya); xc, mc, vc = var_terms(yc)
            tot += float((xa ** 2 * xc ** 2 * (va * vc + va * mc ** 2 + vc * ma ** 2)).sum())
        return tot / trials
    assert mean_var(0.1, True) < mean_var(0.1, False)
    assert abs(mean_var(0.0, True) / mean_var(0.0, False) - 1.0) < 0.25


def test_bias_grad_closed_forms(ref):
    """dL/db = 1 dL/dy (problem statement): closed forms a transposed index, a dropped row or a wrong stride would break."""
    b, m = 96, 40
    # dY[i, j] = j + 1: every column sums to b (j + 1)
    dY = np.tile(np.arange(1, m + 1, dtype=np.float64), (b, 1))
    assert np.array_equal(ref.bias_grad(wl.to_bf16_bits(dY)), b * np.arange(1, m + 1, dtype=np.float64))
    # dY[i, j] = i for j == 3 only: Gauss sum in one column, zeros elsewhere
    dY = np.zeros((b, m)); dY[:, 3] = np.arange(b)
    want = np.zeros(m); want[3] = b * (b - 1) / 2
    assert np.array_equal(ref.bias_grad(wl.to_bf16_bits(dY)), want)
    # alternating signs cancel exactly; a lone last row survives
    dY = np.ones((b + 1, m)); dY[1::2] = -1.0; dY[-1] = 0.25
    assert np.array_equal(ref.bias_grad(wl.to_bf16_bits(dY)), np.full(m, 0.25))
    # random bf16 data against numpy's own sum of the exactly converted values
    rng = np.random.default_rng(7)
    bits = wl.to_bf16_bits(rng.standard_normal((300, 24)) * 1e-3)
    np.testing.assert_allclose(ref.bias_grad(bits), wl.bf16_bits_to_f64(bits).sum(axis=0), rtol=1e-13, atol=0)
