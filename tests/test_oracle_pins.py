"""Pins for the fp64 CPU oracle: everything here is fixed by mathematics, a textbook value, exact
rational brute force or an independent library routine -- never by the oracle itself and never
by the CUDA path.  Each test is aimed at one plausible mistake (dropped term, wrong sign or
index, transposed operand, wrong order of epilogue steps, biased/unbiased variance, ...).
"""
import math
from decimal import Decimal, getcontext
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest

from oracle import kfo
from paper_2603_12440_b200 import inputs

GOLD = {}
for line in (Path(__file__).parent / "golden" / "closed_forms.txt").read_text().splitlines():
    line = line.split("#")[0].strip()
    if line:
        key, *vals = line.split()
        GOLD[key] = [float(v) for v in vals]


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


# ----------------------------------------------------------------------------- activations
def test_activation_textbook_values():
    assert kfo.act("gelu_erf", 1.0) == pytest.approx(GOLD["Phi_1.0"][0], abs=1e-15)
    assert kfo.act("gelu_erf", 2.0) == pytest.approx(2 * GOLD["Phi_2.0"][0], abs=1e-15)
    # GELU(z) = z/2 (1 + erf(z/sqrt2)): at z = sqrt2 * t this exposes erf(t) from the tables
    for t, key in ((0.5, "erf_0.5"), (1.0, "erf_1.0"), (2.0, "erf_2.0")):
        z = math.sqrt(2.0) * t
        assert kfo.act("gelu_erf", z) == pytest.approx(0.5 * z * (1 + GOLD[key][0]), abs=1e-15)
    assert kfo.act("silu", 1.0) == pytest.approx(GOLD["sigmoid_1.0"][0], abs=1e-15)
    assert kfo.act("silu", 2.0) == pytest.approx(2 * GOLD["sigmoid_2.0"][0], abs=1e-15)
    assert kfo.act("sigmoid", 1.0) == pytest.approx(GOLD["sigmoid_1.0"][0], abs=1e-15)
    assert kfo.act("gelu_tanh", 1.0) == pytest.approx(GOLD["tanh_gelu_1.0"][0], abs=1e-15)
    assert kfo.act("silu", GOLD["silu_argmin"][0]) == pytest.approx(GOLD["silu_min"][0], abs=1e-15)
    # the minimiser really is one: neighbours are larger
    xm = GOLD["silu_argmin"][0]
    assert kfo.act("silu", xm - 1e-3) > kfo.act("silu", xm) < kfo.act("silu", xm + 1e-3)


def test_activation_identities():
    for z in np.linspace(-6, 6, 49):
        z = float(z)
        assert kfo.act("none", z) == z
        assert kfo.act("relu", z) == max(z, 0.0)
        # odd-part identities: f(z) - f(-z) = z for GELU (both forms) and SiLU
        for name in ("gelu_erf", "gelu_tanh", "silu"):
            assert kfo.act(name, z) - kfo.act(name, -z) == pytest.approx(z, abs=1e-14)
        assert kfo.act("sigmoid", z) + kfo.act("sigmoid", -z) == pytest.approx(1.0, abs=1e-15)
        assert kfo.act("silu", z) == pytest.approx(z * kfo.act("sigmoid", z), abs=1e-15)
    for name in ("gelu_erf", "gelu_tanh", "silu", "relu", "none"):
        assert kfo.act(name, 0.0) == 0.0
    assert kfo.act("gelu_erf", 10.0) == pytest.approx(10.0, abs=1e-15)
    assert abs(kfo.act("gelu_erf", -10.0)) < 1e-20
    assert kfo.act("silu", 40.0) == pytest.approx(40.0, abs=1e-14)
    assert abs(kfo.act("silu", -40.0)) < 1e-15
    # the two GELU forms are different functions (max gap a few 1e-4): a silent swap must show
    gap = max(abs(kfo.act("gelu_erf", z) - kfo.act("gelu_tanh", z)) for z in np.linspace(-4, 4, 801))
    assert 1e-4 < gap < 1e-3


def _erf_series(x: Decimal) -> Decimal:
    """erf by its Maclaurin series in 60-digit decimal arithmetic (brute force, |x| < 4)."""
    getcontext().prec = 60
    term = x
    total = x
    n = 0
    while abs(term) > Decimal(10) ** -50:
        n += 1
        term = -term * x * x / n
        total += term / (2 * n + 1)
    pi = Decimal("3.14159265358979323846264338327950288419716939937510582097494")
    return 2 * total / pi.sqrt()


def test_gelu_erf_against_series_bruteforce():
    getcontext().prec = 60
    for z in (-3.7, -2.0, -0.9, -0.1, 0.3, 0.77, 1.5, 2.9, 3.9):
        zd = Decimal(z)                     # exact decimal value of the double
        ref = zd / 2 * (1 + _erf_series(zd / Decimal(2).sqrt()))
        # 1 + erf(.) cancels for negative z, so the double formula is good to ~1e-16 absolute
        assert kfo.act("gelu_erf", z) == pytest.approx(float(ref), rel=4e-15, abs=1e-15)


# ----------------------------------------------------------------------------- linear
def _exact_linear(X, W):
    """Exact rational X W^T of float arrays."""
    M, K = X.shape
    N = W.shape[0]
    out = np.empty((M, N))
    for i in range(M):
        for n in range(N):
            s = Fraction(0)
            for k in range(K):
                s += Fraction(float(X[i, k])) * Fraction(float(W[n, k]))
            out[i, n] = float(s)
    return out


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f64"])
def test_linear_bruteforce_exact_rational(dtype):
    r = rng(11)
    for M in (1, 2, 3, 5):
        for N in (1, 2, 3, 5):
            for K in (1, 2, 3, 5):
                X64 = r.standard_normal((M, K))
                W64 = r.standard_normal((N, K))
                if dtype == "f64":
                    X, W = X64, W64
                else:
                    X, W = inputs._store(X64, dtype), inputs._store(W64, dtype)
                ref = _exact_linear(inputs.to_f64(X), inputs.to_f64(W))
                got = kfo.linear_epilogue(X, W)
                assert got.shape == (M, N)
                np.testing.assert_allclose(got, ref, rtol=0, atol=1e-15 * K * 16)


def test_linear_nonsquare_catches_transposes_and_pitches():
    r = rng(12)
    M, N, K = 7, 11, 13
    Xbig = r.standard_normal((M, K + 5)).astype(np.float32)
    Wbig = r.standard_normal((N, K + 3)).astype(np.float32)
    X, W = Xbig[:, :K], Wbig[:, :K]          # row pitches larger than K
    ref = _exact_linear(X.astype(np.float64), W.astype(np.float64))
    np.testing.assert_allclose(kfo.linear_epilogue(X, W), ref, rtol=0, atol=1e-14)
    # element (i,n) depends on row i of X and row n of W only
    X2 = X.copy(); X2[3, :] = 0
    got = kfo.linear_epilogue(X2, W)
    assert np.all(got[3] == 0) and np.allclose(np.delete(got, 3, 0), np.delete(ref, 3, 0), atol=1e-14)


def test_linear_small_integers_are_exact():
    M, N, K = 6, 9, 17
    ones = np.ones((M, K), np.float32)
    assert np.all(kfo.linear_epilogue(ones, np.ones((N, K), np.float32)) == K)
    r = rng(13)
    Xi = r.integers(-8, 9, (M, K)).astype(np.float32)
    Wi = r.integers(-8, 9, (N, K)).astype(np.float32)
    assert np.array_equal(kfo.linear_epilogue(Xi, Wi), (Xi.astype(np.int64) @ Wi.astype(np.int64).T).astype(np.float64))
    # one-hot row of X selects column k of W (as a row of the output)
    Xh = np.zeros((K, K), np.float32); Xh[np.arange(K), np.arange(K)] = 1
    assert np.array_equal(kfo.linear_epilogue(Xh, Wi), Wi.T.astype(np.float64))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_identity_weight_reproduces_x_bit_exactly(dtype):
    r = rng(14)
    K = 24
    X = inputs._store(r.standard_normal((10, K)), dtype)
    I = inputs._store(np.eye(K), dtype)
    assert np.array_equal(kfo.linear_epilogue(X, I), inputs.to_f64(X))


def test_linear_power_of_two_scaling_is_exact():
    r = rng(15)
    X = r.standard_normal((5, 33)).astype(np.float32)
    W = r.standard_normal((4, 33)).astype(np.float32)
    assert np.array_equal(kfo.linear_epilogue(X * np.float32(4), W), 4 * kfo.linear_epilogue(X, W))


def test_bf16_bit_patterns_widen_exactly():
    bits = np.array([[0x3F80, 0x4049, 0xC000, 0x0000, 0x3F00]], dtype=np.uint16)   # 1, 3.140625, -2, 0, .5
    one = np.array([[0x3F80]], dtype=np.uint16)
    for j, want in enumerate((1.0, 3.140625, -2.0, 0.0, 0.5)):
        assert kfo.linear_epilogue(np.ascontiguousarray(bits[:, j:j + 1]), one)[0, 0] == want
    assert np.array_equal(kfo.row_norm(bits, "none"), [[1.0, 3.140625, -2.0, 0.0, 0.5]])


def test_linear_matches_library_matmul():
    torch = pytest.importorskip("torch")
    r = rng(16)
    X = r.standard_normal((37, 300)).astype(np.float32)
    W = r.standard_normal((53, 300)).astype(np.float32)
    ref = (torch.from_numpy(X).double() @ torch.from_numpy(W).double().T).numpy()
    np.testing.assert_allclose(kfo.linear_epilogue(X, W), ref, rtol=0, atol=1e-12)


# ----------------------------------------------------------------------------- epilogue
def test_epilogue_order_bias_act_scale_residual():
    # acc = 1, bias = 1, SiLU, scale 0.5, residual 3  ->  SiLU(2) * 0.5 + 3; any other order differs
    one = np.ones((1, 1), np.float32)
    got = kfo.linear_epilogue(one, one, bias=np.ones(1, np.float32), act="silu", scale=0.5,
                              residual=np.full((1, 1), 3, np.float32))[0, 0]
    assert got == pytest.approx(2 * GOLD["sigmoid_2.0"][0] * 0.5 + 3.0, abs=1e-15)
    # ReLU makes the position of the bias visible: relu(-1 + 0.25) = 0, not relu(-1) + 0.25
    got = kfo.linear_epilogue(-one, one, bias=np.full(1, 0.25, np.float32), act="relu", scale=2.0)[0, 0]
    assert got == 0.0
    got = kfo.linear_epilogue(one, one, bias=np.full(1, 0.25, np.float32), act="relu", scale=2.0,
                              residual=np.full((1, 1), -1, np.float32))[0, 0]
    assert got == 1.5


def test_scale_is_the_float32_value_widened():
    one = np.ones((1, 1), np.float32)
    got = kfo.linear_epilogue(one, one, scale=0.1)[0, 0]
    assert got == float(np.float32(0.1)) and got != 0.1


def test_zero_x_yields_epilogue_of_bias_alone():
    r = rng(17)
    M, N, K = 4, 9, 12
    W = r.standard_normal((N, K)).astype(np.float32)
    b = r.standard_normal(N).astype(np.float32)
    R = r.standard_normal((M, N)).astype(np.float32)
    got = kfo.linear_epilogue(np.zeros((M, K), np.float32), W, bias=b, act="gelu_erf", scale=0.5, residual=R)
    want = np.array([[0.5 * float(b[n]) * GOLD_PHI(float(b[n])) * 0.5 + float(R[i, n]) for n in range(N)]
                     for i in range(M)])
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-15)
    # K = 0 is the same statement with an empty sum
    got0 = kfo.linear_epilogue(np.zeros((M, 0), np.float32), np.zeros((N, 0), np.float32), bias=b, act="silu")
    want0 = np.array([[float(b[n]) / (1 + math.exp(-float(b[n]))) for n in range(N)]] * M)
    np.testing.assert_allclose(got0, want0, rtol=0, atol=1e-15)


def GOLD_PHI(z):
    """2*Phi(z) = 1 + erf(z/sqrt 2) through Python's own libm binding (not the oracle's code)."""
    return 1.0 + math.erf(z / math.sqrt(2.0))


# ----------------------------------------------------------------------------- softmax
def test_softmax_closed_forms():
    a = np.array([[0.0, math.log(2.0), math.log(3.0)]])
    np.testing.assert_allclose(kfo.row_softmax(a)[0], GOLD["softmax_0_ln2_ln3"], rtol=0, atol=1e-15)
    for N in (1, 2, 7, 256):
        assert np.all(kfo.row_softmax(np.full((3, N), 2.5, np.float32)) == 1.0 / N)
    # N = 2 is the logistic function of the difference
    for d in (-3.0, -0.5, 0.0, 1.0, 2.0):
        y = kfo.row_softmax(np.array([[d, 0.0]]))[0]
        sig = GOLD["sigmoid_1.0"][0] if d == 1.0 else (GOLD["sigmoid_2.0"][0] if d == 2.0 else 1 / (1 + math.exp(-d)))
        assert y[0] == pytest.approx(sig, abs=1e-15) and y[1] == pytest.approx(1 - sig, abs=1e-15)


def test_softmax_invariants_and_stability():
    r = rng(21)
    a = r.standard_normal((16, 133)) * 3
    y = kfo.row_softmax(a)
    np.testing.assert_allclose(y.sum(1), 1.0, rtol=0, atol=1e-13)
    assert np.all(y > 0)
    for c in (90.0, -90.0, 1000.0):
        np.testing.assert_allclose(kfo.row_softmax(a + c), y, rtol=1e-10, atol=0)
    # order preserving, row-wise
    assert np.array_equal(np.argsort(a, axis=1, kind="stable"), np.argsort(y, axis=1, kind="stable"))
    # ratio rule y_i / y_j = exp(a_i - a_j) pins the exponent's sign and base
    assert y[2, 5] / y[2, 9] == pytest.approx(math.exp(a[2, 5] - a[2, 9]), rel=1e-12)
    # logits that overflow a naive exp stay finite
    big = np.array([[1000.0, 999.0, -1000.0]])
    yb = kfo.row_softmax(big)[0]
    assert np.all(np.isfinite(yb)) and yb[0] == pytest.approx(1 / (1 + math.exp(-1.0)), abs=1e-15)
    # rows are independent
    a2 = a.copy(); a2[0] += 5 * r.standard_normal(133)
    assert np.array_equal(kfo.row_softmax(a2)[1:], y[1:])


def test_softmax_matches_library():
    torch = pytest.importorskip("torch")
    a = rng(22).standard_normal((9, 77)) * 4
    ref = torch.softmax(torch.from_numpy(a), dim=1).numpy()
    np.testing.assert_allclose(kfo.row_softmax(a), ref, rtol=1e-13, atol=0)


# ----------------------------------------------------------------------------- layernorm / rmsnorm
def test_layernorm_arithmetic_progression_closed_form():
    for N in (2, 5, 64, 1000):
        eps = 1e-5
        a = np.arange(N, dtype=np.float64)[None, :]
        mu = (N - 1) / 2.0
        v = (N * N - 1) / 12.0                  # biased variance of 0..N-1
        want = (a[0] - mu) / math.sqrt(v + float(np.float32(eps)))
        np.testing.assert_allclose(kfo.row_layernorm(a, eps=eps)[0], want, rtol=1e-14, atol=1e-15)
    # unbiased variance (N/(N-1)) would give a different, detectable answer at N = 2:
    y = kfo.row_layernorm(np.array([[0.0, 1.0]]), eps=0.0)[0]
    np.testing.assert_allclose(y, [-1.0, 1.0], atol=1e-15)


def test_layernorm_invariants():
    r = rng(31)
    N = 257
    a = r.standard_normal((12, N)) * 2 + 0.7
    eps = 1e-5
    e = float(np.float32(eps))
    y = kfo.row_layernorm(a, eps=eps)
    v = a.var(axis=1)
    np.testing.assert_allclose(y.mean(1), 0.0, atol=1e-14)
    np.testing.assert_allclose(y.var(axis=1), v / (v + e), rtol=1e-12)
    np.testing.assert_allclose(kfo.row_layernorm(a + 123.0, eps=eps), y, rtol=0, atol=1e-11)
    # LN(c x; c^2 eps) = LN(x; eps) for a power-of-two c (exact scaling of float32 eps)
    np.testing.assert_allclose(kfo.row_layernorm(a * 4.0, eps=16 * eps), y, rtol=1e-13, atol=1e-15)
    # eps sits inside the square root: with tiny variance the output shrinks by sqrt(v/(v+eps))
    tiny = np.array([[0.0, 2e-3]])              # v = 1e-6
    yt = kfo.row_layernorm(tiny, eps=eps)[0]
    assert yt[1] == pytest.approx(1e-3 / math.sqrt(1e-6 + e), rel=1e-12)
    # affine: gamma multiplies, beta adds, per column
    g = r.standard_normal(N); b = r.standard_normal(N)
    np.testing.assert_allclose(kfo.row_layernorm(a, g, b, eps), y * g + b, rtol=0, atol=1e-13)
    # degenerate rows
    assert np.array_equal(kfo.row_layernorm(np.full((2, 5), 3.25), None, np.arange(5.0), eps), [np.arange(5.0)] * 2)
    assert np.array_equal(kfo.row_layernorm(np.array([[7.0]]), np.array([2.0]), np.array([-1.5]), eps), [[-1.5]])


def test_layernorm_matches_library():
    torch = pytest.importorskip("torch")
    r = rng(32)
    a = r.standard_normal((6, 99)); g = r.standard_normal(99); b = r.standard_normal(99)
    eps = float(np.float32(1e-5))
    ref = torch.nn.functional.layer_norm(torch.from_numpy(a), (99,), torch.from_numpy(g), torch.from_numpy(b), eps).numpy()
    np.testing.assert_allclose(kfo.row_layernorm(a, g, b, 1e-5), ref, rtol=0, atol=1e-13)


def test_rmsnorm_closed_forms():
    eps = 1e-5
    e = float(np.float32(eps))
    y = kfo.row_rmsnorm(np.array([[3.0, 4.0]]), eps=0.0)[0]          # mean square 12.5
    np.testing.assert_allclose(y, [3 / math.sqrt(12.5), 4 / math.sqrt(12.5)], rtol=1e-15)
    c = -2.5
    y = kfo.row_rmsnorm(np.full((1, 9), c), np.arange(9.0), eps)[0]
    np.testing.assert_allclose(y, c / math.sqrt(c * c + e) * np.arange(9.0), rtol=1e-15)
    a = rng(33).standard_normal((5, 40))
    y = kfo.row_rmsnorm(a, eps=eps)
    ms = (a * a).mean(1)
    np.testing.assert_allclose((y * y).mean(1), ms / (ms + e), rtol=1e-12)   # no mean subtraction
    assert abs(kfo.row_rmsnorm(a + 10.0, eps=eps).mean()) > 0.5              # and not shift invariant


# ----------------------------------------------------------------------------- fused = composition
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("norm", ["softmax", "layernorm", "rmsnorm"])
def test_fused_equals_composition_and_library_chain(dtype, norm):
    torch = pytest.importorskip("torch")
    F = torch.nn.functional
    r = rng(41)
    M, N, K = 9, 37, 50
    X = inputs._store(r.standard_normal((M, K)) / 4, dtype)
    W = inputs._store(r.standard_normal((N, K)) / 4, dtype)
    b = inputs._store(r.standard_normal(N) / 4, dtype)
    R = inputs._store(r.standard_normal((M, N)), dtype)
    g = inputs._store(1 + r.standard_normal(N) / 10, dtype)
    be = inputs._store(r.standard_normal(N) / 10, dtype)
    eps = 1e-5
    for act, tact in (("gelu_erf", lambda t: F.gelu(t)), ("gelu_tanh", lambda t: F.gelu(t, approximate="tanh")),
                      ("silu", F.silu), ("relu", F.relu), ("sigmoid", torch.sigmoid), ("none", lambda t: t)):
        fused = kfo.linear_epilogue_rownorm(X, W, b, act, 0.5, R, norm, g, be, eps)
        pre = kfo.linear_epilogue(X, W, b, act, 0.5, R)
        g64, be64 = inputs.to_f64(g), inputs.to_f64(be)
        comp = kfo.row_norm(pre, norm, g64, be64 if norm == "layernorm" else None, eps)
        np.testing.assert_allclose(fused, comp, rtol=0, atol=1e-14)
        # independent library chain in float64
        t = F.linear(torch.from_numpy(inputs.to_f64(X)), torch.from_numpy(inputs.to_f64(W)), torch.from_numpy(inputs.to_f64(b)))
        t = tact(t) * float(np.float32(0.5)) + torch.from_numpy(inputs.to_f64(R))
        e = float(np.float32(eps))
        if norm == "softmax":
            t = torch.softmax(t, dim=1)
        elif norm == "layernorm":
            t = F.layer_norm(t, (N,), torch.from_numpy(g64), torch.from_numpy(be64), e)
        else:
            t = t / torch.sqrt((t * t).mean(dim=1, keepdim=True) + e) * torch.from_numpy(g64)
        np.testing.assert_allclose(fused, t.numpy(), rtol=0, atol=2e-12)


def test_degenerate_shapes():
    X = np.zeros((0, 4), np.float32); W = np.ones((3, 4), np.float32)
    assert kfo.linear_epilogue_rownorm(X, W, norm="softmax").shape == (0, 3)
    assert kfo.linear_epilogue_rownorm(np.ones((2, 4), np.float32), np.zeros((0, 4), np.float32), norm="layernorm").shape == (2, 0)
    y = kfo.linear_epilogue_rownorm(np.ones((2, 4), np.float32), np.ones((1, 4), np.float32), norm="softmax")
    assert np.array_equal(y, [[1.0], [1.0]])


# ----------------------------------------------------------------------------- input generator
def test_bf16_rounding_is_nearest_even_and_matches_library():
    torch = pytest.importorskip("torch")
    f = np.array([1.0, 1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -20, -1 - 2.0 ** -8, 0.0, 3.14159265],
                 dtype=np.float32)
    bits = inputs.f32_to_bf16_bits(f)
    assert list(bits[:5]) == [0x3F80, 0x3F80, 0x3F82, 0x3F81, 0xBF80]
    x = (rng(51).standard_normal(100000) * np.exp(rng(52).standard_normal(100000) * 5)).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(inputs.f32_to_bf16_bits(x), ref)
    assert np.array_equal(inputs.bf16_bits_to_f32(ref), torch.from_numpy(ref.view(np.int16)).view(torch.bfloat16).float().numpy())


def test_config_recipes_are_seeded_and_shaped():
    p = inputs.config(1)
    assert (p.M, p.N, p.K, p.dtype, p.act, p.norm) == (128, 256, 256, "f32", "gelu_erf", "softmax")
    assert p.flops == 16_777_216 and p.algorithmic_bytes == 525_312
    q = inputs.config(1)
    assert np.array_equal(p.X, q.X) and np.array_equal(p.W, q.W) and np.array_equal(p.bias, q.bias)
    assert abs(float(p.X.std()) - 1 / 16) < 2e-3
    p4 = inputs.config(4, rows=8)
    assert p4.X.shape == (8, 2048) and p4.W.shape == (8192, 2048) and p4.X.dtype == np.uint16
    assert abs(float(inputs.to_f64(p4.W).std()) - 0.02) < 1e-4
    assert abs(float(inputs.to_f64(p4.gamma).mean()) - 1.0) < 1e-2
