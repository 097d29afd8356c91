"""Pins for the quantized EMA (Eq. 2-4) against the paper's analysis.

Theorem 3.1 (sufficient condition for a swamped state), Corollary 3.2 and the
spec swamping demonstration, Example 3.3, Proposition 3.5 (exact decay),
Theorem 3.6 (stochastic rounding is unbiased, variance bound).
"""
import math

import numpy as np
import pytest

import oracle


def radius(y, q):
    """r of Thm 3.1: half the smaller gap to a neighbouring level."""
    gaps = []
    if q > 0:
        gaps.append(y[q] - y[q - 1])
    if q < len(y) - 1:
        gaps.append(y[q + 1] - y[q])
    return 0.5 * float(min(gaps))


@pytest.mark.parametrize("kind", [oracle.LINEAR_UNSIGNED, oracle.DE_UNSIGNED, oracle.LINEAR_NOZERO,
                                  oracle.DE_SIGNED])
def test_theorem_3_1_swamping_condition(kind):
    """Whenever r >= (1-beta)|z/D' - y_q| + |D/D' - 1| the code does not move."""
    rng = np.random.default_rng(kind)
    held = 0
    for trial in range(400):
        bits = int(rng.choice([2, 3, 4]))
        y = oracle.codebook(kind, bits)
        n = 64
        signed = kind == oracle.DE_SIGNED
        codes = rng.integers(0, len(y), n).astype(np.int32)
        codes[0] = len(y) - 1                       # one element sits on the top level
        delta = float(np.float32(math.exp(rng.uniform(-8, 2))))
        beta = float(rng.choice([0.9, 0.99, 0.999, 0.5]))
        z = (rng.uniform(-1 if signed else 0, 1, n) * delta * rng.choice([0.01, 0.5, 1.0])).astype(np.float32)
        before = codes.copy()
        new_delta, _ = oracle.qema(oracle.NEAREST, kind, bits, codes, delta, 0.5, z, beta)
        assert new_delta > 0
        for i in range(n):
            q = int(before[i])
            rhs = (1 - beta) * abs(float(z[i]) / new_delta - float(y[q])) + abs(delta / new_delta - 1)
            if radius(y, q) >= rhs + 1e-6:          # small slack for binary32 rounding
                assert codes[i] == q
                held += 1
    assert held > 1000                              # the condition was actually exercised


def test_swamping_linear_stuck_log_moves():
    """A small second-moment increment moves the log-quantized state where a linear unsigned
    quantizer leaves it unchanged (Cor. 3.2: beta >= 0.967 / 0.833 swamps every level)."""
    n, beta = 128, 0.999
    rng = np.random.default_rng(0)
    for bits in (4, 2):
        y = oracle.codebook(oracle.LINEAR_UNSIGNED, bits)
        mid = len(y) // 2
        codes = np.full(n, mid, np.int32)
        codes[0] = len(y) - 1
        start = codes.copy()
        delta = 1.0
        z = np.full(n, 0.01, np.float32)            # signal far below the state (0.5)
        z[0] = 1.0                                  # keeps Delta pinned at 1
        for _ in range(300):
            delta, _ = oracle.qema(oracle.NEAREST, oracle.LINEAR_UNSIGNED, bits, codes, delta, 0.5,
                                   z, beta)
        assert delta == 1.0 and np.array_equal(codes, start)       # swamped: never moved

        # SOLO: same start value (0.5 -> a level of the log codebook), same signal
        K = 1 << bits
        lcodes = np.full(n, 1, np.int32)
        lcodes[0] = 0
        ldelta, lalpha = 1.0, 0.5                   # level 1 = 0.5
        first = None
        for it in range(300):
            rnd = rng.integers(0, 1 << 32, n, dtype=np.uint64).astype(np.uint32)
            ldelta, lalpha = oracle.qema(oracle.LOG, 0, bits, lcodes, ldelta, lalpha, z, beta,
                                         p_quantile=0.1, rnd=rnd)
            if first is None and np.any(lcodes[1:] != 1):
                first = it
        state = np.array([oracle.pow_sm(lalpha, int(q)) * ldelta for q in lcodes[1:]])
        true = 0.5 * beta ** 300 + 0.01 * (1 - beta ** 300)
        assert first is not None and first < 50
        assert state.mean() < 0.46                                  # moved toward the signal
        assert abs(state.mean() - true) < 0.05                      # and tracks the true EMA


def test_example_3_3_uniform_signals():
    """X in R^1000, states and signals ~ U[0,1]: with beta -> 1 linear / DE stay where they
    started while the log quantizer follows the full-precision EMA towards E[z] = 0.5."""
    n, iters, beta, bits = 1000, 100, 0.99, 4
    rng = np.random.default_rng(33)
    x0 = rng.uniform(0, 1, n).astype(np.float32)
    signals = rng.uniform(0, 1, (iters, n)).astype(np.float32)
    exact = x0.astype(np.float64)
    for t in range(iters):
        exact = beta * exact + (1 - beta) * signals[t]

    def run(mode, kind):
        delta = float(x0.max())
        if mode == oracle.LOG:
            alpha, inv = oracle.log_base(float(np.sort(x0)[99]), delta, 1 << bits)
            codes = np.array([oracle.quant_log(float(x / delta), inv, 0.0, 1 << bits) for x in x0], np.int32)
        else:
            alpha = 0.5
            y = oracle.codebook(kind, bits)
            codes = np.array([oracle.quant_nearest(y, float(x / delta)) for x in x0], np.int32)
        start = codes.copy()
        for t in range(iters):
            rnd = rng.integers(0, 1 << 32, n, dtype=np.uint64).astype(np.uint32)
            delta, alpha = oracle.qema(mode, kind, bits, codes, delta, alpha, signals[t], beta, rnd=rnd)
        if mode == oracle.LOG:
            val = np.array([oracle.pow_sm(alpha, int(q)) for q in codes]) * delta
        else:
            val = oracle.codebook(kind, bits)[codes] * delta
        return val, float(np.mean(codes != start))

    lin, lin_changed = run(oracle.NEAREST, oracle.LINEAR_UNSIGNED)
    de, de_changed = run(oracle.NEAREST, oracle.DE_UNSIGNED)
    log, log_changed = run(oracle.LOG, 0)
    # 4-bit linear is swamped for beta >= 0.967, 4-bit DE for half its levels at beta >= 0.966:
    # their states keep the spread of the initial U[0,1] draw instead of contracting to 0.5
    assert lin_changed < 0.02 and de_changed < 0.1 and log_changed > 0.5
    err = lambda v: float(np.mean(np.abs(v - exact)))
    assert err(log) < 0.5 * err(lin) and err(log) < 0.5 * err(de)
    assert lin.std() > 2 * exact.std() and de.std() > 2 * exact.std()
    assert abs(log.std() - exact.std()) < 0.03 and abs(log.mean() - exact.mean()) < 0.05


@pytest.mark.parametrize("c,beta", [(4, 0.9), (2, 0.8), (10, 0.99)])
def test_proposition_3_5_exact_decay(c, beta):
    """Zero signals, base alpha = beta^c: a level drops with probability 1/c per step, so s
    levels take c*s steps on average."""
    n, bits, s = 100_001, 8, 5
    alpha = float(np.float32(beta ** c))
    rng = np.random.default_rng(c)
    codes = np.full(n, 3, np.int32)
    codes[0] = 0
    z = np.zeros(n, np.float32)
    z[0] = 1.0                                      # element 0 stays at Delta = 1
    delta, a = 1.0, alpha
    reached = np.zeros(n, np.int64)
    drops = []
    for it in range(1, 40 * c + 1):
        before = codes.copy()
        rnd = rng.integers(0, 1 << 32, n, dtype=np.uint64).astype(np.uint32)
        delta, a = oracle.qema(oracle.LOG, 0, bits, codes, delta, a, z, beta, fixed_alpha=alpha, rnd=rnd)
        assert delta == 1.0 and codes[0] == 0
        step = codes[1:] - before[1:]
        assert set(np.unique(step)) <= {0, 1}       # a level is never skipped, never regained
        if it <= 5:
            drops.append(step.mean())
        newly = (codes >= 3 + s) & (reached == 0)
        reached[newly] = it
    assert np.all(reached[1:] > 0)
    p = float(np.mean(drops))
    assert abs(p - 1 / c) < 4 * math.sqrt((1 / c) * (1 - 1 / c) / (5 * n)) + 2e-5
    mean_steps = reached[1:].mean()
    sd = math.sqrt(s * (1 - 1 / c)) * c             # negative binomial
    assert abs(mean_steps - c * s) < 5 * sd / math.sqrt(n) + 1e-3 * c * s


@pytest.mark.parametrize("bits", [2, 4])
def test_theorem_3_6_stochastic_rounding(bits):
    """Eq. 5 is unbiased and its variance is at most (r_max * Delta)^2."""
    y = oracle.codebook(oracle.DE_SIGNED, bits)
    r_max = float(np.max(np.diff(y)) / 2)
    n = 400_001
    rng = np.random.default_rng(bits)
    for x in (0.3, -0.2, 0.013, 0.77, -0.5):
        z = np.full(n, x, np.float32)
        z[0] = 1.0                                  # Delta = 1
        codes = np.zeros(n, np.int32)
        rnd = rng.integers(0, 1 << 32, n, dtype=np.uint64).astype(np.uint32)
        delta, _ = oracle.qema(oracle.STOCHASTIC, oracle.DE_SIGNED, bits, codes, 0.0, 0.5, z, 0.0, rnd=rnd)
        assert delta == 1.0
        v = y[codes[1:]].astype(np.float64)
        assert len(np.unique(codes[1:])) <= 2       # only the two bracketing levels
        assert v.var() <= r_max ** 2 + 1e-9
        assert abs(v.mean() - x) < 5 * math.sqrt(max(v.var(), 1e-12) / n) + 1e-6
