"""Pins for the oracle's full optimizer step (Sec. 3.1 Eq. 2-4, Sec. 3.4).

Textbook Adam / AdamW through the full-precision switch, the first step from a
zero state, per-block scales / quantile / codes re-derived with numpy, tails,
all-zero blocks, zeros inside a block, threading and the random stream.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2505_00347_b200 import synth


def rand_inputs(n, seed, gscale=1e-3):
    rng = np.random.default_rng(seed)
    p = rng.normal(0, 0.02, n).astype(np.float32)
    g = torch.from_numpy(rng.normal(0, gscale, n).astype(np.float32)).to(torch.bfloat16)
    return p, synth.bf16_bits(g), g.float().numpy()


@pytest.mark.parametrize("adamw", [1, 0])
def test_full_precision_switch_is_textbook_adam(adamw):
    """With quantization switched off the same EMA / update lines must reproduce
    torch.optim.AdamW (decoupled decay) and torch.optim.Adam (L2 in the gradient)."""
    n, steps = 1000, 10
    p0, _, _ = rand_inputs(n, 1)
    h = oracle.hyper(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1, adamw=adamw)
    tp = torch.nn.Parameter(torch.from_numpy(p0.copy()).double())
    cls = torch.optim.AdamW if adamw else torch.optim.Adam
    opt = cls([tp], lr=1e-2, betas=(float(np.float32(0.9)), float(np.float32(0.999))), eps=1e-8,
              weight_decay=float(np.float32(0.1)))
    p = p0.copy()
    st = oracle.State(n, 4, 4, 128)
    m32, v32 = np.zeros(n, np.float32), np.zeros(n, np.float32)
    for t in range(1, steps + 1):
        _, gb, gf = rand_inputs(n, 100 + t)
        tp.grad = torch.from_numpy(gf).double()
        opt.step()
        oracle.step(p, gb, st, h, t, m32=m32, v32=v32)
        ref = tp.detach().numpy()
        # binary32 storage of p: half an ulp of |p| <= 0.1 per step, plus 1e-6 relative
        assert np.all(np.abs(p - ref) <= 1e-6 * np.abs(ref) + 4e-9 * t), t
    assert np.allclose(m32, opt.state[tp]["exp_avg"].numpy(), rtol=1e-5, atol=1e-9)
    assert np.allclose(v32, opt.state[tp]["exp_avg_sq"].numpy(), rtol=1e-5, atol=1e-15)
    assert np.all(st.codes_m == 0) and np.all(st.scale_m == 0)      # packed state untouched


def test_full_precision_switch_is_textbook_adabelief():
    """AdaBelief (Zhuang et al. 2020) written out in binary64 numpy: m = b1 m + (1-b1) g,
    s = b2 s + (1-b2) (g - m)^2 + eps, p <- p (1 - lr wd) - lr (m / bc1) / (sqrt(s / bc2) + eps).
    With quantization switched off the oracle's belief mode must follow it."""
    n, steps = 1000, 12
    p0, _, _ = rand_inputs(n, 7)
    lr, wd, eps = 1e-2, 0.1, 1e-10
    b1, b2 = float(np.float32(0.9)), float(np.float32(0.999))
    h = oracle.hyper(lr=lr, beta1=0.9, beta2=0.999, eps=eps, weight_decay=wd, belief=1)
    lr, wd, eps = float(np.float32(lr)), float(np.float32(wd)), float(np.float32(eps))
    ref, m, sv = p0.astype(np.float64), np.zeros(n), np.zeros(n)
    p = p0.copy()
    st = oracle.State(n, 4, 4, 128)
    m32, v32 = np.zeros(n, np.float32), np.zeros(n, np.float32)
    for t in range(1, steps + 1):
        _, gb, gf = rand_inputs(n, 300 + t)
        g = gf.astype(np.float64)
        m = b1 * m + (1 - b1) * g
        sv = b2 * sv + (1 - b2) * (g - m) ** 2 + eps
        ref = ref * (1 - lr * wd) - lr * (m / (1 - b1 ** t)) / (np.sqrt(sv / (1 - b2 ** t)) + eps)
        oracle.step(p, gb, st, h, t, m32=m32, v32=v32)
        assert np.all(np.abs(p - ref) <= 2e-6 * np.abs(ref) + 4e-9 * t), t
    assert np.allclose(m32, m, rtol=1e-5, atol=1e-9) and np.allclose(v32, sv, rtol=1e-4, atol=1e-16)
    # and it is not Adam: the same run without the flag ends elsewhere
    q = p0.copy()
    m32b, v32b = np.zeros(n, np.float32), np.zeros(n, np.float32)
    hb = oracle.hyper(lr=lr, beta1=0.9, beta2=0.999, eps=eps, weight_decay=wd)
    for t in range(1, steps + 1):
        _, gb, _ = rand_inputs(n, 300 + t)
        oracle.step(q, gb, st, hb, t, m32=m32b, v32=v32b)
    assert np.abs(q - p).max() > 1e-4


def test_fixed_base_mode_is_plain_logarithmic_quantization():
    """fixed_alpha keeps the base (the standard logarithmic quantizer the paper contrasts with,
    alpha = 1/2, and the setting of Prop. 3.5): every block stores that base and every code is
    the rounded log_alpha(v^/Delta) + xi, re-derived here in binary64."""
    n, block, bits = 128 * 5 + 40, 128, 3
    p, _, _ = rand_inputs(n, 11)
    st = oracle.State(n, 4, bits, block)
    for alpha in (0.5, 0.8):
        h = oracle.hyper(seed=5, fixed_alpha=alpha)
        for t in (1, 2, 3):
            _, gb, _ = rand_inputs(n, 40 + t)
            _, vh, _ = oracle.step(p, gb, st, h, t, want_hat=True)
            assert np.all(st.alpha == np.float32(alpha))
            for j in range(st.nblk):
                sl = slice(j * block, min(n, (j + 1) * block))
                assert st.scale_v[j] == vh[sl].max()
                r = vh[sl].astype(np.float64) / float(st.scale_v[j])
                for e in range(sl.stop - sl.start):
                    xi = oracle.xi(oracle.philox_draw16(5, t, 0, sl.start + e, 0))
                    tt = math.log(r[e]) / math.log(float(np.float32(alpha))) + xi if r[e] > 0 else 99
                    q_ref = int(min(max(round(tt), 0), (1 << bits) - 1))
                    q = oracle.get_code(st.codes_v[j * (block * bits // 8):], e, bits)
                    assert q == q_ref or abs(tt - math.floor(tt) - 0.5) < 2e-4, (alpha, t, j, e, tt, q)
    # the quantile mode chooses its own base: a different state from the same inputs
    st2 = oracle.State(n, 4, bits, block)
    _, gb, _ = rand_inputs(n, 41)
    oracle.step(p.copy(), gb, st2, oracle.hyper(seed=5), 1)
    assert not np.all(st2.alpha == np.float32(0.8))


def test_first_step_from_zero_state():
    """From the zero state the EMA sees no quantization: m^ = (1-b1) g, v^ = (1-b2) g^2 and the
    parameter moves by the bias-corrected AdamW step."""
    n = 128 * 5 + 17
    p, gb, gf = rand_inputs(n, 2)
    p0 = p.copy()
    h = oracle.hyper(lr=1e-3, beta1=0.8, beta2=0.999, weight_decay=0.01)
    st = oracle.State(n, 4, 4, 128)
    mh, vh, _ = oracle.step(p, gb, st, h, 1, want_hat=True)
    b1, b2 = np.float32(0.8), np.float32(0.999)
    assert np.allclose(mh, (1 - b1) * gf, rtol=1e-6, atol=0)
    assert np.allclose(vh, (1 - b2) * gf * gf, rtol=1e-6, atol=0)
    g64 = gf.astype(np.float64)
    ref = p0 * (1 - 1e-3 * 0.01) - 1e-3 * g64 / (np.abs(g64) + 1e-8)   # m^/bc1 = g, sqrt(v^/bc2) = |g|
    assert np.allclose(p, ref, rtol=2e-6, atol=1e-9)


@pytest.mark.parametrize("bits_m,bits_v,block", [(4, 4, 128), (2, 3, 128), (3, 3, 64), (8, 8, 256),
                                                 (4, 2, 2048)])
def test_block_quantities_rederived(bits_m, bits_v, block):
    """After a few steps: scales are block maxima, the base puts level K-1 on the p-quantile,
    codes are the nearest levels (re-derived with numpy in binary64)."""
    n = block * 6 + block // 3 + 1
    p, _, _ = rand_inputs(n, 3)
    h = oracle.hyper(beta1=0.8, seed=99)
    st = oracle.State(n, bits_m, bits_v, block)
    Km, Kv = 1 << bits_m, 1 << bits_v
    ym = oracle.codebook(oracle.DE_SIGNED, bits_m).astype(np.float64)
    mids = 0.5 * (ym[:-1] + ym[1:])
    for t in range(1, 5):
        _, gb, _ = rand_inputs(n, 30 + t, gscale=1e-3 * t)
        mh, vh, fl = oracle.step(p, gb, st, h, t, tensor=2, want_hat=True, want_flags=True)
        dm, dv = oracle.dequant(st, 0), oracle.dequant(st, 1)
        for j in range(st.nblk):
            sl = slice(j * block, min(n, (j + 1) * block))
            nb = sl.stop - sl.start
            assert st.scale_m[j] == np.abs(mh[sl]).max() and st.scale_v[j] == vh[sl].max()
            k = max(1, math.ceil(float(np.float32(0.1)) * nb))
            x_p = np.sort(vh[sl])[k - 1]
            rho = min(max(float(x_p) / float(st.scale_v[j]), 2.0 ** -48), 1 - 2.0 ** -10)
            a = float(st.alpha[j])
            assert 0 < a < 1 and a ** (Kv - 1) == pytest.approx(rho, rel=2e-4)
            # first moment: nearest level
            r = mh[sl].astype(np.float64) / float(st.scale_m[j])
            q_ref = (r[:, None] > mids[None, :]).sum(1)
            q = np.array([oracle.get_code(st.codes_m[j * (block * bits_m // 8):], e, bits_m) for e in range(nb)])
            near = np.min(np.abs(r[:, None] - mids[None, :]), axis=1) < 1e-6
            assert np.all((q == q_ref) | near)
            # second moment: Eq. 6 with the element's own xi
            rv = vh[sl].astype(np.float64) / float(st.scale_v[j])
            qv = np.array([oracle.get_code(st.codes_v[j * (block * bits_v // 8):], e, bits_v) for e in range(nb)])
            for e in range(nb):
                w = oracle.philox_draw16(99, t, 2, sl.start + e, 0)
                tt = math.log(rv[e]) / math.log(a) + oracle.xi(w) if rv[e] > 0 else Kv
                q_ref_v = int(min(max(round(tt), 0), Kv - 1))
                assert qv[e] == q_ref_v or abs(tt - math.floor(tt) - 0.5) < 2e-4, (j, e, tt, qv[e])
            # dequantized state: sign / positivity, never above the scale
            assert np.all(dv[sl] > 0) and np.all(dv[sl] <= st.scale_v[j])
            assert np.all((dm[sl] == 0) | (np.sign(dm[sl]) == np.sign(mh[sl])))
            assert np.all(np.abs(dm[sl]) <= st.scale_m[j])
        # bf16 gradients make exact ties (e.g. g_i / g_max = -11/40 on the 2-bit midpoint
        # -0.275) possible at step 1; they are rare
        assert fl.mean() < 0.01


def test_zero_gradients_and_zero_blocks():
    n, block = 128 * 3 + 5, 128
    p, gb, _ = rand_inputs(n, 4)
    gb[128:256] = 0                      # one all-zero block
    gb[300] = 0                          # a zero inside a non-zero block
    h = oracle.hyper(weight_decay=0.0)
    st = oracle.State(n, 2, 3, block)
    p0 = p.copy()
    oracle.step(p, gb, st, h, 1)
    assert st.scale_m[1] == 0 and st.scale_v[1] == 0 and st.alpha[1] == 0.5
    assert np.all(st.codes_m[32:64] == 0) and np.all(st.codes_v[48:96] == 0)
    assert np.array_equal(p[128:256], p0[128:256])          # no gradient, no decay: unchanged
    dv, dm = oracle.dequant(st, 1), oracle.dequant(st, 0)
    assert np.all(dv[128:256] == 0) and np.all(dm[128:256] == 0)
    assert oracle.get_code(st.codes_v[2 * 48:], 300 - 256, 3) == 7   # zero element -> smallest level
    assert dv[300] > 0 and dm[300] == 0
    # >= 10 % zeros in a block: the quantile is 0 and the base is clamped, not 0
    gb2 = gb.copy()
    gb2[0:20] = 0
    st2 = oracle.State(n, 2, 3, block)
    oracle.step(p0.copy(), gb2, st2, h, 1)
    assert st2.alpha[0] == pytest.approx(2.0 ** (-48 / 7), rel=1e-6)
    # a block that goes quiet decays; its scale shrinks by beta each step, never negative
    zeros = np.zeros(n, np.uint16)
    before = oracle.dequant(st, 1).copy()
    for t in range(2, 6):
        oracle.step(p, zeros, st, h, t)
    after = oracle.dequant(st, 1)
    assert np.all(after >= 0) and after[:128].max() == pytest.approx(before[:128].max() * 0.999 ** 4, rel=1e-5)


@pytest.mark.parametrize("n", [1, 2, 63, 64, 65, 127, 129])
def test_tiny_and_ragged_tensors(n):
    p, gb, gf = rand_inputs(n, 5 + n)
    h = oracle.hyper()
    st = oracle.State(n, 4, 4, 128)
    assert st.nblk == (n + 127) // 128 and st.codes_m.size == st.nblk * 64
    for t in range(1, 4):
        mh, vh, _ = oracle.step(p, gb, st, h, t, want_hat=True)
    assert st.scale_m[0] == np.abs(mh[:128]).max()
    assert np.all(np.isfinite(p))
    tail = n % 128
    if tail:    # padding codes of the tail block stay zero
        last = st.codes_m[(st.nblk - 1) * 64:]
        assert all(oracle.get_code(last, e, 4) == 0 for e in range(tail, 128))
    if n == 1:  # a single element is its own maximum and its own quantile
        assert oracle.get_code(st.codes_m, 0, 4) in (0, 15)
        assert oracle.get_code(st.codes_v, 0, 4) in (0, 1)
        assert st.alpha[0] == pytest.approx((1 - 2.0 ** -10) ** (1 / 15), rel=1e-6)


def test_threads_slices_and_stream():
    n, block = 128 * 37 + 11, 128
    p, gb, _ = rand_inputs(n, 6)
    h = oracle.hyper(seed=7)
    runs = []
    for nthreads in (1, 4):
        pp, st = p.copy(), oracle.State(n, 3, 3, block)
        for t in range(1, 4):
            oracle.step(pp, gb, st, h, t, nthreads=nthreads)
        runs.append((pp, st))
    for k in ("codes_m", "codes_v", "scale_m", "scale_v", "alpha"):
        assert np.array_equal(getattr(runs[0][1], k), getattr(runs[1][1], k))
    assert np.array_equal(runs[0][0], runs[1][0])
    # a slice that starts at block 5 with elem_offset set reproduces the full run's blocks
    full_p, full = p.copy(), oracle.State(n, 3, 3, block)
    oracle.step(full_p, gb, full, h, 1, tensor=4)
    lo = 5 * block
    sl_p, sl = p[lo:].copy(), oracle.State(n - lo, 3, 3, block)
    oracle.step(sl_p, gb[lo:].copy(), sl, h, 1, tensor=4, elem_offset=lo)
    assert np.array_equal(sl.codes_v, full.codes_v[5 * 48:]) and np.array_equal(sl_p, full_p[lo:])
    # the stream depends on seed, step and tensor
    other = oracle.State(n, 3, 3, block)
    oracle.step(p.copy(), gb, other, h, 1, tensor=5)
    assert not np.array_equal(other.codes_v, full.codes_v)
    assert np.array_equal(other.codes_m, full.codes_m)          # nearest rounding draws nothing
    det = oracle.State(n, 3, 3, block)
    oracle.step(p.copy(), gb, det, oracle.hyper(seed=7, round_v=0), 1, tensor=5)
    det2 = oracle.State(n, 3, 3, block)
    oracle.step(p.copy(), gb, det2, oracle.hyper(seed=8, round_v=0), 1, tensor=9)
    assert np.array_equal(det.codes_v, det2.codes_v)            # xi = 0: no randomness


def test_bf16_parameters_and_stochastic_m():
    n = 128 * 4
    p, gb, _ = rand_inputs(n, 8)
    pb = synth.bf16_bits(torch.from_numpy(p).to(torch.bfloat16))
    pf = synth.bits_to_bf16(pb).float().numpy().copy()
    h16 = oracle.hyper(param_dtype=1, lr=1e-2)
    h32 = oracle.hyper(param_dtype=0, lr=1e-2)
    s16, s32 = oracle.State(n, 4, 4, 128), oracle.State(n, 4, 4, 128)
    oracle.step(pb, gb, s16, h16, 1)
    oracle.step(pf, gb, s32, h32, 1)
    want = synth.bf16_bits(torch.from_numpy(pf).to(torch.bfloat16))     # torch rounds to nearest even
    assert np.array_equal(pb, want)
    assert np.array_equal(s16.codes_v, s32.codes_v)
    # stochastic first moment: codes bracket the nearest ones and differ somewhere
    hs = oracle.hyper(round_m=1, seed=3)
    ss, sn = oracle.State(n, 4, 4, 128), oracle.State(n, 4, 4, 128)
    oracle.step(p.copy(), gb, ss, hs, 1)
    oracle.step(p.copy(), gb, sn, oracle.hyper(seed=3), 1)
    a = np.array([oracle.get_code(ss.codes_m, e, 4) for e in range(128)])
    b = np.array([oracle.get_code(sn.codes_m, e, 4) for e in range(128)])
    assert np.max(np.abs(a - b)) <= 1 and np.any(a != b)


def test_bf16_parameters_stochastic_rounding():
    """bf16 parameters with param_round=1: each stored value is the binary32 result of the same
    step rounded with the element's own purpose-2 draw; the states do not depend on the rounding
    of the parameter; over many elements the rounding error averages out (nearest does not when
    the update is far below half an ulp)."""
    import struct
    n, seed, tensor = 128 * 5 + 17, 0xABCDEF0123, 4
    p, gb, _ = rand_inputs(n, 11)
    pb = synth.bf16_bits(torch.from_numpy(p).to(torch.bfloat16))
    pf = synth.bits_to_bf16(pb).float().numpy().copy()
    hs = oracle.hyper(param_dtype=1, param_round=1, lr=1e-2, seed=seed)
    hf = oracle.hyper(param_dtype=0, lr=1e-2, seed=seed)
    s16, s32 = oracle.State(n, 2, 3, 128), oracle.State(n, 2, 3, 128)
    for t in (1, 2):
        before = synth.bits_to_bf16(pb).float().numpy().copy()
        pf[:] = before
        oracle.step(pb, gb, s16, hs, t, tensor=tensor, elem_offset=1280)
        oracle.step(pf, gb, s32, hf, t, tensor=tensor, elem_offset=1280)
        for i in range(n):
            d = oracle.philox_draw16(seed, t, tensor, 1280 + i, 2)
            bits = struct.unpack("<I", struct.pack("<f", float(pf[i])))[0]
            assert int(pb[i]) == ((bits + d) >> 16) & 0xffff, (t, i)
        assert np.array_equal(s16.codes_v, s32.codes_v) and np.array_equal(s16.codes_m, s32.codes_m)
    # an update of 1/64 ulp: nearest rounding never moves the parameter, stochastic rounding
    # moves it by the right amount on average
    n = 1 << 15
    ones = np.full(n, 0x3F80, np.uint16)                       # 1.0; ulp(bf16) = 2^-7 above 1
    g = synth.bf16_bits(torch.full((n,), -1.0).to(torch.bfloat16))
    lr = 2.0 ** -13
    for rnd, moved in ((0, False), (1, True)):
        pb = ones.copy()
        h = oracle.hyper(param_dtype=1, param_round=rnd, lr=lr, weight_decay=0.0, seed=5,
                         bias_correction=1, eps=0.0)
        oracle.step(pb, g, oracle.State(n, 4, 4, 128), h, 1)   # first Adam step: p += lr exactly
        val = synth.bits_to_bf16(pb).float().numpy().astype(np.float64)
        if moved:
            assert abs(val.mean() - (1.0 + lr)) < 4 * (2.0 ** -7) * math.sqrt(1 / 64 / n)
        else:
            assert np.all(val == 1.0)


@pytest.mark.parametrize("sel,kind", [(1, "DE_UNSIGNED"), (2, "LINEAR_UNSIGNED"), (3, "LINEAR_NOZERO")])
@pytest.mark.parametrize("bits_v", [2, 4])
def test_baseline_second_moment_codebooks(sel, kind, bits_v):
    """v_codebook != 0 (Sec. 4, "Baselines"): block-wise absmax scaling, codes are the nearest
    level by exhaustive search, dequantization is level times scale, the base is not touched."""
    n, block = 128 * 4 + 40, 128
    p, _, _ = rand_inputs(n, 21)
    y = oracle.codebook(getattr(oracle, kind), bits_v).astype(np.float64)
    h = oracle.hyper(beta1=0.8, seed=3, v_codebook=sel)
    st = oracle.State(n, 4, bits_v, block)
    for t in range(1, 4):
        _, gb, _ = rand_inputs(n, 40 + t)
        prev = oracle.dequant(st, 1).astype(np.float64) if t > 1 else np.zeros(n)
        _, vh, _ = oracle.step(p, gb, st, h, t, want_hat=True)
        g = synth.bits_to_bf16(gb).float().numpy().astype(np.float64)
        b2 = float(np.float32(0.999))
        assert np.allclose(vh, b2 * prev + (1 - b2) * g * g, rtol=1e-5, atol=1e-20)   # Eq. 3 on Eq. 2
        dv = oracle.dequant(st, 1)
        for j in range(st.nblk):
            sl = slice(j * block, min(n, (j + 1) * block))
            assert st.scale_v[j] == vh[sl].max() and st.alpha[j] == 0.5
            r = vh[sl].astype(np.float64) / float(st.scale_v[j])
            dist = np.abs(r[:, None] - y[None, :])
            q_ref = dist.argmin(1)
            q = np.array([oracle.get_code(st.codes_v[j * (block * bits_v // 8):], e, bits_v)
                          for e in range(sl.stop - sl.start)])
            srt = np.sort(dist, axis=1)
            tie = (srt[:, 1] - srt[:, 0]) < 1e-6
            assert np.all((q == q_ref) | tie)
            assert np.array_equal(dv[sl], (y[q].astype(np.float32) * st.scale_v[j]).astype(np.float32))


def test_swamping_through_the_full_step():
    """Sec. 3.2 (Corollary 3.2) on the whole step: one large element pins the block scale; with
    the 4-bit linear codebook (beta2 = 0.999 >= 0.967) the small entries stay at level 0 under
    a constant signal whose per-step increment is below half a gap, although the exact EMA
    climbs to most of the scale; SOLO's logarithmic quantizer follows the exact EMA."""
    n, b2 = 128, float(np.float32(0.999))
    gvals = np.full(n, 1e-3, np.float32)
    gvals[0] = 1.0
    g_big = synth.bf16_bits(torch.from_numpy(gvals).to(torch.bfloat16))
    gvals[1:] = 0.2
    gvals[0] = 0.0                                              # the scale only decays from here
    g_sig_t = torch.from_numpy(gvals).to(torch.bfloat16)
    g_sig = synth.bf16_bits(g_sig_t)
    gs = float(g_sig_t[1]) ** 2
    exact, track = 0.0, {}
    for t in range(1, 4):
        exact = b2 * exact + (1 - b2) * 1e-6
    for t in range(4, 64):
        exact = b2 * exact + (1 - b2) * gs
    for sel in (2, 0):
        h = oracle.hyper(beta1=0.8, beta2=0.999, bias_correction=0, v_codebook=sel, seed=1, lr=0.0)
        st = oracle.State(n, 4, 4, 128)
        p = np.zeros(n, np.float32)
        for t in range(1, 4):
            oracle.step(p, g_big, st, h, t)
        for t in range(4, 64):
            oracle.step(p, g_sig, st, h, t)
            # per-step increment relative to the scale: below half a gap of the linear codebook
            assert (1 - b2) * gs / float(st.scale_v[0]) < 0.5 / 15
        track[sel] = oracle.dequant(st, 1)[1:].astype(np.float64)
        assert exact / float(st.scale_v[0]) > 0.5                  # the exact EMA is far from 0
    assert np.all(track[2] == 0.0)                                  # swamped
    assert abs(track[0].mean() / exact - 1) < 0.1                   # SOLO tracks
