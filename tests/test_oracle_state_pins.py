"""Pins for the two places where the oracle's full step reads or writes the PACKED state.

1. Eq. 2 (Sec. 3.1): the moments that enter the EMA are decoded from the codes and scales the
   step before left behind.  The decode is redone here in binary64 numpy straight from the
   packed bytes: the signed dynamic-exponent levels are typed out from the rule of Appendix A,
   the logarithmic levels are alpha^q (Sec. 3.2.2), both times the block scale; then Eq. 3.
   The run starts from a random packed state, so every code value and every level is hit.
2. Eq. 5 inside the step (stochastic rounding of the signed state, which Thm 3.6 assumes):
   every stored code is the bracket index plus one exactly when the element's own draw
   (Philox purpose 1, the element's global index) falls below the fractional position.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_00347_b200 import synth


def de_signed_levels(bits: int) -> np.ndarray:
    """Appendix A, signed dynamic exponent, typed out: one sign bit; the other bits-1 bits are E
    leading zeros, an indicator bit and F = bits-2-E fraction bits; the magnitude is the midpoint
    of cell j of the 2^F equal cells of [0.1, 1], divided by 10^E.  Zero and +1 complete the set;
    codes count the levels in ascending order."""
    mags = []
    for E in range(bits - 1):
        F = bits - 2 - E
        width = 0.9 / 2 ** F
        mags += [(0.1 + (j + 0.5) * width) / 10 ** E for j in range(2 ** F)]
    lv = sorted([-a for a in mags] + [0.0] + mags + [1.0])
    assert len(lv) == 2 ** bits
    return np.array(lv, np.float64)


# the small codebooks as plain numbers, so that the generator above is itself checked
PRINTED = {
    2: [-0.55, 0, 0.55, 1],
    3: [-0.775, -0.325, -0.055, 0, 0.055, 0.325, 0.775, 1],
    4: [-0.8875, -0.6625, -0.4375, -0.2125, -0.0775, -0.0325, -0.0055, 0,
        0.0055, 0.0325, 0.0775, 0.2125, 0.4375, 0.6625, 0.8875, 1],
}


def unpack(packed: np.ndarray, bits: int, block: int) -> np.ndarray:
    """Bytes -> [n_blocks, block] codes; element e sits at bits [e*b, e*b+b) of its block's
    little-endian bit string (numpy only, no oracle call)."""
    nb = packed.size // (block * bits // 8)
    b = np.unpackbits(packed.reshape(nb, -1), axis=1, bitorder="little").reshape(nb, block, bits)
    return (b.astype(np.int64) << np.arange(bits)).sum(axis=2)


def rand_grad(n, seed, scale):
    rng = np.random.default_rng(seed)
    g = torch.from_numpy(rng.normal(0, scale, n).astype(np.float32)).to(torch.bfloat16)
    return synth.bf16_bits(g), g.float().numpy().astype(np.float64)


def test_typed_out_levels_match_the_small_codebooks():
    for b, want in PRINTED.items():
        assert np.allclose(de_signed_levels(b), want, rtol=0, atol=1e-15)


@pytest.mark.parametrize("bits_m,bits_v,block", [(2, 3, 128), (3, 2, 64), (4, 4, 128), (8, 8, 256),
                                                 (4, 2, 2048), (2, 8, 128)])
def test_moments_are_decoded_from_the_previous_packed_state(bits_m, bits_v, block):
    n = block * 5 + block // 3 + 1                               # a short last block
    rng = np.random.default_rng(17 * bits_m + bits_v)
    p = rng.normal(0, 0.02, n).astype(np.float32)
    sd = synth.make_state((n,), bits_m, bits_v, block, seed=500 + bits_m * 10 + bits_v)
    st = oracle.State(n, bits_m, bits_v, block)
    for k in ("codes_m", "codes_v", "scale_m", "scale_v", "alpha"):
        getattr(st, k)[:] = sd[k].numpy()
    h = oracle.hyper(beta1=0.7, beta2=0.99, seed=41)
    b1, b2 = float(np.float32(0.7)), float(np.float32(0.99))
    y = de_signed_levels(bits_m)
    seen_m, seen_v = set(), set()
    for t in range(1, 5):
        qm = unpack(st.codes_m, bits_m, block).reshape(-1)[:n]
        qv = unpack(st.codes_v, bits_v, block).reshape(-1)[:n]
        seen_m |= set(qm.tolist())
        seen_v |= set(qv.tolist())
        dm = np.repeat(st.scale_m.astype(np.float64), block)[:n]
        dv = np.repeat(st.scale_v.astype(np.float64), block)[:n]
        al = np.repeat(st.alpha.astype(np.float64), block)[:n]
        m_tilde = y[qm] * dm                                     # Eq. 2, signed state
        v_tilde = al ** qv * dv                                  # Eq. 2, levels alpha^q
        gb, g = rand_grad(n, 900 + t, 1e-3 * t)
        mh, vh, _ = oracle.step(p, gb, st, h, t, tensor=3, want_hat=True)
        m_ref = b1 * m_tilde + (1 - b1) * g                      # Eq. 3
        v_ref = b2 * v_tilde + (1 - b2) * g * g
        # binary32 roundings of the decode, the two products and the sum; the signed sum can cancel,
        # so the bound is relative to the size of its terms
        m_tol = 1e-6 * (np.abs(b1 * m_tilde) + np.abs((1 - b1) * g)) + 1e-40
        assert np.all(np.abs(mh - m_ref) <= m_tol), t
        # alpha^q by repeated squaring in binary32 carries a relative error of about q * 2^-24
        bad = np.abs(vh - v_ref) > (4e-6 + 1.2e-7 * qv) * v_ref + 1e-38
        assert not bad.any(), (t, np.nonzero(bad)[0][:4], vh[bad][:4], v_ref[bad][:4], qv[bad][:4], al[bad][:4])
    # the random start makes the run visit (nearly) every code of the small codebooks
    if bits_m <= 4:
        assert seen_m == set(range(1 << bits_m))
    if bits_v <= 4:
        assert seen_v == set(range(1 << bits_v))


@pytest.mark.parametrize("bits_m", [2, 3, 4, 8])
def test_stochastic_first_moment_codes_use_the_elements_own_draw(bits_m):
    block, tensor, off, seed = 128, 6, 128 * 11, 0x1234567
    n = block * 3 + 37
    rng = np.random.default_rng(bits_m)
    p = rng.normal(0, 0.02, n).astype(np.float32)
    st = oracle.State(n, bits_m, 3, block)
    h = oracle.hyper(beta1=0.6, round_m=1, seed=seed)
    y = oracle.codebook(oracle.DE_SIGNED, bits_m)
    y64 = y.astype(np.float64)
    assert np.allclose(y64, de_signed_levels(bits_m), rtol=1e-7, atol=0)
    differs_from_v_stream = 0
    for t in (1, 2, 3):
        gb, _ = rand_grad(n, 70 + t, 1e-3)
        mh, _, _ = oracle.step(p, gb, st, h, t, tensor=tensor, elem_offset=off, want_hat=True)
        q = unpack(st.codes_m, bits_m, block).reshape(-1)[:n]
        for j in range(st.nblk):
            lo, hi = j * block, min(n, (j + 1) * block)
            delta = np.float32(np.abs(mh[lo:hi]).max())
            assert st.scale_m[j] == delta
            inv = np.float32(1.0) / delta
            for i in range(lo, hi):
                r = np.float32(mh[i]) * inv                       # binary32, as the step computes it
                k = int(np.clip(np.searchsorted(y, r, side="right") - 1, 0, len(y) - 2))
                frac = (float(r) - y64[k]) / (y64[k + 1] - y64[k])
                d = oracle.philox_draw16(seed, t, tensor, off + i, 1)
                u = d / 65536.0
                if abs(u - frac) > 1e-6:                          # binary32 vs binary64 fraction
                    assert q[i] == k + (1 if u < frac else 0), (t, i, r, k, frac, u, q[i])
                dv = oracle.philox_draw16(seed, t, tensor, off + i, 0)
                differs_from_v_stream += int((dv / 65536.0 < frac) != (u < frac))
    # the check above can tell the first-moment stream from the second-moment one
    assert differs_from_v_stream > n // 20
