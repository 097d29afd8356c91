"""GPU parity: the CUDA library against the CPU oracle on the same seeded inputs,
through the C ABI (ctypes binding).  Run with -m gpu on a B200."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_00347_b200 import synth
import parity
from parity import run_lockstep

pytestmark = pytest.mark.gpu

# Extra parameter tolerance, as a fraction of the update |p_new - p_old|, for runs that start from a
# random packed state or use a learning rate of 0.1 (see parity.run_lockstep); everything else is held
# to the plain 1e-6 relative / 1e-9 absolute bar.
RANDOM_STATE_TOL = 3e-7


def _inputs(w, device="cpu"):
    params = [synth.make_param(w, i) for i in range(len(w.sizes))]
    return params, lambda t: [synth.make_grad(w, i, t) for i in range(len(w.sizes))]


def test_config1_lockstep_and_free_run():
    """1 Mi elements, 4/4 bit, block 128, AdamW lr 1e-3 wd 0.01, 10 steps."""
    w = synth.workload(1)
    hk = dict(lr=w.lr, beta1=w.beta1, beta2=w.beta2, weight_decay=w.weight_decay, seed=11)
    params, gf = _inputs(w)
    rep = run_lockstep(w.sizes, 4, 4, 128, hk, 10, gf, params, update_tol=0.0)
    print("lock-step", rep)
    assert rep.exempt_m + rep.exempt_v <= 1e-5 * rep.elements + 2
    rep = run_lockstep(w.sizes, 4, 4, 128, hk, 10, gf, params, free_run=True, update_tol=0.0)
    print("free run", rep)


def test_gpt125m_set_free_run_100_steps():
    """GPT-style 125M set (148 tensors, 124,439,808 parameters, 3-bit / 3-bit, block 128): the
    library runs 100 steps on its own state, the oracle likewise; the packed state is compared bit
    for bit at steps 10, 50 and 100 (any difference would compound, so equality at 100 covers every
    step), the parameters within the plain per-step tolerance accumulated over the steps."""
    from paper_2505_00347_b200 import binding as B
    w = synth.workload(2)
    T = len(w.sizes)
    dev = torch.device("cuda")
    gparams = [synth.make_param(w, i, device=dev) for i in range(T)]
    oparams = [p.cpu().numpy().copy() for p in gparams]
    gstate = B.State(list(w.sizes), 3, 3, 128)
    ostates = [oracle.State(n, 3, 3, 128) for n in w.sizes]
    kw = dict(lr=w.lr, beta1=w.beta1, beta2=w.beta2, weight_decay=w.weight_decay, seed=2024)
    ho, hg = parity.hyper_pair(**kw)
    threads = oracle.hardware_threads()
    for t in range(1, 101):
        grads = [synth.make_grad(w, i, t, device=dev) for i in range(T)]
        B.solo_multi_step(B.TensorSet(gparams, grads, gstate), hg, t)
        for i in range(T):
            oracle.step(oparams[i], synth.bf16_bits(grads[i]), ostates[i], ho, t, tensor=i, nthreads=threads)
        if t in (10, 50, 100):
            torch.cuda.synchronize()
            assert gstate.status() == 0
            got = parity.download_state(gstate)
            want = parity.join_state(ostates)
            for k in parity.KEYS:
                assert np.array_equal(got[k].view(np.uint8), want[k].view(np.uint8)), (t, k)
            for i in range(T):
                gp = gparams[i].cpu().numpy().astype(np.float64)
                wp = oparams[i].astype(np.float64)
                # the plain bar, 1e-6 relative / 1e-9 absolute per step, accumulated over the steps
                tol = parity.RTOL * np.abs(wp) + parity.ATOL * t
                assert np.all(np.abs(gp - wp) <= tol), (t, i, float(np.max(np.abs(gp - wp) - tol)))
    gstate.destroy()


@pytest.mark.parametrize("block", [64, 128, 256, 2048])
@pytest.mark.parametrize("bits_m,bits_v", [(2, 2), (2, 3), (3, 3), (4, 2), (4, 4), (8, 8), (3, 8), (8, 2)])
def test_bits_and_blocks_random_state(bits_m, bits_v, block):
    """Every width / block size from a random packed state (all codes, scales and bases in
    use), ragged sizes, multi-tensor launch, two lock-step steps."""
    sizes = (block * 9 + 5, 1, block, block + 1, 7 * 2048 + 3, 2047, 2049, block - 1)
    w = synth.workload(2, sizes=sizes)
    params, gf = _inputs(w)
    st0 = synth.make_state(sizes, bits_m, bits_v, block, seed=bits_m * 100 + bits_v * 10 + block)
    hk = dict(lr=1e-3, beta1=0.8, beta2=0.999, weight_decay=0.01, seed=5)
    # block 128 with widths up to 4 bits: policy 3 is the sixteen-per-thread kernel plus the
    # streamlined kernel for the tails (policy 0 picks it for large sets only)
    policies = (0, 3, 1) if block in (64, 128, 256) and max(bits_m, bits_v) <= 4 else (0, 1)
    # a random packed state pairs huge first moments with tiny second moments: update terms far above
    # the parameters themselves, where the faster kernels' quotient (a few 1e-7 of the term) shows
    rep = run_lockstep(sizes, bits_m, bits_v, block, hk, 2, gf, params, state0=st0, policies=policies,
                       update_tol=RANDOM_STATE_TOL)
    print(rep)
    assert rep.exempt_m + rep.exempt_v <= 3 * len(policies)
    assert rep.allowance_elems <= 1e-3 * rep.elements


@pytest.mark.parametrize("bits_m,bits_v,block", [(2, 3, 128), (3, 2, 64), (4, 4, 256), (2, 2, 2048), (8, 4, 64),
                                                 (2, 8, 256)])
@pytest.mark.parametrize("hk", [dict(adamw=0, weight_decay=0.1), dict(round_v=0, belief=1),
                                dict(fixed_alpha=0.5, param_dtype=1), dict(round_m=1, seed=0xABCDEF012345),
                                dict(round_m=1, v_codebook=2, adamw=0)])
def test_mode_flags_at_other_widths(bits_m, bits_v, block, hk):
    """The streamlined kernel has one instantiation for the paper's plain step and one that reads
    the mode flags at run time; the latter at other widths and block sizes than the mode test."""
    sizes = (2048 * 3 + block + 7, 500)
    w = synth.workload(1, sizes=sizes)
    dtype = torch.bfloat16 if hk.get("param_dtype") == 1 else torch.float32
    params = [synth.make_param(w, i, dtype=dtype) for i in range(2)]
    gf = lambda t: [synth.make_grad(w, i, t) for i in range(2)]
    base = dict(lr=1e-3, beta1=0.6, beta2=0.999, weight_decay=0.01, seed=13)
    base.update(hk)
    st0 = synth.make_state(sizes, bits_m, bits_v, block, seed=19)
    # policy 3: the sixteen-per-thread kernel's instantiation that reads the modes (where it exists)
    print(run_lockstep(sizes, bits_m, bits_v, block, base, 2, gf, params, state0=st0, update_tol=RANDOM_STATE_TOL,
                       policies=(0, 3, 1)))


@pytest.mark.parametrize("bits_m,bits_v,block", [(2, 3, 128), (3, 3, 64), (4, 2, 256), (4, 4, 128), (8, 3, 128)])
@pytest.mark.parametrize("beta1", [0.5, 0.75])
def test_eq5_rounding_on_the_levels_themselves(bits_m, bits_v, block, beta1):
    """Eq. 5 where its bracket search is decided by equality: with zero gradients the first moment is
    beta1 times a level times the scale, so in every block that holds the level 1 the ratio
    m^ / Delta' lands on a level of the codebook or an ulp beside it (the fractional position is 0, an
    ulp, or an ulp short of 1), for every level of the random packed state; zero elements give r = +-0.  The
    sixteen-per-thread kernel counts the levels r reaches with saturated multiply-adds, the general
    kernel and the oracle compare; all three must agree on every code."""
    sizes = (2048 * 4 + 3 * block + 5, 2048 * 2)
    w = synth.workload(1, sizes=sizes)
    params = [synth.make_param(w, i) for i in range(2)]
    zero = lambda t: [torch.zeros(n, dtype=torch.bfloat16) for n in sizes]
    st0 = synth.make_state(sizes, bits_m, bits_v, block, seed=77 + bits_m)
    hk = dict(lr=1e-3, beta1=beta1, beta2=0.999, weight_decay=0.0, seed=31, round_m=1)
    run_lockstep(sizes, bits_m, bits_v, block, hk, 3, zero, params, state0=st0, policies=(0, 3, 1),
                 update_tol=RANDOM_STATE_TOL)


@pytest.mark.parametrize("hk", [
    dict(adamw=0, weight_decay=0.1),
    dict(bias_correction=0),
    dict(round_m=1, seed=99),
    dict(round_v=0),
    dict(p_quantile=0.0),
    dict(p_quantile=0.3, beta2=0.95),
    dict(param_dtype=1, lr=1e-2),
    dict(eps=1e-3, lr=0.1, weight_decay=0.0),
    dict(belief=1),
    dict(fixed_alpha=0.5),
    dict(fixed_alpha=0.9, round_v=0),
    dict(belief=1, eps=1e-12, beta2=0.99, adamw=0, weight_decay=0.05),
    dict(param_dtype=1, param_round=1, lr=1e-2, seed=77),
    dict(param_dtype=1, param_round=1, lr=3e-5, weight_decay=0.0, round_m=1),
    dict(v_codebook=1),
    dict(v_codebook=2, belief=1),
    dict(v_codebook=3),
    dict(v_codebook=3, param_dtype=1, param_round=1, adamw=0),
])
def test_hyper_parameter_modes(hk):
    sizes = (128 * 40 + 17, 300)
    w = synth.workload(1, sizes=sizes)
    dtype = torch.bfloat16 if hk.get("param_dtype") == 1 else torch.float32
    params = [synth.make_param(w, i, dtype=dtype) for i in range(2)]
    gf = lambda t: [synth.make_grad(w, i, t) for i in range(2)]
    base = dict(lr=1e-3, beta1=0.8, beta2=0.999, weight_decay=0.01, seed=3)
    base.update(hk)
    st0 = synth.make_state(sizes, 4, 3, 128, seed=17)
    print(run_lockstep(sizes, 4, 3, 128, base, 3, gf, params, state0=st0, update_tol=RANDOM_STATE_TOL,
                       policies=(0, 3, 1)))
    # from the zero state the plain bar holds, except at a learning rate of 0.1 (updates of the
    # parameters' own size)
    print(run_lockstep(sizes, 4, 3, 128, base, 3, gf, params, policies=(0, 3, 1),
                       update_tol=RANDOM_STATE_TOL if base["lr"] > 1e-2 else 0.0))


@pytest.mark.parametrize("sel", [1, 2, 3])
@pytest.mark.parametrize("bits_m,bits_v,block", [(4, 2, 64), (4, 3, 128), (4, 4, 2048), (4, 8, 256), (2, 4, 256),
                                                 (3, 4, 128), (2, 2, 128), (3, 3, 64)])
def test_baseline_second_moment_codebooks(sel, bits_m, bits_v, block):
    """Sec. 4 baselines for the unsigned state (unsigned DE, linear, linear without zero;
    Appendix A) at every width, from a random packed state and from zero, ragged sizes.
    Policy 3: full tiles in the sixteen-per-thread kernel (widths up to 4 bits, blocks up to 256),
    the rest in the general kernel; policy 1: the general kernel alone."""
    sizes = (block * 5 + 3, 1, 2048 * 2 + 9, block - 1, 2048 * 3)
    w = synth.workload(4, sizes=sizes)                            # zero blocks and zero elements
    params, gf = _inputs(w)
    hk = dict(lr=1e-3, beta1=0.8, beta2=0.999, weight_decay=0.01, seed=5, v_codebook=sel)
    st0 = synth.make_state(sizes, bits_m, bits_v, block, seed=sel * 1000 + bits_v * 10 + block)
    run_lockstep(sizes, bits_m, bits_v, block, hk, 2, gf, params, state0=st0, policies=(0, 3, 1),
                 update_tol=RANDOM_STATE_TOL)
    run_lockstep(sizes, bits_m, bits_v, block, hk, 3, gf, params, policies=(0, 3, 1))


@pytest.mark.parametrize("param_round", [0, 1])
@pytest.mark.parametrize("bits_m,bits_v,block", [(2, 3, 128), (4, 4, 64), (3, 2, 256), (4, 3, 2048), (8, 8, 128)])
def test_bf16_parameters_every_kernel(bits_m, bits_v, block, param_round):
    """bf16 parameters through the streamlined kernel (full tiles from the staged copies, ragged
    tails from direct loads) and the general one, nearest and stochastic rounding; run_lockstep
    compares the stored bf16 patterns bit for bit."""
    sizes = (2048 * 5 + block * 3 + 1, 77, 2048 * 2, 2048 + 8)
    w = synth.workload(2, sizes=sizes)
    params = [synth.make_param(w, i, dtype=torch.bfloat16) for i in range(len(sizes))]
    gf = lambda t: [synth.make_grad(w, i, t) for i in range(len(sizes))]
    hk = dict(lr=1e-2, beta1=0.6, beta2=0.999, weight_decay=0.01, seed=41, param_dtype=1,
              param_round=param_round)
    st0 = synth.make_state(sizes, bits_m, bits_v, block, seed=block + bits_m)
    # (2, 3, 128): policy 3 adds the sixteen-per-thread kernel (policy 0 uses it for large sets only)
    policies = (0, 3, 1) if block in (64, 128, 256) and max(bits_m, bits_v) <= 4 else (0, 1)
    run_lockstep(sizes, bits_m, bits_v, block, hk, 2, gf, params, state0=st0, policies=policies)
    run_lockstep(sizes, bits_m, bits_v, block, hk, 3, gf, params, policies=policies)


def test_stochastic_bf16_rounding_is_unbiased_on_the_device():
    """Updates of 1/64 ulp(bf16): nearest rounding leaves every parameter where it is, stochastic
    rounding moves the mean by the update (first Adam step from zero state: p += lr exactly)."""
    from paper_2505_00347_b200 import binding as B
    n, lr = 1 << 20, 2.0 ** -13
    g = torch.full((n,), -1.0, dtype=torch.bfloat16, device="cuda")
    for rnd in (0, 1):
        p = torch.ones(n, dtype=torch.bfloat16, device="cuda")
        st = B.State(n, 4, 4, 128)
        B.solo_step(p, g, st, B.hyper(param_dtype=1, param_round=rnd, lr=lr, weight_decay=0.0, seed=5, eps=0.0), 1)
        torch.cuda.synchronize()
        mean = float(p.double().mean())
        if rnd:
            assert abs(mean - (1.0 + lr)) < 5 * 2.0 ** -7 * (1 / 64 / n) ** 0.5
            assert set(p.unique().tolist()) == {1.0, 1.0 + 2.0 ** -7}
        else:
            assert mean == 1.0
        st.destroy()


@pytest.mark.parametrize("bits_m,bits_v", [(2, 3), (2, 2), (2, 4), (3, 3), (4, 2), (4, 4), (3, 4), (4, 3), (3, 2)])
def test_block_128_plain_step_all_three_kernels(bits_m, bits_v):
    """Block 128, plain step: the sixteen-per-thread kernel (policy 3: full tiles there, the rest in
    the streamlined kernel), the streamlined kernel alone (2) and the general kernel (1) against
    one oracle run; tensors with many full tiles, tails and tiny tensors, zero blocks, ties, from a
    random state and from zero."""
    sizes = (2048 * 9 + 700, 3, 2048 * 4, 2048 + 128, 127, 2048 * 2 + 1)
    w = synth.workload(4, sizes=sizes)
    params, gf = _inputs(w)
    hk = dict(lr=2e-5, beta1=0.5, beta2=0.999, weight_decay=0.0, seed=1234)
    st0 = synth.make_state(sizes, bits_m, bits_v, 128, seed=5)
    print(run_lockstep(sizes, bits_m, bits_v, 128, hk, 3, gf, params, state0=st0, policies=(3, 2, 1),
                       update_tol=RANDOM_STATE_TOL))
    run_lockstep(sizes, bits_m, bits_v, 128, hk, 4, gf, params, policies=(3, 2, 1))
    w1 = synth.workload(1, sizes=(2048 * 6,))
    p1, g1 = _inputs(w1)
    run_lockstep(w1.sizes, bits_m, bits_v, 128, hk, 3, g1, p1, policies=(3, 2), multi=False)   # one launch: all tiles full


@pytest.mark.parametrize("block", [64, 256])
@pytest.mark.parametrize("bits_m,bits_v", [(2, 3), (2, 2), (3, 3), (4, 2), (3, 4), (4, 3), (4, 4)])
def test_blocks_64_and_256_plain_step_all_three_kernels(bits_m, bits_v, block):
    """The sixteen-per-thread kernel at the other two block sizes it exists for (four and sixteen
    lanes per block: six and twenty-five selection rounds, 3-bit codes of 64-element blocks that start
    off a 16-byte boundary, threads that run out of keys) against the streamlined and the general
    kernel and one oracle run: many full tiles, tails, tiny tensors, ties and zero blocks."""
    sizes = (2048 * 9 + 700, 3, 2048 * 4, block * 3, 2048 + block, 127, 2048 * 2 + 1, block)
    w = synth.workload(4, sizes=sizes)
    params, gf = _inputs(w)
    hk = dict(lr=2e-5, beta1=0.5, beta2=0.999, weight_decay=0.0, seed=4321)
    st0 = synth.make_state(sizes, bits_m, bits_v, block, seed=6)
    print(run_lockstep(sizes, bits_m, bits_v, block, hk, 3, gf, params, state0=st0, policies=(3, 2, 1),
                       update_tol=RANDOM_STATE_TOL))
    run_lockstep(sizes, bits_m, bits_v, block, hk, 4, gf, params, policies=(3, 2, 1))

    def ties(t):                                # duplicated second moments: tied keys, one lane with most of the smallest
        gs = [synth.make_grad(w, i, t) for i in range(len(sizes))]
        m = gs[0][1::3].numel()
        gs[0][0:3 * m:3] = gs[0][1::3]
        gs[2][:16] = 0.0
        gs[2][2048:2048 + 16] = 1e-30
        return gs

    run_lockstep(sizes, bits_m, bits_v, block, dict(hk, weight_decay=0.01), 3, ties, params, policies=(3, 2, 1))


def test_streamlined_kernel_rounding_guard_is_sound():
    """The streamlined kernel trusts lg2.approx to within abs + rel |log2 x| of the exact
    operation sequence; checked here for EVERY binary32 in [2^-100, 2) with half the constants."""
    from paper_2505_00347_b200 import binding as B
    excess, abs_bound = B.debug_check_fast_log(0x0D800000, 0x3FFFFFFF)
    print("largest excess", excess, "assumed absolute bound", abs_bound)
    assert excess <= 0.5 * abs_bound


def test_quantile_ranks_and_ties_on_full_tiles():
    """Several quantile ranks on tensors that span whole 2048-element tiles, with duplicated
    second moments (tied keys) in many blocks."""
    sizes = (2048 * 3, 2048 * 2 + 100)
    w = synth.workload(1, sizes=sizes)
    params, _ = _inputs(w)

    def gf(t):
        gs = [synth.make_grad(w, i, t) for i in range(2)]
        gs[0][::3] = gs[0][1::3]            # duplicates inside blocks
        gs[1][: 2048] = 0.0                 # all-zero blocks in a full tile
        gs[1][2048:4096:2] = 0.0            # half zeros: the quantile sits on a tie
        return gs

    for p_q, block in ((0.1, 128), (0.0, 64), (0.3, 256), (0.05, 128), (0.9, 64), (0.1, 2048), (0.0, 2048),
                       (0.95, 2048)):
        hk = dict(seed=5, p_quantile=p_q, weight_decay=0.0)
        run_lockstep(sizes, 2, 3, block, hk, 3, gf, params)
        run_lockstep(sizes, 4, 2, block, hk, 2, gf, params)


def test_single_tensor_entry_point_matches_multi():
    sizes = (128 * 33 + 9,)
    w = synth.workload(1, sizes=sizes)
    params, gf = _inputs(w)
    hk = dict(seed=21)
    run_lockstep(sizes, 2, 3, 128, hk, 3, gf, params, multi=False)
    run_lockstep(sizes, 2, 3, 128, hk, 3, gf, params, multi=True)


def test_ragged_zero_blocks_and_zero_elements():
    """Exact-zero blocks, N(0,1e-6) and N(0,1) blocks, elementwise zeros, tiny tensors."""
    sizes = synth.RAGGED_FORCED + (128 * 50, 128 * 7 + 1, 5000)
    w = synth.workload(4, sizes=sizes)
    params = [synth.make_param(w, i) for i in range(len(sizes))]
    # tensor index 7 mod 20 gets elementwise zeros: place the 5000-element tensor there
    order = list(range(len(sizes)))
    gf = lambda t: [synth.make_grad(w, i, t) for i in order]
    for bm, bv in ((2, 2), (3, 3), (4, 4), (2, 3), (4, 2)):
        rep = run_lockstep(sizes, bm, bv, 128, dict(seed=8, weight_decay=0.0), 4, gf, params)
        assert rep.exempt_m + rep.exempt_v <= 3


@pytest.mark.parametrize("bits_m,bits_v,block", [(2, 3, 128), (4, 4, 128), (3, 2, 64), (2, 2, 2048), (8, 4, 256),
                                                 (4, 3, 256)])
def test_nan_and_inf_gradients_follow_one_rule(bits_m, bits_v, block):
    """The paper says nothing about non-finite gradients; the rule here is that they propagate: a
    NaN in a block makes that block's scale NaN and its codes 0, an infinity makes the scale
    infinite, the element's parameter becomes NaN, and nothing outside the block changes.  Every
    kernel (sixteen-per-thread where it exists, streamlined, general) must reproduce the oracle's
    state bit for bit (NaN equal to NaN) and leave the other blocks' parameters finite."""
    sizes = (2048 * 3 + 300, 700)
    w = synth.workload(1, sizes=sizes)
    params, _ = _inputs(w)

    def gf(t):
        gs = [synth.make_grad(w, i, t) for i in range(2)]
        gs[0][5] = float("nan")                 # full tile, first block
        gs[0][2048 + 200] = float("inf")        # full tile, another block
        gs[0][2048 + 700] = float("-inf")
        gs[0][2048 * 3 + 17] = float("nan")     # tail tile
        gs[1][650] = float("inf")
        if t == 2:
            gs[0][4096:4096 + 128] = float("nan")   # a whole block of NaN
        return gs

    policies = (3, 2, 1) if block in (64, 128, 256) and max(bits_m, bits_v) <= 4 else (0, 1)
    run_lockstep(sizes, bits_m, bits_v, block, dict(seed=9, weight_decay=0.0), 3, gf, params, policies=policies)
    # and on its own state for three steps: no hang, status clean, untouched blocks finite
    from paper_2505_00347_b200 import binding as B
    st = B.State(list(sizes), bits_m, bits_v, block)
    ps = [p.cuda() for p in params]
    for t in (1, 2, 3):
        B.solo_multi_step(B.TensorSet(ps, [g.cuda() for g in gf(t)], st), B.hyper(), t)
    torch.cuda.synchronize()
    assert st.status() == 0
    for i in range(2):                          # blocks that never saw a non-finite gradient stay finite
        bad = torch.zeros(sizes[i], dtype=torch.bool)
        for t in (1, 2, 3):
            bad |= ~torch.isfinite(gf(t)[i].float())
        nb = -(-sizes[i] // block)
        pad = torch.zeros(nb * block, dtype=torch.bool)
        pad[: sizes[i]] = bad
        clean = ~pad.view(nb, block).any(dim=1).repeat_interleave(block)[: sizes[i]]
        assert clean.any() or block == 2048
        assert torch.isfinite(ps[i].cpu()[clean]).all()
    st.destroy()


def test_bounded_wait_runs_out_and_nothing_is_stored():
    """A copy of a tile's inputs that announces more bytes than it brings never completes its
    barrier phase: the kernel's bounded wait gives up, status bit 1 is set, the warps concerned store
    nothing (that tile's parameters and state keep their old values), every other tile is stepped
    as usual and the kernel returns.  Both kernels that stage their inputs."""
    from paper_2505_00347_b200 import binding as B
    tiles = 24
    sizes = (2048 * tiles,)
    w = synth.workload(3, sizes=sizes)
    p0 = synth.make_param(w, 0)
    g = synth.make_grad(w, 0, 1).cuda()
    st0 = synth.make_state(sizes, 2, 3, 128, seed=31)
    h = B.hyper(lr=1e-3, beta1=0.5, weight_decay=0.0, seed=4)
    for policy, stalled in ((3, 7), (2, 11)):
        B.set_kernel_policy(policy)
        try:
            ref, hit = B.State(sizes[0], 2, 3, 128), B.State(sizes[0], 2, 3, 128)
            for s_ in (ref, hit):
                for k, v in st0.items():
                    s_.raw_set(k, v)
            p_ref, p_hit = p0.clone().cuda(), p0.clone().cuda()
            B.solo_step(p_ref, g, ref, h, 1)
            B.debug_stall_copy(stalled)
            B.solo_step(p_hit, g, hit, h, 1)
            torch.cuda.synchronize()
            assert ref.status() == 0 and hit.status() == 2
            lo, hi = stalled * 2048, (stalled + 1) * 2048
            same = torch.ones(sizes[0], dtype=torch.bool)
            same[lo:hi] = False
            assert torch.equal(p_hit.cpu()[same], p_ref.cpu()[same])
            assert torch.equal(p_hit.cpu()[lo:hi], p0[lo:hi])                  # untouched
            for key, per_tile in (("codes_m", 512), ("codes_v", 768), ("scale_m", 16), ("scale_v", 16), ("alpha", 16)):
                got, want, old = hit.raw_get(key), ref.raw_get(key), st0[key]
                a, b = stalled * per_tile, (stalled + 1) * per_tile
                assert torch.equal(got[:a], want[:a]) and torch.equal(got[b:], want[b:]), key
                assert torch.equal(got[a:b], old[a:b]), key
            # the hook is one-shot: the next step is an ordinary one (the status word is sticky)
            B.solo_step(p_hit, g, hit, h, 2)
            B.solo_step(p_ref, g, ref, h, 2)
            torch.cuda.synchronize()
            assert torch.equal(p_hit.cpu()[same], p_ref.cpu()[same])
            assert hit.status() == 2
            ref.destroy()
            hit.destroy()
        finally:
            B.set_kernel_policy(0)


@pytest.mark.parametrize("bits_m,bits_v,block,extra,chunk", [
    (2, 3, 128, dict(), 2048 * 3),
    (4, 4, 64, dict(param_dtype=1, param_round=1), 2048),
    (8, 3, 2048, dict(round_m=1), 2048 * 2),
    (3, 3, 256, dict(v_codebook=2), 2048 * 5),
    (2, 3, 128, dict(), 0),
    (2, 3, 128, dict(policy=3), 2048 * 3),
    (2, 4, 128, dict(policy=3, param_dtype=1, param_round=1), 2048 * 2),
    (4, 3, 128, dict(policy=3, round_m=1, v_codebook=3), 2048 * 3),    # the general kernel takes what is left of each chunk
    (3, 2, 256, dict(policy=3, v_codebook=1, adamw=0), 2048),
])
def test_host_buffer_entry_point(bits_m, bits_v, block, extra, chunk):
    """solo_multi_step_host (gradients from host memory, parameters copied back, chunked over three
    streams) against solo_multi_step on the same inputs: identical state and parameters, chunk
    boundaries inside tensors, more chunks than staging slots, tiny tensors, two steps."""
    from paper_2505_00347_b200 import binding as B
    extra = dict(extra)
    policy = extra.pop("policy", 0)            # 3: the sixteen-per-thread kernel on the chunks' tile ranges
    sizes = (2048 * 7 + 300, 5, 2048 * 2, 129, 2048 * 4 + 1, 2047)
    w = synth.workload(2, sizes=sizes)
    dtype = torch.bfloat16 if extra.get("param_dtype") == 1 else torch.float32
    params = [synth.make_param(w, i, dtype=dtype) for i in range(len(sizes))]
    p_dev = [p.clone().cuda() for p in params]
    p_hst = [p.clone().cuda() for p in params]
    out = [torch.zeros_like(p).pin_memory() for p in params]
    h = B.hyper(lr=1e-3, beta1=0.6, beta2=0.999, weight_decay=0.01, seed=77, **extra)
    st_dev = B.State(list(sizes), bits_m, bits_v, block)
    st_hst = B.State(list(sizes), bits_m, bits_v, block)
    for t in (1, 2):
        grads = [synth.make_grad(w, i, t) for i in range(len(sizes))]
        pinned = [g.pin_memory() for g in grads]
        # (the same kernels on both sides: the general kernel's IEEE division and the faster kernels'
        # refined reciprocal differ in the last bits of an fp32 parameter)
        B.set_kernel_policy(policy)
        try:
            B.solo_multi_step(B.TensorSet(p_dev, [g.cuda() for g in grads], st_dev), h, t)
            B.solo_multi_step_host(p_hst, pinned, out if t == 2 else None, st_hst, h, t, chunk_elems=chunk)
            torch.cuda.synchronize()
        finally:
            B.set_kernel_policy(0)
        assert st_hst.status() == 0
        assert torch.equal(st_dev.export(), st_hst.export()), t
        for a, b in zip(p_dev, p_hst):
            assert torch.equal(a, b), t
    for a, o in zip(p_dev, out):
        assert torch.equal(a.cpu(), o)
    with pytest.raises(B.SoloError):
        B.solo_multi_step_host(p_hst[:2], pinned[:2], None, st_hst, h, 3)       # other list than the state's
    st_dev.destroy()
    st_hst.destroy()


@pytest.mark.parametrize("v_codebook", [0, 3])
def test_checkpoint_export_import(v_codebook):
    """solo_state_export / solo_state_import: the byte string holds the header and the five
    arrays in the documented order, equal to the oracle's state after the same steps; a state
    restored from it continues bit-identically; a checkpoint of another geometry is refused."""
    import struct
    from paper_2505_00347_b200 import binding as B
    sizes, bits_m, bits_v, block = (128 * 9 + 5, 77, 4096), 2, 3, 128
    w = synth.workload(2, sizes=sizes)
    hk = dict(lr=1e-3, beta1=0.6, beta2=0.999, weight_decay=0.01, seed=21, v_codebook=v_codebook)
    ho, hg = parity.hyper_pair(**hk)
    params = [synth.make_param(w, i) for i in range(3)]
    gp = [p.clone().cuda() for p in params]
    op = [p.numpy().copy() for p in params]
    st = B.State(list(sizes), bits_m, bits_v, block)
    ost = [oracle.State(n, bits_m, bits_v, block) for n in sizes]
    for t in (1, 2):
        grads = [synth.make_grad(w, i, t) for i in range(3)]
        B.solo_multi_step(B.TensorSet(gp, [g.cuda() for g in grads], st), hg, t)
        for i in range(3):
            oracle.step(op[i], synth.bf16_bits(grads[i]), ost[i], ho, t, tensor=i)
    blob = st.export().numpy()
    nblk = sum(-(-n // block) for n in sizes)
    assert bytes(blob[:8]) == b"SOLOST1\0"
    assert struct.unpack("<6i", blob[8:32].tobytes()) == (bits_m, bits_v, block, 3, v_codebook, 0)
    assert struct.unpack("<q3q", blob[32:64].tobytes()) == (nblk, *sizes)
    off = 64
    pad = lambda n: (n + 15) // 16 * 16
    for key, per in (("codes_m", block * bits_m // 8), ("codes_v", block * bits_v // 8),
                     ("scale_m", 4), ("scale_v", 4), ("alpha", 4)):
        want = np.concatenate([getattr(o, key).view(np.uint8) for o in ost])
        assert want.size == nblk * per
        assert np.array_equal(blob[off:off + want.size], want), key
        off += pad(want.size)
    assert off == blob.size
    # restore into a fresh state and continue on both
    st2 = B.State(list(sizes), bits_m, bits_v, block)
    st2.load(torch.from_numpy(blob))
    gp2 = [p.clone() for p in gp]
    grads = [synth.make_grad(w, i, 3).cuda() for i in range(3)]
    B.solo_multi_step(B.TensorSet(gp, grads, st), hg, 3)
    B.solo_multi_step(B.TensorSet(gp2, grads, st2), hg, 3)
    torch.cuda.synchronize()
    assert torch.equal(st.export(), st2.export())
    assert all(torch.equal(a, b) for a, b in zip(gp, gp2))
    assert torch.equal(B.solo_dequant(st, 1), B.solo_dequant(st2, 1))
    # refused: other geometry, foreign bytes, short buffer
    other = B.State(list(sizes), bits_m, 4, block)
    with pytest.raises(B.SoloError) as e:
        other.load(torch.from_numpy(blob))
    assert e.value.status == B.SOLO_ESTATE
    with pytest.raises(B.SoloError):
        st2.load(torch.zeros(blob.size, dtype=torch.uint8))
    with pytest.raises(B.SoloError):
        st2.load(torch.from_numpy(blob[:100].copy()))
    for s_ in (st, st2, other):
        s_.destroy()


def test_argument_validation():
    from paper_2505_00347_b200 import binding as B
    with pytest.raises(B.SoloError):
        B.State(100, 5, 4, 128)
    with pytest.raises(B.SoloError):
        B.State(100, 4, 4, 100)
    with pytest.raises(B.SoloError):
        B.State(0, 4, 4, 128)
    st = B.State(1024, 4, 4, 128)
    p = torch.zeros(1032, device="cuda")
    g = torch.zeros(1032, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(B.SoloError) as e:
        B.solo_step(p[1:1025], g[:1024], st, B.hyper(), 1)       # misaligned parameter pointer
    assert e.value.status == B.SOLO_EALIGN
    with pytest.raises(B.SoloError):
        B.solo_step(p[:1024], g[:1024], st, B.hyper(beta1=1.0), 1)
    with pytest.raises(B.SoloError):
        B.solo_step(p[:1024], g[:1024], st, B.hyper(), 0)
    multi = B.State([10, 20], 4, 4, 128)
    with pytest.raises(B.SoloError) as e:
        B.solo_step(p[:1024], g[:1024], multi, B.hyper(), 1)     # wrong kind of state
    assert e.value.status == B.SOLO_ESTATE
    # a descriptor whose numel disagrees with the state is refused by the kernel, not executed
    ps = [torch.zeros(10, device="cuda"), torch.zeros(20, device="cuda")]
    gs = [torch.zeros(10, device="cuda", dtype=torch.bfloat16), torch.ones(20, device="cuda", dtype=torch.bfloat16)]
    ts = B.TensorSet(ps, gs, multi)
    ts.numel[1] = 19
    B.solo_multi_step(ts, B.hyper(), 1)
    assert multi.status() == 1 and float(ps[1].abs().sum()) == 0.0
    st.destroy()
    multi.destroy()


def _full_size_sampled(cfg: int, random_per_tensor: int, need_bytes: float, overrides=None, step: int = 3,
                       param_bf16: int = 0, hyper_kw=None):
    """A benchmark workload at its full size, one solo_multi_step launch in the configuration
    bench.py times, from a seeded random packed state.  Blocks are independent, so the oracle
    recomputes a sample of them one by one from copies of their inputs taken before the step:
    the first and the last block of every tensor plus `random_per_tensor` random ones.
    param_bf16: 0 fp32 parameters, 1 bf16 rounded to nearest, 2 bf16 rounded stochastically (the
    stored patterns are then compared bit for bit).  hyper_kw: other fields of the step's hyper-parameters."""
    from paper_2505_00347_b200 import binding as B
    free, _ = torch.cuda.mem_get_info()
    if free < need_bytes:
        pytest.skip(f"needs about {need_bytes / 1e9:.0f} GB of free device memory")
    w = synth.workload(cfg, **(overrides or {}))
    bm, bv, block = w.bits_m, w.bits_v, w.block
    dev = torch.device("cuda")
    pdtype = torch.bfloat16 if param_bf16 else torch.float32
    params = [synth.make_param(w, i, device=dev, dtype=pdtype) for i in range(len(w.sizes))]
    grads = [synth.make_grad(w, i, 1, device=dev) for i in range(len(w.sizes))]
    st0 = synth.make_state(w.sizes, bm, bv, block, seed=33 + cfg, device=dev)
    gstate = B.State(list(w.sizes), bm, bv, block)
    for key in parity.KEYS:
        ptr, nbytes = gstate.raw_ptr(key)
        src = st0[key].contiguous().view(torch.uint8)
        assert src.numel() == nbytes
        B._cuda_memcpy(ptr, src.data_ptr(), nbytes, 3)           # device to device
    rng = np.random.default_rng(5 + cfg)
    nblk = [-(-n // block) for n in w.sizes]
    bstart = np.concatenate([[0], np.cumsum(nblk)])
    sample = []
    for t, nb in enumerate(nblk):
        picks = {0, nb - 1} | set(int(x) for x in rng.integers(0, nb, size=random_per_tensor if nb > 2 else 0))
        sample += [(t, j) for j in sorted(picks)]
    sm, sv = block * bm // 8, block * bv // 8
    before = []
    for t, j in sample:
        lo, hi = j * block, min(w.sizes[t], (j + 1) * block)
        jb = int(bstart[t]) + j
        before.append(dict(
            p=(synth.bf16_bits(params[t][lo:hi]) if param_bf16 else params[t][lo:hi].cpu().numpy().copy()),
            g=synth.bf16_bits(grads[t][lo:hi]),
            codes_m=st0["codes_m"][jb * sm:(jb + 1) * sm].cpu().numpy().copy(),
            codes_v=st0["codes_v"][jb * sv:(jb + 1) * sv].cpu().numpy().copy(),
            scale_m=st0["scale_m"][jb:jb + 1].cpu().numpy().copy(),
            scale_v=st0["scale_v"][jb:jb + 1].cpu().numpy().copy(),
            alpha=st0["alpha"][jb:jb + 1].cpu().numpy().copy()))
    del st0
    kw = dict(lr=w.lr, beta1=w.beta1, beta2=w.beta2, weight_decay=w.weight_decay, seed=1234)
    if param_bf16:
        kw.update(param_dtype=1, param_round=1 if param_bf16 == 2 else 0)
    kw.update(hyper_kw or {})
    ho, hg = parity.hyper_pair(**kw)
    B.solo_multi_step(B.TensorSet(params, grads, gstate), hg, step)
    torch.cuda.synchronize()
    assert gstate.status() == 0
    ptrs = {k: gstate.raw_ptr(k)[0] for k in parity.KEYS}

    def fetch(key, off, nbytes, dtype):
        out = torch.empty(nbytes, dtype=torch.uint8)
        B._cuda_memcpy(out.data_ptr(), ptrs[key] + off, nbytes, 2)
        return out.numpy().view(dtype)

    worst, beyond, excess, checked = 0.0, 0, -1.0, 0
    for (t, j), b in zip(sample, before):
        n = b["p"].size
        ost = oracle.State(n, bm, bv, block)
        for k in parity.KEYS:
            getattr(ost, k)[:] = b[k]
        p = b["p"].copy()
        oracle.step(p, b["g"], ost, ho, step, tensor=t, elem_offset=j * block)
        jb = int(bstart[t]) + j
        assert np.array_equal(fetch("codes_m", jb * sm, sm, np.uint8), ost.codes_m), (t, j)
        assert np.array_equal(fetch("codes_v", jb * sv, sv, np.uint8), ost.codes_v), (t, j)
        for k in ("scale_m", "scale_v", "alpha"):
            assert np.array_equal(fetch(k, jb * 4, 4, np.uint32), getattr(ost, k).view(np.uint32)), (t, j, k)
        if param_bf16:
            assert np.array_equal(synth.bf16_bits(params[t][j * block: j * block + n]), p), (t, j)
            continue
        gp = params[t][j * block: j * block + n].cpu().numpy()
        err = np.abs(gp.astype(np.float64) - p)
        # random states pair huge first moments with tiny second moments: allow the streamlined
        # kernel's 3e-7 of the update term on top of the 1e-6 / 1e-9 bar, and count who needs it
        plain = parity.RTOL * np.abs(p) + parity.ATOL
        tol = plain + 3e-7 * np.abs(p - b["p"].astype(np.float64))
        assert np.all(err <= tol), (t, j, float(err.max()))
        beyond += int((err > plain).sum())
        excess = max(excess, float((err - plain).max()))
        checked += n
        worst = max(worst, float(err.max()))
    print(f"workload {cfg}: {len(sample)} blocks of {len(w.sizes)} tensors checked, "
          f"largest parameter difference {worst:.3g}; {beyond} of {checked} parameters beyond the plain "
          f"1e-6 / 1e-9 bar (largest excess {max(excess, 0.0):.3g}), all within 3e-7 of their update")
    gstate.destroy()


def test_full_size_7b_set_sampled_blocks():
    """LLaMA-7B-shaped set, 6.74 B parameters, 2-bit / 3-bit, block 128 (the headline workload)."""
    _full_size_sampled(3, 12, 60e9)


def test_full_size_7b_set_ten_steps_from_zero_plain_bar():
    """The headline workload on realistic values: from the zero state, ten steps with fresh gradients,
    the library running on its own state.  Sampled blocks (first, last and four random ones per tensor)
    are stepped by the oracle alongside; their packed state must be identical at steps 1, 5 and 10 and
    their parameters within the plain bar, 1e-6 relative / 1e-9 absolute per step, with no allowance
    for the approximate division."""
    from paper_2505_00347_b200 import binding as B
    free, _ = torch.cuda.mem_get_info()
    if free < 62e9:
        pytest.skip("needs about 62 GB of free device memory")
    w = synth.workload(3)
    bm, bv, block = w.bits_m, w.bits_v, w.block
    dev = torch.device("cuda")
    T = len(w.sizes)
    params = [synth.make_param(w, i, device=dev) for i in range(T)]
    gstate = B.State(list(w.sizes), bm, bv, block)
    rng = np.random.default_rng(77)
    nblk = [-(-n // block) for n in w.sizes]
    bstart = np.concatenate([[0], np.cumsum(nblk)])
    picks = [sorted({0, nb - 1} | set(int(x) for x in rng.integers(0, nb, size=4 if nb > 2 else 0))) for nb in nblk]
    idx = []                                                   # per tensor: element indices of its sampled blocks
    for t in range(T):
        e = np.concatenate([np.arange(j * block, min(w.sizes[t], (j + 1) * block)) for j in picks[t]])
        idx.append(torch.from_numpy(e).to(dev))
    osts, ops = [], []
    for t in range(T):
        for j in picks[t]:
            n = min(w.sizes[t], (j + 1) * block) - j * block
            osts.append(oracle.State(n, bm, bv, block))
            ops.append(params[t][j * block: j * block + n].cpu().numpy().copy())
    kw = dict(lr=w.lr, beta1=w.beta1, beta2=w.beta2, weight_decay=w.weight_decay, seed=1234)
    ho, hg = parity.hyper_pair(**kw)
    ptrs = {k: gstate.raw_ptr(k)[0] for k in parity.KEYS}
    sm, sv = block * bm // 8, block * bv // 8

    def fetch(key, off, nbytes, dtype):
        out = torch.empty(nbytes, dtype=torch.uint8)
        B._cuda_memcpy(out.data_ptr(), ptrs[key] + off, nbytes, 2)
        return out.numpy().view(dtype)

    worst = 0.0
    for step in range(1, 11):
        grads = [synth.make_grad(w, i, step, device=dev) for i in range(T)]
        gs = [synth.bf16_bits(grads[t][idx[t]]) for t in range(T)]
        B.solo_multi_step(B.TensorSet(params, grads, gstate), hg, step)
        torch.cuda.synchronize()
        del grads
        k = 0
        for t in range(T):
            pos = 0
            for j in picks[t]:
                n = osts[k].numel
                oracle.step(ops[k], gs[t][pos:pos + n], osts[k], ho, step, tensor=t, elem_offset=j * block)
                pos += n
                k += 1
        if step in (1, 5, 10):
            assert gstate.status() == 0
            k = 0
            for t in range(T):
                for j in picks[t]:
                    jb, ost = int(bstart[t]) + j, osts[k]
                    assert np.array_equal(fetch("codes_m", jb * sm, sm, np.uint8), ost.codes_m), (step, t, j)
                    assert np.array_equal(fetch("codes_v", jb * sv, sv, np.uint8), ost.codes_v), (step, t, j)
                    for key in ("scale_m", "scale_v", "alpha"):
                        assert np.array_equal(fetch(key, jb * 4, 4, np.uint32), getattr(ost, key).view(np.uint32)), (step, t, j, key)
                    gp = params[t][j * block: j * block + ost.numel].cpu().numpy().astype(np.float64)
                    err = np.abs(gp - ops[k])
                    assert np.all(err <= parity.RTOL * np.abs(ops[k]) + parity.ATOL * step), (step, t, j, float(err.max()))
                    worst = max(worst, float(err.max()))
                    k += 1
    print(f"7B set, 10 steps from zero: {len(osts)} blocks followed, largest parameter difference {worst:.3g}")
    gstate.destroy()


def test_full_size_7b_set_bf16_parameters_stochastic_rounding():
    """The same set with bf16 parameters rounded stochastically (streamlined kernel, IEEE update)."""
    _full_size_sampled(3, 6, 45e9, param_bf16=2)


def test_full_size_ragged_set_sampled_blocks():
    """4,096 ragged tensors, 1.12 B parameters: block tails, tiny tensors, all-zero gradient blocks."""
    _full_size_sampled(4, 2, 12e9)


def test_full_size_gpt125m_set_sampled_blocks():
    """GPT-style 125M set, 3-bit states."""
    _full_size_sampled(2, 12, 3e9)


@pytest.mark.parametrize("bits,block", [(4, 64), (2, 256), (3, 2048), (8, 128)])
def test_full_size_sweep_tensor_sampled_blocks(bits, block):
    """One 268,435,456-element tensor at other widths and block sizes."""
    _full_size_sampled(5, 400, 6e9, overrides=dict(bits_m=bits, bits_v=bits, block=block))


@pytest.mark.parametrize("bits,block,hk", [
    (3, 128, dict(v_codebook=3)),
    (4, 256, dict(round_m=1)),
    (2, 64, dict(fixed_alpha=0.5, belief=1)),
    (4, 128, dict(v_codebook=1, round_m=1, adamw=0, weight_decay=0.01)),
    (2, 256, dict(round_v=0, v_codebook=2)),
])
def test_full_size_sweep_tensor_other_modes(bits, block, hk):
    """The same tensor in the modes that the sixteen-per-thread kernel reads at run time (baseline
    second-moment codebooks, Eq. 5 rounding, fixed base, AdaBelief, L2 term), in the launch
    configuration the default policy picks for a set of this size."""
    _full_size_sampled(5, 400, 6e9, overrides=dict(bits_m=bits, bits_v=bits, block=block), hyper_kw=hk)
