"""Sharded stepping on one GPU: a tensor list cut into block-aligned pieces (as a ZeRO / FSDP style
partition of the flattened optimizer state would), every piece stepped with a state of its own whose
origin names the piece's tensor and first element.  Blocks are independent and the rounding noise
is addressed by (tensor, element index), so the pieces' codes, scales and parameters, put back
together, must be bit-identical to stepping the whole list at once -- for the logarithmic
quantizer's xi, for stochastic rounding of the first moment and for stochastically rounded bf16
parameters, in every kernel.  One piece is also checked directly against the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_00347_b200 import shard, synth
import parity

pytestmark = pytest.mark.gpu


def _step_whole(B, sizes, params, grads_fn, bm, bv, block, h, steps, st0):
    st = B.State(list(sizes), bm, bv, block)
    for k, v in st0.items():
        st.raw_set(k, v)
    ps = [p.clone().cuda() for p in params]
    for t in range(1, steps + 1):
        B.solo_multi_step(B.TensorSet(ps, [g.cuda() for g in grads_fn(t)], st), h, t)
    torch.cuda.synchronize()
    assert st.status() == 0
    out = parity.download_state(st), [p.cpu() for p in ps]
    st.destroy()
    return out


def _step_sharded(B, sizes, params, grads_fn, bm, bv, block, h, steps, st0, world):
    parts = shard.partition(sizes, block, world)
    nblk = [-(-n // block) for n in sizes]
    bstart = np.concatenate([[0], np.cumsum(nblk)])
    sm, sv = block * bm // 8, block * bv // 8
    ps = [p.clone().cuda() for p in params]
    states = []
    for pieces in parts:
        if not pieces:
            states.append(None)
            continue
        st = B.State([p.numel for p in pieces], bm, bv, block)
        st.set_origin([p.tensor for p in pieces], [p.elem_offset for p in pieces])
        # this rank's slice of the initial state: its blocks are contiguous in the global block order
        b0 = int(bstart[pieces[0].tensor]) + pieces[0].elem_offset // block
        nb = sum(-(-p.numel // block) for p in pieces)
        st.raw_set("codes_m", st0["codes_m"][b0 * sm:(b0 + nb) * sm])
        st.raw_set("codes_v", st0["codes_v"][b0 * sv:(b0 + nb) * sv])
        for k in ("scale_m", "scale_v", "alpha"):
            st.raw_set(k, st0[k][b0:b0 + nb])
        states.append(st)
    for t in range(1, steps + 1):
        gs = [g.cuda() for g in grads_fn(t)]
        for pieces, st in zip(parts, states):
            if st is None:
                continue
            pv = [ps[p.tensor][p.elem_offset:p.elem_offset + p.numel] for p in pieces]
            gv = [gs[p.tensor][p.elem_offset:p.elem_offset + p.numel] for p in pieces]
            B.solo_multi_step(B.TensorSet(pv, gv, st), h, t)
    torch.cuda.synchronize()
    got = {k: [] for k in parity.KEYS}
    for st in states:
        if st is None:
            continue
        assert st.status() == 0
        d = parity.download_state(st)
        for k in parity.KEYS:
            got[k].append(d[k])
        st.destroy()
    return {k: np.concatenate(v) for k, v in got.items()}, [p.cpu() for p in ps], parts


@pytest.mark.parametrize("bm,bv,block,extra,policies", [
    (2, 3, 128, dict(), (3, 2, 1)),
    (4, 4, 128, dict(round_m=1), (0,)),
    (2, 3, 128, dict(param_dtype=1, param_round=1), (3, 2, 1)),
    (3, 2, 64, dict(), (3, 0, 1)),
    (2, 3, 256, dict(), (3, 0, 1)),
    (4, 2, 2048, dict(param_dtype=1, param_round=1), (0, 1)),
])
def test_pieces_reproduce_the_whole(bm, bv, block, extra, policies):
    from paper_2505_00347_b200 import binding as B
    sizes = (2048 * 9 + 700, block * 5 + 3, 2048 * 4, 77, 2048 * 6 + block)
    w = synth.workload(2, sizes=sizes)
    dtype = torch.bfloat16 if extra.get("param_dtype") == 1 else torch.float32
    params = [synth.make_param(w, i, dtype=dtype) for i in range(len(sizes))]
    gf = lambda t: [synth.make_grad(w, i, t) for i in range(len(sizes))]
    st0 = synth.make_state(sizes, bm, bv, block, seed=71)
    h = B.hyper(lr=1e-3, beta1=0.6, weight_decay=0.01, seed=0xC0FFEE, **extra)
    for policy in policies:
        B.set_kernel_policy(policy)
        try:
            want_state, want_params = _step_whole(B, sizes, params, gf, bm, bv, block, h, 2, st0)
            for world in (2, 3, 7):
                got_state, got_params, parts = _step_sharded(B, sizes, params, gf, bm, bv, block, h, 2, st0, world)
                assert any(p.elem_offset > 0 for r in parts for p in r)        # some tensor really is cut
                for k in parity.KEYS:
                    assert np.array_equal(got_state[k].view(np.uint8), want_state[k].view(np.uint8)), (policy, world, k)
                for a, b in zip(got_params, want_params):
                    assert torch.equal(a.view(torch.int16 if dtype == torch.bfloat16 else torch.int32),
                                       b.view(torch.int16 if dtype == torch.bfloat16 else torch.int32)), (policy, world)
        finally:
            B.set_kernel_policy(0)


def test_a_piece_against_the_oracle_and_argument_checks():
    from paper_2505_00347_b200 import binding as B
    block, n_total, lo = 128, 128 * 40 + 9, 128 * 17
    w = synth.workload(1, sizes=(n_total,))
    p = synth.make_param(w, 0)
    g = synth.make_grad(w, 0, 1)
    n = n_total - lo
    kw = dict(lr=1e-3, beta1=0.8, seed=99, round_m=1)
    ho, hg = parity.hyper_pair(**kw)
    st = B.State(n, 4, 3, block)
    st.set_origin([6], [lo])
    pg = p[lo:].clone().cuda()
    B.solo_step(pg, g[lo:].clone().cuda(), st, hg, 1)
    torch.cuda.synchronize()
    ost = oracle.State(n, 4, 3, block)
    po = p[lo:].numpy().copy()
    oracle.step(po, synth.bf16_bits(g[lo:]), ost, ho, 1, tensor=6, elem_offset=lo)
    got = parity.download_state(st)
    for k in parity.KEYS:
        assert np.array_equal(got[k].view(np.uint8), getattr(ost, k).view(np.uint8)), k
    assert parity.close(pg.cpu().numpy(), po).all()
    # without the origin the noise differs
    st2 = B.State(n, 4, 3, block)
    B.solo_step(p[lo:].clone().cuda(), g[lo:].clone().cuda(), st2, hg, 1)
    torch.cuda.synchronize()
    assert not np.array_equal(parity.download_state(st2)["codes_v"], got["codes_v"])
    # offsets must sit on block boundaries; the defaults come back with no arguments
    with pytest.raises(B.SoloError):
        st2.set_origin([0], [block // 2])
    with pytest.raises(B.SoloError):
        st2.set_origin([-1], [0])
    st2.set_origin([6], [lo])
    st2.set_origin(None, None)
    st.destroy()
    st2.destroy()
