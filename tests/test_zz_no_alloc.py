"""The allocation-free entry point solo_multi_step_static against solo_multi_step.

Callers that run under a memory pool which owns all of the GPU's memory, or that must not
trigger the device-wide synchronisation of cudaMalloc / cudaFree in the middle of a training
step, bring their own state buffers; the library keeps the few tables it needs besides them in a
fixed array of its own.  Both entry points launch the same kernels, so on equal inputs the packed
state and the parameters must come out identical; this is checked on two consecutive calls (the
fixed array is rewritten by every call, the second one with a different tensor list).

Collected last on purpose: a failure here leaves every other test already run.
"""
import numpy as np
import pytest
import torch

from paper_2505_00347_b200 import synth

pytestmark = pytest.mark.gpu


def pad4(n: int) -> int:
    return (n + 3) // 4 * 4


def _fresh_buffers(sizes, bits_m, bits_v, block, state0=None):
    nb = sum(-(-int(n) // block) for n in sizes)
    if state0 is not None:
        out = {}
        for k, v in state0.items():
            if v.dtype == torch.float32:                        # per-block arrays: padded allocation
                buf = torch.zeros(pad4(v.numel()), dtype=torch.float32, device="cuda")
                buf[: v.numel()] = v.cuda()
                out[k] = buf[: v.numel()]
            else:                                                # codes: 16 readable bytes follow
                buf = torch.zeros(v.numel() + 16, dtype=torch.uint8, device="cuda")
                buf[: v.numel()] = v.cuda()
                out[k] = buf[: v.numel()]
        return out
    return {
        # 16 readable bytes follow the codes
        "codes_m": torch.zeros(nb * block * bits_m // 8 + 16, dtype=torch.uint8, device="cuda")[:nb * block * bits_m // 8],
        "codes_v": torch.zeros(nb * block * bits_v // 8 + 16, dtype=torch.uint8, device="cuda")[:nb * block * bits_v // 8],
        # the three per-block arrays are allocated in multiples of 16 bytes
        "scale_m": torch.zeros(pad4(nb), dtype=torch.float32, device="cuda")[:nb],
        "scale_v": torch.zeros(pad4(nb), dtype=torch.float32, device="cuda")[:nb],
        "alpha": torch.full((pad4(nb),), 0.5, dtype=torch.float32, device="cuda")[:nb],
    }


def _run_pair(B, sizes, bits_m, bits_v, block, steps, seed, state0=None, **hyper_kw):
    w = synth.workload(2, sizes=tuple(sizes))
    h = B.hyper(lr=1e-3, beta1=0.6, beta2=0.999, weight_decay=0.01, seed=seed, **hyper_kw)
    params = [synth.make_param(w, i) for i in range(len(sizes))]
    p_lib = [p.clone().cuda() for p in params]
    p_sta = [p.clone().cuda() for p in params]
    lib_state = B.State(list(sizes), bits_m, bits_v, block)
    bufs = _fresh_buffers(sizes, bits_m, bits_v, block, state0)
    if state0 is not None:
        for k, v in state0.items():
            lib_state.raw_set(k, v)
    for t in range(1, steps + 1):
        grads = [synth.make_grad(w, i, t).cuda() for i in range(len(sizes))]
        B.solo_multi_step(B.TensorSet(p_lib, grads, lib_state), h, t)
        # the pointer arrays are made with torch before the measurement: what is measured is the library call
        pp = torch.tensor([p.data_ptr() for p in p_sta], dtype=torch.int64, device="cuda")
        gp = torch.tensor([g.data_ptr() for g in grads], dtype=torch.int64, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.solo_multi_step_static(p_sta, grads, list(sizes), bufs, bits_m, bits_v, block, h, t,
                                 param_ptrs=pp, grad_ptrs=gp)
        assert B.static_status() == 0                     # waits for the stream; no mismatch, no copy given up on
        if t > 1:     # (the very first call on a device may load the library's kernels and looks the fixed array up)
            assert torch.cuda.mem_get_info()[0] == free_before   # free device memory did not move: nothing was allocated
        for key in ("codes_m", "codes_v", "scale_m", "scale_v", "alpha"):
            got = bufs[key].cpu().numpy().view(np.uint8)
            want = lib_state.raw_get(key).numpy().view(np.uint8)
            assert np.array_equal(got, want), (key, t)
        for a, b in zip(p_sta, p_lib):
            assert torch.equal(a, b), t          # same kernel, same inputs: bit-identical parameters
    lib_state.destroy()


def test_static_entry_point_matches_library_state_twice():
    from paper_2505_00347_b200 import binding as B
    # first call sequence: streamlined kernel (2/3 bit, block 128), ragged multi-tensor list
    _run_pair(B, (2048 * 3 + 77, 1, 128, 5000), 2, 3, 128, steps=2, seed=7)
    # second, with another list and widths (8-bit first moment, block 2048), from a random state
    sizes = (2048 * 2 + 5, 300, 4097)
    st0 = synth.make_state(sizes, 8, 4, 2048, seed=99)
    _run_pair(B, sizes, 8, 4, 2048, steps=2, seed=8, state0=st0)
    # and through the general kernel (stochastic rounding of the first moment)
    _run_pair(B, sizes, 8, 4, 2048, steps=2, seed=8, state0=st0, round_m=1)
    # third: a baseline codebook for the second moment (its table also lives in the fixed array)
    _run_pair(B, (2048 + 9, 640), 4, 4, 128, steps=2, seed=9, v_codebook=3)


def test_static_entry_point_refuses_a_capturing_stream():
    """The call copies its tables from its own stack frame; recorded into a graph those copies would
    read a dead frame at replay, so a capturing stream is refused before anything is queued."""
    from paper_2505_00347_b200 import binding as B
    sizes = [2048 + 5]
    ps = [torch.zeros(sizes[0], device="cuda")]
    gs = [torch.zeros(sizes[0], device="cuda", dtype=torch.bfloat16)]
    bufs = _fresh_buffers(sizes, 2, 3, 128)
    pp = torch.tensor([ps[0].data_ptr()], dtype=torch.int64, device="cuda")
    gp = torch.tensor([gs[0].data_ptr()], dtype=torch.int64, device="cuda")
    B.solo_multi_step_static(ps, gs, sizes, bufs, 2, 3, 128, B.hyper(), 1, param_ptrs=pp, grad_ptrs=gp)   # looks the array up
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        try:
            with pytest.raises(B.SoloError) as e:
                B.solo_multi_step_static(ps, gs, sizes, bufs, 2, 3, 128, B.hyper(), 2, param_ptrs=pp, grad_ptrs=gp)
            assert e.value.status == B.SOLO_EINVAL
        finally:
            graph.capture_end()
    torch.cuda.synchronize()
    B.solo_multi_step_static(ps, gs, sizes, bufs, 2, 3, 128, B.hyper(), 2, param_ptrs=pp, grad_ptrs=gp)   # still usable
    assert B.static_status() == 0


def test_static_entry_point_rejects_what_it_cannot_hold():
    from paper_2505_00347_b200 import binding as B
    n = B.STATIC_MAX_TENSORS + 1
    sizes = [8] * n
    ps = [torch.zeros(8, device="cuda") for _ in range(2)]
    gs = [torch.zeros(8, device="cuda", dtype=torch.bfloat16) for _ in range(2)]
    bufs = _fresh_buffers(sizes, 4, 4, 128)
    ptrs = torch.zeros(n, dtype=torch.int64, device="cuda")
    with pytest.raises(B.SoloError) as e:
        B.solo_multi_step_static(ps, gs, sizes, bufs, 4, 4, 128, B.hyper(), 1, param_ptrs=ptrs, grad_ptrs=ptrs)
    assert e.value.status == B.SOLO_ELIMIT and "SOLO_STATIC_MAX_TENSORS" in str(e.value)
    with pytest.raises(B.SoloError):
        B.solo_multi_step_static(ps, gs, [8, 0], bufs, 4, 4, 128, B.hyper(), 1)
