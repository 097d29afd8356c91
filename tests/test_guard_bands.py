"""Guard bands around every device buffer the step touches (the memory checker of the CUDA toolkit
is not available where these tests run).

Through the entry point that takes caller-owned state buffers, parameters, gradients and the five
state arrays are each placed between two 256-byte bands of a known pattern.  The kernels may READ up
to 16 bytes past the codes and the per-block arrays rounded up to 16 bytes (documented in the header);
they must never WRITE outside the arrays proper.  Ragged sizes (1, 2, 63 ... 129, 2047, 2049, whole
tiles plus a tail) through every kernel policy and several widths and block sizes; afterwards every
band, and the documented slack between array and band, still holds the pattern.
"""
import numpy as np
import pytest
import torch

from paper_2505_00347_b200 import synth

pytestmark = pytest.mark.gpu

BAND = 256
PATTERN = 0xA5


class Guarded:
    """`nbytes` usable bytes, 256-byte aligned, followed by `slack` bytes that may be read, between two bands."""

    def __init__(self, nbytes: int, slack: int = 0, fill: int = 0):
        self.nbytes, self.slack = nbytes, slack
        self.raw = torch.full((BAND + nbytes + slack + BAND + 256,), PATTERN, dtype=torch.uint8, device="cuda")
        off = (-self.raw.data_ptr()) % 256
        self.lo = off
        self.body = self.raw[off + BAND: off + BAND + nbytes]
        self.body.fill_(fill)
        assert self.body.data_ptr() % 256 == 0

    def view(self, dtype):
        return self.body.view(dtype)

    def intact(self) -> bool:
        r = self.raw.cpu().numpy()
        a = self.lo + BAND
        return bool((r[:a] == PATTERN).all() and (r[a + self.nbytes:] == PATTERN).all())


def pad4(n):
    return (n + 3) // 4 * 4


@pytest.mark.parametrize("bits_m,bits_v,block,policies", [
    (2, 3, 128, (3, 2, 1)), (4, 4, 128, (3, 2, 1)), (3, 3, 64, (3, 0, 1)), (4, 2, 256, (3, 0, 1)),
    (2, 2, 2048, (0, 1)), (8, 8, 128, (0, 1)), (3, 8, 64, (0, 1)),
])
def test_nothing_is_written_outside_the_arrays(bits_m, bits_v, block, policies):
    from paper_2505_00347_b200 import binding as B
    sizes = list(synth.RAGGED_FORCED) + [2048 * 3, 2048 * 2 + 77, 2048 + 2047, 5 * block + 1]
    w = synth.workload(4, sizes=tuple(sizes))
    nb = sum(-(-n // block) for n in sizes)
    h = B.hyper(lr=1e-3, beta1=0.6, weight_decay=0.01, seed=12)
    for policy in policies:
        B.set_kernel_policy(policy)
        try:
            gp = [Guarded(4 * n) for n in sizes]
            gg = [Guarded(2 * n) for n in sizes]
            params = [x.view(torch.float32) for x in gp]
            for p_, i in zip(params, range(len(sizes))):
                p_.copy_(synth.make_param(w, i))
            # state arrays: the documented readable slack (16 bytes after the codes; the per-block arrays
            # allocated in multiples of 16 bytes) lies inside the guarded region and must stay untouched too
            gs = {
                "codes_m": Guarded(nb * block * bits_m // 8, slack=16),
                "codes_v": Guarded(nb * block * bits_v // 8, slack=16),
                "scale_m": Guarded(4 * nb, slack=4 * (pad4(nb) - nb)),
                "scale_v": Guarded(4 * nb, slack=4 * (pad4(nb) - nb)),
                "alpha": Guarded(4 * nb, slack=4 * (pad4(nb) - nb)),
            }
            bufs = {k: (v.view(torch.float32) if k in ("scale_m", "scale_v", "alpha") else v.body) for k, v in gs.items()}
            bufs["alpha"].fill_(0.5)
            pp = torch.tensor([p_.data_ptr() for p_ in params], dtype=torch.int64, device="cuda")
            for t in (1, 2, 3):
                grads = [x.view(torch.bfloat16) for x in gg]
                for g_, i in zip(grads, range(len(sizes))):
                    g_.copy_(synth.make_grad(w, i, t))
                gptr = torch.tensor([g_.data_ptr() for g_ in grads], dtype=torch.int64, device="cuda")
                B.solo_multi_step_static(params, grads, sizes, bufs, bits_m, bits_v, block, h, t,
                                         param_ptrs=pp, grad_ptrs=gptr)
                assert B.static_status() == 0
            torch.cuda.synchronize()
            for name, arr in [("param", x) for x in gp] + [("grad", x) for x in gg] + list(gs.items()):
                assert arr.intact(), (policy, name)
            assert all(torch.isfinite(p_).all() for p_ in params)
            assert float(bufs["scale_v"].max()) > 0                      # the steps did run
        finally:
            B.set_kernel_policy(0)
