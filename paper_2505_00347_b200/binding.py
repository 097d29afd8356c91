"""ctypes binding of the C ABI in include/solo.h (argument marshalling only).

Every step of the optimizer runs in the CUDA library; this module passes raw device
pointers of torch tensors and the current CUDA stream.  If the shared library is not
there, loading raises: there is no other implementation to fall back to.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libsolo_b200.so"

SOLO_OK, SOLO_EINVAL, SOLO_EALIGN, SOLO_ENOMEM, SOLO_ECUDA, SOLO_ESTATE = 0, -1, -2, -3, -4, -5
SOLO_ELIMIT = -6
STATIC_MAX_TENSORS = 1024


class SoloError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {strerror(status)} ({status})")


class Hyper(C.Structure):
    """solo_hyper_t"""

    _fields_ = [
        ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
        ("weight_decay", C.c_float), ("p_quantile", C.c_float), ("fixed_alpha", C.c_float),
        ("adamw", C.c_int32), ("bias_correction", C.c_int32), ("round_m", C.c_int32),
        ("round_v", C.c_int32), ("param_dtype", C.c_int32), ("belief", C.c_int32),
        ("param_round", C.c_int32), ("v_codebook", C.c_int32),
        ("seed", C.c_uint64),
    ]


class TensorList(C.Structure):
    """solo_tensor_list_t"""

    _fields_ = [
        ("num_tensors", C.c_int32), ("param", C.c_void_p), ("grad", C.c_void_p),
        ("numel", C.c_void_p), ("state", C.c_void_p),
    ]


class HostList(C.Structure):
    """solo_host_list_t: every pointer is a host array"""

    _fields_ = [
        ("num_tensors", C.c_int32), ("param_dev", C.c_void_p), ("grad_host", C.c_void_p),
        ("param_out_host", C.c_void_p), ("numel", C.c_void_p), ("chunk_elems", C.c_int64),
        ("state", C.c_void_p),
    ]


class RawState(C.Structure):
    """solo_raw_state_t: caller-owned state buffers for solo_multi_step_static"""

    _fields_ = [
        ("codes_m", C.c_void_p), ("codes_v", C.c_void_p), ("scale_m", C.c_void_p),
        ("scale_v", C.c_void_p), ("alpha", C.c_void_p),
        ("bits_m", C.c_int32), ("bits_v", C.c_int32), ("block", C.c_int32),
    ]


def hyper(lr=1e-3, beta1=0.8, beta2=0.999, eps=1e-8, weight_decay=0.01, p_quantile=0.1,
          adamw=1, bias_correction=1, round_m=0, round_v=1, param_dtype=0, seed=0, belief=0, fixed_alpha=0.0,
          param_round=0, v_codebook=0) -> Hyper:
    return Hyper(lr, beta1, beta2, eps, weight_decay, p_quantile, fixed_alpha, adamw, bias_correction,
                 round_m, round_v, param_dtype, belief, param_round, v_codebook, seed)


_lib = None


def lib() -> C.CDLL:
    """Loads libsolo_b200.so from the package directory; raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2505_00347_b200._build` "
            "(nvcc, sm_100a).  There is no CPU or PyTorch fallback.")
    L = C.CDLL(str(LIB_PATH))
    vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int
    L.solo_state_create.argtypes = [i64, i32, i32, i32, C.POINTER(vp)]
    L.solo_state_create_multi.argtypes = [C.POINTER(C.c_int64), i32, i32, i32, i32, C.POINTER(vp)]
    L.solo_state_destroy.argtypes = [vp]
    L.solo_state_bytes.argtypes = [i64, i32, i32, i32, C.POINTER(C.c_size_t)]
    L.solo_step.argtypes = [vp, vp, vp, C.POINTER(Hyper), i64, vp]
    L.solo_multi_step.argtypes = [C.POINTER(TensorList), C.POINTER(Hyper), i64, vp]
    L.solo_dequant.argtypes = [vp, i32, vp, vp]
    L.solo_state_raw.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(C.c_size_t)]
    L.solo_state_info.argtypes = [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                                  C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                  C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    L.solo_state_status.argtypes = [vp, C.POINTER(C.c_int)]
    L.solo_codebook_m.argtypes = [i32, C.POINTER(C.c_float)]
    L.solo_codebook_v.argtypes = [i32, i32, C.POINTER(C.c_float)]
    L.solo_codebook_v.restype = C.c_int
    L.solo_default_beta1.argtypes = [i32, i32]
    L.solo_default_beta1.restype = C.c_float
    L.solo_set_kernel_policy.argtypes = [i32]
    L.solo_debug_check_fast_log.argtypes = [C.c_uint32, C.c_uint32, C.POINTER(C.c_float),
                                            C.POINTER(C.c_float)]
    L.solo_multi_step_static.argtypes = [C.c_int32, vp, vp, C.POINTER(C.c_int64), C.POINTER(RawState),
                                         C.POINTER(Hyper), i64, vp]
    L.solo_multi_step_static.restype = C.c_int
    L.solo_multi_step_host.argtypes = [C.POINTER(HostList), C.POINTER(Hyper), i64, vp]
    L.solo_multi_step_host.restype = C.c_int
    L.solo_state_export_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
    L.solo_state_export.argtypes = [vp, vp, C.c_size_t, vp]
    L.solo_state_import.argtypes = [vp, vp, C.c_size_t, vp]
    L.solo_state_set_origin.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
    L.solo_state_set_origin.restype = C.c_int
    L.solo_static_status.argtypes = [C.POINTER(C.c_int), vp]
    L.solo_static_status.restype = C.c_int
    L.solo_debug_stall_copy.argtypes = [i64]
    L.solo_debug_stall_copy.restype = C.c_int
    L.solo_launch_count.argtypes = []
    L.solo_launch_count.restype = C.c_int64
    L.solo_strerror.argtypes = [i32]
    L.solo_strerror.restype = C.c_char_p
    for name in ("solo_state_create", "solo_state_create_multi", "solo_state_destroy",
                 "solo_state_bytes", "solo_step", "solo_multi_step", "solo_dequant",
                 "solo_state_raw", "solo_state_info", "solo_state_status", "solo_codebook_m",
                 "solo_set_kernel_policy", "solo_debug_check_fast_log", "solo_state_export_bytes",
                 "solo_state_export", "solo_state_import"):
        getattr(L, name).restype = C.c_int
    _lib = L
    return L


def strerror(status: int) -> str:
    return lib().solo_strerror(status).decode()


def _check(rc: int, what: str) -> None:
    if rc != SOLO_OK:
        raise SoloError(rc, what)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


RAW = {"codes_m": 0, "codes_v": 1, "scale_m": 2, "scale_v": 3, "alpha": 4}
_RAW_DTYPE = {0: torch.uint8, 1: torch.uint8, 2: torch.float32, 3: torch.float32, 4: torch.float32}


class State:
    """Owner of a solo_state_t handle (single tensor or tensor list)."""

    def __init__(self, numel, bits_m: int, bits_v: int, block: int = 128):
        self.handle = C.c_void_p()
        self.sizes = [int(numel)] if isinstance(numel, int) else [int(n) for n in numel]
        if isinstance(numel, int):
            rc = lib().solo_state_create(numel, bits_m, bits_v, block, C.byref(self.handle))
        else:
            arr = (C.c_int64 * len(self.sizes))(*self.sizes)
            rc = lib().solo_state_create_multi(arr, len(self.sizes), bits_m, bits_v, block,
                                               C.byref(self.handle))
        _check(rc, "solo_state_create")
        self.bits_m, self.bits_v, self.block = bits_m, bits_v, block
        self.device = torch.device("cuda", torch.cuda.current_device())

    def destroy(self) -> None:
        if getattr(self, "handle", None) is not None and self.handle:
            lib().solo_state_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def set_origin(self, stream_ids=None, elem_offsets=None) -> None:
        """solo_state_set_origin: where each tensor of this state sits in the random stream (the
        tensor's stream number and the index of its first element within the whole tensor)."""
        T = len(self.sizes)
        ids = (C.c_int32 * T)(*[int(x) for x in stream_ids]) if stream_ids is not None else None
        offs = (C.c_int64 * T)(*[int(x) for x in elem_offsets]) if elem_offsets is not None else None
        _check(lib().solo_state_set_origin(self.handle, ids, offs), "solo_state_set_origin")

    def info(self) -> dict:
        n, nb = C.c_int64(), C.c_int64()
        t, bm, bv, blk = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
        _check(lib().solo_state_info(self.handle, C.byref(n), C.byref(nb), C.byref(t), C.byref(bm),
                                     C.byref(bv), C.byref(blk)), "solo_state_info")
        return dict(numel=n.value, num_blocks=nb.value, num_tensors=t.value, bits_m=bm.value,
                    bits_v=bv.value, block=blk.value)

    def raw_ptr(self, which) -> tuple[int, int]:
        w = RAW[which] if isinstance(which, str) else which
        p, b = C.c_void_p(), C.c_size_t()
        _check(lib().solo_state_raw(self.handle, w, C.byref(p), C.byref(b)), "solo_state_raw")
        return p.value or 0, b.value

    def raw_get(self, which) -> torch.Tensor:
        """Copy of one state buffer as a CPU tensor (uint8 codes / float32 scales)."""
        w = RAW[which] if isinstance(which, str) else which
        ptr, nbytes = self.raw_ptr(w)
        out = torch.empty(nbytes, dtype=torch.uint8)
        torch.cuda.synchronize()
        _cuda_memcpy(out.data_ptr(), ptr, nbytes, 2)
        return out if _RAW_DTYPE[w] == torch.uint8 else out.view(torch.float32)

    def raw_set(self, which, value: torch.Tensor) -> None:
        """Overwrite one state buffer from a CPU tensor of the same byte size."""
        w = RAW[which] if isinstance(which, str) else which
        ptr, nbytes = self.raw_ptr(w)
        v = value.contiguous().view(torch.uint8).cpu()
        if v.numel() != nbytes:
            raise ValueError(f"expected {nbytes} bytes, got {v.numel()}")
        torch.cuda.synchronize()
        _cuda_memcpy(ptr, v.data_ptr(), nbytes, 1)

    def export(self) -> torch.Tensor:
        """The whole state as one CPU uint8 tensor (solo_state_export)."""
        n = C.c_size_t()
        _check(lib().solo_state_export_bytes(self.handle, C.byref(n)), "solo_state_export_bytes")
        out = torch.empty(n.value, dtype=torch.uint8)
        _check(lib().solo_state_export(self.handle, out.data_ptr(), n.value,
                                       torch.cuda.current_stream().cuda_stream), "solo_state_export")
        return out

    def load(self, blob: torch.Tensor) -> None:
        """Restores a state written by export() into this one (solo_state_import)."""
        b = blob.contiguous().view(torch.uint8).cpu()
        _check(lib().solo_state_import(self.handle, b.data_ptr(), b.numel(),
                                       torch.cuda.current_stream().cuda_stream), "solo_state_import")

    def status(self) -> int:
        s = C.c_int()
        _check(lib().solo_state_status(self.handle, C.byref(s)), "solo_state_status")
        return s.value


_cudart = None


def _cuda_memcpy(dst: int, src: int, nbytes: int, kind: int) -> None:
    """cudaMemcpy through the runtime that torch already loaded (kind 1 = H2D, 2 = D2H)."""
    global _cudart
    if nbytes == 0:
        return
    if _cudart is None:
        _cudart = C.CDLL(_find_cudart())
        _cudart.cudaMemcpy.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_int]
        _cudart.cudaMemcpy.restype = C.c_int
    rc = _cudart.cudaMemcpy(dst, src, nbytes, kind)
    if rc:
        raise RuntimeError(f"cudaMemcpy failed with {rc}")


def _find_cudart() -> str:
    import glob
    import os
    cands = []
    for root in (os.path.join(os.path.dirname(torch.__file__), "lib"),
                 os.path.join(os.path.dirname(os.path.dirname(torch.__file__)), "nvidia",
                              "cuda_runtime", "lib"),
                 "/usr/local/cuda/lib64"):
        cands += sorted(glob.glob(os.path.join(root, "libcudart.so*")))
    if not cands:
        raise ImportError("libcudart.so not found")
    return cands[0]


def state_bytes(numel: int, bits_m: int, bits_v: int, block: int = 128) -> int:
    out = C.c_size_t()
    _check(lib().solo_state_bytes(numel, bits_m, bits_v, block, C.byref(out)), "solo_state_bytes")
    return out.value


def solo_step(param: torch.Tensor, grad: torch.Tensor, state: State, h: Hyper, step: int) -> None:
    """One fused step on a single tensor, on the current stream."""
    _check_tensor(param, grad, h)
    _check(lib().solo_step(param.data_ptr(), grad.data_ptr(), state.handle, C.byref(h), step,
                           _stream()), "solo_step")


def _check_tensor(param: torch.Tensor, grad: torch.Tensor, h: Hyper) -> None:
    want = torch.bfloat16 if h.param_dtype == 1 else torch.float32
    if not (param.is_cuda and grad.is_cuda and param.is_contiguous() and grad.is_contiguous()):
        raise ValueError("param and grad must be contiguous CUDA tensors")
    if param.dtype != want or grad.dtype != torch.bfloat16 or param.numel() != grad.numel():
        raise ValueError("param must be fp32/bf16 per hyper.param_dtype, grad bf16, same numel")


class TensorSet:
    """Device-side descriptor arrays of a tensor list (built once, reused every step)."""

    def __init__(self, params: list[torch.Tensor], grads: list[torch.Tensor], state: State):
        if len(params) != len(grads) or len(params) != len(state.sizes):
            raise ValueError("params, grads and state must have the same number of tensors")
        for p, g, n in zip(params, grads, state.sizes):
            if p.numel() != n or g.numel() != n or g.dtype != torch.bfloat16:
                raise ValueError("tensor sizes / dtypes do not match the state")
            if not (p.is_cuda and g.is_cuda and p.is_contiguous() and g.is_contiguous()):
                raise ValueError("tensors must be contiguous CUDA tensors")
        dev = params[0].device
        self.params, self.grads, self.state = params, grads, state
        self.param_ptrs = torch.tensor([p.data_ptr() for p in params], dtype=torch.int64, device=dev)
        self.grad_ptrs = torch.tensor([g.data_ptr() for g in grads], dtype=torch.int64, device=dev)
        self.numel = torch.tensor(state.sizes, dtype=torch.int64, device=dev)
        self.desc = TensorList(len(params), self.param_ptrs.data_ptr(), self.grad_ptrs.data_ptr(),
                               self.numel.data_ptr(), state.handle)


def solo_multi_step(ts: TensorSet, h: Hyper, step: int) -> None:
    """One fused step over the whole tensor list in one launch, on the current stream."""
    _check(lib().solo_multi_step(C.byref(ts.desc), C.byref(h), step, _stream()), "solo_multi_step")


def solo_dequant(state: State, which: int) -> torch.Tensor:
    """Dequantized first (0) or second (1) moment of every element, as a float32 CUDA tensor."""
    out = torch.empty(sum(state.sizes), dtype=torch.float32, device=state.device)
    _check(lib().solo_dequant(state.handle, which, out.data_ptr(), _stream()), "solo_dequant")
    return out


def solo_multi_step_static(params: list[torch.Tensor], grads: list[torch.Tensor], sizes: list[int],
                           buffers: dict, bits_m: int, bits_v: int, block: int, h: Hyper, step: int,
                           param_ptrs: torch.Tensor = None, grad_ptrs: torch.Tensor = None) -> None:
    """The allocation-free step: `buffers` maps codes_m / codes_v (uint8) and scale_m / scale_v /
    alpha (float32) to CUDA tensors that the caller allocated in the library's state layout.
    `param_ptrs` / `grad_ptrs` are int64 CUDA tensors of the tensors' data pointers (built here,
    with torch, when not given; the library call itself allocates nothing)."""
    if param_ptrs is None:
        param_ptrs = torch.tensor([p.data_ptr() for p in params], dtype=torch.int64, device=params[0].device)
    if grad_ptrs is None:
        grad_ptrs = torch.tensor([g.data_ptr() for g in grads], dtype=torch.int64, device=params[0].device)
    raw = RawState(buffers["codes_m"].data_ptr(), buffers["codes_v"].data_ptr(),
                   buffers["scale_m"].data_ptr(), buffers["scale_v"].data_ptr(),
                   buffers["alpha"].data_ptr(), bits_m, bits_v, block)
    numel = (C.c_int64 * len(sizes))(*[int(n) for n in sizes])
    _check(lib().solo_multi_step_static(len(sizes), param_ptrs.data_ptr(), grad_ptrs.data_ptr(), numel,
                                        C.byref(raw), C.byref(h), step, _stream()),
           "solo_multi_step_static")


def solo_multi_step_host(params: list[torch.Tensor], grads_host: list[torch.Tensor],
                         params_out_host, state: State, h: Hyper, step: int, chunk_elems: int = 0) -> None:
    """The step with gradients in host memory (CPU bf16 tensors, pinned for overlap) and, when
    `params_out_host` is a list of CPU tensors of the parameters' type, a host copy of the updated
    parameters.  `params` are the resident CUDA tensors."""
    T = len(params)
    want = torch.bfloat16 if h.param_dtype == 1 else torch.float32
    for i in range(T):
        if not (params[i].is_cuda and params[i].is_contiguous() and params[i].dtype == want):
            raise ValueError("params must be contiguous CUDA tensors of the type hyper.param_dtype names")
        if grads_host[i].is_cuda or grads_host[i].dtype != torch.bfloat16 or not grads_host[i].is_contiguous() \
                or grads_host[i].numel() != params[i].numel():
            raise ValueError("grads_host must be contiguous CPU bf16 tensors of the parameters' sizes")
        if params_out_host is not None:
            o = params_out_host[i]
            if o.is_cuda or o.dtype != want or not o.is_contiguous() or o.numel() != params[i].numel():
                raise ValueError("params_out_host must be contiguous CPU tensors like the parameters")
    vp = C.c_void_p * T
    pd = vp(*[p.data_ptr() for p in params])
    gh = vp(*[g.data_ptr() for g in grads_host])
    po = vp(*[o.data_ptr() for o in params_out_host]) if params_out_host is not None else None
    numel = (C.c_int64 * T)(*[int(p.numel()) for p in params])
    lst = HostList(T, C.cast(pd, C.c_void_p), C.cast(gh, C.c_void_p),
                   C.cast(po, C.c_void_p) if po is not None else None, C.cast(numel, C.c_void_p),
                   int(chunk_elems), state.handle)
    _check(lib().solo_multi_step_host(C.byref(lst), C.byref(h), step, _stream()), "solo_multi_step_host")


def codebook_m(bits: int) -> torch.Tensor:
    buf = (C.c_float * (1 << bits))()
    _check(lib().solo_codebook_m(bits, buf), "solo_codebook_m")
    return torch.tensor(list(buf), dtype=torch.float32)


def codebook_v(v_codebook: int, bits: int) -> torch.Tensor:
    buf = (C.c_float * (1 << bits))()
    _check(lib().solo_codebook_v(v_codebook, bits, buf), "solo_codebook_v")
    return torch.tensor(list(buf), dtype=torch.float32)


def default_beta1(bits_m: int, from_scratch: bool = False) -> float:
    return float(lib().solo_default_beta1(bits_m, 1 if from_scratch else 0))


def set_kernel_policy(policy: int) -> None:
    """0: fastest kernel that applies (default); 1: always the general kernel; 2: like 0 without the
    sixteen-elements-per-thread kernel; 3: that kernel wherever it exists, whatever the tensor sizes."""
    _check(lib().solo_set_kernel_policy(policy), "solo_set_kernel_policy")


def debug_check_fast_log(lo_bits: int, hi_bits: int) -> tuple[float, float]:
    """(largest excess of the lg2 approximation over the relative bound, assumed absolute bound)."""
    ex, ab = C.c_float(), C.c_float()
    _check(lib().solo_debug_check_fast_log(lo_bits, hi_bits, C.byref(ex), C.byref(ab)),
           "solo_debug_check_fast_log")
    return ex.value, ab.value


def static_status() -> int:
    """Status word of the last solo_multi_step_static call on the current device (waits for the
    current stream)."""
    out = C.c_int(-1)
    _check(lib().solo_static_status(C.byref(out), _stream()), "solo_static_status")
    return out.value


def debug_stall_copy(tile: int) -> None:
    """Test hook: the next step over-announces the input copy of tile `tile`, so the bounded wait
    for it runs out."""
    _check(lib().solo_debug_stall_copy(int(tile)), "solo_debug_stall_copy")


def launch_count() -> int:
    return int(lib().solo_launch_count())
