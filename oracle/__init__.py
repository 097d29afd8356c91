"""Python loader for the CPU oracle (test infrastructure, not the product).

Builds ``solo_oracle.cpp`` into a shared object next to the source on first use
(or when the source changed) and exposes thin numpy wrappers around its C
functions.  Only tests, the smoke check and the benchmark's CPU-baseline leg
import this package; the CUDA library never does, and this package never
imports the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import hashlib
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "solo_oracle.cpp"
_LIB = _HERE / "libsolo_oracle.so"
_STAMP = _HERE / "libsolo_oracle.so.stamp"

# codebook kinds (Appendix A)
DE_SIGNED, DE_UNSIGNED, LINEAR_UNSIGNED, LINEAR_SIGNED, LINEAR_NOZERO = range(5)
# so_qema modes
NEAREST, STOCHASTIC, LOG = range(3)


def _flags() -> list[str]:
    flags = ["-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", "-pthread"]
    try:
        cpu = Path("/proc/cpuinfo").read_text()
        if " fma " in cpu or " fma\n" in cpu:
            flags.append("-mfma")  # lets std::fmaf inline; still one rounding per fma
    except OSError:
        pass
    return flags


def build(force: bool = False) -> Path:
    """Compile the oracle if the shared object is missing or stale."""
    flags = _flags()
    key = hashlib.sha256(_SRC.read_bytes() + " ".join(flags).encode()).hexdigest()
    if not force and _LIB.exists() and _STAMP.exists() and _STAMP.read_text() == key:
        return _LIB
    tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
    subprocess.run(["g++", *flags, "-o", str(tmp), str(_SRC)], check=True)
    os.replace(tmp, _LIB)
    _STAMP.write_text(key)
    return _LIB


class Hyper(C.Structure):
    """Field-for-field the hyper-parameter record of the oracle (``so_hyper``)."""

    _fields_ = [
        ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
        ("weight_decay", C.c_float), ("p_quantile", C.c_float), ("fixed_alpha", C.c_float),
        ("adamw", C.c_int32), ("bias_correction", C.c_int32), ("round_m", C.c_int32),
        ("round_v", C.c_int32), ("param_dtype", C.c_int32), ("belief", C.c_int32),
        ("param_round", C.c_int32), ("v_codebook", C.c_int32),
        ("seed", C.c_uint64),
    ]


def hyper(lr=1e-3, beta1=0.8, beta2=0.999, eps=1e-8, weight_decay=0.01, p_quantile=0.1,
          adamw=1, bias_correction=1, round_m=0, round_v=1, param_dtype=0, seed=0, belief=0, fixed_alpha=0.0,
          param_round=0, v_codebook=0) -> Hyper:
    return Hyper(lr, beta1, beta2, eps, weight_decay, p_quantile, fixed_alpha, adamw, bias_correction,
                 round_m, round_v, param_dtype, belief, param_round, v_codebook, seed)


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    L = C.CDLL(str(build()))
    f32p, u8p, u16p, u32p, i32p = (C.POINTER(t) for t in
                                   (C.c_float, C.c_uint8, C.c_uint16, C.c_uint32, C.c_int32))
    L.so_codebook.argtypes = [C.c_int, C.c_int, f32p]
    L.so_codebook.restype = C.c_int
    for name in ("so_log2_sp", "so_exp2_sp"):
        getattr(L, name).argtypes = [C.c_float]
        getattr(L, name).restype = C.c_float
    L.so_philox4x32_10.argtypes = [u32p, u32p, u32p]
    L.so_philox4x32_10.restype = None
    L.so_philox_draw16.argtypes = [C.c_uint64, C.c_int64, C.c_int32, C.c_int64, C.c_int]
    L.so_philox_draw16.restype = C.c_uint32
    for name in ("so_xi", "so_u"):
        getattr(L, name).argtypes = [C.c_uint32]
        getattr(L, name).restype = C.c_float
    L.so_quant_nearest.argtypes = [f32p, C.c_int, C.c_float]
    L.so_quant_nearest.restype = C.c_int
    L.so_quant_stochastic.argtypes = [f32p, C.c_int, C.c_float, C.c_float]
    L.so_quant_stochastic.restype = C.c_int
    L.so_quant_log.argtypes = [C.c_float, C.c_float, C.c_float, C.c_int]
    L.so_quant_log.restype = C.c_int
    L.so_pow_sm.argtypes = [C.c_float, C.c_int]
    L.so_pow_sm.restype = C.c_float
    L.so_log_base.argtypes = [C.c_float, C.c_float, C.c_int, f32p]
    L.so_log_base.restype = C.c_float
    L.so_get_code.argtypes = [u8p, C.c_int, C.c_int]
    L.so_get_code.restype = C.c_int
    L.so_set_code.argtypes = [u8p, C.c_int, C.c_int, C.c_int]
    L.so_set_code.restype = None
    L.so_state_bytes.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_uint64)]
    L.so_state_bytes.restype = C.c_int
    L.so_beta_prime.argtypes = [C.c_double] * 3
    L.so_beta_prime.restype = C.c_double
    L.so_step.argtypes = [C.c_void_p, u16p, C.c_int64, C.c_int64, C.c_int32, C.c_int, C.c_int,
                          C.c_int, u8p, u8p, f32p, f32p, f32p, C.POINTER(Hyper), C.c_int64,
                          C.c_int, f32p, f32p, u8p, f32p, f32p]
    L.so_step.restype = C.c_int
    L.so_dequant.argtypes = [C.c_int, C.c_int64, C.c_int, C.c_int, u8p, f32p, f32p, C.c_int, f32p]
    L.so_bf16_sr.argtypes = [C.c_float, C.c_uint32]
    L.so_bf16_sr.restype = C.c_uint32
    L.so_bf16_rn.argtypes = [C.c_float]
    L.so_bf16_rn.restype = C.c_uint32
    L.so_dequant.restype = C.c_int
    L.so_hardware_threads.argtypes = []
    L.so_hardware_threads.restype = C.c_int
    L.so_qema.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int64, i32p, f32p, f32p, f32p,
                          C.c_float, C.c_float, C.c_float, u32p, f32p]
    L.so_qema.restype = C.c_int
    _lib = L
    return L


def _p(a, ctype):
    return None if a is None else a.ctypes.data_as(C.POINTER(ctype))


def codebook(kind: int, bits: int) -> np.ndarray:
    out = np.zeros(256, np.float32)
    n = lib().so_codebook(kind, bits, _p(out, C.c_float))
    if n < 0:
        raise ValueError("unsupported codebook")
    return out[:n].copy()


def log2_sp(x: float) -> float:
    return lib().so_log2_sp(C.c_float(x))


def exp2_sp(x: float) -> float:
    return lib().so_exp2_sp(C.c_float(x))


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, np.uint32)
    k = np.asarray(key, np.uint32)
    out = np.zeros(4, np.uint32)
    lib().so_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(out, C.c_uint32))
    return out


def philox_draw16(seed: int, step: int, tensor: int, idx: int, purpose: int) -> int:
    """The 16-bit draw of element ``idx`` (purpose 0: second moment, 1: first moment)."""
    return int(lib().so_philox_draw16(seed, step, tensor, idx, purpose))


def xi(draw16: int) -> float:
    return lib().so_xi(draw16)


def u01(draw16: int) -> float:
    return lib().so_u(draw16)


def bf16_sr(x: float, draw16: int) -> int:
    """bf16 bit pattern of ``x`` rounded stochastically with a 16-bit draw."""
    return int(lib().so_bf16_sr(x, draw16))


def bf16_rn(x: float) -> int:
    return int(lib().so_bf16_rn(x))


def quant_nearest(levels: np.ndarray, r: float) -> int:
    y = np.ascontiguousarray(levels, np.float32)
    return lib().so_quant_nearest(_p(y, C.c_float), len(y), C.c_float(r))


def quant_stochastic(levels: np.ndarray, r: float, u: float) -> int:
    y = np.ascontiguousarray(levels, np.float32)
    return lib().so_quant_stochastic(_p(y, C.c_float), len(y), C.c_float(r), C.c_float(u))


def quant_log(r: float, inv_lambda: float, xi_: float, K: int) -> int:
    return lib().so_quant_log(C.c_float(r), C.c_float(inv_lambda), C.c_float(xi_), K)


def pow_sm(alpha: float, q: int) -> float:
    return lib().so_pow_sm(C.c_float(alpha), q)


def log_base(x_p: float, delta: float, K: int) -> tuple[float, float]:
    """Returns (alpha, 1/log2(alpha))."""
    inv = C.c_float()
    a = lib().so_log_base(C.c_float(x_p), C.c_float(delta), K, C.byref(inv))
    return a, inv.value


def get_code(blk: np.ndarray, e: int, b: int) -> int:
    return lib().so_get_code(_p(blk, C.c_uint8), e, b)


def set_code(blk: np.ndarray, e: int, b: int, v: int) -> None:
    lib().so_set_code(_p(blk, C.c_uint8), e, b, v)


def state_bytes(numel: int, bits_m: int, bits_v: int, block: int) -> int:
    out = C.c_uint64()
    if lib().so_state_bytes(numel, bits_m, bits_v, block, C.byref(out)):
        raise ValueError("bad arguments")
    return out.value


def beta_prime(beta: float, r_med_b: float, r_med_bprime: float) -> float:
    return lib().so_beta_prime(beta, r_med_b, r_med_bprime)


def hardware_threads() -> int:
    return lib().so_hardware_threads()


class State:
    """Packed optimizer state of one tensor slice, as plain numpy arrays."""

    def __init__(self, numel: int, bits_m: int, bits_v: int, block: int):
        self.numel, self.bits_m, self.bits_v, self.block = numel, bits_m, bits_v, block
        self.nblk = (numel + block - 1) // block
        self.codes_m = np.zeros(self.nblk * (block * bits_m // 8), np.uint8)
        self.codes_v = np.zeros(self.nblk * (block * bits_v // 8), np.uint8)
        self.scale_m = np.zeros(self.nblk, np.float32)
        self.scale_v = np.zeros(self.nblk, np.float32)
        self.alpha = np.full(self.nblk, 0.5, np.float32)
        self.v_codebook = 0          # selector the second moment was last written with

    def copy(self) -> "State":
        s = State.__new__(State)
        s.__dict__.update(self.__dict__)
        for k in ("codes_m", "codes_v", "scale_m", "scale_v", "alpha"):
            setattr(s, k, getattr(self, k).copy())
        return s


def step(param: np.ndarray, grad_bf16: np.ndarray, st: State, h: Hyper, step_no: int,
         tensor: int = 0, elem_offset: int = 0, nthreads: int = 1, want_hat: bool = False,
         want_flags: bool = False, m32: np.ndarray | None = None,
         v32: np.ndarray | None = None):
    """One optimizer step in place on ``param`` (float32, or uint16 holding bf16 bits when
    ``h.param_dtype == 1``) and ``st``.  ``grad_bf16`` is uint16 (bf16 bit patterns)."""
    n = st.numel
    assert param.flags.c_contiguous and param.size == n
    assert param.dtype == (np.uint16 if h.param_dtype == 1 else np.float32)
    assert grad_bf16.dtype == np.uint16 and grad_bf16.size == n and grad_bf16.flags.c_contiguous
    mh = np.zeros(n, np.float32) if want_hat else None
    vh = np.zeros(n, np.float32) if want_hat else None
    fl = np.zeros(n, np.uint8) if want_flags else None
    rc = lib().so_step(param.ctypes.data_as(C.c_void_p), _p(grad_bf16, C.c_uint16), n,
                       elem_offset, tensor, st.bits_m, st.bits_v, st.block,
                       _p(st.codes_m, C.c_uint8), _p(st.codes_v, C.c_uint8),
                       _p(st.scale_m, C.c_float), _p(st.scale_v, C.c_float),
                       _p(st.alpha, C.c_float), C.byref(h), step_no, nthreads,
                       _p(mh, C.c_float), _p(vh, C.c_float), _p(fl, C.c_uint8),
                       _p(m32, C.c_float), _p(v32, C.c_float))
    if rc:
        raise ValueError("so_step rejected its arguments")
    if m32 is None:
        st.v_codebook = int(h.v_codebook)
    return mh, vh, fl


def dequant(st: State, which: int) -> np.ndarray:
    out = np.zeros(st.numel, np.float32)
    codes, scale, bits = ((st.codes_m, st.scale_m, st.bits_m) if which == 0
                          else (st.codes_v, st.scale_v, st.bits_v))
    rc = lib().so_dequant(which, st.numel, bits, st.block, _p(codes, C.c_uint8),
                          _p(scale, C.c_float), _p(st.alpha, C.c_float), st.v_codebook,
                          _p(out, C.c_float))
    if rc:
        raise ValueError("so_dequant rejected its arguments")
    return out


def qema(mode: int, kind: int, bits: int, codes: np.ndarray, delta: float, alpha: float,
         z: np.ndarray, beta: float, p_quantile: float = 0.1, fixed_alpha: float = 0.0,
         rnd: np.ndarray | None = None, want_hat: bool = False):
    """One quantized-EMA update (Eq. 2-4) of a single quantization unit of any length.
    ``codes`` (int32) is updated in place; returns (delta, alpha[, x_hat])."""
    n = codes.size
    assert codes.dtype == np.int32 and z.dtype == np.float32 and z.size == n
    d, a = C.c_float(delta), C.c_float(alpha)
    xh = np.zeros(n, np.float32) if want_hat else None
    if rnd is not None:
        assert rnd.dtype == np.uint32 and rnd.size == n
    rc = lib().so_qema(mode, kind, bits, n, _p(codes, C.c_int32), C.byref(d), C.byref(a),
                       _p(z, C.c_float), C.c_float(beta), C.c_float(p_quantile),
                       C.c_float(fixed_alpha), _p(rnd, C.c_uint32), _p(xh, C.c_float))
    if rc:
        raise ValueError("so_qema rejected its arguments")
    return (d.value, a.value, xh) if want_hat else (d.value, a.value)
