"""CPU oracle for the lognormal gradient-compression path -- TEST INFRASTRUCTURE.

Thin ctypes access to ``lgn_oracle.c`` (plain scalar C, fp64).  Only the tests,
the smoke check and the benchmark's CPU-baseline leg import this package.  It
imports nothing from the CUDA package and shares no code with it.

Arrays are numpy: float32 for fp32 tensors, uint16 (raw bfloat16 bit patterns)
for bf16 tensors.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lgn_oracle.c")
_LIB = os.path.join(_HERE, "liblgn_oracle.so")

F32, BF16 = 0, 1
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with the host C compiler (no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fno-fast-math",
             _SRC, "-o", _LIB, "-lm"])
    return _LIB


class _Stats(C.Structure):
    _fields_ = [("n", C.c_uint64), ("nnz", C.c_uint64), ("mu", C.c_double),
                ("sigma", C.c_double), ("zero_frac", C.c_double)]


_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        u32, u64, i32, dbl, vp = C.c_uint32, C.c_uint64, C.c_int, C.c_double, C.c_void_p
        lib.orc_stats.argtypes = [vp, u64, i32, C.POINTER(_Stats)]
        lib.orc_stats.restype = None
        lib.orc_stats_masked.argtypes = [vp, vp, u64, i32, C.POINTER(_Stats), C.POINTER(u64)]
        lib.orc_stats_masked.restype = None
        lib.orc_max_abs.argtypes = [vp, u64, i32]
        lib.orc_max_abs.restype = dbl
        lib.orc_scale_exp_from_max.argtypes = [dbl, i32]
        lib.orc_scale_exp_from_max.restype = i32
        lib.orc_cosine_similarity.argtypes = [dbl, dbl, dbl]
        lib.orc_cosine_similarity.restype = dbl
        lib.orc_threshold_for_cosine.argtypes = [dbl, dbl, dbl]
        lib.orc_threshold_for_cosine.restype = dbl
        lib.orc_allocate_sparsity.argtypes = [i32, vp, vp, vp, vp, i32, vp, dbl, dbl, vp]
        lib.orc_allocate_sparsity.restype = dbl
        lib.orc_quantile_k.argtypes = [vp, u64, i32, dbl, dbl, dbl, C.POINTER(dbl)]
        lib.orc_quantile_k.restype = dbl
        lib.orc_philox4x32.argtypes = [vp, vp, i32, vp]
        lib.orc_philox4x32.restype = None
        lib.orc_rand16.argtypes = [u64, u64]
        lib.orc_rand16.restype = u32
        lib.orc_rand16_fill.argtypes = [u64, u64, u64, vp]
        lib.orc_rand16_fill.restype = None
        lib.orc_sparsity_of.argtypes = [dbl, dbl]
        lib.orc_sparsity_of.restype = dbl
        lib.orc_threshold.argtypes = [dbl, dbl, dbl, dbl, C.POINTER(dbl)]
        lib.orc_threshold.restype = i32
        lib.orc_snap_tau.argtypes = [dbl, i32]
        lib.orc_snap_tau.restype = dbl
        lib.orc_prune_one.argtypes = [dbl, dbl, u32]
        lib.orc_prune_one.restype = dbl
        lib.orc_prune_with_bits.argtypes = [vp, vp, u64, i32, dbl, vp]
        lib.orc_prune_with_bits.restype = None
        lib.orc_prune.argtypes = [vp, vp, u64, i32, dbl, u64, u64]
        lib.orc_prune.restype = None
        lib.orc_expected_rel_err.argtypes = [dbl, i32, i32]
        lib.orc_expected_rel_err.restype = dbl
        lib.orc_fp_format.argtypes = [dbl, dbl, u64, i32, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
        lib.orc_fp_format.restype = i32
        lib.orc_quantize_one.argtypes = [dbl, i32, i32, i32, i32, u32]
        lib.orc_quantize_one.restype = u32
        lib.orc_decode.argtypes = [u32, i32, i32, i32]
        lib.orc_decode.restype = dbl
        lib.orc_quantize_with_bits.argtypes = [vp, vp, u64, i32, i32, i32, i32, i32, vp]
        lib.orc_quantize_with_bits.restype = None
        lib.orc_quantize.argtypes = [vp, vp, u64, i32, i32, i32, i32, i32, u64, u64]
        lib.orc_quantize.restype = None
        lib.orc_packed_bytes.argtypes = [u64, i32]
        lib.orc_packed_bytes.restype = u64
        lib.orc_pack.argtypes = [vp, u64, i32, vp]
        lib.orc_pack.restype = None
        lib.orc_unpack.argtypes = [vp, u64, i32, vp]
        lib.orc_unpack.restype = None
        lib.orc_count_zeros.argtypes = [vp, u64, i32]
        lib.orc_dequantize.argtypes = [vp, u64, i32, i32, i32, i32, i32, vp]
        lib.orc_dequantize.restype = None
        lib.orc_prefix_blocks.argtypes = [u64]
        lib.orc_prefix_blocks.restype = u64
        lib.orc_prefix_bound_words.argtypes = [u64, i32]
        lib.orc_prefix_bound_words.restype = u64
        lib.orc_prefix_class.argtypes = [u32, i32, dbl]
        lib.orc_prefix_class.restype = i32
        lib.orc_prefix_encode.argtypes = [vp, u64, i32, dbl, vp, vp]
        lib.orc_prefix_encode.restype = u64
        lib.orc_prefix_decode.argtypes = [vp, vp, u64, i32, dbl, vp]
        lib.orc_prefix_decode.restype = None
        lib.orc_count_zeros.restype = u64
        _lib = lib
    return _lib


def _dtype_of(g: np.ndarray) -> int:
    if g.dtype == np.float32:
        return F32
    if g.dtype == np.uint16:
        return BF16
    raise TypeError("oracle tensors are float32 or uint16 (bfloat16 bits), got %s" % g.dtype)


def _flat(g: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(g).reshape(-1)


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


# --------------------------------------------------------------------------- stats
def stats(g: np.ndarray) -> dict:
    """nnz, mu, sigma of ln|g| over the nonzero entries; zero fraction l."""
    g = _flat(g)
    st = _Stats()
    _L().orc_stats(_ptr(g), g.size, _dtype_of(g), C.byref(st))
    return {"n": st.n, "nnz": st.nnz, "mu": st.mu, "sigma": st.sigma, "zero_frac": st.zero_frac}


def stats_masked(g: np.ndarray, right_mode: np.ndarray) -> dict:
    """Appendix A.9 steps (1), (3): l from the mask, mu and sigma over the right mode
    (right_mode[i] != 0).  ``n_right`` = size of the right mode."""
    g = _flat(g)
    m = np.ascontiguousarray(right_mode, dtype=np.uint8).reshape(-1)
    assert m.size == g.size
    st = _Stats()
    nr = C.c_uint64()
    _L().orc_stats_masked(_ptr(g), _ptr(m), g.size, _dtype_of(g), C.byref(st), C.byref(nr))
    return {"n": st.n, "nnz": st.nnz, "mu": st.mu, "sigma": st.sigma, "zero_frac": st.zero_frac,
            "n_right": nr.value}


def max_abs(g: np.ndarray) -> float:
    g = _flat(g)
    return float(_L().orc_max_abs(_ptr(g), g.size, _dtype_of(g)))


def scale_exp_from_max(max_abs_: float, exp_bits: int) -> int:
    """Algorithm 1's scale read as: the largest element lands in the top binade."""
    return int(_L().orc_scale_exp_from_max(max_abs_, exp_bits))


def fp_format_max_scale(mu: float, sigma: float, nnz: int, nbits: int, max_abs_: float) -> dict:
    """Split from Eq. 4 as in fp_format; scale from the tensor's maximum."""
    f = fp_format(mu, sigma, nnz, nbits)
    if nnz:
        f["scale_exp"] = scale_exp_from_max(max_abs_, f["exp_bits"])
    return f


# --------------------------------------------------------------------------- rng
PHILOX_ROUNDS = 7      # rounds the method uses (the known-answer vectors are for 10)


def philox4x32(ctr, key, rounds: int = 10):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    o = np.zeros(4, dtype=np.uint32)
    _L().orc_philox4x32(_ptr(c), _ptr(k), rounds, _ptr(o))
    return o


def rand16(seed: int, i: int) -> int:
    """The 16 random bits of element i."""
    return int(_L().orc_rand16(seed, i))


def rand16_fill(seed: int, first: int, n: int) -> np.ndarray:
    o = np.zeros(n, dtype=np.uint16)
    _L().orc_rand16_fill(seed, first, n, _ptr(o))
    return o


# --------------------------------------------------------------------------- threshold / prune
def sparsity_of(u: float, sigma: float) -> float:
    """Eq. 8: expected pruned fraction at threshold alpha = e^(mu+u)."""
    return float(_L().orc_sparsity_of(u, sigma))


def threshold(mu: float, sigma: float, zero_frac: float, S: float) -> float:
    tau = C.c_double()
    rc = _L().orc_threshold(mu, sigma, zero_frac, S, C.byref(tau))
    if rc != 0:
        raise ValueError("orc_threshold: invalid argument")
    return tau.value


def snap_tau(tau: float, dtype: int) -> float:
    return float(_L().orc_snap_tau(tau, dtype))


def prune_one(x: float, tau_used: float, h: int) -> float:
    return float(_L().orc_prune_one(x, tau_used, h))


def prune_with_bits(g: np.ndarray, tau_used: float, h: np.ndarray) -> np.ndarray:
    g = _flat(g)
    h = np.ascontiguousarray(h, dtype=np.uint16)
    assert h.size == g.size
    out = np.empty_like(g)
    _L().orc_prune_with_bits(_ptr(g), _ptr(out), g.size, _dtype_of(g), tau_used, _ptr(h))
    return out


def prune(g: np.ndarray, tau_used: float, seed: int, first: int = 0) -> np.ndarray:
    g = _flat(g)
    out = np.empty_like(g)
    _L().orc_prune(_ptr(g), _ptr(out), g.size, _dtype_of(g), tau_used, seed, first)
    return out


# --------------------------------------------------------------------------- cosine similarity / allocation
def cosine_similarity(u: float, sigma: float, k: float) -> float:
    """Expected cos between X and T(X) at threshold alpha = e^(mu+u), log cut off at k sigma."""
    return float(_L().orc_cosine_similarity(u, sigma, k))


def threshold_for_cosine(min_cos: float, sigma: float, k: float) -> float:
    return float(_L().orc_threshold_for_cosine(min_cos, sigma, k))


def allocate_sparsity(n, sigma, zero_frac, k, min_cos, S: float, s_max: float):
    """Layers deepest first; the first len(min_cos) carry a cosine floor.  Returns
    (per-layer sparsity list, element-weighted mean actually allocated)."""
    L = len(n)
    na = np.ascontiguousarray(n, dtype=np.uint64)
    sa = np.ascontiguousarray(sigma, dtype=np.float64)
    za = np.ascontiguousarray(zero_frac, dtype=np.float64)
    ka = np.ascontiguousarray(k, dtype=np.float64)
    ca = np.ascontiguousarray(list(min_cos) + [0.0], dtype=np.float64)
    out = np.zeros(max(L, 1), dtype=np.float64)
    mean = _L().orc_allocate_sparsity(L, _ptr(na), _ptr(sa), _ptr(za), _ptr(ka), len(min_cos), _ptr(ca), S, s_max, _ptr(out))
    return [float(x) for x in out[:L]], float(mean)


def quantile_k(g: np.ndarray, q: float, mu: float, sigma: float):
    """(k, value): the q-quantile of ln|g| over the nonzeros in sigmas above mu, and the order statistic."""
    g = _flat(g)
    v = C.c_double()
    k = _L().orc_quantile_k(_ptr(g), g.size, _dtype_of(g), q, mu, sigma, C.byref(v))
    return float(k), v.value


# --------------------------------------------------------------------------- format / quantize
def expected_rel_err(sigma: float, n1: int, n2: int) -> float:
    """Eq. 4 for n1 mantissa bits and n2 exponent bits."""
    return float(_L().orc_expected_rel_err(sigma, n1, n2))


def fp_format(mu: float, sigma: float, nnz: int, nbits: int) -> dict:
    e, m, s = C.c_int(), C.c_int(), C.c_int()
    rc = _L().orc_fp_format(mu, sigma, nnz, nbits, C.byref(e), C.byref(m), C.byref(s))
    if rc != 0:
        raise ValueError("orc_fp_format: nbits outside 4..8")
    return {"nbits": nbits, "exp_bits": e.value, "man_bits": m.value, "scale_exp": s.value}


def quantize_one(x: float, n2: int, n1: int, e_s: int, rounding: int, h: int = 0) -> int:
    return int(_L().orc_quantize_one(x, n2, n1, e_s, rounding, h))


def decode(code: int, n2: int, n1: int, e_s: int) -> float:
    return float(_L().orc_decode(code, n2, n1, e_s))


def quantize_with_bits(g, n2, n1, e_s, rounding, h=None) -> np.ndarray:
    g = _flat(g)
    codes = np.empty(g.size, dtype=np.uint8)
    hp = None
    if h is not None:
        h = np.ascontiguousarray(h, dtype=np.uint16)
        assert h.size == g.size
        hp = _ptr(h)
    _L().orc_quantize_with_bits(_ptr(g), _ptr(codes), g.size, _dtype_of(g), n2, n1, e_s, rounding, hp)
    return codes


def quantize(g, n2, n1, e_s, rounding, seed=0, first=0) -> np.ndarray:
    """One code per byte (unpacked)."""
    g = _flat(g)
    codes = np.empty(g.size, dtype=np.uint8)
    _L().orc_quantize(_ptr(g), _ptr(codes), g.size, _dtype_of(g), n2, n1, e_s, rounding, seed, first)
    return codes


def packed_bytes(n: int, nbits: int) -> int:
    return int(_L().orc_packed_bytes(n, nbits))


def pack(codes: np.ndarray, nbits: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.zeros(packed_bytes(codes.size, nbits), dtype=np.uint8)
    _L().orc_pack(_ptr(codes), codes.size, nbits, _ptr(out))
    return out


def unpack(packed: np.ndarray, n: int, nbits: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    codes = np.empty(n, dtype=np.uint8)
    _L().orc_unpack(_ptr(packed), n, nbits, _ptr(codes))
    return codes


def count_zeros(g: np.ndarray) -> int:
    g = _flat(g)
    return int(_L().orc_count_zeros(_ptr(g), g.size, _dtype_of(g)))


# --------------------------------------------------------------------------- prefix code (appendix "Encoding")
PREFIX_BLOCK = 2048


def prefix_blocks(n: int) -> int:
    return int(_L().orc_prefix_blocks(n))


def prefix_bound_words(n: int, dtype: int) -> int:
    return int(_L().orc_prefix_bound_words(n, dtype))


def prefix_class(pattern: int, dtype: int, tau_used: float) -> int:
    """0 zero, 1 +alpha, 2 -alpha, 3 FP value."""
    return int(_L().orc_prefix_class(pattern, dtype, tau_used))


def prefix_encode(v: np.ndarray, tau_used: float):
    """(stream uint32[words], off uint64[nblocks+1]) of a pruned tensor."""
    v = _flat(v)
    dt = _dtype_of(v)
    stream = np.zeros(max(1, prefix_bound_words(v.size, dt)), dtype=np.uint32)
    off = np.zeros(prefix_blocks(v.size) + 1, dtype=np.uint64)
    words = int(_L().orc_prefix_encode(_ptr(v), v.size, dt, tau_used, _ptr(stream), _ptr(off)))
    return stream[:words].copy(), off


def prefix_decode(stream: np.ndarray, off: np.ndarray, n: int, dtype: int, tau_used: float) -> np.ndarray:
    stream = np.ascontiguousarray(stream, dtype=np.uint32)
    off = np.ascontiguousarray(off, dtype=np.uint64)
    if stream.size == 0:
        stream = np.zeros(1, dtype=np.uint32)
    out = np.empty(n, dtype=np.uint16 if dtype == BF16 else np.float32)
    _L().orc_prefix_decode(_ptr(stream), _ptr(off), n, dtype, tau_used, _ptr(out))
    return out


# --------------------------------------------------------------------------- decode of a packed stream (Algorithm 1)
def dequantize(packed: np.ndarray, n: int, fmt: dict, out_dtype: int) -> np.ndarray:
    """The tensor a packed code stream stands for, as float32 or bf16 bit patterns (uint16)."""
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    if packed.size == 0:
        packed = np.zeros(1, dtype=np.uint8)
    out = np.empty(n, dtype=np.uint16 if out_dtype == BF16 else np.float32)
    _L().orc_dequantize(_ptr(packed), n, fmt["nbits"], fmt["exp_bits"], fmt["man_bits"], fmt["scale_exp"],
                        out_dtype, _ptr(out))
    return out
