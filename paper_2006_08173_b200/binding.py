"""ctypes binding of ``liblgn.so`` (declared in ``include/lgn.h``).

Argument marshalling only: torch supplies device memory and the current CUDA
stream, every step of the path runs in the library's kernels.  There is no CPU
fallback: if the shared library is missing or cannot be loaded, importing this
module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "liblgn.so")      # the in-tree build, and nothing else

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} not found: build it with `python -m paper_2006_08173_b200.build` "
        "(nvcc, sm_100a); this package has no CPU fallback")
_lib = C.CDLL(LIB_PATH)

LGN_OK = 0
F32, BF16 = 0, 1
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1
MODE_PRUNE, MODE_QUANTIZE = 0, 1
SCALE_CENTRED, SCALE_FROM_MAX = 0, 1


class StatsT(C.Structure):
    _fields_ = [("n", C.c_uint64), ("nnz", C.c_uint64), ("sum_ln", C.c_double),
                ("sum_ln2", C.c_double), ("mu", C.c_double), ("sigma", C.c_double)]


class FpFormatT(C.Structure):
    _fields_ = [("nbits", C.c_int32), ("exp_bits", C.c_int32), ("man_bits", C.c_int32),
                ("scale_exp", C.c_int32)]


class AllocLayerT(C.Structure):
    _fields_ = [("n", C.c_uint64), ("sigma", C.c_double), ("zero_frac", C.c_double), ("k", C.c_double),
                ("min_cos", C.c_double)]


class QuantileT(C.Structure):
    _fields_ = [("value", C.c_float), ("pad", C.c_uint32), ("nnz", C.c_uint64)]


class LayerT(C.Structure):
    _fields_ = [("g", C.c_void_p), ("out", C.c_void_p), ("n", C.c_uint64),
                ("dt", C.c_int32), ("mode", C.c_int32), ("S", C.c_double),
                ("nbits", C.c_int32), ("rounding", C.c_int32), ("seed", C.c_uint64),
                ("use_override", C.c_int32), ("scale_mode", C.c_int32),
                ("mu_override", C.c_double), ("sigma_override", C.c_double), ("right_mode", C.c_void_p),
                ("counters", C.c_int32), ("reserved", C.c_int32)]


class LayerResultT(C.Structure):
    _fields_ = [("stats", StatsT), ("tau", C.c_double), ("fmt", FpFormatT),
                ("status", C.c_int32), ("max_abs", C.c_float), ("n_right_mode", C.c_uint64),
                ("n_zero_out", C.c_uint64), ("n_snapped", C.c_uint64), ("n_saturated", C.c_uint64),
                ("n_underflow", C.c_uint64)]


assert C.sizeof(StatsT) == 48 and C.sizeof(LayerT) == 96 and C.sizeof(LayerResultT) == 120

_vp, _u64, _sz, _dbl, _i32 = C.c_void_p, C.c_uint64, C.c_size_t, C.c_double, C.c_int
_lib.lgn_status_string.argtypes = [_i32]
_lib.lgn_status_string.restype = C.c_char_p
_lib.lgn_workspace_bytes.argtypes = [C.POINTER(_u64), _i32]
_lib.lgn_workspace_bytes.restype = _sz
_lib.lgn_codes_bytes.argtypes = [_u64, _i32]
_lib.lgn_codes_bytes.restype = _sz
_lib.lgn_stats.argtypes = [_vp, _u64, _i32, _vp, _vp, _sz, _vp]
_lib.lgn_stats.restype = _i32
_lib.lgn_threshold.argtypes = [_dbl, _dbl, _dbl, _dbl, C.POINTER(_dbl)]
_lib.lgn_threshold.restype = _i32
_lib.lgn_snap_threshold.argtypes = [_dbl, _i32]
_lib.lgn_snap_threshold.restype = _dbl
_lib.lgn_fp_format.argtypes = [_dbl, _dbl, _i32, C.POINTER(FpFormatT)]
_lib.lgn_fp_format.restype = _i32
_lib.lgn_cosine_similarity.argtypes = [_dbl, _dbl, _dbl, _dbl, C.POINTER(_dbl)]
_lib.lgn_cosine_similarity.restype = _i32
_lib.lgn_allocate_sparsity.argtypes = [C.POINTER(AllocLayerT), _i32, _i32, _dbl, _dbl, C.POINTER(_dbl), C.POINTER(_dbl)]
_lib.lgn_allocate_sparsity.restype = _i32
_lib.lgn_quantile_workspace_bytes.argtypes = []
_lib.lgn_quantile_workspace_bytes.restype = _sz
_lib.lgn_quantile.argtypes = [_vp, _u64, _i32, _dbl, _vp, _vp, _sz, _vp]
_lib.lgn_quantile.restype = _i32
_lib.lgn_combine_stats.argtypes = [C.POINTER(StatsT), _i32, C.POINTER(StatsT)]
_lib.lgn_combine_stats.restype = _i32
_lib.lgn_scale_from_max.argtypes = [_dbl, _i32, C.POINTER(C.c_int32)]
_lib.lgn_scale_from_max.restype = _i32
_lib.lgn_prune.argtypes = [_vp, _vp, _u64, _i32, _dbl, _u64, _vp]
_lib.lgn_prune.restype = _i32
_lib.lgn_quantize.argtypes = [_vp, _vp, _u64, _i32, C.POINTER(FpFormatT), _i32, _u64, _vp]
_lib.lgn_quantize.restype = _i32
_lib.lgn_compress_layers.argtypes = [C.POINTER(LayerT), _i32, _vp, _vp, _sz, _vp]
_lib.lgn_compress_layers.restype = _i32
_lib.lgn_host_staging_bytes.argtypes = [C.POINTER(LayerT), _i32]
_lib.lgn_host_staging_bytes.restype = _sz
_lib.lgn_compress_layers_host.argtypes = [C.POINTER(LayerT), _i32, C.POINTER(LayerResultT), _vp, _sz, _vp]
_lib.lgn_compress_layers_host.restype = _i32
_lib.lgn_selftest_wait_expires.argtypes = [C.POINTER(LayerT), _i32, _vp, _vp, _sz, _vp]
_lib.lgn_selftest_wait_expires.restype = _i32
_lib.lgn_prefix_blocks.argtypes = [_u64]
_lib.lgn_prefix_blocks.restype = _u64
_lib.lgn_prefix_bound_words.argtypes = [_u64, _i32]
_lib.lgn_prefix_bound_words.restype = _u64
_lib.lgn_prefix_workspace_bytes.argtypes = [_u64]
_lib.lgn_prefix_workspace_bytes.restype = _sz
_lib.lgn_prefix_encode.argtypes = [_vp, _u64, _i32, C.c_double, _u64, _i32, _vp, _vp, _u64, _vp, _vp, _sz, _vp]
_lib.lgn_prefix_encode.restype = _i32
_lib.lgn_prefix_decode.argtypes = [_vp, _vp, _u64, _i32, C.c_double, _vp, _vp, _vp]
_lib.lgn_prefix_decode.restype = _i32
_lib.lgn_dequantize.argtypes = [_vp, _u64, C.POINTER(FpFormatT), _i32, _vp, _vp]
_lib.lgn_dequantize.restype = _i32
_lib.lgn_launches_per_call.argtypes = [_i32]
_lib.lgn_launches_per_call.restype = _i32
_lib.lgn_stats_static_scratch.argtypes = [_vp, _u64, _i32, _vp, _vp]
_lib.lgn_stats_static_scratch.restype = _i32
STATS_STATIC_MAX_ELEMS = 1 << 28


class LgnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_lib.lgn_status_string(code).decode()} (status {code})")


def _check(code: int, where: str) -> None:
    if code != LGN_OK:
        raise LgnError(code, where)


def raw():
    """The loaded ctypes library (for tests of the ABI itself)."""
    return _lib


def dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"gradient tensors are float32 or bfloat16, got {t.dtype}")


def _dev(t: torch.Tensor, what: str) -> int:
    if not t.is_cuda:
        raise ValueError(f"{what} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{what} must be contiguous")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


# --------------------------------------------------------------------------- sizes
def lgn_workspace_bytes(n_per_layer: Sequence[int]) -> int:
    arr = (_u64 * max(1, len(n_per_layer)))(*n_per_layer)
    return int(_lib.lgn_workspace_bytes(arr, len(n_per_layer)))


def lgn_launches_per_call(num_layers: int) -> int:
    return int(_lib.lgn_launches_per_call(num_layers))


def lgn_codes_bytes(n: int, nbits: int) -> int:
    return int(_lib.lgn_codes_bytes(n, nbits))


def new_workspace(n_per_layer: Sequence[int], device) -> torch.Tensor:
    return torch.empty(max(16, lgn_workspace_bytes(n_per_layer)), dtype=torch.uint8, device=device)


# --------------------------------------------------------------------------- host closed forms
def lgn_threshold(mu: float, sigma: float, zero_frac: float, S: float) -> float:
    tau = _dbl()
    _check(_lib.lgn_threshold(mu, sigma, zero_frac, S, C.byref(tau)), "lgn_threshold")
    return tau.value


def lgn_snap_threshold(tau: float, dt: int) -> float:
    return float(_lib.lgn_snap_threshold(tau, dt))


def lgn_fp_format(mu: float, sigma: float, nbits: int) -> Dict[str, int]:
    f = FpFormatT()
    _check(_lib.lgn_fp_format(mu, sigma, nbits, C.byref(f)), "lgn_fp_format")
    return {"nbits": f.nbits, "exp_bits": f.exp_bits, "man_bits": f.man_bits, "scale_exp": f.scale_exp}


def lgn_cosine_similarity(mu: float, sigma: float, k: float, tau: float) -> float:
    c = _dbl()
    _check(_lib.lgn_cosine_similarity(mu, sigma, k, tau, C.byref(c)), "lgn_cosine_similarity")
    return c.value


def lgn_allocate_sparsity(layers: Sequence[Dict[str, float]], num_deep: int, S: float, s_max: float):
    """``layers``: dicts with n, sigma, zero_frac, k and (deep layers) min_cos, deepest first.
    Returns (per-layer sparsity list, element-weighted mean allocated)."""
    L = len(layers)
    arr = (AllocLayerT * max(1, L))(*[AllocLayerT(int(a["n"]), float(a["sigma"]), float(a["zero_frac"]),
                                                  float(a.get("k", 0.0)), float(a.get("min_cos", 0.0))) for a in layers])
    out = (_dbl * max(1, L))()
    mean = _dbl()
    _check(_lib.lgn_allocate_sparsity(arr, L, num_deep, S, s_max, out, C.byref(mean)), "lgn_allocate_sparsity")
    return [out[i] for i in range(L)], mean.value


def lgn_quantile_workspace_bytes() -> int:
    return int(_lib.lgn_quantile_workspace_bytes())


def lgn_quantile(g: torch.Tensor, q: float, ws: Optional[torch.Tensor] = None, stream=None) -> Dict[str, float]:
    """The order statistic of rank ceil(q nnz) of |g| over the nonzeros (synchronises to read it back)."""
    ws = ws if ws is not None else torch.empty(lgn_quantile_workspace_bytes(), dtype=torch.uint8, device=g.device)
    out = torch.empty(16, dtype=torch.uint8, device=g.device)
    _check(_lib.lgn_quantile(_dev(g, "g") if g.numel() else None, g.numel(), dtype_code(g), float(q), _dev(out, "out"),
                             _dev(ws, "ws"), ws.numel(), _stream(stream)), "lgn_quantile")
    r = QuantileT.from_buffer_copy(out.cpu().numpy().tobytes())
    return {"value": float(r.value), "nnz": int(r.nnz)}


def lgn_combine_stats(parts: Sequence[Dict[str, float]]) -> Dict[str, float]:
    """Statistics of the union of tensors from each one's n, nnz, sum_ln, sum_ln2."""
    arr = (StatsT * max(1, len(parts)))(*[StatsT(int(p["n"]), int(p["nnz"]), float(p["sum_ln"]), float(p["sum_ln2"]),
                                                 0.0, 0.0) for p in parts])
    out = StatsT()
    _check(_lib.lgn_combine_stats(arr, len(parts), C.byref(out)), "lgn_combine_stats")
    return {"n": out.n, "nnz": out.nnz, "sum_ln": out.sum_ln, "sum_ln2": out.sum_ln2, "mu": out.mu, "sigma": out.sigma}


def lgn_scale_from_max(max_abs: float, exp_bits: int) -> int:
    e = C.c_int32()
    _check(_lib.lgn_scale_from_max(float(max_abs), int(exp_bits), C.byref(e)), "lgn_scale_from_max")
    return e.value


def _fmt_struct(fmt: Dict[str, int]) -> FpFormatT:
    return FpFormatT(fmt["nbits"], fmt["exp_bits"], fmt["man_bits"], fmt["scale_exp"])


# --------------------------------------------------------------------------- device entry points
def lgn_stats_async(g: torch.Tensor, out_dev: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
    """Enqueue the statistics pass; ``out_dev`` (>= 48 bytes, uint8, CUDA) receives one lgn_stats_t."""
    _check(_lib.lgn_stats(_dev(g, "g"), g.numel(), dtype_code(g), _dev(out_dev, "out_dev"),
                          _dev(ws, "ws"), ws.numel() * ws.element_size(), _stream(stream)), "lgn_stats")


def lgn_stats_static_scratch_async(g: torch.Tensor, out_dev: torch.Tensor, stream=None) -> None:
    """lgn_stats without a workspace argument: the scratch is an array inside
    the library (at most STATS_STATIC_MAX_ELEMS elements; calls that may overlap
    on the GPU must not share a device).  Allocates nothing."""
    _check(_lib.lgn_stats_static_scratch(_dev(g, "g") if g.numel() else None, g.numel(), dtype_code(g),
                                         _dev(out_dev, "out_dev"), _stream(stream)), "lgn_stats_static_scratch")


def read_stats(out_dev: torch.Tensor) -> Dict[str, float]:
    raw_bytes = out_dev.cpu().numpy().tobytes()[:C.sizeof(StatsT)]
    st = StatsT.from_buffer_copy(raw_bytes)
    return {"n": st.n, "nnz": st.nnz, "sum_ln": st.sum_ln, "sum_ln2": st.sum_ln2,
            "mu": st.mu, "sigma": st.sigma}


def lgn_stats(g: torch.Tensor, ws: Optional[torch.Tensor] = None, stream=None) -> Dict[str, float]:
    """Statistics of one tensor, read back to the host (synchronises)."""
    ws = ws if ws is not None else new_workspace([g.numel()], g.device)
    out = torch.empty(64, dtype=torch.uint8, device=g.device)
    lgn_stats_async(g, out, ws, stream)
    return read_stats(out)


def lgn_prune(g: torch.Tensor, tau: float, seed: int, out: Optional[torch.Tensor] = None,
              stream=None) -> torch.Tensor:
    out = out if out is not None else torch.empty_like(g)
    _check(_lib.lgn_prune(_dev(g, "g"), _dev(out, "out"), g.numel(), dtype_code(g), float(tau),
                          int(seed), _stream(stream)), "lgn_prune")
    return out


def lgn_quantize(g: torch.Tensor, fmt: Dict[str, int], rounding: int, seed: int,
                 out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Packed codes as a uint8 tensor of lgn_codes_bytes(n, nbits) bytes."""
    if out is None:
        out = torch.empty(max(16, lgn_codes_bytes(g.numel(), fmt["nbits"])), dtype=torch.uint8, device=g.device)
    f = _fmt_struct(fmt)
    _check(_lib.lgn_quantize(_dev(g, "g"), _dev(out, "codes"), g.numel(), dtype_code(g), C.byref(f),
                             int(rounding), int(seed), _stream(stream)), "lgn_quantize")
    return out


def lgn_dequantize(codes: torch.Tensor, n: int, fmt: Dict[str, int], out: torch.Tensor, stream=None) -> torch.Tensor:
    """Decode ``n`` packed codes (uint8 CUDA tensor) into ``out`` (float32 or bfloat16, n elements)."""
    if out.numel() != n:
        raise ValueError("out must hold n elements")
    if codes.numel() * codes.element_size() < lgn_codes_bytes(n, fmt["nbits"]):
        raise ValueError("codes shorter than lgn_codes_bytes(n, nbits)")
    f = _fmt_struct(fmt)
    _check(_lib.lgn_dequantize(_dev(codes, "codes") if n else None, n, C.byref(f), dtype_code(out),
                               _dev(out, "out") if n else None, _stream(stream)), "lgn_dequantize")
    return out


def make_layer(g: torch.Tensor, out: torch.Tensor, mode: int, S: float = 0.0, nbits: int = 0,
               rounding: int = ROUND_NEAREST, seed: int = 0, mu_override: Optional[float] = None,
               sigma_override: Optional[float] = None, scale_mode: int = SCALE_CENTRED,
               right_mode: Optional[torch.Tensor] = None, counters: bool = False) -> LayerT:
    """``right_mode``: uint8/bool CUDA tensor of g.numel() bytes (bi-modal pruning), or None.
    ``counters``: have the apply pass fill n_zero_out .. n_underflow of the layer's result."""
    use = mu_override is not None and sigma_override is not None
    mask = None
    if right_mode is not None:
        if right_mode.element_size() != 1 or right_mode.numel() != g.numel():
            raise ValueError("right_mode must hold one byte per element of g")
        mask = _dev(right_mode, "right_mode") if g.numel() else None
    return LayerT(_dev(g, "g") if g.numel() else (g.data_ptr() or None),
                  _dev(out, "out") if out.numel() else (out.data_ptr() or None), g.numel(), dtype_code(g),
                  mode, float(S), int(nbits), int(rounding), int(seed), 1 if use else 0, int(scale_mode),
                  float(mu_override) if use else 0.0, float(sigma_override) if use else 0.0, mask,
                  1 if counters else 0, 0)


def lgn_compress_layers(layers: Sequence[LayerT], results_dev: torch.Tensor, ws: torch.Tensor,
                        stream=None) -> None:
    """Enqueue the grouped path.  ``results_dev``: uint8 CUDA tensor of at least
    120 bytes per layer; ``ws``: uint8 CUDA tensor of lgn_workspace_bytes(...)."""
    L = len(layers)
    arr = (LayerT * max(1, L))(*layers)
    if results_dev.numel() * results_dev.element_size() < L * C.sizeof(LayerResultT):
        raise ValueError("results_dev too small")
    _check(_lib.lgn_compress_layers(arr, L, _dev(results_dev, "results_dev"), _dev(ws, "ws"),
                                    ws.numel() * ws.element_size(), _stream(stream)), "lgn_compress_layers")


def lgn_selftest_wait_expires(layers: Sequence[LayerT], results_dev: torch.Tensor, ws: torch.Tensor,
                              stream=None) -> None:
    """lgn_compress_layers with one statistics tile of layer 0 withheld: layer 0
    must come back with status LGN_ERR_TIMEOUT after about a second."""
    L = len(layers)
    arr = (LayerT * max(1, L))(*layers)
    _check(_lib.lgn_selftest_wait_expires(arr, L, _dev(results_dev, "results_dev"), _dev(ws, "ws"),
                                          ws.numel() * ws.element_size(), _stream(stream)),
           "lgn_selftest_wait_expires")


def new_results(num_layers: int, device) -> torch.Tensor:
    return torch.zeros(max(1, num_layers) * C.sizeof(LayerResultT), dtype=torch.uint8, device=device)


def read_results(results_dev: torch.Tensor, num_layers: int) -> List[Dict]:
    """Host copy of the per-layer results (synchronises)."""
    buf = results_dev.cpu().numpy().tobytes()
    out = []
    for k in range(num_layers):
        r = LayerResultT.from_buffer_copy(buf[k * C.sizeof(LayerResultT):(k + 1) * C.sizeof(LayerResultT)])
        out.append({"n": r.stats.n, "nnz": r.stats.nnz, "sum_ln": r.stats.sum_ln, "sum_ln2": r.stats.sum_ln2,
                    "mu": r.stats.mu, "sigma": r.stats.sigma, "tau": r.tau,
                    "fmt": {"nbits": r.fmt.nbits, "exp_bits": r.fmt.exp_bits, "man_bits": r.fmt.man_bits,
                            "scale_exp": r.fmt.scale_exp},
                    "status": r.status, "max_abs": r.max_abs, "n_right_mode": r.n_right_mode,
                    "n_zero_out": r.n_zero_out, "n_snapped": r.n_snapped, "n_saturated": r.n_saturated,
                    "n_underflow": r.n_underflow})
    return out


# --------------------------------------------------------------------------- host-buffer form
def _result_dict(r: LayerResultT) -> Dict:
    return {"n": r.stats.n, "nnz": r.stats.nnz, "sum_ln": r.stats.sum_ln, "sum_ln2": r.stats.sum_ln2,
            "mu": r.stats.mu, "sigma": r.stats.sigma, "tau": r.tau,
            "fmt": {"nbits": r.fmt.nbits, "exp_bits": r.fmt.exp_bits, "man_bits": r.fmt.man_bits,
                    "scale_exp": r.fmt.scale_exp},
            "status": r.status, "max_abs": r.max_abs, "n_right_mode": r.n_right_mode,
            "n_zero_out": r.n_zero_out, "n_snapped": r.n_snapped, "n_saturated": r.n_saturated,
            "n_underflow": r.n_underflow}


def make_host_layer(g: torch.Tensor, out: torch.Tensor, mode: int, **kw) -> LayerT:
    """Descriptor whose g/out are HOST tensors (pinned memory recommended)."""
    if g.is_cuda or out.is_cuda or not g.is_contiguous() or not out.is_contiguous():
        raise ValueError("host layers take contiguous CPU tensors")
    lay = LayerT(g.data_ptr() or None, out.data_ptr() or None, g.numel(), dtype_code(g), mode,
                 float(kw.get("S", 0.0)), int(kw.get("nbits", 0)), int(kw.get("rounding", ROUND_NEAREST)),
                 int(kw.get("seed", 0)), 0, int(kw.get("scale_mode", SCALE_CENTRED)), 0.0, 0.0,
                 (kw["right_mode"].data_ptr() or None) if kw.get("right_mode") is not None else None,
                 1 if kw.get("counters") else 0, 0)
    return lay


def lgn_host_staging_bytes(layers: Sequence[LayerT]) -> int:
    arr = (LayerT * max(1, len(layers)))(*layers)
    return int(_lib.lgn_host_staging_bytes(arr, len(layers)))


def lgn_compress_layers_host(layers: Sequence[LayerT], dev_buf: torch.Tensor, stream=None) -> List[Dict]:
    """Host tensors in, host tensors out; copies and the kernel run inside the
    call, which returns when everything has landed."""
    L = len(layers)
    arr = (LayerT * max(1, L))(*layers)
    res = (LayerResultT * max(1, L))()
    _check(_lib.lgn_compress_layers_host(arr, L, res, _dev(dev_buf, "dev_buf"),
                                         dev_buf.numel() * dev_buf.element_size(), _stream(stream)),
           "lgn_compress_layers_host")
    return [_result_dict(res[k]) for k in range(L)]


# --------------------------------------------------------------------------- prefix code (appendix "Encoding")
PREFIX_BLOCK = 2048


def lgn_prefix_blocks(n: int) -> int:
    return int(_lib.lgn_prefix_blocks(n))


def lgn_prefix_bound_words(n: int, dtype_code_: int) -> int:
    return int(_lib.lgn_prefix_bound_words(n, dtype_code_))


def lgn_prefix_workspace_bytes(n: int) -> int:
    return int(_lib.lgn_prefix_workspace_bytes(n))


def lgn_prefix_encode(g: torch.Tensor, tau: float, seed: int, apply_prune: bool, stream_dev: torch.Tensor,
                      off_dev: torch.Tensor, ws: torch.Tensor, tau_from_dev: Optional[int] = None,
                      stream=None) -> None:
    """``stream_dev``: int32/uint32 CUDA tensor (capacity = its length in words);
    ``off_dev``: int64 CUDA tensor of lgn_prefix_blocks(n) + 1 entries;
    ``tau_from_dev``: device address of a layer result record, or None."""
    if off_dev.numel() < lgn_prefix_blocks(g.numel()) + 1 or off_dev.element_size() != 8:
        raise ValueError("off_dev too small")
    if stream_dev.element_size() != 4:
        raise ValueError("stream_dev must hold 32-bit words")
    _check(_lib.lgn_prefix_encode(_dev(g, "g") if g.numel() else None, g.numel(), dtype_code(g), float(tau), int(seed),
                                  1 if apply_prune else 0, tau_from_dev,
                                  _dev(stream_dev, "stream_dev") if stream_dev.numel() else None, stream_dev.numel(),
                                  _dev(off_dev, "off_dev"), _dev(ws, "ws"), ws.numel() * ws.element_size(),
                                  _stream(stream)), "lgn_prefix_encode")


def lgn_prefix_decode(stream_dev: torch.Tensor, off_dev: torch.Tensor, out: torch.Tensor, tau: float,
                      tau_from_dev: Optional[int] = None, stream=None) -> torch.Tensor:
    _check(_lib.lgn_prefix_decode(_dev(stream_dev, "stream_dev") if stream_dev.numel() else None,
                                  _dev(off_dev, "off_dev"), out.numel(), dtype_code(out), float(tau), tau_from_dev,
                                  _dev(out, "out") if out.numel() else None, _stream(stream)), "lgn_prefix_decode")
    return out
