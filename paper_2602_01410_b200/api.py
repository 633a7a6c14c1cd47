"""Thin Python binding of the C-ABI library declared in include/snip.h.

Argument marshalling only: every function takes torch CUDA tensors (used here purely as device
memory) and forwards raw pointers and sizes to the entry point of the same name.  All work runs
in the library's CUDA kernels on torch's current stream.  There is no fallback: if the shared
library is missing or fails to load, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

FMT_BF16, FMT_FP8_E4M3, FMT_FP4_E2M1 = 0, 1, 2
BLOCK_ROW, BLOCK_COL, BLOCK_BLK = 0, 1, 2
BLOCK_ROW32, BLOCK_COL32 = 3, 4   # 32-long tiles, power-of-two scales only
BLOCK_ROW16, BLOCK_COL16 = 5, 6   # 16-long tiles of the two-level option
OUT_BF16, OUT_FP32 = 0, 1
OP_FWD, OP_DGRAD, OP_WGRAD = 0, 1, 2
Q_TRANSPOSED, Q_STATS, Q_NO_CODES = 1, 2, 4
OK = 0
ERR_ARG, ERR_SHAPE, ERR_ALIGN, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(1, 8)

LIB_PATH = os.environ.get("SNIP_B200_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsnip_b200.so")

EXPORTS = (
    "snip_version", "snip_status_string", "snip_last_cuda_error", "snip_quantize_sizes",
    "snip_quantize", "snip_quantize_noalloc", "snip_quantize_mx_sizes", "snip_quantize_mx", "snip_quantize_dual_workspace", "snip_quantize_dual", "snip_quantize_sr", "snip_workspace_size", "snip_gemm_quantized", "snip_gemm_mx", "snip_quantize_nvfp4_sizes", "snip_quantize_nvfp4_dual", "snip_gemm_nvfp4", "snip_linear_fwd_bwd_nvfp4_workspace", "snip_linear_fwd_bwd_nvfp4", "snip_linear_fwd",
    "snip_linear_dgrad", "snip_linear_wgrad", "snip_linear_mx", "snip_linear_mx_workspace", "snip_linear_fwd_bwd_workspace", "snip_linear_fwd_bwd", "snip_layer_stats", "snip_layer_stats_workspace", "snip_adamw_sensitivity_workspace", "snip_adamw_sensitivity", "snip_loss_divergence", "snip_weight_divergence", "snip_select_scheme",
    "snip_poll_status", "snip_debug_set",
)


class SnipError(RuntimeError):
    def __init__(self, fn, status):
        self.status = status
        name = _lib.snip_status_string(status).decode()
        detail = _lib.snip_last_cuda_error().decode() if status == ERR_CUDA else ""
        super().__init__(f"{fn} failed: {name} {detail}".strip())


class QTensor(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("rows", ctypes.c_int64),
                ("cols", ctypes.c_int64), ("fmt", ctypes.c_int32), ("block", ctypes.c_int32),
                ("transposed", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class QOut(ctypes.Structure):
    _fields_ = [("fmt", ctypes.c_int32), ("rounding", ctypes.c_int32), ("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p),
                ("sf", ctypes.c_void_p), ("stats", ctypes.c_void_p), ("seed", ctypes.c_uint64)]


DUAL_ROW_COLT, DUAL_BLK_BLKT, DUAL_ROW32_COL32T = 0, 1, 2
ROUND_NEAREST_EVEN, ROUND_STOCHASTIC = 0, 1
DEBUG_WAIT_LIMIT_NS, DEBUG_TX_SKEW_BYTES, DEBUG_GEMM_KERNEL, DEBUG_GEMM_SLICING = 0, 1, 2, 3
GEMM_KERNEL_AUTO, GEMM_KERNEL_SINGLE, GEMM_KERNEL_PAIR = 0, 1, 2


class LayerTensors(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("X", "W", "Y", "dY", "dX", "dW")] + \
               [(n, ctypes.c_int64) for n in ("M", "N", "K")]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2602_01410_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    i32, i64, u32, vp, sz = ctypes.c_int, ctypes.c_int64, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_size_t
    psz = ctypes.POINTER(sz)
    lib.snip_version.restype = i32
    lib.snip_status_string.restype = ctypes.c_char_p
    lib.snip_status_string.argtypes = [i32]
    lib.snip_last_cuda_error.restype = ctypes.c_char_p
    lib.snip_quantize_sizes.argtypes = [i64, i64, i32, i32, u32, psz, psz, psz]
    lib.snip_quantize.argtypes = [vp, i64, i64, i64, i32, i32, u32, vp, vp, vp, vp, vp, sz, vp]
    lib.snip_quantize_noalloc.argtypes = [vp, i64, i64, i64, i32, i32, u32, vp, vp, vp, vp]
    lib.snip_quantize_mx_sizes.argtypes = [i64, i64, psz]
    lib.snip_quantize_mx.argtypes = [vp, i64, i64, i64, i32, i32, u32, vp, vp, vp, vp, vp, sz, vp]
    lib.snip_quantize_dual_workspace.argtypes = [i64, i64, psz]
    lib.snip_quantize_dual.argtypes = [vp, i64, i64, i64, i32, i32, ctypes.POINTER(QOut), ctypes.POINTER(QOut), vp, sz, vp]
    lib.snip_quantize_sr.argtypes = [vp, i64, i64, i64, i32, u32, ctypes.c_uint64, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.snip_workspace_size.argtypes = [i32, i64, i64, i64, i32, i32, psz, psz]
    lib.snip_gemm_quantized.argtypes = [i32, ctypes.POINTER(QTensor), ctypes.POINTER(QTensor), vp, i32, i32, vp, sz, vp]
    lib.snip_gemm_mx.argtypes = [i32, ctypes.POINTER(QTensor), vp, ctypes.POINTER(QTensor), vp, vp, i32, vp, sz, vp]
    lib.snip_quantize_nvfp4_sizes.argtypes = [i64, i64, psz, psz]
    lib.snip_quantize_nvfp4_dual.argtypes = [vp, i64, i64, i64, vp, vp, vp, vp, vp, vp, vp, i32, ctypes.c_uint64, vp, sz, vp]
    lib.snip_gemm_nvfp4.argtypes = [i32, ctypes.POINTER(QTensor), vp, vp, ctypes.POINTER(QTensor), vp, vp, vp, i32, vp, sz, vp]
    lib.snip_linear_fwd_bwd_nvfp4_workspace.argtypes = [i64, i64, i64, psz]
    lib.snip_linear_fwd_bwd_nvfp4.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, vp, i32, ctypes.c_uint64, vp, vp, sz, vp]
    lin = [vp, vp, vp, i64, i64, i64, i32, i32, i32, vp, vp, vp, sz, vp]
    lib.snip_linear_fwd.argtypes = lin
    lib.snip_linear_dgrad.argtypes = lin
    lib.snip_linear_wgrad.argtypes = [vp, vp, vp, i64, i64, i64, i32, i32, i32, i32, vp, vp, vp, sz, vp]
    lib.snip_linear_mx.argtypes = [i32, vp, vp, vp, i64, i64, i64, i32, i32, i32, vp, vp, vp, sz, vp]
    lib.snip_linear_mx_workspace.argtypes = [i32, i64, i64, i64, i32, i32, psz]
    lib.snip_linear_fwd_bwd_workspace.argtypes = [i64, i64, i64, i32, i32, i32, i32, psz]
    lib.snip_linear_fwd_bwd.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i32, i32, i32, i32, i32, ctypes.c_uint64, vp, vp, sz, vp]
    lib.snip_layer_stats.argtypes = [ctypes.POINTER(LayerTensors), u32, vp, vp, sz, vp]
    lib.snip_layer_stats_workspace.argtypes = [i64, i64, i64, psz]
    lib.snip_adamw_sensitivity_workspace.argtypes = [i64, psz]
    lib.snip_adamw_sensitivity.argtypes = [vp, vp, vp, i32, i64, ctypes.c_float, ctypes.c_float, ctypes.c_float, vp, vp, sz, vp]
    dbl = ctypes.c_double
    lib.snip_loss_divergence.restype = dbl
    lib.snip_loss_divergence.argtypes = [dbl, dbl, i64, i64, dbl, dbl, i64, dbl]
    lib.snip_weight_divergence.restype = dbl
    lib.snip_weight_divergence.argtypes = [dbl, dbl, i64, i64, dbl, dbl, dbl, i64, dbl, i64]
    lib.snip_select_scheme.argtypes = [i32, i32, vp, vp, i64, i32, vp, vp, vp]
    lib.snip_poll_status.argtypes = [vp, ctypes.POINTER(i32)]
    lib.snip_debug_set.argtypes = [i32, ctypes.c_longlong]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is ctypes.c_int and name not in ("snip_version",):
            fn.restype = i32
    return lib


_lib = _load()


def _check(fn, status):
    if status != OK:
        raise SnipError(fn, status)


def _p(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def snip_version() -> int:
    return int(_lib.snip_version())


def snip_status_string(status: int) -> str:
    return _lib.snip_status_string(status).decode()


def snip_quantize_sizes(rows, cols, fmt, block, flags=0):
    cb, sb, wb = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    _check("snip_quantize_sizes", _lib.snip_quantize_sizes(rows, cols, fmt, block, flags, ctypes.byref(cb),
                                                            ctypes.byref(sb), ctypes.byref(wb)))
    return cb.value, sb.value, wb.value


def stats_to_host(stats: torch.Tensor) -> dict:
    """Decode a snip_stats_t held in a 24-byte uint8 tensor (synchronizes)."""
    raw = stats.cpu().numpy().tobytes()
    import struct
    sx, se, am, _ = struct.unpack("<ddfI", raw[:24])
    return {"sumsq_x": sx, "sumsq_err": se, "amax": am}


def snip_quantize(x: torch.Tensor, fmt: int, block: int, flags: int = 0, *, codes=None, scales=None,
                  stats=None, row_stats=None, ws=None, want_row_stats=False):
    """x: bf16 CUDA tensor [rows, cols] (row stride = x.stride(0)).  Allocates any output not
    supplied, through torch, and returns (codes, scales, stats, row_stats) as uint8 / float32 /
    uint8[24] / float64[rows,2] tensors (None where not produced)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    cb, sb, wb = snip_quantize_sizes(rows, cols, fmt, block, flags)
    dev = x.device
    if cb and codes is None:
        codes = torch.empty(cb, dtype=torch.uint8, device=dev)
    if sb and scales is None:
        scales = torch.empty(sb // 4, dtype=torch.float32, device=dev)
    if (flags & Q_STATS) and stats is None:
        stats = torch.empty(24, dtype=torch.uint8, device=dev)
    if want_row_stats and row_stats is None:
        row_stats = torch.empty((rows, 2), dtype=torch.float64, device=dev)
    if ws is None and ((flags & Q_STATS) or row_stats is not None):
        ws = torch.empty(wb, dtype=torch.uint8, device=dev)
    _check("snip_quantize", _lib.snip_quantize(_p(x), rows, cols, x.stride(0), fmt, block, flags, _p(codes), _p(scales),
                                               _p(stats), _p(row_stats), _p(ws), 0 if ws is None else ws.numel(), _stream()))
    return codes, scales, stats, row_stats


def snip_quantize_noalloc(x: torch.Tensor, fmt: int, block: int, flags: int, codes, scales, stats):
    """Same work as snip_quantize with the statistics scratch taken from the array built into the
    library, for hosts that cannot give it any.  The caller passes every output buffer: this wrapper,
    like the entry point, allocates nothing."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    _check("snip_quantize_noalloc", _lib.snip_quantize_noalloc(_p(x), rows, cols, x.stride(0), fmt, block, flags, _p(codes),
                                                               _p(scales), _p(stats), _stream()))


def snip_quantize_mx(x: torch.Tensor, fmt: int, block: int, flags: int = 0, *, want_sf=True):
    """Power-of-two scale option.  Returns (codes, scales, sf, stats): uint8, float32, uint8 (UE8M0
    atoms, None unless want_sf) and a 32-byte stats buffer (None unless Q_STATS)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    cb, sb, wb = snip_quantize_sizes(rows, cols, fmt, block, flags)
    dev = x.device
    codes = torch.empty(cb, dtype=torch.uint8, device=dev)
    scales = torch.empty(sb // 4, dtype=torch.float32, device=dev)
    sf = None
    if want_sf:
        n = ctypes.c_size_t()
        _check("snip_quantize_mx_sizes", _lib.snip_quantize_mx_sizes(rows, cols, ctypes.byref(n)))
        sf = torch.empty(n.value, dtype=torch.uint8, device=dev)
    stats = torch.empty(32, dtype=torch.uint8, device=dev) if (flags & Q_STATS) else None
    ws = torch.empty(wb, dtype=torch.uint8, device=dev) if (flags & Q_STATS) else None
    _check("snip_quantize_mx", _lib.snip_quantize_mx(_p(x), rows, cols, x.stride(0), fmt, block, flags, _p(codes), _p(scales), _p(sf),
                                                     _p(stats), _p(ws), 0 if ws is None else ws.numel(), _stream()))
    return codes, scales, sf, stats


def snip_quantize_dual_workspace(rows, cols):
    n = ctypes.c_size_t()
    _check("snip_quantize_dual_workspace", _lib.snip_quantize_dual_workspace(rows, cols, ctypes.byref(n)))
    return n.value


def snip_quantize_sr(x: torch.Tensor, block: int, flags: int, seed: int, *, pow2_scale=False, want_sf=False):
    """FP4 codes with stochastic rounding.  Returns (codes, scales, sf, stats) like snip_quantize_mx."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    cb, sb, wb = snip_quantize_sizes(rows, cols, FMT_FP4_E2M1, block, flags)
    dev = x.device
    codes = torch.empty(cb, dtype=torch.uint8, device=dev)
    scales = torch.empty(sb // 4, dtype=torch.float32, device=dev)
    sf = None
    if want_sf:
        n = ctypes.c_size_t()
        _check("snip_quantize_mx_sizes", _lib.snip_quantize_mx_sizes(rows, cols, ctypes.byref(n)))
        sf = torch.empty(n.value, dtype=torch.uint8, device=dev)
    stats = torch.empty(32, dtype=torch.uint8, device=dev) if (flags & Q_STATS) else None
    ws = torch.empty(wb, dtype=torch.uint8, device=dev) if (flags & Q_STATS) else None
    _check("snip_quantize_sr", _lib.snip_quantize_sr(_p(x), rows, cols, x.stride(0), block, flags, seed, int(pow2_scale), _p(codes), _p(scales),
                                                     _p(sf), _p(stats), _p(ws), 0 if ws is None else ws.numel(), _stream()))
    return codes, scales, sf, stats


def snip_quantize_dual(x: torch.Tensor, kind: int, fmt_stored: int, fmt_transposed: int, *, pow2_scale=False, want_stats=True,
                       want_sf=False, bufs=None, ws=None, sr_seeds=(None, None)):
    """One read, two outputs.  Returns two dicts (as stored, transposed) with codes / scales / sf / stats
    tensors (sf, stats None unless asked for).  bufs = (dict, dict) reuses buffers of an earlier call."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    dev = x.device
    blocks = {DUAL_ROW_COLT: (BLOCK_ROW, BLOCK_COL), DUAL_BLK_BLKT: (BLOCK_BLK, BLOCK_BLK), DUAL_ROW32_COL32T: (BLOCK_ROW32, BLOCK_COL32)}[kind]
    outs, structs = [], []
    for i, fmt in enumerate((fmt_stored, fmt_transposed)):
        if bufs is not None:
            o = bufs[i]
        else:
            cb, sb, _ = snip_quantize_sizes(rows, cols, fmt, blocks[i], Q_TRANSPOSED if i else 0)
            o = {"codes": torch.empty(cb, dtype=torch.uint8, device=dev), "scales": torch.empty(sb // 4, dtype=torch.float32, device=dev),
                 "sf": None, "stats": torch.empty(32, dtype=torch.uint8, device=dev) if want_stats else None}
            if want_sf:
                n = ctypes.c_size_t()
                _check("snip_quantize_mx_sizes", _lib.snip_quantize_mx_sizes(rows, cols, ctypes.byref(n)))
                o["sf"] = torch.empty(n.value, dtype=torch.uint8, device=dev)
        outs.append(o)
        seed = sr_seeds[i]
        structs.append(QOut(fmt, ROUND_NEAREST_EVEN if seed is None else ROUND_STOCHASTIC, _p(o["codes"]), _p(o["scales"]), _p(o["sf"]),
                            _p(o["stats"]), 0 if seed is None else seed))
    if ws is None and outs[0]["stats"] is not None:
        ws = torch.empty(snip_quantize_dual_workspace(rows, cols), dtype=torch.uint8, device=dev)
    _check("snip_quantize_dual", _lib.snip_quantize_dual(_p(x), rows, cols, x.stride(0), kind, int(pow2_scale), ctypes.byref(structs[0]),
                                                         ctypes.byref(structs[1]), _p(ws), 0 if ws is None else ws.numel(), _stream()))
    return outs[0], outs[1]


def snip_workspace_size(op, M, N, K, fmt_a, fmt_b):
    g, l = ctypes.c_size_t(), ctypes.c_size_t()
    _check("snip_workspace_size", _lib.snip_workspace_size(op, M, N, K, fmt_a, fmt_b, ctypes.byref(g), ctypes.byref(l)))
    return g.value, l.value


def make_qtensor(codes, scales, rows, cols, fmt, block, transposed=False) -> QTensor:
    return QTensor(codes.data_ptr(), 0 if scales is None else scales.data_ptr(), rows, cols, fmt, block,
                   int(transposed), 0)


def _out(shape, out_dtype, device, out):
    if out is not None:
        return out
    return torch.empty(shape, dtype=torch.bfloat16 if out_dtype == OUT_BF16 else torch.float32, device=device)


def snip_gemm_quantized(op, a: QTensor, b: QTensor, out_shape, out_dtype=OUT_BF16, accumulate=False, *, out=None,
                        ws=None, device="cuda"):
    out = _out(out_shape, out_dtype, device, out)
    if ws is None:
        M, N = out_shape
        g, _ = snip_workspace_size(op, *_mnk(op, a, b), a.fmt, b.fmt)
        ws = torch.zeros(g, dtype=torch.uint8, device=out.device)
    _check("snip_gemm_quantized", _lib.snip_gemm_quantized(op, ctypes.byref(a), ctypes.byref(b), _p(out), out_dtype,
                                                           int(accumulate), _p(ws), ws.numel(), _stream()))
    return out


def snip_gemm_mx(op, a: QTensor, sf_a, b: QTensor, sf_b, out_shape, out_dtype=OUT_BF16, *, out=None, ws=None, device="cuda"):
    out = _out(out_shape, out_dtype, device, out)
    if ws is None:
        ws = torch.zeros(256, dtype=torch.uint8, device=out.device)
    _check("snip_gemm_mx", _lib.snip_gemm_mx(op, ctypes.byref(a), _p(sf_a), ctypes.byref(b), _p(sf_b), _p(out), out_dtype, _p(ws),
                                             ws.numel(), _stream()))
    return out


def snip_quantize_nvfp4_sizes(rows, cols):
    cb, sb = ctypes.c_size_t(), ctypes.c_size_t()
    _check("snip_quantize_nvfp4_sizes", _lib.snip_quantize_nvfp4_sizes(rows, cols, ctypes.byref(cb), ctypes.byref(sb)))
    return cb.value, sb.value


def snip_quantize_nvfp4_dual(x: torch.Tensor, tensor_amax: torch.Tensor, *, want_stats=True, bufs=None, ws=None, sr_seed=None):
    """Two-level option, both copies from one read.  tensor_amax: float32 CUDA tensor with one element (the bound of |x|).
    Returns two dicts (as stored, transposed) with codes / sf / stats tensors."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    assert tensor_amax.is_cuda and tensor_amax.dtype == torch.float32
    rows, cols = x.shape
    dev = x.device
    if bufs is None:
        cb, sb = snip_quantize_nvfp4_sizes(rows, cols)
        bufs = tuple({"codes": torch.empty(cb, dtype=torch.uint8, device=dev), "sf": torch.empty(sb, dtype=torch.uint8, device=dev),
                      "stats": torch.empty(32, dtype=torch.uint8, device=dev) if want_stats else None} for _ in range(2))
    if ws is None and bufs[0]["stats"] is not None:
        ws = torch.empty(snip_quantize_dual_workspace(rows, cols), dtype=torch.uint8, device=dev)
    a, b = bufs
    _check("snip_quantize_nvfp4_dual", _lib.snip_quantize_nvfp4_dual(_p(x), rows, cols, x.stride(0), _p(tensor_amax), _p(a["codes"]), _p(a["sf"]),
                                                                     _p(a["stats"]), _p(b["codes"]), _p(b["sf"]), _p(b["stats"]),
                                                                     ROUND_NEAREST_EVEN if sr_seed is None else ROUND_STOCHASTIC, 0 if sr_seed is None else sr_seed,
                                                                     _p(ws), 0 if ws is None else ws.numel(), _stream()))
    return a, b


def snip_gemm_nvfp4(op, a: QTensor, sf_a, amax_a, b: QTensor, sf_b, amax_b, out_shape, out_dtype=OUT_BF16, *, out=None, ws=None, device="cuda"):
    out = _out(out_shape, out_dtype, device, out)
    if ws is None:
        ws = torch.zeros(256, dtype=torch.uint8, device=out.device)
    _check("snip_gemm_nvfp4", _lib.snip_gemm_nvfp4(op, ctypes.byref(a), _p(sf_a), _p(amax_a), ctypes.byref(b), _p(sf_b), _p(amax_b), _p(out), out_dtype,
                                                   _p(ws), ws.numel(), _stream()))
    return out


def _mnk(op, a: QTensor, b: QTensor):
    if op == OP_FWD:      # a = X[M,K], b = W[N,K]
        return a.rows, b.rows, a.cols
    if op == OP_DGRAD:    # a = dY[M,N], b = W[N,K]
        return a.rows, a.cols, b.cols
    return a.rows, a.cols, b.cols  # wgrad: a = dY[M,N], b = X[M,K]


def _linear(fn_name, A, B, out_shape, M, N, K, fmt_a, fmt_b, out_dtype, op, out, ws, want_stats, extra=()):
    out = _out(out_shape, out_dtype, A.device, out)
    if ws is None:
        _, l = snip_workspace_size(op, M, N, K, fmt_a, fmt_b)
        ws = torch.zeros(l, dtype=torch.uint8, device=A.device)
    sa = torch.empty(24, dtype=torch.uint8, device=A.device) if want_stats else None
    sb = torch.empty(24, dtype=torch.uint8, device=A.device) if want_stats else None
    fn = getattr(_lib, fn_name)
    _check(fn_name, fn(_p(A), _p(B), _p(out), M, N, K, fmt_a, fmt_b, out_dtype, *extra, _p(sa), _p(sb), _p(ws),
                       ws.numel(), _stream()))
    return out, sa, sb


def snip_linear_fwd(X, W, fmt_x, fmt_w, out_dtype=OUT_BF16, *, out=None, ws=None, want_stats=False):
    M, K = X.shape
    N = W.shape[0]
    return _linear("snip_linear_fwd", X, W, (M, N), M, N, K, fmt_x, fmt_w, out_dtype, OP_FWD, out, ws, want_stats)


def snip_linear_dgrad(dY, W, fmt_dy, fmt_w, out_dtype=OUT_BF16, *, out=None, ws=None, want_stats=False):
    M, N = dY.shape
    K = W.shape[1]
    return _linear("snip_linear_dgrad", dY, W, (M, K), M, N, K, fmt_dy, fmt_w, out_dtype, OP_DGRAD, out, ws, want_stats)


def snip_linear_wgrad(dY, X, fmt_dy, fmt_x, out_dtype=OUT_BF16, accumulate=False, *, out=None, ws=None,
                      want_stats=False):
    M, N = dY.shape
    K = X.shape[1]
    return _linear("snip_linear_wgrad", dY, X, (N, K), M, N, K, fmt_dy, fmt_x, out_dtype, OP_WGRAD, out, ws,
                   want_stats, extra=(int(accumulate),))


def snip_linear_mx_workspace(op, M, N, K, fmt_a, fmt_b):
    w = ctypes.c_size_t()
    _check("snip_linear_mx_workspace", _lib.snip_linear_mx_workspace(op, M, N, K, fmt_a, fmt_b, ctypes.byref(w)))
    return w.value


def snip_linear_mx(op, A, B, fmt_a, fmt_b, out_dtype=OUT_BF16, *, out=None, ws=None, want_stats=False):
    """Power-of-two scale option.  op FWD: (X, W) -> Y; DGRAD: (dY, W) -> dX; WGRAD: (dY, X) -> dW."""
    if op == OP_FWD:
        (M, K), N = A.shape, B.shape[0]
        shape = (M, N)
    elif op == OP_DGRAD:
        (M, N), K = A.shape, B.shape[1]
        shape = (M, K)
    else:
        (M, N), K = A.shape, B.shape[1]
        shape = (N, K)
    out = _out(shape, out_dtype, A.device, out)
    if ws is None:
        ws = torch.zeros(snip_linear_mx_workspace(op, M, N, K, fmt_a, fmt_b), dtype=torch.uint8, device=A.device)
    sa = torch.empty(32, dtype=torch.uint8, device=A.device) if want_stats else None
    sb = torch.empty(32, dtype=torch.uint8, device=A.device) if want_stats else None
    _check("snip_linear_mx", _lib.snip_linear_mx(op, _p(A), _p(B), _p(out), M, N, K, fmt_a, fmt_b, out_dtype, _p(sa), _p(sb), _p(ws),
                                                 ws.numel(), _stream()))
    return out, sa, sb


def snip_linear_fwd_bwd_workspace(M, N, K, fmt_fwd, fmt_dgrad, fmt_wgrad, pow2_scale=False):
    n = ctypes.c_size_t()
    _check("snip_linear_fwd_bwd_workspace", _lib.snip_linear_fwd_bwd_workspace(M, N, K, fmt_fwd, fmt_dgrad, fmt_wgrad, int(pow2_scale),
                                                                               ctypes.byref(n)))
    return n.value


def snip_linear_fwd_bwd(x, w, dy, fmt_fwd, fmt_dgrad, fmt_wgrad, out_dtype=OUT_BF16, *, pow2_scale=False, dy_sr_seed=None, y=None,
                        dx=None, dw=None, stats=None, ws=None):
    """Forward and both gradients of one linear layer, each tensor read once.  Returns (y, dx, dw, stats)
    with stats a uint8 tensor holding six 24-byte snip_stats_t."""
    M, K = x.shape
    N = w.shape[0]
    dev = x.device
    y, dx, dw = _out((M, N), out_dtype, dev, y), _out((M, K), out_dtype, dev, dx), _out((N, K), out_dtype, dev, dw)
    if stats is None:
        stats = torch.zeros(6 * 24, dtype=torch.uint8, device=dev)
    if ws is None:
        ws = torch.zeros(snip_linear_fwd_bwd_workspace(M, N, K, fmt_fwd, fmt_dgrad, fmt_wgrad, pow2_scale), dtype=torch.uint8, device=dev)
    _check("snip_linear_fwd_bwd", _lib.snip_linear_fwd_bwd(_p(x), _p(w), _p(dy), _p(y), _p(dx), _p(dw), M, N, K, fmt_fwd, fmt_dgrad, fmt_wgrad,
                                                           out_dtype, int(pow2_scale), ROUND_NEAREST_EVEN if dy_sr_seed is None else ROUND_STOCHASTIC,
                                                           0 if dy_sr_seed is None else dy_sr_seed, _p(stats), _p(ws), ws.numel(), _stream()))
    return y, dx, dw, stats


def snip_linear_fwd_bwd_nvfp4(x, w, dy, bounds3, out_dtype=OUT_BF16, *, dy_sr_seed=None, stats=None, ws=None):
    """Forward and both gradients under the two-level option.  bounds3: float32 CUDA tensor [3] (bounds of |X|, |W|, |dY|).
    Returns (y, dx, dw, stats) with stats a uint8 tensor holding six 24-byte snip_stats_t."""
    M, K = x.shape
    N = w.shape[0]
    dev = x.device
    y, dx, dw = _out((M, N), out_dtype, dev, None), _out((M, K), out_dtype, dev, None), _out((N, K), out_dtype, dev, None)
    if stats is None:
        stats = torch.zeros(6 * 24, dtype=torch.uint8, device=dev)
    if ws is None:
        n = ctypes.c_size_t()
        _check("snip_linear_fwd_bwd_nvfp4_workspace", _lib.snip_linear_fwd_bwd_nvfp4_workspace(M, N, K, ctypes.byref(n)))
        ws = torch.zeros(n.value, dtype=torch.uint8, device=dev)
    _check("snip_linear_fwd_bwd_nvfp4", _lib.snip_linear_fwd_bwd_nvfp4(_p(x), _p(w), _p(dy), _p(y), _p(dx), _p(dw), M, N, K, out_dtype, _p(bounds3),
                                                                       ROUND_NEAREST_EVEN if dy_sr_seed is None else ROUND_STOCHASTIC,
                                                                       0 if dy_sr_seed is None else dy_sr_seed, _p(stats), _p(ws), ws.numel(), _stream()))
    return y, dx, dw, stats


def snip_layer_stats_workspace(M, N, K):
    w = ctypes.c_size_t()
    _check("snip_layer_stats_workspace", _lib.snip_layer_stats_workspace(M, N, K, ctypes.byref(w)))
    return w.value


def snip_layer_stats(X=None, W=None, Y=None, dY=None, dX=None, dW=None, *, M, N, K, fmt_mask=0b110, out=None, ws=None):
    """Returns a float64 CUDA tensor of 24 values: sumsq[6] then sumsq_err[3][2][3]."""
    dev = next(t for t in (X, W, Y, dY, dX, dW) if t is not None).device
    lt = LayerTensors(*[0 if t is None else t.data_ptr() for t in (X, W, Y, dY, dX, dW)], M, N, K)
    if out is None:
        out = torch.zeros(24, dtype=torch.float64, device=dev)
    if ws is None:
        ws = torch.empty(snip_layer_stats_workspace(M, N, K), dtype=torch.uint8, device=dev)
    _check("snip_layer_stats", _lib.snip_layer_stats(ctypes.byref(lt), fmt_mask, _p(out), _p(ws), ws.numel(), _stream()))
    return out


def snip_adamw_sensitivity(m: torch.Tensor, v: torch.Tensor, g: torch.Tensor, beta1: float, beta2: float, eps: float, *, out=None, ws=None):
    """Sum of T^2 (AdamW sensitivity term) over a parameter tensor; returns a 1-element float64 CUDA tensor."""
    assert m.dtype == torch.float32 and v.dtype == torch.float32 and g.dtype in (torch.bfloat16, torch.float32)
    assert m.is_contiguous() and v.is_contiguous() and g.is_contiguous() and m.numel() == v.numel() == g.numel()
    n = m.numel()
    if out is None:
        out = torch.zeros(1, dtype=torch.float64, device=m.device)
    if ws is None:
        w = ctypes.c_size_t()
        _check("snip_adamw_sensitivity_workspace", _lib.snip_adamw_sensitivity_workspace(n, ctypes.byref(w)))
        ws = torch.empty(w.value, dtype=torch.uint8, device=m.device)
    _check("snip_adamw_sensitivity", _lib.snip_adamw_sensitivity(_p(m), _p(v), _p(g), OUT_BF16 if g.dtype == torch.bfloat16 else OUT_FP32, n, beta1, beta2,
                                                                 eps, _p(out), _p(ws), ws.numel(), _stream()))
    return out


def snip_loss_divergence(grad_x_norm, err_x_norm, M, K, grad_w_norm, err_w_norm, N, loss) -> float:
    return float(_lib.snip_loss_divergence(grad_x_norm, err_x_norm, M, K, grad_w_norm, err_w_norm, N, loss))


def snip_weight_divergence(sens_norm, grad_err_norm, N, K, lr, beta1, beta2, step, weight_norm, num_layers) -> float:
    return float(_lib.snip_weight_divergence(sens_norm, grad_err_norm, N, K, lr, beta1, beta2, step, weight_norm, num_layers))


def snip_select_scheme(q, w, target: int, num_groups: int = 1):
    """q: m x n floats, w: m x n ints.  Returns (choice list, total loss, total work)."""
    import numpy as np
    qa = np.ascontiguousarray(np.asarray(q, dtype=np.float64))
    wa = np.ascontiguousarray(np.asarray(w, dtype=np.int64))
    m, n = qa.shape
    assert wa.shape == (m, n)
    choice = np.zeros(m, dtype=np.int32)
    qt, wt = ctypes.c_double(), ctypes.c_int64()
    _check("snip_select_scheme", _lib.snip_select_scheme(m, n, qa.ctypes.data_as(ctypes.c_void_p), wa.ctypes.data_as(ctypes.c_void_p), int(target),
                                                         num_groups, choice.ctypes.data_as(ctypes.c_void_p), ctypes.byref(qt), ctypes.byref(wt)))
    return [int(c) for c in choice], qt.value, wt.value


def snip_debug_set(key: int, value: int) -> None:
    """Testing hooks of the library (process-wide, off by default): see include/snip.h."""
    _check("snip_debug_set", _lib.snip_debug_set(key, value))


def snip_poll_status(ws: torch.Tensor) -> int:
    st = ctypes.c_int(0)
    _check("snip_poll_status", _lib.snip_poll_status(_p(ws), ctypes.byref(st)))
    return st.value
