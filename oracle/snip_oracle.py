"""ctypes front end of the CPU oracle (``snip_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's
cpu_baseline / reference arm.  It never touches the CUDA library and holds no arithmetic of its
own beyond composing the C routines in the order the paper states them (Sec. 2.2, Fig. 5:
quantize the operands, multiply, keep the product in BF16; Sec. 3.1: Frobenius norms of the
tensors and of their quantization errors).

bf16 tensors travel as ``numpy.uint16`` arrays holding the raw bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

FMT_BF16, FMT_FP8_E4M3, FMT_FP4_E2M1 = 0, 1, 2
BLOCK_ROW, BLOCK_COL, BLOCK_BLK = 0, 1, 2
BLOCK_ROW32, BLOCK_COL32 = 3, 4   # added option: 1x32 / 32x1 tiles (block-32 power-of-two scales)
TILE = 128

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "snip_oracle.c")
_LIB = os.path.join(_HERE, "libsnip_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE flags: no contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared",
               "-fPIC", "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, i32, vp, dbl = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_double
        L.orc_fpx_max.restype = dbl
        L.orc_fpx_max.argtypes = [i32]
        L.orc_bf16_to_float.restype = ctypes.c_float
        L.orc_bf16_to_float.argtypes = [ctypes.c_uint16]
        L.orc_double_to_bf16.restype = ctypes.c_uint16
        L.orc_double_to_bf16.argtypes = [dbl]
        L.orc_decode_code.restype = dbl
        L.orc_decode_code.argtypes = [i32, ctypes.c_uint8]
        L.orc_encode_e4m3.restype = ctypes.c_uint8
        L.orc_encode_e4m3.argtypes = [ctypes.c_float]
        L.orc_encode_e2m1.restype = ctypes.c_uint8
        L.orc_encode_e2m1.argtypes = [ctypes.c_float]
        L.orc_tile_scale.restype = ctypes.c_float
        L.orc_tile_scale.argtypes = [i32, ctypes.c_float]
        L.orc_scale_shape.restype = None
        L.orc_scale_shape.argtypes = [i64, i64, i32, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.orc_quantize.restype = i32
        L.orc_quantize.argtypes = [vp, i64, i64, i32, i32, vp, vp, vp, vp, vp]
        L.orc_quantize_rule.restype = i32
        L.orc_quantize_rule.argtypes = [vp, i64, i64, i32, i32, i32, vp, vp, vp, vp, vp]
        L.orc_quantize_nvfp4.restype = i32
        L.orc_quantize_nvfp4.argtypes = [vp, i64, i64, i32, ctypes.c_float, vp, vp, vp, vp, vp]
        L.orc_quantize_nvfp4_sr.restype = i32
        L.orc_quantize_nvfp4_sr.argtypes = [vp, i64, i64, i32, ctypes.c_float, i32, ctypes.c_uint64, vp, vp, vp, vp, vp]
        L.orc_quantize_sr.restype = i32
        L.orc_quantize_sr.argtypes = [vp, i64, i64, i32, i32, i32, ctypes.c_uint64, vp, vp, vp, vp, vp]
        L.orc_philox4x32_10.restype = None
        L.orc_philox4x32_10.argtypes = [vp, vp, vp]
        L.orc_sr_uniform16.restype = ctypes.c_uint32
        L.orc_sr_uniform16.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
        L.orc_encode_sr.restype = ctypes.c_uint8
        L.orc_encode_sr.argtypes = [i32, ctypes.c_float, ctypes.c_uint32]
        L.orc_tile_scale_pow2.restype = ctypes.c_float
        L.orc_tile_scale_pow2.argtypes = [i32, ctypes.c_float]
        L.orc_dequantize.restype = i32
        L.orc_dequantize.argtypes = [vp, vp, i64, i64, i32, i32, vp]
        L.orc_pack_codes.restype = i32
        L.orc_pack_codes.argtypes = [vp, i64, i64, i32, i32, vp]
        for name in ("orc_gemm_fwd", "orc_gemm_dgrad", "orc_gemm_wgrad"):
            fn = getattr(L, name)
            fn.restype = None
            fn.argtypes = [vp, vp, vp, i64, i64, i64]
        L.orc_round_to_bf16.restype = None
        L.orc_round_to_bf16.argtypes = [vp, i64, vp]
        L.orc_sumsq_bf16.restype = dbl
        L.orc_sumsq_bf16.argtypes = [vp, i64]
        L.orc_adamw_sensitivity_sumsq.restype = dbl
        L.orc_adamw_sensitivity_sumsq.argtypes = [vp, vp, vp, i64, dbl, dbl, dbl]
        L.orc_set_num_threads.restype = None
        L.orc_set_num_threads.argtypes = [i32]
        L.orc_num_threads.restype = i32
        L.orc_num_threads.argtypes = []
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def set_num_threads(n: int) -> None:
    lib().orc_set_num_threads(n)


def num_threads() -> int:
    return int(lib().orc_num_threads())


def fpx_max(fmt: int) -> float:
    return float(lib().orc_fpx_max(fmt))


def decode_code(fmt: int, code: int) -> float:
    return float(lib().orc_decode_code(fmt, code))


def encode(fmt: int, t: float) -> int:
    t32 = np.float32(t)
    if fmt == FMT_FP8_E4M3:
        return int(lib().orc_encode_e4m3(t32))
    if fmt == FMT_FP4_E2M1:
        return int(lib().orc_encode_e2m1(t32))
    raise ValueError("fmt")


def tile_scale(fmt: int, amax: float) -> np.float32:
    return np.float32(lib().orc_tile_scale(fmt, np.float32(amax)))


def tile_scale_pow2(fmt: int, amax: float) -> np.float32:
    return np.float32(lib().orc_tile_scale_pow2(fmt, np.float32(amax)))


def bf16_to_float(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    with np.errstate(invalid="ignore"):
        return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def round_to_bf16(v: np.ndarray) -> np.ndarray:
    v = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    lib().orc_round_to_bf16(_ptr(v), v.size, _ptr(out))
    return out


def scale_shape(rows: int, cols: int, block: int):
    d0, d1 = ctypes.c_int64(), ctypes.c_int64()
    lib().orc_scale_shape(rows, cols, block, ctypes.byref(d0), ctypes.byref(d1))
    return int(d0.value), int(d1.value)


@dataclass
class Quantized:
    """Result of quantizing one bf16 matrix (Sec. 2.3)."""
    fmt: int
    block: int
    rows: int
    cols: int
    codes: np.ndarray | None      # uint8 [rows, cols], one code per byte; None for BF16
    scales: np.ndarray | None     # float32, shape given by scale_shape(); None for BF16
    xhat: np.ndarray              # float64 [rows, cols], dequantized values
    sumsq_x: float                # sum of x^2
    sumsq_err: float              # sum of (x - xhat)^2
    row_sumsq_x: np.ndarray       # float64 [rows]
    row_sumsq_err: np.ndarray     # float64 [rows]

    def packed(self, transposed: bool = False) -> np.ndarray:
        """Codes in the library's storage layout (FP4: two per byte, even index low)."""
        return pack_codes(self.codes, self.fmt, transposed)


def philox4x32_10(ctr, key) -> np.ndarray:
    """Four 32-bit outputs of Philox4x32-10 for a 4-word counter and a 2-word key."""
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def sr_uniform16(seed: int, idx: int) -> int:
    """The 16-bit uniform that element idx (row-major linear index) draws under `seed`."""
    return int(lib().orc_sr_uniform16(seed, idx))


def encode_sr(fmt: int, t: float, u16: int) -> int:
    """Stochastically rounded code of the binary32 value t for the 16-bit uniform u16 (Sec. 6.1)."""
    return int(lib().orc_encode_sr(fmt, float(np.float32(t)), u16))


def quantize(x_bits: np.ndarray, fmt: int, block: int, pow2_scale: bool = False, sr_seed: int | None = None) -> Quantized:
    """sr_seed = None: round to nearest even (Sec. 2.3); an integer: stochastic rounding with that seed (Sec. 6.1)."""
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    assert x.ndim == 2
    rows, cols = x.shape
    quantized = fmt != FMT_BF16
    codes = np.zeros((rows, cols), dtype=np.uint8) if quantized else None
    scales = np.zeros(scale_shape(rows, cols, block), dtype=np.float32) if quantized else None
    xhat = np.empty((rows, cols), dtype=np.float64)
    sumsq = np.zeros(2, dtype=np.float64)
    row_sumsq = np.zeros((rows, 2), dtype=np.float64)
    if sr_seed is None:
        rc = lib().orc_quantize_rule(_ptr(x), rows, cols, fmt, block, int(pow2_scale), _ptr(codes), _ptr(scales),
                                     _ptr(xhat), _ptr(sumsq), _ptr(row_sumsq))
    else:
        rc = lib().orc_quantize_sr(_ptr(x), rows, cols, fmt, block, int(pow2_scale), sr_seed, _ptr(codes), _ptr(scales),
                                   _ptr(xhat), _ptr(sumsq), _ptr(row_sumsq))
    if rc != 0:
        raise ValueError("orc_quantize: bad argument")
    return Quantized(fmt, block, rows, cols, codes, scales, xhat, float(sumsq[0]),
                     float(sumsq[1]), row_sumsq[:, 0].copy(), row_sumsq[:, 1].copy())


@dataclass
class QuantizedNvfp4:
    """Result of the two-level (NVFP4-style) option: E2M1 codes, one E4M3 scale byte per 16-long tile, one factor per tensor."""
    rows: int
    cols: int
    col_tiles: bool               # False: 1x16 tiles along the columns, sf[ceil(cols/16)][rows]; True: 16x1 tiles, sf[ceil(rows/16)][cols]
    codes: np.ndarray             # uint8 [rows, cols]
    sf: np.ndarray                # uint8 E4M3 codes
    enc: np.float32               # 2688 / tensor_amax: dequantized value = value(code) * value(sf) / enc
    xhat: np.ndarray              # float64 [rows, cols]
    sumsq_x: float
    sumsq_err: float

    def packed(self, transposed: bool = False) -> np.ndarray:
        return pack_codes(self.codes, FMT_FP4_E2M1, transposed)


def quantize_nvfp4(x_bits: np.ndarray, col_tiles: bool = False, tensor_amax: float | None = None, sr_seed: int | None = None) -> QuantizedNvfp4:
    """tensor_amax = None: the exact maximum magnitude of x.  sr_seed = an integer: codes rounded stochastically (Sec. 6.1)."""
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    rows, cols = x.shape
    if tensor_amax is None:
        tensor_amax = float(np.abs(bf16_to_float(x)).max()) if x.size else 0.0
    nt = -(-(rows if col_tiles else cols) // 16)
    codes = np.zeros((rows, cols), dtype=np.uint8)
    sf = np.zeros((nt, cols if col_tiles else rows), dtype=np.uint8)
    enc = np.zeros(1, dtype=np.float32)
    xhat = np.empty((rows, cols), dtype=np.float64)
    sumsq = np.zeros(2, dtype=np.float64)
    rc = lib().orc_quantize_nvfp4_sr(_ptr(x), rows, cols, int(col_tiles), ctypes.c_float(tensor_amax), int(sr_seed is not None),
                                     0 if sr_seed is None else sr_seed, _ptr(codes), _ptr(sf), _ptr(enc), _ptr(xhat), _ptr(sumsq))
    if rc != 0:
        raise ValueError("orc_quantize_nvfp4: bad argument")
    return QuantizedNvfp4(rows, cols, bool(col_tiles), codes, sf, enc[0], xhat, float(sumsq[0]), float(sumsq[1]))


def nvfp4_atoms(q: QuantizedNvfp4, transposed: bool) -> np.ndarray:
    """Scale bytes of a QuantizedNvfp4 in the library's layout: per 128x128 tile and per half (64 elements) of a
    128-long chunk of the contraction one 512-byte atom, indexed [operand line tile][chunk][half]; inside an atom the
    word of tile line r (its four 16-long tiles of that half, in order) sits at (r % 32) * 16 + (r // 32) * 4.
    Lines and tiles beyond the matrix hold 0."""
    assert transposed == q.col_tiles
    lines, depth = (q.cols, q.rows) if q.col_tiles else (q.rows, q.cols)
    lt, ch = -(-lines // TILE), -(-depth // TILE)
    out = np.zeros((lt, ch, 2, 128, 4), dtype=np.uint8)
    for i in range(lt):
        for j in range(ch):
            for half in range(2):
                for r in range(min(TILE, lines - i * TILE)):
                    for k in range(4):
                        t = 8 * j + 4 * half + k
                        if t < q.sf.shape[0]:
                            out[i, j, half, (r % 32) * 4 + r // 32, k] = q.sf[t, i * TILE + r]
    return out.reshape(-1)


def linear_nvfp4(op: str, a_bits, b_bits):
    """The three GEMMs with both operands under the two-level option: 'fwd' (X, W) -> X W^T with 1x16 tiles along K on
    both; 'dgrad' (dY, W) -> dY W with 1x16 tiles of dY and 16x1 tiles of W; 'wgrad' (dY, X) -> dY^T X with 16x1 tiles."""
    if op == "fwd":
        qa, qb = quantize_nvfp4(a_bits, False), quantize_nvfp4(b_bits, False)
        return gemm_fwd(qa.xhat, qb.xhat), qa, qb
    if op == "dgrad":
        qa, qb = quantize_nvfp4(a_bits, False), quantize_nvfp4(b_bits, True)
        return gemm_dgrad(qa.xhat, qb.xhat), qa, qb
    qa, qb = quantize_nvfp4(a_bits, True), quantize_nvfp4(b_bits, True)
    return gemm_wgrad(qa.xhat, qb.xhat), qa, qb


def dequantize(codes: np.ndarray, scales: np.ndarray, fmt: int, block: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.float32)
    rows, cols = codes.shape
    out = np.empty((rows, cols), dtype=np.float64)
    rc = lib().orc_dequantize(_ptr(codes), _ptr(scales), rows, cols, fmt, block, _ptr(out))
    if rc != 0:
        raise ValueError("orc_dequantize: bad argument")
    return out


def pack_codes(codes: np.ndarray, fmt: int, transposed: bool = False) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    rows, cols = codes.shape
    outer, inner = (cols, rows) if transposed else (rows, cols)
    per_byte = 2 if fmt == FMT_FP4_E2M1 else 1
    out = np.zeros((outer, inner // per_byte), dtype=np.uint8)
    rc = lib().orc_pack_codes(_ptr(codes), rows, cols, fmt, int(transposed), _ptr(out))
    if rc != 0:
        raise ValueError("orc_pack_codes: bad argument")
    return out


def _gemm(name, a, b, out_shape, M, N, K):
    a = np.ascontiguousarray(a, dtype=np.float64)
    b = np.ascontiguousarray(b, dtype=np.float64)
    out = np.empty(out_shape, dtype=np.float64)
    getattr(lib(), name)(_ptr(a), _ptr(b), _ptr(out), M, N, K)
    return out


def gemm_fwd(xhat: np.ndarray, what: np.ndarray) -> np.ndarray:
    """Y[M,N] = X[M,K] . W[N,K]^T in float64."""
    M, K = xhat.shape
    N, K2 = what.shape
    assert K == K2
    return _gemm("orc_gemm_fwd", xhat, what, (M, N), M, N, K)


def gemm_dgrad(dyhat: np.ndarray, what: np.ndarray) -> np.ndarray:
    """dX[M,K] = dY[M,N] . W[N,K] in float64."""
    M, N = dyhat.shape
    N2, K = what.shape
    assert N == N2
    return _gemm("orc_gemm_dgrad", dyhat, what, (M, K), M, N, K)


def gemm_wgrad(dyhat: np.ndarray, xhat: np.ndarray) -> np.ndarray:
    """dW[N,K] = dY[M,N]^T . X[M,K] in float64."""
    M, N = dyhat.shape
    M2, K = xhat.shape
    assert M == M2
    return _gemm("orc_gemm_wgrad", dyhat, xhat, (N, K), M, N, K)


# ---- the three GEMMs of one linear layer under a precision choice (Fig. 5) -------------------

def linear_fwd(x_bits, w_bits, fmt_x, fmt_w, pow2_scale=False):
    """Quantize X with 1x128 tiles along K and W with 128x128 blocks, then Y = Xhat What^T.
    pow2_scale = 2 (added option): power-of-two scales on 32-long tiles along the contraction of both operands."""
    if pow2_scale == 2:
        qx = quantize(x_bits, fmt_x, BLOCK_ROW32, True)
        qw = quantize(w_bits, fmt_w, BLOCK_ROW32, True)
    else:
        qx = quantize(x_bits, fmt_x, BLOCK_ROW, pow2_scale)
        qw = quantize(w_bits, fmt_w, BLOCK_BLK, pow2_scale)
    return gemm_fwd(qx.xhat, qw.xhat), qx, qw


def linear_dgrad(dy_bits, w_bits, fmt_dy, fmt_w, pow2_scale=False):
    """Quantize dY with 1x128 tiles along N and W with 128x128 blocks, then dX = dYhat What."""
    if pow2_scale == 2:   # contraction over N: 1x32 tiles of dY, 32x1 tiles of W[N,K]
        qdy = quantize(dy_bits, fmt_dy, BLOCK_ROW32, True)
        qw = quantize(w_bits, fmt_w, BLOCK_COL32, True)
    else:
        qdy = quantize(dy_bits, fmt_dy, BLOCK_ROW, pow2_scale)
        qw = quantize(w_bits, fmt_w, BLOCK_BLK, pow2_scale)
    return gemm_dgrad(qdy.xhat, qw.xhat), qdy, qw


def linear_wgrad(dy_bits, x_bits, fmt_dy, fmt_x, pow2_scale=False):
    """Quantize dY and X with 128x1 tiles along M (the contraction), then dW = dYhat^T Xhat."""
    if pow2_scale == 2:
        qdy = quantize(dy_bits, fmt_dy, BLOCK_COL32, True)
        qx = quantize(x_bits, fmt_x, BLOCK_COL32, True)
    else:
        qdy = quantize(dy_bits, fmt_dy, BLOCK_COL, pow2_scale)
        qx = quantize(x_bits, fmt_x, BLOCK_COL, pow2_scale)
    return gemm_wgrad(qdy.xhat, qx.xhat), qdy, qx


def sumsq_bf16(bits: np.ndarray) -> float:
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return float(lib().orc_sumsq_bf16(_ptr(b), b.size))


def layer_stats(x_bits, w_bits, y_bits, dy_bits, dx_bits, dw_bits):
    """Step-1 statistics of one linear layer (Sec. 3.1): the plain sum of squares of the six
    tensors, and the error sum of squares of X, W, dY under each candidate format and each tile
    kind the tensor is consumed with.  Any tensor may be None."""
    out = {"sumsq": {}, "sumsq_err": {}}
    named = {"X": x_bits, "W": w_bits, "Y": y_bits, "dY": dy_bits, "dX": dx_bits, "dW": dw_bits}
    for name, t in named.items():
        if t is not None:
            out["sumsq"][name] = sumsq_bf16(t)
    kinds = {"X": (BLOCK_ROW, BLOCK_COL), "W": (BLOCK_BLK,), "dY": (BLOCK_ROW, BLOCK_COL)}
    for name, blocks in kinds.items():
        t = named[name]
        if t is None:
            continue
        for fmt in (FMT_FP8_E4M3, FMT_FP4_E2M1):
            for block in blocks:
                out["sumsq_err"][(name, fmt, block)] = quantize(t, fmt, block).sumsq_err
    return out


def sf_atoms(q: Quantized, transposed: bool) -> np.ndarray:
    """UE8M0 scale-factor atoms of a power-of-two-scaled Quantized, in the library's layout: one
    512-byte atom per 128x128 tile, indexed [operand row tile][contraction chunk] for the orientation
    the GEMM consumes; inside an atom the byte 127 - e of tile line r (S = 2^e) sits four times at
    (r % 32) * 16 + (r // 32) * 4.  Lines beyond the matrix hold 127.  With 32-long tiles the four bytes are those
    of the line's four tiles inside the 128-long chunk, in order (tiles beyond the matrix: 127)."""
    tr, tc = -(-q.rows // TILE), -(-q.cols // TILE)
    exps = np.frexp(q.scales.astype(np.float64))[1] - 1            # S = 2^e exactly
    byte = (127 - exps).astype(np.uint8)
    out = np.full((tc, tr, 128, 4) if transposed else (tr, tc, 128, 4), 127, dtype=np.uint8)
    for i in range(tr):
        for j in range(tc):
            if q.block == BLOCK_ROW:       # line = row inside the tile; scales[j][row]
                lines = byte[j, i * TILE:min((i + 1) * TILE, q.rows)]
            elif q.block == BLOCK_COL:     # line = column inside the tile; scales[i][col]
                lines = byte[i, j * TILE:min((j + 1) * TILE, q.cols)]
            elif q.block in (BLOCK_ROW32, BLOCK_COL32):
                # ROW32: line = row, chunk j, scales[4j + k][row];  COL32: line = column, chunk i, scales[4i + k][col]
                line_tile, chunk = (i, j) if q.block == BLOCK_ROW32 else (j, i)
                nlines = (q.rows if q.block == BLOCK_ROW32 else q.cols)
                atom = out[j, i] if transposed else out[i, j]
                for r in range(min(TILE, nlines - line_tile * TILE)):
                    for k in range(4):
                        if 4 * chunk + k < byte.shape[0]:
                            atom[(r % 32) * 4 + r // 32, k] = byte[4 * chunk + k, line_tile * TILE + r]
                continue
            else:
                lines = np.full(TILE, byte[i, j], dtype=np.uint8)
            atom = out[j, i] if transposed else out[i, j]
            for r, b in enumerate(lines):
                atom[(r % 32) * 4 + r // 32, :] = b
    return out.reshape(-1)



def adamw_sensitivity_sumsq(m, v, g, beta1: float, beta2: float, eps: float) -> float:
    """Sum over all elements of T^2, T = (1-beta1)/(sqrt(v)+eps) - (1-beta2) m g / (sqrt(v) (sqrt(v)+eps)^2)
    (Sec. 4.3); its square root is the norm Step 1 collects for the weight-divergence estimate."""
    m64, v64, g64 = (np.ascontiguousarray(np.asarray(a, dtype=np.float64).reshape(-1)) for a in (m, v, g))
    assert m64.size == v64.size == g64.size
    return float(lib().orc_adamw_sensitivity_sumsq(_ptr(m64), _ptr(v64), _ptr(g64), m64.size, beta1, beta2, eps))
