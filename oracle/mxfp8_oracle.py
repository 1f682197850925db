"""ctypes/numpy front end of the CPU oracle -- TEST INFRASTRUCTURE, not the product.

The conversion arithmetic lives in ``mxfp8_oracle.c`` (scalar C, binary64); this file
marshals numpy arrays to it and adds the two pieces that are plain definitions on top
of it: the 128x4 scale-factor layout (an index permutation) and the block-scaled GEMM
(two binary64 matrix products over the decoded operands, Sec. 2 and App. A.3).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

E4M3, E5M2 = 0, 1
E2M3, E3M2, E2M1 = 3, 4, 5      # the 6- and 4-bit element formats of Table 1
RULE_PAPER, RULE_OCP = 0, 1
ROW, COL = 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mxfp8_oracle.c")
_SO = os.path.join(_HERE, "libmxfp8_oracle.so")
_lib = None
_lock = threading.Lock()


def build_oracle(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, no fast-math) if the library is stale."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build_oracle())
            c_i, c_i64, c_p = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p
            lib.orc_fp8_decode.restype = ctypes.c_double
            lib.orc_fp8_decode.argtypes = [c_i, c_i]
            lib.orc_fp8_encode.restype = c_i
            lib.orc_fp8_encode.argtypes = [ctypes.c_double, c_i]
            lib.orc_scale_byte.restype = c_i
            lib.orc_scale_byte.argtypes = [ctypes.c_float, c_i, c_i]
            lib.orc_quantize.restype = c_i
            lib.orc_quantize.argtypes = [c_p, c_i64, c_i64, c_i, c_i, c_i, c_p, c_p]
            lib.orc_dequantize.restype = c_i
            lib.orc_dequantize.argtypes = [c_p, c_p, c_i64, c_i64, c_i, c_i, c_p]
            lib.orc_round_to_f32.restype = None
            lib.orc_round_to_f32.argtypes = [c_p, c_i64, c_p]
            lib.orc_round_to_bf16.restype = None
            lib.orc_round_to_bf16.argtypes = [c_p, c_i64, c_p]
            _lib = lib
    return _lib


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def fp8_decode(code: int, elem: int = E4M3) -> float:
    """Value of one FP8 code (Table 1)."""
    return float(_load().orc_fp8_decode(int(code), elem))


def fp8_encode(x: float, elem: int = E4M3) -> int:
    """Quantize_to_fp8: RNE onto the element grid, saturating (Sec. 3.3, App. A.2)."""
    return int(_load().orc_fp8_encode(float(x), elem))


def scale_byte(amax, elem: int = E4M3, rule: int = RULE_PAPER) -> int:
    """UE8M0 byte of a block with this amax (Algorithm 1 / App. A.1, or the OCP rule)."""
    return int(_load().orc_scale_byte(np.float32(amax), elem, rule))


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float32."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def quantize(src: np.ndarray, orientation: int, rule: int = RULE_PAPER, elem: int = E4M3):
    """Convert a [rows, cols] float32 array to MXFP8.

    Returns (q, s): q uint8 [rows, cols]; s uint8 in the linear layout, [rows, cols/32]
    for ROW blocks and [rows/32, cols] for COL blocks.
    """
    src = np.ascontiguousarray(src, dtype=np.float32)
    rows, cols = src.shape
    q = np.empty((rows, cols), dtype=np.uint8)
    s = np.empty((rows, cols // 32) if orientation == ROW else (rows // 32, cols), dtype=np.uint8)
    rc = _load().orc_quantize(_ptr(src), rows, cols, orientation, rule, elem, _ptr(q), _ptr(s))
    if rc != 0:
        raise ValueError("blocked dimension is not a multiple of 32")
    return q, s


def quantize_threads(src: np.ndarray, orientation: int, rule: int, elem: int, threads: int):
    """The same conversion with row slabs handed to ``threads`` host threads.

    Blocks are independent, so slabs of whole 32-row groups give the same bytes; the C
    call releases the GIL.  Used by the benchmark's CPU-baseline leg only.
    """
    src = np.ascontiguousarray(src, dtype=np.float32)
    rows, cols = src.shape
    q = np.empty((rows, cols), dtype=np.uint8)
    s = np.empty((rows, cols // 32) if orientation == ROW else (rows // 32, cols), dtype=np.uint8)
    lib = _load()
    groups = rows // 32
    bounds = [32 * (groups * t // threads) for t in range(threads + 1)]
    bounds[-1] = rows

    def work(t):
        r0, r1 = bounds[t], bounds[t + 1]
        if r1 <= r0:
            return
        s0 = r0 if orientation == ROW else r0 // 32
        lib.orc_quantize(_ptr(src[r0:r1]), r1 - r0, cols, orientation, rule, elem,
                         _ptr(q[r0:r1]), _ptr(s[s0:]))

    ths = [threading.Thread(target=work, args=(t,)) for t in range(threads)]
    for t in ths:
        t.start()
    for t in ths:
        t.join()
    return q, s


def dequantize_f64(q: np.ndarray, s: np.ndarray, orientation: int, elem: int = E4M3) -> np.ndarray:
    """Decoded values Q*X as float64 (exact), Sec. 2."""
    q = np.ascontiguousarray(q, dtype=np.uint8)
    s = np.ascontiguousarray(s, dtype=np.uint8)
    rows, cols = q.shape
    out = np.empty((rows, cols), dtype=np.float64)
    rc = _load().orc_dequantize(_ptr(q), _ptr(s), rows, cols, orientation, elem, _ptr(out))
    if rc != 0:
        raise ValueError("blocked dimension is not a multiple of 32")
    return out


def dequantize(q, s, orientation: int, elem: int = E4M3, dst: str = "f32") -> np.ndarray:
    """Decoded values rounded (RNE, once) to float32, or to bfloat16 bit patterns (uint16)."""
    d = dequantize_f64(q, s, orientation, elem)
    if dst == "f32":
        out = np.empty(d.shape, dtype=np.float32)
        _load().orc_round_to_f32(_ptr(d), d.size, _ptr(out))
    elif dst == "bf16":
        out = np.empty(d.shape, dtype=np.uint16)
        _load().orc_round_to_bf16(_ptr(d), d.size, _ptr(out))
    else:
        raise ValueError(dst)
    return out


def sf_offset_swizzled(mn: int, kb: int, n_kblocks: int) -> int:
    """Byte offset of the scale of (row-or-column mn, K-block kb) in the 128x4 layout.

    The scale matrix, logically [MN, n_kblocks], is cut into atoms of 128 MN-indices by
    4 K-blocks, 512 bytes each, atoms ordered MN-major-outer / K-inner.  Inside an atom
    the byte of (mn, kb) sits at (mn % 32) * 16 + ((mn % 128) // 32) * 4 + kb % 4.
    """
    atoms_k = (n_kblocks + 3) // 4
    return ((mn // 128) * atoms_k + kb // 4) * 512 + (mn % 32) * 16 + ((mn % 128) // 32) * 4 + kb % 4


def swizzle_scales(s_logical: np.ndarray) -> np.ndarray:
    """Lay a logical [MN, n_kblocks] scale matrix out in the 128x4 layout (pad bytes 0)."""
    mn_n, nkb = s_logical.shape
    out = np.zeros(((mn_n + 127) // 128) * ((nkb + 3) // 4) * 512, dtype=np.uint8)
    for mn in range(mn_n):
        for kb in range(nkb):
            out[sf_offset_swizzled(mn, kb, nkb)] = s_logical[mn, kb]
    return out


def _operand_f64(q, s, major: str, elem: int) -> np.ndarray:
    """Logical [MN, K] float64 operand.  'k': stored [MN, K], ROW blocks, scales [MN, K/32].
    'mn': stored [K, MN], COL blocks (blocks run down K), scales [K/32, MN]."""
    if major == "k":
        return dequantize_f64(q, s, ROW, elem)
    return np.ascontiguousarray(dequantize_f64(q, s, COL, elem).T)


def gemm_f64(aq, a_s, bq, b_s, a_major: str = "k", b_major: str = "k",
             a_elem: int = E4M3, b_elem: int = E4M3):
    """Block-scaled product D[m,n] = sum_k A[m,k] * B[n,k] over the decoded operands.

    Each decoded element is Q*X with X a power of two, so every product of two of them
    is exact in binary64 and the block-wise application of the scales (Sec. 2, App. A.3)
    equals the plain product of the decoded matrices.  Returns (D, S) with
    S[m,n] = sum_k |A[m,k] * B[n,k]|, the magnitude sum the per-element bound uses.
    """
    a = _operand_f64(aq, a_s, a_major, a_elem)
    b = _operand_f64(bq, b_s, b_major, b_elem)
    with np.errstate(invalid="ignore", over="ignore"):
        d = a @ b.T
        sabs = np.abs(a) @ np.abs(b).T
    return d, sabs


def grouped_gemm_f64(aq, a_s, bq, b_s, offsets, mode: str = "m", b_major: str = "k",
                     a_elem: int = E4M3, b_elem: int = E4M3):
    """Per-expert block-scaled products of a mixture-of-experts layer (App. A.4 trains one with the
    same recipe: every expert's GEMMs are the products of Sec. 2 on that expert's tokens).

    `offsets` (length G+1, non-decreasing, multiples of 32) splits the token axis into G groups;
    group g owns tokens offsets[g] .. offsets[g+1]-1.

    mode "m" (fprop / dgrad): A stored [T, K] with ROW blocks; B holds the G expert matrices stacked:
        b_major "k":  stored [G*N, K], ROW blocks, expert g = rows g*N .. (g+1)*N-1
        b_major "mn": stored [G*K, N], COL blocks, expert g = rows g*K .. (g+1)*K-1
      D [T, N]: D[t, :] = A[t, :] . B_g^T for t in group g.
    mode "k" (wgrad): A stored [T, M] and B stored [T, N], both with COL blocks (blocks run down the
      token axis); D [G*M, N]: D_g = A_g^T . B_g summed over the tokens of group g (zeros for an
      empty group).
    Returns (D, S), S the matching sums of |a*b|.
    """
    offsets = [int(o) for o in offsets]
    G = len(offsets) - 1
    if mode == "m":
        a = dequantize_f64(aq, a_s, ROW, a_elem)
        T, K = a.shape
        if b_major == "k":
            b = dequantize_f64(bq, b_s, ROW, b_elem)
            N = b.shape[0] // G
            experts = [b[g * N:(g + 1) * N, :] for g in range(G)]
        else:
            b = dequantize_f64(bq, b_s, COL, b_elem)
            N = b.shape[1]
            experts = [b[g * K:(g + 1) * K, :].T for g in range(G)]
        d = np.zeros((T, N))
        sabs = np.zeros((T, N))
        with np.errstate(invalid="ignore", over="ignore"):
            for g in range(G):
                lo, hi = offsets[g], offsets[g + 1]
                d[lo:hi] = a[lo:hi] @ experts[g].T
                sabs[lo:hi] = np.abs(a[lo:hi]) @ np.abs(experts[g]).T
        return d, sabs
    if mode != "k":
        raise ValueError(mode)
    a = dequantize_f64(aq, a_s, COL, a_elem)
    b = dequantize_f64(bq, b_s, COL, b_elem)
    M, N = a.shape[1], b.shape[1]
    d = np.zeros((G * M, N))
    sabs = np.zeros((G * M, N))
    with np.errstate(invalid="ignore", over="ignore"):
        for g in range(G):
            lo, hi = offsets[g], offsets[g + 1]
            d[g * M:(g + 1) * M] = a[lo:hi].T @ b[lo:hi]
            sabs[g * M:(g + 1) * M] = np.abs(a[lo:hi]).T @ np.abs(b[lo:hi])
    return d, sabs


def concat_swizzled_scales_k(parts, mn: int, nkb_part: int) -> np.ndarray:
    """Swizzled scales of logical [mn, len(parts) * nkb_part] from the swizzled arrays of its parts, each logical
    [mn, nkb_part]: byte by byte through the layout's offset formula."""
    nkb = len(parts) * nkb_part
    out = np.zeros(((mn + 127) // 128) * ((nkb + 3) // 4) * 512, dtype=np.uint8)
    for r, part in enumerate(parts):
        for m in range(mn):
            for kb in range(nkb_part):
                out[sf_offset_swizzled(m, r * nkb_part + kb, nkb)] = part[sf_offset_swizzled(m, kb, nkb_part)]
    return out


def data_parallel_linear_f64(xs, w_shards, dys, rule: int = RULE_PAPER, elem: int = E4M3):
    """One linear-layer step (Sec. 3.2: FPROP, DGRAD and WGRAD on MXFP8 copies blocked along each product's
    reduction axis) when rank r holds tokens xs[r] [T_r, H] with output gradients dys[r] [T_r, F] and owns
    rows w_shards[r] [F_r, H] of the weight.  The paper states the single-device arithmetic only; sharded, it
    reads: every rank converts its own tensors (blocks never cross a shard: T_r and F_r are multiples of 32);
    the weight operand of every rank is the shards' conversions one under another; Y_r and dX_r use the rank's
    own tokens; dW sums the ranks' partial products over their tokens and rank r keeps its rows.

    Returns (ys, dxs, dw_shards, sabs) as lists per rank of float64 arrays; sabs = matching lists of |a*b| sums
    (for dW the sum over ranks)."""
    R, C = ROW, COL
    wq = {o: [quantize(w, o, rule, elem) for w in w_shards] for o in (R, C)}
    w_row = (np.concatenate([q for q, _ in wq[R]]), np.concatenate([sc for _, sc in wq[R]]))     # [F, H], [F, H/32]
    w_col = (np.concatenate([q for q, _ in wq[C]]), np.concatenate([sc for _, sc in wq[C]]))     # [F, H], [F/32, H]
    ys, dxs, s_y, s_dx = [], [], [], []
    dw = None
    s_dw = None
    for x, dy in zip(xs, dys):
        xq = {o: quantize(x, o, rule, elem) for o in (R, C)}
        dyq = {o: quantize(dy, o, rule, elem) for o in (R, C)}
        y, sy = gemm_f64(xq[R][0], xq[R][1], w_row[0], w_row[1], "k", "k", elem, elem)
        dx, sdx = gemm_f64(dyq[R][0], dyq[R][1], w_col[0], w_col[1], "k", "mn", elem, elem)
        part, spart = gemm_f64(dyq[C][0], dyq[C][1], xq[C][0], xq[C][1], "mn", "mn", elem, elem)
        ys.append(y); dxs.append(dx); s_y.append(sy); s_dx.append(sdx)
        dw = part if dw is None else dw + part
        s_dw = spart if s_dw is None else s_dw + spart
    bounds = np.cumsum([0] + [w.shape[0] for w in w_shards])
    dw_shards = [dw[bounds[r]:bounds[r + 1]] for r in range(len(w_shards))]
    s_dw_shards = [s_dw[bounds[r]:bounds[r + 1]] for r in range(len(w_shards))]
    return ys, dxs, dw_shards, (s_y, s_dx, s_dw_shards)


def code_bits(elem: int) -> int:
    return {E4M3: 8, E5M2: 8, E2M3: 6, E3M2: 6, E2M1: 4}[elem]


def pack_codes16(codes: np.ndarray, elem: int) -> np.ndarray:
    """Storage layout of 6- and 4-bit codes (Table 1's MXFP6 / MXFP4 elements) as the tensor cores
    read them: every 16 consecutive codes of a row become one 16-byte slot; code i of the slot
    occupies bits [w*i, w*i + w) of the slot read as a little-endian integer (w = 6 or 4), the
    remaining bytes are zero.  8-bit codes are returned unchanged.  `codes`: [rows, cols] uint8,
    one code per byte, cols a multiple of 16.  An index/bit permutation, no arithmetic."""
    w = code_bits(elem)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    if w == 8:
        return codes.copy()
    rows, cols = codes.shape
    if cols % 16:
        raise ValueError("packed slots need cols % 16 == 0")
    out = np.zeros((rows, cols), dtype=np.uint8)
    for r in range(rows):
        for g in range(cols // 16):
            slot = 0
            for i in range(16):
                slot |= int(codes[r, 16 * g + i]) << (w * i)
            out[r, 16 * g:16 * g + 16] = np.frombuffer(slot.to_bytes(16, "little"), dtype=np.uint8)
    return out


def unpack_codes16(packed: np.ndarray, elem: int) -> np.ndarray:
    """Inverse of pack_codes16 (padding bytes are ignored)."""
    w = code_bits(elem)
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    if w == 8:
        return packed.copy()
    rows, cols = packed.shape
    out = np.zeros((rows, cols), dtype=np.uint8)
    for r in range(rows):
        for g in range(cols // 16):
            slot = int.from_bytes(packed[r, 16 * g:16 * g + 16].tobytes(), "little")
            for i in range(16):
                out[r, 16 * g + i] = (slot >> (w * i)) & ((1 << w) - 1)
    return out


ACT_NONE, ACT_RELU, ACT_RELU2, ACT_SILU, ACT_GELU_TANH = 0, 1, 2, 3, 4


def activation(x: np.ndarray, act: int, dst: str = "f32") -> np.ndarray:
    """Elementwise activation ahead of the conversion (Sec. 3.2 keeps the activation function in high
    precision and converts its result): the function's plain definition in binary64, rounded once to
    binary32 and, for dst "bf16", once more to bfloat16 (returned as float32 values / uint16 patterns).
        relu: x > 0 ? x : 0 (NaN -> 0);  relu2: x > 0 ? x*x : 0;  silu: x / (1 + exp(-x));
        gelu_tanh: 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))
    """
    v = np.asarray(x, dtype=np.float64)
    with np.errstate(over="ignore", invalid="ignore"):
        if act == ACT_NONE:
            y = v.copy()
        elif act == ACT_RELU:
            y = np.where(v > 0, v, 0.0)
        elif act == ACT_RELU2:
            y = np.where(v > 0, v * v, 0.0)
        elif act == ACT_SILU:
            y = v / (1.0 + np.exp(-v))
        elif act == ACT_GELU_TANH:
            y = 0.5 * v * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (v + 0.044715 * v * v * v)))
        else:
            raise ValueError(act)
        y32 = y.astype(np.float32)
    if dst == "f32":
        return y32
    out = np.empty(y32.shape, dtype=np.uint16)
    y64 = np.ascontiguousarray(y32, dtype=np.float64)
    _load().orc_round_to_bf16(_ptr(y64), y64.size, _ptr(out))
    return out


def activation_grad(z: np.ndarray, dh: np.ndarray, act: int, dst: str = "f32") -> np.ndarray:
    """Backward of the elementwise activation ahead of the conversion: the gradient with respect to the activation's
    input, dz = act'(z) * dh, is an activation gradient and is converted like one (Sec. 3.2).  act'(z) is the plain
    derivative in binary64 rounded once to binary32; the product with dh is one binary32 operation; for dst "bf16"
    the result is rounded once more to bfloat16.
        relu': z > 0 ? 1 : 0;  relu2': z > 0 ? 2z : 0;  silu': s (1 + z (1 - s)) with s = 1 / (1 + exp(-z));
        gelu_tanh': 0.5 (1 + t) + 0.5 z (1 - t^2) sqrt(2/pi) (1 + 3 * 0.044715 z^2) with t = tanh(sqrt(2/pi) (z + 0.044715 z^3))
    """
    v = np.asarray(z, dtype=np.float64)
    g32 = np.ascontiguousarray(dh, dtype=np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        if act == ACT_NONE:
            d = np.ones_like(v)
        elif act == ACT_RELU:
            d = np.where(v > 0, 1.0, 0.0)
        elif act == ACT_RELU2:
            d = np.where(v > 0, 2.0 * v, 0.0)
        elif act == ACT_SILU:
            sg = 1.0 / (1.0 + np.exp(-v))
            d = sg * (1.0 + v * (1.0 - sg))
        elif act == ACT_GELU_TANH:
            c = np.sqrt(2.0 / np.pi)
            t = np.tanh(c * (v + 0.044715 * v * v * v))
            d = 0.5 * (1.0 + t) + 0.5 * v * (1.0 - t * t) * c * (1.0 + 3.0 * 0.044715 * v * v)
        else:
            raise ValueError(act)
        y32 = d.astype(np.float32) * g32          # one binary32 product
    if dst == "f32":
        return y32
    out = np.empty(y32.shape, dtype=np.uint16)
    y64 = np.ascontiguousarray(y32, dtype=np.float64)
    _load().orc_round_to_bf16(_ptr(y64), y64.size, _ptr(out))
    return out


def rmsnorm(x: np.ndarray, gamma: np.ndarray, eps: float, dst: str = "f32", rstd: np.ndarray | None = None):
    """RMS normalisation ahead of the conversion (Sec. 3.2 keeps normalisation in high precision and converts its
    output).  rstd[r] = 1 / sqrt(mean_c x[r,c]^2 + eps) in binary64, rounded to binary32 (or the `rstd` passed in, one
    binary32 value per row); y = (x * rstd) * gamma as two binary32 products in that order, rounded once more to
    bfloat16 for dst "bf16".  Returns (y, rstd): y as float32 values ("f32") or uint16 patterns ("bf16")."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    g32 = np.ascontiguousarray(gamma, dtype=np.float32)
    if rstd is None:
        v = x32.astype(np.float64)
        rstd = (1.0 / np.sqrt((v * v).mean(axis=1) + float(eps))).astype(np.float32)
    rstd = np.ascontiguousarray(rstd, dtype=np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        y32 = (x32 * rstd[:, None]) * g32[None, :]          # numpy float32 products are IEEE single operations
    if dst == "f32":
        return y32, rstd
    out = np.empty(y32.shape, dtype=np.uint16)
    y64 = np.ascontiguousarray(y32, dtype=np.float64)
    _load().orc_round_to_bf16(_ptr(y64), y64.size, _ptr(out))
    return out, rstd


def layernorm(x: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float, dst: str = "f32",
              mean: np.ndarray | None = None, rstd: np.ndarray | None = None):
    """Layer normalisation ahead of the conversion (Sec. 3.2 keeps normalisation in high precision and converts its
    output).  mean[r] = mean_c x[r,c] and rstd[r] = 1 / sqrt(mean_c (x[r,c] - mean[r])^2 + eps) in binary64, each
    rounded to binary32 (or the values passed in); y = ((x - mean) * rstd) * gamma + beta as binary32 operations in
    that order (a subtraction, two products, an addition: four roundings), rounded once more to bfloat16 for dst
    "bf16".  Returns (y, mean, rstd)."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    g32 = np.ascontiguousarray(gamma, dtype=np.float32)
    b32 = np.ascontiguousarray(beta, dtype=np.float32)
    v = x32.astype(np.float64)
    if mean is None:
        mean = v.mean(axis=1).astype(np.float32)
    mean = np.ascontiguousarray(mean, dtype=np.float32)
    if rstd is None:
        d = v - v.mean(axis=1)[:, None]
        rstd = (1.0 / np.sqrt((d * d).mean(axis=1) + float(eps))).astype(np.float32)
    rstd = np.ascontiguousarray(rstd, dtype=np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        y32 = ((x32 - mean[:, None]) * rstd[:, None]) * g32[None, :] + b32[None, :]   # numpy float32 operations are IEEE single operations
    if dst == "f32":
        return y32, mean, rstd
    out = np.empty(y32.shape, dtype=np.uint16)
    y64 = np.ascontiguousarray(y32, dtype=np.float64)
    _load().orc_round_to_bf16(_ptr(y64), y64.size, _ptr(out))
    return out, mean, rstd


def glu(x: np.ndarray, act: int, dst: str = "f32") -> np.ndarray:
    """Gated activation ahead of the conversion: x is [rows, 2*cols] = (gate | up); y = act(gate) * up, with act(gate)
    as in `activation` (binary64 definition rounded to binary32), then one binary32 product, then one rounding to
    bfloat16 for dst "bf16".  Returns [rows, cols] float32 values ("f32") or uint16 patterns ("bf16")."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    cols = x32.shape[1] // 2
    a = activation(x32[:, :cols], act, "f32")
    with np.errstate(over="ignore", invalid="ignore"):
        y32 = a * x32[:, cols:]                 # numpy float32 product: one IEEE single operation
    if dst == "f32":
        return y32
    out = np.empty(y32.shape, dtype=np.uint16)
    y64 = np.ascontiguousarray(y32, dtype=np.float64)
    _load().orc_round_to_bf16(_ptr(y64), y64.size, _ptr(out))
    return out
