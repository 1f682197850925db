"""Shared test plumbing: run the CUDA library on numpy inputs, compare with the oracle."""
import numpy as np

import oracle as orc

GUARD = 256          # sentinel bytes on each side of every output buffer
SENTINEL = 0xA5


def nan_code_mask(q: np.ndarray, elem: int) -> np.ndarray:
    m = q & 0x7F
    return (m == 0x7F) if elem == orc.E4M3 else (m > 0x7C)


def assert_q_equal(got: np.ndarray, want: np.ndarray, elem: int, what=""):
    """Bit-exact, except that any two NaN codes count as equal (several are valid)."""
    gn, wn = nan_code_mask(got, elem), nan_code_mask(want, elem)
    assert np.array_equal(gn, wn), "NaN positions differ " + what
    bad = (got != want) & ~gn
    if bad.any():
        idx = np.argwhere(bad)[:5]
        raise AssertionError("%d Q bytes differ %s; first at %s: got %s want %s" % (
            bad.sum(), what, idx.tolist(), got[bad][:5], want[bad][:5]))


def logical_scales_from_swizzled(buf: np.ndarray, mn: int, nkb: int) -> np.ndarray:
    """Gather the logical [mn, nkb] scale matrix out of a 128x4-atom buffer (oracle's formula)."""
    m_idx, k_idx = np.meshgrid(np.arange(mn), np.arange(nkb), indexing="ij")
    atoms_k = (nkb + 3) // 4
    off = ((m_idx // 128) * atoms_k + k_idx // 4) * 512 + (m_idx % 32) * 16 + ((m_idx % 128) // 32) * 4 + k_idx % 4
    assert off[-1, -1] == orc.sf_offset_swizzled(mn - 1, nkb - 1, nkb)
    assert off[mn // 2, nkb // 2] == orc.sf_offset_swizzled(mn // 2, nkb // 2, nkb)
    return buf[off]


def swizzled_pad_mask(mn: int, nkb: int) -> np.ndarray:
    size = ((mn + 127) // 128) * ((nkb + 3) // 4) * 512
    used = np.zeros(size, dtype=bool)
    m_idx, k_idx = np.meshgrid(np.arange(mn), np.arange(nkb), indexing="ij")
    atoms_k = (nkb + 3) // 4
    off = ((m_idx // 128) * atoms_k + k_idx // 4) * 512 + (m_idx % 32) * 16 + ((m_idx % 128) // 32) * 4 + k_idx % 4
    used[off.reshape(-1)] = True
    return ~used


class Guarded:
    """A device byte buffer with sentinel bands before and after the payload."""

    def __init__(self, nbytes: int, device="cuda"):
        import torch
        self.n = nbytes
        self.buf = torch.full((nbytes + 2 * GUARD,), SENTINEL, dtype=torch.uint8, device=device)
        self.view = self.buf[GUARD:GUARD + nbytes]

    def check(self, what=""):
        b = self.buf.cpu().numpy()
        assert (b[:GUARD] == SENTINEL).all() and (b[GUARD + self.n:] == SENTINEL).all(), "guard band overwritten " + what

    def numpy(self):
        return self.view.cpu().numpy()


def gpu_quantize(src_np, dtype: str, orientation: int, rule: int, elem: int, sf_layout: int):
    """src_np: float32 array (dtype 'fp32') or uint16 bf16 bit patterns (dtype 'bf16').
    Returns dict with 'q_row','s_row','q_col','s_col' numpy arrays (scales logical, linear
    shape) plus the raw swizzled buffers when sf_layout is swizzled."""
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = src_np.shape
    if dtype == "bf16":
        src = torch.from_numpy(src_np.view(np.int16)).cuda().view(torch.bfloat16)
    else:
        src = torch.from_numpy(src_np).cuda()
    bufs = {}
    args = []
    for o, name in ((B.ROW, "row"), (B.COL, "col")):
        if orientation & o:
            q = Guarded(rows * cols)
            s = Guarded(B.mxfp8_scale_bytes(rows, cols, o, sf_layout))
            bufs[name] = (q, s)
            args += [q.view.view(rows, cols), s.view]
        else:
            args += [None, None]
    B.mxfp8_quantize(src, orientation, rule, elem, args[0], args[1], args[2], args[3], sf_layout)
    torch.cuda.synchronize()
    out = {}
    for name, (q, s) in bufs.items():
        q.check("q_" + name)
        s.check("s_" + name)
        raw_q = q.numpy().reshape(rows, cols)
        if orc.code_bits(elem) < 8:
            # 6- and 4-bit codes come in packed 16-byte slots: padding must be zero, then compare code by code
            pad_from = 12 if orc.code_bits(elem) == 6 else 8
            assert not raw_q.reshape(rows, cols // 16, 16)[:, :, pad_from:].any(), "slot padding must be 0"
            out["packed_q_" + name] = raw_q
            raw_q = orc.unpack_codes16(raw_q, elem)
        out["q_" + name] = raw_q
        raw = s.numpy()
        if name == "row":
            mn, nkb = rows, cols // 32
        else:
            mn, nkb = cols, rows // 32
        if sf_layout == B.SF_SWIZZLED:
            out["raw_s_" + name] = raw
            logical = logical_scales_from_swizzled(raw, mn, nkb)
            assert (raw[swizzled_pad_mask(mn, nkb)] == 0).all(), "pad bytes must be 0"
        else:
            logical = raw.reshape(rows, cols // 32) if name == "row" else raw.reshape(rows // 32, cols).T
        out["s_" + name] = logical if name == "row" else np.ascontiguousarray(logical.T)
    return out


def check_against_oracle(src_np, dtype, orientation, rule, elem, sf_layout, what=""):
    from paper_2506_08027_b200 import binding as B
    x = orc.bf16_bits_to_f32(src_np) if dtype == "bf16" else src_np
    got = gpu_quantize(src_np, dtype, orientation, rule, elem, sf_layout)
    for o, name in ((B.ROW, "row"), (B.COL, "col")):
        if orientation & o:
            wq, ws = orc.quantize(x, orc.ROW if o == B.ROW else orc.COL, rule, elem)
            assert np.array_equal(got["s_" + name], ws), "scale bytes differ (%s) %s" % (name, what)
            assert_q_equal(got["q_" + name], wq, elem, "(%s) %s" % (name, what))
    return got


def swizzle_np(s_logical: np.ndarray) -> np.ndarray:
    """Vectorised form of oracle.swizzle_scales (checked against it in the CPU tests)."""
    mn, nkb = s_logical.shape
    out = np.zeros(((mn + 127) // 128) * ((nkb + 3) // 4) * 512, dtype=np.uint8)
    m_idx, k_idx = np.meshgrid(np.arange(mn), np.arange(nkb), indexing="ij")
    atoms_k = (nkb + 3) // 4
    off = ((m_idx // 128) * atoms_k + k_idx // 4) * 512 + (m_idx % 32) * 16 + ((m_idx % 128) // 32) * 4 + k_idx % 4
    out[off.reshape(-1)] = s_logical.reshape(-1)
    return out


def gpu_gemm(aq, a_s, bq, b_s, a_major="k", b_major="k", a_elem=0, b_elem=0, out="fp32"):
    """aq/bq: uint8 arrays as stored ([MN,K] for 'k', [K,MN] for 'mn'); a_s/b_s: linear scale
    arrays as the oracle returns them for that storage.  Returns D as numpy (float32, or
    uint16 bf16 bit patterns)."""
    import torch
    from paper_2506_08027_b200 import binding as B
    if a_major == "k":
        M, K = aq.shape
        sa_log = a_s
    else:
        K, M = aq.shape
        sa_log = np.ascontiguousarray(a_s.T)
    if b_major == "k":
        N, _ = bq.shape
        sb_log = b_s
    else:
        _, N = bq.shape
        sb_log = np.ascontiguousarray(b_s.T)
    dA, dB = torch.from_numpy(np.ascontiguousarray(aq)).cuda(), torch.from_numpy(np.ascontiguousarray(bq)).cuda()   # fancy-indexed inputs may be strided
    dSA, dSB = torch.from_numpy(swizzle_np(sa_log)).cuda(), torch.from_numpy(swizzle_np(sb_log)).cuda()
    D = torch.full((M, N), float("nan"), dtype=torch.float32 if out == "fp32" else torch.bfloat16, device="cuda")
    B.mxfp8_gemm(dA, dSA, dB, dSB, M, N, K, B.MN_MAJOR if a_major == "mn" else B.K_MAJOR,
                 B.MN_MAJOR if b_major == "mn" else B.K_MAJOR, a_elem, b_elem, D)
    assert B.mxfp8_device_status() == 0, "device status word reports a timeout"
    if out == "fp32":
        return D.cpu().numpy()
    return D.view(torch.int16).cpu().numpy().view(np.uint16)


def check_gemm_tolerance(d_gpu, d64, sabs, what=""):
    """The GEMM acceptance bounds: relative Frobenius error <= 1e-5 and every element within
    2^-16 * sum_k |a_k b_k| (plus an absolute floor of 2^-126 at the edge of the FP32 range)."""
    d = d_gpu.astype(np.float64)
    assert np.array_equal(np.isnan(d), np.isnan(d64)), "NaN positions differ " + what
    ok = ~np.isnan(d64)
    err = np.abs(d[ok] - d64[ok])
    bound = 2.0 ** -16 * sabs[ok] + 2.0 ** -126
    worst = float((err / bound).max()) if err.size else 0.0
    assert worst <= 1.0, "element bound exceeded %s: worst err/bound = %.3g" % (what, worst)
    fro = np.sqrt((err ** 2).sum()) / max(np.sqrt((d64[ok] ** 2).sum()), 1e-300)
    assert fro <= 1e-5, "relative Frobenius error %.3g %s" % (fro, what)
    return worst, fro
