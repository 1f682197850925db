"""mxfp8_rmsnorm_quantize_static: the RMS-normalisation + conversion call whose row statistics live in a fixed
array inside the library, so that it needs no scratch from the caller and allocates nothing."""
import numpy as np
import pytest

from paper_2506_08027_b200 import synth


def test_symbols_are_declared_and_exported():
    import os
    import re
    here = os.path.dirname(os.path.abspath(__file__))
    header = open(os.path.join(here, "..", "include", "mxfp8.h")).read()
    assert re.search(r"\bmxfp8_rmsnorm_quantize_static\s*\(", header)
    assert re.search(r"\bmxfp8_rmsnorm_quantize_static_max_rows\s*\(", header)
    from paper_2506_08027_b200 import binding as B
    assert "mxfp8_rmsnorm_quantize_static" in B.EXPORTS
    lib = B.lib()
    assert hasattr(lib, "mxfp8_rmsnorm_quantize_static") and B.mxfp8_rmsnorm_quantize_static_max_rows() == 65536


def _inputs(rows, cols, seed):
    import torch
    x = synth.device_tensor("activation", (rows, cols), seed)
    gamma = (1.0 + 0.1 * torch.randn(cols, generator=torch.Generator().manual_seed(seed))).to(torch.bfloat16).cuda()
    return x, gamma


@pytest.mark.gpu
@pytest.mark.parametrize("shape", [(256, 512), (160, 352), (65536, 32)])
def test_same_result_as_the_call_with_a_caller_buffer(shape):
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = shape
    x, gamma = _inputs(rows, cols, 5)
    a = B.alloc_quantize_outputs(rows, cols, B.BOTH, B.SF_SWIZZLED)
    b = B.alloc_quantize_outputs(rows, cols, B.BOTH, B.SF_SWIZZLED)
    for t in a + b:
        t.zero_()
    rstd = torch.empty(rows, dtype=torch.float32, device="cuda")
    B.mxfp8_rmsnorm_quantize(x, gamma, 1e-5, rstd, B.BOTH, B.RULE_PAPER, B.E4M3, *a, B.SF_SWIZZLED)
    B.mxfp8_rmsnorm_quantize_static(x, gamma, 1e-5, B.BOTH, B.RULE_PAPER, B.E4M3, *b, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    for u, v in zip(a, b):
        assert torch.equal(u, v)


@pytest.mark.gpu
def test_allocates_nothing_on_host_or_device():
    import ctypes
    import torch
    from paper_2506_08027_b200 import binding as B

    class Mallinfo2(ctypes.Structure):        # glibc: bytes in use by the C heap are `uordblks`
        _fields_ = [(n, ctypes.c_size_t) for n in ("arena", "ordblks", "smblks", "hblks", "hblkhd", "usmblks", "fsmblks",
                                                    "uordblks", "fordblks", "keepcost")]
    libc = ctypes.CDLL(None)
    libc.mallinfo2.restype = Mallinfo2
    lib = B.lib()
    rows, cols = 4096, 2048
    x, gamma = _inputs(rows, cols, 6)
    outs = B.alloc_quantize_outputs(rows, cols, B.BOTH, B.SF_SWIZZLED)
    # first call: module load and the one-time address lookup
    B.mxfp8_rmsnorm_quantize_static(x, gamma, 1e-5, B.BOTH, B.RULE_PAPER, B.E4M3, *outs, B.SF_SWIZZLED)
    torch.cuda.synchronize()
    stats0 = torch.cuda.memory_stats()
    unchanged = False
    for _ in range(3):          # the free-memory figure is device-wide: repeat if something else moved it meanwhile
        free0, _ = torch.cuda.mem_get_info()
        for _ in range(20):
            B.mxfp8_rmsnorm_quantize_static(x, gamma, 1e-5, B.BOTH, B.RULE_PAPER, B.E4M3, *outs, B.SF_SWIZZLED)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        if free1 == free0:
            unchanged = True
            break
    assert unchanged, "device memory in use changed across the calls"
    stats1 = torch.cuda.memory_stats()
    assert stats1["allocation.all.allocated"] == stats0["allocation.all.allocated"]
    assert stats1["allocated_bytes.all.current"] == stats0["allocated_bytes.all.current"]
    # the host side: the C heap of this process around 20 calls made straight through the C ABI (arguments
    # marshalled beforehand, so that nothing of Python's runs between the two readings but the foreign calls)
    args = (x.data_ptr(), B.BF16, rows, cols, gamma.data_ptr(), ctypes.c_float(1e-5), B.BOTH, B.RULE_PAPER, B.E4M3,
            outs[0].data_ptr(), outs[1].data_ptr(), outs[2].data_ptr(), outs[3].data_ptr(), B.SF_SWIZZLED, None)
    call = lib.mxfp8_rmsnorm_quantize_static
    assert call(*args) == 0
    grew = []
    for _ in range(3):
        before = libc.mallinfo2().uordblks
        rc = [call(*args) for _ in range(20)]
        grew.append(libc.mallinfo2().uordblks - before)
        assert not any(rc)
    torch.cuda.synchronize()
    # the list of 20 return codes is Python's own (a few hundred bytes at most): a buffer of any size that the
    # library allocated and kept per call would show far above that
    assert max(grew) < 4096, grew


@pytest.mark.gpu
def test_rejects_more_rows_than_the_array_holds():
    import torch
    from paper_2506_08027_b200 import binding as B
    rows, cols = 65536 + 32, 32
    x, gamma = _inputs(rows, cols, 7)
    outs = B.alloc_quantize_outputs(rows, cols, B.ROW, B.SF_LINEAR)
    for t in outs[:2]:
        t.fill_(0xA5)
    with pytest.raises(B.Mxfp8Error) as e:
        B.mxfp8_rmsnorm_quantize_static(x, gamma, 1e-5, B.ROW, B.RULE_PAPER, B.E4M3, *outs, B.SF_LINEAR)
    assert e.value.status == -5
    torch.cuda.synchronize()
    assert (outs[0] == 0xA5).all() and (outs[1] == 0xA5).all()      # nothing was launched
