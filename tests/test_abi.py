"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header declares,
validates arguments, and refuses to compute without a device (there is no CPU fallback)."""
import ctypes
import os
import re

import pytest
import torch

from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import build as dma_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    dma_build.build()
    return dma.lib()


def test_header_symbols_are_exported(lib):
    text = open(os.path.join(ROOT, "include", "dma.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(dma_[a-z_0-9]+)\s*\(", text))
    assert {"dma_mask_build", "dma_attn_fwd", "dma_attn_bwd", "dma_query_workspace"} <= names
    for n in names:
        assert hasattr(lib, n), n
    assert names == set(dma.ENTRY_POINTS)


def test_struct_layout_matches_header():
    # 12 four-byte fields then four int64[3] arrays
    assert ctypes.sizeof(dma.dma_problem_t) == 12 * 4 + 4 * 24
    assert dma.dma_problem_t.q_stride.offset == 48


def test_argument_validation(lib):
    ok = dma.problem(1, 4, 2, 256, 64, 32)
    assert dma.dma_query_workspace(ok)[0] > 256
    assert dma.dma_bitmap_words(ok) == 4 * 2 * 1
    for bad, code in ((dma.problem(1, 3, 2, 256, 64, 32), -2), (dma.problem(1, 4, 2, 0, 64, 32), -2),
                      (dma.problem(1, 4, 2, 256, 64, 0), -2), (dma.problem(1, 4, 2, 256, 96, 32), -4),
                      (dma.problem(1, 4, 2, 256, 64, 32, causal=2), -4), (dma.problem(1, 4, 2, 256, 64, 32, tile_m=64), -2)):
        with pytest.raises(dma.DmaError) as e:
            dma.dma_query_workspace(bad)
        assert e.value.status == code
    s = dma.problem(1, 4, 2, 256, 64, 32)
    s.q_stride[0], s.q_stride[1], s.q_stride[2] = 256 * 4 * 64, 4 * 64 + 4, 64       # stride not a multiple of 8
    with pytest.raises(dma.DmaError) as e:
        dma.dma_query_workspace(s)
    assert e.value.status == -3
    # NULL pointers and a short workspace are refused before anything touches a device
    z = ctypes.c_void_p(0)
    assert lib.dma_mask_build(ctypes.byref(ok), z, z, z, z, z, z, z, ctypes.c_size_t(0), z) == -1
    assert lib.dma_attn_fwd(ctypes.byref(ok), z, z, z, z, z, z, z, z, z, ctypes.c_size_t(0), z) == -1
    assert lib.dma_attn_bwd(ctypes.byref(ok), *([z] * 15), ctypes.c_size_t(0), z) == -1
    a = ctypes.c_void_p(4096)
    assert lib.dma_mask_build(ctypes.byref(ok), a, a, a, a, a, a, z, ctypes.c_size_t(0), z) == -5
    assert lib.dma_mask_build(ctypes.byref(ok), ctypes.c_void_p(4100), a, a, a, a, a, a, ctypes.c_size_t(1 << 30), z) == -3
    assert "workspace" in dma.dma_strerror(-5)


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device behaviour")
def test_no_cpu_fallback(lib):
    ok = dma.problem(1, 4, 2, 256, 64, 32)
    a = ctypes.c_void_p(4096)
    assert lib.dma_mask_build(ctypes.byref(ok), a, a, a, a, a, a, a, ctypes.c_size_t(1 << 30), ctypes.c_void_p(0)) == -6
    assert lib.dma_attn_fwd(ctypes.byref(ok), *([a] * 9), ctypes.c_size_t(1 << 30), ctypes.c_void_p(0)) == -6


def test_binding_refuses_tensors_of_another_element_type():
    # the library would read them with the problem's element size; the binding stops that before any call
    p = dma.problem(1, 2, 2, 8, 64, 4, dtype=dma.DMA_FP32)
    assert p.dtype == dma.DMA_FP32 and dma.problem(1, 2, 2, 8, 64, 4).dtype == dma.DMA_BF16
    V = torch.zeros(1, 8, 2, 64, dtype=torch.bfloat16)
    with pytest.raises(TypeError):
        dma.dma_mask_build(p, V, None, None)
    with pytest.raises(TypeError):
        dma.dma_attn_fwd(p, V, V, V, None, None, None)
    with pytest.raises(TypeError):
        dma.problem(1, 2, 2, 8, 64, 4, dtype=torch.float16)
