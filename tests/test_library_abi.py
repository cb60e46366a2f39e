"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, sizes its workspace and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2106_06998_b200 import binding as xb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return xb.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "xconv.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(xconv_[a-z0-9_]+)\s*\(", header))
    assert declared == set(xb.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def _desc(**kw):
    base = dict(B=8, Cin=16, Cout=16, H=32, W=32, r=8, dtype=xb.XCONV_F32, K=3)
    base.update(kw)
    return xb.make_desc(**base)


def test_workspace_sizes_are_positive_and_monotone_in_r(lib):
    a = xb.workspace_bytes(_desc(r=8), xb.OP_WGRAD)
    b = xb.workspace_bytes(_desc(r=64), xb.OP_WGRAD)
    assert 0 < a < b
    assert xb.workspace_bytes(_desc(), xb.OP_SKETCH) > 0
    assert xb.workspace_bytes(_desc(), xb.OP_DGRAD) > 0
    assert xb.workspace_bytes(_desc(), 17) == 0


def test_invalid_descriptors_are_rejected(lib):
    assert xb.workspace_bytes(_desc(B=0), xb.OP_SKETCH) == 0
    assert xb.engine_for(_desc(r=-1), xb.OP_SKETCH) == "none"
    d = _desc(Cin=64, Cout=64, dtype=xb.XCONV_BF16)
    assert xb.engine_for(d, xb.OP_CONTRACT) == "tcgen05_bf16" and xb.engine_for(d, xb.OP_FORWARD) == "tcgen05_bf16"
    d.circular = 1                       # circular shifts are served for planar layers, by the FP32-FMA kernels ...
    assert xb.workspace_bytes(d, xb.OP_WGRAD) > 0
    assert xb.engine_for(d, xb.OP_CONTRACT) == "simt_f32" and xb.engine_for(d, xb.OP_FORWARD) == "simt_f32"
    assert xb.engine_for(d, xb.OP_SKETCH) == "tcgen05_bf16"       # the sketch shifts nothing
    d.D, d.KD, d.pad_d = 4, 3, 1         # ... not for volumes
    assert lib.xconv_sketch(ctypes.byref(d), 16, 16, 16, 16, 1 << 20, None) == 2
    d = _desc()
    d.circular = 2                       # a flag, not a count
    assert lib.xconv_sketch(ctypes.byref(d), 16, 16, 16, 16, 1 << 20, None) == 1
    d = _desc(K=7)                       # kernel sizes beyond 5 x 5 have no kernel
    assert lib.xconv_sketch(ctypes.byref(d), 16, 16, 16, 16, 1 << 20, None) == 2
    d = _desc()
    d.pad_h = 0                          # not a "same" convolution
    assert lib.xconv_wgrad(ctypes.byref(d), 16, 16, 16, 16, 16, 1 << 20, None) == 2
    d = _desc()
    d.dtype = 7
    assert lib.xconv_dgrad(ctypes.byref(d), 16, 16, 16, 16, 1 << 20, None) == 1


def test_null_misaligned_and_short_workspace_return_codes_without_launching(lib):
    d = _desc()
    need = xb.workspace_bytes(d, xb.OP_SKETCH)
    assert lib.xconv_sketch(None, 16, 16, 16, 16, need, None) == 1
    assert lib.xconv_sketch(ctypes.byref(d), None, 16, 16, 16, need, None) == 1
    assert lib.xconv_sketch(ctypes.byref(d), 16, 24, 16, 16, need, None) == 3      # 24 is not 16-aligned
    assert lib.xconv_sketch(ctypes.byref(d), 16, 16, 16, None, need, None) == 4
    assert lib.xconv_sketch(ctypes.byref(d), 16, 16, 16, 16, need - 1, None) == 4
    needw = xb.workspace_bytes(d, xb.OP_WGRAD)
    assert lib.xconv_wgrad(ctypes.byref(d), 16, 16, 16, 16, 16, needw - 1, None) == 4
    assert lib.xconv_forward(ctypes.byref(d), 16, 16, 16, 16, 16, 16, 0, None) == 4
    assert lib.xconv_sketch_wgrad_host(ctypes.byref(d), 16, 16, 16, 16, 16, 256, 10, None) == 4
    assert xb.host_arena_bytes(d) > need
    assert b"workspace" in lib.xconv_status_string(4)


def test_binding_refuses_host_tensors_and_wrong_layout(lib):
    import torch
    X = torch.zeros(2, 4, 5, 5)
    Z = torch.zeros(3, 4, 5, 5)
    with pytest.raises(ValueError):
        xb.xconv_sketch(X, Z)


def test_zero_block_mask_changes_the_plan_only_where_it_is_used(lib):
    """Host arithmetic only (the mask pointer is never followed): the contraction of wide 16-bit layers plans a list
    of non-zero probes behind its partial sums; everywhere else the field changes nothing."""
    def pair(**kw):
        plain = _desc(**kw)
        masked = _desc(**kw)
        masked.zero_blocks = 256
        return plain, masked
    plain, masked = pair(B=512, Cin=256, Cout=256, H=28, W=28, r=64, dtype=xb.XCONV_BF16)
    assert not xb.zero_blocks_used(plain) and xb.zero_blocks_used(masked)
    grown = xb.workspace_bytes(masked, xb.OP_WGRAD) - xb.workspace_bytes(plain, xb.OP_WGRAD)
    assert 4 * (64 + 2) <= grown <= 4 * (64 + 2) + 512          # one column tile: count, 64 entries, terminator
    plain, masked = pair(B=512, Cin=512, Cout=256, H=28, W=28, r=64, dtype=xb.XCONV_F16)
    assert xb.zero_blocks_used(masked)
    assert xb.workspace_bytes(masked, xb.OP_WGRAD) - xb.workspace_bytes(plain, xb.OP_WGRAD) >= 2 * 4 * (64 + 2)
    for kw in (dict(B=8, Cin=64, Cout=32, H=8, W=8, r=4, dtype=xb.XCONV_F32),           # FP32-FMA kernels
               dict(B=32, Cin=128, Cout=64, H=12, W=20, r=24, dtype=xb.XCONV_BF16),     # small 16-bit layer
               dict(B=8, Cin=96, Cout=64, H=16, W=16, r=8, dtype=xb.XCONV_BF16)):       # not whole 64-channel blocks
        plain, masked = pair(**kw)
        assert not xb.zero_blocks_used(masked)
        assert xb.workspace_bytes(masked, xb.OP_WGRAD) == xb.workspace_bytes(plain, xb.OP_WGRAD)
    # a planar kernel on a volume: the mask is per probing vector, the contraction walks planes
    plain, masked = pair(B=8, Cin=128, Cout=128, H=16, W=16, r=6, dtype=xb.XCONV_BF16, D=3, KD=1)
    assert not xb.zero_blocks_used(masked)
    plain, masked = pair(B=8, Cin=128, Cout=128, H=16, W=16, r=6, dtype=xb.XCONV_BF16, D=3, KD=3)
    assert xb.zero_blocks_used(masked)


def test_planning_survives_random_descriptors(lib):
    """Host arithmetic only: 3000 seeded random layers (odd sizes, all storage types, volumes, kernel sizes, with and
    without a zero-block mask) through every size and engine query -- no crash, no absurd size, and an engine
    answer for every layer that validates."""
    import numpy as np
    import torch
    g = np.random.Generator(np.random.PCG64(20210612))
    ops = [xb.OP_FORWARD, xb.OP_SKETCH, xb.OP_WGRAD, xb.OP_DGRAD, xb.OP_SKETCH_SEEDED, xb.OP_WGRAD_SEEDED]
    for _ in range(3000):
        B = int(g.choice([1, 2, 3, 8, 16, 17, 64, 100, 512, 1000]))
        Cin = int(g.choice([1, 3, 8, 16, 32, 48, 64, 96, 128, 192, 256, 320, 512, 1024]))
        Cout = int(g.choice([1, 3, 8, 16, 32, 48, 64, 96, 128, 192, 256, 320, 512]))
        H, W = (int(g.choice([1, 2, 3, 4, 7, 8, 14, 16, 28, 31, 32, 56, 64, 100, 256])) for _ in range(2))
        r = int(g.choice([1, 2, 5, 8, 16, 24, 64, 100, 256, 1000, 1024]))
        K = int(g.choice([1, 3, 5]))
        D = int(g.choice([1, 1, 1, 2, 3, 5]))
        KD = 3 if (K == 3 and g.random() < 0.3) else 1
        dt = [torch.float32, torch.bfloat16, torch.float16][int(g.integers(0, 3))]
        d = xb.make_desc(B, Cin, Cout, H, W, r, dt, K, D=D, KD=KD)
        if g.random() < 0.5:
            d.zero_blocks = 256                      # never followed on the host
        sizes = [xb.workspace_bytes(d, op) for op in ops]
        assert all(0 < s < (1 << 46) for s in sizes), (B, Cin, Cout, H, W, r, K, D, KD, sizes)
        assert all(xb.engine_for(d, op) != "none" for op in ops[:4])
        assert xb.zero_blocks_used(d) in (False, True)
