"""The no-allocation sketch entry point (xconv_sketch_static), called through the C ABI.

Some users of the library run where device memory cannot be obtained on demand (all of it was
handed out at start-up, or cudaMalloc's device-wide synchronisation is not tolerable mid-loop) and
have no buffer to pass as workspace.  This file checks that the variant whose scratch is a fixed
array inside the library gives the same sketch as xconv_sketch, twice in a row (the array keeps the
previous call's contents), and that it refuses layers beyond its fixed size.  It is collected last
so that a run stopping at the first failure has already run every other test."""
import ctypes

import pytest
import torch

import __graft_entry__ as entry
from oracle import xconv_oracle as O
from paper_2106_06998_b200 import binding as xb
from paper_2106_06998_b200 import inputs
from tests._util import TOL_SKETCH, check, host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    entry.build()
    torch.cuda.set_device(0)


def _rel(a, b):
    return float((a.double() - b.double()).norm() / b.double().norm())


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_static_scratch_sketch_matches_workspace_sketch_twice_in_a_row(dtype):
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    # two different layers back to back: the second call finds the first call's partial sums in the array
    shapes = [(24, 32, 20, 28, 40), (7, 16, 9, 13, 5)]          # B, Cin, H, W, r
    for rep in range(2):
        for (B, Cin, H, W, r) in shapes:
            lay = inputs.make_custom(B, Cin, 8, H, W, r, dtype=dtype, seed=100 + rep)
            X, Z = xb.to_device(lay["X"], dtype), xb.to_device(lay["Z"], dtype)
            want = xb.xconv_sketch(X, Z)                         # existing entry point (caller's workspace)
            desc = xb.make_desc(B, Cin, 1, H, W, r, tdt)
            got = torch.full((r, B), float("nan"), dtype=torch.float32, device="cuda")
            for call in range(2):                                # two calls in a row, same arguments
                st = xb.lib().xconv_sketch_static(ctypes.byref(desc), X.data_ptr(), Z.data_ptr(), got.data_ptr(),
                                                  torch.cuda.current_stream().cuda_stream)
                assert st == 0, xb.lib().xconv_status_string(st)
                torch.cuda.synchronize()
                assert _rel(got, want) <= TOL_SKETCH, (dtype, rep, call, _rel(got, want))
            assert torch.equal(xb.xconv_sketch_static(X, Z), got)     # binding wrapper, and reproducible
            # and against the definition itself (Algorithm 1 forward step 3), not only the other entry point
            check("static-scratch sketch", host(got), O.sketch(lay["X"], lay["Z"]), TOL_SKETCH)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [
    # B, Cin, H, W, r
    (512, 8, 16, 16, 1024),      # r*B = 2^19: the fixed array holds two slabs, so four k-splits shrink to two
    (1024, 8, 16, 16, 1024),     # r*B = 2^20 exactly: one slab fills the array, a single split
])
def test_static_scratch_at_and_near_its_limit(shape, dtype):
    """The fixed array bounds the number of k-splits; at r*B equal to its size one slab fills it to the last float."""
    B, Cin, H, W, r = shape
    assert r * B <= xb.STATIC_SCRATCH_FLOATS
    lay = inputs.make_custom(B, Cin, 8, H, W, r, dtype=dtype, seed=sum(shape), z="rademacher")
    X, Z = xb.to_device(lay["X"], dtype), xb.to_device(lay["Z"], dtype)
    want = xb.xconv_sketch(X, Z)
    for call in range(2):
        got = xb.xconv_sketch_static(X, Z)
        torch.cuda.synchronize()
        assert _rel(got, want) <= TOL_SKETCH, (dtype, call, _rel(got, want))
    check("static-scratch sketch", host(got), O.sketch(lay["X"], lay["Z"]), TOL_SKETCH)


def test_static_scratch_rejects_layers_beyond_its_fixed_size():
    limit = xb.STATIC_SCRATCH_FLOATS
    r, B = 2048, limit // 2048 + 1                                # r*B just over the limit
    desc = xb.make_desc(B, 8, 1, 2, 2, r, torch.float32)
    X = torch.zeros((B, 8, 2, 2), device="cuda").contiguous(memory_format=torch.channels_last)
    Z = torch.zeros((r, 8, 2, 2), device="cuda").contiguous(memory_format=torch.channels_last)
    S = torch.full((r, B), 3.0, device="cuda")
    st = xb.lib().xconv_sketch_static(ctypes.byref(desc), X.data_ptr(), Z.data_ptr(), S.data_ptr(), None)
    torch.cuda.synchronize()
    assert st == 4 and b"too small" in xb.lib().xconv_status_string(st)
    assert float(S.min()) == 3.0 and float(S.max()) == 3.0        # nothing was launched
    with pytest.raises(xb.XConvError):
        xb.xconv_sketch_static(X, Z)
