"""GPU parity of the estimator applied to each channel pair on its own ("independent" probing: first sentence of
the multi-channel case, Section 3): per-channel sketch and crosstalk-free estimate against the oracle."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from oracle import xconv_oracle as O
from paper_2106_06998_b200 import binding as xb
from paper_2106_06998_b200 import inputs
from tests._util import TOL, TOL_SKETCH, check, dev, host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    entry.build()
    torch.cuda.set_device(0)


SHAPES = [
    # dtype, (B, Cin, Cout, H, W, r), K
    ("f32", (3, 5, 7, 9, 11, 5), 3),           # odd everything
    ("f32", (1, 1, 1, 1, 1, 1), 3),
    ("f32", (8, 16, 32, 32, 32, 32), 5),       # the CIFAR-10 network's second layer (5 x 5), r = 32 as in Section 5.5
    ("bf16", (8, 32, 32, 16, 16, 32), 5),      # its third layer; the contraction over the batch runs on tcgen05
    ("bf16", (16, 64, 128, 12, 20, 24), 3),
    ("f16", (16, 64, 64, 12, 12, 40), 3),
    ("bf16", (9, 40, 24, 7, 9, 13), 3),        # channel counts off every tile, odd batch
    ("f32", (12, 70, 8, 6, 6, 9), 1),          # pointwise kernel, channels beyond two 32-lane blocks
]


@pytest.mark.parametrize("dtype,shape,K", SHAPES)
def test_independent_probing_matches_the_oracle(dtype, shape, K):
    B, Cin, Cout, H, W, r = shape
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype=dtype, seed=sum(shape) + 3, KH=K, KW=K, z="gaussian", x="relu")
    if dtype == "f16":
        lay["dY"] = inputs.round_to_storage(lay["dY"] * np.float32(0.1), "f16")
    d = dev(lay)
    S = xb.xconv_sketch_independent(d["X"], d["Z"])
    So = O.sketch_independent(lay["X"], lay["Z"])
    check("per-channel sketch", host(S), So, TOL_SKETCH)
    dW = xb.xconv_wgrad_independent(S, d["dY"], d["Z"], kernel_size=K)
    dWo = O.wgrad_estimate_independent(So, lay["dY"], lay["Z"], K, K)
    check("dW (independent)", host(dW), dWo, TOL[dtype])
    # the estimator alone, fed the oracle's sketch rounded to float
    dW2 = xb.xconv_wgrad_independent(torch.from_numpy(So.astype(np.float32)).cuda(), d["dY"], d["Z"], kernel_size=K)
    check("dW (independent, oracle sketch in)", host(dW2), dWo, TOL[dtype])
    # summed over the channels the per-channel sketch is the multi-channel one
    check("sum over channels", host(S).sum(axis=1), O.sketch(lay["X"], lay["Z"]), TOL_SKETCH)


def test_independent_probing_with_an_orthogonal_basis_per_channel_is_exact_on_gpu():
    Cin, H, W, N = 3, 4, 4, 16
    lay = inputs.make_custom(4, Cin, 5, H, W, N, dtype="f32", seed=8)
    g = np.random.Generator(np.random.PCG64(2))
    lay["Z"] = np.stack([np.sqrt(N) * np.linalg.qr(g.standard_normal((N, N)))[0].T.reshape(N, H, W)
                         for _ in range(Cin)], axis=1).astype(np.float32)
    d = dev(lay)
    dW = xb.xconv_wgrad_independent(xb.xconv_sketch_independent(d["X"], d["Z"]), d["dY"], d["Z"])
    check("exact recovery", host(dW), O.dw_exact(lay["X"], lay["dY"]), 1e-5)
