"""GPU parity with circular shifts (desc.circular = 1): the operator T_k of the paper's Section 3 taken
literally, i.e. a convolution with circular padding, its exact input gradient and the estimator of Eq. 6
with the same T_k.  Every element against the float64 oracle's circular mode, through the C ABI."""
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
    # B, Cin, Cout, H, W, r, K
    (1, 1, 1, 1, 1, 1, 3),            # one pixel: every shift is the identity
    (2, 3, 2, 2, 2, 3, 5),            # image smaller than the kernel: the shifts wrap around more than once
    (3, 5, 7, 9, 11, 5, 3),           # odd everything
    (4, 16, 16, 8, 8, 8, 3),
    (2, 4, 8, 6, 40, 6, 3),           # wider than one 32-pixel chunk: the halo of the second chunk wraps to column 0
    (5, 33, 65, 7, 35, 17, 3),
    (4, 64, 64, 12, 12, 16, 3),       # a layer the tensor-core kernels would take with zero padding
    (8, 64, 64, 10, 14, 24, 3),       # r > B: the probes are summed first, the circular shift then acts on the rebuilt activation
    (4, 16, 32, 16, 16, 8, 5),
    (6, 8, 8, 5, 9, 4, 1),            # pointwise kernel: nothing to shift
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES)
def test_circular_layer_all_elements(shape, dtype):
    B, Cin, Cout, H, W, r, K = shape
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype=dtype, seed=sum(shape) + 77, KH=K, KW=K, z="rademacher")
    tol = TOL[dtype]
    d = dev(lay)
    Y, S = xb.xconv_forward(d["X"], d["W"], d["Z"], circular=True)
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"], kernel_size=K, circular=True)
    dX = xb.xconv_dgrad(d["dY"], d["W"], circular=True)
    torch.cuda.synchronize()
    Yo, So, dWo, dXo = O.xconv_layer(lay["X"], lay["W"], lay["dY"], lay["Z"], circular=True)
    check("Y", host(Y), Yo, tol)
    check("sketch", host(S), So, TOL_SKETCH)
    check("dX", host(dX), dXo, tol)
    check("dW", host(dW), dWo, tol)
    # the contraction alone (Algorithm 1 backward step 4), from the oracle's own L rounded to the storage type
    Lr = inputs.round_to_storage(O.backprobe(So.astype(np.float32), lay["dY"]).astype(np.float32), dtype)
    dWc = xb.xconv_contract(xb.to_device(Lr, dtype), d["Z"], kernel_size=K, circular=True)
    check("dW (contraction alone)", host(dWc), O.wgrad_contract(Lr, lay["Z"], K, K, circular=True),
          1e-5 if dtype == "f32" else 1e-4)
    if H > 1 or W > 1:
        # and the two kinds of shift do differ on these inputs (a flag that did nothing would still pass the above
        # only if the oracle ignored it too)
        Yz, _ = xb.xconv_forward(d["X"], d["W"], d["Z"])
        assert K == 1 or O.rel_fro(host(Yz), Yo) > 10 * tol


def test_circular_estimate_recovers_the_exact_circular_gradient_with_an_orthogonal_basis():
    """r = Cin*N probing vectors with (1/r) Z Z^T = I: the estimate equals the exact weight gradient of the
    circularly padded convolution (the trace identity of Eq. 2-3 with the permutation T_k)."""
    B, Cin, Cout, H, W = 3, 2, 3, 4, 4
    r = Cin * H * W
    rng = np.random.default_rng(31)
    Q, _ = np.linalg.qr(rng.standard_normal((r, r)))
    Z = (np.sqrt(r) * Q).reshape(r, Cin, H, W).astype(np.float32)
    X = rng.standard_normal((B, Cin, H, W)).astype(np.float32)
    dY = rng.standard_normal((B, Cout, H, W)).astype(np.float32)
    S = xb.xconv_sketch(xb.to_device(X, "f32"), xb.to_device(Z, "f32"))
    dW = xb.xconv_wgrad(S, xb.to_device(dY, "f32"), xb.to_device(Z, "f32"), circular=True)
    torch.cuda.synchronize()
    exact = O.dw_exact(X, dY, circular=True)
    assert O.rel_fro(host(dW), exact) < 1e-5
    assert O.rel_fro(host(dW), O.dw_exact(X, dY)) > 1e-2          # not the zero-padded gradient


def test_circular_shifts_per_channel_pair():
    B, Cin, Cout, H, W, r = 4, 6, 5, 7, 9, 8
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype="f32", seed=123, z="rademacher")
    d = dev(lay)
    S = xb.xconv_sketch_independent(d["X"], d["Z"])
    dW = xb.xconv_wgrad_independent(S, d["dY"], d["Z"], circular=True)
    torch.cuda.synchronize()
    So = O.sketch_independent(lay["X"], lay["Z"])
    check("dW (per pair, circular)", host(dW), O.wgrad_estimate_independent(So, lay["dY"], lay["Z"], circular=True), 1e-5)


def test_circular_shifts_over_volumes_are_refused():
    desc = xb.make_desc(2, 4, 4, 6, 6, 4, torch.float32, D=3, KD=3, circular=True)
    assert xb.workspace_bytes(desc, xb.OP_WGRAD) == 0
    assert xb.engine_for(desc, xb.OP_CONTRACT) == "none"


def _draw_case(seed):
    g = np.random.Generator(np.random.PCG64(seed))
    dtype = ["f32", "bf16", "f16"][int(g.integers(0, 3))]
    K = [1, 3, 3, 5][int(g.integers(0, 4))]
    chans = [1, 3, 8, 16, 24, 32, 40, 64, 96, 128]
    Cin, Cout = int(g.choice(chans)), int(g.choice(chans))
    H, W = int(g.integers(1, 15)), int(g.integers(1, 41))
    B, r = int(g.integers(1, 25)), int(g.integers(1, 41))
    return dict(dtype=dtype, K=K, Cin=Cin, Cout=Cout, H=H, W=W, B=B, r=r)


@pytest.mark.parametrize("seed", range(48))
def test_random_circular_layer(seed):
    """Seeded random planar layers with circular shifts: every storage type and kernel size, channel counts on and off
    the tensor-core tiles (the flag must take those layers off them), batch above and below the probe count, images
    narrower than the kernel and wider than a 32-pixel chunk; stored and redrawn probes."""
    c = _draw_case(31000 + seed)
    dtype, K = c["dtype"], c["K"]
    B, Cin, Cout, H, W, r = c["B"], c["Cin"], c["Cout"], c["H"], c["W"], c["r"]
    note = str(c)
    lay = dict(X=inputs.draw("relu", (B, Cin, H, W), seed * 10 + 40, dtype),
               W=inputs.draw("normal", (Cout, Cin, K, K), seed * 10 + 41, dtype, (2.0 / (Cin * K * K)) ** 0.5),
               dY=inputs.draw("normal", (B, Cout, H, W), seed * 10 + 42, dtype, 0.1 if dtype == "f16" else 1.0),
               Z=inputs.draw(["rademacher", "gaussian"][seed % 2], (r, Cin, H, W), seed * 10 + 43, dtype))
    d = {k: xb.to_device(v, dtype) for k, v in lay.items()}
    tol = TOL[dtype]
    Y, S = xb.xconv_forward(d["X"], d["W"], d["Z"], circular=True)
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"], kernel_size=K, circular=True)
    dX = xb.xconv_dgrad(d["dY"], d["W"], circular=True)
    torch.cuda.synchronize()
    So = O.sketch(lay["X"], lay["Z"])
    check("sketch " + note, host(S), So, TOL_SKETCH)
    check("Y " + note, host(Y), O.conv_forward(lay["X"], lay["W"], circular=True), tol)
    check("dX " + note, host(dX), O.dx_exact(lay["dY"], lay["W"], circular=True), tol)
    dWo = O.wgrad_estimate(So, lay["dY"], lay["Z"], K, K, circular=True)
    check("dW " + note, host(dW), dWo, tol)
    # the paper's order through the two halves, whatever order xconv_wgrad took
    L = xb.xconv_backprobe(torch.from_numpy(So.astype(np.float32)).cuda(), d["dY"])
    check("dW (halves) " + note, host(xb.xconv_contract(L, d["Z"], kernel_size=K, circular=True)), dWo, tol)
    # probes redrawn from a seed
    zseed = 910000 + seed
    Zo = O.rademacher_probes(zseed, r, Cin, H, W)
    Ss = xb.xconv_sketch_seeded(d["X"], zseed, r)
    dWs = xb.xconv_wgrad_seeded(Ss, d["dY"], zseed, Cin, kernel_size=K, circular=True)
    check("seeded dW " + note, host(dWs), O.wgrad_estimate(host(Ss), lay["dY"], Zo, K, K, circular=True), tol)
