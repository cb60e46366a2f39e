"""GPU parity on volumes (three-dimensional layers, Section 5.5's 3-D segmentation network): 3 x 3 x 3 kernels
and planar kernels applied plane by plane, against the oracle's volume functions."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from oracle import xconv_oracle as O
from paper_2106_06998_b200 import binding as xb
from paper_2106_06998_b200 import inputs
from tests._util import TOL, TOL_SKETCH, check, host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    entry.build()
    torch.cuda.set_device(0)


def _volume_layer(B, Cin, Cout, D, H, W, r, KD, K, dtype, seed):
    dy_scale = 0.1 if dtype == "f16" else 1.0
    return dict(X=inputs.draw("relu", (B, Cin, D, H, W), seed * 10, dtype),
                W=inputs.draw("normal", (Cout, Cin, KD, K, K), seed * 10 + 1, dtype, (2.0 / (Cin * KD * K * K)) ** 0.5),
                dY=inputs.draw("normal", (B, Cout, D, H, W), seed * 10 + 2, dtype, dy_scale),
                Z=inputs.draw("rademacher", (r, Cin, D, H, W), seed * 10 + 3, dtype))


SHAPES = [
    # dtype, (B, Cin, Cout, D, H, W, r), KD, K
    ("f32", (2, 3, 4, 3, 5, 4, 5), 3, 3),             # odd everything
    ("f32", (1, 1, 1, 1, 1, 1, 1), 3, 3),             # a single voxel: only the centre weight sees data
    ("f32", (3, 16, 8, 4, 6, 6, 6), 3, 3),
    ("bf16", (4, 32, 32, 4, 8, 8, 8), 3, 3),          # tcgen05 throughout: planes moved by the depth offset, 32-channel groups
    ("bf16", (2, 64, 128, 6, 12, 12, 16), 3, 3),      # tcgen05, 27 offsets, r > B (contraction over image planes)
    ("f16", (6, 64, 64, 3, 10, 7, 4), 3, 3),          # tcgen05, r < B (contraction over probe planes), ragged patches
    ("bf16", (3, 64, 64, 1, 9, 9, 8), 3, 3),          # a volume one plane deep: two thirds of the offsets see only padding
    ("bf16", (8, 64, 64, 3, 6, 12, 16), 1, 3),        # planar kernel on every plane: tcgen05 throughout
    ("f16", (8, 64, 32, 2, 8, 8, 24), 1, 3),          # the same with r > B
    ("bf16", (4, 32, 16, 5, 6, 6, 12), 3, 3),         # r > B on a volume
    ("f32", (2, 6, 5, 3, 4, 5, 4), 1, 1),             # pointwise kernel
    ("f32", (2, 5, 4, 2, 4, 4, 3), 1, 5),             # 5 x 5 planar kernel on a volume
]


@pytest.mark.parametrize("dtype,shape,KD,K", SHAPES)
def test_volume_layers_match_the_oracle(dtype, shape, KD, K):
    B, Cin, Cout, D, H, W, r = shape
    lay = _volume_layer(B, Cin, Cout, D, H, W, r, KD, K, dtype, seed=sum(shape) + KD)
    tol = TOL[dtype]
    if dtype != "f32" and Cin % 32 == 0 and Cout % 32 == 0:
        desc = xb.make_desc(B, Cin, Cout, H, W, r, {"bf16": torch.bfloat16, "f16": torch.float16}[dtype], K, D=D, KD=KD)
        tc = "tcgen05_" + dtype
        assert xb.engine_for(desc, xb.OP_CONTRACT) == tc and xb.engine_for(desc, xb.OP_FORWARD) == tc
    d = {k: xb.to_device(v, dtype) for k, v in lay.items()}
    Y, S = xb.xconv_forward(d["X"], d["W"], d["Z"])
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"], kernel_size=K, kernel_depth=KD)
    dX = xb.xconv_dgrad(d["dY"], d["W"])
    torch.cuda.synchronize()
    So = O.sketch(lay["X"], lay["Z"])
    check("sketch", host(S), So, TOL_SKETCH)
    check("Y", host(Y), O.conv_forward3d(lay["X"], lay["W"]), tol)
    check("dX", host(dX), O.dx_exact3d(lay["dY"], lay["W"]), tol)
    dWo = O.wgrad_estimate3d(So, lay["dY"], lay["Z"], (KD, K, K))
    check("dW", host(dW), dWo, tol)
    # the two halves in the paper's order, fed the oracle's sketch
    So32 = So.astype(np.float32)
    L = xb.xconv_backprobe(torch.from_numpy(So32).cuda(), d["dY"])
    Lo = O.backprobe(So32, lay["dY"])
    check("L", host(L), Lo, tol)
    Lr = inputs.round_to_storage(Lo.astype(np.float32), dtype)
    dWc = xb.xconv_contract(xb.to_device(Lr, dtype), d["Z"], kernel_size=K, kernel_depth=KD)
    check("dW (contraction alone)", host(dWc), O.wgrad_contract3d(Lr, lay["Z"], (KD, K, K)), 1e-5 if dtype == "f32" else 1e-4)


def test_volume_with_depth_one_equals_the_planar_layer():
    lay = inputs.make_custom(4, 8, 8, 6, 7, 5, dtype="f32", seed=91)
    d4 = {k: xb.to_device(lay[k], "f32") for k in ("X", "W", "dY", "Z")}
    d5 = {k: xb.to_device(lay[k][:, :, None], "f32") for k in ("X", "W", "dY", "Z")}
    Y4, S4 = xb.xconv_forward(d4["X"], d4["W"], d4["Z"])
    Y5, S5 = xb.xconv_forward(d5["X"], d5["W"], d5["Z"])
    assert torch.equal(S4, S5) and torch.equal(Y4, Y5[:, :, 0])
    assert torch.equal(xb.xconv_wgrad(S4, d4["dY"], d4["Z"]), xb.xconv_wgrad(S5, d5["dY"], d5["Z"])[:, :, 0])


def test_independent_probing_on_a_volume():
    B, Cin, Cout, D, H, W, r = 4, 6, 5, 3, 4, 5, 7
    lay = _volume_layer(B, Cin, Cout, D, H, W, r, 3, 3, "f32", seed=17)
    d = {k: xb.to_device(v, "f32") for k, v in lay.items()}
    S = xb.xconv_sketch_independent(d["X"], d["Z"])
    So = np.stack([O.sketch(lay["X"][:, n:n + 1], lay["Z"][:, n:n + 1]) for n in range(Cin)], axis=1)
    check("per-channel sketch", host(S), So, TOL_SKETCH)
    dW = xb.xconv_wgrad_independent(S, d["dY"], d["Z"], kernel_size=3, kernel_depth=3)
    want = np.concatenate([O.wgrad_estimate3d(So[:, n, :], lay["dY"], lay["Z"][:, n:n + 1]) for n in range(Cin)], axis=1)
    check("dW (independent, volume)", host(dW), want, TOL["f32"])


@pytest.mark.parametrize("seed", range(24))
def test_random_medium_volumes(seed):
    """Seeded random volumes on the tensor-core tiles (depth 2-6, planar and 3 x 3 x 3 kernels, both orders of
    summation), every entry point, stored and redrawn probes."""
    g = np.random.Generator(np.random.PCG64(120000 + seed))
    dtype = ["bf16", "f16"][int(g.integers(0, 2))]
    D, KD = int(g.choice([2, 3, 4, 6])), int(g.choice([1, 3]))
    Cin, Cout = int(g.choice([32, 64, 96])), int(g.choice([32, 64, 128]))
    H, W = int(g.integers(5, 17)), int(g.integers(5, 17))
    B, r = int(g.integers(1, 7)), int(g.choice([4, 8, 12, 24, 40]))
    note = str(dict(dtype=dtype, D=D, KD=KD, Cin=Cin, Cout=Cout, H=H, W=W, B=B, r=r))
    X = inputs.draw("relu", (B, Cin, D, H, W), seed * 7 + 1, dtype)
    Wt = inputs.draw("normal", (Cout, Cin, KD, 3, 3), seed * 7 + 2, dtype, (2.0 / (Cin * KD * 9)) ** 0.5)
    dY = inputs.draw("normal", (B, Cout, D, H, W), seed * 7 + 3, dtype, 0.1 if dtype == "f16" else 1.0)
    zseed = 5 + seed
    Zo = O.rademacher_probes(zseed, r, Cin, D * H, W).reshape(r, Cin, D, H, W)      # numbered like an image of D*H rows
    d = {k: xb.to_device(v, dtype) for k, v in dict(X=X, W=Wt, dY=dY).items()}
    Zg = xb.xconv_probes_from_seed(zseed, r, Cin, H, W, d["X"].dtype, D=D)
    assert np.array_equal(host(Zg), Zo)
    Y, S = xb.xconv_forward(d["X"], d["W"], Zg)
    check("S " + note, host(S), O.sketch(X, Zo), TOL_SKETCH)
    check("Y " + note, host(Y), O.conv_forward3d(X, Wt), TOL[dtype])
    check("dX " + note, host(xb.xconv_dgrad(d["dY"], d["W"])), O.dx_exact3d(dY, Wt), TOL[dtype])
    dW = xb.xconv_wgrad(S, d["dY"], Zg, kernel_depth=KD)
    check("dW " + note, host(dW), O.wgrad_estimate3d(host(S), dY, Zo, (KD, 3, 3)), TOL[dtype])
    assert torch.equal(dW, xb.xconv_wgrad_seeded(S, d["dY"], zseed, Cin, kernel_depth=KD))
    L = xb.xconv_backprobe(S, d["dY"])
    check("dW (halves) " + note, host(xb.xconv_contract(L, Zg, kernel_depth=KD)),
          O.wgrad_contract3d(host(L), Zo, (KD, 3, 3)), 1e-5)
