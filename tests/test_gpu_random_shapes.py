"""Seeded random layer shapes through every entry point of the layer API, against the oracle: storage type,
kernel size, depth, channel counts on and off the tensor-core tiles, batch above and below the probe count."""
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


def _draw_case(seed):
    g = np.random.Generator(np.random.PCG64(seed))
    dtype = ["f32", "bf16", "f16"][int(g.integers(0, 3))]
    K = [1, 3, 3, 5][int(g.integers(0, 4))]
    D = [1, 1, 2, 3][int(g.integers(0, 4))]
    KD = 3 if (D > 1 and K == 3 and g.random() < 0.6) else 1
    chans = [1, 3, 8, 16, 24, 32, 40, 64, 96, 128]
    Cin, Cout = int(g.choice(chans)), int(g.choice(chans))
    if dtype != "f32" and g.random() < 0.6:            # steer half of the 16-bit cases onto the tensor-core tiles
        Cin, Cout = int(g.choice([32, 64, 96, 128])), int(g.choice([32, 64, 128, 160]))
    H, W = int(g.integers(1, 15)), int(g.integers(1, 15))
    B, r = int(g.integers(1, 41)), int(g.integers(1, 49))
    return dict(dtype=dtype, K=K, D=D, KD=KD, Cin=Cin, Cout=Cout, H=H, W=W, B=B, r=r)


@pytest.mark.parametrize("seed", range(128))
def test_random_layer(seed):
    c = _draw_case(1000 + seed)
    dtype, K, D, KD = c["dtype"], c["K"], c["D"], c["KD"]
    B, Cin, Cout, H, W, r = c["B"], c["Cin"], c["Cout"], c["H"], c["W"], c["r"]
    geo = (D, H, W) if D > 1 else (H, W)
    kgeo = (KD, K, K) if D > 1 else (K, K)
    dy_scale = 0.1 if dtype == "f16" else 1.0
    lay = dict(X=inputs.draw("relu", (B, Cin) + geo, seed * 10, dtype),
               W=inputs.draw("normal", (Cout, Cin) + kgeo, seed * 10 + 1, dtype, (2.0 / (Cin * KD * K * K)) ** 0.5),
               dY=inputs.draw("normal", (B, Cout) + geo, seed * 10 + 2, dtype, dy_scale),
               Z=inputs.draw(["rademacher", "gaussian"][seed % 2], (r, Cin) + geo, seed * 10 + 3, dtype))
    d = {k: xb.to_device(v, dtype) for k, v in lay.items()}
    tol = TOL[dtype]
    Y, S = xb.xconv_forward(d["X"], d["W"], d["Z"])
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"], kernel_size=K, kernel_depth=KD)
    dX = xb.xconv_dgrad(d["dY"], d["W"])
    torch.cuda.synchronize()
    So = O.sketch(lay["X"], lay["Z"])
    if D > 1:
        Yo, dXo = O.conv_forward3d(lay["X"], lay["W"]), O.dx_exact3d(lay["dY"], lay["W"])
        dWo = O.wgrad_estimate3d(So, lay["dY"], lay["Z"], (KD, K, K))
    else:
        Yo, dXo = O.conv_forward(lay["X"], lay["W"]), O.dx_exact(lay["dY"], lay["W"])
        dWo = O.wgrad_estimate(So, lay["dY"], lay["Z"], K, K)
    note = str(c)
    check("sketch " + note, host(S), So, TOL_SKETCH)
    check("Y " + note, host(Y), Yo, tol)
    check("dX " + note, host(dX), dXo, tol)
    check("dW " + note, host(dW), dWo, tol)
    # the paper's order through the two halves, and the per-pair estimator, on the same tensors
    So32 = So.astype(np.float32)
    L = xb.xconv_backprobe(torch.from_numpy(So32).cuda(), d["dY"])
    check("L " + note, host(L), O.backprobe(So32, lay["dY"]), tol)
    dW2 = xb.xconv_contract(L, d["Z"], kernel_size=K, kernel_depth=KD)
    check("dW (halves) " + note, host(dW2), dWo, tol)
    Si = xb.xconv_sketch_independent(d["X"], d["Z"])
    Sio = np.stack([O.sketch(lay["X"][:, n:n + 1], lay["Z"][:, n:n + 1]) for n in range(Cin)], axis=1)
    check("per-channel sketch " + note, host(Si), Sio, TOL_SKETCH)
    dWi = xb.xconv_wgrad_independent(torch.from_numpy(Sio.astype(np.float32)).cuda(), d["dY"], d["Z"], kernel_size=K, kernel_depth=KD)
    if D > 1:
        want = np.concatenate([O.wgrad_estimate3d(Sio[:, n, :], lay["dY"], lay["Z"][:, n:n + 1], (KD, K, K)) for n in range(Cin)], axis=1)
    else:
        want = O.wgrad_estimate_independent(Sio, lay["dY"], lay["Z"], K, K)
    check("dW (independent) " + note, host(dWi), want, tol)
    if D == 1:        # the sketch through the entry point that takes no workspace
        check("sketch (no workspace) " + note, host(xb.xconv_sketch_static(d["X"], d["Z"])), So, TOL_SKETCH)
    # the same layer with its probing vectors redrawn from a seed (Algorithm 1 keeps the seed, not Z); a volume's
    # probing vector is numbered in memory order like an image of D*H rows
    zseed = 900000 + seed
    Zo = O.rademacher_probes(zseed, r, Cin, D * H, W)
    if D > 1:
        Zo = Zo.reshape(r, Cin, D, H, W)
    Ss = xb.xconv_sketch_seeded(d["X"], zseed, r)
    check("seeded sketch " + note, host(Ss), O.sketch(lay["X"], Zo), TOL_SKETCH)
    dWs = xb.xconv_wgrad_seeded(Ss, d["dY"], zseed, Cin, kernel_size=K, kernel_depth=KD)
    Zg = xb.xconv_probes_from_seed(zseed, r, Cin, H, W, d["X"].dtype, D=D)
    assert np.array_equal(host(Zg), Zo)
    assert torch.equal(dWs, xb.xconv_wgrad(Ss, d["dY"], Zg, kernel_size=K, kernel_depth=KD))
    if D > 1:
        check("seeded dW " + note, host(dWs), O.wgrad_estimate3d(host(Ss), lay["dY"], Zo, (KD, K, K)), tol)
    else:
        check("seeded dW " + note, host(dWs), O.wgrad_estimate(host(Ss), lay["dY"], Zo, K, K), tol)


def _draw_medium(seed):
    g = np.random.Generator(np.random.PCG64(seed))
    dtype = ["bf16", "f16"][int(g.integers(0, 2))]
    Cin, Cout = int(g.choice([32, 64, 96])), int(g.choice([32, 64]))
    H, W = int(g.integers(9, 41)), int(g.integers(9, 41))
    B, r = int(g.choice([4, 8, 13, 24, 40])), int(g.choice([8, 16, 40, 72, 136, 200]))
    return dict(dtype=dtype, Cin=Cin, Cout=Cout, H=H, W=W, B=B, r=r)


@pytest.mark.parametrize("seed", range(40))
def test_random_medium_layer(seed):
    """Larger images on the tensor-core tiles (several tiles per CTA, rings of stages that wrap, ragged tiles, probing
    vectors of every length modulo 128), the estimator in both orders of summation, stored and redrawn probes."""
    c = _draw_medium(5000 + seed)
    dtype = c["dtype"]
    B, Cin, Cout, H, W, r = c["B"], c["Cin"], c["Cout"], c["H"], c["W"], c["r"]
    note = str(c)
    lay = dict(X=inputs.draw("relu", (B, Cin, H, W), seed * 10 + 7, dtype),
               dY=inputs.draw("normal", (B, Cout, H, W), seed * 10 + 8, dtype, 0.1 if dtype == "f16" else 1.0))
    d = {k: xb.to_device(v, dtype) for k, v in lay.items()}
    zseed = 7000 + seed
    Zo = O.rademacher_probes(zseed, r, Cin, H, W)
    Zg = xb.xconv_probes_from_seed(zseed, r, Cin, H, W, d["X"].dtype)
    assert np.array_equal(host(Zg), Zo)
    So = O.sketch(lay["X"], Zo)
    S = xb.xconv_sketch(d["X"], Zg)
    Ss = xb.xconv_sketch_seeded(d["X"], zseed, r)
    check("sketch " + note, host(S), So, TOL_SKETCH)
    check("seeded sketch " + note, host(Ss), So, TOL_SKETCH)
    want = O.wgrad_estimate(host(S), lay["dY"], Zo)
    dW = xb.xconv_wgrad(S, d["dY"], Zg)
    check("dW " + note, host(dW), want, TOL[dtype])
    assert torch.equal(dW, xb.xconv_wgrad_seeded(S, d["dY"], zseed, Cin))
    L = xb.xconv_backprobe(S, d["dY"])
    check("L " + note, host(L), O.backprobe(host(S), lay["dY"]), TOL[dtype])
    check("dW (halves) " + note, host(xb.xconv_contract(L, Zg)), O.wgrad_contract(host(L), Zo), 1e-5)


@pytest.mark.parametrize("seed", range(40))
def test_random_medium_convolution(seed):
    """Forward convolution and exact input gradient on larger images (ragged patches, channel counts on and off the
    tensor-core tiles, all kernel sizes and storage types), against the plain-C statement of the oracle."""
    from oracle import c_oracle as C
    g = np.random.Generator(np.random.PCG64(90000 + seed))
    dtype = ["bf16", "f16", "f32"][int(g.integers(0, 3))]
    K = int(g.choice([1, 3, 3, 5]))
    Cin, Cout = int(g.choice([8, 32, 64, 96, 128, 160])), int(g.choice([8, 32, 64, 96, 128, 160]))
    H, W = int(g.integers(5, 41)), int(g.integers(5, 41))
    B = int(g.integers(1, 7))
    note = str(dict(dtype=dtype, K=K, Cin=Cin, Cout=Cout, H=H, W=W, B=B))
    X = inputs.draw("relu", (B, Cin, H, W), seed * 7 + 1, dtype)
    Wt = inputs.draw("normal", (Cout, Cin, K, K), seed * 7 + 2, dtype, (2.0 / (Cin * K * K)) ** 0.5)
    dY = inputs.draw("normal", (B, Cout, H, W), seed * 7 + 3, dtype, 0.1 if dtype == "f16" else 1.0)
    Z = inputs.draw("rademacher", (4, Cin, H, W), seed * 7 + 4, dtype)
    d = {k: xb.to_device(v, dtype) for k, v in dict(X=X, W=Wt, dY=dY, Z=Z).items()}
    Y, _ = xb.xconv_forward(d["X"], d["W"], d["Z"])
    dX = xb.xconv_dgrad(d["dY"], d["W"])
    check("Y " + note, host(Y), C.conv_forward(X, Wt), TOL[dtype])
    check("dX " + note, host(dX), C.dx_exact(dY, Wt), TOL[dtype])
