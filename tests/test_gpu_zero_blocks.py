"""GPU parity for block-sparse probing vectors (Eq. 7) whose all-zero 64-channel blocks are named to the
contraction (descriptor field zero_blocks) so that wide layers neither fetch nor multiply them, with the
1/nnz(Z_n) scale of Eq. 8.  The oracle knows nothing of masks: it gets the probing vectors themselves."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from oracle import xconv_oracle as O
from paper_2106_06998_b200 import binding as xb
from paper_2106_06998_b200 import inputs
from tests._util import TOL, check, host

pytestmark = pytest.mark.gpu

TORCH = {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}


@pytest.fixture(scope="module", autouse=True)
def _built():
    entry.build()
    torch.cuda.set_device(0)


def _sparse_layer(B, Cin, Cout, H, W, r, dtype, seed, p_group, K=3, D=None, KD=1):
    """A layer whose probing vectors keep a 64-channel group with probability p_group, and a channel inside a
    kept group with probability 1/2 (Eq. 7 with blocks of one channel); group 1 is never probed."""
    sp = (H, W) if D is None else (D, H, W)
    ones = (1,) * len(sp)
    g = np.random.Generator(np.random.PCG64(seed))
    groups = Cin // 64
    keep_g = g.random((r, groups)) < p_group
    if groups > 1:
        keep_g[:, 1] = False
    keep_g[0, 0] = True
    keep_c = np.repeat(keep_g, 64, axis=1) & (g.random((r, Cin)) < 0.5)
    Z = inputs.draw("rademacher", (r, Cin) + sp, seed * 10 + 3, dtype) * keep_c.reshape((r, Cin) + ones)
    # a group may come out empty although it was kept: the mask is what the probes say, not what was drawn
    zero = ~np.any(Z.reshape(r, groups, -1) != 0, axis=2)
    wshape = (Cout, Cin, K, K) if D is None else (Cout, Cin, KD, K, K)
    return dict(X=inputs.draw("relu", (B, Cin) + sp, seed * 10, dtype),
                W=inputs.draw("normal", wshape, seed * 10 + 1, dtype),
                dY=inputs.draw("normal", (B, Cout) + sp, seed * 10 + 2, dtype, 0.1 if dtype == "f16" else 1.0),
                Z=Z, zero=zero.astype(np.uint8))


CASES = [
    # dtype, (B, Cin, Cout, H, W, r), K, p_group, blocks skipped?
    ("bf16", (64, 256, 256, 28, 28, 16), 3, 0.3, True),      # four blocks per tile, two row tiles, unrolled k-steps
    ("bf16", (32, 128, 256, 16, 16, 12), 3, 0.5, True),      # two blocks per tile
    ("f16", (32, 320, 256, 16, 16, 12), 3, 0.4, True),       # two column tiles, the second one block wide; float16
    ("bf16", (32, 512, 128, 16, 16, 12), 3, 0.25, True),     # two full column tiles, one row tile
    ("bf16", (32, 256, 256, 16, 16, 12), 5, 0.3, True),      # 5 x 5 kernel
    ("bf16", (32, 256, 256, 14, 14, 12), 1, 0.5, True),      # pointwise kernel, ragged patches
    ("bf16", (8, 256, 256, 10, 24, 40), 3, 0.3, True),       # r > B: xconv_wgrad sums over the probes first, xconv_contract skips
    ("bf16", (32, 128, 64, 12, 20, 24), 3, 0.5, False),      # small layers: the mask is ignored
    ("f16", (48, 192, 128, 9, 14, 40), 3, 0.4, False),
]


@pytest.mark.parametrize("dtype,shape,K,p_group,skips", CASES)
def test_contraction_with_named_zero_blocks(dtype, shape, K, p_group, skips):
    B, Cin, Cout, H, W, r = shape
    lay = _sparse_layer(B, Cin, Cout, H, W, r, dtype, seed=sum(shape) + K, p_group=p_group, K=K)
    d = {k: xb.to_device(lay[k], dtype) for k in ("X", "dY", "Z")}
    sc = O.channel_scale(lay["Z"])
    cs = torch.from_numpy(sc.astype(np.float32)).cuda()
    # the mask, computed on the device from Z, is the one the probes define
    zb = xb.xconv_zero_blocks(d["Z"])
    assert zb.dtype == torch.uint8 and np.array_equal(zb.cpu().numpy(), lay["zero"])
    assert 0 < int(zb.sum()) < zb.numel()
    desc = xb.make_desc(B, Cin, Cout, H, W, r, TORCH[dtype], K, zero_blocks=zb)
    assert xb.engine_for(desc, xb.OP_CONTRACT) == "tcgen05_" + dtype
    assert xb.zero_blocks_used(desc) == skips
    S = xb.xconv_sketch(d["X"], d["Z"])
    So = O.sketch(lay["X"], lay["Z"])
    want = O.wgrad_estimate(So, lay["dY"], lay["Z"], KH=K, KW=K, scale=sc)
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"], kernel_size=K, chan_scale=cs, zero_blocks=zb)
    check("dW, zero blocks named", host(dW), want, TOL[dtype])
    assert float(dW[:, 64:128].abs().max()) == 0.0            # the group that is never probed
    # the two halves on their own, against the oracle's contraction of the library's L
    L = xb.xconv_backprobe(S, d["dY"])
    dW2 = xb.xconv_contract(L, d["Z"], kernel_size=K, chan_scale=cs, zero_blocks=zb)
    want2 = O.wgrad_contract(host(L), lay["Z"], KH=K, KW=K, scale=sc)
    check("contraction, zero blocks named", host(dW2), want2, 1e-5)
    assert float(dW2[:, 64:128].abs().max()) == 0.0
    # the same mask gives the same bits again (the list of non-zero blocks keeps the probes in order)
    assert torch.equal(dW2, xb.xconv_contract(L, d["Z"], kernel_size=K, chan_scale=cs, zero_blocks=zb))


def test_many_probes_few_of_them_non_zero():
    """More probing vectors than one pass of the list kernel takes (1024), and more listed probes per work unit than
    its shared-memory copy of the list holds (128).  The oracle gets only the probes that are not zero
    altogether: the others add nothing to its sum."""
    Cin, Cout, H, W, r = 128, 128, 8, 16, 2300
    g = np.random.Generator(np.random.PCG64(2300))
    keep = g.random((r, 2)) < 0.1
    keep[100:700] |= g.random((600, 2)) < 0.7                 # a dense stretch: one unit's slice of the list is long
    Z = inputs.draw("rademacher", (r, Cin, H, W), 23001, "bf16") * np.repeat(keep, 64, axis=1)[:, :, None, None]
    Lh = inputs.draw("normal", (r, Cout, H, W), 23002, "bf16")
    zb = torch.from_numpy((~keep).astype(np.uint8)).cuda()
    Zd, Ld = xb.to_device(Z, "bf16"), xb.to_device(Lh, "bf16")
    assert torch.equal(xb.xconv_zero_blocks(Zd), zb)
    assert xb.zero_blocks_used(xb.make_desc(1, Cin, Cout, H, W, r, torch.bfloat16, zero_blocks=zb))
    got = xb.xconv_contract(Ld, Zd, zero_blocks=zb)
    rows = np.flatnonzero(keep.any(axis=1))
    want = O.wgrad_contract(Lh[rows], Z[rows], scale=np.full(Cin, 1.0 / r))
    check("contraction over a long, sparse list", host(got), want, 1e-5)


def test_a_masked_probe_is_not_read():
    """The mask is a promise, not a hint that is checked: a probing vector whose blocks are all named zero drops
    out of the sum although it is not zero.  (What the oracle computes when that vector is set to zero.)"""
    Cin, Cout, H, W, r = 256, 128, 16, 16, 12
    Z = inputs.draw("rademacher", (r, Cin, H, W), 771, "bf16")          # dense probes
    Lh = inputs.draw("normal", (r, Cout, H, W), 772, "bf16")
    mask = np.zeros((r, 4), np.uint8)
    mask[[0, 7, 11], :] = 1
    Zm = Z.copy()
    Zm[[0, 7, 11]] = 0
    zb = torch.from_numpy(mask).cuda()
    assert xb.zero_blocks_used(xb.make_desc(1, Cin, Cout, H, W, r, torch.bfloat16, zero_blocks=zb))
    got = xb.xconv_contract(xb.to_device(Lh, "bf16"), xb.to_device(Z, "bf16"), zero_blocks=zb)
    check("contraction under a mask", host(got), O.wgrad_contract(Lh, Zm), 1e-5)
    assert O.rel_fro(host(got), O.wgrad_contract(Lh, Z)) > 1e-2


def test_all_blocks_masked_gives_zero():
    Cin, Cout, H, W, r = 128, 128, 16, 16, 8
    Z = xb.to_device(inputs.draw("rademacher", (r, Cin, H, W), 5, "bf16"), "bf16")
    L = xb.to_device(inputs.draw("normal", (r, Cout, H, W), 6, "bf16"), "bf16")
    zb = torch.ones((r, 2), dtype=torch.uint8, device="cuda")
    assert xb.zero_blocks_used(xb.make_desc(1, Cin, Cout, H, W, r, torch.bfloat16, zero_blocks=zb))
    got = xb.xconv_contract(L, Z, zero_blocks=zb)
    assert float(got.abs().max()) == 0.0


@pytest.mark.parametrize("KD", [3, 1])
def test_zero_blocks_on_volumes(KD):
    """3 x 3 x 3 kernels skip the planes of a masked probe; a planar kernel on a volume ignores the mask.  Both
    give the oracle's estimate."""
    B, Cin, Cout, D, H, W, r = 8, 128, 128, 3, 16, 16, 6
    lay = _sparse_layer(B, Cin, Cout, H, W, r, "bf16", seed=90 + KD, p_group=0.5, D=D, KD=KD)
    d = {k: xb.to_device(lay[k], "bf16") for k in ("X", "dY", "Z")}
    sc = O.channel_scale(lay["Z"])
    cs = torch.from_numpy(sc.astype(np.float32)).cuda()
    zb = xb.xconv_zero_blocks(d["Z"])
    assert np.array_equal(zb.cpu().numpy(), lay["zero"])
    assert xb.zero_blocks_used(xb.make_desc(B, Cin, Cout, H, W, r, torch.bfloat16, D=D, KD=KD, zero_blocks=zb)) == (KD == 3)
    S = xb.xconv_sketch(d["X"], d["Z"])
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"], kernel_depth=KD, chan_scale=cs, zero_blocks=zb)
    So = O.sketch(lay["X"].reshape(B, Cin, D * H, W), lay["Z"].reshape(r, Cin, D * H, W))
    want = O.wgrad_estimate3d(So, lay["dY"], lay["Z"], K=(KD, 3, 3), scale=sc)
    check("dW on a volume, zero blocks named", host(dW), want, TOL["bf16"])


@pytest.mark.parametrize("dtype,shape", [
    ("f32", (8, 64, 32, 6, 6, 4)),           # FP32-FMA kernels ignore the mask
    ("f32", (4, 128, 64, 8, 8, 12)),
])
def test_paths_that_ignore_the_mask_still_match(dtype, shape):
    B, Cin, Cout, H, W, r = shape
    lay = _sparse_layer(B, Cin, Cout, H, W, r, dtype, seed=sum(shape), p_group=0.5)
    d = {k: xb.to_device(lay[k], dtype) for k in ("X", "dY", "Z")}
    sc = O.channel_scale(lay["Z"])
    cs = torch.from_numpy(sc.astype(np.float32)).cuda()
    zb = xb.xconv_zero_blocks(d["Z"])
    assert np.array_equal(zb.cpu().numpy(), lay["zero"])
    S = xb.xconv_sketch(d["X"], d["Z"])
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"], chan_scale=cs, zero_blocks=zb)
    want = O.wgrad_estimate(O.sketch(lay["X"], lay["Z"]), lay["dY"], lay["Z"], scale=sc)
    check("dW", host(dW), want, TOL[dtype])


def test_mask_shape_is_checked():
    with pytest.raises(ValueError):
        xb.make_desc(4, 96, 64, 8, 8, 4, torch.bfloat16, zero_blocks=torch.zeros((4, 1), dtype=torch.uint8, device="cuda"))
    with pytest.raises(ValueError):
        xb.make_desc(4, 128, 64, 8, 8, 4, torch.bfloat16, zero_blocks=torch.zeros((4, 3), dtype=torch.uint8, device="cuda"))


def test_back_to_back_calls_give_the_same_bits():
    """Ten masked contractions in a row on one stream (each kernel's preamble overlaps the tail of the one before):
    the list kernel, the main kernel and the reduce kernel of every call see the state their own call left."""
    Cin, Cout, H, W, r = 256, 256, 28, 28, 16
    g = np.random.Generator(np.random.PCG64(123))
    keep = g.random((r, 4)) < 0.4
    keep[0, 0] = True
    Z = inputs.draw("rademacher", (r, Cin, H, W), 1231, "bf16") * np.repeat(keep, 64, axis=1)[:, :, None, None]
    Zd = xb.to_device(Z, "bf16")
    Ld = xb.to_device(inputs.draw("normal", (r, Cout, H, W), 1232, "bf16"), "bf16")
    zb = torch.from_numpy((~keep).astype(np.uint8)).cuda()
    desc = xb.make_desc(1, Cin, Cout, H, W, r, torch.bfloat16, zero_blocks=zb)
    assert xb.zero_blocks_used(desc)
    ws = xb.workspace(xb.workspace_bytes(desc, xb.OP_WGRAD), Ld.device)
    outs = [torch.empty((Cout, Cin, 3, 3), dtype=torch.float32, device="cuda", memory_format=torch.channels_last) for _ in range(10)]
    for o in outs:
        xb.contract_into(desc, Ld, Zd, o, ws)
    torch.cuda.synchronize()
    assert xb.workspace_status(ws) == 0
    assert all(torch.equal(outs[0], o) for o in outs[1:])
    check("contraction, ten calls", host(outs[-1]), O.wgrad_contract(host(Ld), Z), 1e-5)


def _draw_masked(seed):
    g = np.random.Generator(np.random.PCG64(seed))
    return dict(dtype=["bf16", "f16"][int(g.integers(0, 2))], Cin=int(g.choice([128, 192, 256, 320, 512])),
                Cout=int(g.choice([64, 128, 256])), H=int(g.choice([12, 14, 16, 20, 24, 28])),
                W=int(g.choice([12, 14, 16, 20, 24, 28])), r=int(g.integers(4, 49)), K=int(g.choice([1, 3, 3])),
                p=float(g.choice([0.1, 0.3, 0.6, 0.9])))


@pytest.mark.parametrize("seed", range(32))
def test_random_masked_contraction(seed):
    """Seeded random wide layers and masks (some skip, some ignore the mask; whole probes, whole tiles and single
    blocks zero): the contraction against the oracle, which gets the probes that are not zero altogether."""
    c = _draw_masked(3000 + seed)
    dtype, Cin, Cout, H, W, r, K = c["dtype"], c["Cin"], c["Cout"], c["H"], c["W"], c["r"], c["K"]
    g = np.random.Generator(np.random.PCG64(4000 + seed))
    keep = g.random((r, Cin // 64)) < c["p"]
    keep[g.integers(0, r)] = False                          # one probe zero altogether
    keep[g.integers(0, r), 0] = True                        # and at least one block that is not
    Z = inputs.draw("rademacher", (r, Cin, H, W), seed * 10 + 1, dtype) * np.repeat(keep, 64, axis=1)[:, :, None, None]
    Lh = inputs.draw("normal", (r, Cout, H, W), seed * 10 + 2, dtype)
    Zd, Ld = xb.to_device(Z, dtype), xb.to_device(Lh, dtype)
    zb = xb.xconv_zero_blocks(Zd)
    assert np.array_equal(zb.cpu().numpy(), (~keep).astype(np.uint8))
    got = xb.xconv_contract(Ld, Zd, kernel_size=K, zero_blocks=zb)
    rows = np.flatnonzero(keep.any(axis=1))
    want = O.wgrad_contract(Lh[rows], Z[rows], KH=K, KW=K, scale=np.full(Cin, 1.0 / r))
    check("masked contraction " + str(c), host(got), want, 1e-5)
