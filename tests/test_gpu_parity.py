"""GPU parity: libxconv (through the C ABI) against the float64 oracle, element by element on the
same seeded inputs.  Tolerances: relative Frobenius error <= 1e-5 for float storage, <= 1e-2 for
bfloat16 storage with float accumulation; the estimate is compared with the oracle's ESTIMATE for
the same Z, never with the exact gradient."""
import ctypes

import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from oracle import xconv_oracle as O
from paper_2106_06998_b200 import binding as xb
from paper_2106_06998_b200 import inputs
from tests._util import TOL, TOL_SKETCH, check, dev, host, sketch_oracle_chunked, sketch_tol

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    entry.build()
    torch.cuda.set_device(0)


def _full_layer_parity(lay, K=3):
    tol = TOL[lay["dtype"]]
    d = dev(lay)
    Y, S = xb.xconv_forward(d["X"], d["W"], d["Z"])
    S2 = xb.xconv_sketch(d["X"], d["Z"])
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"], kernel_size=K)
    dX = xb.xconv_dgrad(d["dY"], d["W"])
    torch.cuda.synchronize()
    assert torch.equal(S, S2)
    Yo, So, dWo, dXo = O.xconv_layer(lay["X"], lay["W"], lay["dY"], lay["Z"])
    errs = dict(Y=check("Y", host(Y), Yo, tol), S=check("sketch", host(S), So, TOL_SKETCH),
                dX=check("dX", host(dX), dXo, tol))
    # the estimator alone, from the oracle's own sketch (float), so that its error is not inherited
    So32 = torch.from_numpy(So.astype(np.float32)).cuda()
    dW_from_oracle_S = xb.xconv_wgrad(So32, d["dY"], d["Z"], kernel_size=K)
    # the two halves on their own: L against Algorithm 1 backward step 3, the contraction against step 4
    L = xb.xconv_backprobe(So32, d["dY"])
    Lo = O.backprobe(So.astype(np.float32), lay["dY"])
    errs["L"] = check("L", host(L), Lo, tol)
    Lr = inputs.round_to_storage(Lo.astype(np.float32), lay["dtype"])
    dWc = xb.xconv_contract(xb.to_device(Lr, lay["dtype"]), d["Z"], kernel_size=K)
    check("dW (contraction alone)", host(dWc), O.wgrad_contract(Lr, lay["Z"], K, K), 1e-5 if lay["dtype"] == "f32" else 1e-4)
    errs["dW"] = check("dW (end to end)", host(dW), dWo, tol)
    check("dW (oracle sketch in)", host(dW_from_oracle_S), dWo, tol)
    return errs


# ------------------------------------------------------------------ small layers, every element

EDGE_SHAPES = [
    # B, Cin, Cout, H, W, r   -- odd sizes, ragged tiles, B = 1, r not a multiple of any tile
    (1, 1, 1, 1, 1, 1),
    (1, 3, 2, 5, 4, 3),
    (3, 5, 7, 9, 11, 5),
    (2, 16, 16, 8, 8, 8),
    (5, 33, 65, 7, 35, 17),
    (4, 64, 32, 12, 40, 70),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", EDGE_SHAPES)
def test_edge_shapes_all_elements(shape, dtype):
    B, Cin, Cout, H, W, r = shape
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype=dtype, seed=sum(shape))
    _full_layer_parity(lay)


# The 3 x 3 layers of the paper's two MNIST networks (appendix, network tables): 1 -> 16 on 28 x 28, 16 -> 32 on
# 14 x 14, 32 -> 32 on 7 x 7 (the Julia network), 1 -> 32 and 32 -> 64 on 28 x 28 (the PyTorch network, whose
# code figure in Section 4.2 uses 32 probing vectors).
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [
    # B, Cin, Cout, H, W, r
    (16, 1, 16, 28, 28, 8),
    (16, 16, 32, 14, 14, 8),
    (16, 32, 32, 7, 7, 8),
    (8, 1, 32, 28, 28, 32),
    (8, 32, 64, 28, 28, 32),
])
def test_layers_of_the_papers_mnist_networks(shape, dtype):
    B, Cin, Cout, H, W, r = shape
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype=dtype, seed=sum(shape) + 28, z="rademacher",
                             x="normal" if Cin == 1 else "relu")
    _full_layer_parity(lay)


# Shapes that reach the tcgen05 kernels with ragged tiles: channel counts that are not powers of two
# (several 64- or 32-channel groups, partial last tile), images that no patch tiles exactly, probe counts
# and batches that are not multiples of the MMA tile, r > B (re-associated wgrad) and r < B.
TENSOR_EDGE_SHAPES = [
    # B, Cin, Cout, H, W, r
    (24, 192, 320, 9, 13, 40),        # Cout 320 = 256 + 64: two row tiles, the second half empty
    (40, 320, 64, 10, 6, 24),         # Cin 320: column tiles 256 + 64
    (16, 96, 160, 12, 20, 48),        # multiples of 32 only: 64-byte-swizzle contraction, several groups
    (8, 32, 32, 40, 24, 72),          # one 32-channel group, r > B
    (72, 64, 128, 7, 9, 136),         # r just above a 128-row tile, B % 64 != 0
    (136, 128, 64, 5, 5, 8),          # tiny image (25 pixels), B above a tile, few probes
    (8, 64, 64, 3, 70, 16),           # wide flat image
    (9, 64, 64, 6, 12, 16),           # odd batch: the last image pair of the convolution is half empty
]


@pytest.mark.parametrize("shape", TENSOR_EDGE_SHAPES)
def test_tensor_path_edge_shapes_all_elements(shape):
    B, Cin, Cout, H, W, r = shape
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype="bf16", seed=sum(shape), z="rademacher", x="relu")
    desc = xb.make_desc(B, Cin, Cout, H, W, r, torch.bfloat16)
    assert xb.engine_for(desc, xb.OP_CONTRACT) == "tcgen05_bf16"
    _full_layer_parity(lay)


@pytest.mark.parametrize("shape", [
    # B, Cin, H, W, r
    (8, 24, 11, 13, 16),      # K = 3432: a multiple of 8 but not of 64 -> one k-block per stage, short A tile
    (24, 8, 17, 19, 8),       # K = 2584, samples on the MMA rows
    (8, 64, 6, 35, 8),        # K = 13440 = 64 * 210: four k-blocks per stage, the last stage half past K
    (200, 64, 5, 10, 8),      # two 128-row tiles, the second ragged
    (520, 8, 16, 16, 504),    # r*B/(r+B) > 250: pairs of row tiles share the column tile; both axes ragged
])
def test_sketch_tensor_path_k_blocking(shape):
    B, Cin, H, W, r = shape
    lay = inputs.make_custom(B, Cin, 8, H, W, r, dtype="bf16", seed=sum(shape), z="gaussian", x="normal")
    desc = xb.make_desc(B, Cin, 8, H, W, r, torch.bfloat16)
    assert xb.engine_for(desc, xb.OP_SKETCH) == "tcgen05_bf16"
    d = dev(lay)
    S = xb.xconv_sketch(d["X"], d["Z"])
    torch.cuda.synchronize()
    check("sketch", host(S), O.sketch(lay["X"], lay["Z"]), TOL_SKETCH)


@pytest.mark.parametrize("shape", [
    # B, Cout, H, W, r -- the persistent grid runs several rounds of column tiles of unequal width
    (16, 64, 24, 40, 136),    # 960 blocks of 64 positions, two probe tiles (the second has 8 rows)
    (24, 64, 30, 33, 40),     # 990 blocks: tiles of four and of three blocks, r not a multiple of 32
    (8, 128, 31, 29, 200),    # 1798 blocks, B below one 64-wide k-block
])
def test_backprobe_tensor_path_column_tiles(shape):
    B, Cout, H, W, r = shape
    lay = inputs.make_custom(B, 8, Cout, H, W, r, dtype="bf16", seed=sum(shape), z="gaussian", x="normal")
    desc = xb.make_desc(B, 8, Cout, H, W, r, torch.bfloat16)
    assert xb.engine_for(desc, xb.OP_BACKPROBE) == "tcgen05_bf16"
    S = np.random.Generator(np.random.PCG64(sum(shape))).standard_normal((r, B)).astype(np.float32)
    L = xb.xconv_backprobe(torch.from_numpy(S).cuda(), dev(lay)["dY"])
    torch.cuda.synchronize()
    check("L", host(L), O.backprobe(S, lay["dY"]), TOL["bf16"])


@pytest.mark.parametrize("shape", [
    # B, Cin, Cout, H, W, r -- wide layers whose contraction copies every k-block in two halves
    (16, 256, 256, 8, 28, 40),    # 28 x 4 patches: halves of 56 pixels, one MMA step spans the two halves
    (16, 256, 256, 16, 16, 36),   # 16 x 8 patches: halves of 64 pixels, no step across the halves
    (16, 256, 128, 8, 28, 24),    # one 128-row tile of output channels
    (8, 256, 192, 12, 28, 33),    # 192 output channels: the second row tile half empty; odd probe count
])
def test_contraction_in_half_stages(shape):
    B, Cin, Cout, H, W, r = shape
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype="bf16", seed=sum(shape), z="rademacher", x="relu")
    desc = xb.make_desc(B, Cin, Cout, H, W, r, torch.bfloat16)
    assert xb.engine_for(desc, xb.OP_CONTRACT) == "tcgen05_bf16"
    d = dev(lay)
    g = np.random.Generator(np.random.PCG64(sum(shape)))
    Lr = inputs.round_to_storage(g.standard_normal((r, Cout, H, W)).astype(np.float32), "bf16")
    dW = xb.xconv_contract(xb.to_device(Lr, "bf16"), d["Z"])
    torch.cuda.synchronize()
    check("dW (contraction alone)", host(dW), O.wgrad_contract(Lr, lay["Z"], 3, 3), 1e-4)


def test_pointwise_kernel_on_the_tensor_path():
    lay = inputs.make_custom(16, 64, 128, 8, 12, 32, dtype="bf16", seed=78, KH=1, KW=1)
    desc = xb.make_desc(16, 64, 128, 8, 12, 32, torch.bfloat16, 1)
    assert xb.engine_for(desc, xb.OP_CONTRACT) == "tcgen05_bf16" and xb.engine_for(desc, xb.OP_FORWARD) == "tcgen05_bf16"
    _full_layer_parity(lay, K=1)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_pointwise_kernel(dtype):
    lay = inputs.make_custom(3, 12, 20, 6, 10, 9, dtype=dtype, seed=77, KH=1, KW=1)
    _full_layer_parity(lay, K=1)


# 5 x 5 kernels: the layers of the paper's CIFAR-10 network (appendix, network tables): 3 -> 16 and
# 16 -> 32 channels on 32 x 32 images, 32 -> 32 on 16 x 16, plus a wide layer for the tcgen05 kernels.
@pytest.mark.parametrize("dtype,shape", [
    # B, Cin, Cout, H, W, r
    ("f32", (4, 3, 16, 32, 32, 8)),
    ("f32", (4, 16, 32, 32, 32, 8)),
    ("bf16", (4, 16, 32, 32, 32, 16)),
    ("f32", (6, 32, 32, 16, 16, 12)),
    ("bf16", (16, 32, 32, 16, 16, 12)),       # 32-channel groups: tcgen05, 64-byte-swizzle tiles
    ("bf16", (16, 128, 64, 9, 11, 24)),       # tcgen05, ragged patches, 25 offsets
    ("bf16", (8, 64, 64, 12, 12, 40)),        # r > B: the probes are summed first
    ("f32", (2, 5, 7, 6, 9, 5)),              # odd everything
])
def test_five_by_five_kernels(dtype, shape):
    B, Cin, Cout, H, W, r = shape
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype=dtype, seed=sum(shape) + 5, KH=5, KW=5,
                             z="rademacher", x="relu")
    _full_layer_parity(lay, K=5)


# float16 storage (the paper's "half precision", Section 5.2).  Tolerance 2e-3: S and L are each rounded once
# to float16 (2^-11 / sqrt(3) = 2.8e-4 relative rms each, about 4e-4 together); five times that.
@pytest.mark.parametrize("shape,K", [
    # B, Cin, Cout, H, W, r
    ((3, 5, 7, 9, 11, 5), 3),              # FP32-FMA kernels, odd sizes
    ((16, 128, 128, 28, 28, 32), 3),       # the ImageNet-stage recipe, shrunk: tcgen05 with float16 operands
    ((16, 128, 128, 28, 28, 128), 3),      # r > B
    ((24, 192, 320, 9, 13, 40), 3),        # ragged tiles
    ((8, 32, 32, 40, 24, 72), 3),          # 32-channel groups (64-byte swizzle)
    ((16, 32, 32, 16, 16, 12), 5),         # 5 x 5 kernel
    ((16, 64, 128, 8, 12, 32), 1),         # pointwise kernel
])
def test_float16_storage(shape, K):
    B, Cin, Cout, H, W, r = shape
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype="f16", seed=sum(shape) + 16, KH=K, KW=K,
                             z="rademacher", x="relu")
    lay["dY"] = inputs.round_to_storage(lay["dY"] * np.float32(0.1), "f16")     # the recipe's N(0, 1e-2)
    if Cin >= 32:
        desc = xb.make_desc(B, Cin, Cout, H, W, r, torch.float16, K)
        assert xb.engine_for(desc, xb.OP_CONTRACT) == "tcgen05_f16" and xb.engine_for(desc, xb.OP_SKETCH) == "tcgen05_f16"
    _full_layer_parity(lay, K=K)


@pytest.mark.parametrize("cfg,r,shrink", [
    (1, 8, {}),                                   # the small configuration at full size
    (2, 16, dict(B=32)), (2, 64, dict(B=32)),
    (3, 32, dict(B=16, H=28, W=28)), (3, 128, dict(B=16, H=28, W=28)),
    (4, 64, dict(B=16, H=48, W=40)),
    (5, 16, dict(B=128, H=14, W=14)), (5, 64, dict(B=128, H=14, W=14)), (5, 256, dict(B=256, H=14, W=14)),
])
def test_config_recipes_reduced_all_elements(cfg, r, shrink):
    """The five workload recipes (shapes shrunk where the oracle would take too long), all elements."""
    _full_layer_parity(inputs.make_layer(cfg, r, **shrink))


# ------------------------------------------------------------------ full sizes, sampled outputs

FULL = [(2, 16), (2, 64), (3, 32), (3, 128), (4, 64), (4, 256), (5, 16), (5, 64), (5, 256), (5, 1024)]


@pytest.mark.parametrize("cfg,r", FULL)
def test_full_size_sampled(cfg, r):
    """Full-size layers in the launch configuration the benchmark times.  The sketch is compared in
    full (one float64 matrix product per slab of probes); dW, Y and dX on channel / sample subsets,
    each of which the oracle computes as a smaller layer of its own."""
    lay = inputs.make_layer(cfg, r)
    tol = TOL[lay["dtype"]]
    d = dev(lay)
    Y, S = xb.xconv_forward(d["X"], d["W"], d["Z"])
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"])
    dX = xb.xconv_dgrad(d["dY"], d["W"])
    torch.cuda.synchronize()
    assert xb.workspace_status(xb.workspace(256, S.device)) == 0
    So = sketch_oracle_chunked(lay["X"], lay["Z"])
    check("sketch", host(S), So, sketch_tol(lay["Cin"] * lay["H"] * lay["width"]))
    g = np.random.Generator(np.random.PCG64(cfg * 1000 + r))
    # output / input channels at the ends of the channel range, either side of the 128-row tile boundary, and at random
    ms = np.unique(np.concatenate([[0, lay["Cout"] - 1, min(127, lay["Cout"] - 1), min(128, lay["Cout"] - 1)],
                                   g.choice(lay["Cout"], size=min(2, lay["Cout"]), replace=False)]))
    ns = np.unique(np.concatenate([[0, lay["Cin"] - 1], g.choice(lay["Cin"], size=min(4, lay["Cin"]), replace=False)]))
    dWo = O.wgrad_estimate(So, lay["dY"][:, ms], lay["Z"][:, ns])
    check("dW block", host(dW)[np.ix_(ms, ns)], dWo, tol)
    # the two halves as the benchmark calls them (Algorithm 1's order, which xconv_wgrad leaves when r > B),
    # fed the oracle's own sketch rounded to float
    So32 = So.astype(np.float32)
    L = xb.xconv_backprobe(torch.from_numpy(So32).cuda(), d["dY"])
    dW2 = xb.xconv_contract(L, d["Z"])
    torch.cuda.synchronize()
    check("dW block (back-probe + contraction)", host(dW2)[np.ix_(ms, ns)], dWo, tol)
    # L itself (Algorithm 1 backward step 3) on a few probes x output channels, all pixels
    js = np.sort(g.choice(r, size=min(5, r), replace=False))
    Lo = O.backprobe(So32[js], lay["dY"][:, ms])
    check("L rows", host(L[torch.from_numpy(js).cuda()][:, torch.from_numpy(ms).cuda()]), Lo, tol)
    del L, dW2
    bs = np.sort(g.choice(lay["B"], size=min(2, lay["B"]), replace=False))
    check("Y samples", host(Y[bs]), O.conv_forward(lay["X"][bs], lay["W"]), tol)
    check("dX samples", host(dX[bs]), O.dx_exact(lay["dY"][bs], lay["W"]), tol)


# ------------------------------------------------------------------ properties and options

def test_results_are_bit_reproducible():
    lay = inputs.make_layer(5, 64, B=128, H=14, W=14)
    d = dev(lay)
    S1 = xb.xconv_sketch(d["X"], d["Z"]).clone()
    W1 = xb.xconv_wgrad(S1, d["dY"], d["Z"]).clone()
    for _ in range(3):
        S2 = xb.xconv_sketch(d["X"], d["Z"])
        W2 = xb.xconv_wgrad(S2, d["dY"], d["Z"])
        assert torch.equal(S1, S2) and torch.equal(W1, W2)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_block_sparse_probes_with_channel_scale(dtype):
    """Eq. (7) probes with the 1/nnz(Z_n) scale of Eq. (8) passed as chan_scale."""
    lay = inputs.make_custom(4, 16, 24, 10, 12, 12, dtype=dtype, seed=5)
    g = np.random.Generator(np.random.PCG64(9))
    mask = (g.random((12, 16, 1, 1)) < 0.5).astype(np.float32)
    mask[:, 3] = 0                                     # one channel never probed: estimate must be 0
    lay["Z"] = lay["Z"] * mask
    sc = O.channel_scale(lay["Z"])
    d = dev(lay)
    S = xb.xconv_sketch(d["X"], d["Z"])
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"], chan_scale=torch.from_numpy(sc.astype(np.float32)).cuda())
    want = O.wgrad_estimate(O.sketch(lay["X"], lay["Z"]), lay["dY"], lay["Z"], scale=sc)
    check("dW nnz-scaled", host(dW), want, TOL[dtype])
    assert float(dW[:, 3].abs().max()) == 0.0


@pytest.mark.parametrize("shape", [
    # B, Cin, Cout, H, W, r
    (16, 64, 128, 12, 20, 24),        # r > B is false: back-probe, contraction and its reduce kernel on tcgen05
    (8, 32, 32, 40, 24, 72),          # r > B: xconv_wgrad sums over the probes first; 64-byte-swizzle tiles
    (32, 256, 256, 8, 28, 16),        # wide layer: contraction in half-stages
])
def test_block_sparse_probes_with_channel_scale_on_the_tensor_path(shape):
    """Eq. (7) probes (whole channel blocks of a probing vector zero with probability 1 - p_n) and the
    1/nnz(Z_n) scale of Eq. (8) on layers the tcgen05 kernels serve, in both orders of summation."""
    B, Cin, Cout, H, W, r = shape
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype="bf16", seed=sum(shape) + 1, z="rademacher", x="relu")
    desc = xb.make_desc(B, Cin, Cout, H, W, r, torch.bfloat16)
    assert xb.engine_for(desc, xb.OP_CONTRACT) == "tcgen05_bf16" and xb.engine_for(desc, xb.OP_BACKPROBE) == "tcgen05_bf16"
    g = np.random.Generator(np.random.PCG64(sum(shape)))
    mask = (g.random((r, Cin, 1, 1)) < 0.5).astype(np.float32)
    mask[:, 5] = 0                                     # one channel never probed: estimate must be exactly 0
    mask[0, 6] = 1                                     # and its neighbours probed at least once
    lay["Z"] = lay["Z"] * mask
    sc = O.channel_scale(lay["Z"])
    assert sc[5] == 0.0 and sc[6] > 0.0
    d = dev(lay)
    cs = torch.from_numpy(sc.astype(np.float32)).cuda()
    S = xb.xconv_sketch(d["X"], d["Z"])
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"], chan_scale=cs)
    So = O.sketch(lay["X"], lay["Z"])
    want = O.wgrad_estimate(So, lay["dY"], lay["Z"], scale=sc)
    check("sketch (block-sparse probes)", host(S), So, TOL_SKETCH)
    check("dW nnz-scaled", host(dW), want, TOL["bf16"])
    assert float(dW[:, 5].abs().max()) == 0.0
    # the paper's order of summation as well (back-probe, then the contraction with the scale)
    L = xb.xconv_backprobe(S, d["dY"])
    dW2 = xb.xconv_contract(L, d["Z"], chan_scale=cs)
    check("dW nnz-scaled (back-probe + contraction)", host(dW2), want, TOL["bf16"])
    assert float(dW2[:, 5].abs().max()) == 0.0


def test_orthogonal_probe_basis_recovers_exact_gradient_on_gpu():
    """r = Cin*N with (1/r) Z Z^T = I: the float path reproduces the exact gradient."""
    Cin, H, W = 2, 4, 4
    lay = inputs.make_custom(3, Cin, 3, H, W, Cin * H * W, dtype="f32", seed=3)
    from scipy.linalg import hadamard
    lay["Z"] = hadamard(32).astype(np.float32).reshape(32, Cin, H, W)
    d = dev(lay)
    dW = xb.xconv_wgrad(xb.xconv_sketch(d["X"], d["Z"]), d["dY"], d["Z"])
    check("exact recovery", host(dW), O.dw_exact(lay["X"], lay["dY"]), 1e-5)


def test_host_buffer_entry_point_matches_device_entry_points():
    lay = inputs.make_layer(5, 64, B=128, H=14, W=14)
    d = dev(lay)
    S = xb.xconv_sketch(d["X"], d["Z"])
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"])
    desc = xb.make_desc(lay["B"], lay["Cin"], lay["Cout"], lay["H"], lay["width"], 64, torch.bfloat16)
    hX, hdY, hZ = (d[k].cpu().pin_memory() for k in ("X", "dY", "Z"))
    hS = torch.empty((64, lay["B"]), dtype=torch.float32).pin_memory()
    hdW = torch.empty(dW.shape, dtype=torch.float32).contiguous(memory_format=torch.channels_last).pin_memory()
    arena = torch.empty(xb.host_arena_bytes(desc), dtype=torch.uint8, device="cuda")
    xb.xconv_sketch_wgrad_host(desc, hX, hdY, hZ, hS, hdW, arena)
    assert torch.equal(hS, S.cpu()) and torch.equal(hdW, dW.cpu())


def test_errors_launch_nothing_on_gpu():
    lay = inputs.make_custom(2, 8, 8, 6, 6, 4, dtype="f32", seed=1)
    d = dev(lay)
    desc = xb.make_desc(2, 8, 8, 6, 6, 4, torch.float32)
    S = torch.full((4, 2), 7.0, device="cuda")
    ws = torch.empty(xb.workspace_bytes(desc, xb.OP_SKETCH), dtype=torch.uint8, device="cuda")
    short = ws[: ws.numel() - 64]
    st = xb.lib().xconv_sketch(ctypes.byref(desc), d["X"].data_ptr(), d["Z"].data_ptr(), S.data_ptr(),
                               short.data_ptr(), short.numel(), None)
    torch.cuda.synchronize()
    assert st == 4 and float(S.min()) == 7.0 and float(S.max()) == 7.0


def test_bounded_wait_reports_timeout_and_next_call_recovers():
    """A wait that nothing satisfies gives up after its limit, the status says so, the context stays
    usable and the next call on the same workspace reports its own (clean) outcome."""
    lay = inputs.make_layer(5, 16, B=128, H=14, W=14)
    d = dev(lay, ("X", "Z"))
    desc = xb.make_desc(128, 256, 256, 14, 14, 16, torch.bfloat16)
    ws = torch.empty(xb.workspace_bytes(desc, xb.OP_SKETCH), dtype=torch.uint8, device="cuda")
    st = xb.lib().xconv_selftest_wait_limit(ws.data_ptr(), ws.numel(), 50, torch.cuda.current_stream().cuda_stream)
    assert st == 0
    assert xb.workspace_status(ws) == 6                      # XCONV_ERR_TIMEOUT
    S = torch.empty((16, 128), dtype=torch.float32, device="cuda")
    xb.sketch_into(desc, d["X"], d["Z"], S, ws)
    assert xb.workspace_status(ws) == 0
    check("sketch after a timed-out call", host(S), O.sketch(lay["X"], lay["Z"]), TOL_SKETCH)


def test_engines_reported():
    d1 = xb.make_desc(8, 16, 16, 32, 32, 8, torch.float32)
    assert xb.engine_for(d1, xb.OP_SKETCH) == "simt_f32" and xb.engine_for(d1, xb.OP_WGRAD) == "simt_f32"
    d5 = xb.make_desc(512, 256, 256, 28, 28, 64, torch.bfloat16)
    for op in (xb.OP_SKETCH, xb.OP_WGRAD, xb.OP_FORWARD, xb.OP_DGRAD):
        assert xb.engine_for(d5, op) == "tcgen05_bf16"
    d4 = xb.make_desc(16, 32, 32, 256, 256, 64, torch.bfloat16)      # 32 channels: 64-byte-swizzle tiles
    assert xb.engine_for(d4, xb.OP_SKETCH) == "tcgen05_bf16" and xb.engine_for(d4, xb.OP_WGRAD) == "tcgen05_bf16"
    d6 = xb.make_desc(16, 24, 40, 30, 30, 8, torch.bfloat16)         # channels not multiples of 32: FP32 FMA
    assert xb.engine_for(d6, xb.OP_WGRAD) == "simt_f32"


def test_a_step_can_be_captured_into_a_cuda_graph():
    """The library allocates nothing, keeps no per-call state on the host and never synchronises: sketch and
    estimator are captured once and replayed, with the bits of the uncaptured calls."""
    lay = inputs.make_layer(1, 8)
    d = dev(lay)
    B, Cin, H, W = d["X"].shape
    Cout, r = d["dY"].shape[1], d["Z"].shape[0]
    desc = xb.make_desc(B, Cin, Cout, H, W, r, d["X"].dtype)
    S = torch.empty((r, B), dtype=torch.float32, device="cuda")
    dW = torch.empty((Cout, Cin, 3, 3), dtype=torch.float32, device="cuda", memory_format=torch.channels_last)
    ws = xb.workspace(max(xb.workspace_bytes(desc, xb.OP_SKETCH), xb.workspace_bytes(desc, xb.OP_WGRAD)), S.device)

    def step():
        xb.sketch_into(desc, d["X"], d["Z"], S, ws)
        xb.wgrad_into(desc, S, d["dY"], d["Z"], dW, ws)

    step()
    torch.cuda.synchronize()
    S0, W0 = S.clone(), dW.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for _ in range(3):
        S.zero_(); dW.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(S, S0) and torch.equal(dW, W0)
    assert xb.workspace_status(ws) == 0
    check("dW replayed", host(dW), O.wgrad_estimate(O.sketch(lay["X"], lay["Z"]), lay["dY"], lay["Z"]), TOL["f32"])


@pytest.mark.parametrize("dtype,shape", [("f32", (5, 12, 10, 9, 11, 7)), ("bf16", (16, 64, 128, 12, 20, 24))])
def test_against_the_plain_c_oracle(dtype, shape):
    """The same layer against the second statement of the oracle (plain C loop nests, oracle/xconv_oracle.c)."""
    from oracle import c_oracle as C
    B, Cin, Cout, H, W, r = shape
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype=dtype, seed=sum(shape) + 5, z="rademacher", x="relu")
    d = dev(lay)
    Y, S = xb.xconv_forward(d["X"], d["W"], d["Z"])
    dW = xb.xconv_wgrad(S, d["dY"], d["Z"])
    dX = xb.xconv_dgrad(d["dY"], d["W"])
    So = C.sketch(lay["X"], lay["Z"])
    check("sketch", host(S), So, TOL_SKETCH)
    check("Y", host(Y), C.conv_forward(lay["X"], lay["W"]), TOL[dtype])
    check("dX", host(dX), C.dx_exact(lay["dY"], lay["W"]), TOL[dtype])
    check("dW", host(dW), C.wgrad_estimate(So, lay["dY"], lay["Z"]), TOL[dtype])
