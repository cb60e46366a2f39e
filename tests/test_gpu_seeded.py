"""GPU parity of the seeded calls: probing vectors redrawn from a seed (Algorithm 1 stores the seed, not
Z).  The generator is compared bit for bit with the oracle's own implementation of the same published
definition; the seeded sketch with the oracle's sketch on the oracle's Z, and bit for bit with the
library's sketch on the library's Z."""
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


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16, torch.float16])
@pytest.mark.parametrize("shape", [(1, 1, 1, 1), (3, 5, 4, 7), (8, 16, 9, 9), (5, 64, 6, 12), (130, 8, 5, 13)])
def test_probes_from_seed_match_the_oracle_generator_bit_for_bit(shape, dtype):
    r, Cin, H, W = shape
    for seed in (0, 0x1234567890ABCDEF, 2**64 - 1):
        Z = xb.xconv_probes_from_seed(seed, r, Cin, H, W, dtype)
        torch.cuda.synchronize()
        assert np.array_equal(host(Z), O.rademacher_probes(seed, r, Cin, H, W))


SEEDED_SKETCH_SHAPES = [
    # B, Cin, H, W, r
    (24, 8, 16, 16, 8),       # samples on the MMA rows, K = 2048: four k-blocks per stage
    (8, 64, 6, 35, 40),       # probes on the MMA rows (r > B): Z is the A operand; last stage half past K
    (200, 64, 5, 10, 72),     # two 128-row tiles of samples, 72 probes
    (520, 8, 16, 16, 504),    # pairs of row tiles share the redrawn tile; both axes ragged
    (16, 32, 24, 24, 300),    # r > B with three probe tiles, the last one ragged
    (8, 24, 11, 13, 16),      # K = 3432 is not a multiple of 64: Z is written to the workspace first
    (3, 5, 7, 9, 5),          # no tensor-core kernel at all
]


@pytest.mark.parametrize("shape", SEEDED_SKETCH_SHAPES)
def test_seeded_sketch_matches_oracle_and_the_stored_probe_path(shape):
    B, Cin, H, W, r = shape
    seed = 1000003 * sum(shape) + 17
    lay = inputs.make_custom(B, Cin, 8, H, W, r, dtype="bf16", seed=sum(shape), z="rademacher", x="normal")
    X = xb.to_device(lay["X"], "bf16")
    S = xb.xconv_sketch_seeded(X, seed, r)
    Zg = xb.xconv_probes_from_seed(seed, r, Cin, H, W, torch.bfloat16)
    S_stored = xb.xconv_sketch(X, Zg)
    torch.cuda.synchronize()
    # the same sum in a possibly different order (the seeded plan may take more k-blocks per stage)
    check("seeded sketch against the stored-probe sketch", host(S), host(S_stored), 1e-5)
    check("seeded sketch", host(S), O.sketch(lay["X"], O.rademacher_probes(seed, r, Cin, H, W)), TOL_SKETCH)


@pytest.mark.parametrize("shape", [(24, 8, 16, 16, 8), (8, 64, 6, 35, 40)])
def test_seeded_sketch_float16_storage_redraws_float16_signs(shape):
    B, Cin, H, W, r = shape
    seed = 31 * sum(shape)
    lay = inputs.make_custom(B, Cin, 8, H, W, r, dtype="f16", seed=sum(shape), z="rademacher", x="normal")
    X = xb.to_device(lay["X"], "f16")
    assert xb.engine_for(xb.make_desc(B, Cin, 8, H, W, r, torch.float16), xb.OP_SKETCH) == "tcgen05_f16"
    S = xb.xconv_sketch_seeded(X, seed, r)
    torch.cuda.synchronize()
    check("seeded sketch", host(S), O.sketch(lay["X"], O.rademacher_probes(seed, r, Cin, H, W)), TOL_SKETCH)


def test_seeded_sketch_float_storage():
    B, Cin, H, W, r, seed = 6, 16, 8, 8, 12, 99
    lay = inputs.make_custom(B, Cin, 8, H, W, r, dtype="f32", seed=5, z="rademacher", x="normal")
    X = xb.to_device(lay["X"], "f32")
    S = xb.xconv_sketch_seeded(X, seed, r)
    torch.cuda.synchronize()
    check("seeded sketch", host(S), O.sketch(lay["X"], O.rademacher_probes(seed, r, Cin, H, W)), TOL_SKETCH)


@pytest.mark.parametrize("shape,dtype", [
    ((16, 64, 64, 12, 20, 24), "bf16"),
    # r > B on the tensor cores: the estimator sums over the probes first and its first kernel redraws Z on chip
    ((8, 32, 32, 40, 24, 72), "bf16"),       # two k-blocks of probes, the second with 8 of 64 rows
    ((4, 64, 64, 16, 16, 200), "f16"),       # float16 signs, four k-blocks
    ((16, 32, 64, 64, 64, 64), "bf16"),      # one k-block per tile, a few tiles per CTA
    ((16, 32, 32, 128, 128, 64), "bf16"),    # 14 tiles per CTA: the ring of stages wraps, six warps draw in turn
    ((2, 128, 64, 16, 16, 520), "bf16"),     # nine k-blocks per tile: more than the ring holds
    ((5, 64, 32, 8, 24, 24), "bf16"),        # one ragged k-block; an odd number of samples
    ((4, 32, 32, 9, 22, 16), "bf16"),        # a probing vector is 99 x 64 entries long: odd rows start mid Philox block
    ((6, 96, 32, 11, 6, 48), "f16"),         # the same with 96 channels, float16
    ((5, 64, 32, 9, 24, 17), "bf16"),        # 17 probes (not a multiple of 8): Z goes through the workspace
    ((3, 5, 7, 9, 11, 5), "f32"), ((2, 16, 16, 8, 8, 8), "f32")])
def test_seeded_layer_matches_the_oracle_with_redrawn_probes(shape, dtype):
    """Algorithm 1 end to end with nothing but S and the seed kept between the passes."""
    B, Cin, Cout, H, W, r = shape
    seed = 7919 * sum(shape) + 3
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype=dtype, seed=sum(shape), z="rademacher", x="relu")
    X, dY = xb.to_device(lay["X"], dtype), xb.to_device(lay["dY"], dtype)
    S = xb.xconv_sketch_seeded(X, seed, r)
    dW = xb.xconv_wgrad_seeded(S, dY, seed, Cin)
    Zg = xb.xconv_probes_from_seed(seed, r, Cin, H, W, X.dtype)
    dW_stored = xb.xconv_wgrad(S, dY, Zg)
    torch.cuda.synchronize()
    assert torch.equal(dW, dW_stored)
    Zo = O.rademacher_probes(seed, r, Cin, H, W)
    So = O.sketch(lay["X"], Zo)
    check("sketch", host(S), So, TOL_SKETCH)
    check("dW", host(dW), O.wgrad_estimate(So, lay["dY"], Zo), TOL[dtype])


def test_seeded_estimator_back_to_back_calls_give_the_same_bits():
    """r > B, Z redrawn on chip, eight calls in a row on one stream through one workspace."""
    B, Cin, Cout, H, W, r = 16, 32, 32, 96, 96, 64
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype="bf16", seed=77, z="rademacher", x="relu")
    dY = xb.to_device(lay["dY"], "bf16")
    S = torch.from_numpy(O.sketch(lay["X"], O.rademacher_probes(5, r, Cin, H, W)).astype(np.float32)).cuda()
    desc = xb.make_desc(B, Cin, Cout, H, W, r, torch.bfloat16)
    assert xb.workspace_bytes(desc, xb.OP_WGRAD_SEEDED) == xb.workspace_bytes(desc, xb.OP_WGRAD)     # no Z in the workspace
    ws = xb.workspace(xb.workspace_bytes(desc, xb.OP_WGRAD_SEEDED), dY.device)
    outs = [torch.empty((Cout, Cin, 3, 3), dtype=torch.float32, device="cuda", memory_format=torch.channels_last) for _ in range(8)]
    for o in outs:
        xb.wgrad_seeded_into(desc, S, dY, 5, o, ws)
    torch.cuda.synchronize()
    assert xb.workspace_status(ws) == 0
    assert all(torch.equal(outs[0], o) for o in outs[1:])
    Zo = O.rademacher_probes(5, r, Cin, H, W)
    check("dW", host(outs[-1]), O.wgrad_estimate(host(S), lay["dY"], Zo), TOL["bf16"])


# ------------------------------------------------------------------ standard normal probing vectors from a seed

_NP_DT = {torch.float32: "f32", torch.bfloat16: "bf16", torch.float16: "f16"}


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16, torch.float16])
@pytest.mark.parametrize("shape", [(1, 1, 1, 1), (3, 5, 4, 7), (8, 16, 9, 9), (5, 64, 6, 12), (130, 8, 5, 13), (64, 32, 40, 40)])
def test_gaussian_probes_from_seed_match_the_oracle_generator_bit_for_bit(shape, dtype):
    """Every float operation of the generator is a single IEEE operation in a fixed order, on both sides: the float
    values agree bit for bit, and so do their roundings to the 16-bit storage types."""
    r, Cin, H, W = shape
    for seed in (0, 0x1234567890ABCDEF, 2**64 - 1):
        Z = xb.xconv_probes_from_seed(seed, r, Cin, H, W, dtype, gaussian=True)
        torch.cuda.synchronize()
        want = inputs.round_to_storage(O.gaussian_probes(seed, r, Cin, H, W).astype(np.float32), _NP_DT[dtype])
        assert np.array_equal(host(Z), want.astype(np.float64))


def test_gaussian_probes_over_a_volume_are_numbered_in_memory_order():
    r, Cin, D, H, W = 3, 4, 3, 5, 6
    Z = xb.xconv_probes_from_seed(77, r, Cin, H, W, torch.float32, D=D, gaussian=True)
    torch.cuda.synchronize()
    want = O.gaussian_probes(77, r, Cin, D * H, W).reshape(r, Cin, D, H, W)
    assert np.array_equal(host(Z), want)


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("shape", [
    # B, Cin, Cout, H, W, r, K
    (4, 3, 5, 7, 9, 6, 3),           # FP32-FMA kernels, odd sizes
    (16, 64, 64, 12, 12, 24, 3),     # tensor-core kernels for 16-bit storage
    (8, 32, 32, 20, 24, 40, 3),      # r > B
    (6, 16, 32, 16, 16, 8, 5),
])
def test_algorithm_one_with_gaussian_probes_kept_as_a_seed(shape, dtype):
    """Forward: S = Z[seed]^T X; backward: dW from S, dY and the seed -- nothing but S and the seed kept between them.
    Against the oracle run on the oracle's own Z[seed] (rounded to the storage type), and bit for bit against the
    library's stored-Z calls on the library's Z[seed]."""
    B, Cin, Cout, H, W, r, K = shape
    seed = 4242 + sum(shape)
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype=dtype, seed=sum(shape) + 9, KH=K, KW=K, x="relu")
    X, dY = xb.to_device(lay["X"], dtype), xb.to_device(lay["dY"], dtype)
    Zo = inputs.round_to_storage(O.gaussian_probes(seed, r, Cin, H, W).astype(np.float32), dtype)
    S = xb.xconv_sketch_seeded(X, seed, r, gaussian=True)
    dW = xb.xconv_wgrad_seeded(S, dY, seed, Cin, kernel_size=K, gaussian=True)
    torch.cuda.synchronize()
    check("seeded sketch", host(S), O.sketch(lay["X"], Zo), TOL_SKETCH)
    check("seeded dW", host(dW), O.wgrad_estimate(host(S), lay["dY"], Zo, K, K), TOL[dtype])
    Zg = xb.xconv_probes_from_seed(seed, r, Cin, H, W, X.dtype, gaussian=True)
    assert torch.equal(S, xb.xconv_sketch(X, Zg))
    assert torch.equal(dW, xb.xconv_wgrad(S, dY, Zg, kernel_size=K))
    # twice in a row: the same bits
    assert torch.equal(dW, xb.xconv_wgrad_seeded(S, dY, seed, Cin, kernel_size=K, gaussian=True))


def test_gaussian_seeded_calls_refuse_a_short_workspace():
    import ctypes
    desc = xb.make_desc(8, 16, 16, 8, 8, 8, torch.float32)
    need = xb.workspace_bytes(desc, xb.OP_WGRAD_SEEDED_GAUSSIAN)
    assert need >= xb.workspace_bytes(desc, xb.OP_WGRAD) + 8 * 16 * 8 * 8 * 4
    ws = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    S = torch.zeros((8, 8), device="cuda")
    dY = torch.zeros((8, 16, 8, 8), device="cuda").contiguous(memory_format=torch.channels_last)
    dW = torch.full((16, 16, 3, 3), 5.0, device="cuda").contiguous(memory_format=torch.channels_last)
    st = xb.lib().xconv_wgrad_seeded_gaussian(ctypes.byref(desc), S.data_ptr(), dY.data_ptr(), 1, dW.data_ptr(),
                                              ws.data_ptr(), ws.numel(), None)
    torch.cuda.synchronize()
    assert st == 4 and float(dW.min()) == 5.0


# ------------------------------------------------------------------ block-sparse probing vectors (Eq. 7) from a seed

@pytest.mark.parametrize("gaussian", [False, True])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16, torch.float16])
@pytest.mark.parametrize("shape,p", [((1, 1, 1, 1), 0.5), ((7, 5, 4, 6), 0.3), ((40, 64, 6, 6), 0.5), ((33, 130, 3, 5), 0.125),
                                     ((6, 8, 5, 5), 1.0), ((6, 8, 5, 5), 0.0)])
def test_block_sparse_probes_from_seed_match_the_oracle_bit_for_bit(shape, p, dtype, gaussian):
    r, Cin, H, W = shape
    seed = 0xA5A5A5A5DEADBEEF ^ (r * 1000 + Cin)
    Z, keep, scale = xb.xconv_block_sparse_probes_from_seed(seed, p, r, Cin, H, W, dtype, gaussian=gaussian)
    torch.cuda.synchronize()
    Zo = inputs.round_to_storage(O.block_sparse_probes(seed, r, Cin, H, W, p, gaussian).astype(np.float32), _NP_DT[dtype])
    assert np.array_equal(host(Z), Zo.astype(np.float64))
    assert np.array_equal(keep.cpu().numpy().astype(bool), O.block_keep_mask(seed, r, Cin, p))
    np.testing.assert_allclose(scale.cpu().numpy(), O.channel_scale(O.block_sparse_probes(seed, r, Cin, H, W, p, False)),
                               rtol=1e-7, atol=0)


def test_block_sparse_probes_from_seed_through_the_layer_with_the_equation_8_scale():
    """Forward sketch and backward estimate on the probes of Eq. 7 redrawn from (seed, p) in each pass; the estimate
    against the oracle on the oracle's own redraw, with the 1/nnz scale the call returns; the mask the contraction
    takes (xconv_zero_blocks) agrees with the keep mask on 64-channel blocks."""
    B, Cin, Cout, H, W, r, p, seed = 16, 64, 64, 12, 12, 24, 0.5, 31337
    lay = inputs.make_custom(B, Cin, Cout, H, W, r, dtype="bf16", seed=5150, x="relu")
    X, dY = xb.to_device(lay["X"], "bf16"), xb.to_device(lay["dY"], "bf16")
    Z, keep, scale = xb.xconv_block_sparse_probes_from_seed(seed, p, r, Cin, H, W, torch.bfloat16)
    S = xb.xconv_sketch(X, Z)
    del Z
    Z2, keep2, scale2 = xb.xconv_block_sparse_probes_from_seed(seed, p, r, Cin, H, W, torch.bfloat16)     # backward pass
    dW = xb.xconv_wgrad(S, dY, Z2, chan_scale=scale2)
    torch.cuda.synchronize()
    assert torch.equal(keep, keep2) and torch.equal(scale, scale2)
    Zo = O.block_sparse_probes(seed, r, Cin, H, W, p)
    check("sketch", host(S), O.sketch(lay["X"], Zo), TOL_SKETCH)
    check("dW", host(dW), O.wgrad_estimate(host(S), lay["dY"], Zo, scale=O.channel_scale(Zo)), TOL["bf16"])
    zb = xb.xconv_zero_blocks(Z2).cpu().numpy().astype(bool)                  # [r, Cin/64]: all 64 channels dropped
    assert np.array_equal(zb[:, 0], ~O.block_keep_mask(seed, r, Cin, p).any(axis=1))


def test_block_sparse_probes_refuse_a_probability_outside_the_unit_interval():
    import ctypes
    desc = xb.make_desc(1, 8, 1, 4, 4, 4, torch.float32)
    Z = torch.full((4, 8, 4, 4), 7.0, device="cuda").contiguous(memory_format=torch.channels_last)
    keep = torch.zeros((4, 8), dtype=torch.uint8, device="cuda")
    scale = torch.zeros(8, device="cuda")
    for p in (-0.1, 1.5, float("nan")):
        st = xb.lib().xconv_block_sparse_probes_from_seed(ctypes.byref(desc), 1, 0, p, Z.data_ptr(), keep.data_ptr(),
                                                          scale.data_ptr(), None)
        assert st == 1
    torch.cuda.synchronize()
    assert float(Z.min()) == 7.0
