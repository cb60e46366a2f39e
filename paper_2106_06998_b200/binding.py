"""Python binding of libxconv: argument marshalling only -- every step runs in the CUDA library.

Tensors are torch CUDA tensors of logical shape (batch, channel, H, W) / (Cout, Cin, KH, KW) /
(r, Cin, H, W) held in ``torch.channels_last`` memory format (the library's layout), in float32 or
bfloat16 or float16.  torch is used for device memory and streams only.  There is no fallback: if the shared
library is missing or a layer has no kernel, a RuntimeError is raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_char_p, c_float, c_int, c_int32, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libxconv.so")

XCONV_F32, XCONV_BF16, XCONV_F16 = 0, 1, 2
OP_FORWARD, OP_WGRAD, OP_DGRAD, OP_SKETCH, OP_BACKPROBE, OP_CONTRACT, OP_SKETCH_SEEDED, OP_WGRAD_SEEDED, OP_WGRAD_INDEPENDENT = 0, 1, 2, 3, 4, 5, 6, 7, 8
OP_SKETCH_SEEDED_GAUSSIAN, OP_WGRAD_SEEDED_GAUSSIAN = 9, 10
ENGINE_NAMES = {0: "none", 1: "simt_f32", 2: "tcgen05_bf16", 3: "tcgen05_f16"}
STATUS_OK = 0

# every symbol include/xconv.h declares
EXPORTS = ("xconv_workspace_bytes", "xconv_engine_for", "xconv_forward", "xconv_sketch", "xconv_wgrad",
           "xconv_dgrad", "xconv_probes_from_seed", "xconv_sketch_seeded", "xconv_wgrad_seeded", "xconv_backprobe_bytes", "xconv_backprobe", "xconv_contract", "xconv_host_arena_bytes", "xconv_sketch_wgrad_host", "xconv_sketch_static",
           "xconv_workspace_status", "xconv_selftest_wait_limit", "xconv_measure_fma_rate",
           "xconv_sketch_independent", "xconv_wgrad_independent", "xconv_zero_blocks", "xconv_zero_blocks_used",
           "xconv_gaussian_probes_from_seed", "xconv_sketch_seeded_gaussian", "xconv_wgrad_seeded_gaussian",
           "xconv_block_sparse_probes_from_seed",
           "xconv_last_launch_count", "xconv_last_cuda_error", "xconv_status_string")


class XConvDesc(Structure):
    _fields_ = [("B", c_int32), ("Cin", c_int32), ("Cout", c_int32), ("H", c_int32), ("W", c_int32),
                ("KH", c_int32), ("KW", c_int32), ("pad_h", c_int32), ("pad_w", c_int32), ("r", c_int32),
                ("dtype", c_int32), ("circular", c_int32), ("chan_scale", c_void_p),
                ("D", c_int32), ("KD", c_int32), ("pad_d", c_int32), ("zero_blocks", c_void_p)]


class XConvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().xconv_status_string(status).decode()
        extra = f" (cudaError {lib().xconv_last_cuda_error()})" if status == 5 else ""
        super().__init__(f"{where}: {msg}{extra}")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2106_06998_b200.build` "
                           "(libxconv has no CPU or library fallback)")
    L = ctypes.CDLL(LIB_PATH)
    P = POINTER(XConvDesc)
    L.xconv_workspace_bytes.argtypes = [P, c_int]; L.xconv_workspace_bytes.restype = c_size_t
    L.xconv_engine_for.argtypes = [P, c_int]; L.xconv_engine_for.restype = c_int
    L.xconv_forward.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.xconv_forward.restype = c_int
    L.xconv_sketch.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.xconv_sketch.restype = c_int
    L.xconv_probes_from_seed.argtypes = [P, ctypes.c_ulonglong, c_void_p, c_void_p]
    L.xconv_probes_from_seed.restype = c_int
    L.xconv_sketch_seeded.argtypes = [P, c_void_p, ctypes.c_ulonglong, c_void_p, c_void_p, c_size_t, c_void_p]
    L.xconv_sketch_seeded.restype = c_int
    L.xconv_wgrad_seeded.argtypes = [P, c_void_p, c_void_p, ctypes.c_ulonglong, c_void_p, c_void_p, c_size_t, c_void_p]
    L.xconv_wgrad_seeded.restype = c_int
    L.xconv_gaussian_probes_from_seed.argtypes = L.xconv_probes_from_seed.argtypes
    L.xconv_gaussian_probes_from_seed.restype = c_int
    L.xconv_sketch_seeded_gaussian.argtypes = L.xconv_sketch_seeded.argtypes
    L.xconv_sketch_seeded_gaussian.restype = c_int
    L.xconv_wgrad_seeded_gaussian.argtypes = L.xconv_wgrad_seeded.argtypes
    L.xconv_wgrad_seeded_gaussian.restype = c_int
    L.xconv_block_sparse_probes_from_seed.argtypes = [P, ctypes.c_ulonglong, c_int, ctypes.c_double, c_void_p, c_void_p,
                                                      c_void_p, c_void_p]
    L.xconv_block_sparse_probes_from_seed.restype = c_int
    L.xconv_wgrad.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.xconv_wgrad.restype = c_int
    L.xconv_sketch_independent.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p]
    L.xconv_sketch_independent.restype = c_int
    L.xconv_wgrad_independent.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.xconv_wgrad_independent.restype = c_int
    L.xconv_zero_blocks.argtypes = [P, c_void_p, c_void_p, c_void_p]
    L.xconv_zero_blocks.restype = c_int
    L.xconv_zero_blocks_used.argtypes = [P]; L.xconv_zero_blocks_used.restype = c_int
    L.xconv_backprobe_bytes.argtypes = [P]; L.xconv_backprobe_bytes.restype = c_size_t
    L.xconv_backprobe.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.xconv_backprobe.restype = c_int
    L.xconv_contract.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.xconv_contract.restype = c_int
    L.xconv_dgrad.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.xconv_dgrad.restype = c_int
    L.xconv_host_arena_bytes.argtypes = [P]; L.xconv_host_arena_bytes.restype = c_size_t
    L.xconv_sketch_wgrad_host.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t,
                                          c_void_p]
    L.xconv_sketch_wgrad_host.restype = c_int
    L.xconv_sketch_static.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p]
    L.xconv_sketch_static.restype = c_int
    L.xconv_selftest_wait_limit.argtypes = [c_void_p, c_size_t, ctypes.c_uint, c_void_p]
    L.xconv_selftest_wait_limit.restype = c_int
    L.xconv_measure_fma_rate.argtypes = [c_void_p, c_size_t, POINTER(ctypes.c_double), c_void_p]
    L.xconv_measure_fma_rate.restype = c_int
    L.xconv_workspace_status.argtypes = [c_void_p, c_void_p]; L.xconv_workspace_status.restype = c_int
    L.xconv_last_launch_count.argtypes = []; L.xconv_last_launch_count.restype = c_int
    L.xconv_last_cuda_error.argtypes = []; L.xconv_last_cuda_error.restype = c_int
    L.xconv_status_string.argtypes = [c_int]; L.xconv_status_string.restype = c_char_p
    _lib = L
    return L


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.float32:
        return XCONV_F32
    if t == torch.bfloat16:
        return XCONV_BF16
    if t == torch.float16:
        return XCONV_F16
    raise TypeError(f"libxconv stores float32, bfloat16 or float16, got {t}")


def make_desc(B, Cin, Cout, H, W, r, dtype, K=3, chan_scale=None, D=1, KD=1, zero_blocks=None,
              circular=False) -> XConvDesc:
    """Layer descriptor; D > 1 describes a volume (tensors gain a depth axis), KD its kernel depth (1 or 3);
    zero_blocks: uint8 CUDA tensor [r, Cin/64] marking the all-zero 64-channel blocks of the probing vectors;
    circular: the paper's circular shifts T_k (circular padding) instead of zero padding, planar layers only."""
    code = dtype if isinstance(dtype, int) else _dtype_code(dtype)
    cs = chan_scale.data_ptr() if chan_scale is not None else None
    zb = None
    if zero_blocks is not None:
        if (zero_blocks.dtype != torch.uint8 or not zero_blocks.is_cuda or not zero_blocks.is_contiguous()
                or Cin % 64 != 0 or tuple(zero_blocks.shape) != (r, Cin // 64)):
            raise ValueError("zero_blocks must be a contiguous uint8 CUDA tensor [r, Cin/64] (Cin a multiple of 64)")
        zb = zero_blocks.data_ptr()
    return XConvDesc(B, Cin, Cout, H, W, K, K, (K - 1) // 2, (K - 1) // 2, r, code, 1 if circular else 0, cs, D, KD, (KD - 1) // 2, zb)


def zero_blocks_used(desc: XConvDesc) -> bool:
    """Whether the contraction of this layer skips the blocks desc.zero_blocks names (else the field is ignored)."""
    return bool(lib().xconv_zero_blocks_used(ctypes.byref(desc)))


def xconv_zero_blocks(Z: torch.Tensor) -> torch.Tensor:
    """uint8 [r, Cin/64]: 1 where the 64-channel block of a probing vector holds only zeros (the mask that
    xconv_contract / xconv_wgrad take as zero_blocks)."""
    _cl(Z, "Z")
    r, Cin = Z.shape[:2]
    D, H, W = _geo(Z)
    if Cin % 64 != 0:
        raise ValueError("Cin must be a multiple of 64")
    desc = make_desc(1, Cin, 64, H, W, r, Z.dtype, D=D)
    mask = torch.empty((r, Cin // 64), dtype=torch.uint8, device=Z.device)
    _check(lib().xconv_zero_blocks(ctypes.byref(desc), Z.data_ptr(), mask.data_ptr(), _stream()), "xconv_zero_blocks")
    return mask


def _cl(t: torch.Tensor, name: str) -> torch.Tensor:
    """Checks the layout: 4-d tensors in channels_last, 5-d tensors (volumes) in channels_last_3d."""
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    fmt = {4: torch.channels_last, 5: torch.channels_last_3d}.get(t.dim())
    if fmt is None or not t.is_contiguous(memory_format=fmt):
        raise ValueError(f"{name} must be a 4-d tensor in torch.channels_last or a 5-d tensor in "
                         "torch.channels_last_3d memory format")
    return t


def _geo(t: torch.Tensor):
    """(D, H, W) of a 4-d (planar, D = 1) or 5-d (volume) tensor."""
    return (1, t.shape[2], t.shape[3]) if t.dim() == 4 else (t.shape[2], t.shape[3], t.shape[4])


def _like(shape_head, geo, dim, **kw):
    """An empty tensor (head..., [D,] H, W) in the channels-last format of a `dim`-d tensor."""
    D, H, W = geo
    shape = tuple(shape_head) + ((H, W) if dim == 4 else (D, H, W))
    return torch.empty(shape, memory_format=torch.channels_last if dim == 4 else torch.channels_last_3d, **kw)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


_ws_cache: dict = {}


def workspace(nbytes: int, device) -> torch.Tensor:
    """A cached scratch buffer of at least ``nbytes`` on ``device`` (grown on demand)."""
    key = str(device)
    buf = _ws_cache.get(key)
    if buf is None or buf.numel() < nbytes:
        buf = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)
        _ws_cache[key] = buf
    return buf


def workspace_bytes(desc: XConvDesc, op: int) -> int:
    return lib().xconv_workspace_bytes(ctypes.byref(desc), op)


def engine_for(desc: XConvDesc, op: int) -> str:
    return ENGINE_NAMES[lib().xconv_engine_for(ctypes.byref(desc), op)]


def _check(status: int, where: str):
    if status != STATUS_OK:
        raise XConvError(status, where)


# ------------------------------------------------------------------ raw calls (preallocated outputs)

def sketch_into(desc, X, Z, S, ws):
    _check(lib().xconv_sketch(ctypes.byref(desc), X.data_ptr(), Z.data_ptr(), S.data_ptr(), ws.data_ptr(),
                              ws.numel(), _stream()), "xconv_sketch")


def sketch_seeded_into(desc, X, seed, S, ws):
    _check(lib().xconv_sketch_seeded(ctypes.byref(desc), X.data_ptr(), seed, S.data_ptr(), ws.data_ptr(),
                                     ws.numel(), _stream()), "xconv_sketch_seeded")


def wgrad_seeded_into(desc, S, dY, seed, dW, ws):
    _check(lib().xconv_wgrad_seeded(ctypes.byref(desc), S.data_ptr(), dY.data_ptr(), seed, dW.data_ptr(),
                                    ws.data_ptr(), ws.numel(), _stream()), "xconv_wgrad_seeded")


def forward_into(desc, X, W, Z, Y, S, ws):
    _check(lib().xconv_forward(ctypes.byref(desc), X.data_ptr(), W.data_ptr(), Z.data_ptr(), Y.data_ptr(),
                               S.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "xconv_forward")


def wgrad_into(desc, S, dY, Z, dW, ws):
    _check(lib().xconv_wgrad(ctypes.byref(desc), S.data_ptr(), dY.data_ptr(), Z.data_ptr(), dW.data_ptr(),
                             ws.data_ptr(), ws.numel(), _stream()), "xconv_wgrad")


def backprobe_into(desc, S, dY, L, ws):
    _check(lib().xconv_backprobe(ctypes.byref(desc), S.data_ptr(), dY.data_ptr(), L.data_ptr(), ws.data_ptr(),
                                 ws.numel(), _stream()), "xconv_backprobe")


def contract_into(desc, L, Z, dW, ws):
    _check(lib().xconv_contract(ctypes.byref(desc), L.data_ptr(), Z.data_ptr(), dW.data_ptr(), ws.data_ptr(),
                                ws.numel(), _stream()), "xconv_contract")


def dgrad_into(desc, dY, W, dX, ws):
    _check(lib().xconv_dgrad(ctypes.byref(desc), dY.data_ptr(), W.data_ptr(), dX.data_ptr(), ws.data_ptr(),
                             ws.numel(), _stream()), "xconv_dgrad")


def workspace_status(ws) -> int:
    return lib().xconv_workspace_status(ws.data_ptr(), _stream())


def measure_fma_rate(device="cuda") -> float:
    """FP32 FMA rate of the device in TFLOP/s, measured by the library's register-only FMA kernel."""
    scratch = torch.empty(148 * 16 * 256, dtype=torch.float32, device=device)
    out = ctypes.c_double(0.0)
    _check(lib().xconv_measure_fma_rate(scratch.data_ptr(), scratch.numel() * 4, ctypes.byref(out), _stream()),
           "xconv_measure_fma_rate")
    return float(out.value)


def last_launch_count() -> int:
    return lib().xconv_last_launch_count()


# ------------------------------------------------------------------ same names as the C ABI

def xconv_sketch(X: torch.Tensor, Z: torch.Tensor) -> torch.Tensor:
    """S = Z^T X (Algorithm 1 forward step 3): float32 tensor [r, B].  X (B, Cin, [D,] H, W), Z (r, Cin, [D,] H, W)."""
    _cl(X, "X"); _cl(Z, "Z")
    B, Cin = X.shape[:2]
    D, H, W = _geo(X)
    r = Z.shape[0]
    if tuple(Z.shape[1:]) != tuple(X.shape[1:]) or Z.dtype != X.dtype:
        raise ValueError("Z must be (r, Cin, [D,] H, W) in X's dtype")
    desc = make_desc(B, Cin, 1, H, W, r, X.dtype, D=D)
    S = torch.empty((r, B), dtype=torch.float32, device=X.device)
    ws = workspace(workspace_bytes(desc, OP_SKETCH), X.device)
    sketch_into(desc, X, Z, S, ws)
    return S


def xconv_probes_from_seed(seed: int, r: int, Cin: int, H: int, W: int, dtype=torch.bfloat16, device="cuda",
                           D: int = 1, gaussian: bool = False) -> torch.Tensor:
    """Z[seed]: Rademacher (or, with ``gaussian``, standard normal) probing vectors (r, Cin, H, W) (volumes, D > 1:
    (r, Cin, D, H, W)), channels-last, from the library's Philox streams."""
    desc = make_desc(1, Cin, 1, H, W, r, dtype, D=D)
    Z = _like((r, Cin), (D, H, W), 5 if D > 1 else 4, dtype=dtype, device=device)
    fn = lib().xconv_gaussian_probes_from_seed if gaussian else lib().xconv_probes_from_seed
    _check(fn(ctypes.byref(desc), seed, Z.data_ptr(), _stream()), "xconv_probes_from_seed")
    return Z


def xconv_block_sparse_probes_from_seed(seed: int, p: float, r: int, Cin: int, H: int, W: int, dtype=torch.bfloat16,
                                        device="cuda", D: int = 1, gaussian: bool = False):
    """The block-sparse probing vectors of Eq. 7 from a seed: (Z, keep [r, Cin] uint8, chan_scale [Cin] float32 =
    1/nnz(Z_n) of Eq. 8).  Blocks are kept with probability p; the kept ones are those of the dense probes of the seed."""
    desc = make_desc(1, Cin, 1, H, W, r, dtype, D=D)
    Z = _like((r, Cin), (D, H, W), 5 if D > 1 else 4, dtype=dtype, device=device)
    keep = torch.empty((r, Cin), dtype=torch.uint8, device=device)
    scale = torch.empty((Cin,), dtype=torch.float32, device=device)
    _check(lib().xconv_block_sparse_probes_from_seed(ctypes.byref(desc), seed, 1 if gaussian else 0, float(p), Z.data_ptr(),
                                                     keep.data_ptr(), scale.data_ptr(), _stream()),
           "xconv_block_sparse_probes_from_seed")
    return Z, keep, scale


def xconv_sketch_seeded(X: torch.Tensor, seed: int, r: int, gaussian: bool = False) -> torch.Tensor:
    """S = Z[seed]^T X without a stored Z (Algorithm 1 keeps the seed): float32 tensor [r, B].  ``gaussian``: standard
    normal probing vectors (drawn into the workspace) instead of Rademacher ones."""
    _cl(X, "X")
    B, Cin = X.shape[:2]
    D, H, W = _geo(X)
    desc = make_desc(B, Cin, 1, H, W, r, X.dtype, D=D)
    S = torch.empty((r, B), dtype=torch.float32, device=X.device)
    if gaussian:
        ws = workspace(workspace_bytes(desc, OP_SKETCH_SEEDED_GAUSSIAN), X.device)
        _check(lib().xconv_sketch_seeded_gaussian(ctypes.byref(desc), X.data_ptr(), seed, S.data_ptr(), ws.data_ptr(),
                                                  ws.numel(), _stream()), "xconv_sketch_seeded_gaussian")
        return S
    ws = workspace(workspace_bytes(desc, OP_SKETCH_SEEDED), X.device)
    sketch_seeded_into(desc, X, seed, S, ws)
    return S


def xconv_wgrad_seeded(sketch: torch.Tensor, dY: torch.Tensor, seed: int, Cin: int, kernel_size: int = 3,
                       kernel_depth: int = 1, circular: bool = False, gaussian: bool = False) -> torch.Tensor:
    """dW estimate from the sketch and the seed (Algorithm 1 backward steps 2-4): Z[seed] is redrawn on chip or into
    the workspace, never passed in.  float32 (Cout, Cin, [KD,] K, K), channels-last.  ``gaussian``: standard normal
    probing vectors instead of Rademacher ones."""
    _cl(dY, "dY")
    B, Cout = dY.shape[:2]
    D, H, Wd = _geo(dY)
    r = sketch.shape[0]
    if tuple(sketch.shape) != (r, B) or sketch.dtype != torch.float32 or not sketch.is_contiguous():
        raise ValueError("sketch must be a contiguous float32 [r, B] tensor")
    K = kernel_size
    desc = make_desc(B, Cin, Cout, H, Wd, r, dY.dtype, K, D=D, KD=kernel_depth, circular=circular)
    dW = _like((Cout, Cin), (kernel_depth, K, K), dY.dim(), dtype=torch.float32, device=dY.device)
    fn = lib().xconv_wgrad_seeded_gaussian if gaussian else lib().xconv_wgrad_seeded
    ws = workspace(workspace_bytes(desc, OP_WGRAD_SEEDED_GAUSSIAN if gaussian else OP_WGRAD_SEEDED), dY.device)
    _check(fn(ctypes.byref(desc), sketch.data_ptr(), dY.data_ptr(), seed, dW.data_ptr(),
              ws.data_ptr(), ws.numel(), _stream()), "xconv_wgrad_seeded")
    return dW


STATIC_SCRATCH_FLOATS = 1 << 20


def xconv_sketch_static(X: torch.Tensor, Z: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """S = Z^T X through the entry point that takes no workspace and allocates nothing in the library
    (its partial sums live in a fixed 4 MiB array inside the library image).  For callers that may not
    allocate device memory at this point; pass ``out`` to avoid even the output allocation here.
    Raises XConvError (workspace too small) when r*B exceeds STATIC_SCRATCH_FLOATS."""
    _cl(X, "X"); _cl(Z, "Z")
    B, Cin, H, W = X.shape
    r = Z.shape[0]
    if tuple(Z.shape[1:]) != (Cin, H, W) or Z.dtype != X.dtype:
        raise ValueError("Z must be (r, Cin, H, W) in X's dtype")
    desc = make_desc(B, Cin, 1, H, W, r, X.dtype)
    S = out if out is not None else torch.empty((r, B), dtype=torch.float32, device=X.device)
    _check(lib().xconv_sketch_static(ctypes.byref(desc), X.data_ptr(), Z.data_ptr(), S.data_ptr(), _stream()),
           "xconv_sketch_static")
    return S


def xconv_forward(X: torch.Tensor, W: torch.Tensor, Z: torch.Tensor, circular: bool = False):
    """Y = conv(X, W) and the sketch S = Z^T X (Algorithm 1 forward steps 1 and 3).  5-d tensors are volumes."""
    _cl(X, "X"); _cl(W, "W"); _cl(Z, "Z")
    B, Cin = X.shape[:2]
    D, H, Wd = _geo(X)
    Cout, K = W.shape[0], W.shape[-1]
    KD = W.shape[2] if W.dim() == 5 else 1
    r = Z.shape[0]
    if (W.shape[1] != Cin or W.dim() != X.dim() or tuple(Z.shape[1:]) != tuple(X.shape[1:]) or W.dtype != X.dtype
            or Z.dtype != X.dtype):
        raise ValueError("shape or dtype mismatch between X, W and Z")
    desc = make_desc(B, Cin, Cout, H, Wd, r, X.dtype, K, D=D, KD=KD, circular=circular)
    Y = _like((B, Cout), (D, H, Wd), X.dim(), dtype=X.dtype, device=X.device)
    S = torch.empty((r, B), dtype=torch.float32, device=X.device)
    ws = workspace(workspace_bytes(desc, OP_FORWARD), X.device)
    forward_into(desc, X, W, Z, Y, S, ws)
    return Y, S


def xconv_wgrad(sketch: torch.Tensor, dY: torch.Tensor, Z: torch.Tensor, kernel_size: int = 3,
                chan_scale: torch.Tensor | None = None, kernel_depth: int = 1,
                zero_blocks: torch.Tensor | None = None, circular: bool = False) -> torch.Tensor:
    """dW estimate (Algorithm 1 backward steps 3-4): float32 (Cout, Cin, [KD,] K, K), channels-last."""
    _cl(dY, "dY"); _cl(Z, "Z")
    B, Cout = dY.shape[:2]
    D, H, Wd = _geo(dY)
    r, Cin = Z.shape[0], Z.shape[1]
    if tuple(sketch.shape) != (r, B) or sketch.dtype != torch.float32 or not sketch.is_contiguous():
        raise ValueError("sketch must be a contiguous float32 [r, B] tensor")
    if tuple(Z.shape[2:]) != tuple(dY.shape[2:]) or Z.dtype != dY.dtype:
        raise ValueError("shape or dtype mismatch between dY and Z")
    if chan_scale is not None and (chan_scale.dtype != torch.float32 or chan_scale.numel() != Cin):
        raise ValueError("chan_scale must hold Cin float32 values")
    K = kernel_size
    desc = make_desc(B, Cin, Cout, H, Wd, r, dY.dtype, K, chan_scale, D=D, KD=kernel_depth, zero_blocks=zero_blocks,
                     circular=circular)
    dW = _like((Cout, Cin), (kernel_depth, K, K), dY.dim(), dtype=torch.float32, device=dY.device)
    ws = workspace(workspace_bytes(desc, OP_WGRAD), dY.device)
    wgrad_into(desc, sketch, dY, Z, dW, ws)
    return dW


def xconv_sketch_independent(X: torch.Tensor, Z: torch.Tensor) -> torch.Tensor:
    """Per-channel sketch S[j, n, b] = <Z[j, n], X[b, n]> (estimator applied to each channel pair on its own):
    float32 tensor [r, Cin, B]."""
    _cl(X, "X"); _cl(Z, "Z")
    B, Cin = X.shape[:2]
    D, H, W = _geo(X)
    r = Z.shape[0]
    if tuple(Z.shape[1:]) != tuple(X.shape[1:]) or Z.dtype != X.dtype:
        raise ValueError("Z must be (r, Cin, [D,] H, W) in X's dtype")
    desc = make_desc(B, Cin, 1, H, W, r, X.dtype, D=D)
    S = torch.empty((r, Cin, B), dtype=torch.float32, device=X.device)
    _check(lib().xconv_sketch_independent(ctypes.byref(desc), X.data_ptr(), Z.data_ptr(), S.data_ptr(), _stream()),
           "xconv_sketch_independent")
    return S


def xconv_wgrad_independent(sketch: torch.Tensor, dY: torch.Tensor, Z: torch.Tensor, kernel_size: int = 3,
                            kernel_depth: int = 1, circular: bool = False) -> torch.Tensor:
    """dW estimate per channel pair from the per-channel sketch: float32 (Cout, Cin, [KD,] K, K), channels-last."""
    _cl(dY, "dY"); _cl(Z, "Z")
    B, Cout = dY.shape[:2]
    D, H, Wd = _geo(dY)
    r, Cin = Z.shape[0], Z.shape[1]
    if tuple(sketch.shape) != (r, Cin, B) or sketch.dtype != torch.float32 or not sketch.is_contiguous():
        raise ValueError("sketch must be a contiguous float32 [r, Cin, B] tensor")
    if tuple(Z.shape[2:]) != tuple(dY.shape[2:]) or Z.dtype != dY.dtype:
        raise ValueError("shape or dtype mismatch between dY and Z")
    K = kernel_size
    desc = make_desc(B, Cin, Cout, H, Wd, r, dY.dtype, K, D=D, KD=kernel_depth, circular=circular)
    dW = _like((Cout, Cin), (kernel_depth, K, K), dY.dim(), dtype=torch.float32, device=dY.device)
    ws = workspace(workspace_bytes(desc, OP_WGRAD_INDEPENDENT), dY.device)
    _check(lib().xconv_wgrad_independent(ctypes.byref(desc), sketch.data_ptr(), dY.data_ptr(), Z.data_ptr(),
                                         dW.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "xconv_wgrad_independent")
    return dW


def xconv_backprobe(sketch: torch.Tensor, dY: torch.Tensor) -> torch.Tensor:
    """L = S dY^T (Algorithm 1 backward step 3): (r, Cout, [D,] H, W) in dY's dtype, channels-last."""
    _cl(dY, "dY")
    B, Cout = dY.shape[:2]
    D, H, Wd = _geo(dY)
    r = sketch.shape[0]
    if tuple(sketch.shape) != (r, B) or sketch.dtype != torch.float32 or not sketch.is_contiguous():
        raise ValueError("sketch must be a contiguous float32 [r, B] tensor")
    desc = make_desc(B, 1, Cout, H, Wd, r, dY.dtype, D=D)
    L = _like((r, Cout), (D, H, Wd), dY.dim(), dtype=dY.dtype, device=dY.device)
    ws = workspace(workspace_bytes(desc, OP_WGRAD), dY.device)
    backprobe_into(desc, sketch, dY, L, ws)
    return L


def xconv_contract(L: torch.Tensor, Z: torch.Tensor, kernel_size: int = 3,
                   chan_scale: torch.Tensor | None = None, kernel_depth: int = 1,
                   zero_blocks: torch.Tensor | None = None, circular: bool = False) -> torch.Tensor:
    """dW[m,n,k] = scale[n] * sum L[j,m,.] Z[j,n,.+k] (Algorithm 1 backward step 4)."""
    _cl(L, "L"); _cl(Z, "Z")
    r, Cout = L.shape[:2]
    D, H, Wd = _geo(L)
    Cin = Z.shape[1]
    if Z.shape[0] != r or tuple(Z.shape[2:]) != tuple(L.shape[2:]) or Z.dtype != L.dtype:
        raise ValueError("shape or dtype mismatch between L and Z")
    K = kernel_size
    desc = make_desc(1, Cin, Cout, H, Wd, r, L.dtype, K, chan_scale, D=D, KD=kernel_depth, zero_blocks=zero_blocks,
                     circular=circular)
    dW = _like((Cout, Cin), (kernel_depth, K, K), L.dim(), dtype=torch.float32, device=L.device)
    ws = workspace(workspace_bytes(desc, OP_WGRAD), L.device)
    contract_into(desc, L, Z, dW, ws)
    return dW


def xconv_dgrad(dY: torch.Tensor, W: torch.Tensor, circular: bool = False) -> torch.Tensor:
    """Exact dX (transposed convolution)."""
    _cl(dY, "dY"); _cl(W, "W")
    B, Cout = dY.shape[:2]
    D, H, Wd = _geo(dY)
    Cin, K = W.shape[1], W.shape[-1]
    KD = W.shape[2] if W.dim() == 5 else 1
    if W.shape[0] != Cout or W.dtype != dY.dtype or W.dim() != dY.dim():
        raise ValueError("shape or dtype mismatch between dY and W")
    desc = make_desc(B, Cin, Cout, H, Wd, 1, dY.dtype, K, D=D, KD=KD, circular=circular)
    dX = _like((B, Cin), (D, H, Wd), dY.dim(), dtype=dY.dtype, device=dY.device)
    ws = workspace(workspace_bytes(desc, OP_DGRAD), dY.device)
    dgrad_into(desc, dY, W, dX, ws)
    return dX


def host_arena_bytes(desc: XConvDesc) -> int:
    return lib().xconv_host_arena_bytes(ctypes.byref(desc))


def xconv_sketch_wgrad_host(desc: XConvDesc, hX, hdY, hZ, hS, hdW, arena: torch.Tensor):
    """Sketch + dW estimate from host (ideally pinned) tensors; copies are inside the call."""
    _check(lib().xconv_sketch_wgrad_host(ctypes.byref(desc), hX.data_ptr(), hdY.data_ptr(), hZ.data_ptr(),
                                         hS.data_ptr(), hdW.data_ptr(), arena.data_ptr(), arena.numel(), _stream()),
           "xconv_sketch_wgrad_host")


def to_device(a, dtype: str, device="cuda") -> torch.Tensor:
    """Host float32 array (logical NCHW or NCDHW, already rounded to ``dtype``) -> channels-last device tensor."""
    t = torch.from_numpy(a).to(device)
    if dtype == "bf16":
        t = t.to(torch.bfloat16)
    elif dtype == "f16":
        t = t.to(torch.float16)
    return t.contiguous(memory_format=torch.channels_last if t.dim() == 4 else torch.channels_last_3d)
