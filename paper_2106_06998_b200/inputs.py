"""Seeded synthetic inputs for the XConv layer workloads.

This module only draws and rounds numbers.  It holds none of the method's
arithmetic, so that the float64 oracle and the CUDA path can both be fed from
it without sharing anything else.

Every array is generated on the host from ``numpy.random.Generator(PCG64(seed))``
as float32, rounded once to the storage type (float32, bfloat16 or float16,
round-to-nearest-even) and handed out as a float32 array holding exactly the
stored values.  Logical index order is (batch, channel, y, x) for X and dY,
(Cout, Cin, ky, kx) for W and (probe, channel, y, x) for Z.

The five layer shapes follow the workloads the library is measured on; the
value distributions are: X standard normal, optionally rectified (a post-ReLU
activation, about half exact zeros); W normal with the fan-in ("Kaiming")
variance 2/(Cin*KH*KW) or unit variance; dY normal with a stated variance;
Z Rademacher (+1/-1) or standard normal, both of which satisfy E[z z^T] = I,
the only property the trace estimator of Eq. (3) needs.
"""
from __future__ import annotations

import numpy as np

# name -> layer description.  ``r`` lists the probing-vector counts of the sweep.
CONFIGS = {
    1: dict(B=8, Cin=16, Cout=16, H=32, W=32, dtype="f32", r=(8,),
            x="normal", w="normal", dy_var=1.0, z="rademacher"),
    2: dict(B=128, Cin=64, Cout=64, H=32, W=32, dtype="f32", r=(16, 64),
            x="relu", w="kaiming", dy_var=1e-2, z="gaussian"),
    3: dict(B=64, Cin=128, Cout=128, H=56, W=56, dtype="bf16", r=(32, 128),
            x="relu", w="kaiming", dy_var=1e-2, z="rademacher"),
    4: dict(B=16, Cin=32, Cout=32, H=256, W=256, dtype="bf16", r=(64, 256),
            x="normal", w="kaiming", dy_var=1.0, z="gaussian"),
    5: dict(B=512, Cin=256, Cout=256, H=28, W=28, dtype="bf16", r=(16, 64, 256, 1024),
            x="relu", w="kaiming", dy_var=1e-2, z="rademacher"),
}

_TENSOR_ID = {"X": 0, "W": 1, "dY": 2, "Z": 3}


def seed_for(config: int, r: int, tensor: str) -> int:
    """Seed of one tensor: 10000*config + 100*(index of r in the sweep) + tensor id."""
    rs = CONFIGS[config]["r"]
    r_index = rs.index(r) if r in rs else 50 + (r % 49)
    return 10_000 * config + 100 * r_index + _TENSOR_ID[tensor]


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result is float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """The 16-bit patterns of float32 values that are already bfloat16-representable."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def round_to_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "bf16":
        return round_bf16(a)
    if dtype == "f16":      # IEEE half precision, round to nearest even (numpy's conversion)
        return np.ascontiguousarray(a, dtype=np.float32).astype(np.float16).astype(np.float32)
    raise ValueError(f"unknown storage dtype {dtype!r}")


def draw(kind: str, shape, seed: int, dtype: str, scale: float = 1.0) -> np.ndarray:
    """One seeded tensor, rounded to ``dtype`` storage, returned as float32."""
    rng = np.random.Generator(np.random.PCG64(seed))
    if kind == "normal":
        a = rng.standard_normal(shape, dtype=np.float32)
    elif kind == "relu":
        a = np.maximum(rng.standard_normal(shape, dtype=np.float32), np.float32(0))
    elif kind == "rademacher":
        a = rng.integers(0, 2, size=shape, dtype=np.int8).astype(np.float32) * 2 - 1
    elif kind == "gaussian":
        a = rng.standard_normal(shape, dtype=np.float32)
    else:
        raise ValueError(f"unknown distribution {kind!r}")
    if scale != 1.0:
        a = a * np.float32(scale)
    return round_to_storage(a, dtype)


def layer_shape(config: int, **override) -> dict:
    c = dict(CONFIGS[config])
    c.update(override)
    return c


def make_layer(config: int, r: int, *, tensors=("X", "W", "dY", "Z"), KH: int = 3, KW: int = 3,
               **override) -> dict:
    """The tensors of one (config, r) workload (key "W" holds the weights, "width" the image width).  ``override`` may shrink B, H, W, Cin, Cout
    (used by tests that want the same recipe at a size the oracle finishes quickly)."""
    c = layer_shape(config, **override)
    B, Cin, Cout, H, W, dt = c["B"], c["Cin"], c["Cout"], c["H"], c["W"], c["dtype"]
    out = dict(config=config, r=r, B=B, Cin=Cin, Cout=Cout, H=H, width=W, KH=KH, KW=KW, dtype=dt)
    if "X" in tensors:
        out["X"] = draw(c["x"], (B, Cin, H, W), seed_for(config, r, "X"), dt)
    if "W" in tensors:
        wscale = (2.0 / (Cin * KH * KW)) ** 0.5 if c["w"] == "kaiming" else 1.0
        out["W"] = draw("normal", (Cout, Cin, KH, KW), seed_for(config, r, "W"), dt, wscale)
    if "dY" in tensors:
        out["dY"] = draw("normal", (B, Cout, H, W), seed_for(config, r, "dY"), dt, c["dy_var"] ** 0.5)
    if "Z" in tensors:
        out["Z"] = draw(c["z"], (r, Cin, H, W), seed_for(config, r, "Z"), dt)
    return out


def make_custom(B, Cin, Cout, H, W, r, *, dtype="f32", z="gaussian", x="normal", seed=0,
                KH=3, KW=3) -> dict:
    """A free-form layer for edge-case tests (odd sizes, ragged tails)."""
    out = dict(config=0, r=r, B=B, Cin=Cin, Cout=Cout, H=H, width=W, KH=KH, KW=KW, dtype=dtype)
    out["X"] = draw(x, (B, Cin, H, W), seed * 10 + 0, dtype)
    out["W"] = draw("normal", (Cout, Cin, KH, KW), seed * 10 + 1, dtype, (2.0 / (Cin * KH * KW)) ** 0.5)
    out["dY"] = draw("normal", (B, Cout, H, W), seed * 10 + 2, dtype)
    out["Z"] = draw(z, (r, Cin, H, W), seed * 10 + 3, dtype)
    return out
