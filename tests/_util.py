"""Helpers shared by the GPU parity tests: run one layer through libxconv and through the oracle."""
import numpy as np
import torch

from oracle import xconv_oracle as O
from paper_2106_06998_b200 import binding as xb

# Relative Frobenius error per storage type, for everything that inherits a rounding of the storage
# type (Y, dX, L are rounded to it; dW inherits the roundings of S and L).
TOL = {"f32": 1e-5, "bf16": 1e-2, "f16": 2e-3}
# The sketch inherits no rounding: products of two bfloat16 (or float16) values are exact in float, so
# only the float accumulation order differs from the oracle, whatever the storage type.
TOL_SKETCH = 1e-5


def sketch_tol(K):
    """Bar for a sketch whose reduction runs over K = H*W*Cin terms.  The tensor cores add the 16 products of a
    k-step to a float accumulator that is not rounded to nearest, so the error grows with the number of k-steps
    per accumulator (K / 16 / k-splits: 885 on the 2^21-term reduction of the high-resolution workload, where
    1.6e-5 was measured).  1e-5 up to 2^20 terms, 4e-5 beyond."""
    return TOL_SKETCH if K <= (1 << 20) else 4e-5
# Element-wise companion of the Frobenius bound: no single element may be off by more than
# MAX_C * tol * rms(want).  Independent rounding errors at the Frobenius bound itself would peak near 5 rms
# errors over a million elements, so 8 leaves room for them, while one wholly wrong element (an error of
# the order of rms(want)) exceeds the bound by a factor 1 / (8 tol) >= 12.
MAX_C = 8.0


def dev(lay, names=("X", "W", "dY", "Z")):
    return {k: xb.to_device(lay[k], lay["dtype"]) for k in names if k in lay}


def host(t):
    """Device tensor (logical NCHW view) -> float64 numpy array."""
    return t.detach().float().cpu().numpy().astype(np.float64)


def sketch_oracle_chunked(X, Z, chunk=32):
    """Rows of the sketch are independent per probe: call the oracle on slabs of probes to bound memory."""
    X64 = np.asarray(X, np.float64)
    return np.concatenate([O.sketch(X64, Z[j:j + chunk]) for j in range(0, Z.shape[0], chunk)], axis=0)


def check(name, got, want, tol):
    """Relative Frobenius error <= tol, and every element within MAX_C * tol * rms(want)."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    assert got.shape == want.shape, f"{name}: shape {got.shape} != {want.shape}"
    err = O.rel_fro(got, want)
    assert err <= tol, f"{name}: relative Frobenius error {err:.3e} > {tol:.1e}"
    rms = float(np.sqrt(np.mean(want ** 2))) if want.size else 0.0
    worst = float(np.max(np.abs(got - want))) if want.size else 0.0
    assert worst <= MAX_C * tol * rms, (f"{name}: largest element error {worst:.3e} > {MAX_C:g} * {tol:.1e} * "
                                        f"rms(want) = {MAX_C * tol * rms:.3e}")
    return err
