"""Helpers shared by the GPU parity tests: run one layer through libxconv and through the oracle."""
import numpy as np
import torch

from oracle import xconv_oracle as O
from paper_2106_06998_b200 import binding as xb

TOL = {"f32": 1e-5, "bf16": 1e-2}      # relative Frobenius error, per storage type


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
    err = O.rel_fro(got, want)
    assert err <= tol, f"{name}: relative Frobenius error {err:.3e} > {tol:.1e}"
    return err
