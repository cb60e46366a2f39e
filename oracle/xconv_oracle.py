"""Float64 CPU oracle for the XConv layer (test infrastructure, not product code).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may use this
module.  It shares no code with the CUDA path and imports nothing from it.

Everything is plain numpy in float64 on logical (batch, channel, y, x) arrays.
Where a step is a dense contraction, ``numpy.matmul`` / ``numpy.einsum`` serves as
that step; there is no blocking, fusion or reordering beyond what the formulas
state.

Notation (Section 3, "Single channel case" and "Multi-channel case"):
  B batch, Cin/Cout channels, N = H*W pixels, r probing vectors,
  X  [B, Cin, H, W]     layer input
  dY [B, Cout, H, W]    back-propagated residual (delta Y)
  W  [Cout, Cin, KH, KW] weights; the i-th weight has offset k(i) = (ky-ph, kx-pw)
  Z  [r, Cin, H, W]     probing vectors (column j of the paper's Z, reshaped)
  S  [r, B]             the sketch, the paper's X-bar = Z^T X   (text after Eq. 4, Algorithm 1 forward step 3)
  L  [r, Cout, H, W]    backward probe L = X-bar dY^T           (Algorithm 1 backward step 3)

Shift operator.  The paper's T_k is a circular shift; every layer this library is
used on is a zero-padded convolution, for which the matching operator is the
truncating shift (out-of-range pixels read as zero).  ``circular=True`` selects the
paper's literal operator and is used as a second self-check.  In both cases
  (shift(A, dy, dx))[..., y, x] = A[..., y+dy, x+dx].

Direction of the shift in the gradient.  From Y = sum_i w_i T_k(i) X with
(T_k X)[q] = X[q + k], the exact weight gradient is
  dw_i = sum_{b,q} dY[q, b] X[q + k(i), b] = tr(X dY^T S_k),  (S_k z)[q] = z[q + k],
so the paper's T_{-k(i)} in Eq. (2) acts on a probing vector as z -> z[. + k(i)]:
output pixel q pairs with the probe value at input pixel q + k(i).

Pinned by tests/test_oracle_pins.py: brute-force loops and finite differences
(conv_forward, dw_exact, dx_exact), exact recovery with an orthogonal probe basis,
unbiasedness, the closed-form Hutchinson variance, Proposition 1's bound and the
literal block-matrix estimator of Eq. (6) (sketch, backprobe, wgrad_estimate).
philox4x32_10 and rademacher_probes (probing vectors redrawn from a stored seed, Algorithm 1) are pinned
by the generator's published known-answer vectors (tests/golden/philox4x32_10_kat.txt), by the
balance and independence of the signs, and by the unbiasedness of the estimator run on them.
gaussian_probes (standard normal probing vectors from a stored seed: Box-Muller on Philox words, with float32 series
for the logarithm, sine and cosine that a GPU can repeat bit for bit) is pinned by numpy's float64 functions on the
same arguments, by a float64 recomputation of single entries from the stated definition, by its moments, a
Kolmogorov-Smirnov test, E[z z^T] = I, and the unbiasedness of the estimator run on it.
block_keep_mask and block_sparse_probes (the block-sparse probing vectors of Eq. 7 from a seed) are pinned by a
word-by-word recomputation of the mask from the stated definition, by the kept share and the independence of the
mask bits, by the limits p = 0 and p = 1, and by the unbiasedness of the estimator with the Eq. 8 scale on them.
sketch_independent and wgrad_estimate_independent (the estimator applied to each channel pair on its own) are
pinned by exact recovery with one orthogonal basis per channel, by unbiasedness with the crosstalk-free
Hutchinson variance, and by their reduction to the multi-channel functions for a single input channel.
The functions for volumes (shift3, conv_forward3d, dw_exact3d, dx_exact3d, wgrad_contract3d, wgrad_estimate3d) are
pinned by brute-force loops, by their reduction to the two-dimensional functions at depth 1, and by exact recovery.
rel_fro, the metric every parity check passes through, is pinned on a hand-computed pair.
oracle/xconv_oracle.c states the layer's formulas a second time as plain C loop nests (loader: oracle/c_oracle.py); the two
are compared on random layers and the C one is pinned by the same brute-force loops and by exact recovery.
No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def _pads(KH, KW, pad):
    if pad is None:
        return (KH - 1) // 2, (KW - 1) // 2
    return pad


def shift(A: np.ndarray, dy: int, dx: int, circular: bool = False) -> np.ndarray:
    """(shift A)[..., y, x] = A[..., y+dy, x+dx]; zero outside the image unless ``circular``.

    Section 3, text after Eq. (1): the i-th weight applies a shift with offset k(i).
    """
    A = np.asarray(A, dtype=F64)
    if circular:
        return np.roll(A, shift=(-dy, -dx), axis=(-2, -1))
    H, W = A.shape[-2], A.shape[-1]
    out = np.zeros_like(A)
    y0, y1 = max(0, -dy), min(H, H - dy)
    x0, x1 = max(0, -dx), min(W, W - dx)
    if y0 < y1 and x0 < x1:
        out[..., y0:y1, x0:x1] = A[..., y0 + dy:y1 + dy, x0 + dx:x1 + dx]
    return out


def conv_forward(X, W, pad=None, circular=False):
    """Y^m = sum_n W^{n,m} X^n with W^{n,m} = sum_i w_i^{n,m} T_k(i)   (Eq. 5; Algorithm 1 forward step 1).

    Y[b,m,y,x] = sum_{n,ky,kx} W[m,n,ky,kx] X[b,n,y+ky-ph,x+kx-pw]  (cross-correlation, stride 1).
    """
    X = np.asarray(X, F64)
    W = np.asarray(W, F64)
    Cout, Cin, KH, KW = W.shape
    ph, pw = _pads(KH, KW, pad)
    Y = np.zeros((X.shape[0], Cout) + X.shape[2:], F64)
    for ky in range(KH):
        for kx in range(KW):
            Xs = shift(X, ky - ph, kx - pw, circular)
            Y += np.einsum("mn,bnyx->bmyx", W[:, :, ky, kx], Xs)
    return Y


def dw_exact(X, dY, KH=3, KW=3, pad=None, circular=False):
    """Exact weight gradient dw_i^{n,m} = tr(X^n (dY^m)^T T_{-k(i)})   (Eq. 2 and the sentence after Eq. 5).

    dW[m,n,ky,kx] = sum_{b,y,x} dY[b,m,y,x] X[b,n,y+ky-ph,x+kx-pw].
    """
    X = np.asarray(X, F64)
    dY = np.asarray(dY, F64)
    ph, pw = _pads(KH, KW, pad)
    dW = np.zeros((dY.shape[1], X.shape[1], KH, KW), F64)
    for ky in range(KH):
        for kx in range(KW):
            Xs = shift(X, ky - ph, kx - pw, circular)
            dW[:, :, ky, kx] = np.einsum("bmyx,bnyx->mn", dY, Xs)
    return dW


def dx_exact(dY, W, pad=None, circular=False):
    """Exact input gradient: the adjoint of ``conv_forward`` in X (standard back-propagation,
    which the method leaves untouched -- abstract and Section 1).

    dX[b,n,u,v] = sum_{m,ky,kx} W[m,n,ky,kx] dY[b,m,u-ky+ph,v-kx+pw].
    """
    dY = np.asarray(dY, F64)
    W = np.asarray(W, F64)
    Cout, Cin, KH, KW = W.shape
    ph, pw = _pads(KH, KW, pad)
    dX = np.zeros((dY.shape[0], Cin) + dY.shape[2:], F64)
    for ky in range(KH):
        for kx in range(KW):
            dYs = shift(dY, -(ky - ph), -(kx - pw), circular)
            dX += np.einsum("mn,bmyx->bnyx", W[:, :, ky, kx], dYs)
    return dX


def sketch(X, Z):
    """X-bar = Z^T X in R^{r x B}: step (i) of the three-step procedure after Eq. (6);
    Algorithm 1 forward step 3.   S[j,b] = sum_{n,y,x} Z[j,n,y,x] X[b,n,y,x]."""
    X = np.asarray(X, F64)
    Z = np.asarray(Z, F64)
    return Z.reshape(Z.shape[0], -1) @ X.reshape(X.shape[0], -1).T


def backprobe(S, dY):
    """L = X-bar dY^T (Algorithm 1 backward step 3), reshaped per output channel (step ii).

    L[j,m,y,x] = sum_b S[j,b] dY[b,m,y,x]."""
    S = np.asarray(S, F64)
    dY = np.asarray(dY, F64)
    L = S @ dY.reshape(dY.shape[0], -1)
    return L.reshape((S.shape[0],) + dY.shape[1:])


def channel_scale(Z):
    """Scale of the estimator per input channel: 1/nnz(Z_n), nnz = number of probing vectors
    whose block n is not identically zero (Eq. 8).  For dense probes this is 1/r (Eq. 6).
    A channel with no non-zero block gets scale 0 (its estimate is then 0)."""
    Z = np.asarray(Z, F64)
    nnz = np.count_nonzero(np.any(Z.reshape(Z.shape[0], Z.shape[1], -1) != 0, axis=2), axis=0)
    return np.where(nnz > 0, 1.0 / np.maximum(nnz, 1), 0.0)


def wgrad_contract(L, Z, KH=3, KW=3, pad=None, circular=False, scale=None):
    """Step (iii): probe each block from the left, dw_i = (1/r) tr(L T_{-k(i)} Z)
    (Eq. 6 block by block; Algorithm 1 backward step 4).

    dW[m,n,ky,kx] = scale[n] * sum_{j,y,x} L[j,m,y,x] Z[j,n,y+ky-ph,x+kx-pw],
    scale = 1/r unless given (Eq. 8 uses 1/nnz(Z_n))."""
    L = np.asarray(L, F64)
    Z = np.asarray(Z, F64)
    r = Z.shape[0]
    ph, pw = _pads(KH, KW, pad)
    if scale is None:
        scale = np.full(Z.shape[1], 1.0 / r)
    dW = np.zeros((L.shape[1], Z.shape[1], KH, KW), F64)
    for ky in range(KH):
        for kx in range(KW):
            Zs = shift(Z, ky - ph, kx - pw, circular)
            dW[:, :, ky, kx] = np.einsum("jmyx,jnyx->mn", L, Zs) * scale[None, :]
    return dW


def wgrad_estimate(S, dY, Z, KH=3, KW=3, pad=None, circular=False, scale=None):
    """Algorithm 1 backward steps 3-4 in the paper's order: L first, then the offset traces."""
    return wgrad_contract(backprobe(S, dY), Z, KH, KW, pad, circular, scale)


def xconv_layer(X, W, dY, Z, pad=None, circular=False, scale=None):
    """Algorithm 1 end to end for one layer: returns Y, the sketch, the dW estimate and exact dX."""
    KH, KW = W.shape[2], W.shape[3]
    Y = conv_forward(X, W, pad, circular)
    S = sketch(X, Z)
    dW = wgrad_estimate(S, dY, Z, KH, KW, pad, circular, scale)
    dX = dx_exact(dY, W, pad, circular)
    return Y, S, dW, dX


# --- three-dimensional layers (volumes): the same method with one more shift axis ---------------------
# Arrays are (batch, channel, z, y, x); kernels (Cout, Cin, KD, KH, KW).  The sketch and the back-probe do not
# see the geometry (``sketch`` and ``backprobe`` above flatten every pixel axis), only the shifts do.

def shift3(A, dz, dy, dx, circular=False):
    """(shift3 A)[..., z, y, x] = A[..., z+dz, y+dy, x+dx]; zero outside the volume unless ``circular``
    (the shift T_k(i) of Section 3 for a three-dimensional offset k(i))."""
    A = np.asarray(A, dtype=F64)
    if circular:
        return np.roll(A, shift=(-dz, -dy, -dx), axis=(-3, -2, -1))
    D = A.shape[-3]
    out = np.zeros_like(A)
    z0, z1 = max(0, -dz), min(D, D - dz)
    if z0 < z1:
        out[..., z0:z1, :, :] = shift(A[..., z0 + dz:z1 + dz, :, :], dy, dx, False)
    return out


def _pads3(K, pad):
    return tuple((k - 1) // 2 for k in K) if pad is None else tuple(pad)


def conv_forward3d(X, W, pad=None, circular=False):
    """Eq. (5) for volumes: Y[b,m,z,y,x] = sum_{n,kz,ky,kx} W[m,n,kz,ky,kx] X[b,n,z+kz-pd,y+ky-ph,x+kx-pw]."""
    X = np.asarray(X, F64)
    W = np.asarray(W, F64)
    Cout, Cin, KD, KH, KW = W.shape
    pd, ph, pw = _pads3((KD, KH, KW), pad)
    Y = np.zeros((X.shape[0], Cout) + X.shape[2:], F64)
    for kz in range(KD):
        for ky in range(KH):
            for kx in range(KW):
                Y += np.einsum("mn,bnzyx->bmzyx", W[:, :, kz, ky, kx], shift3(X, kz - pd, ky - ph, kx - pw, circular))
    return Y


def dw_exact3d(X, dY, K=(3, 3, 3), pad=None, circular=False):
    """Eq. (2) for volumes: dW[m,n,kz,ky,kx] = sum_{b,z,y,x} dY[b,m,z,y,x] X[b,n,z+kz-pd,y+ky-ph,x+kx-pw]."""
    X = np.asarray(X, F64)
    dY = np.asarray(dY, F64)
    pd, ph, pw = _pads3(K, pad)
    dW = np.zeros((dY.shape[1], X.shape[1]) + tuple(K), F64)
    for kz in range(K[0]):
        for ky in range(K[1]):
            for kx in range(K[2]):
                dW[:, :, kz, ky, kx] = np.einsum("bmzyx,bnzyx->mn", dY, shift3(X, kz - pd, ky - ph, kx - pw, circular))
    return dW


def dx_exact3d(dY, W, pad=None, circular=False):
    """Adjoint of ``conv_forward3d`` in X: dX[b,n,u] = sum_{m,k} W[m,n,k] dY[b,m,u-k+p] (standard back-propagation)."""
    dY = np.asarray(dY, F64)
    W = np.asarray(W, F64)
    Cout, Cin, KD, KH, KW = W.shape
    pd, ph, pw = _pads3((KD, KH, KW), pad)
    dX = np.zeros((dY.shape[0], Cin) + dY.shape[2:], F64)
    for kz in range(KD):
        for ky in range(KH):
            for kx in range(KW):
                dX += np.einsum("mn,bmzyx->bnzyx", W[:, :, kz, ky, kx], shift3(dY, -(kz - pd), -(ky - ph), -(kx - pw), circular))
    return dX


def wgrad_contract3d(L, Z, K=(3, 3, 3), pad=None, circular=False, scale=None):
    """Algorithm 1 backward step 4 for volumes:
    dW[m,n,kz,ky,kx] = scale[n] * sum_{j,z,y,x} L[j,m,z,y,x] Z[j,n,z+kz-pd,y+ky-ph,x+kx-pw], scale = 1/r unless given."""
    L = np.asarray(L, F64)
    Z = np.asarray(Z, F64)
    pd, ph, pw = _pads3(K, pad)
    if scale is None:
        scale = np.full(Z.shape[1], 1.0 / Z.shape[0])
    dW = np.zeros((L.shape[1], Z.shape[1]) + tuple(K), F64)
    for kz in range(K[0]):
        for ky in range(K[1]):
            for kx in range(K[2]):
                Zs = shift3(Z, kz - pd, ky - ph, kx - pw, circular)
                dW[:, :, kz, ky, kx] = np.einsum("jmzyx,jnzyx->mn", L, Zs) * scale[None, :]
    return dW


def wgrad_estimate3d(S, dY, Z, K=(3, 3, 3), pad=None, circular=False, scale=None):
    """Algorithm 1 backward steps 3-4 for volumes (``sketch`` and ``backprobe`` serve any number of pixel axes)."""
    return wgrad_contract3d(backprobe(S, dY), Z, K, pad, circular, scale)


# --- trace estimation applied to every input/output channel pair on its own ---------------------------

def sketch_independent(X, Z):
    """The per-channel sketch X-bar^n = Z_n^T X^n in R^{r x B} for every input channel n: what has to be kept
    when the single-channel estimator (Eq. 4) is applied to each channel pair independently (first sentence
    of the multi-channel case, Section 3) instead of probing the stacked matrix.

    S[j,n,b] = sum_{y,x} Z[j,n,y,x] X[b,n,y,x]; summing it over n gives the multi-channel sketch."""
    X = np.asarray(X, F64)
    Z = np.asarray(Z, F64)
    return np.stack([sketch(X[:, n:n + 1], Z[:, n:n + 1]) for n in range(X.shape[1])], axis=1)


def wgrad_estimate_independent(S, dY, Z, KH=3, KW=3, pad=None, circular=False):
    """dw_i^{n,m} ~ (1/r) sum_j (z_{n,j}^T X^n) ((dY^m)^T T_{-k(i)} z_{n,j}): Eq. (4) for the pair (n, m), with the
    n-th block of the probing vectors and the n-th per-channel sketch.  No other channel enters the estimate
    of a pair, so there is no crosstalk.  S [r, Cin, B] from ``sketch_independent``."""
    S = np.asarray(S, F64)
    Z = np.asarray(Z, F64)
    Cin = Z.shape[1]
    dW = np.zeros((np.asarray(dY).shape[1], Cin, KH, KW), F64)
    for n in range(Cin):
        dW[:, n:n + 1] = wgrad_estimate(S[:, n, :], dY, Z[:, n:n + 1], KH, KW, pad, circular)
    return dW


# --- the literal block-matrix form of Eq. (6), for tiny layers only ---------------------------

def shift_matrix(H, W, dy, dx, circular=False):
    """Dense N x N matrix S_k with (S_k z)[q] = z[q + k], q = y*W + x, built entry by entry."""
    N = H * W
    M = np.zeros((N, N), F64)
    for y in range(H):
        for x in range(W):
            yy, xx = y + dy, x + dx
            if circular:
                yy %= H
                xx %= W
            elif not (0 <= yy < H and 0 <= xx < W):
                continue
            M[y * W + x, yy * W + xx] = 1.0
    return M


def wgrad_estimate_literal(X, dY, Z, KH=3, KW=3, pad=None, circular=False):
    """Eq. (6) as printed: form every block A^{m,n} = (X^n (dY^m)^T T_{-k(i)})^T, stack them into A,
    probe A from the right with the r columns of Z and each block row from the left.
    G^{m,n} = (1/r) sum_j z_{n,j}^T (A z_j)_m.  O(N^2) memory: tiny inputs only."""
    X = np.asarray(X, F64)
    dY = np.asarray(dY, F64)
    Z = np.asarray(Z, F64)
    B, Cin, H, W = X.shape
    Cout = dY.shape[1]
    r = Z.shape[0]
    N = H * W
    ph, pw = _pads(KH, KW, pad)
    Xm = X.reshape(B, Cin, N)
    dYm = dY.reshape(B, Cout, N)
    Zc = Z.reshape(r, Cin * N).T          # the paper's Z in R^{N Cin x r}
    dW = np.zeros((Cout, Cin, KH, KW), F64)
    for ky in range(KH):
        for kx in range(KW):
            Tk = shift_matrix(H, W, ky - ph, kx - pw, circular)
            A = np.zeros((Cout * N, Cin * N), F64)
            for m in range(Cout):
                for n in range(Cin):
                    outer = Xm[:, n, :].T @ dYm[:, m, :]          # X^n (dY^m)^T, N x N
                    A[m * N:(m + 1) * N, n * N:(n + 1) * N] = (outer @ Tk).T
            AZ = A @ Zc                                            # (i) probe from the right
            for m in range(Cout):
                for n in range(Cin):
                    acc = 0.0
                    for j in range(r):
                        acc += Zc[n * N:(n + 1) * N, j] @ AZ[m * N:(m + 1) * N, j]   # (iii)
                    dW[m, n, ky, kx] = acc / r
    return dW


def philox4x32_10(counter, key):
    """Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2,
    3", SC'11, Section 3.3 and Table 2): a counter-based generator, 128-bit counter -> 128 random bits.

    ``counter``: four arrays of 32-bit words (c0 least significant), ``key``: two 32-bit words.
    One round: (hi0, lo0) = M0 * c0, (hi1, lo1) = M1 * c2 (32 x 32 -> 64-bit products),
    c <- (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0); after every round the key is bumped by the Weyl
    constants (k0 += W0, k1 += W1).  Returns the four output words as uint64 arrays below 2^32.
    """
    M0, M1, W0, W1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85
    u = np.uint64
    mask = u(0xFFFFFFFF)
    c = [np.asarray(x, dtype=np.uint64) & mask for x in counter]
    k0, k1 = u(int(key[0]) & 0xFFFFFFFF), u(int(key[1]) & 0xFFFFFFFF)
    for _ in range(10):
        p0, p1 = u(M0) * c[0], u(M1) * c[2]
        hi0, lo0, hi1, lo1 = p0 >> u(32), p0 & mask, p1 >> u(32), p1 & mask
        c = [hi1 ^ c[1] ^ k0, lo1, hi0 ^ c[3] ^ k1, lo0]
        k0, k1 = (k0 + u(W0)) & mask, (k1 + u(W1)) & mask
    return c


def rademacher_probes(seed: int, r: int, Cin: int, H: int, W: int) -> np.ndarray:
    """The probing vectors Z[s] redrawn from the stored seed s (Algorithm 1: forward step 2 draws the seed,
    backward step 2 redraws "Z = randn(N, r)" from it), with Rademacher entries.

    Definition (fixed by this library, the paper leaves the generator open): number the entries of Z by
    e = ((j*H + y)*W + x)*Cin + n (probe j, pixel (y, x), input channel n).  Entry e is +1 if bit (e mod
    128) of philox4x32_10(counter = e div 128 as a 128-bit number, key = the two 32-bit halves of the seed)
    is 0 and -1 if it is 1; bit b is bit (b mod 32) of output word (b div 32).
    Returns Z [r, Cin, H, W] float64.
    """
    total = r * Cin * H * W
    blocks = np.arange((total + 127) // 128, dtype=np.uint64)
    zero = np.zeros_like(blocks)
    words = philox4x32_10((blocks & np.uint64(0xFFFFFFFF), blocks >> np.uint64(32), zero, zero),
                          (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))
    shifts = np.arange(32, dtype=np.uint64)
    bits = np.stack([(w[:, None] >> shifts[None, :]) & np.uint64(1) for w in words], axis=1)   # [block, word, bit]
    signs = 1.0 - 2.0 * bits.reshape(-1)[:total].astype(F64)
    return np.ascontiguousarray(signs.reshape(r, H, W, Cin).transpose(0, 3, 1, 2))


def _ln_f32(t):
    """Natural logarithm of (t * 2^-24) for odd integers 0 < t < 2^24, in float32 arithmetic whose every step is a
    single correctly rounded IEEE operation (+, -, *, /), so that a GPU can repeat it bit for bit.
    t = 2^k * f with f in [1, 2); if f > sqrt(2) halve it; then ln f = 2 artanh(s), s = (f - 1) / (f + 1),
    |s| <= 0.1716, by the odd series up to s^11 (the next term is below 1e-11)."""
    f32 = np.float32
    t = np.asarray(t, dtype=np.int64)
    k = np.floor(np.log2(t.astype(np.float64))).astype(np.int64)          # position of the leading bit (exact: t < 2^24)
    f = (t.astype(np.float64) / np.exp2(k)).astype(f32)                   # exact: a 24-bit integer scaled by a power of two
    big = f > f32(1.41421354)
    f = np.where(big, f * f32(0.5), f).astype(f32)
    e = (k - 24 + big.astype(np.int64)).astype(f32)
    s = ((f - f32(1.0)) / (f + f32(1.0))).astype(f32)
    s2 = (s * s).astype(f32)
    p = f32(1.0 / 11.0)
    for c in (1.0 / 9.0, 1.0 / 7.0, 1.0 / 5.0, 1.0 / 3.0, 1.0):
        p = ((p * s2).astype(f32) + f32(c)).astype(f32)
    lnf = ((f32(2.0) * s).astype(f32) * p).astype(f32)
    return ((e * f32(0.693147182)).astype(f32) + lnf).astype(f32)


def _sincos_2pi_f32(t):
    """(cos, sin) of 2 pi t / 2^24 for odd integers 0 < t < 2^24, in float32 arithmetic of single IEEE operations.
    The top three bits of t pick the octant, the rest is an angle x in (0, pi/4) (taken from the nearer end of the
    octant), where sin and cos are their Taylor polynomials up to x^9 and x^10 (next terms below 2e-9)."""
    f32 = np.float32
    t = np.asarray(t, dtype=np.int64)
    octant = t >> 21
    frac = t & ((1 << 21) - 1)                              # odd, below 2^21: angle frac * 2 pi / 2^24 within the octant
    frac = np.where(octant & 1, (1 << 21) - frac, frac)     # odd octants measure the angle back from their upper end
    x = (frac.astype(f32) * f32(3.74507039e-07)).astype(f32)        # 2 pi / 2^24
    x2 = (x * x).astype(f32)
    ps = f32(1.0 / 362880.0)
    for c in (-1.0 / 5040.0, 1.0 / 120.0, -1.0 / 6.0, 1.0):
        ps = ((ps * x2).astype(f32) + f32(c)).astype(f32)
    sn = (ps * x).astype(f32)
    pc = f32(-1.0 / 3628800.0)
    for c in (1.0 / 40320.0, -1.0 / 720.0, 1.0 / 24.0, -0.5, 1.0):
        pc = ((pc * x2).astype(f32) + f32(c)).astype(f32)
    cs = pc
    # octants 0..7: (cos, sin) of the full angle from (cs, sn) of the reduced one
    swap = ((octant + 1) >> 1) & 1                          # octants 1, 2, 5, 6: the roles of sin and cos trade places
    c_abs = np.where(swap, sn, cs)
    s_abs = np.where(swap, cs, sn)
    c_neg = ((octant + 2) >> 2) & 1                         # cos < 0 in octants 2..5
    s_neg = octant >> 2                                     # sin < 0 in octants 4..7
    return np.where(c_neg, -c_abs, c_abs).astype(f32), np.where(s_neg, -s_abs, s_abs).astype(f32)


def gaussian_probes(seed: int, r: int, Cin: int, H: int, W: int) -> np.ndarray:
    """Probing vectors with standard normal entries redrawn from the stored seed (Algorithm 1, backward step 2:
    "Z = randn(N, r)" from the seed drawn in forward step 2; Section 3 takes z ~ N(0, I)).

    Definition (fixed by this library): number the entries of Z by e = ((j*H + y)*W + x)*Cin + n as for the
    Rademacher probes.  Philox block b = e div 4 has counter (b as 64 bits in words 0-1, word 2 = 1, word 3 = 0) --
    word 2 keeps it apart from the Rademacher stream of the same seed -- and the seed as key.  Its four words
    w0..w3 give two pairs (w0, w1), (w2, w3) of uniforms u = (2 (w >> 9) + 1) / 2^24 in (0, 1), and each pair two
    normals by the Box-Muller transform: sqrt(-2 ln u_a) cos(2 pi u_b) for the even entry, ... sin(...) for the odd
    one.  Logarithm, sine and cosine are the float32 series of _ln_f32 and _sincos_2pi_f32, the square root and the
    products single float32 operations.  Returns Z [r, Cin, H, W] (float32 values in a float64 array)."""
    f32 = np.float32
    total = r * Cin * H * W
    blocks = np.arange((total + 3) // 4, dtype=np.uint64)
    one, zero = np.ones_like(blocks), np.zeros_like(blocks)
    w = philox4x32_10((blocks & np.uint64(0xFFFFFFFF), blocks >> np.uint64(32), one, zero),
                      (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))
    out = np.empty((blocks.size, 4), dtype=f32)
    for pair in range(2):
        ta = ((w[2 * pair] >> np.uint64(9)).astype(np.int64) << 1) | 1
        tb = ((w[2 * pair + 1] >> np.uint64(9)).astype(np.int64) << 1) | 1
        rad = np.sqrt(((f32(-2.0) * _ln_f32(ta)).astype(f32))).astype(f32)
        cs, sn = _sincos_2pi_f32(tb)
        out[:, 2 * pair] = (rad * cs).astype(f32)
        out[:, 2 * pair + 1] = (rad * sn).astype(f32)
    z = out.reshape(-1)[:total].astype(F64)
    return np.ascontiguousarray(z.reshape(r, H, W, Cin).transpose(0, 3, 1, 2))


def block_keep_mask(seed: int, r: int, Cin: int, p: float) -> np.ndarray:
    """Which blocks z_{n,j} of Eq. (7) are non-zero, redrawn from the stored seed: block n of probing vector j is kept
    with probability p, independently for every (n, j).

    Definition (fixed by this library): number the blocks by g = j*Cin + n.  Philox block g div 4 has counter (g div 4
    in words 0-1, word 2 = 2, word 3 = 0) -- word 2 keeps it apart from the two value streams -- and the seed as key;
    block g is kept iff its output word (g mod 4) is below floor(p * 2^32).  Returns a boolean array [r, Cin]."""
    total = r * Cin
    blocks = np.arange((total + 3) // 4, dtype=np.uint64)
    two, zero = np.full_like(blocks, 2), np.zeros_like(blocks)
    w = philox4x32_10((blocks & np.uint64(0xFFFFFFFF), blocks >> np.uint64(32), two, zero),
                      (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))
    words = np.stack(w, axis=1).reshape(-1)[:total]
    threshold = np.uint64(min(max(int(np.floor(float(p) * 4294967296.0)), 0), 1 << 32))
    return (words < threshold).reshape(r, Cin)


def block_sparse_probes(seed: int, r: int, Cin: int, H: int, W: int, p: float, gaussian: bool = False) -> np.ndarray:
    """Probing vectors of Eq. (7) from a seed: the dense probes of the same seed (Rademacher, or standard normal as the
    equation prints them) with the blocks block_keep_mask drops set to zero.  Returns Z [r, Cin, H, W]; the scale of
    Eq. (8) for it is channel_scale(Z)."""
    dense = gaussian_probes(seed, r, Cin, H, W) if gaussian else rademacher_probes(seed, r, Cin, H, W)
    return dense * block_keep_mask(seed, r, Cin, p)[:, :, None, None]


def memory_factor(Cin, H, W, r):
    """Stored elements, exact (X) over sketched (X-bar), per sample: N*Cin / r (Section 3 and 4.1)."""
    return (H * W * Cin) / r


def rel_fro(a, b):
    """||a - b||_F / ||b||_F."""
    a = np.asarray(a, F64)
    b = np.asarray(b, F64)
    d = np.linalg.norm((a - b).ravel())
    n = np.linalg.norm(b.ravel())
    return d / n if n > 0 else d
