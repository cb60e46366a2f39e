"""Pins for the float64 oracle: each check ties it to something other than itself --
brute-force loops, closed forms, invariants, special cases that reduce to a plain
matrix product, values and bounds the paper prints.  CPU only."""
import math
import os

import numpy as np
import pytest

from oracle import xconv_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _tiny(seed=0, B=2, Cin=3, Cout=2, H=5, W=4, KH=3, KW=3):
    g = _rng(seed)
    X = g.standard_normal((B, Cin, H, W))
    Wt = g.standard_normal((Cout, Cin, KH, KW))
    dY = g.standard_normal((B, Cout, H, W))
    return X, Wt, dY


# ---------------------------------------------------------------- P1: brute force (Eq. 1, 2, 5)

def _loops_conv(X, Wt, circular):
    B, Cin, H, W = X.shape
    Cout, _, KH, KW = Wt.shape
    ph, pw = (KH - 1) // 2, (KW - 1) // 2
    Y = np.zeros((B, Cout, H, W))
    for b in range(B):
        for m in range(Cout):
            for y in range(H):
                for x in range(W):
                    acc = 0.0
                    for n in range(Cin):
                        for ky in range(KH):
                            for kx in range(KW):
                                yy, xx = y + ky - ph, x + kx - pw
                                if circular:
                                    yy, xx = yy % H, xx % W
                                elif not (0 <= yy < H and 0 <= xx < W):
                                    continue
                                acc += Wt[m, n, ky, kx] * X[b, n, yy, xx]
                    Y[b, m, y, x] = acc
    return Y


def _loops_dw(X, dY, KH, KW, circular):
    B, Cin, H, W = X.shape
    Cout = dY.shape[1]
    ph, pw = (KH - 1) // 2, (KW - 1) // 2
    dW = np.zeros((Cout, Cin, KH, KW))
    for m in range(Cout):
        for n in range(Cin):
            for ky in range(KH):
                for kx in range(KW):
                    acc = 0.0
                    for b in range(B):
                        for y in range(H):
                            for x in range(W):
                                yy, xx = y + ky - ph, x + kx - pw
                                if circular:
                                    yy, xx = yy % H, xx % W
                                elif not (0 <= yy < H and 0 <= xx < W):
                                    continue
                                acc += dY[b, m, y, x] * X[b, n, yy, xx]
                    dW[m, n, ky, kx] = acc
    return dW


def _loops_dx(dY, Wt, circular):
    B, Cout, H, W = dY.shape
    _, Cin, KH, KW = Wt.shape
    ph, pw = (KH - 1) // 2, (KW - 1) // 2
    dX = np.zeros((B, Cin, H, W))
    # scatter form: every term W*dY of the forward sum sends its gradient to the pixel it read
    for b in range(B):
        for m in range(Cout):
            for y in range(H):
                for x in range(W):
                    for n in range(Cin):
                        for ky in range(KH):
                            for kx in range(KW):
                                yy, xx = y + ky - ph, x + kx - pw
                                if circular:
                                    yy, xx = yy % H, xx % W
                                elif not (0 <= yy < H and 0 <= xx < W):
                                    continue
                                dX[b, n, yy, xx] += Wt[m, n, ky, kx] * dY[b, m, y, x]
    return dX


@pytest.mark.parametrize("circular", [False, True])
@pytest.mark.parametrize("K", [1, 3, 5])
def test_p1_brute_force_loops(circular, K):
    X, Wt, dY = _tiny(seed=K, H=5, W=6 if K == 5 else 4, KH=K, KW=K)
    np.testing.assert_allclose(O.conv_forward(X, Wt, circular=circular), _loops_conv(X, Wt, circular), rtol=0, atol=1e-12)
    np.testing.assert_allclose(O.dw_exact(X, dY, K, K, circular=circular), _loops_dw(X, dY, K, K, circular), rtol=0, atol=1e-12)
    np.testing.assert_allclose(O.dx_exact(dY, Wt, circular=circular), _loops_dx(dY, Wt, circular), rtol=0, atol=1e-12)


def test_p1_gradients_by_finite_difference():
    """f(W, X) = <conv(X, W), G> is bilinear, so one-sided differences are exact up to rounding."""
    X, Wt, G = _tiny(seed=11)
    f0 = np.sum(O.conv_forward(X, Wt) * G)
    dW = O.dw_exact(X, G)
    dX = O.dx_exact(G, Wt)
    g = _rng(5)
    for _ in range(12):
        idx = tuple(g.integers(0, s) for s in Wt.shape)
        Wp = Wt.copy(); Wp[idx] += 1.0
        assert abs((np.sum(O.conv_forward(X, Wp) * G) - f0) - dW[idx]) < 1e-10
        idx = tuple(g.integers(0, s) for s in X.shape)
        Xp = X.copy(); Xp[idx] += 1.0
        assert abs((np.sum(O.conv_forward(Xp, Wt) * G) - f0) - dX[idx]) < 1e-10


def test_conv_is_cross_correlation_of_a_unit_impulse():
    """A unit impulse in X reproduces the flipped kernel around it: fixes the sign of k(i)."""
    H = W = 5
    X = np.zeros((1, 1, H, W)); X[0, 0, 2, 2] = 1.0
    Wt = np.arange(9, dtype=float).reshape(1, 1, 3, 3)
    Y = O.conv_forward(X, Wt)
    # Y[y,x] = W[ky,kx] with y+ky-1 = 2, x+kx-1 = 2
    for ky in range(3):
        for kx in range(3):
            assert Y[0, 0, 3 - ky, 3 - kx] == Wt[0, 0, ky, kx]


# ---------------------------------------------------------------- P2: exact recovery

def _orth_probes(Cin, H, W, seed):
    D = Cin * H * W
    Q, _ = np.linalg.qr(_rng(seed).standard_normal((D, D)))
    return (math.sqrt(D) * Q).reshape(D, Cin, H, W)      # rows j: Z2d^T Z2d = D * I


@pytest.mark.parametrize("circular", [False, True])
def test_p2_exact_recovery_with_orthogonal_basis(circular):
    """With r = Cin*N probes and (1/r) Z Z^T = I the estimator is the exact gradient
    ("recovers the exact gradient in the limit", Section 2)."""
    X, Wt, dY = _tiny(seed=3, B=3, Cin=2, Cout=3, H=4, W=3)
    Z = _orth_probes(2, 4, 3, seed=9)
    S = O.sketch(X, Z)
    est = O.wgrad_estimate(S, dY, Z, circular=circular)
    np.testing.assert_allclose(est, _loops_dw(X, dY, 3, 3, circular), rtol=0, atol=1e-11)


def test_p2_exact_recovery_with_hadamard_rademacher_basis():
    from scipy.linalg import hadamard
    Cin, H, W = 2, 4, 4                      # Cin*N = 32, a power of two
    X, Wt, dY = _tiny(seed=4, B=3, Cin=Cin, Cout=2, H=H, W=W)
    Z = hadamard(Cin * H * W).astype(float).reshape(-1, Cin, H, W)   # +-1 entries, Z^T Z = r I
    est = O.wgrad_estimate(O.sketch(X, Z), dY, Z)
    np.testing.assert_allclose(est, _loops_dw(X, dY, 3, 3, False), rtol=0, atol=1e-11)


def test_p2_wrong_shift_sign_would_fail():
    """The exact gradient is not symmetric under k -> -k on generic data, so P2 pins the direction."""
    X, Wt, dY = _tiny(seed=3, B=3, Cin=2, Cout=3, H=4, W=3)
    dW = _loops_dw(X, dY, 3, 3, False)
    assert O.rel_fro(dW[:, :, ::-1, ::-1], dW) > 0.5


# ---------------------------------------------------------------- literal Eq. (6) vs the three steps

@pytest.mark.parametrize("circular", [False, True])
def test_three_steps_equal_literal_block_estimator(circular):
    X, Wt, dY = _tiny(seed=6, B=2, Cin=2, Cout=2, H=3, W=4)
    Z = _rng(7).standard_normal((5, 2, 3, 4))
    lit = O.wgrad_estimate_literal(X, dY, Z, circular=circular)
    est = O.wgrad_estimate(O.sketch(X, Z), dY, Z, circular=circular)
    np.testing.assert_allclose(est, lit, rtol=0, atol=1e-11)


def test_shift_matrix_is_the_shift():
    g = _rng(2)
    A = g.standard_normal((4, 5))
    for dy in (-1, 0, 1):
        for dx in (-2, 0, 1):
            for circ in (False, True):
                M = O.shift_matrix(4, 5, dy, dx, circ)
                np.testing.assert_array_equal((M @ A.ravel()).reshape(4, 5), O.shift(A, dy, dx, circ))
    # circular shifts are permutations (the paper's T_k), truncating ones are not
    assert np.allclose(O.shift_matrix(4, 5, 1, -1, True).sum(0), 1)
    assert O.shift_matrix(4, 5, 1, -1, False).sum() < 20


# ---------------------------------------------------------------- P8: special cases

def test_p8_single_channel_reduces_to_eq4():
    """Cin = Cout = 1: dw_i ~ (1/r) sum_j (z_j^T X)(dY^T T_{-k(i)} z_j)   (Eq. 4)."""
    H, W, B, r = 4, 5, 3, 6
    g = _rng(8)
    X = g.standard_normal((B, 1, H, W)); dY = g.standard_normal((B, 1, H, W))
    Z = g.standard_normal((r, 1, H, W))
    est = O.wgrad_estimate(O.sketch(X, Z), dY, Z)
    Xm = X.reshape(B, -1).T; dYm = dY.reshape(B, -1).T; Zm = Z.reshape(r, -1).T   # N x B, N x B, N x r
    for ky in range(3):
        for kx in range(3):
            Tk = O.shift_matrix(H, W, ky - 1, kx - 1)
            ref = sum((Zm[:, j] @ Xm) @ (dYm.T @ Tk @ Zm[:, j]) for j in range(r)) / r
            assert abs(est[0, 0, ky, kx] - ref) < 1e-11


def test_p8_pointwise_kernel_is_a_plain_matmul():
    """K = 1: dW = (1/r) L_flat Z_flat^T with L_flat [Cout, r*N], Z_flat [Cin, r*N]."""
    g = _rng(10)
    B, Cin, Cout, H, W, r = 3, 4, 5, 3, 3, 7
    X = g.standard_normal((B, Cin, H, W)); dY = g.standard_normal((B, Cout, H, W))
    Z = g.standard_normal((r, Cin, H, W))
    S = Z.reshape(r, -1) @ X.reshape(B, -1).T
    L = (S @ dY.reshape(B, -1)).reshape(r, Cout, H * W)
    ref = L.transpose(1, 0, 2).reshape(Cout, -1) @ Z.reshape(r, Cin, -1).transpose(1, 0, 2).reshape(Cin, -1).T / r
    est = O.wgrad_estimate(O.sketch(X, Z), dY, Z, KH=1, KW=1)
    np.testing.assert_allclose(est[:, :, 0, 0], ref, rtol=0, atol=1e-11)


def test_estimator_is_exact_wgrad_of_the_reconstructed_activation():
    """Bilinearity: contracting L with Z equals the exact gradient with X replaced by (1/r) Z Z^T X."""
    X, Wt, dY = _tiny(seed=12, B=3, Cin=2, Cout=2, H=4, W=4)
    Z = _rng(13).standard_normal((6, 2, 4, 4))
    S = O.sketch(X, Z)
    Xrec = np.einsum("jb,jnyx->bnyx", S, Z) / 6
    np.testing.assert_allclose(O.wgrad_estimate(S, dY, Z), _loops_dw(Xrec, dY, 3, 3, False), rtol=0, atol=1e-11)


# ---------------------------------------------------------------- P3/P4: unbiasedness and closed-form variance

def _C_blocks(X, dY, m, ky, kx):
    """C_n'[p, q'] = sum_b X[b,n',p] dY[b,m,q'-k]; the estimate of dW[m,n,k] with one probe is
    sum_n' z_n'^T C_n' z_n."""
    B, Cin, H, W = X.shape
    N = H * W
    C = np.zeros((Cin, N, N))
    for n in range(Cin):
        for y in range(H):
            for x in range(W):
                yq, xq = y - (ky - 1), x - (kx - 1)     # q = q' - k
                if 0 <= yq < H and 0 <= xq < W:
                    for b in range(B):
                        C[n, :, y * W + x] += X[b, n].ravel() * dY[b, m, yq, xq]
    return C


def _closed_form_variance(C, n, rademacher):
    v = np.sum(C[n] ** 2) + np.trace(C[n] @ C[n])
    if rademacher:
        v -= 2.0 * np.sum(np.diag(C[n]) ** 2)
    for k in range(C.shape[0]):
        if k != n:
            v += np.sum(C[k] ** 2)
    return v


@pytest.mark.parametrize("kind", ["gaussian", "rademacher"])
def test_p3_p4_unbiased_with_hutchinson_variance(kind):
    """Mean over independent probes tends to the exact gradient (Appendix, proof of Theorem 1, first part);
    the per-probe variance is the textbook Hutchinson expression plus the cross-channel terms."""
    X, Wt, dY = _tiny(seed=20, B=3, Cin=2, Cout=2, H=4, W=4)
    exact = _loops_dw(X, dY, 3, 3, False)
    T = 6000
    g = _rng(21)
    if kind == "gaussian":
        Zall = g.standard_normal((T, 2, 4, 4))
    else:
        Zall = g.integers(0, 2, size=(T, 2, 4, 4)).astype(float) * 2 - 1
    ests = np.stack([O.wgrad_estimate(O.sketch(X, Zall[t:t + 1]), dY, Zall[t:t + 1]) for t in range(T)])
    mean, var = ests.mean(0), ests.var(0, ddof=1)
    for m in range(2):
        for ky in range(3):
            for kx in range(3):
                C = _C_blocks(X, dY, m, ky, kx)
                for n in range(2):
                    assert abs(np.trace(C[n]) - exact[m, n, ky, kx]) < 1e-10
                    v = _closed_form_variance(C, n, kind == "rademacher")
                    z = (mean[m, n, ky, kx] - exact[m, n, ky, kx]) / math.sqrt(v / T)
                    assert abs(z) < 4.5, (m, n, ky, kx, z)
                    assert 0.8 < var[m, n, ky, kx] / v < 1.25, (m, n, ky, kx, var[m, n, ky, kx], v)
    # one r-probe estimate is the average of r one-probe estimates (scale 1/r)
    r = 8
    np.testing.assert_allclose(O.wgrad_estimate(O.sketch(X, Zall[:r]), dY, Zall[:r]), ests[:r].mean(0), atol=1e-11)


def test_p3_block_sparse_probes_with_nnz_scale_are_unbiased():
    """Eq. (7) probes (whole channel blocks zeroed with probability 1-p) with the 1/nnz(Z_n) scale of
    Eq. (8) stay unbiased; with the plain 1/r scale they are biased by the factor nnz/r."""
    X, Wt, dY = _tiny(seed=30, B=3, Cin=3, Cout=2, H=3, W=3)
    exact = _loops_dw(X, dY, 3, 3, False)
    g = _rng(31)
    T, r, p = 1500, 6, 0.6
    acc = np.zeros_like(exact); acc_plain = np.zeros_like(exact)
    for _ in range(T):
        Z = g.standard_normal((r, 3, 3, 3)) * (g.random((r, 3, 1, 1)) < p)
        sc = O.channel_scale(Z)
        S = O.sketch(X, Z)
        acc += O.wgrad_estimate(S, dY, Z, scale=sc)
        acc_plain += O.wgrad_estimate(S, dY, Z)
    # channels with nnz = 0 give 0 (probability (1-p)^r = 0.4%): compare against (1-(1-p)^r) * exact
    keep = 1 - (1 - p) ** r
    assert O.rel_fro(acc / T, keep * exact) < 0.08
    assert O.rel_fro(acc_plain / T, p * exact) < 0.08
    assert O.rel_fro(acc_plain / T, exact) > 0.25


def test_channel_scale_counts_nonzero_blocks():
    Z = np.zeros((4, 3, 2, 2))
    Z[0, 0] = 1; Z[2, 0, 1, 1] = -3; Z[1, 1, 0, 0] = 2
    np.testing.assert_allclose(O.channel_scale(Z), [0.5, 1.0, 0.0])
    np.testing.assert_allclose(O.channel_scale(np.ones((5, 2, 2, 2))), [0.2, 0.2])


# ---------------------------------------------------------------- P5: Proposition 1

def test_p5_proposition1_bound_holds_with_probability_1_minus_delta():
    c2, cF = np.loadtxt(os.path.join(GOLD, "prop1_constants.txt"))
    g = _rng(40)
    H, W, B = 4, 4, 3
    X = g.standard_normal((B, 1, H, W)); dY = g.standard_normal((B, 1, H, W))
    exact = _loops_dw(X, dY, 3, 3, False)
    T = 1500
    for r in (1, 4, 32):
        Zall = g.standard_normal((T, r, 1, H, W))
        ests = np.stack([O.wgrad_estimate(O.sketch(X, Zall[t]), dY, Zall[t]) for t in range(T)])
        for (ky, kx) in ((0, 0), (1, 1), (2, 1)):
            A = _C_blocks(X, dY, 0, ky, kx)[0]
            n2, nF = np.linalg.norm(A, 2), np.linalg.norm(A, "fro")
            dev = np.abs(ests[:, 0, 0, ky, kx] - exact[0, 0, ky, kx])
            for delta in (0.1, 0.01):
                lg = math.log(2 / delta)
                bound = c2 * n2 / r * lg + cF * nF / math.sqrt(r) * math.sqrt(lg)
                frac = np.mean(dev > bound)
                assert frac <= delta + 3 * math.sqrt(delta * (1 - delta) / T), (r, ky, kx, delta, frac)
            # the bound is not vacuous for this estimator: a deviation of that size does occur at 1/50 of it
            assert np.mean(dev > bound / 50) > 0


# ---------------------------------------------------------------- P6: Theorem 1's shape

def test_p6_error_decays_like_inverse_sqrt_r_and_respects_the_row_bound():
    X, Wt, dY = _tiny(seed=50, B=4, Cin=3, Cout=2, H=4, W=4)
    exact = _loops_dw(X, dY, 3, 3, False)
    g = _rng(51)
    rs, rms = (4, 16, 64, 256), []
    for r in rs:
        errs = []
        for _ in range(60):
            Z = g.standard_normal((r, 3, 4, 4))
            errs.append(O.wgrad_estimate(O.sketch(X, Z), dY, Z) - exact)
        rms.append(np.sqrt(np.mean(np.square(errs), axis=0)))
    slope = np.polyfit(np.log(rs), np.log([np.sqrt(np.mean(e ** 2)) for e in rms]), 1)[0]
    assert -0.6 < slope < -0.4, slope
    # RMS error of entry (m,n) <= (sqrt(2)||C_n||_F + sum_{k != n} ||C_k||_F)/sqrt(r): own block plus
    # the other blocks of the same output row (Theorem 1, large-r form, with the constant made explicit)
    r = rs[-1]
    for m in range(2):
        C = _C_blocks(X, dY, m, 1, 2)
        nf = [np.linalg.norm(C[n]) for n in range(3)]
        for n in range(3):
            bound = (math.sqrt(2) * nf[n] + sum(nf[k] for k in range(3) if k != n)) / math.sqrt(r)
            assert rms[-1][m, n, 1, 2] <= 1.25 * bound


# ---------------------------------------------------------------- P7: memory factor

def test_p7_memory_factor_matches_printed_values():
    rows = np.loadtxt(os.path.join(GOLD, "memory_factor.txt"))
    for H, W, Cin, gamma, factor in rows:
        assert O.memory_factor(int(Cin), int(H), int(W), 2 ** int(gamma)) == factor == 2 ** (14 - gamma)
    assert 100 <= O.memory_factor(16, 32, 32, 2 ** 7) <= 130      # "roughly 100x"


# ------------------------------------------------------------------ probes redrawn from a seed (Algorithm 1)

def test_philox_known_answer_vectors():
    rows = [l.split() for l in open(os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for row in rows:
        v = [int(x, 16) for x in row]
        out = O.philox4x32_10([np.array([c]) for c in v[0:4]], v[4:6])
        assert [int(o[0]) for o in out] == v[6:10]


def test_rademacher_probes_follow_the_stated_bit_order():
    # entry e = ((j*H + y)*W + x)*Cin + n takes bit (e mod 128) of block (e div 128): re-derive a few entries
    # one by one, straight from the definition
    r, Cin, H, W, seed = 3, 5, 4, 7, 0x1234567890ABCDEF
    Z = O.rademacher_probes(seed, r, Cin, H, W)
    assert Z.shape == (r, Cin, H, W) and set(np.unique(Z)) == {-1.0, 1.0}
    for (j, n, y, x) in [(0, 0, 0, 0), (0, 4, 0, 0), (1, 2, 3, 6), (2, 4, 3, 6), (2, 0, 1, 5)]:
        e = ((j * H + y) * W + x) * Cin + n
        blk, bit = divmod(e, 128)
        words = O.philox4x32_10([np.array([blk & 0xFFFFFFFF]), np.array([blk >> 32]), np.array([0]), np.array([0])],
                                (seed & 0xFFFFFFFF, seed >> 32))
        b = (int(words[bit // 32][0]) >> (bit % 32)) & 1
        assert Z[j, n, y, x] == (1.0 - 2.0 * b)


def test_rademacher_probes_are_balanced_independent_and_seed_dependent():
    r, Cin, H, W = 4096, 2, 3, 3          # 4096 probes of dimension 18
    Z = O.rademacher_probes(7, r, Cin, H, W).reshape(r, -1)
    assert abs(Z.mean()) < 4.0 / np.sqrt(Z.size)
    C = Z.T @ Z / r                       # E[z z^T] = I, the only property the estimator needs (Section 3)
    assert np.allclose(np.diag(C), 1.0)
    off = C - np.eye(C.shape[0])
    assert np.abs(off).max() < 5.0 / np.sqrt(r)
    Z2 = O.rademacher_probes(8, r, Cin, H, W).reshape(r, -1)
    assert 0.4 < (Z != Z2).mean() < 0.6


def test_estimator_on_redrawn_probes_is_unbiased():
    # mean of the estimate over many seeds -> exact gradient (Section 3: E[z z^T] = I)
    g = np.random.Generator(np.random.PCG64(5))
    B, Cin, Cout, H, W, r, T = 3, 2, 2, 4, 4, 8, 3000
    X, dY = g.standard_normal((B, Cin, H, W)), g.standard_normal((B, Cout, H, W))
    exact = O.dw_exact(X, dY)
    acc = np.zeros_like(exact)
    for t in range(T):
        Z = O.rademacher_probes(1000 + t, r, Cin, H, W)
        acc += O.wgrad_estimate(O.sketch(X, Z), dY, Z)
    err = np.abs(acc / T - exact).max()
    single = np.std([O.wgrad_estimate(O.sketch(X, Z), dY, Z) for Z in (O.rademacher_probes(s, r, Cin, H, W) for s in range(50))], axis=0).max()
    assert err < 5.0 * single / np.sqrt(T)


def test_rel_fro_on_a_hand_computed_pair():
    """The parity metric itself: ||a - b||_F / ||b||_F on values worked out by hand.
    a - b = (3, 4, 0, 0) has norm 5; b = (1, 2, 2, 4) has norm 5; a shifted copy gives a different value, so
    the arguments are not interchangeable and the denominator is the second one."""
    a = np.array([[4.0, 6.0], [2.0, 4.0]])
    b = np.array([[1.0, 2.0], [2.0, 4.0]])
    assert O.rel_fro(a, b) == pytest.approx(1.0, abs=1e-15)
    assert O.rel_fro(b, a) == pytest.approx(5.0 / np.sqrt(72.0), abs=1e-15)
    assert O.rel_fro(b, b) == 0.0
    assert O.rel_fro(2 * b, b) == pytest.approx(1.0, abs=1e-15)          # scale of the error, not of the data
    assert O.rel_fro(np.array([3.0, 4.0]), np.zeros(2)) == pytest.approx(5.0)   # zero reference: absolute norm


# ---------------------------------------------------------------- independent probing (per channel pair)

def test_independent_sketch_sums_to_the_multichannel_sketch_and_reduces_for_one_channel():
    X, Wt, dY = _tiny(seed=40, B=3, Cin=3, Cout=2, H=4, W=5)
    Z = _rng(41).standard_normal((7, 3, 4, 5))
    Si = O.sketch_independent(X, Z)
    assert Si.shape == (7, 3, 3)
    np.testing.assert_allclose(Si.sum(axis=1), O.sketch(X, Z), atol=1e-12)
    # brute force for one entry
    j, n, b = 4, 2, 1
    assert abs(Si[j, n, b] - sum(Z[j, n, y, x] * X[b, n, y, x] for y in range(4) for x in range(5))) < 1e-12
    # a single input channel: both estimators coincide (Eq. 4 is the Cin = Cout = 1 case of Eq. 6)
    X1, Z1 = X[:, :1], Z[:, :1]
    np.testing.assert_allclose(O.wgrad_estimate_independent(O.sketch_independent(X1, Z1), dY, Z1),
                               O.wgrad_estimate(O.sketch(X1, Z1), dY, Z1), atol=1e-12)


def test_independent_probing_recovers_the_exact_gradient_with_one_orthogonal_basis_per_channel():
    """r = N and (1/r) Z_n Z_n^T = I_N for every channel n (a different basis each): every pair's trace is exact."""
    X, Wt, dY = _tiny(seed=42, B=3, Cin=3, Cout=2, H=3, W=4)
    N = 12
    Z = np.stack([np.sqrt(N) * np.linalg.qr(_rng(50 + n).standard_normal((N, N)))[0].T.reshape(N, 3, 4)
                  for n in range(3)], axis=1)                     # [r = N, Cin, H, W]
    est = O.wgrad_estimate_independent(O.sketch_independent(X, Z), dY, Z)
    np.testing.assert_allclose(est, _loops_dw(X, dY, 3, 3, False), atol=1e-10)
    # the multi-channel estimator on the same probes is NOT exact (r = N < N*Cin: crosstalk remains)
    assert O.rel_fro(O.wgrad_estimate(O.sketch(X, Z), dY, Z), _loops_dw(X, dY, 3, 3, False)) > 1e-2


def test_independent_probing_is_unbiased_with_the_crosstalk_free_variance():
    """Per pair the variance is the single-channel Hutchinson expression: the sum over the other channels'
    blocks, which the multi-channel estimator carries, is absent."""
    X, Wt, dY = _tiny(seed=20, B=3, Cin=2, Cout=2, H=4, W=4)
    exact = _loops_dw(X, dY, 3, 3, False)
    T = 6000
    Zall = _rng(43).standard_normal((T, 2, 4, 4))
    ests = np.stack([O.wgrad_estimate_independent(O.sketch_independent(X, Zall[t:t + 1]), dY, Zall[t:t + 1])
                     for t in range(T)])
    mean, var = ests.mean(0), ests.var(0, ddof=1)
    for m in range(2):
        for ky in range(3):
            for kx in range(3):
                C = _C_blocks(X, dY, m, ky, kx)
                for n in range(2):
                    v = np.sum(C[n] ** 2) + np.trace(C[n] @ C[n])
                    z = (mean[m, n, ky, kx] - exact[m, n, ky, kx]) / math.sqrt(v / T)
                    assert abs(z) < 4.5, (m, n, ky, kx, z)
                    assert 0.8 < var[m, n, ky, kx] / v < 1.25, (m, n, ky, kx, var[m, n, ky, kx], v)
                    assert v < _closed_form_variance(C, n, False)


# ---------------------------------------------------------------- volumes (three-dimensional layers)

def _tiny3(seed, B=2, Cin=2, Cout=3, D=3, H=4, W=3, K=(3, 3, 3)):
    g = _rng(seed)
    return (g.standard_normal((B, Cin, D, H, W)), g.standard_normal((Cout, Cin) + K), g.standard_normal((B, Cout, D, H, W)))


@pytest.mark.parametrize("circular", [False, True])
@pytest.mark.parametrize("K", [(3, 3, 3), (1, 3, 3), (3, 1, 5)])
def test_volume_functions_against_brute_force_loops(K, circular):
    X, Wt, dY = _tiny3(60, K=K)
    B, Cin, D, H, W = X.shape
    Cout = Wt.shape[0]
    pd, ph, pw = [(k - 1) // 2 for k in K]
    Y = np.zeros((B, Cout, D, H, W)); dW = np.zeros_like(Wt); dX = np.zeros_like(X)

    def src(z, y, x, kz, ky, kx):
        zz, yy, xx = z + kz - pd, y + ky - ph, x + kx - pw
        if circular:
            return zz % D, yy % H, xx % W
        return (zz, yy, xx) if (0 <= zz < D and 0 <= yy < H and 0 <= xx < W) else None

    for b in range(B):
        for m in range(Cout):
            for n in range(Cin):
                for z in range(D):
                    for y in range(H):
                        for x in range(W):
                            for kz in range(K[0]):
                                for ky in range(K[1]):
                                    for kx in range(K[2]):
                                        s_ = src(z, y, x, kz, ky, kx)
                                        if s_ is None:
                                            continue
                                        Y[b, m, z, y, x] += Wt[m, n, kz, ky, kx] * X[(b, n) + s_]
                                        dW[m, n, kz, ky, kx] += dY[b, m, z, y, x] * X[(b, n) + s_]
                                        dX[(b, n) + s_] += Wt[m, n, kz, ky, kx] * dY[b, m, z, y, x]
    np.testing.assert_allclose(O.conv_forward3d(X, Wt, circular=circular), Y, atol=1e-11)
    np.testing.assert_allclose(O.dw_exact3d(X, dY, K, circular=circular), dW, atol=1e-11)
    np.testing.assert_allclose(O.dx_exact3d(dY, Wt, circular=circular), dX, atol=1e-11)


def test_volume_functions_reduce_to_the_planar_ones_at_depth_one():
    X, Wt, dY = _tiny(seed=61, B=2, Cin=3, Cout=2, H=5, W=4)
    Z = _rng(62).standard_normal((6, 3, 5, 4))
    X3, W3, dY3, Z3 = X[:, :, None], Wt[:, :, None], dY[:, :, None], Z[:, :, None]
    np.testing.assert_allclose(O.conv_forward3d(X3, W3)[:, :, 0], O.conv_forward(X, Wt), atol=1e-12)
    np.testing.assert_allclose(O.dx_exact3d(dY3, W3)[:, :, 0], O.dx_exact(dY, Wt), atol=1e-12)
    np.testing.assert_allclose(O.dw_exact3d(X3, dY3, (1, 3, 3))[:, :, 0], O.dw_exact(X, dY), atol=1e-12)
    S = O.sketch(X3, Z3)
    np.testing.assert_allclose(S, O.sketch(X, Z), atol=1e-12)
    np.testing.assert_allclose(O.wgrad_estimate3d(S, dY3, Z3, (1, 3, 3))[:, :, 0], O.wgrad_estimate(S, dY, Z), atol=1e-12)


def test_volume_estimator_recovers_the_exact_gradient_with_an_orthogonal_basis():
    X, Wt, dY = _tiny3(63, B=2, Cin=2, Cout=2, D=2, H=3, W=2)
    n = 2 * 2 * 3 * 2
    Q, _ = np.linalg.qr(_rng(64).standard_normal((n, n)))
    Z = (np.sqrt(n) * Q.T).reshape(n, 2, 2, 3, 2)
    est = O.wgrad_estimate3d(O.sketch(X, Z), dY, Z)
    np.testing.assert_allclose(est, O.dw_exact3d(X, dY), atol=1e-10)
    # a wrong sign of the depth shift would not recover it
    wrong = O.wgrad_contract3d(O.backprobe(O.sketch(X, Z), dY), Z[:, :, ::-1])
    assert O.rel_fro(wrong, O.dw_exact3d(X, dY)) > 0.1


# ---------------------------------------------------------------- Theorem 1: dependence on the block probabilities p_n

def _masked_estimates(X, dY, r, probs, T, seed):
    """T estimates with Eq. (7) probes (block n of a probing vector non-zero with probability probs[n]) and
    the 1/nnz(Z_n) scale of Eq. (8); trials in which a channel was never probed are dropped."""
    g = _rng(seed)
    Cin, H, W = X.shape[1:]
    out = []
    while len(out) < T:
        mask = g.random((r, Cin, 1, 1)) < np.asarray(probs).reshape(1, Cin, 1, 1)
        if not mask.any(axis=0).all():
            continue
        Z = g.standard_normal((r, Cin, H, W)) * mask
        out.append(O.wgrad_estimate(O.sketch(X, Z), dY, Z, scale=O.channel_scale(Z)))
    return np.stack(out)


def test_theorem1_own_block_error_scales_like_inverse_sqrt_of_p_times_r():
    """Single input channel, so that only the first term of Theorem 1's bound is there: ||A^{n,m}||_F / sqrt(p_n r).
    Quartering p_n doubles the rms error (the estimate then averages nnz(Z_n) ~ p_n r probes instead of r)."""
    X, Wt, dY = _tiny(seed=70, B=3, Cin=1, Cout=2, H=4, W=4)
    exact = _loops_dw(X, dY, 3, 3, False)
    r, T = 64, 600
    rms = {}
    for p_ in (1.0, 0.25):
        est = _masked_estimates(X, dY, r, [p_], T, seed=71)
        rms[p_] = np.sqrt(np.mean((est - exact) ** 2))
    ratio = rms[0.25] / rms[1.0]
    assert 1.75 < ratio < 2.4, ratio            # sqrt(1 / 0.25) = 2, a little more because nnz fluctuates
    # and against r at fixed p: four times the probes halve it
    est4 = _masked_estimates(X, dY, 4 * r, [0.25], T, seed=72)
    assert 1.75 < rms[0.25] / np.sqrt(np.mean((est4 - exact) ** 2)) < 2.3


def test_theorem1_crosstalk_from_channel_j_scales_like_sqrt_p_j():
    """Two input channels; the estimate of block (m, n = 0) carries the crosstalk term sqrt(p_1 / p_0) ||A^{.,1}||_F of
    Theorem 1.  With p_0 = 1 fixed, its variance is the single-channel Hutchinson variance plus p_1 ||C_1||_F^2 / r:
    making the other channel's blocks sparser removes crosstalk in proportion."""
    X, Wt, dY = _tiny(seed=73, B=3, Cin=2, Cout=1, H=3, W=3)
    X[:, 1] *= 3.0                                   # make the crosstalk term the larger one
    r, T = 16, 4000
    var = {p1: _masked_estimates(X, dY, r, [1.0, p1], T, seed=74).var(axis=0, ddof=1) for p1 in (1.0, 0.25)}
    for ky in range(3):
        for kx in range(3):
            C = _C_blocks(X, dY, 0, ky, kx)
            own = (np.sum(C[0] ** 2) + np.trace(C[0] @ C[0])) / r
            cross = np.sum(C[1] ** 2) / r
            for p1 in (1.0, 0.25):
                want = own + p1 * cross
                assert 0.8 < var[p1][0, 0, ky, kx] / want < 1.25, (ky, kx, p1, var[p1][0, 0, ky, kx], want)


# --- the plain-C statement of the oracle (oracle/xconv_oracle.c) -------------------------------------------------
# Pinned by the same brute-force loops and by exact recovery (neither goes through the numpy oracle), and compared
# with the numpy oracle on random layers.

def _c():
    from oracle import c_oracle
    c_oracle.lib()
    return c_oracle


@pytest.mark.parametrize("K", [1, 3, 5])
def test_c_oracle_against_brute_force_loops(K):
    C = _c()
    X, Wt, dY = _tiny(seed=10 + K, H=5, W=6 if K == 5 else 4, KH=K, KW=K)
    np.testing.assert_allclose(C.conv_forward(X, Wt), _loops_conv(X, Wt, False), rtol=0, atol=1e-12)
    np.testing.assert_allclose(C.dw_exact(X, dY, K, K), _loops_dw(X, dY, K, K, False), rtol=0, atol=1e-12)
    np.testing.assert_allclose(C.dx_exact(dY, Wt), _loops_dx(dY, Wt, False), rtol=0, atol=1e-12)


def test_c_oracle_recovers_the_exact_gradient_with_an_orthogonal_basis():
    C = _c()
    X, Wt, dY = _tiny(seed=13, B=3, Cin=2, Cout=3, H=4, W=3)
    Z = _orth_probes(2, 4, 3, seed=19)
    est = C.wgrad_estimate(C.sketch(X, Z), dY, Z)
    np.testing.assert_allclose(est, _loops_dw(X, dY, 3, 3, False), rtol=0, atol=1e-11)


def test_c_oracle_wrong_shift_sign_would_fail():
    """The pin above has teeth for the C loops too: probing with the mirrored offset misses the gradient."""
    C = _c()
    X, Wt, dY = _tiny(seed=14, B=3, Cin=2, Cout=3, H=4, W=3)
    Z = _orth_probes(2, 4, 3, seed=20)
    est = C.wgrad_estimate(C.sketch(X, Z), dY, Z)
    mirrored = est[:, :, ::-1, ::-1]
    assert np.abs(mirrored - _loops_dw(X, dY, 3, 3, False)).max() > 1e-3


@pytest.mark.parametrize("seed", range(6))
def test_c_and_numpy_oracles_agree_on_random_layers(seed):
    C = _c()
    g = np.random.default_rng(100 + seed)
    B, Cin, Cout, H, W, r = (int(g.integers(1, 6)) for _ in range(6))
    K = int(g.choice([1, 3, 5]))
    X, dY = g.standard_normal((B, Cin, H, W)), g.standard_normal((B, Cout, H, W))
    Z, Wt = g.standard_normal((r, Cin, H, W)), g.standard_normal((Cout, Cin, K, K))
    sc = g.random(Cin)
    S = O.sketch(X, Z)
    for got, want in ((C.conv_forward(X, Wt), O.conv_forward(X, Wt)), (C.dx_exact(dY, Wt), O.dx_exact(dY, Wt)),
                      (C.dw_exact(X, dY, K, K), O.dw_exact(X, dY, K, K)), (C.sketch(X, Z), S),
                      (C.backprobe(S, dY), O.backprobe(S, dY)),
                      (C.wgrad_estimate(S, dY, Z, K, K, scale=sc), O.wgrad_estimate(S, dY, Z, K, K, scale=sc))):
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-11)


# ------------------------------------------------------------------ Gaussian probes redrawn from a seed

def test_gaussian_probe_series_against_float64_functions():
    """The float32 series the generator is built from, against numpy's float64 log, cos and sin on the same arguments."""
    t = np.arange(1, 1 << 24, 2, dtype=np.int64)[::53]
    t = np.concatenate([t, [1, 3, (1 << 24) - 1, (1 << 23) - 1, (1 << 23) + 1, 11863283, 11863285]])   # ends, sqrt(2) cut
    ref = np.log(t / 2.0 ** 24)
    assert np.max(np.abs(O._ln_f32(t) - ref) / np.maximum(np.abs(ref), 1e-3)) < 5e-7
    c, s = O._sincos_2pi_f32(t)
    a = 2.0 * np.pi * t / 2.0 ** 24
    assert np.max(np.abs(c - np.cos(a))) < 2.5e-7 and np.max(np.abs(s - np.sin(a))) < 2.5e-7
    # every octant boundary from both sides
    tb = np.array([k * (1 << 21) + d for k in range(8) for d in (1, (1 << 21) - 1)], dtype=np.int64)
    c, s = O._sincos_2pi_f32(tb)
    a = 2.0 * np.pi * tb / 2.0 ** 24
    assert np.max(np.abs(c - np.cos(a))) < 2.5e-7 and np.max(np.abs(s - np.sin(a))) < 2.5e-7


def test_gaussian_probes_follow_the_stated_definition():
    """Entries recomputed one by one from the definition in float64 (Philox block e div 4 with counter word 2 = 1,
    uniforms from the top 23 bits, Box-Muller: cosine for even entries, sine for odd ones), in memory order."""
    import math
    seed, r, Cin, H, W = 0x0123456789ABCDEF, 3, 5, 4, 6
    Z = O.gaussian_probes(seed, r, Cin, H, W)
    flat = Z.transpose(0, 2, 3, 1).reshape(-1)               # entry e = ((j*H + y)*W + x)*Cin + n
    for e in list(range(0, 24)) + [101, 102, 103, 357, 358, 359]:
        b = e // 4
        w = [int(v[0]) for v in O.philox4x32_10(([b & 0xFFFFFFFF], [b >> 32], [1], [0]),
                                             (seed & 0xFFFFFFFF, seed >> 32))]
        pair, odd = (e % 4) // 2, e % 2
        ua = (2 * (w[2 * pair] >> 9) + 1) / 2.0 ** 24
        ub = (2 * (w[2 * pair + 1] >> 9) + 1) / 2.0 ** 24
        rad = math.sqrt(-2.0 * math.log(ua))
        want = rad * (math.sin(2 * math.pi * ub) if odd else math.cos(2 * math.pi * ub))
        assert abs(flat[e] - want) < 2e-6 * max(1.0, abs(want)), (e, flat[e], want)
    assert np.array_equal(Z.astype(np.float32).astype(np.float64), Z)          # float32 values


def test_gaussian_probes_are_standard_normal_independent_and_apart_from_the_rademacher_stream():
    from scipy import stats
    r, Cin, H, W = 64, 8, 20, 20
    Z = O.gaussian_probes(99, r, Cin, H, W)
    z = Z.ravel()
    n = z.size
    assert abs(z.mean()) < 5.0 / np.sqrt(n) and abs(z.var() - 1.0) < 5.0 * np.sqrt(2.0 / n)
    assert abs(np.mean(z ** 3)) < 5.0 * np.sqrt(15.0 / n) and abs(np.mean(z ** 4) - 3.0) < 5.0 * np.sqrt(96.0 / n)
    assert stats.kstest(z[::3], "norm").pvalue > 1e-3
    # E[z z^T] = I (Section 3, "E(z z^T) = I"): Gram matrix of the probes over their entries, off-diagonal ~ 1/sqrt(len)
    G = Z.reshape(r, -1) @ Z.reshape(r, -1).T / (Cin * H * W)
    assert np.abs(G - np.eye(r)).max() < 6.0 / np.sqrt(Cin * H * W) * np.sqrt(2.0)
    # neighbours in memory (the cosine and the sine of one pair, and the two pairs of a block) are uncorrelated
    f = Z.transpose(0, 2, 3, 1).reshape(-1)
    for lag in (1, 2, 3, 4):
        assert abs(np.mean(f[:-lag] * f[lag:])) < 5.0 / np.sqrt(n)
    # another seed, and the Rademacher stream of the same seed, are unrelated to it
    assert abs(np.mean(z * O.gaussian_probes(100, r, Cin, H, W).ravel())) < 5.0 / np.sqrt(n)
    assert abs(np.mean(np.sign(z) * O.rademacher_probes(99, r, Cin, H, W).ravel())) < 5.0 / np.sqrt(n)


def test_estimator_on_gaussian_probes_from_seeds_is_unbiased_with_the_gaussian_variance():
    """Mean over seeds -> exact gradient, and the spread is the closed-form Hutchinson variance with c = 0 (Gaussian)."""
    X, Wt, dY = _tiny(seed=44, B=3, Cin=2, Cout=2, H=4, W=4)
    r, T = 4, 1500
    est = np.stack([O.wgrad_estimate(O.sketch(X, Z), dY, Z) for Z in
                    (O.gaussian_probes(5000 + t, r, 2, 4, 4) for t in range(T))])
    exact = O.dw_exact(X, dY)
    sd = est.std(axis=0)
    assert np.all(np.abs(est.mean(axis=0) - exact) < 4.5 * sd / np.sqrt(T))
    # against Rademacher probes the Gaussian estimator has the larger own-block variance (the -2 sum A_ii^2 term is absent)
    est_r = np.stack([O.wgrad_estimate(O.sketch(X, Z), dY, Z) for Z in
                      (O.rademacher_probes(5000 + t, r, 2, 4, 4) for t in range(T))])
    assert est.var(axis=0).sum() > est_r.var(axis=0).sum()


# ------------------------------------------------------------------ block-sparse probes (Eq. 7) redrawn from a seed

def test_block_keep_mask_follows_the_stated_definition():
    seed, r, Cin, p = 0xFEDCBA9876543210, 7, 5, 0.3
    keep = O.block_keep_mask(seed, r, Cin, p)
    thr = int(np.floor(p * 2.0 ** 32))
    for g in range(r * Cin):
        b = g // 4
        w = [int(v[0]) for v in O.philox4x32_10(([b & 0xFFFFFFFF], [b >> 32], [2], [0]), (seed & 0xFFFFFFFF, seed >> 32))]
        assert bool(keep[g // Cin, g % Cin]) == (w[g % 4] < thr)
    assert O.block_keep_mask(seed, r, Cin, 1.0).all() and not O.block_keep_mask(seed, r, Cin, 0.0).any()


def test_block_keep_mask_keeps_a_share_p_of_independent_blocks():
    r, Cin = 400, 300
    n = r * Cin
    for p in (0.125, 0.5, 0.9):
        k = O.block_keep_mask(11, r, Cin, p).astype(np.float64)
        assert abs(k.mean() - p) < 5.0 * np.sqrt(p * (1 - p) / n)
        c = k - p
        for a, b in ((c[:, :-1], c[:, 1:]), (c[:-1], c[1:])):        # neighbours along the channels, along the probes
            assert abs(np.mean(a * b)) < 5.0 * p * (1 - p) / np.sqrt(a.size)
    # another seed gives another mask; the mask is unrelated to the signs of the same seed
    k1, k2 = O.block_keep_mask(11, r, Cin, 0.5), O.block_keep_mask(12, r, Cin, 0.5)
    assert 0.4 < np.mean(k1 != k2) < 0.6


@pytest.mark.parametrize("gaussian", [False, True])
def test_block_sparse_probes_are_the_dense_ones_with_blocks_dropped_and_keep_the_estimator_unbiased(gaussian):
    r, Cin, H, W, p = 12, 3, 4, 4, 0.5
    Z = O.block_sparse_probes(21, r, Cin, H, W, p, gaussian)
    dense = (O.gaussian_probes if gaussian else O.rademacher_probes)(21, r, Cin, H, W)
    keep = O.block_keep_mask(21, r, Cin, p)
    assert np.array_equal(Z[keep], dense[keep]) and not Z[~keep].any() and 0 < keep.sum() < keep.size
    # Eq. 8: with the 1/nnz(Z_n) scale the mean over seeds is the exact gradient
    X, Wt, dY = _tiny(seed=45, B=3, Cin=Cin, Cout=2, H=H, W=W)
    T = 1200
    est = []
    for t in range(T):
        Zt = O.block_sparse_probes(7000 + t, r, Cin, H, W, p, gaussian)
        est.append(O.wgrad_estimate(O.sketch(X, Zt), dY, Zt, scale=O.channel_scale(Zt)))
    est = np.stack(est)
    # a channel whose r blocks are all dropped (probability 2^-12 per channel and seed) estimates 0: negligible bias
    assert np.all(np.abs(est.mean(axis=0) - O.dw_exact(X, dY)) < 4.5 * est.std(axis=0) / np.sqrt(T) + 1e-3 * np.abs(O.dw_exact(X, dY)).max())
