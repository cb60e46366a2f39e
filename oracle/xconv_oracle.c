/* Float64 CPU oracle for the XConv layer in plain C (test infrastructure, not product code).
 *
 * A second statement of the formulas that oracle/xconv_oracle.py writes in numpy: plain nested loops over logical
 * (batch, channel, y, x) arrays of doubles, one loop nest per formula, no blocking, no reordering beyond what the
 * formula states.  OpenMP spreads the outermost loop over the host's cores; the sums inside run in the order
 * written.  Only the tests and the benchmark's CPU-baseline leg use it; it shares no code with the CUDA path.
 *
 * Shifts are truncating (out-of-range pixels read as zero), matching the zero-padded convolution of the layers this
 * library serves; offset (ky, kx) of a KH x KW kernel moves by (ky - ph, kx - pw), ph = (KH-1)/2, pw = (KW-1)/2.
 *
 * Pinned by tests/test_oracle_pins.py (against the numpy oracle on random layers, against brute-force pins that do
 * not go through either, and by exact recovery with an orthogonal probe basis).
 */
#include <stddef.h>

#define IDX4(a, b, c, d, B_, C_, D_) ((((size_t)(a) * (B_) + (b)) * (C_) + (c)) * (D_) + (d))

/* Eq. 5 / Algorithm 1 forward step 1: Y[b,m,y,x] = sum_{n,ky,kx} W[m,n,ky,kx] X[b,n,y+ky-ph,x+kx-pw]. */
void xo_conv_forward(const double* X, const double* W, double* Y, int B, int Cin, int Cout, int H, int Wd, int KH,
                     int KW) {
  const int ph = (KH - 1) / 2, pw = (KW - 1) / 2;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < B; ++b)
    for (int m = 0; m < Cout; ++m)
      for (int y = 0; y < H; ++y)
        for (int x = 0; x < Wd; ++x) {
          double s = 0.0;
          for (int n = 0; n < Cin; ++n)
            for (int ky = 0; ky < KH; ++ky)
              for (int kx = 0; kx < KW; ++kx) {
                const int yy = y + ky - ph, xx = x + kx - pw;
                if (yy >= 0 && yy < H && xx >= 0 && xx < Wd)
                  s += W[IDX4(m, n, ky, kx, Cin, KH, KW)] * X[IDX4(b, n, yy, xx, Cin, H, Wd)];
              }
          Y[IDX4(b, m, y, x, Cout, H, Wd)] = s;
        }
}

/* Exact input gradient: dX[b,n,y,x] = sum_{m,ky,kx} W[m,n,ky,kx] dY[b,m,y-(ky-ph),x-(kx-pw)]. */
void xo_dx_exact(const double* dY, const double* W, double* dX, int B, int Cin, int Cout, int H, int Wd, int KH,
                 int KW) {
  const int ph = (KH - 1) / 2, pw = (KW - 1) / 2;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < B; ++b)
    for (int n = 0; n < Cin; ++n)
      for (int y = 0; y < H; ++y)
        for (int x = 0; x < Wd; ++x) {
          double s = 0.0;
          for (int m = 0; m < Cout; ++m)
            for (int ky = 0; ky < KH; ++ky)
              for (int kx = 0; kx < KW; ++kx) {
                const int yy = y - (ky - ph), xx = x - (kx - pw);
                if (yy >= 0 && yy < H && xx >= 0 && xx < Wd)
                  s += W[IDX4(m, n, ky, kx, Cin, KH, KW)] * dY[IDX4(b, m, yy, xx, Cout, H, Wd)];
              }
          dX[IDX4(b, n, y, x, Cin, H, Wd)] = s;
        }
}

/* Exact weight gradient (Eq. 2 with the truncating shift): dW[m,n,ky,kx] = sum_{b,y,x} dY[b,m,y,x] X[b,n,y+ky-ph,x+kx-pw]. */
void xo_dw_exact(const double* X, const double* dY, double* dW, int B, int Cin, int Cout, int H, int Wd, int KH,
                 int KW) {
  const int ph = (KH - 1) / 2, pw = (KW - 1) / 2;
#pragma omp parallel for collapse(2)
  for (int m = 0; m < Cout; ++m)
    for (int n = 0; n < Cin; ++n)
      for (int ky = 0; ky < KH; ++ky)
        for (int kx = 0; kx < KW; ++kx) {
          double s = 0.0;
          for (int b = 0; b < B; ++b)
            for (int y = 0; y < H; ++y)
              for (int x = 0; x < Wd; ++x) {
                const int yy = y + ky - ph, xx = x + kx - pw;
                if (yy >= 0 && yy < H && xx >= 0 && xx < Wd)
                  s += dY[IDX4(b, m, y, x, Cout, H, Wd)] * X[IDX4(b, n, yy, xx, Cin, H, Wd)];
              }
          dW[IDX4(m, n, ky, kx, Cin, KH, KW)] = s;
        }
}

/* Algorithm 1 forward step 3 (the sketch, X-bar = Z^T X): S[j,b] = sum_{n,y,x} Z[j,n,y,x] X[b,n,y,x]; K = Cin*H*W. */
void xo_sketch(const double* X, const double* Z, double* S, int B, int r, size_t K) {
#pragma omp parallel for collapse(2)
  for (int j = 0; j < r; ++j)
    for (int b = 0; b < B; ++b) {
      double s = 0.0;
      for (size_t k = 0; k < K; ++k) s += Z[(size_t)j * K + k] * X[(size_t)b * K + k];
      S[(size_t)j * B + b] = s;
    }
}

/* Algorithm 1 backward step 3: L[j,q] = sum_b S[j,b] dY[b,q]; Q = Cout*H*W. */
void xo_backprobe(const double* S, const double* dY, double* L, int r, int B, size_t Q) {
#pragma omp parallel for
  for (int j = 0; j < r; ++j)
    for (size_t q = 0; q < Q; ++q) {
      double s = 0.0;
      for (int b = 0; b < B; ++b) s += S[(size_t)j * B + b] * dY[(size_t)b * Q + q];
      L[(size_t)j * Q + q] = s;
    }
}

/* Algorithm 1 backward step 4 (Eq. 6 block by block; Eq. 8 with scale[n] = 1/nnz(Z_n)):
 * dW[m,n,ky,kx] = scale[n] * sum_{j,y,x} L[j,m,y,x] Z[j,n,y+ky-ph,x+kx-pw]. */
void xo_wgrad_contract(const double* L, const double* Z, const double* scale, double* dW, int r, int Cin, int Cout,
                       int H, int Wd, int KH, int KW) {
  const int ph = (KH - 1) / 2, pw = (KW - 1) / 2;
#pragma omp parallel for collapse(2)
  for (int m = 0; m < Cout; ++m)
    for (int n = 0; n < Cin; ++n)
      for (int ky = 0; ky < KH; ++ky)
        for (int kx = 0; kx < KW; ++kx) {
          double s = 0.0;
          for (int j = 0; j < r; ++j)
            for (int y = 0; y < H; ++y)
              for (int x = 0; x < Wd; ++x) {
                const int yy = y + ky - ph, xx = x + kx - pw;
                if (yy >= 0 && yy < H && xx >= 0 && xx < Wd)
                  s += L[IDX4(j, m, y, x, Cout, H, Wd)] * Z[IDX4(j, n, yy, xx, Cin, H, Wd)];
              }
          dW[IDX4(m, n, ky, kx, Cin, KH, KW)] = scale[n] * s;
        }
}
