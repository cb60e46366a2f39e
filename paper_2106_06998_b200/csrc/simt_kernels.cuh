// FP32-FMA kernels for every step of the layer.  They serve float storage (where the 1e-5 parity
// bar rules out TF32/BF16 tensor-core products) and any bfloat16 shape the tcgen05 kernels do not
// cover.  All tensors are channels-last; all sums are accumulated in float.
#pragma once

#include "common.cuh"

namespace xconv {

// v modulo n for v that may be negative: the pixel a circular shift reads (the paper's T_k; Section 3).
__device__ __forceinline__ int wrap_index(int v, int n) { v %= n; return v < 0 ? v + n : v; }

// ---------------------------------------------------------------------------------------------
// Sketch, S = Z^T X (Algorithm 1 forward step 3): D[m][n] = sum_k A[m,k] * Bm[n,k], both operands
// contiguous along k (k runs over pixel-major, channel-minor positions of one sample / one probe).
// Split over k: block z writes its partial tile to part[z][M][N]; reduce_partials sums them in order.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) gemm_tn_simt(const T* __restrict__ A, const T* __restrict__ Bm,
                                                    float* __restrict__ part, int M, int N, long K,
                                                    long k_per_split, int vec) {
  // 64 x 64 outputs per block, 32 k per step (128 consecutive bytes of a row; rows lie K elements apart);
  // the loads of the next step are issued before the arithmetic of this one.
  constexpr int KS = 32;
  __shared__ __align__(16) float As[KS][68];
  __shared__ __align__(16) float Bs[KS][68];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const long kb = (long)blockIdx.z * k_per_split;
  const long ke = min(K, kb + k_per_split);
  // A warp reads 32 bytes (two threads) of 16 rows at a time, and warps 0..3 / 4..7 cover the eight 16-byte
  // pieces of a step for rows 0..15 / 16..31: the transposing stores below then hit 32 different banks
  // ((lk + c) * 68 + row = 16 * (lane & 1) + (lane >> 1) + const, modulo 32).
  const int lane_ = tid & 31, warp_ = tid >> 5;
  const int lr = (warp_ >> 2) * 16 + (lane_ >> 1), lk = ((warp_ & 3) * 2 + (lane_ & 1)) * 4;   // rows lr and lr + 32
  const int tm = tid >> 4, tn = tid & 15;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 a[2], b[2];
  auto fetch = [&](long k0) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int row = lr + 32 * h;
      a[h] = (m0 + row < M) ? ld4_guard(A + (long)(m0 + row) * K, k0 + lk, ke, vec != 0) : zero;
      b[h] = (n0 + row < N) ? ld4_guard(Bm + (long)(n0 + row) * K, k0 + lk, ke, vec != 0) : zero;
    }
  };
  if (kb < ke) fetch(kb);
  for (long k0 = kb; k0 < ke; k0 += KS) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int row = lr + 32 * h;
      As[lk + 0][row] = a[h].x; As[lk + 1][row] = a[h].y; As[lk + 2][row] = a[h].z; As[lk + 3][row] = a[h].w;
      Bs[lk + 0][row] = b[h].x; Bs[lk + 1][row] = b[h].y; Bs[lk + 2][row] = b[h].z; Bs[lk + 3][row] = b[h].w;
    }
    __syncthreads();
    if (k0 + KS < ke) fetch(k0 + KS);
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
      const float4 av = *reinterpret_cast<const float4*>(&As[kk][tm * 4]);
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tn * 4]);
      const float ar[4] = {av.x, av.y, av.z, av.w};
      const float br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* out = part + (long)blockIdx.z * M * N;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + tm * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tn * 4 + j;
      if (n < N) out[(long)m * N + n] = acc[i][j];
    }
  }
}

// The same for float operands whose rows start on 16-byte boundaries (K a multiple of 4, k ranges multiples of 32):
// the tiles are copied with cp.async straight into k-contiguous rows of shared memory, three stages deep, and the
// arithmetic reads four consecutive k of a row with one 128-bit load (the kernel above transposes every tile
// through registers with scalar stores, and its warps wait on those between the two barriers of a step).  A thread
// owns rows tm + 16 i and columns tn + 16 j, i, j < 4: the sixteen lanes that differ in tn then read consecutive
// rows, 36 floats apart, which spread over all banks.  Dynamic shared memory: GT_STAGES * 128 * GT_LD floats.
constexpr int GT_KS = 32, GT_LD = 36, GT_STAGES = 3;
__device__ __forceinline__ void cp_async16_f(float* dst, const float* src, bool valid) {
  // src-size 0 fills the 16 bytes with zeros without reading (src is then any valid address)
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src),
               "r"(valid ? 16 : 0) : "memory");
}
static __global__ void __launch_bounds__(256) gemm_tn_simt_async(const float* __restrict__ A, const float* __restrict__ Bm,
                                                          float* __restrict__ part, int M, int N, long K, long k_per_split) {
  extern __shared__ __align__(16) float gt_tiles[];       // [stage][A rows 0..63 | B rows 0..63][GT_LD]
  const int tid = threadIdx.x;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const long kb = (long)blockIdx.z * k_per_split;
  const long ke = min(K, kb + k_per_split);
  const int tm = tid >> 4, tn = tid & 15;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  auto fetch = [&](int stage, long k0) {
    float* t = gt_tiles + stage * 128 * GT_LD;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + 256 * i, row = idx >> 3, c = (idx & 7) * 4;       // rows 0..63: A, 64..127: B
      const bool is_a = row < 64;
      const int g = is_a ? m0 + row : n0 + row - 64;
      const bool ok = (is_a ? g < M : g < N) && k0 + c < ke;
      const float* src = (is_a ? A : Bm) + (long)g * K + k0 + c;
      cp_async16_f(t + row * GT_LD + c, ok ? src : A, ok);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  const long steps = kb < ke ? (ke - kb + GT_KS - 1) / GT_KS : 0;
  for (int s = 0; s < GT_STAGES - 1; ++s) {
    if (s < steps) fetch(s, kb + (long)s * GT_KS);
    else asm volatile("cp.async.commit_group;" ::: "memory");          // keeps the group count in step
  }
  for (long st = 0; st < steps; ++st) {
    // the copies of step st are the oldest group but GT_STAGES - 2
    asm volatile("cp.async.wait_group %0;" ::"n"(GT_STAGES - 2) : "memory");
    __syncthreads();             // ... and every thread is done with the stage that the next fetch overwrites
    if (st + GT_STAGES - 1 < steps) fetch((int)((st + GT_STAGES - 1) % GT_STAGES), kb + (st + GT_STAGES - 1) * GT_KS);
    else asm volatile("cp.async.commit_group;" ::: "memory");
    const float* ta = gt_tiles + (int)(st % GT_STAGES) * 128 * GT_LD;
    const float* tb = ta + 64 * GT_LD;
#pragma unroll
    for (int k4 = 0; k4 < GT_KS; k4 += 4) {
      float4 a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const float4*>(ta + (tm + 16 * i) * GT_LD + k4);
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = *reinterpret_cast<const float4*>(tb + (tn + 16 * j) * GT_LD + k4);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(a[i].x, b[j].x, acc[i][j]);
          acc[i][j] = fmaf(a[i].y, b[j].y, acc[i][j]);
          acc[i][j] = fmaf(a[i].z, b[j].z, acc[i][j]);
          acc[i][j] = fmaf(a[i].w, b[j].w, acc[i][j]);
        }
    }
  }
  float* out = part + (long)blockIdx.z * M * N;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + tm + 16 * i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tn + 16 * j;
      if (n < N) out[(long)m * N + n] = acc[i][j];
    }
  }
}

// out[i] = scale(i) * sum_s part[s][i].  Eight threads share an output and take the splits in turn (one
// thread per output would walk a chain of `splits` dependent loads); their eight sums are added in a
// fixed order, so results are reproducible.  scale(i) = chan_scale[i % period] if chan_scale else alpha.
// Launch with 256 threads: 32 outputs per block.
constexpr int RP_OUT = 32, RP_LANES = 8;
static __global__ void __launch_bounds__(RP_OUT * RP_LANES)
reduce_partials(const float* __restrict__ part, float* __restrict__ out, long count, int splits, float alpha,
                const float* __restrict__ chan_scale, int period) {
  __shared__ float acc[RP_LANES][RP_OUT];
  const int o = threadIdx.x % RP_OUT, g = threadIdx.x / RP_OUT;
  const long i = (long)blockIdx.x * RP_OUT + o;
  float s = 0.f;
  if (i < count) {
#pragma unroll 4
    for (int k = g; k < splits; k += RP_LANES) s += part[(long)k * count + i];
  }
  acc[g][o] = s;
  __syncthreads();
  if (g != 0 || i >= count) return;
  float t = acc[0][o];
#pragma unroll
  for (int l = 1; l < RP_LANES; ++l) t += acc[l][o];
  out[i] = t * (chan_scale ? chan_scale[i % period] : alpha);
}

// ---------------------------------------------------------------------------------------------
// Back-probe, L = S dY^T (Algorithm 1 backward step 3): L[j][q] = sum_b S[j,b] * dY[b,q], q running
// over the H*W*Cout positions of one sample.  A block owns 4 * blockDim.x q and 16 probes (the host picks the block
// size, a multiple of 32 up to 256, so that the grid fills whole waves of the SMs).
// ---------------------------------------------------------------------------------------------
template <typename T, typename TL>
__global__ void __launch_bounds__(256) backprobe_simt(const float* __restrict__ S, const T* __restrict__ dY,
                                                      TL* __restrict__ L, int r, int B, long Q, int vec) {
  __shared__ __align__(16) float Ss[128][16];
  const int tid = threadIdx.x;
  const long q = ((long)blockIdx.x * blockDim.x + tid) * 4;
  const int j0 = blockIdx.y * 16;
  float4 acc[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);

  for (int b0 = 0; b0 < B; b0 += 128) {
    for (int idx = tid; idx < 128 * 16; idx += blockDim.x) {
      const int jj = idx >> 7, bb = idx & 127;   // consecutive threads read consecutive b
      Ss[bb][jj] = (b0 + bb < B && j0 + jj < r) ? S[(long)(j0 + jj) * B + b0 + bb] : 0.f;
    }
    __syncthreads();
    if (q < Q) {
      const int nb = min(128, B - b0);
      // eight samples at a time: their loads are issued together (one load in flight per thread keeps
      // only a few KB per SM on the way from HBM), then consumed in order
      for (int bb0 = 0; bb0 < nb; bb0 += 8) {
        float4 d8[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
          d8[u] = bb0 + u < nb ? ld4_guard(dY + (long)(b0 + bb0 + u) * Q, q, Q, vec != 0) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float4 d = d8[u];
          const int bb = min(bb0 + u, 127);          // rows past nb hold zeros in d8; any valid row of Ss will do
#pragma unroll
          for (int j4 = 0; j4 < 4; ++j4) {
            const float4 s = *reinterpret_cast<const float4*>(&Ss[bb][j4 * 4]);
            const float sr[4] = {s.x, s.y, s.z, s.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              float4& a = acc[j4 * 4 + i];
              a.x = fmaf(sr[i], d.x, a.x); a.y = fmaf(sr[i], d.y, a.y);
              a.z = fmaf(sr[i], d.z, a.z); a.w = fmaf(sr[i], d.w, a.w);
            }
          }
        }
      }
    }
    __syncthreads();
  }
  if (q < Q) {
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (j0 + j < r) st4_guard(L + (long)(j0 + j) * Q, q, Q, vec != 0, acc[j]);
  }
}

// ---------------------------------------------------------------------------------------------
// Offset contraction (Algorithm 1 backward step 4; Eq. 6 block by block):
//   part[s][m][tap][n] = sum over the (j, y, x) of split s of L[j,y,x,m] * Z[j,y+ky-p,x+kx-p,n].
// The shift of each kernel offset is an index offset into a haloed probe tile in shared memory, so
// no shifted or im2col copy of Z exists.  A block owns 32 output x 64 input channels and DYS rows of
// the KS x KS offsets (all of them for 3 x 3; one row at a time for 5 x 5, whose 25 x 8 sums per thread
// would not fit the registers); work items are (probe, row, 32-pixel chunk) triples dealt to grid.z
// splits in order.  grid.x = (blocks of 64 input channels) x (KD * KS / DYS groups of offset rows).
// Volumes (D planes per probe, KD planes per kernel): an "offset row" is a (dz, dy) pair, rho = kz * KS + ky,
// and a work item carries its plane z; a row whose plane z + dz lies outside the volume reads zeros.
// ---------------------------------------------------------------------------------------------
template <typename TL, typename TZ, int KS, int KD, int DYS, bool VEC>
__global__ void __launch_bounds__(256) contract_simt(const TL* __restrict__ L, const TZ* __restrict__ Z,
                                                     float* __restrict__ part, int r, int D, int H, int W, int Cin,
                                                     int Cout, long items_per_split, int circ) {
  constexpr int P = (KS - 1) / 2, PD = (KD - 1) / 2, XC = 32, T = DYS * KS, TALL = KD * KS * KS;
  __shared__ __align__(16) float Ls[XC][32];
  __shared__ __align__(16) float Zs[DYS][XC + KS - 1][64];
  const int tid = threadIdx.x;
  const int nblocks = (Cin + 63) / 64;
  const int dy0 = (blockIdx.x / nblocks) * DYS;          // first offset row (kz * KS + ky) of this block
  const int n0 = (blockIdx.x % nblocks) * 64, m0 = blockIdx.y * 32;
  const int tx = tid & 15, ty = tid >> 4;
  const int chunks = (W + XC - 1) / XC;
  const long items = (long)r * D * H * chunks;
  const long ib = (long)blockIdx.z * items_per_split;
  const long ie = min(items, ib + items_per_split);

  float acc[T][2][4];
#pragma unroll
  for (int t = 0; t < T; ++t)
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int k = 0; k < 4; ++k) acc[t][i][k] = 0.f;

  // (x chunk, row, plane) of the first item, then stepped along: a 64-bit division per item costs as much as a
  // sixth of the item's arithmetic
  int xc = (int)(ib % chunks), y = (int)((ib / chunks) % H);
  long jz = ib / ((long)chunks * H);                      // plane index j * D + z
  int z = (int)(jz % D);
  for (long it = ib; it < ie; ++it) {
    const int x0 = xc * XC;
    if (VEC) {
      // channel counts are multiples of 4: four consecutive channels per load (the tiles fill in a quarter
      // of the instructions; the fill costs about as much as the arithmetic otherwise)
      {
        const int mm = (tid & 7) * 4, px = tid >> 3;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (x0 + px < W && m0 + mm < Cout) v = ld4(L + ((jz * H + y) * W + x0 + px) * Cout + m0 + mm);
        *reinterpret_cast<float4*>(&Ls[px][mm]) = v;
      }
      for (int idx = tid; idx < DYS * (XC + KS - 1) * 16; idx += 256) {
        const int nn = (idx & 15) * 4;
        const int px = (idx >> 4) % (XC + KS - 1);
        const int dy = (idx >> 4) / (XC + KS - 1);
        const int rho = dy0 + dy, dz = rho / KS - PD;
        int yy = y + rho % KS - P, xx = x0 + px - P;
        if (circ) { yy = wrap_index(yy, H); xx = wrap_index(xx, W); }   // circular shift instead of zero fill
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (z + dz >= 0 && z + dz < D && yy >= 0 && yy < H && xx >= 0 && xx < W && n0 + nn < Cin)
          v = ld4(Z + (((jz + dz) * H + yy) * W + xx) * Cin + n0 + nn);
        *reinterpret_cast<float4*>(&Zs[dy][px][nn]) = v;
      }
    } else {
    for (int idx = tid; idx < XC * 32; idx += 256) {
      const int mm = idx & 31, px = idx >> 5;
      float v = 0.f;
      if (x0 + px < W && m0 + mm < Cout) v = to_f(L[((jz * H + y) * W + x0 + px) * Cout + m0 + mm]);
      Ls[px][mm] = v;
    }
    for (int idx = tid; idx < DYS * (XC + KS - 1) * 64; idx += 256) {
      const int nn = idx & 63;
      const int px = (idx >> 6) % (XC + KS - 1);
      const int dy = (idx >> 6) / (XC + KS - 1);
      const int rho = dy0 + dy, dz = rho / KS - PD;
      int yy = y + rho % KS - P, xx = x0 + px - P;
      if (circ) { yy = wrap_index(yy, H); xx = wrap_index(xx, W); }
      float v = 0.f;
      if (z + dz >= 0 && z + dz < D && yy >= 0 && yy < H && xx >= 0 && xx < W && n0 + nn < Cin)
        v = to_f(Z[(((jz + dz) * H + yy) * W + xx) * Cin + n0 + nn]);
      Zs[dy][px][nn] = v;
    }
    }
    __syncthreads();
#pragma unroll 4
    for (int px = 0; px < XC; ++px) {
      const float2 l = *reinterpret_cast<const float2*>(&Ls[px][ty * 2]);
#pragma unroll
      for (int dy = 0; dy < DYS; ++dy)
#pragma unroll
        for (int dx = 0; dx < KS; ++dx) {
          const float4 z = *reinterpret_cast<const float4*>(&Zs[dy][px + dx][tx * 4]);
          float* a0 = acc[dy * KS + dx][0];
          float* a1 = acc[dy * KS + dx][1];
          a0[0] = fmaf(l.x, z.x, a0[0]); a0[1] = fmaf(l.x, z.y, a0[1]);
          a0[2] = fmaf(l.x, z.z, a0[2]); a0[3] = fmaf(l.x, z.w, a0[3]);
          a1[0] = fmaf(l.y, z.x, a1[0]); a1[1] = fmaf(l.y, z.y, a1[1]);
          a1[2] = fmaf(l.y, z.z, a1[2]); a1[3] = fmaf(l.y, z.w, a1[3]);
        }
    }
    __syncthreads();
    if (++xc == chunks) { xc = 0; if (++y == H) { y = 0; ++jz; if (++z == D) z = 0; } }
  }
  float* out = part + (long)blockIdx.z * Cout * TALL * Cin;
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int m = m0 + ty * 2 + i;
    if (m >= Cout) continue;
#pragma unroll
    for (int t = 0; t < T; ++t)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int n = n0 + tx * 4 + k;
        if (n < Cin) out[((long)m * TALL + dy0 * KS + t) * Cin + n] = acc[t][i][k];
      }
  }
}

// The same contraction for float storage with channel counts that are multiples of 4, tiles copied with cp.async
// into two sets of buffers: the tiles of the next work item are on their way while this one is multiplied (the kernel
// above loads, waits, multiplies, and leaves the overlap to the second block of the SM).  Dynamic shared memory:
// 2 * contract_async_tile_floats<KS, DYS>() floats.
template <int KS, int DYS>
__host__ __device__ constexpr int contract_async_tile_floats() { return 32 * 32 + DYS * (32 + KS - 1) * 64; }

template <int KS, int KD, int DYS>
__global__ void __launch_bounds__(256) contract_simt_async(const float* __restrict__ L, const float* __restrict__ Z,
                                                           float* __restrict__ part, int r, int D, int H, int W, int Cin,
                                                           int Cout, long items_per_split, int circ) {
  constexpr int P = (KS - 1) / 2, PD = (KD - 1) / 2, XC = 32, T = DYS * KS, TALL = KD * KS * KS, ZW = XC + KS - 1;
  constexpr int TILE = contract_async_tile_floats<KS, DYS>();
  extern __shared__ __align__(16) float tiles[];          // [2][ Ls[XC][32] | Zs[DYS][ZW][64] ]
  const int tid = threadIdx.x;
  const int nblocks = (Cin + 63) / 64;
  const int dy0 = (blockIdx.x / nblocks) * DYS;
  const int n0 = (blockIdx.x % nblocks) * 64, m0 = blockIdx.y * 32;
  const int tx = tid & 15, ty = tid >> 4;
  const int chunks = (W + XC - 1) / XC;
  const long items = (long)r * D * H * chunks;
  const long ib = (long)blockIdx.z * items_per_split;
  const long ie = min(items, ib + items_per_split);

  float acc[T][2][4];
#pragma unroll
  for (int t = 0; t < T; ++t)
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int k = 0; k < 4; ++k) acc[t][i][k] = 0.f;

  // coordinates of the item whose tiles are fetched next (one ahead of the item being multiplied)
  int xc = (int)(ib % chunks), y = (int)((ib / chunks) % H);
  long jz = ib / ((long)chunks * H);
  int z = (int)(jz % D);
  auto fetch = [&](int buf) {
    float* Ls = tiles + buf * TILE;
    float* Zs = Ls + XC * 32;
    const int x0 = xc * XC;
    {
      const int mm = (tid & 7) * 4, px = tid >> 3;
      const bool ok = x0 + px < W && m0 + mm < Cout;
      cp_async16_f(Ls + px * 32 + mm, ok ? L + ((jz * H + y) * W + x0 + px) * Cout + m0 + mm : L, ok);
    }
    for (int idx = tid; idx < DYS * ZW * 16; idx += 256) {
      const int nn = (idx & 15) * 4;
      const int px = (idx >> 4) % ZW;
      const int dy = (idx >> 4) / ZW;
      const int rho = dy0 + dy, dz = rho / KS - PD;
      int yy = y + rho % KS - P, xx = x0 + px - P;
      if (circ) { yy = wrap_index(yy, H); xx = wrap_index(xx, W); }
      const bool ok = z + dz >= 0 && z + dz < D && yy >= 0 && yy < H && xx >= 0 && xx < W && n0 + nn < Cin;
      cp_async16_f(Zs + (dy * ZW + px) * 64 + nn, ok ? Z + (((jz + dz) * H + yy) * W + xx) * Cin + n0 + nn : Z, ok);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (++xc == chunks) { xc = 0; if (++y == H) { y = 0; ++jz; if (++z == D) z = 0; } }
  };

  int buf = 0;
  if (ib < ie) fetch(0);
  for (long it = ib; it < ie; ++it) {
    if (it + 1 < ie) {
      fetch(buf ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");       // this item's copies have landed; the next item's may be in flight
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const float* Ls = tiles + buf * TILE;
    const float* Zs = Ls + XC * 32;
#pragma unroll 4
    for (int px = 0; px < XC; ++px) {
      const float2 l = *reinterpret_cast<const float2*>(Ls + px * 32 + ty * 2);
#pragma unroll
      for (int dy = 0; dy < DYS; ++dy)
#pragma unroll
        for (int dx = 0; dx < KS; ++dx) {
          const float4 zv = *reinterpret_cast<const float4*>(Zs + (dy * ZW + px + dx) * 64 + tx * 4);
          float* a0 = acc[dy * KS + dx][0];
          float* a1 = acc[dy * KS + dx][1];
          a0[0] = fmaf(l.x, zv.x, a0[0]); a0[1] = fmaf(l.x, zv.y, a0[1]);
          a0[2] = fmaf(l.x, zv.z, a0[2]); a0[3] = fmaf(l.x, zv.w, a0[3]);
          a1[0] = fmaf(l.y, zv.x, a1[0]); a1[1] = fmaf(l.y, zv.y, a1[1]);
          a1[2] = fmaf(l.y, zv.z, a1[2]); a1[3] = fmaf(l.y, zv.w, a1[3]);
        }
    }
    __syncthreads();             // all reads of this buffer are done before the copies of the item after next land in it
    buf ^= 1;
  }
  float* out = part + (long)blockIdx.z * Cout * TALL * Cin;
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int m = m0 + ty * 2 + i;
    if (m >= Cout) continue;
#pragma unroll
    for (int t = 0; t < T; ++t)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int n = n0 + tx * 4 + k;
        if (n < Cin) out[((long)m * TALL + dy0 * KS + t) * Cin + n] = acc[t][i][k];
      }
  }
}

// ---------------------------------------------------------------------------------------------
// Direct convolution, used for Y (Algorithm 1 forward step 1; Eq. 5) and, with the weights read
// transposed and flipped, for the exact input gradient dX:
//   out[b,y,x,co] = sum_{tap,ci} w(co,ci,tap) * in[b,y+dy-p,x+dx-p,ci]
//   forward: w(co,ci,tap) = Wt[co][tap][ci]          (Wt is [Cout][T][Cin])
//   dgrad  : w(co,ci,tap) = Wt[ci][T-1-tap][co]
// A block owns 32 pixels of one image row and 64 output channels; input channels go by 16 (by 4 for
// 5 x 5 and 3 x 3 x 3 kernels, whose weight tile would not fit the static shared memory otherwise).
// Volumes: `B` counts planes (images x depth D), KD planes per kernel, offset rows rho = kz * KS + ky.
// ---------------------------------------------------------------------------------------------
template <typename T_, int KS, int KD, bool DGRAD>
__global__ void __launch_bounds__(256) conv_simt(const T_* __restrict__ in, const T_* __restrict__ Wt,
                                                 T_* __restrict__ out, int B, int D, int H, int W, int Ci, int Co,
                                                 int Cin_w, int circ) {
  constexpr int P = (KS - 1) / 2, PD = (KD - 1) / 2, XC = 32, T = KD * KS * KS, CK = T >= 25 ? 4 : 16, R = KD * KS;
  __shared__ __align__(16) float Xs[R][XC + KS - 1][CK];
  __shared__ __align__(16) float Ws[T][CK][64];
  const int tid = threadIdx.x;
  const int chunks = (W + XC - 1) / XC;
  const int xc = blockIdx.x % chunks;
  const int y = (blockIdx.x / chunks) % H;
  const int b = blockIdx.x / (chunks * H);              // plane index: image * D + z
  const int z = b % D;
  const int x0 = xc * XC, co0 = blockIdx.y * 64;
  const int cp = tid & 31, pg = tid >> 5;
  float acc[4][2];
#pragma unroll
  for (int p = 0; p < 4; ++p) acc[p][0] = acc[p][1] = 0.f;

  for (int ci0 = 0; ci0 < Ci; ci0 += CK) {
    for (int idx = tid; idx < R * (XC + KS - 1) * CK; idx += 256) {
      const int cc = idx % CK;
      const int px = (idx / CK) % (XC + KS - 1);
      const int rho = idx / (CK * (XC + KS - 1)), dz = rho / KS - PD;
      int yy = y + rho % KS - P, xx = x0 + px - P;
      if (circ) { yy = wrap_index(yy, H); xx = wrap_index(xx, W); }
      float v = 0.f;
      if (z + dz >= 0 && z + dz < D && yy >= 0 && yy < H && xx >= 0 && xx < W && ci0 + cc < Ci)
        v = to_f(in[(((long)(b + dz) * H + yy) * W + xx) * Ci + ci0 + cc]);
      Xs[rho][px][cc] = v;
    }
    for (int idx = tid; idx < T * CK * 64; idx += 256) {
      int cc, tap, co;
      if (DGRAD) { co = idx & 63; cc = (idx >> 6) % CK; tap = idx / (64 * CK); }
      else       { cc = idx % CK; tap = (idx / CK) % T; co = idx / (CK * T); }
      float v = 0.f;
      if (co0 + co < Co && ci0 + cc < Ci) {
        v = DGRAD ? to_f(Wt[((long)(ci0 + cc) * T + (T - 1 - tap)) * Cin_w + co0 + co])
                  : to_f(Wt[((long)(co0 + co) * T + tap) * Cin_w + ci0 + cc]);
      }
      // pairs of output channels are XOR-swizzled by the input channel so that both the
      // channel-fastest writes above and the pair reads below are free of bank conflicts
      Ws[tap][cc][(((co >> 1) ^ cc) << 1) | (co & 1)] = v;
    }
    __syncthreads();
#pragma unroll 4
    for (int cc = 0; cc < CK; ++cc) {
#pragma unroll
      for (int dy = 0; dy < R; ++dy) {
        float xv[4 + KS - 1];
#pragma unroll
        for (int p = 0; p < 4 + KS - 1; ++p) xv[p] = Xs[dy][pg * 4 + p][cc];
#pragma unroll
        for (int dx = 0; dx < KS; ++dx) {
          const float2 w = *reinterpret_cast<const float2*>(&Ws[dy * KS + dx][cc][(cp ^ cc) << 1]);
#pragma unroll
          for (int p = 0; p < 4; ++p) {
            acc[p][0] = fmaf(xv[p + dx], w.x, acc[p][0]);
            acc[p][1] = fmaf(xv[p + dx], w.y, acc[p][1]);
          }
        }
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    const int x = x0 + pg * 4 + p;
    if (x >= W) continue;
    T_* o = out + (((long)b * H + y) * W + x) * Co;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int co = co0 + cp * 2 + i;
      if (co < Co) o[co] = from_f<T_>(acc[p][i]);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Trace estimation per channel pair ("independent" probing, first sentence of the multi-channel case in
// Section 3): the sketch keeps the input channels apart,
//   S[j][n][b] = sum_{pixels q} Z[j,q,n] * X[b,q,n],
// and the estimate of dW[m,n,k] uses only block n of the probing vectors.  Its cheapest order of summation
// rebuilds every channel of the activation from its own sketch,
//   Xr[b,q,n] = sum_j S[j][n][b] * Z[j,q,n],
// and then runs the offset contraction over the batch (dY in the place of L, Xr in the place of Z).
// Both kernels below put 32 consecutive channels on the lanes of a warp, so every load is one row of
// channels-last memory.
// ---------------------------------------------------------------------------------------------
constexpr int IS_JT = 4, IS_BT = 8;      // probes x samples per thread in the sketch
template <typename T>
__global__ void __launch_bounds__(256) sketch_indep_simt(const T* __restrict__ X, const T* __restrict__ Z,
                                                         float* __restrict__ S, int r, int B, long N, int Cin) {
  __shared__ float red[8][IS_JT * IS_BT][33];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n = blockIdx.y * 32 + lane, b0 = blockIdx.x * IS_BT, j0 = blockIdx.z * IS_JT;
  const bool live = n < Cin;
  float acc[IS_JT][IS_BT];
#pragma unroll
  for (int j = 0; j < IS_JT; ++j)
#pragma unroll
    for (int b = 0; b < IS_BT; ++b) acc[j][b] = 0.f;
  // the eight warps take the pixels in turn; their sums are added below in warp order
  for (long q = warp; q < N; q += 8) {
    float z[IS_JT], x[IS_BT];
#pragma unroll
    for (int j = 0; j < IS_JT; ++j) z[j] = (live && j0 + j < r) ? to_f(Z[((long)(j0 + j) * N + q) * Cin + n]) : 0.f;
#pragma unroll
    for (int b = 0; b < IS_BT; ++b) x[b] = (live && b0 + b < B) ? to_f(X[((long)(b0 + b) * N + q) * Cin + n]) : 0.f;
#pragma unroll
    for (int j = 0; j < IS_JT; ++j)
#pragma unroll
      for (int b = 0; b < IS_BT; ++b) acc[j][b] = fmaf(z[j], x[b], acc[j][b]);
  }
#pragma unroll
  for (int j = 0; j < IS_JT; ++j)
#pragma unroll
    for (int b = 0; b < IS_BT; ++b) red[warp][j * IS_BT + b][lane] = acc[j][b];
  __syncthreads();
  // thread t sums output (t / 32, lane) ... over the eight warps, in order
  for (int o = warp; o < IS_JT * IS_BT; o += 8) {
    float t = red[0][o][lane];
#pragma unroll
    for (int w = 1; w < 8; ++w) t += red[w][o][lane];
    const int j = j0 + o / IS_BT, b = b0 + o % IS_BT;
    if (live && j < r && b < B) S[((long)j * Cin + n) * B + b] = t;
  }
}

// Xr[b,q,n] = sum_j S[j][n][b] Z[j,q,n], written in the storage type.  A block owns 32 channels x 8 pixels
// x 8 samples; the sketch entries of 16 probes at a time are staged in shared memory.
constexpr int IR_BT = 8, IR_JC = 16;
template <typename T>
__global__ void __launch_bounds__(256) rebuild_indep_simt(const float* __restrict__ S, const T* __restrict__ Z,
                                                          T* __restrict__ Xr, int r, int B, long N, int Cin) {
  __shared__ float Ss[IR_JC][32][IR_BT + 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n0 = blockIdx.y * 32, n = n0 + lane, b0 = blockIdx.z * IR_BT;
  const long q = (long)blockIdx.x * 8 + warp;
  const bool live = n < Cin && q < N;
  float acc[IR_BT];
#pragma unroll
  for (int b = 0; b < IR_BT; ++b) acc[b] = 0.f;
  for (int jc = 0; jc < r; jc += IR_JC) {
    for (int idx = threadIdx.x; idx < IR_JC * 32 * IR_BT; idx += 256) {
      const int bb = idx % IR_BT, nn = (idx / IR_BT) % 32, jj = idx / (IR_BT * 32);
      Ss[jj][nn][bb] = (jc + jj < r && n0 + nn < Cin && b0 + bb < B) ? S[((long)(jc + jj) * Cin + n0 + nn) * B + b0 + bb] : 0.f;
    }
    __syncthreads();
    if (live) {
      const int nj = min(IR_JC, r - jc);
      for (int jj = 0; jj < nj; ++jj) {
        const float z = to_f(Z[((long)(jc + jj) * N + q) * Cin + n]);
#pragma unroll
        for (int b = 0; b < IR_BT; ++b) acc[b] = fmaf(Ss[jj][lane][b], z, acc[b]);
      }
    }
    __syncthreads();
  }
  if (live) {
#pragma unroll
    for (int b = 0; b < IR_BT; ++b)
      if (b0 + b < B) Xr[((long)(b0 + b) * N + q) * Cin + n] = from_f<T>(acc[b]);
  }
}

// out[b][j] = in[j][b] for a small [rows][cols] float matrix (the sketch, transposed).
static __global__ void transpose_f32(const float* __restrict__ in, float* __restrict__ out, int rows, int cols) {
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long)rows * cols) return;
  const int j = (int)(i / cols), b = (int)(i % cols);
  out[(long)b * rows + j] = in[i];
}

// float -> 16-bit storage type copy (the sketch as tensor-core operand).
template <typename T>
static __global__ void cast_f32_to_16(const float* __restrict__ in, T* __restrict__ out, long n) {
  pdl_trigger();
  pdl_wait();
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = from_f<T>(in[i]);
}

}  // namespace xconv
