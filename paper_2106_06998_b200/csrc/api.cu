// libxconv C ABI: argument checks, workspace planning and kernel dispatch.
#include <cmath>
#include "../../include/xconv.h"

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstring>

#include "common.cuh"
#include "simt_kernels.cuh"
#include "tc_api.h"
#include <type_traits>

namespace xconv {

thread_local int g_last_cuda_error = 0;
thread_local int g_launches = 0;

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline long cdiv(long a, long b) { return (a + b - 1) / b; }
static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static xconv_status check_launch() {
  ++g_launches;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; return XCONV_ERR_CUDA; }
  return XCONV_OK;
}

// A fresh non-zero tag per API call (see the workspace header in common.cuh).
static std::atomic<unsigned int> g_call_tag{0x51u};
thread_local unsigned int g_tag = 1u;
static void new_call() {
  g_launches = 0;
  g_tag = g_call_tag.fetch_add(2u) | 1u;
}
unsigned int call_tag() { return g_tag; }

// Depth of the volume and of the kernel (0 and 1 both mean a planar layer).
static inline int depth(const xconv_desc* d) { return d->D > 1 ? d->D : 1; }
static inline int kdepth(const xconv_desc* d) { return d->KD > 1 ? d->KD : 1; }

static xconv_status validate(const xconv_desc* d) {
  if (!d) return XCONV_ERR_INVALID_ARG;
  if (d->B <= 0 || d->Cin <= 0 || d->Cout <= 0 || d->H <= 0 || d->W <= 0 || d->r <= 0 || d->KH <= 0 || d->KW <= 0)
    return XCONV_ERR_INVALID_ARG;
  if (d->dtype != XCONV_F32 && d->dtype != XCONV_BF16 && d->dtype != XCONV_F16) return XCONV_ERR_INVALID_ARG;
  if (d->pad_h < 0 || d->pad_w < 0 || d->D < 0 || d->KD < 0 || d->pad_d < 0) return XCONV_ERR_INVALID_ARG;
  if (d->circular != 0 && d->circular != 1) return XCONV_ERR_INVALID_ARG;
  if (d->KH != d->KW || (d->KH != 1 && d->KH != 3 && d->KH != 5)) return XCONV_ERR_UNSUPPORTED;
  if (2 * d->pad_h != d->KH - 1 || 2 * d->pad_w != d->KW - 1) return XCONV_ERR_UNSUPPORTED;
  // kernels over volumes: 3 x 3 x 3, or planar kernels (1 x K x K) applied to every plane
  if (kdepth(d) != 1 && !(kdepth(d) == 3 && d->KH == 3)) return XCONV_ERR_UNSUPPORTED;
  if (2 * d->pad_d != kdepth(d) - 1) return XCONV_ERR_UNSUPPORTED;
  // circular shifts (the operator T_k of the paper's Section 3) are served for planar layers only
  if (d->circular && (depth(d) > 1 || kdepth(d) > 1)) return XCONV_ERR_UNSUPPORTED;
  // 32-bit grid and index limits of the kernels.  r, B and the channel counts land on the y axis of a
  // grid (at most 65535 blocks of 16 or more) in the FP32-FMA kernels, and r and B trade places when
  // xconv_wgrad sums over the probes first.
  const long px = (long)depth(d) * d->H * d->W;
  const long Kdim = px * d->Cin, Q = px * d->Cout;
  if (Kdim > (1L << 40) || Q > (1L << 40) || (long)d->B * depth(d) * d->H * cdiv(d->W, 32) > 2000000000L ||
      (long)depth(d) * d->H > 2000000000L)
    return XCONV_ERR_UNSUPPORTED;
  const long axis_limit = 65535L * 16;
  if (d->r > axis_limit || d->B > axis_limit || d->Cin > axis_limit || d->Cout > axis_limit ||
      (long)d->r * d->B > (1L << 40) || (long)d->r * depth(d) > 2000000000L || (long)d->B * depth(d) > 2000000000L)
    return XCONV_ERR_UNSUPPORTED;
  return XCONV_OK;
}

// The sketch, the back-probe and the per-channel kernels see the pixels of a sample as one flat axis: for
// them a volume is an image with D*H rows.
static xconv_desc flat(const xconv_desc* d) {
  xconv_desc f = *d;
  f.H = d->H * depth(d);
  f.D = 1; f.KD = 1; f.pad_d = 0;
  f.zero_blocks = nullptr;
  return f;
}
// The tensor-core contraction and convolution work plane by plane: D times the probes for the contraction,
// D times the batch for the convolutions.  A planar kernel on a volume treats every plane as an image of its
// own (D = 1 from there on); a 3 x 3 x 3 kernel keeps D, so that the kernels know where a volume ends.
static xconv_desc planes_ct(const xconv_desc* d) {
  xconv_desc f = *d;
  f.r = d->r * depth(d);
  if (kdepth(d) == 1) {
    f.D = 1; f.KD = 1; f.pad_d = 0;
    if (depth(d) > 1) f.zero_blocks = nullptr;      // the mask is per probe, and r now counts planes
  }
  return f;
}
static xconv_desc planes_cv(const xconv_desc* d) {
  xconv_desc f = *d;
  f.B = d->B * depth(d);
  if (kdepth(d) == 1) { f.D = 1; f.KD = 1; f.pad_d = 0; }
  return f;
}
static inline bool volumetric(const xconv_desc* d) { return kdepth(d) == 3; }

// ----------------------------------------------------------------------------------- plans
// A plan fixes every launch shape and workspace offset from the descriptor alone, so that
// xconv_workspace_bytes and the entry points always agree.

static const size_t WS_HEADER = 256;   // word 0: status left by pipelined kernels

struct SketchPlan {
  bool tc;
  int splits; long k_per_split;        // simt
  TcSketchPlan t;                      // tcgen05
  size_t part_off, bytes;
};

static SketchPlan plan_sketch(const xconv_desc* d_, bool seeded = false) {
  const xconv_desc fl = flat(d_);
  const xconv_desc* d = &fl;
  SketchPlan p{};
  const long K = (long)d->H * d->W * d->Cin;
  p.part_off = WS_HEADER;
  p.tc = tc_plan_sketch(d, &p.t, seeded && tc_sketch_can_redraw(d));
  if (p.tc) {
    p.bytes = p.part_off + align_up(p.t.part_bytes, 256);
    return p;
  }
  const long tiles = cdiv(d->r, 64) * cdiv(d->B, 64);
  // short chains: a block walks its k-range step by step with one step of loads in flight, so the time of a
  // sketch is (steps per block) x (load latency) unless the range is dealt to many blocks
  // one full wave of the grid: four blocks of the transposing kernel fit an SM, three of the cp.async kernel that
  // serves float rows on 16-byte boundaries (80 registers, 54 KB)
  const long per_sm = (d->dtype == XCONV_F32 && K % 4 == 0) ? 3 : 4;
  long splits = std::max(1L, std::min(cdiv(per_sm * 148, tiles), cdiv(K, 128)));
  splits = std::min(splits, 2048L);
  p.k_per_split = align_up((size_t)cdiv(K, splits), 32);
  p.splits = (int)cdiv(K, p.k_per_split);
  p.bytes = p.part_off + align_up((size_t)p.splits * d->r * d->B * sizeof(float), 256);
  return p;
}

struct WgradPlan {
  bool tc_bp, tc_ct;
  int splits; long items_per_split;    // simt contraction
  TcWgradPlan t;                       // tcgen05: contraction fields (planned on the per-plane layer)
  TcWgradPlan tb;                      // tcgen05: back-probe fields (planned on the flattened layer)
  size_t l_off, sb_off, part_off, bytes;
};

static WgradPlan plan_wgrad_core(const xconv_desc* d) {
  WgradPlan p{};
  const long Q = (long)depth(d) * d->H * d->W * d->Cout;
  const int T = kdepth(d) * d->KH * d->KW;
  const size_t lsz = d->dtype == XCONV_F32 ? 4 : 2;
  p.l_off = WS_HEADER;
  p.sb_off = p.l_off + align_up((size_t)d->r * Q * lsz, 256);
  p.part_off = p.sb_off + align_up((size_t)d->r * d->B * 2, 256);
  const xconv_desc f = flat(d);
  p.tc_bp = (tc_plan_wgrad(&f, &p.tb) & 1) != 0;
  const xconv_desc c = planes_ct(d);    // the tensor-core contraction works plane by plane
  p.tc_ct = (tc_plan_wgrad(&c, &p.t) & 2) != 0;
  if (p.tc_ct) {
    p.bytes = p.part_off + align_up(p.t.part_bytes, 256);
    return p;
  }
  const long items = (long)d->r * depth(d) * d->H * cdiv(d->W, 32);
  // blocks per split: 5 x 5 kernels take one offset row per block, 3 x 3 x 3 kernels three
  const long tiles = cdiv(d->Cin, 64) * cdiv(d->Cout, 32) * (d->KH == 5 ? 5 : volumetric(d) ? 3 : 1);
  // one wave of the grid: two blocks of this kernel fit an SM (its 72 accumulators per thread)
  long splits = std::max(1L, std::min(std::max(1L, 2L * 148 / tiles), cdiv(items, 2)));
  splits = std::min(splits, 4096L);
  p.items_per_split = cdiv(items, splits);
  p.splits = (int)cdiv(items, p.items_per_split);
  p.bytes = p.part_off + align_up((size_t)p.splits * d->Cout * T * d->Cin * sizeof(float), 256);
  return p;
}

// Re-association for r > B.  The estimate is one bilinear form,
//   dW[m,n,k] = scale_n * sum_{j,b,q} S[j,b] dY[b,m,q] Z[j,n,q+k],
// and Algorithm 1 sums over b first (L = S dY^T, cost r*Cout*N*(B + 9*Cin)).  Summing over j first
// gives Xr[b,n,p] = sum_j S[j,b] Z[j,n,p] -- the activation rebuilt from its sketch -- followed by the
// same offset contraction over the batch, dW = scale * sum_{b,q} dY[b,m,q] Xr[b,n,q+k]
// (cost B*Cin*N*(r + 9*Cout)): cheaper exactly when r > B.  Both steps are the kernels of the other
// order with the roles of the tensors swapped, so xconv_wgrad picks the cheaper order; the explicit
// halves xconv_backprobe / xconv_contract always follow the paper's order.
struct SwappedWgrad {
  bool on;
  xconv_desc d1, d2;       // d1: "back-probe" producing Xr; d2: contraction over the batch
  WgradPlan p1, p2;
  size_t x_off, st_off, sb_off, part_off, bytes;
};

static SwappedWgrad plan_wgrad_swapped(const xconv_desc* d) {
  SwappedWgrad w{};
  w.on = d->r > d->B;
  if (!w.on) return w;
  w.d1 = *d; w.d1.B = d->r; w.d1.r = d->B; w.d1.Cout = d->Cin; w.d1.chan_scale = nullptr;
  w.d2 = *d; w.d2.r = d->B;
  w.d1.zero_blocks = w.d2.zero_blocks = nullptr;      // neither step sums over the probes block by block
  w.p1 = plan_wgrad_core(&w.d1);
  w.p2 = plan_wgrad_core(&w.d2);
  const size_t es = d->dtype == XCONV_F32 ? 4 : 2;
  const int T = kdepth(d) * d->KH * d->KW;
  w.x_off = WS_HEADER;
  w.st_off = w.x_off + align_up((size_t)d->B * depth(d) * d->H * d->W * d->Cin * es, 256);
  w.sb_off = w.st_off + align_up((size_t)d->r * d->B * 4, 256);
  w.part_off = w.sb_off + align_up((size_t)d->r * d->B * 2, 256);
  const size_t part = w.p2.tc_ct ? w.p2.t.part_bytes : (size_t)w.p2.splits * d->Cout * T * d->Cin * sizeof(float);
  w.bytes = w.part_off + align_up(part, 256);
  return w;
}

static WgradPlan plan_wgrad(const xconv_desc* d) {
  WgradPlan p = plan_wgrad_core(d);
  const SwappedWgrad w = plan_wgrad_swapped(d);
  if (w.on) p.bytes = std::max(p.bytes, w.bytes);
  return p;
}

// ----------------------------------------------------------------------------------- probes from a seed

// Z redrawn from a seed: entry e (in memory order) is +1 if bit (e mod 128) of Philox block (e div 128) is 0,
// -1 if it is 1; bit b is bit (b mod 32) of output word (b div 32).  One thread writes eight entries.
template <typename T>
__global__ void __launch_bounds__(256) probes_from_seed_kernel(T* __restrict__ Z, long total, uint32_t k0, uint32_t k1) {
  pdl_trigger();
  pdl_wait();
  const long e0 = ((long)blockIdx.x * blockDim.x + threadIdx.x) * 8;
  if (e0 >= total) return;
  const unsigned long long blk = (unsigned long long)e0 >> 7;
  const uint4 w = philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), k0, k1);
  const int word = (int)((e0 & 127) >> 5);
  const uint32_t wv = word == 0 ? w.x : word == 1 ? w.y : word == 2 ? w.z : w.w;
  const uint32_t bits = (wv >> (e0 & 31)) & 0xFFu;
  if (e0 + 8 <= total) {                     // Z is 16-byte aligned and e0 a multiple of 8: vector stores
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = ((bits >> i) & 1u) ? -1.0f : 1.0f;
    st4(Z + e0, make_float4(v[0], v[1], v[2], v[3]));
    st4(Z + e0 + 4, make_float4(v[4], v[5], v[6], v[7]));
    return;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (e0 + i < total) Z[e0 + i] = from_f<T>(((bits >> i) & 1u) ? -1.0f : 1.0f);
}

static xconv_status run_probes_from_seed(const xconv_desc* d, unsigned long long seed, void* Z, cudaStream_t st) {
  const long total = (long)d->r * depth(d) * d->H * d->W * d->Cin;
  const unsigned grid = (unsigned)cdiv(cdiv(total, 8), 256);
  const uint32_t k0 = (uint32_t)(seed & 0xFFFFFFFFull), k1 = (uint32_t)(seed >> 32);
  cudaError_t e = d->dtype == XCONV_F32
      ? launch_pdl(probes_from_seed_kernel<float>, dim3(grid), dim3(256), 0, st, static_cast<float*>(Z), total, k0, k1)
      : d->dtype == XCONV_F16
      ? launch_pdl(probes_from_seed_kernel<f16>, dim3(grid), dim3(256), 0, st, static_cast<f16*>(Z), total, k0, k1)
      : launch_pdl(probes_from_seed_kernel<bf16>, dim3(grid), dim3(256), 0, st, static_cast<bf16*>(Z), total, k0, k1);
  ++g_launches;
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; return XCONV_ERR_CUDA; }
  return XCONV_OK;
}

// Z with standard normal entries from a seed: Philox block b (counter word 2 = 1, which keeps the stream apart from
// the Rademacher one) gives entries 4b .. 4b+3, two Box-Muller pairs.  One thread per block.
template <typename T>
__global__ void __launch_bounds__(256) gaussian_probes_kernel(T* __restrict__ Z, long total, uint32_t k0, uint32_t k1) {
  pdl_trigger();
  pdl_wait();
  const long b = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const long e0 = b * 4;
  if (e0 >= total) return;
  const uint4 w = philox4x32_10((uint32_t)b, (uint32_t)((unsigned long long)b >> 32), k0, k1, 1u);
  const float2 p0 = box_muller_u24(w.x, w.y), p1 = box_muller_u24(w.z, w.w);
  if (e0 + 4 <= total) { st4(Z + e0, make_float4(p0.x, p0.y, p1.x, p1.y)); return; }
  const float v[4] = {p0.x, p0.y, p1.x, p1.y};
#pragma unroll
  for (int i = 0; i < 4; ++i)
    if (e0 + i < total) Z[e0 + i] = from_f<T>(v[i]);
}

static xconv_status run_gaussian_probes(const xconv_desc* d, unsigned long long seed, void* Z, cudaStream_t st) {
  const long total = (long)d->r * depth(d) * d->H * d->W * d->Cin;
  const unsigned grid = (unsigned)cdiv(cdiv(total, 4), 256);
  const uint32_t k0 = (uint32_t)(seed & 0xFFFFFFFFull), k1 = (uint32_t)(seed >> 32);
  cudaError_t e = d->dtype == XCONV_F32
      ? launch_pdl(gaussian_probes_kernel<float>, dim3(grid), dim3(256), 0, st, static_cast<float*>(Z), total, k0, k1)
      : d->dtype == XCONV_F16
      ? launch_pdl(gaussian_probes_kernel<f16>, dim3(grid), dim3(256), 0, st, static_cast<f16*>(Z), total, k0, k1)
      : launch_pdl(gaussian_probes_kernel<bf16>, dim3(grid), dim3(256), 0, st, static_cast<bf16*>(Z), total, k0, k1);
  ++g_launches;
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; return XCONV_ERR_CUDA; }
  return XCONV_OK;
}

// Block-sparse probing vectors (Eq. 7) from a seed.  keep[g], g = j * Cin + n: block n of probing vector j is non-zero
// iff word (g mod 4) of Philox block (g div 4) -- counter word 2 = 2, apart from the two value streams -- is below the
// threshold floor(p * 2^32).
__global__ void __launch_bounds__(256) block_keep_kernel(unsigned char* __restrict__ keep, long total, uint32_t k0,
                                                         uint32_t k1, unsigned long long threshold) {
  const long b = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (b * 4 >= total) return;
  const uint4 w = philox4x32_10((uint32_t)b, (uint32_t)((unsigned long long)b >> 32), k0, k1, 2u);
  const uint32_t v[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i)
    if (b * 4 + i < total) keep[b * 4 + i] = (unsigned long long)v[i] < threshold ? 1 : 0;
}
// scale[n] = 1 / nnz(Z_n), the number of probing vectors whose block n is kept (Eq. 8); 0 for a channel no vector probes.
__global__ void __launch_bounds__(256) keep_scale_kernel(const unsigned char* __restrict__ keep, int r, int Cin,
                                                         float* __restrict__ scale) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= Cin) return;
  int nnz = 0;
  for (int j = 0; j < r; ++j) nnz += keep[(long)j * Cin + n];
  scale[n] = nnz > 0 ? __fdiv_rn(1.0f, (float)nnz) : 0.0f;
}
// The dropped blocks of a dense Z set to +0.  Entry e belongs to probe e / per_probe and channel e % Cin.
template <typename T>
__global__ void __launch_bounds__(256) drop_blocks_kernel(T* __restrict__ Z, const unsigned char* __restrict__ keep,
                                                          long total, long per_probe, int Cin) {
  const long e0 = ((long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long e = e0 + i;
    if (e < total && !keep[(e / per_probe) * Cin + e % Cin]) Z[e] = from_f<T>(0.0f);
  }
}

static size_t probes_bytes(const xconv_desc* d) {
  return align_up((size_t)d->r * depth(d) * d->H * d->W * d->Cin * (d->dtype == XCONV_F32 ? 4 : 2), 256);
}

// ----------------------------------------------------------------------------------- launchers

template <typename T>
static xconv_status run_sketch_simt(const xconv_desc* d, const SketchPlan& p, const void* X, const void* Z,
                                    float* S, char* ws, cudaStream_t st) {
  const long K = (long)d->H * d->W * d->Cin;
  float* part = reinterpret_cast<float*>(ws + p.part_off);
  dim3 grid((unsigned)cdiv(d->B, 64), (unsigned)cdiv(d->r, 64), (unsigned)p.splits);
  if (std::is_same<T, float>::value && K % 4 == 0 && p.k_per_split % GT_KS == 0) {
    const size_t smem = (size_t)GT_STAGES * 128 * GT_LD * sizeof(float);
    cudaError_t ea = cudaFuncSetAttribute(gemm_tn_simt_async, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (ea != cudaSuccess) { g_last_cuda_error = (int)ea; return XCONV_ERR_CUDA; }
    gemm_tn_simt_async<<<grid, 256, smem, st>>>(reinterpret_cast<const float*>(Z), reinterpret_cast<const float*>(X), part,
                                                d->r, d->B, K, p.k_per_split);
  } else {
    gemm_tn_simt<T><<<grid, 256, 0, st>>>(static_cast<const T*>(Z), static_cast<const T*>(X), part, d->r, d->B, K,
                                          p.k_per_split, (K % 4 == 0) ? 1 : 0);
  }
  xconv_status s = check_launch();
  if (s != XCONV_OK) return s;
  const long count = (long)d->r * d->B;
  reduce_partials<<<(unsigned)cdiv(count, RP_OUT), RP_OUT * RP_LANES, 0, st>>>(part, S, count, p.splits, 1.0f, nullptr, 1);
  return check_launch();
}

// Whether the sketch kernel of this layer redraws Z itself; otherwise the seeded call first writes Z
// into the workspace (behind the regular scratch) and runs the regular kernels on it.
static bool sketch_redraws(const xconv_desc* d, const SketchPlan& p) {
  const xconv_desc fl = flat(d);
  return p.tc && tc_sketch_can_redraw(&fl);
}

static xconv_status run_sketch(const xconv_desc* d_, const void* X, const void* Z, float* S, void* ws,
                               size_t ws_bytes, cudaStream_t st, const unsigned long long* seed = nullptr) {
  const xconv_desc fl = flat(d_);
  const xconv_desc* d = &fl;
  const SketchPlan p = plan_sketch(d, seed != nullptr);
  const bool redraw = seed && sketch_redraws(d, p);
  const size_t need = p.bytes + (seed && !redraw ? probes_bytes(d) : 0);
  if (!ws || ws_bytes < need) return XCONV_ERR_WORKSPACE;
  if (!aligned16(ws)) return XCONV_ERR_ALIGNMENT;
  char* w = static_cast<char*>(ws);
  if (seed && !redraw) {
    xconv_status s = run_probes_from_seed(d, *seed, w + p.bytes, st);
    if (s != XCONV_OK) return s;
    Z = w + p.bytes;
  }
  if (p.tc) return tc_run_sketch(d, p.t, X, Z, S, w, w + p.part_off, st, redraw ? seed : nullptr);
  return d->dtype == XCONV_F32 ? run_sketch_simt<float>(d, p, X, Z, S, w, st)
         : d->dtype == XCONV_F16 ? run_sketch_simt<f16>(d, p, X, Z, S, w, st)
                                 : run_sketch_simt<bf16>(d, p, X, Z, S, w, st);
}

template <typename T, typename TL>
static xconv_status run_backprobe_simt(const xconv_desc* d, const float* S, const void* dY, void* Lv,
                                       cudaStream_t st) {
  const long Q = (long)depth(d) * d->H * d->W * d->Cout;
  // Block size: the kernel holds about 126 registers per thread, so an SM runs floor(65536 / (126 t)) blocks of t
  // threads; the time goes with (waves of the grid) x (threads an SM runs at once).  256 threads leave the last
  // wave of a small layer part empty (256 blocks for 296 places on the 64-channel 32 x 32 layer; 224 threads fill it).
  int threads = 256;
  long best = -1;
  for (int t = 256; t >= 128; t -= 32) {
    const long per_sm = std::min<long>(65536 / (126L * t), 2048 / t);
    const long blocks = cdiv(cdiv(Q, 4), t) * cdiv(d->r, 16);
    const long cost = cdiv(blocks, 148 * per_sm) * per_sm * t;
    if (best < 0 || cost < best) { best = cost; threads = t; }
  }
  dim3 g1((unsigned)cdiv(cdiv(Q, 4), threads), (unsigned)cdiv(d->r, 16));
  backprobe_simt<T, TL><<<g1, threads, 0, st>>>(S, static_cast<const T*>(dY), static_cast<TL*>(Lv), d->r, d->B, Q,
                                                (Q % 4 == 0) ? 1 : 0);
  return check_launch();
}

template <typename T, typename TL>
static xconv_status run_contract_simt(const xconv_desc* d, const WgradPlan& p, const void* Lv, const void* Z,
                                      float* dW, float alpha, float* part, cudaStream_t st) {
  const int T9 = kdepth(d) * d->KH * d->KW;
  const TL* L = static_cast<const TL*>(Lv);
  const T* Zt = static_cast<const T*>(Z);
  const bool vec = d->Cin % 4 == 0 && d->Cout % 4 == 0;      // rows of L and Z then start on 4-element boundaries
  const unsigned gx = (unsigned)cdiv(d->Cin, 64), gy = (unsigned)cdiv(d->Cout, 32), gz = (unsigned)p.splits;
#define XC_CONTRACT(KS, KD, DYS) do { \
    dim3 g2(gx * (KD * KS / DYS), gy, gz); \
    if (vec && std::is_same<TL, float>::value && std::is_same<T, float>::value) { \
      const size_t smem = 2 * contract_async_tile_floats<KS, DYS>() * sizeof(float); \
      auto kern = contract_simt_async<KS, KD, DYS>; \
      cudaError_t ea = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
      if (ea != cudaSuccess) { g_last_cuda_error = (int)ea; return XCONV_ERR_CUDA; } \
      kern<<<g2, 256, smem, st>>>(reinterpret_cast<const float*>(L), reinterpret_cast<const float*>(Zt), part, d->r, depth(d), d->H, d->W, d->Cin, d->Cout, p.items_per_split, d->circular); \
    } else if (vec) contract_simt<TL, T, KS, KD, DYS, true><<<g2, 256, 0, st>>>(L, Zt, part, d->r, depth(d), d->H, d->W, d->Cin, d->Cout, p.items_per_split, d->circular); \
    else contract_simt<TL, T, KS, KD, DYS, false><<<g2, 256, 0, st>>>(L, Zt, part, d->r, depth(d), d->H, d->W, d->Cin, d->Cout, p.items_per_split, d->circular); \
  } while (0)
  if (volumetric(d)) XC_CONTRACT(3, 3, 3);
  else if (d->KH == 3) XC_CONTRACT(3, 1, 3);
  else if (d->KH == 5) XC_CONTRACT(5, 1, 1);
  else XC_CONTRACT(1, 1, 1);
#undef XC_CONTRACT
  xconv_status s = check_launch();
  if (s != XCONV_OK) return s;
  const long count = (long)d->Cout * T9 * d->Cin;
  reduce_partials<<<(unsigned)cdiv(count, RP_OUT), RP_OUT * RP_LANES, 0, st>>>(part, dW, count, p.splits, alpha, d->chan_scale, d->Cin);
  return check_launch();
}

template <typename T>
static xconv_status run_conv_simt(const xconv_desc* d, bool dgrad, const void* in, const void* Wt, void* out,
                                  cudaStream_t st) {
  const int Ci = dgrad ? d->Cout : d->Cin, Co = dgrad ? d->Cin : d->Cout;
  const int D = depth(d), planes = d->B * D;
  dim3 grid((unsigned)((long)planes * d->H * cdiv(d->W, 32)), (unsigned)cdiv(Co, 64));
  const T* i_ = static_cast<const T*>(in);
  const T* w_ = static_cast<const T*>(Wt);
  T* o_ = static_cast<T*>(out);
#define XC_CONV(KS, KD) do { \
    if (dgrad) conv_simt<T, KS, KD, true><<<grid, 256, 0, st>>>(i_, w_, o_, planes, D, d->H, d->W, Ci, Co, d->Cin, d->circular); \
    else       conv_simt<T, KS, KD, false><<<grid, 256, 0, st>>>(i_, w_, o_, planes, D, d->H, d->W, Ci, Co, d->Cin, d->circular); \
  } while (0)
  if (volumetric(d)) XC_CONV(3, 3);
  else if (d->KH == 3) XC_CONV(3, 1);
  else if (d->KH == 5) XC_CONV(5, 1);
  else XC_CONV(1, 1);
#undef XC_CONV
  return check_launch();
}

// Scratch of the convolution calls: the header, and for the tensor-core dgrad the transposed weights.
static size_t conv_ws_bytes(const xconv_desc* d, bool dgrad) {
  TcConvPlan t;
  const xconv_desc c = planes_cv(d);
  if (tc_plan_conv(&c, dgrad, &t)) return WS_HEADER + align_up(t.wt_bytes, 256);
  return WS_HEADER;
}

static xconv_status run_conv(const xconv_desc* d, bool dgrad, const void* in, const void* Wt, void* out,
                             char* ws, cudaStream_t st) {
  TcConvPlan t;
  const xconv_desc c = planes_cv(d);
  if (tc_plan_conv(&c, dgrad, &t)) return tc_run_conv(&c, t, dgrad, in, Wt, out, ws, ws + WS_HEADER, st);
  return d->dtype == XCONV_F32 ? run_conv_simt<float>(d, dgrad, in, Wt, out, st)
         : d->dtype == XCONV_F16 ? run_conv_simt<f16>(d, dgrad, in, Wt, out, st)
                                 : run_conv_simt<bf16>(d, dgrad, in, Wt, out, st);
}

// L = S dY^T into `L`; `Sb` receives the bfloat16 copy of S that the tensor-core kernel reads.
static xconv_status run_backprobe(const xconv_desc* d, const WgradPlan& p, const float* S, const void* dY,
                                  void* L, void* Sb_, char* w, cudaStream_t st, const unsigned long long* seed = nullptr) {
  if (p.tc_bp) {
    const long n = (long)d->r * d->B;
    cudaError_t e = d->dtype == XCONV_F16
        ? launch_pdl(cast_f32_to_16<f16>, dim3((unsigned)cdiv(n, 256)), dim3(256), 0, st, S, static_cast<f16*>(Sb_), n)
        : launch_pdl(cast_f32_to_16<bf16>, dim3((unsigned)cdiv(n, 256)), dim3(256), 0, st, S, static_cast<bf16*>(Sb_), n);
    ++g_launches;
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; return XCONV_ERR_CUDA; }
    const xconv_desc f = flat(d);
    return tc_run_backprobe(&f, p.tb, Sb_, dY, L, w, st, seed);
  }
  return d->dtype == XCONV_F32 ? run_backprobe_simt<float, float>(d, S, dY, L, st)
         : d->dtype == XCONV_F16 ? run_backprobe_simt<f16, f16>(d, S, dY, L, st)
                                 : run_backprobe_simt<bf16, bf16>(d, S, dY, L, st);
}

static xconv_status run_contract(const xconv_desc* d, const WgradPlan& p, const void* L, const void* Z,
                                 float* dW, float alpha, char* part, char* w, cudaStream_t st) {
  if (p.tc_ct) {
    const xconv_desc c = planes_ct(d);
    return tc_run_contract(&c, p.t, L, Z, dW, alpha, w, part, st);
  }
  return d->dtype == XCONV_F32
             ? run_contract_simt<float, float>(d, p, L, Z, dW, alpha, reinterpret_cast<float*>(part), st)
         : d->dtype == XCONV_F16
             ? run_contract_simt<f16, f16>(d, p, L, Z, dW, alpha, reinterpret_cast<float*>(part), st)
             : run_contract_simt<bf16, bf16>(d, p, L, Z, dW, alpha, reinterpret_cast<float*>(part), st);
}

static xconv_status check_ws(void* ws, size_t ws_bytes, size_t need) {
  if (!ws || ws_bytes < need) return XCONV_ERR_WORKSPACE;
  if (!aligned16(ws)) return XCONV_ERR_ALIGNMENT;
  return XCONV_OK;
}

// Whether xconv_wgrad_seeded redraws the probing vectors inside its first kernel (the estimator summed over the
// probes first, r > B, with that step on the tensor cores) instead of writing them to the workspace first.
static bool wgrad_redraws(const xconv_desc* d) {
  const SwappedWgrad sw = plan_wgrad_swapped(d);
  return sw.on && sw.p1.tc_bp;
}

// `seed` != nullptr (only where wgrad_redraws holds): Z is not read.
static xconv_status run_wgrad(const xconv_desc* d, const float* S, const void* dY, const void* Z, float* dW,
                              void* ws, size_t ws_bytes, cudaStream_t st, const unsigned long long* seed = nullptr) {
  const WgradPlan p = plan_wgrad(d);
  xconv_status s = check_ws(ws, ws_bytes, p.bytes);
  if (s != XCONV_OK) return s;
  char* w = static_cast<char*>(ws);
  const float alpha = 1.0f / (float)d->r;
  const SwappedWgrad sw = plan_wgrad_swapped(d);
  if (sw.on) {
    // Xr = S^T Z, then the offset contraction over the batch (see plan_wgrad_swapped)
    if ((s = validate(&sw.d1)) != XCONV_OK || (s = validate(&sw.d2)) != XCONV_OK) return s;
    float* St = reinterpret_cast<float*>(w + sw.st_off);
    const long n = (long)d->r * d->B;
    transpose_f32<<<(unsigned)cdiv(n, 256), 256, 0, st>>>(S, St, d->r, d->B);
    s = check_launch();
    if (s != XCONV_OK) return s;
    s = run_backprobe(&sw.d1, sw.p1, St, Z, w + sw.x_off, w + sw.sb_off, w, st, seed);
    if (s != XCONV_OK) return s;
    return run_contract(&sw.d2, sw.p2, dY, w + sw.x_off, dW, alpha, w + sw.part_off, w, st);
  }
  s = run_backprobe(d, p, S, dY, w + p.l_off, w + p.sb_off, w, st);
  if (s != XCONV_OK) return s;
  return run_contract(d, p, w + p.l_off, Z, dW, alpha, w + p.part_off, w, st);
}

// One block per (probe, 64-channel group): do the H*W (volumes: D*H*W) rows of 64 channels hold anything but +-0?
template <typename T>
__global__ void __launch_bounds__(256) zero_blocks_kernel(const T* __restrict__ Z, unsigned char* __restrict__ mask,
                                                           long pixels, int Cin) {
  constexpr int PER_ROW = 64 * (int)sizeof(T) / 16;          // 16-byte pieces of one row of the block
  constexpr uint32_t ABS = sizeof(T) == 4 ? 0x7FFFFFFFu : 0x7FFF7FFFu;      // a negative zero is a zero
  const int groups = Cin / 64;
  const long j = blockIdx.x / groups;
  const int g = (int)(blockIdx.x % groups);
  const T* base = Z + j * pixels * Cin + (long)g * 64;
  int any = 0;
  for (long i = threadIdx.x; i < pixels * PER_ROW; i += blockDim.x) {
    const uint4 v = *reinterpret_cast<const uint4*>(base + (i / PER_ROW) * Cin + (i % PER_ROW) * (16 / (int)sizeof(T)));
    any |= ((v.x | v.y | v.z | v.w) & ABS) != 0u;
  }
  any = __syncthreads_or(any);
  if (threadIdx.x == 0) mask[blockIdx.x] = any ? 0 : 1;
}

// FP32 FMA throughput probe: every thread runs 16 independent chains of dependent FMAs on registers (no
// memory traffic), 4 blocks of 256 threads per SM's worth of grid; the result is stored so that the
// compiler keeps the arithmetic.
__global__ void __launch_bounds__(256) fma_rate_kernel(float* __restrict__ sink, int iters, float a, float b) {
  float v[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = (float)(threadIdx.x + i);
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = fmaf(v[i], a, b);
  }
  float t = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) t += v[i];
  sink[(long)blockIdx.x * blockDim.x + threadIdx.x] = t;
}

// ----------------------------------------------------------------------------------- per-pair ("independent") probing

// Layout of the scratch of xconv_wgrad_independent: header | Xr (the activation rebuilt per channel) | partial sums
struct IndepPlan { xconv_desc d2; WgradPlan p2; size_t x_off, part_off, bytes; };

static IndepPlan plan_indep(const xconv_desc* d) {
  IndepPlan ip{};
  ip.d2 = *d; ip.d2.r = d->B; ip.d2.chan_scale = nullptr;     // the contraction runs over the batch
  ip.d2.zero_blocks = nullptr;
  ip.p2 = plan_wgrad_core(&ip.d2);
  const size_t es = d->dtype == XCONV_F32 ? 4 : 2;
  const int T = kdepth(d) * d->KH * d->KW;
  ip.x_off = WS_HEADER;
  ip.part_off = ip.x_off + align_up((size_t)d->B * depth(d) * d->H * d->W * d->Cin * es, 256);
  const size_t part = ip.p2.tc_ct ? ip.p2.t.part_bytes : (size_t)ip.p2.splits * d->Cout * T * d->Cin * sizeof(float);
  ip.bytes = ip.part_off + align_up(part, 256);
  return ip;
}

static xconv_status validate_indep(const xconv_desc* d) {
  xconv_status s = validate(d);
  if (s != XCONV_OK) return s;
  if (d->r > 65535L * IS_JT || d->B > 65535L * IR_BT) return XCONV_ERR_UNSUPPORTED;     // grid z axes
  return XCONV_OK;
}

template <typename T>
static xconv_status run_sketch_indep(const xconv_desc* d, const void* X, const void* Z, float* S, cudaStream_t st) {
  const long N = (long)depth(d) * d->H * d->W;
  dim3 grid((unsigned)cdiv(d->B, IS_BT), (unsigned)cdiv(d->Cin, 32), (unsigned)cdiv(d->r, IS_JT));
  sketch_indep_simt<T><<<grid, 256, 0, st>>>(static_cast<const T*>(X), static_cast<const T*>(Z), S, d->r, d->B, N, d->Cin);
  return check_launch();
}

template <typename T>
static xconv_status run_rebuild_indep(const xconv_desc* d, const float* S, const void* Z, void* Xr, cudaStream_t st) {
  const long N = (long)depth(d) * d->H * d->W;
  dim3 grid((unsigned)cdiv(N, 8), (unsigned)cdiv(d->Cin, 32), (unsigned)cdiv(d->B, IR_BT));
  rebuild_indep_simt<T><<<grid, 256, 0, st>>>(S, static_cast<const T*>(Z), static_cast<T*>(Xr), d->r, d->B, N, d->Cin);
  return check_launch();
}

int launches() { return g_launches; }
void count_launch() { ++g_launches; }
void set_cuda_error(int e) { g_last_cuda_error = e; }

}  // namespace xconv

using namespace xconv;

extern "C" {

size_t xconv_workspace_bytes(const xconv_desc* desc, int op) {
  if (validate(desc) != XCONV_OK) return 0;
  switch (op) {
    case XCONV_OP_FORWARD:
    case XCONV_OP_SKETCH: return plan_sketch(desc).bytes;
    case XCONV_OP_WGRAD_SEEDED: return plan_wgrad(desc).bytes + (wgrad_redraws(desc) ? 0 : probes_bytes(desc));
    case XCONV_OP_SKETCH_SEEDED: {
      const SketchPlan p = plan_sketch(desc, true);
      return p.bytes + (sketch_redraws(desc, p) ? 0 : probes_bytes(desc));
    }
    case XCONV_OP_SKETCH_SEEDED_GAUSSIAN: return plan_sketch(desc).bytes + probes_bytes(desc);
    case XCONV_OP_WGRAD_SEEDED_GAUSSIAN: return plan_wgrad(desc).bytes + probes_bytes(desc);
    case XCONV_OP_WGRAD:
    case XCONV_OP_BACKPROBE:
    case XCONV_OP_CONTRACT: return plan_wgrad(desc).bytes;
    case XCONV_OP_DGRAD: return conv_ws_bytes(desc, true);
    case XCONV_OP_WGRAD_INDEPENDENT: return validate_indep(desc) == XCONV_OK ? plan_indep(desc).bytes : 0;
    default: return 0;
  }
}

int xconv_engine_for(const xconv_desc* desc, int op) {
  if (validate(desc) != XCONV_OK) return XCONV_ENGINE_NONE;
  const int tc = desc->dtype == XCONV_F16 ? XCONV_ENGINE_TCGEN05_F16 : XCONV_ENGINE_TCGEN05_BF16;
  switch (op) {
    case XCONV_OP_SKETCH: return plan_sketch(desc).tc ? tc : XCONV_ENGINE_SIMT_F32;
    case XCONV_OP_WGRAD:
    case XCONV_OP_CONTRACT: return plan_wgrad(desc).tc_ct ? tc : XCONV_ENGINE_SIMT_F32;
    case XCONV_OP_BACKPROBE: return plan_wgrad(desc).tc_bp ? tc : XCONV_ENGINE_SIMT_F32;
    case XCONV_OP_FORWARD:
    case XCONV_OP_DGRAD: {
      TcConvPlan t;
      const xconv_desc c = planes_cv(desc);
      return tc_plan_conv(&c, op == XCONV_OP_DGRAD, &t) ? tc : XCONV_ENGINE_SIMT_F32;
    }
    default: return XCONV_ENGINE_NONE;
  }
}

xconv_status xconv_sketch(const xconv_desc* desc, const void* X, const void* Z, float* sketch, void* ws,
                          size_t ws_bytes, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!X || !Z || !sketch) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(Z) || !aligned16(sketch)) return XCONV_ERR_ALIGNMENT;
  new_call();
  return run_sketch(desc, X, Z, sketch, ws, ws_bytes, static_cast<cudaStream_t>(cuda_stream));
}

xconv_status xconv_probes_from_seed(const xconv_desc* desc, unsigned long long seed, void* Z, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!Z) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(Z)) return XCONV_ERR_ALIGNMENT;
  new_call();
  return run_probes_from_seed(desc, seed, Z, static_cast<cudaStream_t>(cuda_stream));
}

xconv_status xconv_sketch_seeded(const xconv_desc* desc, const void* X, unsigned long long seed, float* sketch,
                                 void* ws, size_t ws_bytes, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!X || !sketch) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(sketch)) return XCONV_ERR_ALIGNMENT;
  new_call();
  return run_sketch(desc, X, nullptr, sketch, ws, ws_bytes, static_cast<cudaStream_t>(cuda_stream), &seed);
}

xconv_status xconv_wgrad_seeded(const xconv_desc* desc, const float* sketch, const void* dY, unsigned long long seed,
                                float* dW, void* ws, size_t ws_bytes, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!sketch || !dY || !dW) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(sketch) || !aligned16(dY) || !aligned16(dW)) return XCONV_ERR_ALIGNMENT;
  const size_t base = plan_wgrad(desc).bytes;
  const bool redraw = wgrad_redraws(desc);
  s = check_ws(ws, ws_bytes, base + (redraw ? 0 : probes_bytes(desc)));
  if (s != XCONV_OK) return s;
  new_call();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // r > B on the tensor cores: the first kernel of the estimator redraws its tiles of Z on chip
  if (redraw) return run_wgrad(desc, sketch, dY, nullptr, dW, ws, base, st, &seed);
  // Algorithm 1 backward step 2: redraw Z from the seed (behind the regular scratch), then steps 3-4
  char* Z = static_cast<char*>(ws) + base;
  s = run_probes_from_seed(desc, seed, Z, st);
  if (s != XCONV_OK) return s;
  return run_wgrad(desc, sketch, dY, Z, dW, ws, base, st);
}

xconv_status xconv_gaussian_probes_from_seed(const xconv_desc* desc, unsigned long long seed, void* Z,
                                             void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!Z) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(Z)) return XCONV_ERR_ALIGNMENT;
  new_call();
  return run_gaussian_probes(desc, seed, Z, static_cast<cudaStream_t>(cuda_stream));
}

xconv_status xconv_block_sparse_probes_from_seed(const xconv_desc* desc, unsigned long long seed, int gaussian, double p,
                                                 void* Z, unsigned char* keep, float* chan_scale, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!Z || !keep || !chan_scale || !(p >= 0.0 && p <= 1.0) || (gaussian != 0 && gaussian != 1)) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(Z)) return XCONV_ERR_ALIGNMENT;
  new_call();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  s = gaussian ? run_gaussian_probes(desc, seed, Z, st) : run_probes_from_seed(desc, seed, Z, st);
  if (s != XCONV_OK) return s;
  const long blocks = (long)desc->r * desc->Cin;
  const unsigned long long threshold = (unsigned long long)std::floor(p * 4294967296.0);
  block_keep_kernel<<<(unsigned)cdiv(cdiv(blocks, 4), 256), 256, 0, st>>>(keep, blocks, (uint32_t)(seed & 0xFFFFFFFFull),
                                                                          (uint32_t)(seed >> 32), threshold);
  if ((s = check_launch()) != XCONV_OK) return s;
  keep_scale_kernel<<<(unsigned)cdiv(desc->Cin, 256), 256, 0, st>>>(keep, desc->r, desc->Cin, chan_scale);
  if ((s = check_launch()) != XCONV_OK) return s;
  const long per_probe = (long)depth(desc) * desc->H * desc->W * desc->Cin, total = per_probe * desc->r;
  const unsigned grid = (unsigned)cdiv(cdiv(total, 4), 256);
  if (desc->dtype == XCONV_F32) drop_blocks_kernel<float><<<grid, 256, 0, st>>>(static_cast<float*>(Z), keep, total, per_probe, desc->Cin);
  else if (desc->dtype == XCONV_F16) drop_blocks_kernel<f16><<<grid, 256, 0, st>>>(static_cast<f16*>(Z), keep, total, per_probe, desc->Cin);
  else drop_blocks_kernel<bf16><<<grid, 256, 0, st>>>(static_cast<bf16*>(Z), keep, total, per_probe, desc->Cin);
  return check_launch();
}

xconv_status xconv_sketch_seeded_gaussian(const xconv_desc* desc, const void* X, unsigned long long seed,
                                          float* sketch, void* ws, size_t ws_bytes, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!X || !sketch) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(sketch)) return XCONV_ERR_ALIGNMENT;
  const size_t base = plan_sketch(desc).bytes;
  s = check_ws(ws, ws_bytes, base + probes_bytes(desc));
  if (s != XCONV_OK) return s;
  new_call();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* Z = static_cast<char*>(ws) + base;             // Z[seed] behind the regular scratch, then the regular kernels
  s = run_gaussian_probes(desc, seed, Z, st);
  if (s != XCONV_OK) return s;
  return run_sketch(desc, X, Z, sketch, ws, base, st);
}

xconv_status xconv_wgrad_seeded_gaussian(const xconv_desc* desc, const float* sketch, const void* dY,
                                         unsigned long long seed, float* dW, void* ws, size_t ws_bytes,
                                         void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!sketch || !dY || !dW) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(sketch) || !aligned16(dY) || !aligned16(dW)) return XCONV_ERR_ALIGNMENT;
  const size_t base = plan_wgrad(desc).bytes;
  s = check_ws(ws, ws_bytes, base + probes_bytes(desc));
  if (s != XCONV_OK) return s;
  new_call();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* Z = static_cast<char*>(ws) + base;             // Algorithm 1 backward step 2, then steps 3-4
  s = run_gaussian_probes(desc, seed, Z, st);
  if (s != XCONV_OK) return s;
  return run_wgrad(desc, sketch, dY, Z, dW, ws, base, st);
}

xconv_status xconv_sketch_independent(const xconv_desc* desc, const void* X, const void* Z, float* sketch,
                                      void* cuda_stream) {
  xconv_status s = validate_indep(desc);
  if (s != XCONV_OK) return s;
  if (!X || !Z || !sketch) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(Z) || !aligned16(sketch)) return XCONV_ERR_ALIGNMENT;
  new_call();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  return desc->dtype == XCONV_F32 ? run_sketch_indep<float>(desc, X, Z, sketch, st)
         : desc->dtype == XCONV_F16 ? run_sketch_indep<f16>(desc, X, Z, sketch, st)
                                    : run_sketch_indep<bf16>(desc, X, Z, sketch, st);
}

xconv_status xconv_wgrad_independent(const xconv_desc* desc, const float* sketch, const void* dY, const void* Z,
                                     float* dW, void* ws, size_t ws_bytes, void* cuda_stream) {
  xconv_status s = validate_indep(desc);
  if (s != XCONV_OK) return s;
  if (!sketch || !dY || !Z || !dW) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(sketch) || !aligned16(dY) || !aligned16(Z) || !aligned16(dW)) return XCONV_ERR_ALIGNMENT;
  const IndepPlan ip = plan_indep(desc);
  if ((s = validate(&ip.d2)) != XCONV_OK) return s;
  s = check_ws(ws, ws_bytes, ip.bytes);
  if (s != XCONV_OK) return s;
  new_call();
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* w = static_cast<char*>(ws);
  s = desc->dtype == XCONV_F32 ? run_rebuild_indep<float>(desc, sketch, Z, w + ip.x_off, st)
      : desc->dtype == XCONV_F16 ? run_rebuild_indep<f16>(desc, sketch, Z, w + ip.x_off, st)
                                 : run_rebuild_indep<bf16>(desc, sketch, Z, w + ip.x_off, st);
  if (s != XCONV_OK) return s;
  return run_contract(&ip.d2, ip.p2, dY, w + ip.x_off, dW, 1.0f / (float)desc->r, w + ip.part_off, w, st);
}

xconv_status xconv_forward(const xconv_desc* desc, const void* X, const void* W, const void* Z, void* Y,
                           float* sketch, void* ws, size_t ws_bytes, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!X || !W || !Z || !Y || !sketch) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W) || !aligned16(Z) || !aligned16(Y) || !aligned16(sketch))
    return XCONV_ERR_ALIGNMENT;
  const SketchPlan p = plan_sketch(desc);
  if (!ws || ws_bytes < p.bytes) return XCONV_ERR_WORKSPACE;
  if (!aligned16(ws)) return XCONV_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  new_call();
  s = run_conv(desc, false, X, W, Y, static_cast<char*>(ws), st);
  if (s != XCONV_OK) return s;
  return run_sketch(desc, X, Z, sketch, ws, ws_bytes, st);
}

xconv_status xconv_wgrad(const xconv_desc* desc, const float* sketch, const void* dY, const void* Z, float* dW,
                         void* ws, size_t ws_bytes, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!sketch || !dY || !Z || !dW) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(sketch) || !aligned16(dY) || !aligned16(Z) || !aligned16(dW)) return XCONV_ERR_ALIGNMENT;
  if (desc->chan_scale && (reinterpret_cast<uintptr_t>(desc->chan_scale) & 3u)) return XCONV_ERR_ALIGNMENT;
  new_call();
  return run_wgrad(desc, sketch, dY, Z, dW, ws, ws_bytes, static_cast<cudaStream_t>(cuda_stream));
}

size_t xconv_backprobe_bytes(const xconv_desc* desc) {
  if (validate(desc) != XCONV_OK) return 0;
  return (size_t)desc->r * depth(desc) * desc->H * desc->W * desc->Cout * (desc->dtype == XCONV_F32 ? 4 : 2);
}

xconv_status xconv_backprobe(const xconv_desc* desc, const float* sketch, const void* dY, void* L, void* ws,
                             size_t ws_bytes, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!sketch || !dY || !L) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(sketch) || !aligned16(dY) || !aligned16(L)) return XCONV_ERR_ALIGNMENT;
  const WgradPlan p = plan_wgrad(desc);
  s = check_ws(ws, ws_bytes, p.bytes);
  if (s != XCONV_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  new_call();
  return run_backprobe(desc, p, sketch, dY, L, static_cast<char*>(ws) + p.sb_off, static_cast<char*>(ws), st);
}

xconv_status xconv_contract(const xconv_desc* desc, const void* L, const void* Z, float* dW, void* ws,
                            size_t ws_bytes, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!L || !Z || !dW) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(L) || !aligned16(Z) || !aligned16(dW)) return XCONV_ERR_ALIGNMENT;
  if (desc->chan_scale && (reinterpret_cast<uintptr_t>(desc->chan_scale) & 3u)) return XCONV_ERR_ALIGNMENT;
  const WgradPlan p = plan_wgrad(desc);
  s = check_ws(ws, ws_bytes, p.bytes);
  if (s != XCONV_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  new_call();
  return run_contract(desc, p, L, Z, dW, 1.0f / (float)desc->r, static_cast<char*>(ws) + p.part_off,
                      static_cast<char*>(ws), st);
}

xconv_status xconv_dgrad(const xconv_desc* desc, const void* dY, const void* W, void* dX, void* ws,
                         size_t ws_bytes, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!dY || !W || !dX) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(W) || !aligned16(dX)) return XCONV_ERR_ALIGNMENT;
  if (!ws || ws_bytes < conv_ws_bytes(desc, true)) return XCONV_ERR_WORKSPACE;
  if (!aligned16(ws)) return XCONV_ERR_ALIGNMENT;
  new_call();
  return run_conv(desc, true, dY, W, dX, static_cast<char*>(ws), static_cast<cudaStream_t>(cuda_stream));
}

// Arena layout of the host-buffer entry point: X | dY | Z | S | dW | workspace, each 256-aligned.
struct HostArena { size_t x, dy, z, s, dw, ws, ws_bytes, total, xb, dyb, zb, sb, dwb; };
static HostArena host_arena(const xconv_desc* d) {
  HostArena a{};
  const size_t es = d->dtype == XCONV_F32 ? 4 : 2;
  const size_t px = (size_t)depth(d) * d->H * d->W;
  a.xb = (size_t)d->B * px * d->Cin * es;
  a.dyb = (size_t)d->B * px * d->Cout * es;
  a.zb = (size_t)d->r * px * d->Cin * es;
  a.sb = (size_t)d->r * d->B * 4;
  a.dwb = (size_t)d->Cout * kdepth(d) * d->KH * d->KW * d->Cin * 4;
  a.x = 0;
  a.dy = a.x + align_up(a.xb, 256);
  a.z = a.dy + align_up(a.dyb, 256);
  a.s = a.z + align_up(a.zb, 256);
  a.dw = a.s + align_up(a.sb, 256);
  a.ws = a.dw + align_up(a.dwb, 256);
  a.ws_bytes = std::max(plan_sketch(d).bytes, plan_wgrad(d).bytes);
  a.total = a.ws + a.ws_bytes;
  return a;
}

size_t xconv_host_arena_bytes(const xconv_desc* desc) {
  if (validate(desc) != XCONV_OK) return 0;
  return host_arena(desc).total;
}

xconv_status xconv_sketch_wgrad_host(const xconv_desc* desc, const void* hX, const void* hdY, const void* hZ,
                                     float* hS, float* hdW, void* arena, size_t arena_bytes, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!hX || !hdY || !hZ || !hS || !hdW || !arena) return XCONV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(arena) & 255u) return XCONV_ERR_ALIGNMENT;
  const HostArena a = host_arena(desc);
  if (arena_bytes < a.total) return XCONV_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* base = static_cast<char*>(arena);
  cudaError_t e;
  if ((e = cudaMemcpyAsync(base + a.x, hX, a.xb, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
      (e = cudaMemcpyAsync(base + a.z, hZ, a.zb, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
      (e = cudaMemcpyAsync(base + a.dy, hdY, a.dyb, cudaMemcpyHostToDevice, st)) != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return XCONV_ERR_CUDA;
  }
  new_call();
  float* S = reinterpret_cast<float*>(base + a.s);
  float* dW = reinterpret_cast<float*>(base + a.dw);
  s = run_sketch(desc, base + a.x, base + a.z, S, base + a.ws, a.ws_bytes, st);
  if (s != XCONV_OK) return s;
  s = run_wgrad(desc, S, base + a.dy, base + a.z, dW, base + a.ws, a.ws_bytes, st);
  if (s != XCONV_OK) return s;
  if ((e = cudaMemcpyAsync(hS, S, a.sb, cudaMemcpyDeviceToHost, st)) != cudaSuccess ||
      (e = cudaMemcpyAsync(hdW, dW, a.dwb, cudaMemcpyDeviceToHost, st)) != cudaSuccess ||
      (e = cudaStreamSynchronize(st)) != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return XCONV_ERR_CUDA;
  }
  return XCONV_OK;
}

xconv_status xconv_selftest_wait_limit(void* ws, size_t ws_bytes, unsigned int limit_ms, void* cuda_stream) {
  if (!ws || ws_bytes < WS_HEADER) return XCONV_ERR_WORKSPACE;
  if (!aligned16(ws)) return XCONV_ERR_ALIGNMENT;
  if (limit_ms == 0 || limit_ms > 2000) return XCONV_ERR_INVALID_ARG;
  new_call();
  return tc_run_wait_selftest(static_cast<char*>(ws), (unsigned long long)limit_ms * 1000000ull,
                              static_cast<cudaStream_t>(cuda_stream));
}

xconv_status xconv_workspace_status(const void* ws, void* cuda_stream) {
  if (!ws) return XCONV_ERR_INVALID_ARG;
  unsigned int word[2] = {0, 0};
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemcpyAsync(word, ws, sizeof(word), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; return XCONV_ERR_CUDA; }
  return (word[0] != WS_OK && word[0] == word[1]) ? XCONV_ERR_TIMEOUT : XCONV_OK;
}

int xconv_zero_blocks_used(const xconv_desc* desc) {
  if (validate(desc) != XCONV_OK || desc->zero_blocks == nullptr) return 0;
  const WgradPlan p = plan_wgrad(desc);
  return (p.tc_ct && p.t.ct_masked) ? 1 : 0;
}

xconv_status xconv_zero_blocks(const xconv_desc* desc, const void* Z, unsigned char* mask, void* cuda_stream) {
  xconv_status s = validate(desc);
  if (s != XCONV_OK) return s;
  if (!Z || !mask) return XCONV_ERR_INVALID_ARG;
  if (!aligned16(Z)) return XCONV_ERR_ALIGNMENT;
  if (desc->Cin % 64 != 0 || (long)desc->r * (desc->Cin / 64) > 2000000000L) return XCONV_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const long pixels = (long)depth(desc) * desc->H * desc->W;
  const unsigned blocks = (unsigned)((long)desc->r * (desc->Cin / 64));
  new_call();
  if (desc->dtype == XCONV_F32) zero_blocks_kernel<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(Z), mask, pixels, desc->Cin);
  else zero_blocks_kernel<unsigned short><<<blocks, 256, 0, st>>>(static_cast<const unsigned short*>(Z), mask, pixels, desc->Cin);
  ++g_launches;
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; return XCONV_ERR_CUDA; }
  return XCONV_OK;
}

xconv_status xconv_measure_fma_rate(void* scratch, size_t scratch_bytes, double* tflops, void* cuda_stream) {
  const int blocks = 148 * 16, threads = 256, iters = 4096;
  if (!scratch || !tflops) return XCONV_ERR_INVALID_ARG;
  if (scratch_bytes < (size_t)blocks * threads * sizeof(float)) return XCONV_ERR_WORKSPACE;
  if (!aligned16(scratch)) return XCONV_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaError_t e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  float best_ms = 0.f;
  new_call();
  for (int rep = 0; rep < 6 && e == cudaSuccess; ++rep) {      // the first repetition warms up
    cudaEventRecord(e0, st);
    fma_rate_kernel<<<blocks, threads, 0, st>>>(static_cast<float*>(scratch), iters, 0.999f, 0.001f);
    ++g_launches;
    cudaEventRecord(e1, st);
    e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (rep > 0 && (best_ms == 0.f || ms < best_ms)) best_ms = ms;
  }
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (e != cudaSuccess || best_ms <= 0.f) { g_last_cuda_error = (int)e; return XCONV_ERR_CUDA; }
  *tflops = 2.0 * 16.0 * iters * (double)blocks * threads / (best_ms * 1e-3) / 1e12;
  return XCONV_OK;
}

int xconv_last_launch_count(void) { return g_launches; }
int xconv_last_cuda_error(void) { return g_last_cuda_error; }

const char* xconv_status_string(xconv_status s) {
  switch (s) {
    case XCONV_OK: return "ok";
    case XCONV_ERR_INVALID_ARG: return "invalid argument";
    case XCONV_ERR_UNSUPPORTED: return "unsupported layer or option (no kernel; there is no fallback)";
    case XCONV_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case XCONV_ERR_WORKSPACE: return "workspace missing or too small";
    case XCONV_ERR_CUDA: return "CUDA call failed";
    case XCONV_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    default: return "unknown status";
  }
}

}  // extern "C"
