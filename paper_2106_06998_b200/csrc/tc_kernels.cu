// tcgen05 / TMEM / TMA kernels for bfloat16 storage (sm_100a).
//
// One kernel template, three problem shapes, all dense contractions with float accumulation in
// tensor memory:
//   SKETCH    S = Z^T X       (Algorithm 1 forward step 3)  D[row,col] = sum_k A[row,k] Bm[col,k],
//             both operands contiguous along k = (pixel, channel): K-major tiles, plain 2-D maps.
//   BACKPROBE L = S dY^T      (backward step 3)  D[q,j] = sum_b dY[b,q] S[j,b]: the A tile is read
//             with q (pixel, channel) contiguous, i.e. MN-major; S (bfloat16 copy) is K-major.
//   CONTRACT  dW = tr(L T Z)  (backward step 4, Eq. 6)  D[m,n] = sum_{j,pixel} L[j,pixel,m] Z[j,pixel+k,n]
//             for one kernel offset k per CTA: both tiles MN-major (channels contiguous), the
//             reduction runs over image patches, and the offset is added to the patch coordinates of
//             the TMA box of Z -- out-of-image rows are zero-filled by the TMA unit, which is exactly
//             the zero padding of the convolution.  No shifted or im2col copy of Z is ever made.
//
// Structure of a CTA (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = epilogue (one TMEM lane quadrant each).  A ring of shared-memory stages is handed
// from producer to issuer with mbarriers; tcgen05.commit returns stages and signals the epilogue.
// Every wait is bounded: on expiry the CTA records WS_TIMEOUT in the workspace status word, drains
// its outstanding copies (bounded again), frees its tensor memory and returns.
#include "tc_api.h"

#include <cuda.h>
#include <cudaTypedefs.h>

#include <algorithm>

#include "common.cuh"

namespace xconv {

enum : int { MODE_SKETCH = 0, MODE_BACKPROBE = 1, MODE_CONTRACT = 2 };

struct TcParams {
  int mode;
  int tile_n;              // MMA N (multiple of 16, <= 256)
  int tmem_cols;           // power of two >= max(32, tile_n)
  int stages;
  int ksteps;              // UMMA k-steps (of 16) per stage
  uint32_t a_stage_bytes, b_stage_bytes, tx_bytes;
  int a_boxes, b_boxes;    // TMA boxes per stage and operand
  uint32_t a_box_bytes, b_box_bytes;
  int a_mn_major, b_mn_major;
  uint32_t a_lbo, b_lbo;   // leading byte offsets of the UMMA descriptors
  int tiles_m, tiles_n;    // blockIdx.x = (tap * tiles_m + tm) * tiles_n + tn
  long kblocks, kblocks_per_split;
  // contraction geometry
  int patch_w, patch_h, patches_x, patches_y, pad;
  // extents for the epilogue guards
  long rows, cols;         // valid MMA rows / columns of the whole problem
  // outputs
  float* part;             // SKETCH: [split][rows][cols]; CONTRACT: [split][Cout][T][Cin]
  bf16* L;                 // BACKPROBE: [r][Q]
  long Q;
  int T, Cin;              // CONTRACT output indexing
  unsigned int* status;
};

// ------------------------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: about one second after a short spin.  Returns false (and records the code) on expiry.
__device__ __noinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned int* status) {
  for (int i = 0; i < 4096; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_ns() - t0 > 1000000000ull) {
      atomicExch(status, (unsigned int)WS_TIMEOUT);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], bfloat16 inputs, float accumulate; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// mbarrier arrive once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp receives lane (quadrant*32 + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
// Byte offsets are encoded without their 4 low bits.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}

constexpr int TILE_M = 128;
constexpr int MAX_STAGES = 8;
constexpr int TC_THREADS = 192;

// ------------------------------------------------------------------------------------ the kernel

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t tmem_full_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int go;

  // an earlier CTA gave up: leave at once (one thread reads the word so that the whole CTA agrees)
  if (threadIdx.x == 0) go = (*reinterpret_cast<volatile unsigned int*>(p.status) == WS_OK) ? 1 : 0;
  __syncthreads();
  if (!go) return;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;          // 128B swizzle wants 1024B alignment
  const uint32_t stage_bytes = p.a_stage_bytes + p.b_stage_bytes;

  // tile of this CTA
  int t = blockIdx.x;
  const int tn = t % p.tiles_n; t /= p.tiles_n;
  const int tm = t % p.tiles_m; t /= p.tiles_m;
  const int tap = t;
  const long kb0 = (long)blockIdx.y * p.kblocks_per_split;
  const long kb1 = min(p.kblocks, kb0 + p.kblocks_per_split);
  const int nkb = (int)max(0L, kb1 - kb0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(&tmem_full_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    prefetch_tmap(&map_a);
    prefetch_tmap(&map_b);
  }
  if (warp == 1) tmem_alloc(&tmem_slot, (uint32_t)p.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (int i = 0; i < nkb && ok; ++i) {
        const int s = i % p.stages;
        if (i >= p.stages) ok = mbar_wait(&empty_bar[s], (uint32_t)(((i / p.stages) - 1) & 1), p.status);
        if (!ok) break;
        const long kb = kb0 + i;
        const uint32_t a_dst = tiles_base + (uint32_t)s * stage_bytes;
        const uint32_t b_dst = a_dst + p.a_stage_bytes;
        mbar_arrive_expect_tx(&full_bar[s], p.tx_bytes);
        if (p.mode == MODE_SKETCH) {
          tma_load_2d(a_dst, &map_a, (int)(kb * 64), tm * TILE_M, &full_bar[s]);
          tma_load_2d(b_dst, &map_b, (int)(kb * 64), tn * p.tile_n, &full_bar[s]);
        } else if (p.mode == MODE_BACKPROBE) {
          const int brow = (int)kb * p.ksteps * 16;
          for (int bx = 0; bx < p.a_boxes; ++bx)
            tma_load_2d(a_dst + bx * p.a_box_bytes, &map_a, tm * TILE_M + bx * 64, brow, &full_bar[s]);
          tma_load_2d(b_dst, &map_b, brow, tn * p.tile_n, &full_bar[s]);
        } else {
          long u = kb;
          const int px = (int)(u % p.patches_x); u /= p.patches_x;
          const int py = (int)(u % p.patches_y); u /= p.patches_y;
          const int j = (int)u;
          const int ks = 2 * p.pad + 1;
          const int dy = tap / ks - p.pad, dx = tap % ks - p.pad;
          const int x0 = px * p.patch_w, y0 = py * p.patch_h;
          for (int bx = 0; bx < p.a_boxes; ++bx)
            tma_load_4d(a_dst + bx * p.a_box_bytes, &map_a, tm * TILE_M + bx * 64, x0, y0, j, &full_bar[s]);
          for (int bx = 0; bx < p.b_boxes; ++bx)
            tma_load_4d(b_dst + bx * p.b_box_bytes, &map_b, tn * p.tile_n + bx * 64, x0 + dx, y0 + dy, j,
                        &full_bar[s]);
        }
        issued = i + 1;
      }
      // drain: every copy issued must have landed in this CTA's shared memory before it exits
      // (immediate on the normal path, bounded on the failure path)
      for (int i = max(0, issued - p.stages); i < issued; ++i)
        if (!mbar_wait(&full_bar[i % p.stages], (uint32_t)((i / p.stages) & 1), p.status)) break;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn_major << 15) |
                             ((uint32_t)p.b_mn_major << 16) | ((uint32_t)(p.tile_n >> 3) << 17) |
                             ((uint32_t)(TILE_M >> 4) << 24);
      // K-major: 8-row groups 1024 B apart, k-step = 32 B inside the swizzled row.
      // MN-major: 8-row (k) groups 1024 B apart, 64-column blocks `lbo` apart, k-step = 16 rows = 2048 B.
      const uint32_t a_step = p.a_mn_major ? 2048u : 32u, b_step = p.b_mn_major ? 2048u : 32u;
      const uint32_t a_lbo = p.a_mn_major ? p.a_lbo : 16u, b_lbo = p.b_mn_major ? p.b_lbo : 16u;
      bool ok = true;
      for (int i = 0; i < nkb; ++i) {
        const int s = i % p.stages;
        ok = mbar_wait(&full_bar[s], (uint32_t)((i / p.stages) & 1), p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_src = tiles_base + (uint32_t)s * stage_bytes;
        const uint32_t b_src = a_src + p.a_stage_bytes;
        for (int k = 0; k < p.ksteps; ++k) {
          const uint64_t da = make_desc(a_src + k * a_step, a_lbo, 1024u);
          const uint64_t db = make_desc(b_src + k * b_step, b_lbo, 1024u);
          umma_bf16(tmem_base, da, db, idesc, (i > 0 || k > 0) ? 1u : 0u);
        }
        umma_commit(&empty_bar[s]);          // stage s may be refilled once these MMAs have read it
      }
      if (ok && nkb > 0) umma_commit(&tmem_full_bar);
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;                  // TMEM lanes [32*quad, 32*quad+32)
    bool ok = true;
    if (nkb > 0) {
      if (lane == 0) ok = mbar_wait(&tmem_full_bar, 0u, p.status);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      tc_fence_after();
    }
    if (ok) {
      const long row = (long)tm * TILE_M + quad * 32 + lane;
      const long col0 = (long)tn * p.tile_n;
      for (int c = 0; c < p.tile_n; c += 32) {
        uint32_t v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = 0u;
        if (nkb > 0) {
          const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)c;
          if (p.tile_n - c >= 32) tmem_ld32(taddr, v);
          else { tmem_ld16(taddr, v); }
        }
        const int nc = min(32, p.tile_n - c);
        if (p.mode == MODE_BACKPROBE) {
          // D[q, j] -> L[j][q]: a warp writes 32 consecutive q of one probe per instruction
          if (row < p.rows) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const long j = col0 + c + i;
              if (i < nc && j < p.cols) p.L[j * p.Q + row] = __float2bfloat16_rn(__uint_as_float(v[i]));
            }
          }
        } else {
          float* dst;
          if (p.mode == MODE_SKETCH) dst = p.part + ((long)blockIdx.y * p.rows + row) * p.cols + col0 + c;
          else dst = p.part + (((long)blockIdx.y * p.rows + row) * p.T + tap) * p.Cin + col0 + c;
          if (row < p.rows) {
            const bool vec = ((p.cols & 3) == 0);
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              if (i >= nc) break;
              if (vec && col0 + c + i + 3 < p.cols) {
                *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]),
                                                                  __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
              } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  if (col0 + c + i + e < p.cols) dst[i + e] = __uint_as_float(v[i + e]);
              }
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

// S[j][b] = sum_s part[s][row][col]; (row, col) = (b, j) when the samples were the MMA rows.
__global__ void reduce_sketch_partials(const float* __restrict__ part, float* __restrict__ S, int r, int B,
                                       int splits, int swapped) {
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const long count = (long)r * B;
  if (i >= count) return;
  const int j = (int)(i / B), b = (int)(i % B);
  const long src = swapped ? (long)b * r + j : i;
  float s = 0.f;
  for (int k = 0; k < splits; ++k) s += part[(long)k * count + src];
  S[i] = s;
}

__global__ void reduce_contract_partials(const float* __restrict__ part, float* __restrict__ out, long count,
                                         int splits, float alpha, const float* __restrict__ chan_scale, int period) {
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  float s = 0.f;
  for (int k = 0; k < splits; ++k) s += part[(long)k * count + i];
  out[i] = s * (chan_scale ? chan_scale[i % period] : alpha);
}

// ------------------------------------------------------------------------------------ host side

static inline long cdivl(long a, long b) { return (a + b - 1) / b; }
static inline int round_up(int v, int a) { return (v + a - 1) / a * a; }
static const int SMEM_LIMIT = 227 * 1024;
static const int STATIC_SMEM_SLACK = 2048;     // barriers + alignment slack

static PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ptr);
  }
  return fn;
}

// bfloat16 tensor map with 128-byte swizzle; dims/strides innermost first, strides in bytes for dims 1..rank-1.
static bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides,
                     const uint32_t* box) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  cuuint64_t d[5], st[4];
  cuuint32_t bx[5];
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; bx[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) st[i] = strides[i];
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, st, bx, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

static int pow2_cols(int n) { int c = 32; while (c < n) c *= 2; return c; }

static int pick_stages(uint32_t stage_bytes, int want_ctas_per_sm) {
  const int budget = SMEM_LIMIT / want_ctas_per_sm - STATIC_SMEM_SLACK;
  int s = budget / (int)stage_bytes;
  return std::max(1, std::min(s, MAX_STAGES));
}

static xconv_status launch(const CUtensorMap& ma, const CUtensorMap& mb, const TcParams& p, dim3 grid,
                           cudaStream_t st) {
  const size_t smem = (size_t)p.stages * (p.a_stage_bytes + p.b_stage_bytes) + 1024;
  if (smem > (size_t)(SMEM_LIMIT - 1024)) return XCONV_ERR_UNSUPPORTED;
  {
    cudaError_t e = cudaFuncSetAttribute(tc_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT - 1024);
    if (e != cudaSuccess) { set_cuda_error((int)e); return XCONV_ERR_CUDA; }
  }
  tc_gemm_kernel<<<grid, TC_THREADS, smem, st>>>(ma, mb, p);
  count_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return XCONV_ERR_CUDA; }
  return XCONV_OK;
}

// ---- sketch --------------------------------------------------------------------------------

bool tc_plan_sketch(const xconv_desc* d, TcSketchPlan* p) {
  if (d->dtype != XCONV_BF16) return false;
  const long K = (long)d->H * d->W * d->Cin;
  if (K % 8 != 0 || K < 2048 || K > 2000000000L) return false;
  p->swap = d->B >= d->r ? 1 : 0;
  const int rows = p->swap ? d->B : d->r, cols = p->swap ? d->r : d->B;
  p->tile_m = TILE_M;
  p->tile_n = std::min(256, round_up(cols, 16));
  p->tiles_m = (int)cdivl(rows, TILE_M);
  p->tiles_n = (int)cdivl(cols, p->tile_n);
  p->kblocks = cdivl(K, 64);
  const uint32_t stage = TILE_M * 128 + p->tile_n * 128;
  const int ctas = (stage * 4 + STATIC_SMEM_SLACK <= SMEM_LIMIT / 2 && p->tile_n <= 128) ? 2 : 1;
  p->stages = pick_stages(stage, ctas);
  const long tiles = (long)p->tiles_m * p->tiles_n;
  long splits = std::max(1L, std::min((148L * ctas) / tiles, p->kblocks / 8));
  if (tiles >= 148L * ctas) splits = 1;
  splits = std::max(1L, std::min(splits, 512L));
  p->kblocks_per_split = cdivl(p->kblocks, splits);
  p->splits = (int)cdivl(p->kblocks, p->kblocks_per_split);
  p->part_bytes = (size_t)p->splits * rows * cols * sizeof(float);
  return true;
}

xconv_status tc_run_sketch(const xconv_desc* d, const TcSketchPlan& pl, const void* X, const void* Z, float* S,
                           char* ws_head, char* part, cudaStream_t st) {
  const long K = (long)d->H * d->W * d->Cin;
  const int rows = pl.swap ? d->B : d->r, cols = pl.swap ? d->r : d->B;
  const void* A = pl.swap ? X : Z;
  const void* Bm = pl.swap ? Z : X;
  CUtensorMap ma, mb;
  const uint64_t da[2] = {(uint64_t)K, (uint64_t)rows}, db[2] = {(uint64_t)K, (uint64_t)cols};
  const uint64_t sa[1] = {(uint64_t)K * 2};
  // full boxes always: rows and k positions past the tensor are zero-filled by the TMA unit
  const uint32_t box_a[2] = {64, (uint32_t)TILE_M};
  const uint32_t box_b[2] = {64, (uint32_t)pl.tile_n};
  if (!make_map(&ma, A, 2, da, sa, box_a) || !make_map(&mb, Bm, 2, db, sa, box_b)) return XCONV_ERR_CUDA;
  TcParams p{};
  p.mode = MODE_SKETCH;
  p.tile_n = pl.tile_n;
  p.tmem_cols = pow2_cols(pl.tile_n);
  p.stages = pl.stages;
  p.ksteps = 4;
  p.a_stage_bytes = TILE_M * 128;
  p.b_stage_bytes = (uint32_t)pl.tile_n * 128;
  p.tx_bytes = p.a_stage_bytes + p.b_stage_bytes;
  p.a_boxes = p.b_boxes = 1;
  p.a_mn_major = p.b_mn_major = 0;
  p.tiles_m = pl.tiles_m;
  p.tiles_n = pl.tiles_n;
  p.kblocks = pl.kblocks;
  p.kblocks_per_split = pl.kblocks_per_split;
  p.rows = rows;
  p.cols = cols;
  p.part = reinterpret_cast<float*>(part);
  p.status = reinterpret_cast<unsigned int*>(ws_head);
  xconv_status s = launch(ma, mb, p, dim3((unsigned)(pl.tiles_m * pl.tiles_n), (unsigned)pl.splits), st);
  if (s != XCONV_OK) return s;
  const long count = (long)d->r * d->B;
  reduce_sketch_partials<<<(unsigned)cdivl(count, 256), 256, 0, st>>>(p.part, S, d->r, d->B, pl.splits, pl.swap);
  count_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return XCONV_ERR_CUDA; }
  return XCONV_OK;
}

// ---- weight gradient -----------------------------------------------------------------------

static void pick_patch(int H, int W, int* pw, int* ph) {
  // patch of pw x ph pixels, pw*ph a multiple of 16 and at most 128, covering the image with the
  // least zero-filled overhang; ties go to the larger, then the wider patch
  double best = 1e30; int bw = 16, bh = 1, barea = 0;
  for (int w = 1; w <= std::min(W, 128); ++w)
    for (int h = 1; h * w <= 128 && h <= H; ++h) {
      if ((w * h) % 16) continue;
      const double waste = (double)(cdivl(W, w) * w) * (double)(cdivl(H, h) * h) / ((double)W * H);
      if (waste < best - 1e-9 || (waste < best + 1e-9 && (w * h > barea || (w * h == barea && w > bw)))) {
        best = waste; bw = w; bh = h; barea = w * h;
      }
    }
  if (barea == 0) { bw = std::min(16, 128); bh = 1; }     // tiny images: one 16-pixel row box, mostly zero fill
  *pw = bw; *ph = bh;
}

int tc_plan_wgrad(const xconv_desc* d, TcWgradPlan* p) {
  if (d->dtype != XCONV_BF16) return 0;
  int mask = 0;
  const long Q = (long)d->H * d->W * d->Cout;
  // back-probe: D[q, j], rows = Q, cols = r, k = B
  if (Q % 8 == 0 && d->B % 8 == 0 && Q >= 2048 && Q < 2000000000L) {
    mask |= 1;
    p->bp_tile_n = std::min(256, round_up(d->r, 16));
    p->bp_tiles_q = (int)cdivl(Q, TILE_M);
    p->bp_tiles_r = (int)cdivl(d->r, p->bp_tile_n);
    p->bp_ksteps = std::min(4, (int)cdivl(d->B, 16));
    const uint32_t stage = (uint32_t)p->bp_ksteps * 16 * 128 * 2 + (uint32_t)p->bp_tile_n * 128;
    p->bp_stages = pick_stages(stage, p->bp_tile_n <= 128 ? 2 : 1);
  }
  // contraction: rows = Cout, cols = Cin per offset, k = (probe, patch)
  const int T = d->KH * d->KW;
  if (d->Cout % 8 == 0 && d->Cin % 8 == 0 && d->Cout >= 64 && d->Cin >= 64 && (long)d->H * d->W >= 16) {
    mask |= 2;
    pick_patch(d->H, d->W, &p->patch_w, &p->patch_h);
    p->patches_x = (int)cdivl(d->W, p->patch_w);
    p->patches_y = (int)cdivl(d->H, p->patch_h);
    p->ct_tile_n = std::min(256, round_up(d->Cin, 16));
    p->ct_tiles_m = (int)cdivl(d->Cout, TILE_M);
    p->ct_tiles_n = (int)cdivl(d->Cin, p->ct_tile_n);
    const int bk = p->patch_w * p->patch_h;
    const uint32_t stage = (uint32_t)bk * 128 * (2 + (uint32_t)cdivl(p->ct_tile_n, 64));
    p->ct_stages = pick_stages(stage, 1);
    p->ct_items = (long)d->r * p->patches_x * p->patches_y;
    const long tiles = (long)p->ct_tiles_m * p->ct_tiles_n * T;
    long splits = std::max(1L, std::min(148L / std::max(1L, tiles), p->ct_items / 4));
    splits = std::max(1L, std::min(splits, 512L));
    p->ct_items_per_split = cdivl(p->ct_items, splits);
    p->ct_splits = (int)cdivl(p->ct_items, p->ct_items_per_split);
    p->part_bytes = (size_t)p->ct_splits * d->Cout * T * d->Cin * sizeof(float);
  }
  return mask;
}

xconv_status tc_run_backprobe(const xconv_desc* d, const TcWgradPlan& pl, const void* S_bf16, const void* dY,
                              void* L, char* ws_head, cudaStream_t st) {
  const long Q = (long)d->H * d->W * d->Cout;
  const int bk = pl.bp_ksteps * 16;
  CUtensorMap ma, mb;
  const uint64_t da[2] = {(uint64_t)Q, (uint64_t)d->B}, db[2] = {(uint64_t)d->B, (uint64_t)d->r};
  const uint64_t sa[1] = {(uint64_t)Q * 2}, sb[1] = {(uint64_t)d->B * 2};
  const uint32_t box_a[2] = {64, (uint32_t)bk};
  const uint32_t box_b[2] = {64, (uint32_t)pl.bp_tile_n};     // 128-byte rows whatever bk is (zero fill past B)
  if (!make_map(&ma, dY, 2, da, sa, box_a) || !make_map(&mb, S_bf16, 2, db, sb, box_b)) return XCONV_ERR_CUDA;
  TcParams p{};
  p.mode = MODE_BACKPROBE;
  p.tile_n = pl.bp_tile_n;
  p.tmem_cols = pow2_cols(pl.bp_tile_n);
  p.stages = pl.bp_stages;
  p.ksteps = pl.bp_ksteps;
  p.a_boxes = 2;
  p.b_boxes = 1;
  p.a_box_bytes = (uint32_t)bk * 128;
  p.a_stage_bytes = 2 * p.a_box_bytes;
  p.b_stage_bytes = (uint32_t)pl.bp_tile_n * 128;
  p.b_box_bytes = p.b_stage_bytes;
  p.tx_bytes = p.a_stage_bytes + p.b_stage_bytes;
  p.a_mn_major = 1;
  p.b_mn_major = 0;
  p.a_lbo = p.a_box_bytes;
  p.tiles_m = pl.bp_tiles_q;
  p.tiles_n = pl.bp_tiles_r;
  p.kblocks = cdivl(d->B, bk);
  p.kblocks_per_split = p.kblocks;
  p.rows = Q;
  p.cols = d->r;
  p.L = static_cast<bf16*>(L);
  p.Q = Q;
  p.status = reinterpret_cast<unsigned int*>(ws_head);
  return launch(ma, mb, p, dim3((unsigned)((long)pl.bp_tiles_q * pl.bp_tiles_r), 1), st);
}

xconv_status tc_run_contract(const xconv_desc* d, const TcWgradPlan& pl, const void* L, const void* Z, float* dW,
                             char* ws_head, char* part, cudaStream_t st) {
  const int T = d->KH * d->KW;
  const int bk = pl.patch_w * pl.patch_h;
  CUtensorMap ma, mb;
  const uint64_t da[4] = {(uint64_t)d->Cout, (uint64_t)d->W, (uint64_t)d->H, (uint64_t)d->r};
  const uint64_t sa[3] = {(uint64_t)d->Cout * 2, (uint64_t)d->W * d->Cout * 2, (uint64_t)d->H * d->W * d->Cout * 2};
  const uint64_t db[4] = {(uint64_t)d->Cin, (uint64_t)d->W, (uint64_t)d->H, (uint64_t)d->r};
  const uint64_t sb[3] = {(uint64_t)d->Cin * 2, (uint64_t)d->W * d->Cin * 2, (uint64_t)d->H * d->W * d->Cin * 2};
  const uint32_t box[4] = {64, (uint32_t)pl.patch_w, (uint32_t)pl.patch_h, 1};
  if (!make_map(&ma, L, 4, da, sa, box) || !make_map(&mb, Z, 4, db, sb, box)) return XCONV_ERR_CUDA;
  TcParams p{};
  p.mode = MODE_CONTRACT;
  p.tile_n = pl.ct_tile_n;
  p.tmem_cols = pow2_cols(pl.ct_tile_n);
  p.stages = pl.ct_stages;
  p.ksteps = bk / 16;
  p.a_boxes = 2;
  p.b_boxes = (int)cdivl(pl.ct_tile_n, 64);
  p.a_box_bytes = p.b_box_bytes = (uint32_t)bk * 128;
  p.a_stage_bytes = 2 * p.a_box_bytes;
  p.b_stage_bytes = (uint32_t)p.b_boxes * p.b_box_bytes;
  p.tx_bytes = p.a_stage_bytes + p.b_stage_bytes;
  p.a_mn_major = p.b_mn_major = 1;
  p.a_lbo = p.a_box_bytes;
  p.b_lbo = p.b_box_bytes;
  p.tiles_m = pl.ct_tiles_m;
  p.tiles_n = pl.ct_tiles_n;
  p.kblocks = pl.ct_items;
  p.kblocks_per_split = pl.ct_items_per_split;
  p.patch_w = pl.patch_w;
  p.patch_h = pl.patch_h;
  p.patches_x = pl.patches_x;
  p.patches_y = pl.patches_y;
  p.pad = (d->KH - 1) / 2;
  p.rows = d->Cout;
  p.cols = d->Cin;
  p.T = T;
  p.Cin = d->Cin;
  p.part = reinterpret_cast<float*>(part);
  p.status = reinterpret_cast<unsigned int*>(ws_head);
  xconv_status s = launch(ma, mb, p, dim3((unsigned)(pl.ct_tiles_m * pl.ct_tiles_n * T), (unsigned)pl.ct_splits), st);
  if (s != XCONV_OK) return s;
  const long count = (long)d->Cout * T * d->Cin;
  reduce_contract_partials<<<(unsigned)cdivl(count, 256), 256, 0, st>>>(p.part, dW, count, pl.ct_splits,
                                                                       1.0f / (float)d->r, d->chan_scale, d->Cin);
  count_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return XCONV_ERR_CUDA; }
  return XCONV_OK;
}

}  // namespace xconv
