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
//   CONV      Y = conv(X, w)  (forward step 1, Eq. 5) and, with transposed and flipped weights, the exact
//             dX: D[pixel, co] = sum_{offset, ci} In[pixel + offset, ci] W[co, offset, ci] for one image
//             patch per work unit; both tiles K-major (channels contiguous), the reduction runs over
//             (offset, 64-channel block), and the offset again moves the TMA box of the input.
//
// Structure of a CTA (192 or 320 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 (2..9) = epilogue, one (two) per TMEM lane quadrant; two share the columns of a tile.  A ring of shared-memory stages is handed
// from producer to issuer with mbarriers; tcgen05.commit returns stages and signals the epilogue.
// Every wait is bounded: on expiry the CTA records the call's tag in the workspace header, drains
// its outstanding copies (bounded again), frees its tensor memory and returns.
#include "tc_api.h"

#include <cuda.h>
#include <cudaTypedefs.h>

#include <algorithm>

#include "common.cuh"

namespace xconv {

enum : int { MODE_SKETCH = 0, MODE_BACKPROBE = 1, MODE_CONTRACT = 2, MODE_CONV = 3 };

struct TcParams {
  int mode;
  int tile_n;              // MMA N (multiple of 16, <= 256)
  int m_sub;               // 128-row MMA tiles per work unit that share the B tile (1 or 2)
  int acc_bufs;            // accumulator sets in tensor memory (2 = epilogue overlaps the next unit)
  int tmem_cols;           // power of two >= max(32, tile_n * m_sub * acc_bufs)
  int stages;
  int ksteps;              // UMMA k-steps (of 16) per stage
  int kgroup;              // SKETCH: 64-wide k-blocks per stage (each its own K-major tile), 1 elsewhere
  uint32_t a_jump, b_jump; // kgroup > 1: descriptor start-address step (>>4) from the last k-step of a block to the next block
  uint32_t a_stage_bytes, b_stage_bytes, tx_bytes;
  int a_boxes, b_boxes;    // TMA boxes per stage: A per 128-row tile, B in all
  uint32_t a_box_bytes, b_box_bytes, a_sub_bytes;
  int a_mn_major, b_mn_major;
  uint32_t a_lbo, b_lbo;   // leading byte offsets of the UMMA descriptors
  // swizzle of the stage tiles: 128-byte rows (layout 2, 8-row groups 1024 B apart) everywhere except
  // the contraction of layers with 32-channel multiples, which uses 64-byte rows (layout 4, 512 B)
  uint32_t sbo, mn_step, layout;
  int cw_shift;            // log2 of the channels per tile block (6 or 5)
  // BACKPROBE: behind the stages every epilogue warp owns a ring of epi_slots staging slots of 4 KB (32 rows x
  // 64 positions) from which it stores L with tensor stores; epi_bytes = epilogue warps x epi_slots x 4 KB (0 elsewhere).
  // Column tiles have bp_base blocks of 64 positions, the first bp_rem tiles one more (at most 4).
  uint32_t epi_bytes;
  int epi_slots;
  long bp_base, bp_rem;
  uint32_t smem_pad;       // bytes kept free behind the last stage: a 128-row MMA reads that far past a shorter A tile
  int tiles_m, tiles_n, taps;
  // CONTRACT: kernel offsets per work unit (1, 3 or 9).  The offsets of a unit share the L tile of every
  // stage; their Z tiles lie one behind the other in the stage as consecutive column blocks, so one MMA
  // spans several offsets: columns [0, tpu * tile_n) of the accumulator, in `pieces` MMAs of whole blocks.
  // CONTRACT, one offset per unit: a k-block's tiles arrive as two halves (the upper and the lower image rows of
  // the patch), each with barriers of its own, in a ring of `stages` half-slots.  A half is released as soon
  // as the last MMA that reads it is done, so four halves cover the load latency where two whole stages
  // cannot.  `ks_h0` k-steps lie wholly in the first half, then (if the half has an odd number of 8-row
  // groups) one k-step takes its first 8 rows from the end of the first half and its last 8 from the start
  // of the second -- the descriptor's stride between 8-row groups, `sbo_x`, spans the gap -- then `ks_h1`.
  int halves, ks_h0, ks_x, ks_h1;
  uint32_t a_half_bytes, sbo_x;
  int tpu, pieces;
  uint32_t b_tap_bytes;    // bytes of one offset's Z tile
  int piece_cols[2];       // N of each MMA
  long units;              // work units = tiles x k-splits, dealt round-robin to the CTAs
  long kblocks, kblocks_per_split;
  long kb_rem;             // the first kb_rem k-splits take one k-block more than kblocks_per_split
  // SKETCH: k-split s takes the k-blocks s, s + k_weave, s + 2 k_weave, ... (k_weave = number of splits) instead
  // of a run of consecutive ones, so that the CTAs of a row tile read neighbouring pieces of the same rows at
  // the same time.  0: consecutive k-blocks.
  int k_weave;
  // contraction geometry
  int patch_w, patch_h, patches_x, patches_y, pad;
  // extents for the epilogue guards
  long rows, cols;         // valid MMA rows / columns of the whole problem
  // outputs
  float* part;             // SKETCH: [split][rows][cols]; CONTRACT: [split][Cout][T][Cin]
  bf16* L;                 // BACKPROBE: [r][Q]; CONV: output [B][H][W][Co]
  long Q;
  int T, Cin;              // CONTRACT output indexing; CONV: offsets and input channels
  int H, W, cgroups;       // CONV: image size and input-channel blocks of 64
  int nimg;                // CONV: images; with m_sub = 2 a unit covers the same patch of images img and img + 1
  // Probing vectors redrawn inside the kernel (Algorithm 1 keeps the seed, not Z): the tile of Z is not copied
  // from global memory; the epilogue warps write it into the stage from the Philox stream of the seed.
  int seeded;              // 0: Z is read from memory
  uint32_t seed_lo, seed_hi;
  int z_is_a;              // SKETCH: Z is the A operand (probes on the MMA rows) instead of the B operand
  long z_row_len;          // entries of one probing vector, H*W*Cin
  long rows_z;             // probing vectors (rows of Z)
  // Volumes: the planes (probe x depth for CONTRACT, image x depth for CONV) are the outermost tensor axis; a
  // kernel offset with a depth component dz reads plane + dz, and where that leaves the volume the box is
  // sent to row H of the plane instead, which lies outside the image: the copy engine fills it with zeros.
  // CONTRACT in halves with block-sparse probes (Eq. 7) whose all-zero 64-channel blocks the caller has named.  Row tn of
  // `zlist` (zlist_ld words apart) serves column tile tn: word 0 = number n of probing vectors with at least one non-zero
  // block in that tile, words 1..n = their indices in rising order, word n+1 = 0.  The k-blocks of a tile are those of
  // its n listed probes only, dealt evenly to the zsplits k-splits; the others are neither copied nor multiplied.
  // (A listed probe takes whole k-blocks, zero blocks included: an MMA into columns that the MMA before it wrote waits
  // some 250 clocks for it whatever its width, so narrower MMAs for the non-zero blocks alone took as long.)  Null: dense.
  const uint32_t* zlist;
  int zlist_ld, zsplits;
  int epi_groups;          // epilogue warps per tensor-memory lane quadrant (1 or 2): the launch has 64 + 128 * epi_groups threads
  int depth, pad_d;        // planes per probe or image (1: planar layer), depth padding of the kernel
  int f16;                 // storage type of the 16-bit operands: 0 = bfloat16, 1 = float16 (both operands alike)
  unsigned int* status;    // workspace header: [0] tag of a timed-out call, [1] tag of the last call
  unsigned int tag;        // tag of this call
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
// Bounded wait: about one second after a short spin.  Returns false (and records the tag) on expiry.
__device__ __noinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, unsigned int* status, unsigned int tag,
                                            unsigned long long limit_ns = 1000000000ull) {
  for (int i = 0; i < 4096; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_ns() - t0 > limit_ns) {
      atomicExch(status, tag);
      return false;
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned int* status, unsigned int tag) {
  if (mbar_try_wait(bar, parity)) return true;       // the common case costs one instruction
  return mbar_wait_slow(bar, parity, status, tag);
}

// The same operations on a 32-bit shared-memory address the caller keeps in a register.
__device__ __forceinline__ bool mbar_try_wait_a(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ void umma_commit_a(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4),
        "r"(smem_u32(bar)) : "memory");
}
// Tensor store shared -> global (bulk async-group completion) and its bookkeeping.
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all earlier bulk stores of this thread have finished READING shared memory / have completed
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
// at most `pending` (1, 3 or 7) of this thread's bulk stores may still be reading shared memory
__device__ __forceinline__ void bulk_wait_read_upto(int pending) {
  if (pending >= 7) bulk_wait_read<7>();
  else if (pending >= 3) bulk_wait_read<3>();
  else if (pending >= 1) bulk_wait_read<1>();
  else bulk_wait_read<0>();
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

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

// D[tmem] (+)= A[smem] * B[smem], 16-bit inputs (bfloat16 or float16, per the instruction descriptor), float
// accumulate; issued by one thread.  The two
// shared-memory descriptors come as 32-bit halves: only the low half (start address) changes between
// k-steps, so the issuing thread -- whose own instruction stream is the critical path of the CTA when
// the tiles are small -- spends one 32-bit add per operand and k-step.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// All MMAs of one stage, fully unrolled.  The issuing thread runs alone in its warp, so every instruction
// it executes costs a full dependent-issue slot (~6 cycles): a 128x64x16 MMA occupies the tensor pipe for
// 32 cycles, i.e. about five instructions.  KS k-steps, TWO = two 128-row tiles share the B tile.
// GROUPED: the stage holds KS/4 K-major tiles of 64 k each; after every fourth k-step the start
// addresses jump to the next tile.
template <int KS, bool TWO, bool GROUPED = false>
__device__ __forceinline__ void umma_stage(uint32_t d, uint32_t tile_n, uint32_t a_lo, uint32_t b_lo, uint32_t hi,
                                           uint32_t idesc, uint32_t acc, uint32_t a_step, uint32_t b_step,
                                           uint32_t a_sub, uint32_t a_jump = 0, uint32_t b_jump = 0) {
#pragma unroll
  for (int k = 0; k < KS; ++k) {
    umma_bf16(d, a_lo, hi, b_lo, hi, idesc, k == 0 ? acc : 1u);
    if (TWO) umma_bf16(d + tile_n, a_lo + a_sub, hi, b_lo, hi, idesc, k == 0 ? acc : 1u);
    if (GROUPED && (k & 3) == 3) { a_lo += a_jump; b_lo += b_jump; }
    else { a_lo += a_step; b_lo += b_step; }
  }
}

// The same for a CONTRACT unit with several kernel offsets: per k-step one MMA per piece of the unit's
// columns (`b_piece` = start-address step to the second piece's Z blocks) and per row tile.
template <int KS, bool TWO, bool PIECES2>
__device__ __forceinline__ void umma_stage_taps(uint32_t d, uint32_t unit_cols, uint32_t piece0_cols, uint32_t a_lo,
                                                uint32_t b_lo, uint32_t b_piece, uint32_t hi, uint32_t id0, uint32_t id1,
                                                uint32_t acc, uint32_t a_step, uint32_t b_step, uint32_t a_sub) {
#pragma unroll
  for (int k = 0; k < KS; ++k) {
    const uint32_t ac = k == 0 ? acc : 1u;
    umma_bf16(d, a_lo, hi, b_lo, hi, id0, ac);
    if (PIECES2) umma_bf16(d + piece0_cols, a_lo, hi, b_lo + b_piece, hi, id1, ac);
    if (TWO) {
      umma_bf16(d + unit_cols, a_lo + a_sub, hi, b_lo, hi, id0, ac);
      if (PIECES2) umma_bf16(d + unit_cols + piece0_cols, a_lo + a_sub, hi, b_lo + b_piece, hi, id1, ac);
    }
    a_lo += a_step;
    b_lo += b_step;
  }
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

// The 64 sign bits of entries e0 .. e0+63 of Z (e0 a multiple of 64): entry e takes bit (e mod 128) of the
// Philox block (e div 128); bit b is bit (b mod 32) of output word (b div 32).
__device__ __forceinline__ uint2 z_sign_bits64(long e0, uint32_t k0, uint32_t k1) {
  const unsigned long long blk = (unsigned long long)e0 >> 7;
  const uint4 w = philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), k0, k1);
  return (e0 & 64) ? make_uint2(w.z, w.w) : make_uint2(w.x, w.y);
}
// Eight consecutive entries as bfloat16 (+1 = 0x3F80, -1 = 0xBF80; `ones` = 0x3F803F80) or float16 (+1 = 0x3C00,
// `ones` = 0x3C003C00) from bits 0..7 of `t` (higher bits are ignored).  Two sign bits b0, b1 at positions 2i, 2i+1 go to bits 15 and 31 of a word: the product of
// (t & (3 << 2i)) with (0x40008000 >> 2i) holds b0 at bits 15 and 30 and b1 at bits 16 and 31.
__device__ __forceinline__ uint4 z_pack8(uint32_t t, uint32_t ones) {
  uint4 o;
  o.x = (((t & 0x03u) * 0x40008000u) & 0x80008000u) | ones;
  o.y = (((t & 0x0Cu) * 0x10002000u) & 0x80008000u) | ones;
  o.z = (((t & 0x30u) * 0x04000800u) & 0x80008000u) | ones;
  o.w = (((t & 0xC0u) * 0x01000200u) & 0x80008000u) | ones;
  return o;
}

// 64 entries of one row of a K-major, 128-byte-swizzled tile (row base `rbase`): eight 16-byte pieces.
__device__ __forceinline__ void z_store64(uint32_t rbase, int row, uint2 bits, uint32_t ones) {
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint4 o = z_pack8((c < 4 ? bits.x : bits.y) >> ((c & 3) * 8), ones);
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(rbase + (((uint32_t)c ^ ((uint32_t)row & 7u)) << 4)),
                 "r"(o.x), "r"(o.y), "r"(o.z), "r"(o.w) : "memory");
  }
}
// The same with every piece looked up by its eight sign bits in the table at shared-memory address `lut` (256 x 16
// bytes: z_pack8 of every byte): one load per piece instead of sixteen integer instructions.  Pays where a warp draws
// a stage alone and its instruction stream is the limit (the back-probe: 260 -> 220 us on the 256 x 256 images); where
// all warps draw together beside a copy engine and a tensor pipe that fill shared memory's bandwidth (the sketch) the
// extra loads cost more than the instructions (63 -> 76 us there).
__device__ __forceinline__ void z_store64_lut(uint32_t rbase, int row, uint2 bits, uint32_t lut) {
  const uint32_t r7 = (uint32_t)row & 7u;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint32_t word = c < 4 ? bits.x : bits.y;
    const uint32_t off = (c & 3) == 0 ? (word << 4) & 0xFF0u : (word >> ((c & 3) * 8 - 4)) & 0xFF0u;
    uint4 o;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(o.x), "=r"(o.y), "=r"(o.z), "=r"(o.w) : "r"(lut + off));
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(rbase + (((uint32_t)c ^ r7) << 4)),
                 "r"(o.x), "r"(o.y), "r"(o.z), "r"(o.w) : "memory");
  }
}
// 128 entries: the same row of two consecutive k-block tiles, `tile_bytes` apart.
__device__ __forceinline__ void z_store128(uint32_t rbase, uint32_t tile_bytes, int row, uint4 w, uint32_t ones) {
  z_store64(rbase, row, make_uint2(w.x, w.y), ones);
  z_store64(rbase + tile_bytes, row, make_uint2(w.z, w.w), ones);
}

// The MMAs of `nkb` k-blocks that arrive in two halves (see TcParams::halves), with the numbers of k-steps known at
// compile time so that the issuing thread runs straight-line code: it executes about one instruction per six
// clocks, and every instruction between two tcgen05.mma counts.  Returns false if a wait ran out.
template <int K0, int KX, int K1, bool TWO>
__device__ __forceinline__ bool umma_halves_items(int nkb, int& s, uint32_t& parity, uint32_t& acc, int slots,
                                                  uint64_t* full_bar, uint64_t* empty_bar, uint32_t base16, uint32_t slot16,
                                                  uint32_t a_lo0, uint32_t b_lo0, uint32_t a_half16, uint32_t a_sub,
                                                  uint32_t step, uint32_t sbo16, uint32_t hi, uint32_t hi_x, uint32_t idesc,
                                                  uint32_t d, uint32_t tile_n, unsigned int* status, unsigned int tag) {
  for (int i = 0; i < nkb; ++i) {
    const uint32_t h0 = base16 + (uint32_t)s * slot16, h1 = h0 + slot16;
    if (!mbar_wait(&full_bar[s], parity, status, tag)) return false;
    tc_fence_after();
    uint32_t a = a_lo0 | h0, b = b_lo0 | (h0 + a_half16);
#pragma unroll
    for (int k = 0; k < K0; ++k) {
      umma_bf16(d, a, hi, b, hi, idesc, acc);
      if (TWO) umma_bf16(d + tile_n, a + a_sub, hi, b, hi, idesc, acc);
      acc = 1u; a += step; b += step;
    }
    if (!mbar_wait(&full_bar[s + 1], parity, status, tag)) return false;
    tc_fence_after();
    if (KX) {
      umma_bf16(d, a, hi_x, b, hi_x, idesc, acc);
      if (TWO) umma_bf16(d + tile_n, a + a_sub, hi_x, b, hi_x, idesc, acc);
      acc = 1u;
    }
    umma_commit(&empty_bar[s]);
    a = (a_lo0 | h1) + (KX ? sbo16 : 0u);
    b = (b_lo0 | (h1 + a_half16)) + (KX ? sbo16 : 0u);
#pragma unroll
    for (int k = 0; k < K1; ++k) {
      umma_bf16(d, a, hi, b, hi, idesc, acc);
      if (TWO) umma_bf16(d + tile_n, a + a_sub, hi, b, hi, idesc, acc);
      acc = 1u; a += step; b += step;
    }
    umma_commit(&empty_bar[s + 1]);
    s += 2;
    if (s == slots) { s = 0; parity ^= 1u; }
  }
  return true;
}

// Two floats rounded to the 16-bit storage type, packed (first in the low half).
__device__ __forceinline__ uint32_t pack2(uint32_t a, uint32_t b, bool f16) {
  if (f16) { __half2 h = __floats2half2_rn(__uint_as_float(a), __uint_as_float(b)); return *reinterpret_cast<uint32_t*>(&h); }
  __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(a), __uint_as_float(b));
  return *reinterpret_cast<uint32_t*>(&h);
}

constexpr int TILE_M = 128;
constexpr int MAX_STAGES = 8;
constexpr int ZLIST_SMEM = 128;      // list entries of a unit held in shared memory (the rest are read from global memory)
// Epilogue warps per tensor-memory lane quadrant: one, or two where a tile's epilogue outlasts its mainloop (the
// back-probe of small batches).  More epilogue warps than needed only take issue slots from the two
// single-thread roles: with two everywhere the wide layers lost 10-25 %.
constexpr int MAX_EPI_GROUPS = 2;
constexpr int TC_THREADS = 64 + 128 * MAX_EPI_GROUPS;     // launch bound; a launch has 64 + 128 * epi_groups threads

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

struct Unit { int tm, tn, tap; long split, kb0; int nkb; int px, py, img; int blk0, nblk; };

// Work unit u -> tile, offset, k-split.  32-bit divisions throughout (a launch has far fewer than 2^31 units):
// every role of a CTA decodes each of its units on its own critical path, one instruction per ~6 clocks, and a
// 64-bit division is a 100-instruction routine -- with one-stage tiles the decode alone was half the time per tile.
__device__ __forceinline__ Unit decode_unit(const TcParams& p, long u_) {
  Unit w;
  const uint32_t u = (uint32_t)u_;
  w.px = w.py = w.img = 0;
  w.blk0 = w.nblk = 0;
  if (p.mode == MODE_CONV) {                 // channel tiles innermost, then patches of one image
    uint32_t q = u;
    const uint32_t tn = (uint32_t)p.tiles_n, px = (uint32_t)p.patches_x, py = (uint32_t)p.patches_y;
    w.tn = (int)(q % tn); q /= tn;
    w.px = (int)(q % px); q /= px;
    w.py = (int)(q % py); q /= py;
    w.img = (int)q * p.m_sub;
    w.tm = 0; w.tap = 0; w.split = 0;
  } else if (p.mode == MODE_BACKPROBE) {     // probe tiles innermost: the dY tile is re-read while hot in L2
    const uint32_t tm = (uint32_t)p.tiles_m;
    w.tm = tm == 1 ? 0 : (int)(u % tm);
    w.tn = tm == 1 ? (int)u : (int)(u / tm);
    w.tap = 0;
    w.split = 0;
    // column tile tn covers blocks [blk0, blk0 + nblk) of 64 positions
    w.blk0 = w.tn * (int)p.bp_base + min(w.tn, (int)p.bp_rem);
    w.nblk = (int)p.bp_base + (w.tn < (int)p.bp_rem ? 1 : 0);
  } else {                                   // tiles of one k-split are adjacent: they share operands in L2
    const int tpu = p.mode == MODE_CONTRACT ? p.tpu : 1;
    const uint32_t tiles = (uint32_t)((p.taps / tpu) * p.tiles_m * p.tiles_n);
    uint32_t t = u % tiles;
    w.split = u / tiles;
    w.tn = (int)(t % (uint32_t)p.tiles_n); t /= (uint32_t)p.tiles_n;
    w.tm = (int)(t % (uint32_t)p.tiles_m); t /= (uint32_t)p.tiles_m;
    w.tap = (int)t * tpu;                      // first offset of the unit
  }
  if (p.zlist != nullptr) {                  // k-blocks of the listed probes only, dealt evenly to the k-splits
    const uint32_t n = p.zlist[(uint32_t)w.tn * (uint32_t)p.zlist_ld];
    const uint32_t K = n * (uint32_t)(p.patches_x * p.patches_y * p.depth), zs = (uint32_t)p.zsplits;
    const uint32_t q = K / zs, rem = K % zs, sp = (uint32_t)w.split;
    w.kb0 = (long)(sp * q + min(sp, rem));
    w.nkb = (int)(q + (sp < rem ? 1u : 0u));
    return w;
  }
  w.kb0 = w.split * p.kblocks_per_split + min(w.split, p.kb_rem);
  const long kb1 = min(p.kblocks, w.kb0 + p.kblocks_per_split + (w.split < p.kb_rem ? 1 : 0));
  w.nkb = (int)max(0L, kb1 - w.kb0);
  return w;
}

// ------------------------------------------------------------------------------------ the kernel

// F16: the 16-bit storage type is float16 instead of bfloat16 (a compile-time constant, so that the epilogues'
// conversions carry no selection between the two).
template <bool F16>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_c, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t tmem_full_bar[2];
  __shared__ __align__(8) uint64_t tmem_empty_bar[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int go;
  __shared__ uint32_t zl[ZLIST_SMEM];        // block-sparse probes: the list entries of this CTA's one work unit

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;          // 128B swizzle wants 1024B alignment
  const uint32_t stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  const int unit_cols = p.mode == MODE_CONTRACT ? p.tile_n * p.tpu : p.tile_n;  // columns of one row tile's accumulator
  const int acc_cols = unit_cols * p.m_sub;                                   // columns of one accumulator set

  // Seeded calls: the epilogue warps redraw the tiles of Z, all of them together stage by stage -- except in a
  // back-probe with one tile of at most 96 rows: there the warps of the lane quadrants that hold rows (below
  // gen_quad0) are busy with the epilogue of every unit, the slowest role of that kernel, and the warps of the
  // other quadrants, which have nothing to store, do nothing but draw, each whole stages by itself in turn.
  const int gen_quad0 = (p.seeded && p.mode == MODE_BACKPROBE && p.tiles_m == 1 && p.m_sub == 1 && p.rows <= 96)
                            ? (int)((p.rows + 31) / 32) : 0;
  // preamble: touches no global memory, so it may overlap the tail of the previous kernel
  if (threadIdx.x == 0) {
    // a stage is full when the producer's copies have landed and (seeded) the drawing warps have arrived: all epilogue
    // warps, or the one drawing warp whose turn the stage is; an accumulator set is free when the storing warps are done
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&full_bar[s], !p.seeded ? 1 : gen_quad0 > 0 ? 2 : 1 + 4 * p.epi_groups);
      mbar_init(&empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&tmem_full_bar[b], 1);
      mbar_init(&tmem_empty_bar[b], (gen_quad0 > 0 ? gen_quad0 : 4) * p.epi_groups);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    prefetch_tmap(&map_a);
    prefetch_tmap(&map_b);
    if (p.mode == MODE_BACKPROBE) prefetch_tmap(&map_c);
  }
  // seeded back-probe: the table of sign patterns behind everything else in shared memory
  const uint32_t z_lut = tiles_base + (uint32_t)p.stages * stage_bytes + p.epi_bytes + p.smem_pad;
  if (p.seeded && p.mode == MODE_BACKPROBE)
    for (uint32_t i = threadIdx.x; i < 256u; i += blockDim.x) {
      const uint4 o = z_pack8(i, F16 ? 0x3C003C00u : 0x3F803F80u);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(z_lut + (i << 4)), "r"(o.x), "r"(o.y), "r"(o.z), "r"(o.w) : "memory");
    }
  if (warp == 1) tmem_alloc(&tmem_slot, (uint32_t)p.tmem_cols);
  pdl_trigger();
  pdl_wait();                              // from here on the previous kernel's results are visible
  // Block-sparse probes (one unit per CTA): the unit's stretch of its tile's list, zl_len entries (and the entry behind
  // the last, which the producer may fetch but never uses), goes to shared memory.
  const uint32_t* zl_row = nullptr;
  int zl_len = 0;
  if (p.zlist != nullptr) {
    const Unit w0 = decode_unit(p, blockIdx.x);
    const uint32_t per_probe = (uint32_t)(p.patches_x * p.patches_y * p.depth);
    const uint32_t first = (uint32_t)w0.kb0 / per_probe;
    zl_len = w0.nkb > 0 ? (int)(((uint32_t)w0.kb0 + (uint32_t)w0.nkb - 1u) / per_probe - first) + 1 : 0;
    zl_row = p.zlist + (size_t)w0.tn * p.zlist_ld + 1 + first;
    for (int i = threadIdx.x; i <= zl_len && i < ZLIST_SMEM; i += blockDim.x) zl[i] = zl_row[i];
  }
  auto zent = [&](int i) -> uint32_t { return i < ZLIST_SMEM ? zl[i] : zl_row[i]; };
  if (threadIdx.x == 0) {
    // a CTA of this call gave up earlier: skip the work (one thread reads so that the whole CTA agrees)
    go = (*reinterpret_cast<volatile unsigned int*>(p.status) != p.tag) ? 1 : 0;
    if (blockIdx.x == 0) reinterpret_cast<volatile unsigned int*>(p.status)[1] = p.tag;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);

  if (!go) {
    // fall through to the teardown
  } else if (warp == 0 && p.mode == MODE_CONTRACT && p.tpu > 1) {
    // ------------------------------------------------------------------ TMA producer, several offsets per unit
    // A 5-d tensor copy costs its issuing thread some 150-200 cycles, and a stage takes one per offset
    // plus one: lane 0 waits for the stage, arms its barrier and fetches the L tile, lanes 1..tpu
    // fetch the Z tile of one offset each, all at once.  Every lane walks the same loop.
    const int stages = p.stages;
    const int ks = 2 * p.pad + 1;
    int s = 0;
    long fill = 0, it = 0;
    bool ok = true;
    for (long u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
      const Unit w = decode_unit(p, u);
      const int row0 = w.tm * p.m_sub * TILE_M;
      const int col0 = w.tn * p.tile_n;
      uint32_t q = (uint32_t)w.kb0;
      int px = (int)(q % (uint32_t)p.patches_x); q /= (uint32_t)p.patches_x;
      int py = (int)(q % (uint32_t)p.patches_y); q /= (uint32_t)p.patches_y;
      int pj = (int)q;
      const int tap = w.tap + max(0, min(lane - 1, p.tpu - 1));          // this lane's offset
      const int dy = tap / ks - p.pad, dx = tap % ks - p.pad;
      for (int i = 0; i < w.nkb; ++i) {
        if (fill > 0) {
          if (lane == 0) ok = mbar_wait(&empty_bar[s], (uint32_t)((fill - 1) & 1), p.status, p.tag);
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) break;
        }
        const uint32_t a_dst = tiles_base + (uint32_t)s * stage_bytes;
        const uint32_t b_dst = a_dst + p.a_stage_bytes;
        const int x0 = px * p.patch_w, y0 = py * p.patch_h;
        if (lane == 0) {
          mbar_arrive_expect_tx(&full_bar[s], p.tx_bytes);
          tma_load_5d(a_dst, &map_a, 0, x0, y0, row0 >> p.cw_shift, pj, &full_bar[s]);
        }
        __syncwarp();                                 // the barrier is armed before any Z tile can land
        if (lane >= 1 && lane <= p.tpu)
          tma_load_5d(b_dst + (uint32_t)(lane - 1) * p.b_tap_bytes, &map_b, 0, x0 + dx, y0 + dy, col0 >> p.cw_shift, pj,
                      &full_bar[s]);
        if (++px == p.patches_x) { px = 0; if (++py == p.patches_y) { py = 0; ++pj; } }
        ++it;
        if (++s == stages) { s = 0; ++fill; }
      }
    }
    // drain: every copy issued must have landed in this CTA's shared memory before it exits
    if (lane == 0)
      for (long i = max(0L, it - stages); i < it; ++i)
        if (!mbar_wait(&full_bar[i % stages], (uint32_t)((i / stages) & 1), p.status, p.tag)) break;
  } else if (warp == 0 && p.mode == MODE_CONTRACT && p.halves) {
    // ------------------------------------------------------------------ TMA producer, k-blocks in two halves
    if (lane == 0) {
      const int slots = p.stages;          // half-slots
      int s = 0;
      long fill = 0, it = 0;
      bool ok = true;
      const int hrows = p.patch_h >> 1;    // image rows per half
      for (long u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
        const Unit w = decode_unit(p, u);
        const int row0 = w.tm * p.m_sub * TILE_M, col0 = w.tn * p.tile_n;
        uint32_t q = (uint32_t)w.kb0;
        int px = (int)(q % (uint32_t)p.patches_x); q /= (uint32_t)p.patches_x;
        int py = (int)(q % (uint32_t)p.patches_y); q /= (uint32_t)p.patches_y;
        int pj = (int)q;
        const int ks = 2 * p.pad + 1, tp = w.tap % (ks * ks), dy = tp / ks - p.pad, dx = tp % ks - p.pad;
        const int dz = w.tap / (ks * ks) - p.pad_d;
        int pz = pj % p.depth;               // depth of plane pj inside its volume
        if (p.zlist != nullptr) {
          // block-sparse probes: pj counted the planes of the listed probes; the plane in memory is that of the probe
          // the list entry names
          int li = 0;
          int plane = (int)zent(0) * p.depth + pz;
          for (int i = 0; i < 2 * w.nkb; ++i) {
            if (fill > 0) {
              ok = mbar_wait(&empty_bar[s], (uint32_t)((fill - 1) & 1), p.status, p.tag);
              if (!ok) break;
            }
            const uint32_t a_dst = tiles_base + (uint32_t)s * stage_bytes, b_dst = a_dst + p.a_half_bytes;
            const int x0 = px * p.patch_w, y0 = py * p.patch_h + (i & 1) * hrows;
            mbar_arrive_expect_tx(&full_bar[s], stage_bytes);
            tma_load_5d(a_dst, &map_a, 0, x0, y0, row0 >> p.cw_shift, plane, &full_bar[s]);
            const bool inside = (unsigned)(pz + dz) < (unsigned)p.depth;
            tma_load_5d(b_dst, &map_b, 0, x0 + dx, inside ? y0 + dy : p.H, col0 >> p.cw_shift, plane + dz, &full_bar[s]);
            ++it;
            if (++s == slots) { s = 0; ++fill; }
            if ((i & 1) && ++px == p.patches_x) {
              px = 0;
              if (++py == p.patches_y) {
                py = 0;
                if (++pz == p.depth) { pz = 0; ++li; }
                plane = (int)zent(li) * p.depth + pz;
              }
            }
          }
        } else
        for (int i = 0; i < 2 * w.nkb; ++i) {
          if (fill > 0) {
            ok = mbar_wait(&empty_bar[s], (uint32_t)((fill - 1) & 1), p.status, p.tag);
            if (!ok) break;
          }
          const uint32_t a_dst = tiles_base + (uint32_t)s * stage_bytes, b_dst = a_dst + p.a_half_bytes;
          const int x0 = px * p.patch_w, y0 = py * p.patch_h + (i & 1) * hrows;
          mbar_arrive_expect_tx(&full_bar[s], stage_bytes);
          tma_load_5d(a_dst, &map_a, 0, x0, y0, row0 >> p.cw_shift, pj, &full_bar[s]);
          const bool inside = (unsigned)(pz + dz) < (unsigned)p.depth;
          tma_load_5d(b_dst, &map_b, 0, x0 + dx, inside ? y0 + dy : p.H, col0 >> p.cw_shift, pj + dz, &full_bar[s]);
          if ((i & 1) && ++px == p.patches_x) {
            px = 0;
            if (++py == p.patches_y) { py = 0; ++pj; if (++pz == p.depth) pz = 0; }
          }
          ++it;
          if (++s == slots) { s = 0; ++fill; }
        }
      }
      for (long i = max(0L, it - slots); i < it; ++i)
        if (!mbar_wait(&full_bar[i % slots], (uint32_t)((i / slots) & 1), p.status, p.tag)) break;
    }
  } else if (warp == 1 && p.mode == MODE_CONTRACT && p.halves) {
    // ------------------------------------------------------------------ MMA issuer, k-blocks in two halves
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (F16 ? 0u : (1u << 7) | (1u << 10)) | (1u << 15) | (1u << 16) |
                             ((uint32_t)(p.tile_n >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
      const uint32_t step = p.mn_step >> 4;                                   // 16 rows
      const uint32_t a_lo0 = (p.a_lbo >> 4) << 16, b_lo0 = (p.b_lbo >> 4) << 16;
      const uint32_t hi = (p.sbo >> 4) | (1u << 14) | (p.layout << 29);
      const uint32_t hi_x = (p.sbo_x >> 4) | (1u << 14) | (p.layout << 29);    // the k-step across the two halves
      const uint32_t a_sub = p.a_sub_bytes >> 4, a_half16 = p.a_half_bytes >> 4, slot16 = stage_bytes >> 4;
      const uint32_t base16 = (tiles_base & 0x3FFFFu) >> 4;
      const bool two = p.m_sub == 2;
      const uint32_t tile_n = (uint32_t)p.tile_n;
      int s = 0;                           // half-slot of the next first half (always even)
      uint32_t parity = 0;
      bool ok = true;
      for (long u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
        const Unit w = decode_unit(p, u);
        if (w.nkb == 0) { mbar_arrive(&tmem_full_bar[0]); continue; }      // nothing to multiply: the epilogue stores zeros
        const uint32_t d = tmem_base;      // one unit per CTA and accumulator set (acc_bufs = 1)
        uint32_t acc = 0;
        if (p.ks_h0 == 3 && p.ks_x == 1 && p.ks_h1 == 3) {      // halves of 56 pixels (28-wide images): unrolled
          ok = two ? umma_halves_items<3, 1, 3, true>(w.nkb, s, parity, acc, p.stages, full_bar, empty_bar, base16, slot16,
                                                       a_lo0, b_lo0, a_half16, a_sub, step, p.sbo >> 4, hi, hi_x, idesc, d,
                                                       tile_n, p.status, p.tag)
                   : umma_halves_items<3, 1, 3, false>(w.nkb, s, parity, acc, p.stages, full_bar, empty_bar, base16, slot16,
                                                        a_lo0, b_lo0, a_half16, a_sub, step, p.sbo >> 4, hi, hi_x, idesc, d,
                                                        tile_n, p.status, p.tag);
          if (ok) umma_commit(&tmem_full_bar[0]);
          continue;
        }
        for (int i = 0; i < w.nkb; ++i) {
          const uint32_t h0 = base16 + (uint32_t)s * slot16, h1 = h0 + slot16;
          ok = mbar_wait(&full_bar[s], parity, p.status, p.tag);
          if (!ok) break;
          tc_fence_after();
          uint32_t a = a_lo0 | h0, b = b_lo0 | (h0 + a_half16);
          for (int k = 0; k < p.ks_h0; ++k) {
            umma_bf16(d, a, hi, b, hi, idesc, acc);
            if (two) umma_bf16(d + tile_n, a + a_sub, hi, b, hi, idesc, acc);
            acc = 1u; a += step; b += step;
          }
          ok = mbar_wait(&full_bar[s + 1], parity, p.status, p.tag);
          if (!ok) break;
          tc_fence_after();
          if (p.ks_x) {                     // rows [16 ks_h0, +8) of the first half and [0, 8) of the second
            umma_bf16(d, a, hi_x, b, hi_x, idesc, acc);
            if (two) umma_bf16(d + tile_n, a + a_sub, hi_x, b, hi_x, idesc, acc);
            acc = 1u;
          }
          umma_commit(&empty_bar[s]);       // the first half may be refilled
          a = (a_lo0 | h1) + (p.ks_x ? (p.sbo >> 4) : 0u);
          b = (b_lo0 | (h1 + a_half16)) + (p.ks_x ? (p.sbo >> 4) : 0u);
          for (int k = 0; k < p.ks_h1; ++k) {
            umma_bf16(d, a, hi, b, hi, idesc, acc);
            if (two) umma_bf16(d + tile_n, a + a_sub, hi, b, hi, idesc, acc);
            acc = 1u; a += step; b += step;
          }
          umma_commit(&empty_bar[s + 1]);
          s += 2;
          if (s == p.stages) { s = 0; parity ^= 1u; }
        }
        if (ok) umma_commit(&tmem_full_bar[0]);
      }
    }
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // One thread; its loop is kept free of divisions (coordinates advance incrementally).
    if (lane == 0) {
      const int stages = p.stages;
      int s = 0;                           // stage to fill next
      long fill = 0;                       // how often the ring has wrapped
      long it = 0;                         // stages filled so far, across units
      bool ok = true;
      for (long u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
        const Unit w = decode_unit(p, u);
        const int row0 = w.tm * p.m_sub * TILE_M;
        const int col0 = w.tn * p.tile_n;
        // running coordinates of the k-block
        int kc = 0, px = 0, py = 0, pj = 0, dx = 0, dy = 0, dz = 0, pz = 0;
        if (p.mode == MODE_SKETCH) kc = (int)((p.k_weave ? w.split : w.kb0) * 64 * p.kgroup);
        else if (p.mode == MODE_BACKPROBE) kc = (int)w.kb0 * p.ksteps * 16;
        else if (p.mode == MODE_CONV) {      // pj counts channel blocks, kc = offset * Cin; w.img is a plane
          dx = dy = -p.pad;
          dz = -p.pad_d;
          pz = w.img % p.depth;
        } else {
          uint32_t q = (uint32_t)w.kb0;
          px = (int)(q % (uint32_t)p.patches_x); q /= (uint32_t)p.patches_x;
          py = (int)(q % (uint32_t)p.patches_y); q /= (uint32_t)p.patches_y;
          pj = (int)q;
          pz = pj % p.depth;
          const int ks = 2 * p.pad + 1, tp = w.tap % (ks * ks);
          dz = w.tap / (ks * ks) - p.pad_d;
          dy = tp / ks - p.pad;
          dx = tp % ks - p.pad;
        }
        for (int i = 0; i < w.nkb; ++i) {
          if (fill > 0) {
            ok = mbar_wait(&empty_bar[s], (uint32_t)((fill - 1) & 1), p.status, p.tag);
            if (!ok) break;
          }
          const uint32_t a_dst = tiles_base + (uint32_t)s * stage_bytes;
          const uint32_t b_dst = a_dst + p.a_stage_bytes;
          mbar_arrive_expect_tx(&full_bar[s], p.mode == MODE_BACKPROBE
                                                  ? p.a_stage_bytes + (p.seeded ? 0u : (uint32_t)w.nblk * p.b_box_bytes)
                                                  : p.tx_bytes);
          if (p.mode == MODE_SKETCH) {
            // one box per operand: 128*m_sub rows of A, tile_n rows of B, 64 k each
            const bool get_a = !(p.seeded && p.z_is_a), get_b = !(p.seeded && !p.z_is_a);
            if (p.kgroup > 1) {
              // kgroup consecutive k-blocks per operand in one 3-d box (64 k, rows, k-blocks)
              if (get_a) tma_load_3d(a_dst, &map_a, 0, row0, kc >> 6, &full_bar[s]);
              if (get_b) tma_load_3d(b_dst, &map_b, 0, col0, kc >> 6, &full_bar[s]);
              kc += 64 * p.kgroup * (p.k_weave ? p.k_weave : 1);
            } else {
              if (get_a) tma_load_2d(a_dst, &map_a, kc, row0, &full_bar[s]);
              if (get_b) tma_load_2d(b_dst, &map_b, kc, col0, &full_bar[s]);
              kc += 64 * (p.k_weave ? p.k_weave : 1);
            }
          } else if (p.mode == MODE_BACKPROBE) {
            tma_load_2d(a_dst, &map_a, kc, row0, &full_bar[s]);
            // dY tile: one box (64 positions x k rows) per block of the column tile, one behind the other
            // (seeded: the streamed operand is Z, and the epilogue warps write its tile themselves)
            if (!p.seeded)
              for (int b = 0; b < w.nblk; ++b)
                tma_load_3d(b_dst + (uint32_t)b * p.b_box_bytes, &map_b, 0, kc, w.blk0 + b, &full_bar[s]);
            kc += p.ksteps * 16;
          } else if (p.mode == MODE_CONV) {
            // input patch moved by the kernel offset (zero fill outside the image) and the matching
            // [tile_n output channels x 64 input channels] block of the weights
            const bool inside = (unsigned)(pz + dz) < (unsigned)p.depth;
            tma_load_5d(a_dst, &map_a, 0, w.px * p.patch_w + dx, inside ? w.py * p.patch_h + dy : p.H, pj, w.img + dz,
                        &full_bar[s]);
            tma_load_2d(b_dst, &map_b, kc + (pj << p.cw_shift), col0, &full_bar[s]);
            if (++pj == p.cgroups) {
              pj = 0; kc += p.Cin;
              if (++dx > p.pad) { dx = -p.pad; if (++dy > p.pad) { dy = -p.pad; ++dz; } }
            }
          } else {
            // one 5-d box per operand: (64 channels, patch x, patch y, channel groups of 64, probe)
            const int x0 = px * p.patch_w, y0 = py * p.patch_h;
            tma_load_5d(a_dst, &map_a, 0, x0, y0, row0 >> p.cw_shift, pj, &full_bar[s]);
            const bool inside = (unsigned)(pz + dz) < (unsigned)p.depth;
            tma_load_5d(b_dst, &map_b, 0, x0 + dx, inside ? y0 + dy : p.H, col0 >> p.cw_shift, pj + dz, &full_bar[s]);
            if (++px == p.patches_x) { px = 0; if (++py == p.patches_y) { py = 0; ++pj; if (++pz == p.depth) pz = 0; } }
          }
          ++it;
          if (++s == stages) { s = 0; ++fill; }
        }
      }
      // drain: every copy issued must have landed in this CTA's shared memory before it exits
      // (immediate on the normal path, bounded on the failure path)
      for (long i = max(0L, it - stages); i < it; ++i)
        if (!mbar_wait(&full_bar[i % stages], (uint32_t)((i / stages) & 1), p.status, p.tag)) break;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // One thread.  With small tiles the time between two tcgen05.mma is set by this thread's own
    // instruction stream, so the loop carries descriptors as 32-bit halves and does no division.
    if (lane == 0) {
      // instruction descriptor: float accumulator (bit 4), A and B formats (bits 7-9, 10-12: 0 = float16, 1 = bfloat16,
      // always the same for both), operand majorness (bits 15, 16), N >> 3 (bits 17-22), M >> 4 (bits 24-28)
      const uint32_t idesc = (1u << 4) | (F16 ? 0u : (1u << 7) | (1u << 10)) | ((uint32_t)p.a_mn_major << 15) |
                             ((uint32_t)p.b_mn_major << 16) | ((uint32_t)(p.tile_n >> 3) << 17) |
                             ((uint32_t)(TILE_M >> 4) << 24);
      // Shared-memory descriptor (128-byte swizzle): start address >> 4 | (lbo >> 4) << 16 in the low
      // word; (sbo >> 4) | version 1 << 14 | layout (2 = SWIZZLE_128B, 4 = SWIZZLE_64B) << 29 in the high word.
      // K-major: 8-row groups `sbo` = 1024 B apart, k-step = 32 B inside the swizzled row.
      // MN-major: 8-row (k) groups `sbo` apart, column blocks `lbo` apart, k-step = 16 rows = `mn_step` bytes.
      const uint32_t a_step = (p.a_mn_major ? p.mn_step : 32u) >> 4, b_step = (p.b_mn_major ? p.mn_step : 32u) >> 4;
      const uint32_t a_lo0 = ((p.a_mn_major ? p.a_lbo : 16u) >> 4) << 16;
      const uint32_t b_lo0 = ((p.b_mn_major ? p.b_lbo : 16u) >> 4) << 16;
      const uint32_t desc_hi = (p.sbo >> 4) | (1u << 14) | (p.layout << 29);
      const uint32_t a_sub = p.a_sub_bytes >> 4;
      const uint32_t a_stage16 = p.a_stage_bytes >> 4, stage16 = stage_bytes >> 4;
      const uint32_t base16 = (tiles_base & 0x3FFFFu) >> 4;
      const int ksteps = p.ksteps, stages = p.stages;
      const bool two = p.m_sub == 2;
      const uint32_t tile_n = (uint32_t)p.tile_n;
      int s = 0;
      uint32_t full_parity = 0, s16 = base16;
      const uint32_t full_a0 = smem_u32(&full_bar[0]), empty_a0 = smem_u32(&empty_bar[0]);
      uint32_t full_a = full_a0, empty_a = empty_a0;
      long lu = 0;
      bool ok = true;
      for (long u = blockIdx.x; u < p.units && ok; u += gridDim.x, ++lu) {
        const Unit w = decode_unit(p, u);
        const int buf = p.acc_bufs == 2 ? (int)(lu & 1) : 0;          // (no division: this thread's stream is the critical path)
        const long use = p.acc_bufs == 2 ? lu >> 1 : lu;
        if (use > 0) {                      // the epilogue must have emptied this accumulator set
          ok = mbar_wait(&tmem_empty_bar[buf], (uint32_t)((use - 1) & 1), p.status, p.tag);
          if (!ok) break;
          tc_fence_after();
        }
        // Nothing to multiply: the barriers still take their turn, so that their phases keep counting units, and the
        // epilogue stores zeros without reading the accumulator.
        if (w.nkb == 0) { mbar_arrive(&tmem_full_bar[buf]); continue; }
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * acc_cols);
        uint32_t acc = 0;
        // BACKPROBE: the MMA spans the blocks this column tile has
        const uint32_t idesc_u = p.mode == MODE_BACKPROBE
                                     ? (idesc & ~(0x3Fu << 17)) | ((uint32_t)(w.nblk * 8) << 17) : idesc;
        for (int i = 0; i < w.nkb; ++i) {
          if (!mbar_try_wait_a(full_a, full_parity)) ok = mbar_wait_slow(&full_bar[s], full_parity, p.status, p.tag);
          if (!ok) break;
          tc_fence_after();
          uint32_t a_lo = a_lo0 | s16;
          uint32_t b_lo = b_lo0 | (s16 + a_stage16);
#define XC_STAGE(KS, TWO) umma_stage<KS, TWO>(d_tmem, tile_n, a_lo, b_lo, desc_hi, idesc_u, acc, a_step, b_step, a_sub)
#define XC_GROUP(KS, TWO) umma_stage<KS, TWO, true>(d_tmem, tile_n, a_lo, b_lo, desc_hi, idesc, acc, a_step, b_step, \
                                                    a_sub, p.a_jump, p.b_jump)
          if (p.mode == MODE_CONTRACT && p.tpu > 1) {
            // several offsets per unit: per k-step one MMA per piece (and row tile), each spanning whole
            // column blocks of consecutive offsets
            const uint32_t b_piece = (uint32_t)(p.piece_cols[0] >> p.cw_shift) * (p.b_lbo >> 4);
            const uint32_t id0 = (idesc & ~(0x3Fu << 17)) | ((uint32_t)(p.piece_cols[0] >> 3) << 17);
            const uint32_t id1 = (idesc & ~(0x3Fu << 17)) | ((uint32_t)(p.piece_cols[1] >> 3) << 17);
#define XC_TAPS(KS, TWO, P2) umma_stage_taps<KS, TWO, P2>(d_tmem, (uint32_t)unit_cols, (uint32_t)p.piece_cols[0], a_lo, \
                                                         b_lo, b_piece, desc_hi, id0, id1, acc, a_step, b_step, a_sub)
            const int shape = (two ? 2 : 0) | (p.pieces > 1 ? 1 : 0);
            if (ksteps == 7 && shape == 0) XC_TAPS(7, false, false);
            else if (ksteps == 7 && shape == 1) XC_TAPS(7, false, true);
            else if (ksteps == 7 && shape == 2) XC_TAPS(7, true, false);
            else if (ksteps == 7 && shape == 3) XC_TAPS(7, true, true);
            else if (ksteps == 8 && shape == 0) XC_TAPS(8, false, false);
            else if (ksteps == 8 && shape == 1) XC_TAPS(8, false, true);
            else if (ksteps == 8 && shape == 2) XC_TAPS(8, true, false);
            else if (ksteps == 8 && shape == 3) XC_TAPS(8, true, true);
            else
              for (int k = 0; k < ksteps; ++k) {
                if (shape == 0) XC_TAPS(1, false, false);
                else if (shape == 1) XC_TAPS(1, false, true);
                else if (shape == 2) XC_TAPS(1, true, false);
                else XC_TAPS(1, true, true);
                acc = 1u; a_lo += a_step; b_lo += b_step;
              }
#undef XC_TAPS
          } else if (p.kgroup > 1) {
            if (two) { if (ksteps == 8) XC_GROUP(8, true); else XC_GROUP(16, true); }
            else { if (ksteps == 8) XC_GROUP(8, false); else XC_GROUP(16, false); }
          } else if (two) {
            switch (ksteps) {
              case 4: XC_STAGE(4, true); break;
              case 7: XC_STAGE(7, true); break;
              case 8: XC_STAGE(8, true); break;
              default:
                for (int k = 0; k < ksteps; ++k) {
                  XC_STAGE(1, true);
                  acc = 1u; a_lo += a_step; b_lo += b_step;
                }
            }
          } else {
            switch (ksteps) {
              case 1: XC_STAGE(1, false); break;
              case 4: XC_STAGE(4, false); break;
              case 7: XC_STAGE(7, false); break;
              case 8: XC_STAGE(8, false); break;
              default:
                for (int k = 0; k < ksteps; ++k) {
                  XC_STAGE(1, false);
                  acc = 1u; a_lo += a_step; b_lo += b_step;
                }
            }
          }
#undef XC_STAGE
#undef XC_GROUP
          acc = 1u;
          umma_commit_a(empty_a);            // stage s may be refilled once these MMAs have read it
          s16 += stage16; full_a += 8; empty_a += 8;
          if (++s == stages) { s = 0; s16 = base16; full_a = full_a0; empty_a = empty_a0; full_parity ^= 1u; }
        }
        if (ok) umma_commit(&tmem_full_bar[buf]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..)
    // A warp reads the 32 tensor-memory lanes of its quadrant (warp index mod 4); the epi_groups warps of a
    // quadrant deal the column chunks (back-probe: the 64-position blocks) of a tile among themselves.
    const int quad = warp & 3;                  // TMEM lanes [32*quad, 32*quad+32)
    const int eg = (warp - 2) >> 2;             // which of the quadrant's warps
    const uint32_t epi_base = tiles_base + (uint32_t)p.stages * stage_bytes;
    uint32_t epi_slot = 0;                    // BACKPROBE: next staging slot of this warp's ring
    int gen_s = 0;                            // seeded: stage the generator fills next, and how often the ring wrapped
    long gen_fill = 0;
    long lu = 0;
    bool ok = true;
    // BACKPROBE with Z as the streamed operand: the Z tile of one stage (probes kc .., the blocks of unit w), items
    // t0, t0 + stride, ... of it.  An item is one Philox block = 128 entries = one row of an even 64-position block and
    // of the odd block behind it; two items per round, so that their dependent chains interleave.
    auto fill_bp_stage = [&](uint32_t zbase, long kc, const Unit& w, int t0, int stride) {
            const int rows_k = p.ksteps * 16;
      if ((p.z_row_len & 127) != 0) {
        // rows of Z that start in the middle of a Philox block (their length is an odd multiple of 64): a row's even
        // blocks are not the first halves of Philox blocks in every row, so each (row, block) takes its own half
        for (int i = t0; i < rows_k * w.nblk; i += stride) {
          const int row = i % rows_k, b = i / rows_k;
          const uint2 bits = z_sign_bits64((kc + row) * p.z_row_len + (long)(w.blk0 + b) * 64, p.seed_lo, p.seed_hi);
          z_store64_lut(zbase + (uint32_t)b * p.b_box_bytes + (uint32_t)row * 128u, row, bits, z_lut);
        }
        return;
      }
      const int even0 = w.blk0 & ~1, n = rows_k * ((w.blk0 + w.nblk - even0 + 1) >> 1);
      for (int i0 = t0; i0 < n; i0 += 2 * stride) {
        const int i1 = i0 + stride;
        const bool two = i1 < n;
        const int row0_ = i0 % rows_k, blk0_ = even0 + 2 * (i0 / rows_k);
        const int row1_ = two ? i1 % rows_k : row0_, blk1_ = two ? even0 + 2 * (i1 / rows_k) : blk0_;
        const unsigned long long e0 = (unsigned long long)((kc + row0_) * p.z_row_len + (long)blk0_ * 64);
        const unsigned long long e1 = (unsigned long long)((kc + row1_) * p.z_row_len + (long)blk1_ * 64);
        const uint4 o0 = philox4x32_10((uint32_t)(e0 >> 7), (uint32_t)(e0 >> 39), p.seed_lo, p.seed_hi);
        const uint4 o1 = philox4x32_10((uint32_t)(e1 >> 7), (uint32_t)(e1 >> 39), p.seed_lo, p.seed_hi);
        const int b0 = blk0_ - w.blk0, b1 = blk1_ - w.blk0;       // block of the tile that takes the first 64 entries
        const uint32_t r0 = zbase + (uint32_t)row0_ * 128u, r1 = zbase + (uint32_t)row1_ * 128u;
        if (b0 >= 0) z_store64_lut(r0 + (uint32_t)b0 * p.b_box_bytes, row0_, make_uint2(o0.x, o0.y), z_lut);
        if (b0 + 1 < w.nblk) z_store64_lut(r0 + (uint32_t)(b0 + 1) * p.b_box_bytes, row0_, make_uint2(o0.z, o0.w), z_lut);
        if (two && b1 >= 0) z_store64_lut(r1 + (uint32_t)b1 * p.b_box_bytes, row1_, make_uint2(o1.x, o1.y), z_lut);
        if (two && b1 + 1 < w.nblk) z_store64_lut(r1 + (uint32_t)(b1 + 1) * p.b_box_bytes, row1_, make_uint2(o1.z, o1.w), z_lut);
      }
    };
    // Probing vectors redrawn from the seed: the tiles of Z of one work unit, written by these warps.
    auto redraw_unit = [&](const Unit& w) {
      if (p.mode == MODE_SKETCH) {
        // Redraw this unit's tiles of Z, stage by stage, in step with the producer (same ring, same parity):
        // wait until the MMAs have released the stage, write the signs in the K-major swizzled layout the
        // copy would have produced, hand the stage over with one arrival per warp.
        const int gtid = (int)threadIdx.x - 64;                       // 0 .. GEN-1
        const int GEN = 128 * p.epi_groups;
        const int tile_rows = p.z_is_a ? (int)(p.a_stage_bytes / (128u * p.kgroup)) : p.tile_n;
        const long first = p.z_is_a ? (long)w.tm * p.m_sub * TILE_M : (long)w.tn * p.tile_n;
        const int nrows = (int)max(0L, min((long)tile_rows, p.rows_z - first));
        const uint32_t z_off = p.z_is_a ? 0u : p.a_stage_bytes;
        const uint32_t z_ones = F16 ? 0x3C003C00u : 0x3F803F80u;
        long kc = (p.k_weave ? w.split : w.kb0) * 64 * p.kgroup;
        for (int i = 0; i < w.nkb && ok; ++i) {
          if (gen_fill > 0) {
            if (lane == 0) ok = mbar_wait(&empty_bar[gen_s], (uint32_t)((gen_fill - 1) & 1), p.status, p.tag);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
          }
          const uint32_t zbase = tiles_base + (uint32_t)gen_s * stage_bytes + z_off;
          const uint32_t tile_bytes = (uint32_t)tile_rows * 128u;
          if ((p.kgroup & 1) == 0 && (p.z_row_len & 127) == 0) {
            // one Philox block = 128 entries = the same row of two consecutive k-blocks; two blocks per
            // round of the loop so that the two dependent chains interleave (a warp runs alone on its scheduler)
            const int nitems = nrows * (p.kgroup >> 1);
            for (int it0 = gtid; it0 < nitems; it0 += 2 * GEN) {
              const int it1 = it0 + GEN;
              const bool two = it1 < nitems;
              const int row0_ = it0 % nrows, pr0 = it0 / nrows, row1_ = two ? it1 % nrows : 0, pr1 = two ? it1 / nrows : 0;
              const unsigned long long b0 = (unsigned long long)((first + row0_) * p.z_row_len + kc + pr0 * 128) >> 7;
              const unsigned long long b1 = (unsigned long long)((first + row1_) * p.z_row_len + kc + pr1 * 128) >> 7;
              const uint4 w0 = philox4x32_10((uint32_t)b0, (uint32_t)(b0 >> 32), p.seed_lo, p.seed_hi);
              const uint4 w1 = philox4x32_10((uint32_t)b1, (uint32_t)(b1 >> 32), p.seed_lo, p.seed_hi);
              z_store128(zbase + (uint32_t)(2 * pr0) * tile_bytes + (uint32_t)row0_ * 128u, tile_bytes, row0_, w0, z_ones);
              if (two) z_store128(zbase + (uint32_t)(2 * pr1) * tile_bytes + (uint32_t)row1_ * 128u, tile_bytes, row1_, w1, z_ones);
            }
          } else {
            for (int item = gtid; item < nrows * p.kgroup; item += GEN) {
              const int row = item % nrows, g = item / nrows;
              const uint2 bits = z_sign_bits64((first + row) * p.z_row_len + kc + g * 64, p.seed_lo, p.seed_hi);
              z_store64(zbase + (uint32_t)g * tile_bytes + (uint32_t)row * 128u, row, bits, z_ones);
            }
          }
          fence_async_smem();                 // the MMA reads the stage through the asynchronous proxy
          __syncwarp();
          if (lane == 0) mbar_arrive(&full_bar[gen_s]);
          kc += 64 * p.kgroup * (p.k_weave ? p.k_weave : 1);
          if (++gen_s == p.stages) { gen_s = 0; ++gen_fill; }
        }
      } else {
        // BACKPROBE with Z as the streamed operand (the estimator summed over the probes first): a stage holds, per
        // 64-position block of the column tile, ksteps*16 rows (probes) of 128 bytes, swizzled by the row like the
        // copy would have left them.  One Philox block = 128 entries = the same row of an even block and the odd
        // block behind it.  Rows past the last probe are drawn too: their partners in the A tile are zero.
        const int gtid = (quad * p.epi_groups + eg) * 32 + lane, GEN = 128 * p.epi_groups;
        const int rows_k = p.ksteps * 16;
        long kc = w.kb0 * rows_k;
        for (int i = 0; i < w.nkb && ok; ++i) {
          if (gen_fill > 0) {
            if (lane == 0) ok = mbar_wait(&empty_bar[gen_s], (uint32_t)((gen_fill - 1) & 1), p.status, p.tag);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
          }
          fill_bp_stage(tiles_base + (uint32_t)gen_s * stage_bytes + p.a_stage_bytes, kc, w, gtid, GEN);
          fence_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(&full_bar[gen_s]);
          kc += rows_k;
          if (++gen_s == p.stages) { gen_s = 0; ++gen_fill; }
        }
      }
    };
    // SKETCH: a unit's tiles are drawn when its turn comes (its epilogue is a few stores).  BACKPROBE: one unit ahead, so
    // that the MMAs of the next unit run during this unit's epilogue -- needs the second accumulator set: with one,
    // the next unit's MMAs wait for this epilogue, which would wait behind stages only those MMAs can free.
    const bool redraw_ahead = p.seeded && p.mode == MODE_BACKPROBE && p.acc_bufs == 2 && gen_quad0 == 0;
    if (redraw_ahead && blockIdx.x < p.units) redraw_unit(decode_unit(p, blockIdx.x));
    if (gen_quad0 > 0 && quad >= gen_quad0) {
      // A warp that only draws: it walks the stages of this CTA's units like the producer does and fills, alone, those
      // that fall into the slots of the ring it owns (slot mod n_gen), as far ahead of the MMAs as the ring allows.  The
      // slots have fixed owners because a wait by parity is only right for a thread that has seen every earlier phase
      // of the barrier: a warp that came to a slot two rounds late would take the phase before last for the last.
      // (numbered so that the first warps, the ones a short ring keeps busy, sit on different schedulers)
      const int n_gen = (4 - gen_quad0) * p.epi_groups, mine = eg * (4 - gen_quad0) + (quad - gen_quad0);
      const int rows_k = p.ksteps * 16;
      int turn = 0;                         // gen_s mod n_gen
      for (long u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
        const Unit w = decode_unit(p, u);
        long kc = w.kb0 * rows_k;
        for (int i = 0; i < w.nkb && ok; ++i) {
          if (turn == mine) {
            if (gen_fill > 0) {
              if (lane == 0) ok = mbar_wait(&empty_bar[gen_s], (uint32_t)((gen_fill - 1) & 1), p.status, p.tag);
              ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
              if (!ok) break;
            }
            fill_bp_stage(tiles_base + (uint32_t)gen_s * stage_bytes + p.a_stage_bytes, kc, w, lane, 32);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&full_bar[gen_s]);
          }
          kc += rows_k;
          if (++turn == n_gen) turn = 0;
          if (++gen_s == p.stages) { gen_s = 0; turn = 0; ++gen_fill; }
        }
      }
    } else
    for (long u = blockIdx.x; u < p.units && ok; u += gridDim.x, ++lu) {
      const Unit w = decode_unit(p, u);
      const int buf = p.acc_bufs == 2 ? (int)(lu & 1) : 0;
      const long use = p.acc_bufs == 2 ? lu >> 1 : lu;
      if (p.seeded && gen_quad0 == 0) {
        if (!redraw_ahead) redraw_unit(w);
        else if (u + gridDim.x < p.units) redraw_unit(decode_unit(p, u + gridDim.x));
        if (!ok) break;
      }
      if (lane == 0) ok = mbar_wait(&tmem_full_bar[buf], (uint32_t)(use & 1), p.status, p.tag);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      tc_fence_after();
      const long col0 = (long)w.tn * p.tile_n;
      if (p.mode == MODE_BACKPROBE) {
        // D[j, q] -> L[j][q].  Each warp stages 32 rows x 64 positions at a time in the layout the tensor store
        // wants (128-byte rows, 16-byte pieces swizzled by the row; lane = row) and stores the block with one
        // instruction; rows past the last probe are clipped by the TMA unit.  Storing straight from the
        // accumulator layout would send the 32 lanes of every store instruction to 32 different rows of L.
        for (int mt = 0; mt < p.m_sub; ++mt) {
          const long row_w = ((long)w.tm * p.m_sub + mt) * TILE_M + quad * 32;
          if (row_w >= p.rows) continue;                                       // warp-uniform
          for (int b = eg; b < w.nblk; b += p.epi_groups) {
            // the store that used this slot epi_slots blocks ago must have read it
            if (lane == 0) bulk_wait_read_upto(p.epi_slots - 1);
            __syncwarp();
            const uint32_t slot_base = epi_base + ((uint32_t)(quad * p.epi_groups + eg) * p.epi_slots + epi_slot) * 4096u;
            const uint32_t rowbase = slot_base + (uint32_t)lane * 128u;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              uint32_t v[32];
              tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) +
                            (uint32_t)(buf * acc_cols + mt * unit_cols + b * 64 + half * 32), v);
#pragma unroll
              for (int i = 0; i < 32; i += 8) {
                const uint32_t sdst = rowbase + ((((uint32_t)half * 4u + (uint32_t)(i >> 3)) ^ ((uint32_t)lane & 7u)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sdst),
                             "r"(pack2(v[i + 0], v[i + 1], F16)), "r"(pack2(v[i + 2], v[i + 3], F16)),
                             "r"(pack2(v[i + 4], v[i + 5], F16)), "r"(pack2(v[i + 6], v[i + 7], F16)) : "memory");
              }
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_3d(&map_c, slot_base, 0, (int)row_w, w.blk0 + b);
              bulk_commit();
            }
            if (++epi_slot == (uint32_t)p.epi_slots) epi_slot = 0;
          }
        }
      } else
      for (int mt = 0; mt < p.m_sub; ++mt) {
        // first row of this warp; CONV: rows are the pixels of the patch, the row tile picks the image
        const long row_w = (p.mode == MODE_CONV ? 0L : ((long)w.tm * p.m_sub + mt) * TILE_M) + quad * 32;
        if (row_w >= p.rows) continue;                                         // warp-uniform
        if (p.mode == MODE_CONV && w.img + mt >= p.nimg) continue;
        const long row = row_w + lane;
        for (int cu = eg * 32; cu < unit_cols; cu += 32 * p.epi_groups) {
          // several offsets per unit (CONTRACT): tile_n is then a multiple of 32 and a chunk lies in one offset
          const int tap_l = unit_cols > p.tile_n ? cu / p.tile_n : 0;
          const int c = cu - tap_l * p.tile_n;
          if (col0 + c >= p.cols) continue;
          uint32_t v[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = 0u;
          if (w.nkb > 0) {
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * acc_cols + mt * unit_cols + cu);
            if (p.tile_n - c >= 32) tmem_ld32(taddr, v);
            else tmem_ld16(taddr, v);
          }
          const int nc = min(32, p.tile_n - c);
          if (row >= p.rows) continue;
          if (p.mode == MODE_CONV) {
            // D[pixel of the patch, co] -> out[img][y][x][co]: 32 consecutive channels per thread
            const int pr = (int)row / p.patch_w, pc = (int)row % p.patch_w;
            const int y = w.py * p.patch_h + pr, x = w.px * p.patch_w + pc;
            if (y < p.H && x < p.W) {
              bf16* dst = p.L + (((long)(w.img + mt) * p.H + y) * p.W + x) * p.cols + col0 + c;
              if (nc == 32 && col0 + c + 32 <= p.cols) {
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                  uint4 o;
                  o.x = pack2(v[i + 0], v[i + 1], F16); o.y = pack2(v[i + 2], v[i + 3], F16);
                  o.z = pack2(v[i + 4], v[i + 5], F16); o.w = pack2(v[i + 6], v[i + 7], F16);
                  *reinterpret_cast<uint4*>(dst + i) = o;
                }
              } else {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (i < nc && col0 + c + i < p.cols)
                    reinterpret_cast<unsigned short*>(dst)[i] = (unsigned short)(pack2(v[i], v[i], F16) & 0xFFFFu);
              }
            }
          } else {
            // SKETCH / CONTRACT: partial tile in the order the accumulator comes out of tensor memory:
            // block(split, offset, tile) [128-row tile][32-column chunk][4-column group][row][4 floats],
            // so that the 32 lanes of every store write 512 contiguous bytes.  The reduce kernels undo it.
            const int chunks = (p.tile_n + 31) >> 5, qn = p.tile_n < 32 ? p.tile_n >> 2 : 8;   // 4-column groups per chunk
            float* blk = p.part + ((((long)w.split * p.taps + w.tap + tap_l) * p.tiles_m + w.tm) * p.tiles_n + w.tn) *
                                      ((long)p.m_sub * TILE_M * chunks * qn * 4);
            float* dst = blk + ((long)(mt * chunks + (c >> 5)) * qn * TILE_M + quad * 32 + lane) * 4;
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              if (i >= nc) break;
              *reinterpret_cast<float4*>(dst + (long)(i >> 2) * TILE_M * 4) =
                  make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]), __uint_as_float(v[i + 2]),
                              __uint_as_float(v[i + 3]));
            }
          }
        }
      }
      // this accumulator set may be overwritten by the unit after next
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty_bar[buf]);
    }
    // the tensor stores read this CTA's shared memory: they must be done before it exits
    if (p.mode == MODE_BACKPROBE && lane == 0) bulk_wait_all();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

// S[j][b] = sum over splits of the partial tiles, which are stored in accumulator order (see the
// epilogue).  Sixteen threads share a group of four columns and take the splits in turn (with some 150
// splits of a small tile the kernel is a chain of dependent loads otherwise); their sums are added in a
// fixed order, so the result is reproducible.  (row, col) = (b, j) when the samples were the MMA rows.
constexpr int RS_LANES = 16, RS_GROUPS = 16;
__global__ void __launch_bounds__(RS_LANES * RS_GROUPS)
reduce_sketch_partials(const float* __restrict__ part, float* __restrict__ S, long groups, long split_stride,
                       int splits, int tiles_n, int m_sub, int tile_n, int rows, int cols, int B, int swapped) {
  __shared__ float4 acc[RS_LANES][RS_GROUPS];
  pdl_trigger();
  pdl_wait();
  const int o = threadIdx.x % RS_GROUPS, g = threadIdx.x / RS_GROUPS;
  const long idx = (long)blockIdx.x * RS_GROUPS + o;   // group of four columns, in stored order
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  if (idx < groups) {
#pragma unroll 4
    for (int k = g; k < splits; k += RS_LANES) {
      const float4 v = *reinterpret_cast<const float4*>(part + (long)k * split_stride + idx * 4);
      s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
  }
  acc[g][o] = s;
  __syncthreads();
  if (g != 0 || idx >= groups) return;
  float t4[4] = {acc[0][o].x, acc[0][o].y, acc[0][o].z, acc[0][o].w};
#pragma unroll
  for (int l = 1; l < RS_LANES; ++l) {
    t4[0] += acc[l][o].x; t4[1] += acc[l][o].y; t4[2] += acc[l][o].z; t4[3] += acc[l][o].w;
  }
  uint32_t t = (uint32_t)idx;                   // (32-bit divisions: far fewer than 2^31 groups)
  const uint32_t qn = tile_n < 32 ? tile_n >> 2 : 8;
  const int row = (int)(t % TILE_M); t /= TILE_M;
  const int q = (int)(t % qn); t /= qn;
  const uint32_t chunks = (uint32_t)(tile_n + 31) >> 5;
  const int chunk = (int)(t % chunks); t /= chunks;
  const int mt = (int)(t % (uint32_t)m_sub); t /= (uint32_t)m_sub;
  const int tn = (int)(t % (uint32_t)tiles_n); t /= (uint32_t)tiles_n;
  const int tm = (int)t;
  const long rr = (long)(tm * m_sub + mt) * TILE_M + row;
  const int cl = chunk * 32 + q * 4;
  if (rr >= rows || cl >= tile_n) return;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const long cc = (long)tn * tile_n + cl + e;
    if (cc >= cols) break;
    if (swapped) S[cc * B + rr] = t4[e];      // rows are samples, columns probes
    else S[rr * B + cc] = t4[e];              // rows are probes, columns samples
  }
}

// out[m][offset][n] = scale(n) * sum_s block_s[...]: walks one split's blocks in their stored order (see the
// epilogue of MODE_CONTRACT), four consecutive input channels per group.  LANES threads share a group and take the
// splits in turn (one thread per group would walk a chain of `splits` dependent loads: 41 us for the 296 splits
// of a 32-channel layer); their sums are added in lane order, so the result is reproducible.
template <int LANES>
__global__ void __launch_bounds__(256) reduce_contract_partials(const float* __restrict__ part, float* __restrict__ out,
                                                                long groups, long split_stride, int splits, int T,
                                                                int tiles_m, int tiles_n, int m_sub, int tile_n,
                                                                int Cout, int Cin, float alpha,
                                                                const float* __restrict__ chan_scale) {
  constexpr int GROUPS = 256 / LANES;
  __shared__ float4 acc[LANES][GROUPS];
  pdl_trigger();
  pdl_wait();
  const int o = threadIdx.x % GROUPS, g = threadIdx.x / GROUPS;
  const long idx = (long)blockIdx.x * GROUPS + o;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  if (idx < groups) {
#pragma unroll 4
    for (int k = g; k < splits; k += LANES) {
      const float4 v = *reinterpret_cast<const float4*>(part + (long)k * split_stride + idx * 4);
      s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
  }
  if (LANES > 1) {
    acc[g][o] = s;
    __syncthreads();
    if (g != 0) return;
#pragma unroll
    for (int l = 1; l < LANES; ++l) { s.x += acc[l][o].x; s.y += acc[l][o].y; s.z += acc[l][o].z; s.w += acc[l][o].w; }
  }
  if (idx >= groups) return;
  uint32_t t = (uint32_t)idx;                   // (32-bit divisions: far fewer than 2^31 groups)
  const int row = (int)(t % TILE_M); t /= TILE_M;
  const int q = (int)(t % 8u); t /= 8u;
  const uint32_t chunks = (uint32_t)tile_n >> 5;
  const int chunk = (int)(t % chunks); t /= chunks;
  const int mt = (int)(t % (uint32_t)m_sub); t /= (uint32_t)m_sub;
  const int tn = (int)(t % (uint32_t)tiles_n); t /= (uint32_t)tiles_n;
  const int tm = (int)(t % (uint32_t)tiles_m); t /= (uint32_t)tiles_m;
  const int tap = (int)t;
  const int m = (tm * m_sub + mt) * TILE_M + row;
  const int n = tn * tile_n + chunk * 32 + q * 4;
  if (m >= Cout || n >= Cin) return;
  float4 sc = make_float4(alpha, alpha, alpha, alpha);
  if (chan_scale) sc = make_float4(chan_scale[n], chan_scale[n + 1], chan_scale[n + 2], chan_scale[n + 3]);
  *reinterpret_cast<float4*>(out + ((long)m * T + tap) * Cin + n) = make_float4(s.x * sc.x, s.y * sc.y, s.z * sc.z, s.w * sc.w);
}

// ------------------------------------------------------------------------------------ host side

static inline long cdivl(long a, long b) { return (a + b - 1) / b; }
static inline int round_up(int v, int a) { return (v + a - 1) / a * a; }
static const int SMEM_LIMIT = 227 * 1024;
static const int STATIC_SMEM_SLACK = 2048;     // barriers + alignment slack
static const int NUM_SMS = 148;
static const int BP_SLOT_BYTES = 4 * 32 * 128;      // back-probe output staging: per slot and epilogue group, 4 warps x 32 rows x 64 positions

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

// Tensor map over 16-bit elements (bfloat16, or float16 if `f16`), 128-byte swizzle unless told otherwise;
// dims/strides innermost first, strides in bytes for dims 1..rank-1.
static bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides,
                     const uint32_t* box, bool f16, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  cuuint64_t d[5], st[4];
  cuuint32_t bx[5];
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; bx[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) st[i] = strides[i];
  CUresult r = fn(m, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, st, bx, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Columns a partial tile occupies in its stored (accumulator-order) layout.
static int tile_cols_stored(int tile_n) { return tile_n < 32 ? tile_n : (tile_n + 31) / 32 * 32; }

static int pow2_cols(int n) { int c = 32; while (c < n) c *= 2; return c; }

static int pick_stages(uint32_t stage_bytes, int want_ctas_per_sm) {
  const int budget = SMEM_LIMIT / want_ctas_per_sm - STATIC_SMEM_SLACK;
  int s = budget / (int)stage_bytes;
  return std::max(1, std::min(s, MAX_STAGES));
}

static xconv_status launch(const CUtensorMap& ma, const CUtensorMap& mb, const TcParams& p, unsigned grid,
                           cudaStream_t st, const CUtensorMap* mc = nullptr) {
  TcParams q = p;
  // the seeded back-probe keeps a 4 KB table of sign patterns behind the stages: a stage gives way if it has to
  const size_t table = (p.seeded && p.mode == MODE_BACKPROBE) ? 4096 : 0;
  auto bytes = [&]() { return (size_t)q.stages * (q.a_stage_bytes + q.b_stage_bytes) + 1024 + (size_t)q.epi_bytes + q.smem_pad + table; };
  while (table && q.stages > 2 && bytes() > (size_t)(SMEM_LIMIT - 1024)) --q.stages;
  const size_t smem = bytes();
  if (smem > (size_t)(SMEM_LIMIT - 1024) || p.tmem_cols > 512 || p.stages > MAX_STAGES) return XCONV_ERR_UNSUPPORTED;
  void (*kernel)(CUtensorMap, CUtensorMap, CUtensorMap, TcParams) = p.f16 ? tc_gemm_kernel<true> : tc_gemm_kernel<false>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT - 1024);
  if (e != cudaSuccess) { set_cuda_error((int)e); return XCONV_ERR_CUDA; }
  q.tag = call_tag();
  if (q.layout == 0) { q.sbo = 1024; q.mn_step = 2048; q.layout = 2; q.cw_shift = 6; }
  if (q.depth < 1) q.depth = 1;
  if (q.epi_groups < 1) q.epi_groups = 1;
  e = launch_pdl(kernel, dim3(grid), dim3(64 + 128 * q.epi_groups), smem, st, ma, mb, mc ? *mc : ma, q);
  count_launch();
  if (e != cudaSuccess) { set_cuda_error((int)e); return XCONV_ERR_CUDA; }
  return XCONV_OK;
}

// ---- sketch --------------------------------------------------------------------------------

bool tc_plan_sketch(const xconv_desc* d, TcSketchPlan* p, bool redraw) {
  if (d->dtype != XCONV_BF16 && d->dtype != XCONV_F16) return false;
  const long K = (long)d->H * d->W * d->Cin;
  if (K % 8 != 0 || K < 2048 || K > 2000000000L) return false;
  p->swap = d->B >= d->r ? 1 : 0;
  const int rows = p->swap ? d->B : d->r, cols = p->swap ? d->r : d->B;
  p->tile_n = std::min(256, round_up(cols, 16));
  // Two row tiles that share each tile of the other operand halve the traffic into the SM per MMA, which
  // pays once the sketch is bound by the tensor pipe (r*B/(r+B) flops per byte against the machine's
  // ~250); below that it only doubles the split-k partial sums each CTA writes and the reduce re-reads.
  p->m_sub = (rows > TILE_M && (long)d->r * d->B > 250L * (d->r + d->B)) ? 2 : 1;
  p->tile_m = TILE_M * p->m_sub;
  p->tiles_m = (int)cdivl(rows, p->tile_m);
  p->tiles_n = (int)cdivl(cols, p->tile_n);
  // Small tiles: the cost of a stage is set by the two single-thread roles (barrier waits, copy issue,
  // commit), not by its bytes, so a stage takes up to four 64-wide k-blocks of each operand at once.
  p->rows_box = p->m_sub == 1 ? std::min(TILE_M, round_up(rows, 8)) : TILE_M * 2;
  const uint32_t block = (uint32_t)p->rows_box * 128 + p->tile_n * 128;
  p->kgroup = 1;
  if (K % 64 == 0) p->kgroup = block <= 12 * 1024 ? 4 : block <= 36 * 1024 ? 2 : 1;
  // Z redrawn in the kernel: a Philox block covers 128 consecutive entries of a row, i.e. two k-blocks
  if (redraw && K % 128 == 0 && p->kgroup == 1 && 2 * 2 * block + TILE_M * 128 <= (uint32_t)(SMEM_LIMIT - STATIC_SMEM_SLACK))
    p->kgroup = 2;
  p->kblocks = cdivl(K, 64L * p->kgroup);
  p->stages = std::max(1, std::min(MAX_STAGES, (SMEM_LIMIT - STATIC_SMEM_SLACK - TILE_M * 128) / (int)(block * p->kgroup)));
  const long tiles = (long)p->tiles_m * p->tiles_n;
  long splits = std::max(1L, std::min((long)NUM_SMS / tiles, cdivl(K, 64) / 8));
  splits = std::max(1L, std::min(splits, 512L));
  // k-blocks dealt as evenly as they go: every split takes kblocks_per_split, the first kb_rem one more
  splits = std::min(splits, p->kblocks);
  p->splits = (int)splits;
  p->kblocks_per_split = p->kblocks / splits;
  p->kb_rem = p->kblocks % splits;
  p->part_bytes = (size_t)p->splits * p->tiles_m * p->tiles_n * p->m_sub * TILE_M * tile_cols_stored(p->tile_n) *
                  sizeof(float);
  return true;
}

bool tc_sketch_can_redraw(const xconv_desc* d) {
  return ((long)d->H * d->W * d->Cin) % 64 == 0;     // a row of Z starts on a 64-entry boundary of the stream
}

xconv_status tc_run_sketch(const xconv_desc* d, const TcSketchPlan& pl, const void* X, const void* Z, float* S,
                           char* ws_head, char* part, cudaStream_t st, const unsigned long long* seed) {
  const long K = (long)d->H * d->W * d->Cin;
  const bool f16 = d->dtype == XCONV_F16;
  const int rows = pl.swap ? d->B : d->r, cols = pl.swap ? d->r : d->B;
  if (seed) Z = X;                                   // the map of Z is built but never used: any valid base
  const void* A = pl.swap ? X : Z;
  const void* Bm = pl.swap ? Z : X;
  CUtensorMap ma, mb;
  // Rows and k positions past the tensor are zero-filled by the TMA unit.  When the whole operand has
  // fewer rows than a tile the box stops at the last row (rounded to the 8-row swizzle group): rows the
  // box never writes only feed accumulator rows that are never stored.
  const uint32_t rows_box = (uint32_t)pl.rows_box;
  if (pl.kgroup > 1) {
    // (64 k, rows, k-blocks): one box brings kgroup K-major tiles, one behind the other in shared memory
    const uint64_t da[3] = {64, (uint64_t)rows, (uint64_t)(K / 64)}, db[3] = {64, (uint64_t)cols, (uint64_t)(K / 64)};
    const uint64_t sa[2] = {(uint64_t)K * 2, 128};
    const uint32_t box_a[3] = {64, rows_box, (uint32_t)pl.kgroup};
    const uint32_t box_b[3] = {64, (uint32_t)pl.tile_n, (uint32_t)pl.kgroup};
    if (!make_map(&ma, A, 3, da, sa, box_a, f16) || !make_map(&mb, Bm, 3, db, sa, box_b, f16)) return XCONV_ERR_CUDA;
  } else {
    const uint64_t da[2] = {(uint64_t)K, (uint64_t)rows}, db[2] = {(uint64_t)K, (uint64_t)cols};
    const uint64_t sa[1] = {(uint64_t)K * 2};
    const uint32_t box_a[2] = {64, rows_box};
    const uint32_t box_b[2] = {64, (uint32_t)pl.tile_n};
    if (!make_map(&ma, A, 2, da, sa, box_a, f16) || !make_map(&mb, Bm, 2, db, sa, box_b, f16)) return XCONV_ERR_CUDA;
  }
  TcParams p{};
  p.f16 = f16 ? 1 : 0;
  p.mode = MODE_SKETCH;
  p.tile_n = pl.tile_n;
  p.m_sub = pl.m_sub;
  p.acc_bufs = 1;
  p.tmem_cols = pow2_cols(pl.tile_n * pl.m_sub);
  p.stages = pl.stages;
  p.kgroup = pl.kgroup;
  p.ksteps = 4 * pl.kgroup;
  p.a_sub_bytes = TILE_M * 128;
  const uint32_t a_tile = rows_box * 128, b_tile = (uint32_t)pl.tile_n * 128;
  p.a_stage_bytes = a_tile * pl.kgroup;
  p.b_stage_bytes = b_tile * pl.kgroup;
  p.a_jump = (a_tile >> 4) - 6;
  p.b_jump = (b_tile >> 4) - 6;
  p.tx_bytes = p.a_stage_bytes + p.b_stage_bytes;
  if (seed) {                                        // Z is written by the generator warps, only X is copied
    p.seeded = 1;
    p.seed_lo = (uint32_t)(*seed & 0xFFFFFFFFull);
    p.seed_hi = (uint32_t)(*seed >> 32);
    p.z_is_a = pl.swap ? 0 : 1;
    p.z_row_len = K;
    p.rows_z = d->r;
    p.tx_bytes = p.z_is_a ? p.b_stage_bytes : p.a_stage_bytes;
  }
  // The MMA always reads 128 rows of A.  Behind a shorter tile it reads whatever follows (the rows it
  // produces are never stored), which must still be this CTA's shared memory.
  p.smem_pad = TILE_M * 128 - std::min<uint32_t>(a_tile, TILE_M * 128);
  p.a_boxes = p.b_boxes = 1;
  p.a_mn_major = p.b_mn_major = 0;
  p.tiles_m = pl.tiles_m;
  p.tiles_n = pl.tiles_n;
  p.taps = 1;
  p.kblocks = pl.kblocks;
  p.kblocks_per_split = pl.kblocks_per_split;
  p.kb_rem = pl.kb_rem;
  p.k_weave = pl.splits;
  p.units = (long)pl.tiles_m * pl.tiles_n * pl.splits;
  p.rows = rows;
  p.cols = cols;
  p.part = reinterpret_cast<float*>(part);
  p.status = reinterpret_cast<unsigned int*>(ws_head);
  xconv_status s = launch(ma, mb, p, (unsigned)p.units, st);
  if (s != XCONV_OK) return s;
  const long split_stride = (long)pl.tiles_m * pl.tiles_n * pl.m_sub * TILE_M * tile_cols_stored(pl.tile_n);
  const long groups = split_stride / 4;
  cudaError_t e = launch_pdl(reduce_sketch_partials, dim3((unsigned)cdivl(groups, RS_GROUPS)),
                             dim3(RS_LANES * RS_GROUPS), 0, st, p.part, S,
                             groups, split_stride, pl.splits, pl.tiles_n, pl.m_sub, pl.tile_n, rows, cols, d->B,
                             pl.swap);
  count_launch();
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
  if (barea == 0) { bw = 16; bh = 1; }     // tiny images: one 16-pixel row box, mostly zero fill
  *pw = bw; *ph = bh;
}

int tc_plan_wgrad(const xconv_desc* d, TcWgradPlan* p) {
  if (d->dtype != XCONV_BF16 && d->dtype != XCONV_F16) return 0;
  int mask = 0;
  const long Q = (long)d->H * d->W * d->Cout;
  // back-probe: D[j, q], rows = r, cols = Q, k = B
  if (Q % 64 == 0 && d->B % 8 == 0 && Q >= 2048 && Q < 2000000000L) {
    mask |= 1;
    p->bp_tile_n = 256;
    p->bp_m_sub = 1;
    p->bp_acc_bufs = (2 * p->bp_m_sub * p->bp_tile_n <= 512) ? 2 : 1;
    p->bp_tiles_r = (int)cdivl(d->r, TILE_M * p->bp_m_sub);
    // Column tiles of up to four 64-position blocks, sized so that every CTA of the persistent grid gets
    // the same number of units and (to within one block) the same number of blocks: with tiles of a fixed
    // width the CTAs that run one tile more than the rest finish alone, at a fraction of the bandwidth.
    const long NB = Q / 64, TM = p->bp_tiles_r;
    const long rounds = cdivl(NB * TM, 4L * NUM_SMS), units = rounds * NUM_SMS;
    long NT = cdivl(NB, 4);
    if (units % TM == 0 && units / TM <= NB && units / TM >= NT) NT = units / TM;
    p->bp_tiles_q = (int)NT;
    p->bp_base = NB / NT;
    p->bp_rem = NB % NT;
    p->bp_ksteps = std::min(4, (int)cdivl(d->B, 16));
    // the S tile of a stage holds only the probes there are (in 8-row swizzle groups): the 128-row MMA then
    // reads on into the dY tile and whatever lies behind it in this CTA's shared memory, and the rows it
    // makes of that are never stored
    p->bp_rows_box = p->bp_m_sub == 1 ? std::min(TILE_M, round_up(d->r, 8)) : TILE_M * p->bp_m_sub;
    const int stage = p->bp_rows_box * 128 + p->bp_ksteps * 16 * 128 * (p->bp_tile_n / 64);
    // Behind the stages: the epilogue warps' rings of staging slots.  Deeper rings let more tensor stores
    // be in flight, but a unit's k-blocks should all fit the stage ring (at least four stages otherwise).
    const int budget = SMEM_LIMIT - STATIC_SMEM_SLACK;
    const int want = std::min(4, (int)cdivl(d->B, p->bp_ksteps * 16) + 1);
    // a tile whose reduction over the batch is one or two stages long is over before its epilogue: two warps per quadrant
    p->bp_groups = cdivl(d->B, p->bp_ksteps * 16) <= 2 ? 2 : 1;
    const int slot_bytes = BP_SLOT_BYTES * p->bp_groups;
    p->bp_slots = 2;
    for (int slots = 8; slots >= 2; slots /= 2)
      if ((budget - slots * slot_bytes) / stage >= want) { p->bp_slots = slots; break; }
    p->bp_stages = std::max(1, std::min(MAX_STAGES, (budget - p->bp_slots * slot_bytes) / stage));
  }
  // contraction: rows = Cout, cols = Cin per offset, k = (probe, patch); volumes: d->r counts planes
  const int T = d->KH * d->KW * (d->KD > 1 ? d->KD : 1);
  p->ct_cw = (d->Cout % 64 == 0 && d->Cin % 64 == 0) ? 64 : ((d->Cout % 32 == 0 && d->Cin % 32 == 0) ? 32 : 0);
  // a circular shift wraps around the image, which a copy-engine box cannot (it fills with zeros): FP32-FMA kernels
  if (p->ct_cw && (long)d->H * d->W >= 16 && !d->circular) {
    mask |= 2;
    pick_patch(d->H, d->W, &p->patch_w, &p->patch_h);
    p->patches_x = (int)cdivl(d->W, p->patch_w);
    p->patches_y = (int)cdivl(d->H, p->patch_h);
    p->ct_tile_n = std::min(256, round_up(d->Cin, 16));
    // two output-channel tiles share each probe tile, unless the reduction is so short (few probes)
    // that more, smaller work units finish sooner
    p->ct_m_sub = (d->Cout > TILE_M && d->r >= 32) ? 2 : 1;
    p->ct_tiles_m = (int)cdivl(d->Cout, TILE_M * p->ct_m_sub);
    p->ct_tiles_n = (int)cdivl(d->Cin, p->ct_tile_n);
    const int bk = p->patch_w * p->patch_h;
    const uint32_t a_groups = d->Cout == p->ct_cw ? 1u : (uint32_t)((TILE_M / p->ct_cw) * p->ct_m_sub);
    const uint32_t b_groups = (uint32_t)cdivl(p->ct_tile_n, p->ct_cw);
    const uint32_t block = (uint32_t)bk * (uint32_t)p->ct_cw * 2;
    // Several kernel offsets per work unit while the accumulators fit tensor memory and two stages fit
    // shared memory: the L tile of a stage is fetched once for all of them, and with few input channels
    // one MMA spans the Z tiles of several offsets instead of issuing a narrow MMA for each.
    p->ct_tpu = 1;
    if (T == 9 && p->ct_tiles_n == 1 && p->ct_tile_n % 32 == 0 && p->ct_tile_n % p->ct_cw == 0)
      for (int t = 9; t > 1; t /= 3)
        if (t * p->ct_tile_n * p->ct_m_sub <= 512 && t * p->ct_tile_n <= 512 &&
            2 * block * (a_groups + t * b_groups) <= (uint32_t)(SMEM_LIMIT - STATIC_SMEM_SLACK)) {
          p->ct_tpu = t;
          break;
        }
    const uint32_t stage = block * (a_groups + (uint32_t)p->ct_tpu * b_groups);
    // narrow tiles are bound by the one MMA-issuing thread of a CTA: run two CTAs per SM then
    const int ct_ctas = (p->ct_tpu * p->ct_tile_n * p->ct_m_sub <= 128 && stage * 2 <= 100 * 1024) ? 2 : 1;
    p->ct_stages = pick_stages(stage, ct_ctas);
    p->ct_items = (long)d->r * p->patches_x * p->patches_y;
    const long tiles = (long)p->ct_tiles_m * p->ct_tiles_n * (T / p->ct_tpu);
    long splits = std::max(1L, std::min((long)NUM_SMS * ct_ctas / std::max(1L, tiles), p->ct_items / 4));
    splits = std::max(1L, std::min(splits, 512L));
    splits = std::min(splits, p->ct_items);
    p->ct_splits = (int)splits;
    p->ct_items_per_split = p->ct_items / splits;
    p->ct_items_rem = p->ct_items % splits;
    p->part_bytes = (size_t)p->ct_splits * T * p->ct_tiles_m * p->ct_tiles_n * p->ct_m_sub * TILE_M * p->ct_tile_n *
                    sizeof(float);
    // k-blocks in two halves (upper and lower image rows of the patch): four half-slots cover the load
    // latency that two whole stages cannot.  Needs halves of whole 8-row swizzle groups and one unit per CTA.
    const int hrows = (p->patch_h / 2) * p->patch_w;
    p->ct_halves = (p->ct_tpu == 1 && p->ct_cw == 64 && p->patch_h % 2 == 0 && hrows % 8 == 0 && hrows >= 16 &&
                    tiles * p->ct_splits <= NUM_SMS && ct_ctas == 1 && block * (a_groups + b_groups) >= 64 * 1024) ? 1 : 0;
    if (p->ct_halves) {
      const int half = (int)(block / 2 * (a_groups + b_groups));
      p->ct_stages = std::min(MAX_STAGES, (SMEM_LIMIT - STATIC_SMEM_SLACK) / half) & ~1;      // half-slots, an even number
      if (p->ct_stages < 4) p->ct_halves = 0, p->ct_stages = pick_stages(stage, ct_ctas);
    }
    // Block-sparse probes whose zero blocks are named (one work unit per CTA, which the halves guarantee): a list of
    // the probes with a non-zero block, per column tile, behind the partial sums
    p->ct_masked = (d->zero_blocks != nullptr && p->ct_halves && p->ct_tile_n % 64 == 0) ? 1 : 0;
    p->ct_list_bytes = 0;
    if (p->ct_masked) {
      const long probes = d->r / (d->D > 1 ? d->D : 1);
      p->part_bytes = (p->part_bytes + 255) & ~(size_t)255;
      p->ct_list_bytes = (size_t)p->ct_tiles_n * (size_t)(probes + 2) * sizeof(uint32_t);
      p->part_bytes += p->ct_list_bytes;
    }
  }
  return mask;
}

// Block-sparse probes: the list TcParams::zlist describes, from the caller's mask (zmask[j * groups + g] != 0: channels
// [64 g, 64 g + 64) of probing vector j are all zero).  One block per column tile of `gpt` channel groups; the probes
// keep their order, so that the sums of the contraction are taken in the same order whenever the mask is the same.
__global__ void __launch_bounds__(1024) list_nonzero_blocks(const unsigned char* __restrict__ zmask, int groups, int gpt,
                                                            int probes, uint32_t* __restrict__ list, int ld) {
  __shared__ int warp_count[32];
  pdl_trigger();
  pdl_wait();
  const int tn = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* row = list + (size_t)tn * ld;
  int base = 0;
  for (int j0 = 0; j0 < probes; j0 += 1024) {
    const int j = j0 + (int)threadIdx.x;
    uint32_t bits = 0;
    if (j < probes)
      for (int g = 0; g < gpt; ++g) {
        const int gg = tn * gpt + g;
        if (gg < groups && zmask[(size_t)j * groups + gg] == 0) bits |= 1u << g;
      }
    const unsigned vote = __ballot_sync(0xffffffffu, bits != 0u);
    if (lane == 0) warp_count[warp] = __popc(vote);
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < 32; ++w) { before += w < warp ? warp_count[w] : 0; total += warp_count[w]; }
    if (bits != 0u) row[1 + base + before + __popc(vote & ((1u << lane) - 1u))] = (uint32_t)j;
    base += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) { row[0] = (uint32_t)base; row[1 + base] = 0u; }
}

xconv_status tc_run_backprobe(const xconv_desc* d, const TcWgradPlan& pl, const void* S_bf16, const void* dY,
                              void* L, char* ws_head, cudaStream_t st, const unsigned long long* seed) {
  const long Q = (long)d->H * d->W * d->Cout;
  const int bk = pl.bp_ksteps * 16;
  const bool f16 = d->dtype == XCONV_F16;
  CUtensorMap ma, mb;
  // A = S (bfloat16) [r][B], k = b contiguous; B operand = dY [B][Q], q contiguous (MN-major tile)
  // dY as (64 positions, B rows, Q/64 blocks of 64 positions): one box fetches the [bk x 64] piece of one
  // block as 128-byte rows; the blocks of a column tile lie one behind the other in the stage
  const uint64_t da[2] = {(uint64_t)d->B, (uint64_t)d->r};
  const uint64_t db[3] = {64, (uint64_t)d->B, (uint64_t)(Q / 64)};
  const uint64_t sa[1] = {(uint64_t)d->B * 2}, sb[2] = {(uint64_t)Q * 2, 128};
  const uint32_t box_a[2] = {64, (uint32_t)pl.bp_rows_box};           // 128-byte rows whatever bk is (zero fill past B)
  const uint32_t box_b[3] = {64, (uint32_t)bk, 1};
  // (seeded: the streamed operand is never read, and its map stands in with the output's address)
  if (!make_map(&ma, S_bf16, 2, da, sa, box_a, f16) || !make_map(&mb, seed ? L : dY, 3, db, sb, box_b, f16)) return XCONV_ERR_CUDA;
  // L [r][Q] for the epilogue's stores, as (64 positions, r rows, Q/64 groups): one box = the 32 rows of one
  // epilogue warp x one block of positions
  CUtensorMap mc;
  const uint64_t dc[3] = {64, (uint64_t)d->r, (uint64_t)(Q / 64)};
  const uint32_t box_c[3] = {64, 32, 1};
  if (!make_map(&mc, L, 3, dc, sb, box_c, f16)) return XCONV_ERR_CUDA;
  TcParams p{};
  p.f16 = f16 ? 1 : 0;
  p.mode = MODE_BACKPROBE;
  p.tile_n = pl.bp_tile_n;
  p.m_sub = pl.bp_m_sub;
  p.acc_bufs = pl.bp_acc_bufs;
  p.tmem_cols = pow2_cols(pl.bp_acc_bufs * pl.bp_m_sub * pl.bp_tile_n);
  p.stages = pl.bp_stages;
  int slots = pl.bp_slots;
  int staging_quads = 4;                 // lane quadrants whose warps store (and own staging rings)
  if (seed) {
    // Z drawn on chip: a stage is filled by one warp alone, which takes longer than a copy, so the ring should hold a
    // stage for every drawing warp; the staging rings of the epilogue give up the room (and where only the first
    // quadrants hold rows -- the others do nothing but draw -- only those have rings at all)
    slots = 2;
    if (pl.bp_tiles_r == 1 && pl.bp_m_sub == 1 && d->r <= 96) staging_quads = (int)cdivl(d->r, 32);
    const int stage = pl.bp_rows_box * 128 + bk * 128 * (pl.bp_tile_n / 64);
    const int other = slots * (BP_SLOT_BYTES / 4) * staging_quads * pl.bp_groups + 4096;      // staging + table of signs
    p.stages = std::max(1, std::min(MAX_STAGES, (SMEM_LIMIT - STATIC_SMEM_SLACK - other) / stage));
  }
  p.ksteps = pl.bp_ksteps;
  p.a_boxes = 1;
  p.b_boxes = pl.bp_tile_n / 64;
  p.a_sub_bytes = TILE_M * 128;
  p.a_stage_bytes = (uint32_t)pl.bp_rows_box * 128;
  p.a_box_bytes = p.a_stage_bytes;
  p.b_box_bytes = (uint32_t)bk * 128;
  p.b_stage_bytes = (uint32_t)p.b_boxes * p.b_box_bytes;
  p.tx_bytes = p.a_stage_bytes + p.b_stage_bytes;
  p.a_mn_major = 0;
  p.b_mn_major = 1;
  p.b_lbo = p.b_box_bytes;
  p.epi_groups = pl.bp_groups;
  p.epi_bytes = (uint32_t)slots * (BP_SLOT_BYTES / 4) * staging_quads * pl.bp_groups;
  p.epi_slots = slots;
  p.bp_base = pl.bp_base;
  p.bp_rem = pl.bp_rem;
  p.tiles_m = pl.bp_tiles_r;
  p.tiles_n = pl.bp_tiles_q;
  p.taps = 1;
  p.kblocks = cdivl(d->B, bk);
  p.kblocks_per_split = p.kblocks;
  p.units = (long)pl.bp_tiles_q * pl.bp_tiles_r;
  p.rows = d->r;
  p.cols = Q;
  p.L = static_cast<bf16*>(L);
  p.Q = Q;
  if (seed) {
    p.seeded = 1;
    p.seed_lo = (uint32_t)(*seed & 0xFFFFFFFFull);
    p.seed_hi = (uint32_t)(*seed >> 32);
    p.z_row_len = Q;
  }
  p.status = reinterpret_cast<unsigned int*>(ws_head);
  return launch(ma, mb, p, (unsigned)std::min<long>(p.units, (long)NUM_SMS), st, &mc);
}

xconv_status tc_run_contract(const xconv_desc* d, const TcWgradPlan& pl, const void* L, const void* Z, float* dW,
                             float alpha, char* ws_head, char* part, cudaStream_t st) {
  const int T = d->KH * d->KW * (d->KD > 1 ? d->KD : 1);
  const int bk = pl.patch_w * pl.patch_h;
  const bool f16 = d->dtype == XCONV_F16;
  CUtensorMap ma, mb;
  // (cw channels, x, y, groups of cw channels, probe), cw = 64 or 32: one box = a whole
  // [patch x channels] tile laid out as consecutive blocks of (2*cw)-byte rows, one block per channel
  // group.  A layer with a single group of output channels loads just that block and gives the UMMA
  // descriptor a zero leading-dimension offset: all 128/cw row blocks of the MMA then read the same
  // block, and the accumulator rows past Cout hold copies that are never stored.
  const int cw = pl.ct_cw;
  const uint32_t row_bytes = (uint32_t)cw * 2;
  const bool one_group = d->Cout == cw;
  const int groups_a = one_group ? 1 : (TILE_M / cw) * pl.ct_m_sub, groups_b = (int)cdivl(pl.ct_tile_n, cw);
  const CUtensorMapSwizzle swz = cw == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
  const uint64_t da[5] = {(uint64_t)cw, (uint64_t)d->W, (uint64_t)d->H, (uint64_t)(d->Cout / cw), (uint64_t)d->r};
  const uint64_t sa[4] = {(uint64_t)d->Cout * 2, (uint64_t)d->W * d->Cout * 2, row_bytes,
                          (uint64_t)d->H * d->W * d->Cout * 2};
  const uint64_t db[5] = {(uint64_t)cw, (uint64_t)d->W, (uint64_t)d->H, (uint64_t)(d->Cin / cw), (uint64_t)d->r};
  const uint64_t sb[4] = {(uint64_t)d->Cin * 2, (uint64_t)d->W * d->Cin * 2, row_bytes,
                          (uint64_t)d->H * d->W * d->Cin * 2};
  const uint32_t box_h = (uint32_t)(pl.ct_halves ? pl.patch_h / 2 : pl.patch_h);   // image rows per copy
  const uint32_t box_a[5] = {(uint32_t)cw, (uint32_t)pl.patch_w, box_h, (uint32_t)groups_a, 1};
  const uint32_t box_b[5] = {(uint32_t)cw, (uint32_t)pl.patch_w, box_h, (uint32_t)groups_b, 1};
  if (!make_map(&ma, L, 5, da, sa, box_a, f16, swz) || !make_map(&mb, Z, 5, db, sb, box_b, f16, swz)) return XCONV_ERR_CUDA;
  TcParams p{};
  p.f16 = f16 ? 1 : 0;
  p.mode = MODE_CONTRACT;
  p.tile_n = pl.ct_tile_n;
  p.m_sub = pl.ct_m_sub;
  p.acc_bufs = 1;
  p.tpu = pl.ct_tpu;
  const int n_total = pl.ct_tpu * pl.ct_tile_n, blocks = n_total / cw;
  p.pieces = n_total > 256 ? 2 : 1;
  p.piece_cols[0] = p.pieces == 2 ? (blocks + 1) / 2 * cw : n_total;
  p.piece_cols[1] = n_total - p.piece_cols[0];
  p.tmem_cols = pow2_cols(n_total * pl.ct_m_sub);
  p.stages = pl.ct_stages;
  p.ksteps = bk / 16;
  p.a_boxes = one_group ? 1 : TILE_M / cw;
  p.b_boxes = groups_b;
  p.a_box_bytes = p.b_box_bytes = (uint32_t)bk * row_bytes;
  p.a_sub_bytes = (uint32_t)p.a_boxes * p.a_box_bytes;
  p.a_stage_bytes = (uint32_t)pl.ct_m_sub * p.a_sub_bytes;
  p.sbo = 8 * row_bytes;
  p.mn_step = 16 * row_bytes;
  p.layout = cw == 64 ? 2u : 4u;
  p.cw_shift = cw == 64 ? 6 : 5;
  p.b_tap_bytes = (uint32_t)p.b_boxes * p.b_box_bytes;
  p.b_stage_bytes = (uint32_t)pl.ct_tpu * p.b_tap_bytes;
  p.tx_bytes = p.a_stage_bytes + p.b_stage_bytes;
  p.a_mn_major = p.b_mn_major = 1;
  p.a_lbo = one_group ? 0u : p.a_box_bytes;
  p.b_lbo = p.b_box_bytes;
  p.tiles_m = pl.ct_tiles_m;
  p.tiles_n = pl.ct_tiles_n;
  p.taps = T;
  if (pl.ct_halves) {
    // every tile shrinks to half its rows; a "stage" of the ring is a half-slot
    const int hrows = bk / 2;
    p.halves = 1;
    p.a_box_bytes = p.b_box_bytes = (uint32_t)hrows * row_bytes;
    p.a_sub_bytes = (uint32_t)p.a_boxes * p.a_box_bytes;
    p.a_stage_bytes = p.a_half_bytes = (uint32_t)pl.ct_m_sub * p.a_sub_bytes;
    p.b_tap_bytes = (uint32_t)p.b_boxes * p.b_box_bytes;
    p.b_stage_bytes = p.b_tap_bytes;
    p.tx_bytes = p.a_stage_bytes + p.b_stage_bytes;
    p.a_lbo = one_group ? 0u : p.a_box_bytes;
    p.b_lbo = p.b_box_bytes;
    p.ks_h0 = hrows / 16;
    p.ks_x = (hrows % 16) ? 1 : 0;
    p.ks_h1 = p.ks_x ? (hrows - 8) / 16 : hrows / 16;
    // from the last 8-row group of a first half to the first group of the second half (same block, same operand)
    p.sbo_x = (p.a_stage_bytes + p.b_stage_bytes) - (uint32_t)(p.ks_h0 * 16) * row_bytes;
  }
  p.kblocks = pl.ct_items;
  p.kblocks_per_split = pl.ct_items_per_split;
  p.kb_rem = pl.ct_items_rem;
  p.units = (long)pl.ct_tiles_m * pl.ct_tiles_n * (T / pl.ct_tpu) * pl.ct_splits;
  p.patch_w = pl.patch_w;
  p.patch_h = pl.patch_h;
  p.patches_x = pl.patches_x;
  p.patches_y = pl.patches_y;
  p.pad = (d->KH - 1) / 2;
  p.depth = d->D > 1 ? d->D : 1;
  p.pad_d = d->KD > 1 ? (d->KD - 1) / 2 : 0;
  p.H = d->H;
  p.rows = d->Cout;
  p.cols = d->Cin;
  p.T = T;
  p.Cin = d->Cin;
  p.part = reinterpret_cast<float*>(part);
  p.status = reinterpret_cast<unsigned int*>(ws_head);
  if (pl.ct_masked) {
    const int probes = d->r / p.depth;
    uint32_t* list = reinterpret_cast<uint32_t*>(part + (pl.part_bytes - pl.ct_list_bytes));
    p.zlist = list;
    p.zlist_ld = probes + 2;
    p.zsplits = pl.ct_splits;
    const cudaError_t el = launch_pdl(list_nonzero_blocks, dim3((unsigned)pl.ct_tiles_n), dim3(1024), 0, st, d->zero_blocks,
                                      d->Cin / 64, pl.ct_tile_n / 64, probes, list, p.zlist_ld);
    count_launch();
    if (el != cudaSuccess) { set_cuda_error((int)el); return XCONV_ERR_CUDA; }
  }
  xconv_status s = launch(ma, mb, p, (unsigned)std::min<long>(p.units, 4L * NUM_SMS), st);
  if (s != XCONV_OK) return s;
  const long split_stride = (long)T * pl.ct_tiles_m * pl.ct_tiles_n * pl.ct_m_sub * TILE_M * pl.ct_tile_n;
  const long groups = split_stride / 4;
  cudaError_t e;
#define XC_REDUCE(LANES) launch_pdl(reduce_contract_partials<LANES>, dim3((unsigned)cdivl(groups, 256 / LANES)), dim3(256), 0, st, \
                                    p.part, dW, groups, split_stride, pl.ct_splits, T, pl.ct_tiles_m, pl.ct_tiles_n, \
                                    pl.ct_m_sub, pl.ct_tile_n, d->Cout, d->Cin, alpha, d->chan_scale)
  if (pl.ct_splits >= 64) e = XC_REDUCE(16);
  else if (pl.ct_splits >= 12) e = XC_REDUCE(4);
  else e = XC_REDUCE(1);
#undef XC_REDUCE
  count_launch();
  if (e != cudaSuccess) { set_cuda_error((int)e); return XCONV_ERR_CUDA; }
  return XCONV_OK;
}

// ---- self-test of the bounded wait ------------------------------------------------------------

// One warp waits on an mbarrier that nothing will ever complete; the wait gives up after `limit_ns`,
// records the call's tag in the workspace header exactly as a pipelined kernel would, and returns.
__global__ void wait_limit_selftest_kernel(unsigned int* status, unsigned int tag, unsigned long long limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  pdl_wait();
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    status[1] = tag;
    mbar_wait_slow(&bar, 0u, status, tag, limit_ns);
  }
}

xconv_status tc_run_wait_selftest(char* ws_head, unsigned long long limit_ns, cudaStream_t st) {
  wait_limit_selftest_kernel<<<1, 32, 0, st>>>(reinterpret_cast<unsigned int*>(ws_head), call_tag(), limit_ns);
  count_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return XCONV_ERR_CUDA; }
  return XCONV_OK;
}

// ---- exact convolution and input gradient -----------------------------------------------------

// Wd[n][T-1-t][m] = W[m][t][n]: the weights of the transposed convolution, laid out like W.
__global__ void __launch_bounds__(256) flip_transpose_weights(const bf16* __restrict__ W, bf16* __restrict__ Wd,
                                                              int Cout, int Cin, int T) {
  pdl_trigger();
  pdl_wait();
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const long count = (long)Cout * T * Cin;
  if (i >= count) return;
  const int m = (int)(i % Cout);
  const int t = (int)((i / Cout) % T);
  const int n = (int)(i / ((long)Cout * T));
  Wd[i] = W[((long)m * T + (T - 1 - t)) * Cin + n];
}

static void pick_patch_conv(int H, int W, int* pw, int* ph) {
  // patch of at most 128 pixels (the MMA rows) covering the image with the least work per pixel:
  // overhang and unused MMA rows both count
  double best = 1e30; int bw = 1, bh = 1;
  for (int w = 1; w <= std::min(W, 128); ++w)
    for (int h = 1; h * w <= 128 && h <= H; ++h) {
      const double cost = (double)cdivl(W, w) * (double)cdivl(H, h) * 128.0 / ((double)W * H);
      if (cost < best - 1e-9 || (cost < best + 1e-9 && w > bw)) { best = cost; bw = w; bh = h; }
    }
  *pw = bw; *ph = bh;
}

bool tc_plan_conv(const xconv_desc* d, bool dgrad, TcConvPlan* p) {
  if (d->dtype != XCONV_BF16 && d->dtype != XCONV_F16) return false;
  const int Ci = dgrad ? d->Cout : d->Cin, Co = dgrad ? d->Cin : d->Cout;
  if (Ci % 32 != 0 || Co % 8 != 0 || Co < 16 || d->circular) return false;   // circular padding: FP32-FMA kernels
  p->tile_n = std::min(256, round_up(Co, 16));
  p->tiles_n = (int)cdivl(Co, p->tile_n);
  pick_patch_conv(d->H, d->W, &p->patch_w, &p->patch_h);
  p->patches_x = (int)cdivl(d->W, p->patch_w);
  p->patches_y = (int)cdivl(d->H, p->patch_h);
  // Two images share each weight tile when the patch is a whole number of 8-row swizzle groups (the
  // second image's rows then start on a group boundary): the traffic into the SM per MMA cycle falls
  // from 94 to 62.5 bytes, which is what bounded the convolution.
  const int px = p->patch_w * p->patch_h;
  // (a kernel with a depth component shifts every plane on its own: one plane per unit then)
  p->m_sub = (px % 8 == 0 && d->B >= 2 && d->KD <= 1) ? 2 : 1;
  // Input channels go by 64 per stage (128-byte tile rows); layers whose channel count is a multiple of 32
  // only take 32 per stage (64-byte rows, 64-byte swizzle).  (32 per stage everywhere, for more and smaller
  // stages, was slower: 557 against 485 us on the 256-channel layer.)
  const uint32_t rows = (uint32_t)(p->m_sub == 2 ? px + TILE_M : TILE_M) + (uint32_t)p->tile_n;
  p->cw = Ci % 64 == 0 ? 64 : 32;
  p->stages = pick_stages(rows * 2 * (uint32_t)p->cw, 1);
  p->wt_bytes = dgrad ? (size_t)d->Cout * d->KH * d->KW * (d->KD > 1 ? d->KD : 1) * d->Cin * 2 : 0;
  return true;
}

xconv_status tc_run_conv(const xconv_desc* d, const TcConvPlan& pl, bool dgrad, const void* in, const void* W,
                         void* out, char* ws_head, char* wt, cudaStream_t st) {
  const int T = d->KH * d->KW * (d->KD > 1 ? d->KD : 1);
  const int Ci = dgrad ? d->Cout : d->Cin, Co = dgrad ? d->Cin : d->Cout;
  const bool f16 = d->dtype == XCONV_F16;
  const void* Wk = W;
  if (dgrad) {
    const long count = (long)d->Cout * T * d->Cin;
    cudaError_t e = launch_pdl(flip_transpose_weights, dim3((unsigned)cdivl(count, 256)), dim3(256), 0, st,
                               static_cast<const bf16*>(W), reinterpret_cast<bf16*>(wt), d->Cout, d->Cin, T);
    count_launch();
    if (e != cudaSuccess) { set_cuda_error((int)e); return XCONV_ERR_CUDA; }
    Wk = wt;
  }
  CUtensorMap ma, mb;
  // input as (cw channels, x, y, channel blocks of cw, image); weights as [Co][T*Ci]; cw = 64 or 32
  const uint32_t cw = (uint32_t)pl.cw, rb = 2 * cw;                      // channels and bytes per tile row
  const CUtensorMapSwizzle swz = cw == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
  const uint64_t da[5] = {cw, (uint64_t)d->W, (uint64_t)d->H, (uint64_t)(Ci / cw), (uint64_t)d->B};
  const uint64_t sa[4] = {(uint64_t)Ci * 2, (uint64_t)d->W * Ci * 2, rb, (uint64_t)d->H * d->W * Ci * 2};
  const uint32_t box_a[5] = {cw, (uint32_t)pl.patch_w, (uint32_t)pl.patch_h, 1, (uint32_t)pl.m_sub};
  const uint64_t db[2] = {(uint64_t)T * Ci, (uint64_t)Co};
  const uint64_t sb[1] = {(uint64_t)T * Ci * 2};
  const uint32_t box_b[2] = {cw, (uint32_t)pl.tile_n};
  if (!make_map(&ma, in, 5, da, sa, box_a, f16, swz) || !make_map(&mb, Wk, 2, db, sb, box_b, f16, swz)) return XCONV_ERR_CUDA;
  TcParams p{};
  p.f16 = f16 ? 1 : 0;
  p.mode = MODE_CONV;
  p.tile_n = pl.tile_n;
  const uint32_t px = (uint32_t)(pl.patch_w * pl.patch_h);
  p.m_sub = pl.m_sub;
  p.acc_bufs = (2 * pl.m_sub * pl.tile_n <= 512) ? 2 : 1;
  p.tmem_cols = pow2_cols(p.acc_bufs * pl.m_sub * pl.tile_n);
  p.stages = pl.stages;
  p.ksteps = (int)cw / 16;
  p.a_boxes = p.b_boxes = 1;
  // one image: the patch fills the first px rows of a 128-row tile.  Two images: the second image's px
  // rows follow the first's directly and its MMA tile starts there; 128 rows behind that start belong to the stage.
  p.a_sub_bytes = (pl.m_sub == 2 ? px : (uint32_t)TILE_M) * rb;
  p.a_stage_bytes = (pl.m_sub == 2 ? px + TILE_M : (uint32_t)TILE_M) * rb;
  p.b_stage_bytes = (uint32_t)pl.tile_n * rb;
  p.tx_bytes = (uint32_t)pl.m_sub * px * rb + p.b_stage_bytes;
  if (cw == 32) { p.layout = 4; p.sbo = 8 * rb; p.mn_step = 16 * rb; p.cw_shift = 5; }   // 64-byte swizzle
  p.a_mn_major = p.b_mn_major = 0;
  p.tiles_m = 1;
  p.tiles_n = pl.tiles_n;
  p.taps = 1;
  p.kblocks = (long)T * (Ci / cw);
  p.kblocks_per_split = p.kblocks;
  p.units = cdivl(d->B, pl.m_sub) * pl.patches_y * pl.patches_x * pl.tiles_n;
  p.nimg = d->B;
  p.patch_w = pl.patch_w;
  p.patch_h = pl.patch_h;
  p.patches_x = pl.patches_x;
  p.patches_y = pl.patches_y;
  p.pad = (d->KH - 1) / 2;
  p.depth = d->D > 1 ? d->D : 1;
  p.pad_d = d->KD > 1 ? (d->KD - 1) / 2 : 0;
  p.rows = (long)pl.patch_w * pl.patch_h;
  p.cols = Co;
  p.L = static_cast<bf16*>(out);
  p.T = T;
  p.Cin = Ci;
  p.H = d->H;
  p.W = d->W;
  p.cgroups = Ci / cw;
  p.status = reinterpret_cast<unsigned int*>(ws_head);
  return launch(ma, mb, p, (unsigned)std::min<long>(p.units, NUM_SMS), st);
}

}  // namespace xconv

