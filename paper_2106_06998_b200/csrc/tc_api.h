// Interface between the C ABI layer and the tcgen05 (5th-generation tensor core) kernels.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>

#include "../../include/xconv.h"

namespace xconv {

struct TcSketchPlan {
  int swap;            // 0: MMA rows = probes, columns = samples; 1: rows = samples, columns = probes
  int tile_m, tile_n, m_sub;  // output tile of one work unit; m_sub 128-row MMA tiles share the other operand
  int tiles_m, tiles_n, splits;
  int kgroup, rows_box;      // 64-wide k-blocks per stage; rows of the A box
  long kblocks, kblocks_per_split, kb_rem;   // the first kb_rem splits take one k-block more
  int stages;
  size_t part_bytes;
};

struct TcWgradPlan {
  // back-probe
  int bp_tile_n, bp_m_sub, bp_acc_bufs, bp_tiles_q, bp_tiles_r, bp_stages, bp_ksteps, bp_rows_box, bp_slots;
  int bp_groups;             // epilogue warps per tensor-memory lane quadrant
  long bp_base, bp_rem;      // column tiles: bp_base blocks of 64 positions each, the first bp_rem one more
  // contraction
  int ct_cw, ct_tile_n, ct_m_sub, ct_tiles_m, ct_tiles_n, ct_splits, ct_stages;
  int ct_tpu;                // kernel offsets per work unit (they share the L tile of every stage)
  int ct_halves;             // k-blocks copied and released in two halves; ct_stages then counts half-slots
  int ct_masked;             // block-sparse probes whose zero blocks are named: the contraction walks a list of the
                             // probes with a non-zero block per column tile (ct_list_bytes at the end of the partials)
  size_t ct_list_bytes;
  int patch_h, patch_w, patches_y, patches_x;
  long ct_items, ct_items_per_split, ct_items_rem;   // the first ct_items_rem splits take one item more
  size_t part_bytes;
};

struct TcConvPlan {
  int tile_n, tiles_n, stages, patch_w, patch_h, patches_x, patches_y;
  int m_sub;           // 2 = a work unit covers the same patch of two images, which share the weight tile
  int cw;              // input channels per stage: 64 (128-byte tile rows) or 32 (64-byte rows, more stages)
  size_t wt_bytes;     // dgrad only: transposed, flipped copy of the weights
};

// Fill the plan and say whether the tcgen05 kernels cover this layer.  tc_plan_wgrad returns a mask:
// bit 0 = back-probe covered, bit 1 = contraction covered.
bool tc_plan_sketch(const xconv_desc* d, TcSketchPlan* p, bool redraw = false);   // redraw: plan for a seeded call
int tc_plan_wgrad(const xconv_desc* d, TcWgradPlan* p);

bool tc_plan_conv(const xconv_desc* d, bool dgrad, TcConvPlan* p);
xconv_status tc_run_conv(const xconv_desc* d, const TcConvPlan& p, bool dgrad, const void* in, const void* W,
                         void* out, char* ws_head, char* wt, cudaStream_t st);

// `seed` != nullptr: Z is not read; its tiles are redrawn inside the kernel from the Philox stream of *seed
// (Rademacher entries; see xconv_probes_from_seed).  Only for layers tc_sketch_can_redraw accepts.
xconv_status tc_run_sketch(const xconv_desc* d, const TcSketchPlan& p, const void* X, const void* Z, float* S,
                           char* ws_head, char* part, cudaStream_t st, const unsigned long long* seed = nullptr);
bool tc_sketch_can_redraw(const xconv_desc* d);
// `seed` != nullptr: the streamed operand (`dY`) is a set of probing vectors that is not read but redrawn inside
// the kernel from the Philox stream of *seed -- the first step of the estimator when it sums over the probes first.
xconv_status tc_run_backprobe(const xconv_desc* d, const TcWgradPlan& p, const void* S_bf16, const void* dY,
                              void* L, char* ws_head, cudaStream_t st, const unsigned long long* seed = nullptr);
xconv_status tc_run_contract(const xconv_desc* d, const TcWgradPlan& p, const void* L, const void* Z, float* dW,
                             float alpha, char* ws_head, char* part, cudaStream_t st);

xconv_status tc_run_wait_selftest(char* ws_head, unsigned long long limit_ns, cudaStream_t st);

// bookkeeping shared with the ABI layer
void count_launch();
void set_cuda_error(int e);
unsigned int call_tag();   // tag of the API call in progress on this host thread

}  // namespace xconv
