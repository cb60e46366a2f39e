/*
 * libxconv -- XConv layer kernels for NVIDIA B200 (sm_100a), C ABI.
 *
 * XConv ("Low-memory stochastic backpropagation for convolutional layers") replaces the stored
 * input activation X of a convolutional layer by its projection onto r random probing vectors,
 * and estimates the weight gradient from that projection with a multi-channel randomized trace
 * estimator (Section 3, Eq. 2-6; Section 4.1, Algorithm 1).  This library exposes the steps of
 * Algorithm 1 for one layer:
 *
 *   forward :  Y = conv(X, w)            (Algorithm 1, forward step 1; Eq. 5)
 *              S = Z^T X  in R^{r x B}   (forward step 3; the paper's X-bar, text after Eq. 4)
 *   backward:  L = S dY^T                (backward step 3)
 *              dw_i = (1/r) tr(L T_{-k(i)} Z)   for every kernel offset k(i)  (backward step 4; Eq. 6)
 *              dX = conv^T(dY, w)        (standard back-propagation, which the method keeps exact)
 *
 * Index conventions (b batch, n input channel, m output channel, j probe, (y,x) pixel, (ky,kx) offset):
 *   Y [b,m,y,x]      = sum_{n,ky,kx} W[m,n,ky,kx] * X[b,n,y+ky-pad_h,x+kx-pad_w]
 *   S [j,b]          = sum_{n,y,x}   Z[j,n,y,x]   * X[b,n,y,x]
 *   L [j,m,y,x]      = sum_b         S[j,b]       * dY[b,m,y,x]
 *   dW[m,n,ky,kx]    = scale[n] * sum_{j,y,x} L[j,m,y,x] * Z[j,n,y+ky-pad_h,x+kx-pad_w]
 *   dX[b,n,u,v]      = sum_{m,ky,kx} W[m,n,ky,kx] * dY[b,m,u-ky+pad_h,v-kx+pad_w]
 * A pixel index outside [0,H)x[0,W) reads as zero (the truncating shift that matches a zero-padded
 * convolution), or, with desc.circular = 1, wraps around the image: the paper's circular shift T_k
 * (Section 3), i.e. a convolution with circular padding, its exact dX and the estimator written with the
 * same T_k.  scale[n] = 1/r (Eq. 6) unless
 * chan_scale is given (Eq. 8: 1/nnz(Z_n) for block-sparse probes).
 *
 * MEMORY LAYOUT.  Every tensor is dense and channels-last: the channel index is the fastest one.
 *   X, dY, Y, dX : element (b,c,y,x) at ((b*H + y)*W + x)*C + c
 *   Z            : element (j,n,y,x) at ((j*H + y)*W + x)*Cin + n
 *   W, dW        : element (m,n,ky,kx) at ((m*KH + ky)*KW + kx)*Cin + n
 *   S            : element (j,b) at j*B + b, always float
 * (This is torch's channels_last memory format of the logical NCHW / OIHW tensors.)
 * X, W, dY, Z, Y, dX are stored in desc.dtype (float, bfloat16, or float16 -- the "half precision" of
 * the paper's Section 5.2); S and dW are always float.
 * With 16-bit storage all sums are accumulated in float; L is kept in the storage type and S is rounded to
 * it where it feeds the tensor cores.  (float16 storage: values beyond 65504 in magnitude overflow, as in
 * any half-precision pipeline; the library does not rescale.)
 *
 * OWNERSHIP AND EXECUTION.  All pointers are device pointers owned by the caller, 16-byte aligned,
 * unless a parameter is documented as a host pointer.  The library allocates no device memory and
 * keeps no state between calls; scratch memory is passed in as `ws` (size from
 * xconv_workspace_bytes).  (One documented exception: xconv_sketch_static, whose scratch is a fixed
 * array inside the library image and whose first call per device resolves that array's address.)
 * Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*,
 * NULL = default stream) and the call returns without synchronising.  Outputs are overwritten, never
 * accumulated into.  The same Z must be given to the forward and to the backward call of a layer.
 * Results are bit-reproducible run to run (fixed reduction order, no atomics).
 *
 * ERRORS.  Every entry point returns an xconv_status.  Every check of the arguments is made before the
 * first launch: a call that returns XCONV_ERR_INVALID_ARG, XCONV_ERR_UNSUPPORTED, XCONV_ERR_ALIGNMENT
 * or XCONV_ERR_WORKSPACE has launched nothing and touched no buffer.  XCONV_ERR_CUDA reports a CUDA
 * runtime or driver call that failed in the middle of a call (a launch, a tensor-map encoding, a copy);
 * kernels the call enqueued before that point still run, and the outputs are then undefined.
 * Shapes or options without a kernel return XCONV_ERR_UNSUPPORTED; there is no CPU or library
 * fallback.  Pipelined kernels bound every device-side wait; a wait that runs
 * out records a code in the first word of the workspace, which xconv_workspace_status() reads back.
 */
#ifndef XCONV_H_
#define XCONV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { XCONV_F32 = 0, XCONV_BF16 = 1, XCONV_F16 = 2 } xconv_dtype;

typedef enum {
  XCONV_OK = 0,
  XCONV_ERR_INVALID_ARG = 1, /* NULL descriptor/pointer, non-positive size */
  XCONV_ERR_UNSUPPORTED = 2, /* valid request without a kernel (stride, even kernel size, circular shifts over volumes ...) */
  XCONV_ERR_ALIGNMENT = 3,   /* a pointer is not 16-byte aligned */
  XCONV_ERR_WORKSPACE = 4,   /* ws is NULL or smaller than xconv_workspace_bytes */
  XCONV_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed; see xconv_last_cuda_error */
  XCONV_ERR_TIMEOUT = 6      /* a bounded device-side wait ran out (reported by xconv_workspace_status) */
} xconv_status;

typedef enum { XCONV_OP_FORWARD = 0, XCONV_OP_WGRAD = 1, XCONV_OP_DGRAD = 2, XCONV_OP_SKETCH = 3,
               XCONV_OP_BACKPROBE = 4, XCONV_OP_CONTRACT = 5, XCONV_OP_SKETCH_SEEDED = 6,
               XCONV_OP_WGRAD_SEEDED = 7, XCONV_OP_WGRAD_INDEPENDENT = 8,
               XCONV_OP_SKETCH_SEEDED_GAUSSIAN = 9, XCONV_OP_WGRAD_SEEDED_GAUSSIAN = 10 } xconv_op;

/* Which arithmetic engine a call will use for its dominant kernel. */
typedef enum { XCONV_ENGINE_NONE = 0, XCONV_ENGINE_SIMT_F32 = 1, XCONV_ENGINE_TCGEN05_BF16 = 2,
               XCONV_ENGINE_TCGEN05_F16 = 3 } xconv_engine;

/* One convolutional layer: stride 1, dilation 1, one group, no bias, "same" output size
 * (2*pad_h = KH-1, 2*pad_w = KW-1; KH = KW in {1, 3, 5}).
 *
 * Volumes (three-dimensional layers, as in the paper's 3-D segmentation experiment, Section 5.5): set D > 1.
 * Every tensor gains a depth axis between the sample (or probe) index and the rows: X, dY, Y, dX
 * [B,D,H,W,C], Z [r,D,H,W,Cin], W and dW [Cout,KD,KH,KW,Cin] (torch's channels_last_3d of NCDHW / OIDHW),
 * and every formula above gains the matching sum over kz and shift z + kz - pad_d.  KD = 3 (with KH = KW = 3,
 * pad_d = 1) is a 3 x 3 x 3 kernel; KD = 1 (pad_d = 0) applies a planar kernel to every plane.  D, KD and
 * pad_d of 0 (a zero-initialised tail) mean a planar layer, the same as D = KD = 1.
 *
 * zero_blocks (block-sparse probes, Eq. 7: block n of probing vector j is zero with probability 1 - p_n, so a
 * share of the terms of Eq. 8's sum over j vanishes and need not be formed).  Byte [j*(Cin/64) + g] non-zero is the
 * caller's promise that Z[j, ..., 64g .. 64g+63] is identically zero.  On the layers for which
 * xconv_zero_blocks_used returns 1 -- wide layers on the tensor cores (Cin and Cout multiples of 64, the whole
 * contraction one work unit per SM), planar or 3 x 3 x 3 volumes -- xconv_contract and xconv_wgrad (in the paper's
 * order of summation, r <= B) then work on column tiles of up to 256 input channels and, for each tile, neither
 * fetch nor multiply the probing vectors whose blocks in that tile are all named zero; their work falls in
 * proportion.  Everywhere else the field is ignored, which gives the same result since the blocks are zero.
 * The mask is read, never written; xconv_zero_blocks computes it from Z.  A block that is named zero but is not
 * either enters the sum or drops out of it (it drops out when all blocks of its probing vector in its tile are
 * named zero); no error is raised.  The workspace an op needs depends on whether the field is NULL: ask
 * xconv_workspace_bytes with the descriptor the call will get.  A zero-initialised tail means no mask. */
typedef struct {
  int32_t B, Cin, Cout, H, W;
  int32_t KH, KW, pad_h, pad_w;
  int32_t r;                /* number of probing vectors */
  int32_t dtype;            /* xconv_dtype: storage of X, W, dY, Z, Y, dX */
  int32_t circular;         /* 0: truncating shifts (zero padding); 1: circular shifts T_k of Section 3 (planar layers
                               only; the offset contraction and the convolutions then run on the FP32-FMA kernels,
                               whatever the storage type: a copy-engine box cannot wrap around an image) */
  const float* chan_scale;  /* NULL: scale 1/r.  Else device pointer to Cin floats (Eq. 8). */
  int32_t D, KD, pad_d;     /* depth of the volume and of the kernel; 0 or 1: planar layer */
  const unsigned char* zero_blocks;  /* NULL, or device pointer to r * (Cin/64) bytes: see below */
} xconv_desc;

/* Scratch bytes `op` needs for this layer (0 is possible).  Returns 0 for an invalid descriptor. */
size_t xconv_workspace_bytes(const xconv_desc* desc, int op);

/* Engine the dominant kernel of `op` runs on for this layer (XCONV_ENGINE_NONE if unsupported). */
int xconv_engine_for(const xconv_desc* desc, int op);

/* Algorithm 1, forward pass: Y = conv(X, W) (step 1, Eq. 5) and S = Z^T X (step 3).
 * X [B,H,W,Cin], W [Cout,KH,KW,Cin], Z [r,H,W,Cin] in desc.dtype; Y [B,H,W,Cout] in desc.dtype;
 * sketch [r,B] float.  After this call the caller may drop X and keep only `sketch` and Z (or the
 * seed it drew Z from): a memory factor of N*Cin/r per sample (Section 3). */
xconv_status xconv_forward(const xconv_desc* desc, const void* X, const void* W, const void* Z,
                           void* Y, float* sketch, void* ws, size_t ws_bytes, void* cuda_stream);

/* Forward step 3 alone, S = Z^T X (for callers whose convolution runs elsewhere). */
xconv_status xconv_sketch(const xconv_desc* desc, const void* X, const void* Z, float* sketch,
                          void* ws, size_t ws_bytes, void* cuda_stream);

/* Probing vectors redrawn from a seed.  Algorithm 1 stores the random seed s in the forward pass (step 2)
 * and redraws Z[s] in the backward pass (step 2) instead of keeping Z; the paper leaves the generator
 * open.  This library fixes it as follows (Rademacher entries, for which E[z z^T] = I holds as Section 3
 * requires): number the entries of Z in memory order, e = ((j*H + y)*W + x)*Cin + n.  Entry e is +1 if bit
 * (e mod 128) of the Philox-4x32-10 block with counter (e div 128) and key (seed & 0xffffffff, seed >> 32)
 * is 0, and -1 if it is 1; bit b of a block is bit (b mod 32) of its output word (b div 32).  (Philox:
 * Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC'11.)
 *
 * xconv_probes_from_seed writes Z [r,H,W,Cin] in desc.dtype (desc.B, Cout, KH.. are ignored beyond validity).
 * xconv_sketch_seeded computes S = Z[seed]^T X (Algorithm 1 forward step 3) without reading Z from memory:
 * where the tensor-core kernel covers the layer and H*W*Cin is a multiple of 64 the tiles of Z are redrawn
 * inside the kernel, so that only X leaves HBM; otherwise Z is first written into `ws` and the regular
 * kernels run on it (xconv_workspace_bytes(desc, XCONV_OP_SKETCH_SEEDED) covers both cases).  The result
 * equals xconv_sketch on xconv_probes_from_seed's Z up to the order of summation.
 * xconv_wgrad_seeded is Algorithm 1's backward pass from the stored seed.  Where r > B and the tensor-core
 * kernels cover the layer, xconv_wgrad sums over the probes first (S^T Z, then the offset contraction over the
 * batch), Z is the streamed operand of its first kernel, and that kernel redraws its tiles of Z on chip: Z
 * neither enters nor leaves HBM.  Elsewhere step 2 redraws Z[seed] into `ws` and steps 3-4 are xconv_wgrad on
 * it (xconv_workspace_bytes(desc, XCONV_OP_WGRAD_SEEDED) covers both cases: the scratch of xconv_wgrad, plus
 * one Z in the second).  Either way the estimate equals xconv_wgrad(sketch, dY, xconv_probes_from_seed(seed))
 * bit for bit.  With these two calls a layer keeps S (r*B floats) and the 8-byte seed between its forward and its
 * backward pass, the memory factor the paper quotes. */
xconv_status xconv_probes_from_seed(const xconv_desc* desc, unsigned long long seed, void* Z, void* cuda_stream);
xconv_status xconv_sketch_seeded(const xconv_desc* desc, const void* X, unsigned long long seed, float* sketch,
                                 void* ws, size_t ws_bytes, void* cuda_stream);
xconv_status xconv_wgrad_seeded(const xconv_desc* desc, const float* sketch, const void* dY, unsigned long long seed,
                                float* dW, void* ws, size_t ws_bytes, void* cuda_stream);

/* The same with standard normal probing vectors, the distribution of the paper's theory (Section 3: z ~ N(0, I);
 * Algorithm 1 backward step 2: "Z = randn(N, r)" redrawn from the stored seed).  Definition: entries numbered in
 * memory order as above; Philox-4x32-10 block b = e div 4 has counter (b in words 0-1, word 2 = 1, word 3 = 0) --
 * word 2 keeps it apart from the Rademacher stream of the same seed -- and the seed as key; its words w0..w3 give
 * two pairs (w0, w1), (w2, w3) of uniforms u = (2 (w >> 9) + 1) / 2^24, and each pair (u_a, u_b) two normals by the
 * Box-Muller transform: sqrt(-2 ln u_a) cos(2 pi u_b) for the even entry, sqrt(-2 ln u_a) sin(2 pi u_b) for the
 * odd one, rounded to desc.dtype.  Logarithm, sine and cosine are short float series of single IEEE operations
 * (relative error 2e-7, absolute 1e-7), so that a host program can reproduce every entry bit for bit.
 *
 * xconv_gaussian_probes_from_seed writes Z [r,H,W,Cin] (volumes [r,D,H,W,Cin]) in desc.dtype; no scratch.
 * Drawing a normal costs more than reading it back from memory (one Philox block per four entries against one per
 * 128 signs, plus the series), so these probes are not redrawn inside the sketch and estimator kernels:
 * xconv_sketch_seeded_gaussian and xconv_wgrad_seeded_gaussian write Z[seed] into `ws` (behind the regular scratch:
 * xconv_workspace_bytes(desc, XCONV_OP_SKETCH_SEEDED_GAUSSIAN / XCONV_OP_WGRAD_SEEDED_GAUSSIAN) bytes) and run
 * xconv_sketch / xconv_wgrad on it -- Algorithm 1 taken literally.  Between the passes a layer keeps S and the seed. */
xconv_status xconv_gaussian_probes_from_seed(const xconv_desc* desc, unsigned long long seed, void* Z,
                                             void* cuda_stream);
xconv_status xconv_sketch_seeded_gaussian(const xconv_desc* desc, const void* X, unsigned long long seed,
                                          float* sketch, void* ws, size_t ws_bytes, void* cuda_stream);
xconv_status xconv_wgrad_seeded_gaussian(const xconv_desc* desc, const float* sketch, const void* dY,
                                         unsigned long long seed, float* dW, void* ws, size_t ws_bytes,
                                         void* cuda_stream);

/* The block-sparse probing vectors of Eq. 7 from a seed: block n of probing vector j (the H*W entries of input
 * channel n) is kept with probability p and is zero otherwise, independently for every (n, j); the kept blocks are
 * those of the dense probes of the same seed (gaussian = 0: xconv_probes_from_seed, 1: xconv_gaussian_probes_from_seed;
 * Eq. 7 prints the normal ones).  Definition of the mask: blocks numbered g = j*Cin + n; Philox-4x32-10 block g div 4
 * with counter (g div 4 in words 0-1, word 2 = 2, word 3 = 0) and the seed as key; block g is kept iff output word
 * (g mod 4) is below floor(p * 2^32).  Outputs, all device pointers: Z [r,H,W,Cin] (volumes [r,D,H,W,Cin]) in
 * desc.dtype, 16-byte aligned; keep, r*Cin bytes (1 = kept); chan_scale, Cin floats, 1/nnz(Z_n) of Eq. 8 (0 for a
 * channel none of the r vectors probes) -- what desc.chan_scale takes.  p outside [0, 1]: XCONV_ERR_INVALID_ARG.
 * Four small launches (dense probes, mask, scale, zeroing); no scratch.  A caller that keeps the seed and p between the
 * passes redraws the same Z, keep and chan_scale in the backward pass. */
xconv_status xconv_block_sparse_probes_from_seed(const xconv_desc* desc, unsigned long long seed, int gaussian, double p,
                                                 void* Z, unsigned char* keep, float* chan_scale, void* cuda_stream);

/* Algorithm 1, backward steps 3-4: L = S dY^T, then dW[m,n,k] = scale[n] * tr(L^m T_{-k} Z_n) for
 * every offset (Eq. 6; three-step procedure of Section 3).  sketch [r,B] float as written by
 * xconv_forward; dY [B,H,W,Cout], Z [r,H,W,Cin] in desc.dtype; dW [Cout,KH,KW,Cin] float.
 * L lives in the workspace only. */
xconv_status xconv_wgrad(const xconv_desc* desc, const float* sketch, const void* dY, const void* Z,
                         float* dW, void* ws, size_t ws_bytes, void* cuda_stream);

/* The two halves of xconv_wgrad as calls of their own (for callers that overlap them with other work
 * and for per-step timing).  xconv_backprobe: L = S dY^T (Algorithm 1 backward step 3), L [r,H,W,Cout]
 * in desc.dtype (element (j,m,y,x) at ((j*H + y)*W + x)*Cout + m), xconv_backprobe_bytes(desc) bytes.
 * xconv_contract: dW[m,n,k] = scale[n] * sum_{j,y,x} L[j,m,y,x] Z[j,n,(y,x)+k] (backward step 4; Eq. 6).
 * xconv_wgrad(ws) is exactly xconv_backprobe + xconv_contract with L placed inside ws. */
size_t xconv_backprobe_bytes(const xconv_desc* desc);
xconv_status xconv_backprobe(const xconv_desc* desc, const float* sketch, const void* dY, void* L,
                             void* ws, size_t ws_bytes, void* cuda_stream);
xconv_status xconv_contract(const xconv_desc* desc, const void* L, const void* Z, float* dW,
                            void* ws, size_t ws_bytes, void* cuda_stream);

/* mask[j*(Cin/64) + g] = 1 if every element of Z[j, ..., 64g .. 64g+63] is +0 or -0, else 0 (the mask
 * desc.zero_blocks takes).  Z [r,H,W,Cin] (volumes [r,D,H,W,Cin])
 * in desc.dtype, mask r*(Cin/64) bytes, both device pointers.  Cin must be a multiple of 64
 * (XCONV_ERR_UNSUPPORTED otherwise).  One pass over Z; no scratch. */
xconv_status xconv_zero_blocks(const xconv_desc* desc, const void* Z, unsigned char* mask, void* cuda_stream);

/* 1 if xconv_contract skips the blocks that desc.zero_blocks names on this layer (and with it xconv_wgrad,
 * unless r > B makes that call sum over the probes first), 0 if the field is ignored there (or NULL, or the
 * descriptor invalid).  Host-side arithmetic only. */
int xconv_zero_blocks_used(const xconv_desc* desc);

/* Trace estimation applied to every input/output channel pair on its own ("independent" probing: first
 * sentence of the multi-channel case in Section 3; Eq. 4 per pair).  The probing vectors have the same shape
 * as for the multi-channel estimator, Z [r,H,W,Cin], but block n of a vector only ever meets channel n:
 *   sketch[j,n,b]  = sum_{y,x} Z[j,n,y,x] * X[b,n,y,x]                  (r*Cin*B floats, element (j,n,b) at (j*Cin + n)*B + b)
 *   dW[m,n,ky,kx]  = (1/r) * sum_{j,b,y,x} sketch[j,n,b] * dY[b,m,y,x] * Z[j,n,y+ky-pad_h,x+kx-pad_w]
 * No other input channel enters the estimate of a pair (no crosstalk), at the price of a sketch Cin times
 * larger: the memory factor per sample is N/r instead of N*Cin/r.  xconv_sketch_independent needs no scratch.
 * xconv_wgrad_independent takes xconv_workspace_bytes(desc, XCONV_OP_WGRAD_INDEPENDENT) bytes; it sums over
 * the probes first (the activation rebuilt channel by channel from its sketch, held in `ws` in desc.dtype) and
 * then runs the offset contraction over the batch -- the same sum as the formula above in another order.
 * desc.chan_scale is ignored (the scale is 1/r). */
xconv_status xconv_sketch_independent(const xconv_desc* desc, const void* X, const void* Z, float* sketch,
                                      void* cuda_stream);
xconv_status xconv_wgrad_independent(const xconv_desc* desc, const float* sketch, const void* dY, const void* Z,
                                     float* dW, void* ws, size_t ws_bytes, void* cuda_stream);

/* Exact input gradient (the transposed convolution; the method leaves it as in standard
 * back-propagation, Section 1).  dY [B,H,W,Cout], W [Cout,KH,KW,Cin]; dX [B,H,W,Cin] in desc.dtype. */
xconv_status xconv_dgrad(const xconv_desc* desc, const void* dY, const void* W, void* dX,
                         void* ws, size_t ws_bytes, void* cuda_stream);

/* Sketch + weight-gradient estimate from HOST buffers (Algorithm 1 forward step 3 and backward
 * steps 3-4 back to back).  hX, hdY, hZ are host pointers to desc.dtype data (pinned memory makes the
 * copies asynchronous), hS [r,B] and hdW [Cout,KH,KW,Cin] host float outputs.  `arena` is caller-owned
 * device memory of at least xconv_host_arena_bytes(desc) bytes that receives the inputs, the
 * outputs and the workspace.  Copies in, runs xconv_sketch and xconv_wgrad, copies out and
 * synchronises `cuda_stream` before returning. */
size_t xconv_host_arena_bytes(const xconv_desc* desc);
xconv_status xconv_sketch_wgrad_host(const xconv_desc* desc, const void* hX, const void* hdY, const void* hZ,
                                     float* hS, float* hdW, void* arena, size_t arena_bytes,
                                     void* cuda_stream);

/* The sketch S = Z^T X without any workspace argument and without any allocation.  (The paper has no
 * counterpart to this call; it computes exactly what xconv_sketch computes.)
 *
 * It is meant for callers that cannot allocate device memory when they need the sketch and have no
 * spare buffer to lend as `ws`: code running inside a host application or framework that gave out
 * all device memory at start-up and forbids cudaMalloc afterwards, or a latency-critical loop in
 * which cudaMalloc's device-wide synchronisation is not acceptable.  The split-k partial sums go to
 * a fixed array of XCONV_STATIC_SCRATCH_FLOATS floats (4 MiB) that is part of the library image:
 * every GPU that loads the library holds it until the process exits.
 *
 *  - X [B,H,W,Cin] and Z [r,H,W,Cin] in desc.dtype and sketch [r,B] float are caller-owned device
 *    pointers, 16-byte aligned, as for xconv_sketch.  desc.Cout, KH, KW and pad_* are ignored.
 *  - Limit: r*B <= XCONV_STATIC_SCRATCH_FLOATS.  A larger layer returns XCONV_ERR_WORKSPACE ("too
 *    small": the fixed array cannot hold even one [r,B] slab) and launches nothing.
 *  - The call performs no cudaMalloc, cudaFree or other allocating call.  The first call on a device
 *    resolves the device address of the array (cudaGetSymbolAddress, with that device current).  With
 *    CUDA's lazy module loading that first call is also the moment at which the driver loads the
 *    library's device code, fixed array included, onto that device: it can take the 4 MiB then,
 *    synchronise, or fail if no device memory is left.  So make one warm-up call per device at
 *    start-up -- before the memory budget is handed out, outside any stream capture and outside the
 *    latency-critical loop; later calls on that device only launch kernels.
 *  - All calls on a device share the one array.  Nothing in it has to start at zero -- every call
 *    overwrites the slabs it then sums -- so stale contents of an earlier call are harmless, but two
 *    calls that overlap on the GPU (different streams, no dependency) race on it.  Serialise them.
 *  - Always runs the FP32-FMA kernel; results agree with xconv_sketch to rounding (summation order). */
#define XCONV_STATIC_SCRATCH_FLOATS (1 << 20)
xconv_status xconv_sketch_static(const xconv_desc* desc, const void* X, const void* Z, float* sketch,
                                 void* cuda_stream);

/* Reads the status the kernels of the last call left in the header of `ws` (synchronises
 * `cuda_stream`).  XCONV_OK, or XCONV_ERR_TIMEOUT if a bounded device-side wait ran out in that call.
 * The header never needs clearing: every call tags it afresh, so a later call on the same `ws`
 * reports its own outcome.  (Only the tensor-core kernels wait on anything; calls served by the
 * FP32-FMA kernels leave the header as it was.) */
xconv_status xconv_workspace_status(const void* ws, void* cuda_stream);

/* Self-test of the failure path: one warp waits, with the same bounded wait the pipelined kernels use,
 * on a barrier that nothing completes; after `limit_ms` (1..2000) it gives up and records the
 * time-out in the header of `ws` (at least 256 bytes), where xconv_workspace_status then reports
 * XCONV_ERR_TIMEOUT.  Nothing faults or hangs; the context stays usable.  (No counterpart in the
 * paper.) */
xconv_status xconv_selftest_wait_limit(void* ws, size_t ws_bytes, unsigned int limit_ms, void* cuda_stream);

/* Measurement aid (no counterpart in the paper): the FP32 fused-multiply-add rate this GPU sustains,
 * which is the arithmetic ceiling of the FP32-FMA kernels that serve float storage.  Runs a kernel of
 * register-only FMA chains a few times on `cuda_stream`, times it with CUDA events, synchronises, and
 * writes the best rate in TFLOP/s (2 flops per FMA) to the HOST double `tflops`.  `scratch` is device
 * memory of at least 148*16*256*4 bytes that the kernel writes its (meaningless) sums to. */
xconv_status xconv_measure_fma_rate(void* scratch, size_t scratch_bytes, double* tflops, void* cuda_stream);

/* Number of kernels the last successful call on this host thread enqueued. */
int xconv_last_launch_count(void);

/* cudaError_t (as int) of the last failing CUDA call on this host thread, 0 if none. */
int xconv_last_cuda_error(void);

const char* xconv_status_string(xconv_status s);

#ifdef __cplusplus
}
#endif
#endif /* XCONV_H_ */
