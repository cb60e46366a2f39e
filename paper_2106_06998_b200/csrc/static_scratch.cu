// xconv_sketch_static: the sketch S = Z^T X for callers that cannot hand the library a workspace.
//
// Some callers have no way to obtain scratch memory at the point where they need the sketch: their
// device memory was handed out once at start-up (a framework's caching allocator owns all of it, or
// an embedding application fixed the budget), and calling cudaMalloc later is either forbidden by
// their host environment or unacceptable because it synchronises the whole device in the middle of
// a latency-critical loop.  For them the split-k partial sums of the sketch kernel live in a
// fixed-size array that is part of the library image itself; every GPU that loads the library
// carries these XCONV_STATIC_SCRATCH_FLOATS * 4 bytes until the process exits.
//
// The array below is a device symbol.  In host code its name is only a host-side stand-in, not a
// device address, so the entry point resolves the real address once per device with
// cudaGetSymbolAddress and hands that pointer to the kernels.
#include "../../include/xconv.h"

#include <mutex>

#include "common.cuh"
#include "simt_kernels.cuh"

namespace xconv {

extern thread_local int g_last_cuda_error;
extern thread_local int g_launches;

static __device__ __align__(256) float g_static_scratch[XCONV_STATIC_SCRATCH_FLOATS];

static const int MAX_DEVICES = 64;
static float* g_scratch_ptr[MAX_DEVICES];      // resolved device address of g_static_scratch, per device
static std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device (resolved on the first call there).
static xconv_status static_scratch_address(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
    g_last_cuda_error = (int)e;
    return XCONV_ERR_CUDA;
  }
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    float* ptr = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch);
    if (e != cudaSuccess || !ptr) {
      g_last_cuda_error = (int)e;
      return XCONV_ERR_CUDA;
    }
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return XCONV_OK;
}

template <typename T>
static xconv_status sketch_static_run(const xconv_desc* d, const void* X, const void* Z, float* S, float* scratch,
                                      cudaStream_t st) {
  const long K = (long)(d->D > 1 ? d->D : 1) * d->H * d->W * d->Cin;
  const long out_elems = (long)d->r * d->B;
  // as many k-splits as fill the GPU, capped by what the fixed array can hold
  const long tiles = ((d->r + 63) / 64) * (long)((d->B + 63) / 64);
  long splits = std::max(1L, std::min((4L * 148 + tiles - 1) / tiles, (K + 511) / 512));
  splits = std::min(splits, (long)XCONV_STATIC_SCRATCH_FLOATS / out_elems);
  long k_per_split = ((K + splits - 1) / splits + 15) / 16 * 16;
  splits = (K + k_per_split - 1) / k_per_split;
  dim3 grid((unsigned)((d->B + 63) / 64), (unsigned)((d->r + 63) / 64), (unsigned)splits);
  gemm_tn_simt<T><<<grid, 256, 0, st>>>(static_cast<const T*>(Z), static_cast<const T*>(X), scratch, d->r, d->B, K,
                                        k_per_split, (K % 4 == 0) ? 1 : 0);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; return XCONV_ERR_CUDA; }
  reduce_partials<<<(unsigned)((out_elems + RP_OUT - 1) / RP_OUT), RP_OUT * RP_LANES, 0, st>>>(scratch, S, out_elems, (int)splits, 1.0f,
                                                                       nullptr, 1);
  e = cudaGetLastError();
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; return XCONV_ERR_CUDA; }
  g_launches = 2;
  return XCONV_OK;
}

}  // namespace xconv

using namespace xconv;

extern "C" xconv_status xconv_sketch_static(const xconv_desc* desc, const void* X, const void* Z, float* sketch,
                                            void* cuda_stream) {
  if (!desc || !X || !Z || !sketch) return XCONV_ERR_INVALID_ARG;
  if (desc->B <= 0 || desc->Cin <= 0 || desc->H <= 0 || desc->W <= 0 || desc->r <= 0) return XCONV_ERR_INVALID_ARG;
  if (desc->dtype != XCONV_F32 && desc->dtype != XCONV_BF16 && desc->dtype != XCONV_F16) return XCONV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(Z) | reinterpret_cast<uintptr_t>(sketch)) & 15u)
    return XCONV_ERR_ALIGNMENT;
  // the one partial-sum slab [r][B] must fit the fixed array; beyond that there is nowhere to put it
  if ((long)desc->r * desc->B > (long)XCONV_STATIC_SCRATCH_FLOATS) return XCONV_ERR_WORKSPACE;
  if (desc->D < 0 || (long)(desc->D > 1 ? desc->D : 1) * desc->H * desc->W * desc->Cin > (1L << 40)) return XCONV_ERR_UNSUPPORTED;
  float* scratch = nullptr;
  xconv_status s = static_scratch_address(&scratch);
  if (s != XCONV_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  return desc->dtype == XCONV_F32 ? sketch_static_run<float>(desc, X, Z, sketch, scratch, st)
         : desc->dtype == XCONV_F16 ? sketch_static_run<f16>(desc, X, Z, sketch, scratch, st)
                                    : sketch_static_run<bf16>(desc, X, Z, sketch, scratch, st);
}
