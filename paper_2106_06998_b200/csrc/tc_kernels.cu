// tcgen05 kernels (placeholder translation unit: plans report "not covered" until the kernels land).
#include "tc_api.h"

namespace xconv {
bool tc_plan_sketch(const xconv_desc*, TcSketchPlan*) { return false; }
bool tc_plan_wgrad(const xconv_desc*, TcWgradPlan*) { return false; }
xconv_status tc_run_sketch(const xconv_desc*, const TcSketchPlan&, const void*, const void*, float*, char*, char*,
                           cudaStream_t) { return XCONV_ERR_UNSUPPORTED; }
xconv_status tc_run_backprobe(const xconv_desc*, const TcWgradPlan&, const void*, const void*, void*, char*,
                              cudaStream_t) { return XCONV_ERR_UNSUPPORTED; }
xconv_status tc_run_contract(const xconv_desc*, const TcWgradPlan&, const void*, const void*, float*, char*, char*,
                             cudaStream_t) { return XCONV_ERR_UNSUPPORTED; }
}  // namespace xconv
