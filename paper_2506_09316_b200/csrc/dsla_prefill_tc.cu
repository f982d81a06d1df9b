// Tensor-core (tcgen05) prefill: placeholder until the kernel lands; reports itself unavailable so
// that DSLA_IMPL_AUTO resolves to the CUDA-core kernel and DSLA_IMPL_TENSOR is refused.
#include "dsla_internal.cuh"

namespace dsla {
bool prefill_tc_available() { return false; }
size_t prefill_tc_workspace_bytes(const dsla_prefill_args*) { return 0; }
dsla_status launch_prefill_tc(const PrefillParams&, const dsla_prefill_args*, cudaStream_t) { return DSLA_ERR_UNSUPPORTED; }
}  // namespace dsla
