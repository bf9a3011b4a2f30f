// tcgen05 / TMEM chunk-wise GKA forward (bf16 operands, fp32 accumulation) for sm_100a.
#include "gka_common.cuh"

namespace gka {

bool fwd_tc_available() { return false; }

cudaError_t launch_fwd_tc(const FwdArgs &, cudaStream_t) { return cudaErrorNotSupported; }

}  // namespace gka
