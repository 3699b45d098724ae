// Tensor-core (tcgen05 + TMA) kernels: placeholder until the sm_100a kernels land.
#include "common.cuh"

namespace linattn {
bool umma_supported(const Problem&) { return false; }
size_t umma_partial_bytes(const Problem&) { return 0; }
int umma_state(const Problem&, const void*, const void*, float*, bool, void*, cudaStream_t) { return LINATTN_ERR_UNSUPPORTED; }
int umma_apply(const Problem&, const void*, const float*, void*, float, cudaStream_t) { return LINATTN_ERR_UNSUPPORTED; }
}  // namespace linattn
