#include "chain.cuh"

namespace lrd {
bool chain_eligible(const ChainArgs&) { return false; }
lrd_status_t chain_launch(const ChainArgs&, cudaStream_t) { return LRD_ERR_UNSUPPORTED; }
}  // namespace lrd
