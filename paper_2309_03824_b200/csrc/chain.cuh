// Fused two-product chain  Out[M x N2] = (In[M x K1] P[K1 x r]) Q[N2 x r]^T (+ bias)  with the
// rank-r intermediate T[M x r] kept on chip (tensor memory -> bf16 -> shared memory), written to
// memory only when the caller asks for it (T_save).  The forward pass is the chain (X, V, U),
// the backward data pass is the chain (dY, U, V).
#pragma once
#include "common.cuh"

namespace lrd {

struct ChainArgs {
    int64_t M, K1, r, N2;
    const void* In; int64_t ld_in;     // [M x K1]
    const void* P; int64_t ldp;        // [K1 x r]
    const void* Q; int64_t ldq;        // [N2 x r]
    const void* bias;                  // [N2] or nullptr
    void* Out; int64_t ld_out;         // [M x N2]
    void* T_save; int64_t ldt;         // [M x r] or nullptr
    lrd_dtype_t dtype;
    int sm_share = 0;                  // SMs this launch can count on when it runs beside others (0: all of them)
};

// Overrides of the launch shape for benchmarking sweeps: cluster size, k-blocks per phase-1 stage,
// phase-2 chunk width.  0 = automatic.  Not thread-safe against concurrent launches.
void chain_tuning(int C, int G1, int BN2);
bool chain_eligible(const ChainArgs& c);
// Eligible, and expected to beat the two separate products (the automatic path's test).
bool chain_preferred(const ChainArgs& c);
lrd_status_t chain_launch(const ChainArgs& c, cudaStream_t stream);

// The same chain on pairs of SMs (tcgen05 cta_group::2): a cluster of 2 S blocks owns 256 rows.  `layers` are
// n <= kChainMaxLayers independent layers of equal shape that run in one launch (gridDim.z).  Needs more than
// 128 rows and a rank that splits into S slices of whole 32-column groups.
constexpr int kChainMaxLayers = 4;
// Overrides for sweeps and tests: pairs per cluster (1-4), k-blocks per phase-1 stage, phase-2 chunk width; 0 = automatic.
void chain_pair_tuning(int S, int G1, int BN2);
bool chain_pair_eligible(const ChainArgs* layers, int n);
bool chain_pair_preferred(const ChainArgs* layers, int n);
bool chain_pair_roomy(const ChainArgs* layers, int n);
lrd_status_t chain_pair_launch(const ChainArgs* layers, int n, cudaStream_t stream);

}  // namespace lrd
