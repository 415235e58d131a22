// Internal interface of the tensor-core (tcgen05) kernels.
#pragma once
#include "common.cuh"

namespace lrd {

constexpr int kNumSms = 148;   // B200: tile and split choices are made against this count

// bf16, 16-byte aligned bases, leading dimensions multiples of 8 elements.
bool tc_gemm_eligible(const GemmArgs& g);
int tc_pick_bn(int64_t M, int64_t N);
int tc_pick_splits(int64_t M, int64_t N, int64_t K);
// fp32 partial-tile scratch a split product of this shape needs (0 when it is not split).
size_t tc_split_workspace_bytes(int64_t M, int64_t N, int64_t K);
// True when tc_gemm can also deliver g.a_colsum for this product (bf16, both operands MN-major, aligned).
bool tc_gemm_colsum_ok(const GemmArgs& g);
// Unsplit product with a bf16 result on the persistent kernel (one block per SM walks over the tiles, the
// epilogue of a tile overlaps the MMAs of the next).  Same eligibility as tc_gemm; no column sums.
lrd_status_t tc_gemm_persistent(const GemmArgs& g, cudaStream_t stream);
void tc_gemm_persistent_force_pairs(int blocks_per_mma);     // 0: automatic; 1 or 2: forced where the shape allows
// allow_split: the reduction dimension may be split over blocks (weight gradients).
lrd_status_t tc_gemm(const GemmArgs& g, bool allow_split, float* partials, size_t partial_bytes, cudaStream_t stream);

}  // namespace lrd
