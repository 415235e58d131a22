// Shared host/device declarations of the library (internal).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lrd.h"

namespace lrd {

// Per-device host-side caches (function attributes set, occupancy answers, symbol addresses) are kept in tables
// indexed by the current device's ordinal; devices past the table share its last row.
constexpr int kMaxDevices = 16;
inline int device_slot() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) dev = 0;
    return dev < kMaxDevices ? dev : kMaxDevices - 1;
}

// Device address (on the current device) of the flag a bounded wait raises when it runs out (one word, zero = fine);
// nullptr if the address cannot be obtained.  Read and cleared by lrd_check_device_status().
unsigned int* device_timeout_flag();
lrd_status_t read_and_clear_device_timeout(bool* raised);
// One block whose bounded wait is left to run out (see lrd_selftest_wait_timeout).
lrd_status_t selftest_wait_runs_out(cudaStream_t stream);

// One matrix product  C[M x N] = op(A) op(B) (+ bias over columns), fp32 accumulate.
//   a_mn_major = false: A stored [M x K] (k contiguous);  true: A stored [K x M] (m contiguous)
//   b_mn_major = false: B stored [N x K] (k contiguous);  true: B stored [K x N] (n contiguous)
struct GemmArgs {
    int64_t M, N, K;
    const void* A; int64_t lda; bool a_mn_major;
    const void* B; int64_t ldb; bool b_mn_major;
    void* C; int64_t ldc;
    const void* bias;          // [N] or nullptr, same dtype as C
    void* a_colsum = nullptr;  // optional [M]: sum over k of A(m, k) (the bias gradient when A is dY); only on the
                               // tensor-core path with both operands MN-major, see tc_gemm_colsum_ok()
    lrd_dtype_t dtype;         // storage type of A, B, C, bias
    int max_cluster_split = 0; // split weight gradients: largest cluster to split the reduction over (0 = automatic).  A
                               // launch meant to run BESIDE others asks for 2: clusters of 4 or 8 need that many free
                               // SMs inside one GPC, which a chain kernel on 128 of the 148 SMs never leaves
};

// True when the CUDA call succeeded.  With the environment variable LRD_LOG_ERRORS set, a failure is also written to
// stderr with the call's name and CUDA's error string (the C ABI itself only returns LRD_ERR_CUDA).
bool cuda_ok(cudaError_t e, const char* what);

// Host-side count of kernels enqueued (see lrd_launch_count).
void count_launch(int n = 1);

inline size_t elem_size(int dtype) { return dtype == LRD_BF16 ? 2 : 4; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// General fp32-FMA path (any shape, any alignment).
lrd_status_t simt_gemm(const GemmArgs& g, cudaStream_t stream);
lrd_status_t simt_colsum(const void* A, int64_t lda, int64_t M, int64_t N, void* out, lrd_dtype_t dtype,
                         cudaStream_t stream);

// Column sums of A[M x N] (bias gradient), rows added in a fixed order.  With `scratch` of at least
// colsum_scratch_bytes(M, N) the sum runs in two stages over many blocks; without, in one kernel.
size_t colsum_scratch_bytes(int64_t M, int64_t N);
lrd_status_t colsum(const void* A, int64_t lda, int64_t M, int64_t N, void* out, lrd_dtype_t dtype, float* scratch,
                    size_t scratch_bytes, cudaStream_t stream);

// One product on the path chosen by `path` (an lrd_path_t): the tensor-core kernel when the
// operands qualify, else the general kernel.
lrd_status_t run_gemm(const GemmArgs& g, int path, bool allow_split, float* partials, size_t partial_bytes,
                      cudaStream_t s);
GemmArgs make_gemm(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, bool a_mn, const void* B, int64_t ldb,
                   bool b_mn, void* C, int64_t ldc, const void* bias, lrd_dtype_t dt);
lrd_status_t zero_fill(void* p, int64_t rows, int64_t cols, int64_t ld, lrd_dtype_t dt, cudaStream_t s);
// dst[row][0 .. cols_dst) = src[row][0 .. min(cols_src, cols_dst)) then zeros; bf16, any leading dimensions.
lrd_status_t copy2d_bf16(void* dst, int64_t ldd, const void* src, int64_t lds, int64_t rows, int64_t cols_src, int64_t cols_dst,
                         cudaStream_t s);

}  // namespace lrd
