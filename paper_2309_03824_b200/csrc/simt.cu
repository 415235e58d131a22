// General path: shared-memory tiled fp32-FMA matrix product for any shape, leading dimension and
// operand orientation, and a deterministic column sum.  Used for fp32 layers (which must not use
// reduced-precision tensor math) and for bf16 layers whose ranks or strides do not meet the
// 16-byte alignment the tensor-core path needs.
#include "common.cuh"
#include "conv.cuh"

namespace lrd {

__device__ unsigned int g_device_timeout = 0;

unsigned int* device_timeout_flag() {
    static unsigned int* ptr_on[kMaxDevices] = {};          // every device has its own copy of the symbol
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    void* p = nullptr;
    if (dev < 0 || dev >= kMaxDevices)                      // past the table: look it up every time
        return cudaGetSymbolAddress(&p, g_device_timeout) == cudaSuccess ? (unsigned int*)p : nullptr;
    if (!ptr_on[dev] && cudaGetSymbolAddress(&p, g_device_timeout) == cudaSuccess) ptr_on[dev] = (unsigned int*)p;
    return ptr_on[dev];
}

lrd_status_t read_and_clear_device_timeout(bool* raised) {
    unsigned int flag = 0;
    if (cudaMemcpyFromSymbol(&flag, g_device_timeout, sizeof(flag)) != cudaSuccess) return LRD_ERR_CUDA;
    *raised = flag != 0;
    if (flag) {
        const unsigned int zero = 0;
        if (cudaMemcpyToSymbol(g_device_timeout, &zero, sizeof(zero)) != cudaSuccess) return LRD_ERR_CUDA;
    }
    return LRD_OK;
}

namespace {

// 64 x 64 output tile, 64-deep k-tile: the layers that land here are small or oddly shaped, their grids a handful of
// blocks, and what a block waits for is the latency of a tile's loads -- a deep tile has fewer of those waits
// (16-deep tiles: 41 us for 256 x 512 -> 40 on 4 blocks).
constexpr int TM = 64, TN = 64, TK = 64, NT = 256;
constexpr int kFetch = TM * TK / NT;        // elements of each operand a thread brings in per tile

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Operand loaders: element (m, k) of A and (k, n) of B as fp32, zero outside the problem.
template <typename T> struct PlainA {          // [M x K] (k contiguous) or [K x M] (m contiguous)
    const T* p; int64_t ld; int mn;
    __device__ bool k_fastest() const { return !mn; }
    __device__ float operator()(int64_t m, int64_t k) const { return to_f32(mn ? p[k * ld + m] : p[m * ld + k]); }
};
template <typename T> struct PlainB {          // [N x K] (k contiguous) or [K x N] (n contiguous)
    const T* p; int64_t ld; int mn;
    __device__ bool k_fastest() const { return !mn; }
    __device__ float operator()(int64_t k, int64_t n) const { return to_f32(mn ? p[k * ld + n] : p[n * ld + k]); }
};
// k x k taps of an NHWC image as the A operand of the core's forward product: m = output pixel (b, ho, wo),
// kidx = tap * C + channel; the tap (kh, kw) of output pixel (ho, wo) is input pixel (ho * stride + kh - pad,
// wo * stride + kw - pad); pixels outside the image read as zero.
template <typename T> struct ConvFwdA {
    const T* p; ConvGeom g; int C;
    __device__ bool k_fastest() const { return true; }
    __device__ float operator()(int64_t m, int64_t kidx) const {
        const int t = (int)(kidx / C), c = (int)(kidx % C);
        const int wo = (int)(m % g.Wo), ho = (int)((m / g.Wo) % g.Ho);
        const int64_t b = m / ((int64_t)g.Wo * g.Ho);
        const int h = ho * g.stride + t / g.k - g.pad, w = wo * g.stride + t % g.k - g.pad;
        if (h < 0 || h >= g.H || w < 0 || w >= g.W) return 0.f;
        return to_f32(p[((b * g.H + h) * g.W + w) * C + c]);
    }
};
// The same taps seen from the input side, as the A operand of the data gradient: m = input pixel (b, h, w),
// kidx = tap * C + o; input pixel (h, w) met tap (kh, kw) of output pixel ((h + pad - kh) / stride,
// (w + pad - kw) / stride) where both divisions are exact and the result lies inside the output.
template <typename T> struct ConvBwdA {
    const T* p; ConvGeom g; int C;
    __device__ bool k_fastest() const { return true; }
    __device__ float operator()(int64_t m, int64_t kidx) const {
        const int t = (int)(kidx / C), c = (int)(kidx % C);
        const int w = (int)(m % g.W), h = (int)((m / g.W) % g.H);
        const int64_t b = m / ((int64_t)g.W * g.H);
        const int hs = h + g.pad - t / g.k, ws = w + g.pad - t % g.k;
        if (hs < 0 || ws < 0 || hs % g.stride || ws % g.stride) return 0.f;
        const int ho = hs / g.stride, wo = ws / g.stride;
        if (ho >= g.Ho || wo >= g.Wo) return 0.f;
        return to_f32(p[((b * g.Ho + ho) * g.Wo + wo) * C + c]);
    }
};
// One tap of an NHWC image as the B operand of the filter gradient: kidx = output pixel, n = channel.
template <typename T> struct ConvTapB {
    const T* p; ConvGeom g; int C, kh, kw;
    __device__ bool k_fastest() const { return false; }
    __device__ float operator()(int64_t kidx, int64_t n) const {
        const int wo = (int)(kidx % g.Wo), ho = (int)((kidx / g.Wo) % g.Ho);
        const int64_t b = kidx / ((int64_t)g.Wo * g.Ho);
        const int h = ho * g.stride + kh - g.pad, w = wo * g.stride + kw - g.pad;
        if (h < 0 || h >= g.H || w < 0 || w >= g.W) return 0.f;
        return to_f32(p[((b * g.H + h) * g.W + w) * C + n]);
    }
};
// The core G[o][tap][i] as the B operand of the data gradient: kidx = tap * Co + o, n = i.
template <typename T> struct CoreTransposedB {
    const T* p; int Ci, Co, taps;
    __device__ bool k_fastest() const { return false; }
    __device__ float operator()(int64_t kidx, int64_t n) const {
        const int64_t t = kidx / Co, o = kidx % Co;
        return to_f32(p[(o * taps + t) * Ci + n]);
    }
};

template <typename T, typename LA, typename LB>
__global__ void __launch_bounds__(NT) simt_gemm_kernel(int64_t M, int64_t N, int64_t K, const LA la, const LB lb,
                                                       T* __restrict__ C, int64_t ldc, const T* __restrict__ bias) {
    __shared__ float As[TK][TM + 4];
    __shared__ float Bs[TK][TN + 4];
    const int t = threadIdx.x;
    const int64_t m0 = (int64_t)blockIdx.y * TM, n0 = (int64_t)blockIdx.x * TN;
    const int tx = t % 16, ty = t / 16;  // thread computes rows ty*4.., cols tx*4..
    float acc[4][4] = {};
    // The next tile's elements are fetched into registers before the current tile is multiplied: their global-memory
    // latency then runs beside the arithmetic instead of in front of it (the order of the additions is unchanged).
    float ra[kFetch], rb[kFetch];
    auto fetch = [&](int64_t k0) {
#pragma unroll
        for (int i = 0; i < kFetch; ++i) {
            int mm, kk;
            if (la.k_fastest()) { mm = t / 16 + 16 * (i % 4); kk = t % 16 + 16 * (i / 4); } else { kk = t / 64 + 4 * i; mm = t % 64; }
            const int64_t m = m0 + mm, k = k0 + kk;
            ra[i] = (m < M && k < K) ? la(m, k) : 0.f;
            int nn;
            if (lb.k_fastest()) { nn = t / 16 + 16 * (i % 4); kk = t % 16 + 16 * (i / 4); } else { kk = t / 64 + 4 * i; nn = t % 64; }
            const int64_t n = n0 + nn, kb = k0 + kk;
            rb[i] = (n < N && kb < K) ? lb(kb, n) : 0.f;
        }
    };
    fetch(0);
    for (int64_t k0 = 0; k0 < K; k0 += TK) {
#pragma unroll
        for (int i = 0; i < kFetch; ++i) {
            int mm, kk;
            if (la.k_fastest()) { mm = t / 16 + 16 * (i % 4); kk = t % 16 + 16 * (i / 4); } else { kk = t / 64 + 4 * i; mm = t % 64; }
            As[kk][mm] = ra[i];
            int nn;
            if (lb.k_fastest()) { nn = t / 16 + 16 * (i % 4); kk = t % 16 + 16 * (i / 4); } else { kk = t / 64 + 4 * i; nn = t % 64; }
            Bs[kk][nn] = rb[i];
        }
        __syncthreads();
        if (k0 + TK < K) fetch(k0 + TK);
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t n = n0 + tx * 4 + j;
            if (n >= N) continue;
            float v = acc[i][j];
            if (bias) v += to_f32(bias[n]);
            C[m * ldc + n] = from_f32<T>(v);
        }
    }
}

// out[n] = sum_m A[m][n], rows added in a fixed order (thread-strided partials, then a tree in
// shared memory whose shape does not depend on timing).
template <typename T>
__global__ void __launch_bounds__(256) simt_colsum_kernel(const T* __restrict__ A, int64_t lda, int64_t M, int64_t N,
                                                          T* __restrict__ out) {
    __shared__ float part[8][33];
    const int c = threadIdx.x % 32, g = threadIdx.x / 32;
    const int64_t n = (int64_t)blockIdx.x * 32 + c;
    float s = 0.f;
    if (n < N)
        for (int64_t m = g; m < M; m += 8) s += to_f32(A[m * lda + n]);
    part[g][c] = s;
    __syncthreads();
    if (g == 0 && n < N) {
        float tot = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) tot += part[i][c];
        out[n] = from_f32<T>(tot);
    }
}

// Two-stage column sum for tall matrices: stage 1 adds the rows of one of S row ranges for 64 columns
// (4 row lanes per column, fixed order), stage 2 adds the S partial rows in ascending order.
template <typename T>
__global__ void __launch_bounds__(256) colsum_stage1_kernel(const T* __restrict__ A, int64_t lda, int64_t M, int64_t N,
                                                            int64_t rows_per_split, float* __restrict__ partial) {
    __shared__ float part[4][64];
    const int c = threadIdx.x % 64, g = threadIdx.x / 64;
    const int64_t n = (int64_t)blockIdx.x * 64 + c;
    const int64_t m_begin = (int64_t)blockIdx.y * rows_per_split;
    const int64_t m_end = m_begin + rows_per_split < M ? m_begin + rows_per_split : M;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    if (n < N) {
        int64_t m = m_begin + g;
        for (; m + 12 < m_end; m += 16) {          // four independent loads in flight per thread
            s0 += to_f32(A[m * lda + n]);
            s1 += to_f32(A[(m + 4) * lda + n]);
            s2 += to_f32(A[(m + 8) * lda + n]);
            s3 += to_f32(A[(m + 12) * lda + n]);
        }
        for (; m < m_end; m += 4) s0 += to_f32(A[m * lda + n]);
    }
    part[g][c] = (s0 + s1) + (s2 + s3);
    __syncthreads();
    if (g == 0 && n < N) partial[(int64_t)blockIdx.y * N + n] = (part[0][c] + part[1][c]) + (part[2][c] + part[3][c]);
}

template <typename T>
__global__ void __launch_bounds__(256) colsum_stage2_kernel(const float* __restrict__ partial, int splits, int64_t N,
                                                            T* __restrict__ out) {
    const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N) return;
    float tot = 0.f;
    for (int z = 0; z < splits; ++z) tot += partial[(int64_t)z * N + n];
    out[n] = from_f32<T>(tot);
}

template <typename T>
lrd_status_t colsum_two_stage_t(const void* A, int64_t lda, int64_t M, int64_t N, void* out, float* scratch, int splits,
                                cudaStream_t stream) {
    const int64_t rows = (M + splits - 1) / splits;
    dim3 grid((unsigned)((N + 63) / 64), (unsigned)splits);
    colsum_stage1_kernel<T><<<grid, 256, 0, stream>>>((const T*)A, lda, M, N, rows, scratch);
    colsum_stage2_kernel<T><<<(unsigned)((N + 255) / 256), 256, 0, stream>>>(scratch, splits, N, (T*)out);
    count_launch(2);
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

template <typename T>
lrd_status_t simt_gemm_t(const GemmArgs& g, cudaStream_t stream) {
    dim3 grid((unsigned)((g.N + TN - 1) / TN), (unsigned)((g.M + TM - 1) / TM));
    PlainA<T> la{(const T*)g.A, g.lda, g.a_mn_major};
    PlainB<T> lb{(const T*)g.B, g.ldb, g.b_mn_major};
    simt_gemm_kernel<T><<<grid, NT, 0, stream>>>(g.M, g.N, g.K, la, lb, (T*)g.C, g.ldc, (const T*)g.bias);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

template <typename T>
lrd_status_t conv_fwd_t(const void* in, const void* G, void* out, int64_t B, const ConvGeom& g, int ci, int co, cudaStream_t stream) {
    // M = output pixels, N = co, K = taps * ci, B = G as [co x taps * ci] (k contiguous)
    const int64_t P = B * g.Ho * g.Wo, K = (int64_t)g.k * g.k * ci;
    dim3 grid((unsigned)((co + TN - 1) / TN), (unsigned)((P + TM - 1) / TM));
    ConvFwdA<T> la{(const T*)in, g, ci};
    PlainB<T> lb{(const T*)G, K, 0};
    simt_gemm_kernel<T><<<grid, NT, 0, stream>>>(P, co, K, la, lb, (T*)out, co, (const T*)nullptr);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

template <typename T>
lrd_status_t conv_bwd_data_t(const void* dout, const void* G, void* din, int64_t B, const ConvGeom& g, int ci, int co,
                             cudaStream_t stream) {
    // M = input pixels, N = ci, K = taps * co, B = G regrouped as (tap, o) x i
    const int64_t P = B * g.H * g.W, K = (int64_t)g.k * g.k * co;
    dim3 grid((unsigned)((ci + TN - 1) / TN), (unsigned)((P + TM - 1) / TM));
    ConvBwdA<T> la{(const T*)dout, g, co};
    CoreTransposedB<T> lb{(const T*)G, ci, co, g.k * g.k};
    simt_gemm_kernel<T><<<grid, NT, 0, stream>>>(P, ci, K, la, lb, (T*)din, ci, (const T*)nullptr);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

template <typename T>
lrd_status_t conv_filter_t(const void* dout, const void* in, void* dG, int64_t B, const ConvGeom& g, int ci, int co,
                           cudaStream_t stream) {
    const int taps = g.k * g.k;
    const int64_t P = B * g.Ho * g.Wo;
    dim3 grid((unsigned)((ci + TN - 1) / TN), (unsigned)((co + TM - 1) / TM));
    for (int t = 0; t < taps; ++t) {   // one product per tap: M = co, N = ci, K = output pixels (single block owns all of K)
        PlainA<T> la{(const T*)dout, co, 1};
        ConvTapB<T> lb{(const T*)in, g, ci, t / g.k, t % g.k};
        simt_gemm_kernel<T><<<grid, NT, 0, stream>>>(co, ci, P, la, lb, (T*)dG + (int64_t)t * ci, (int64_t)taps * ci,
                                                     (const T*)nullptr);
    }
    count_launch(taps);
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

}  // namespace

lrd_status_t simt_gemm(const GemmArgs& g, cudaStream_t stream) {
    if (g.M <= 0 || g.N <= 0) return LRD_OK;
    return g.dtype == LRD_F32 ? simt_gemm_t<float>(g, stream) : simt_gemm_t<__nv_bfloat16>(g, stream);
}

lrd_status_t simt_conv_fwd(const void* in, const void* G, void* out, int64_t B, const ConvGeom& g, int64_t ci, int64_t co,
                           lrd_dtype_t dt, cudaStream_t s) {
    return dt == LRD_F32 ? conv_fwd_t<float>(in, G, out, B, g, (int)ci, (int)co, s)
                         : conv_fwd_t<__nv_bfloat16>(in, G, out, B, g, (int)ci, (int)co, s);
}
lrd_status_t simt_conv_bwd_data(const void* dout, const void* G, void* din, int64_t B, const ConvGeom& g, int64_t ci,
                                int64_t co, lrd_dtype_t dt, cudaStream_t s) {
    return dt == LRD_F32 ? conv_bwd_data_t<float>(dout, G, din, B, g, (int)ci, (int)co, s)
                         : conv_bwd_data_t<__nv_bfloat16>(dout, G, din, B, g, (int)ci, (int)co, s);
}
lrd_status_t simt_conv_bwd_filter(const void* dout, const void* in, void* dG, int64_t B, const ConvGeom& g, int64_t ci,
                                  int64_t co, lrd_dtype_t dt, cudaStream_t s) {
    return dt == LRD_F32 ? conv_filter_t<float>(dout, in, dG, B, g, (int)ci, (int)co, s)
                         : conv_filter_t<__nv_bfloat16>(dout, in, dG, B, g, (int)ci, (int)co, s);
}

int colsum_splits(int64_t M) {
    int64_t s = M / 64;
    return (int)(s < 1 ? 1 : (s > 64 ? 64 : s));
}

size_t colsum_scratch_bytes(int64_t M, int64_t N) {
    const int s = colsum_splits(M);
    return s > 1 ? align_up((size_t)s * (size_t)N * sizeof(float), 256) : 0;
}

lrd_status_t colsum(const void* A, int64_t lda, int64_t M, int64_t N, void* out, lrd_dtype_t dtype, float* scratch,
                    size_t scratch_bytes, cudaStream_t stream) {
    if (N <= 0) return LRD_OK;
    const int s = colsum_splits(M);
    if (s > 1 && scratch && scratch_bytes >= (size_t)s * (size_t)N * sizeof(float))
        return dtype == LRD_F32 ? colsum_two_stage_t<float>(A, lda, M, N, out, scratch, s, stream)
                                : colsum_two_stage_t<__nv_bfloat16>(A, lda, M, N, out, scratch, s, stream);
    return simt_colsum(A, lda, M, N, out, dtype, stream);
}

lrd_status_t simt_colsum(const void* A, int64_t lda, int64_t M, int64_t N, void* out, lrd_dtype_t dtype,
                         cudaStream_t stream) {
    if (N <= 0) return LRD_OK;
    const unsigned grid = (unsigned)((N + 31) / 32);
    if (dtype == LRD_F32)
        simt_colsum_kernel<float><<<grid, 256, 0, stream>>>((const float*)A, lda, M, N, (float*)out);
    else
        simt_colsum_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>((const __nv_bfloat16*)A, lda, M, N,
                                                                     (__nv_bfloat16*)out);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

}  // namespace lrd

// ---- bias gradient without any caller-provided or allocated scratch -----------------------------------
// The partial column sums of the two-stage kernels live in a file-scope device array, so a caller
// that may not allocate device memory can still get the many-block version.
namespace {

constexpr int64_t kNoAllocMaxN = 8192;                           // widest dY this entry point accepts
constexpr int kNoAllocMaxSplits = 64;
constexpr size_t kNoAllocFloats = (size_t)kNoAllocMaxN * kNoAllocMaxSplits;   // 2 MiB per GPU that loads the library
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocFloats];

constexpr int kNoallocMaxDevices = 64;
float* g_noalloc_ptr[kNoallocMaxDevices] = {};                          // device address of the array, per device

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel can use:
// the device address is asked for once per device (with that device current) and cached.
lrd_status_t noalloc_scratch(float** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoallocMaxDevices) return LRD_ERR_CUDA;
    if (!g_noalloc_ptr[dev]) {
        float* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return LRD_ERR_CUDA;
        g_noalloc_ptr[dev] = ptr;
    }
    *out = g_noalloc_ptr[dev];
    return LRD_OK;
}

}  // namespace

extern "C" lrd_status_t lrd_bias_grad_noalloc(const void* dY, int64_t ldy, int64_t M, int64_t N, void* dbias,
                                              lrd_dtype_t dtype, void* cuda_stream) {
    if (M < 0 || N < 1 || (dtype != LRD_F32 && dtype != LRD_BF16)) return LRD_ERR_INVALID_ARG;
    if (!dbias || (M > 0 && !dY)) return LRD_ERR_INVALID_ARG;
    if (ldy == 0) ldy = N;
    if (ldy < N) return LRD_ERR_INVALID_ARG;
    if (N > kNoAllocMaxN) return LRD_ERR_TOO_LARGE;
    const size_t e = lrd::elem_size(dtype);
    if (((uintptr_t)dbias % e) || ((uintptr_t)dY % e)) return LRD_ERR_ALIGNMENT;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return LRD_ERR_CUDA;
    if (major != 10) return LRD_ERR_ARCH;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (M == 0) return cudaMemsetAsync(dbias, 0, (size_t)N * e, stream) == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
    float* scratch = nullptr;
    const lrd_status_t st = noalloc_scratch(&scratch);
    if (st != LRD_OK) return st;
    // Same kernels and same row split as the workspace path (splits <= 64, so the partial sums fit);
    // stage 1 writes every partial that stage 2 reads, so nothing left by an earlier call is ever used.
    const int splits = lrd::colsum_splits(M);
    return dtype == LRD_F32 ? lrd::colsum_two_stage_t<float>(dY, ldy, M, N, dbias, scratch, splits, stream)
                            : lrd::colsum_two_stage_t<__nv_bfloat16>(dY, ldy, M, N, dbias, scratch, splits, stream);
}
