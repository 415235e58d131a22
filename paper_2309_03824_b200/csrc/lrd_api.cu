// C-ABI entry points: argument checks, freeze-mask dispatch and path selection.  Every step of
// the layer runs in this library's own kernels; nothing here falls back to the host.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "chain.cuh"
#include "common.cuh"
#include "conv.cuh"
#include "streams.cuh"
#include "tc.cuh"

using namespace lrd;

namespace {

std::atomic<int> g_path{LRD_PATH_AUTO};
std::atomic<int> g_chain_mma_blocks{0};     // 0: automatic; 1: single-block chain only; 2: the chain on pairs of SMs wherever it is eligible
std::atomic<uint64_t> g_launches{0};

lrd_status_t check_arch() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LRD_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return LRD_ERR_CUDA;
    return major == 10 ? LRD_OK : LRD_ERR_ARCH;
}

bool elem_aligned(const void* p, int dtype) { return ((uintptr_t)p % elem_size(dtype)) == 0; }

struct Linear {
    int64_t M, K, N, r, ldx, ldv, ldu, ldy, ldz;
    lrd_dtype_t dt;
};

lrd_status_t parse_linear(const lrd_linear_desc_t* d, Linear* L, bool dense) {
    if (!d) return LRD_ERR_INVALID_ARG;
    if (d->M < 0 || d->K < 1 || d->N < 1) return LRD_ERR_INVALID_ARG;
    if (d->dtype != LRD_F32 && d->dtype != LRD_BF16) return LRD_ERR_INVALID_ARG;
    L->M = d->M; L->K = d->K; L->N = d->N; L->dt = (lrd_dtype_t)d->dtype;
    if (dense) {
        L->r = 0;
        L->ldv = d->ldv ? d->ldv : d->K;
        if (L->ldv < d->K) return LRD_ERR_INVALID_ARG;
        L->ldu = L->ldz = 0;
    } else {
        if (d->r < 1 || d->r > (d->K < d->N ? d->K : d->N)) return LRD_ERR_BAD_RANK;
        L->r = d->r;
        L->ldv = d->ldv ? d->ldv : d->r;
        L->ldu = d->ldu ? d->ldu : d->r;
        L->ldz = d->ldz ? d->ldz : d->r;
        if (L->ldv < d->r || L->ldu < d->r || L->ldz < d->r) return LRD_ERR_INVALID_ARG;
    }
    L->ldx = d->ldx ? d->ldx : d->K;
    L->ldy = d->ldy ? d->ldy : d->N;
    if (L->ldx < d->K || L->ldy < d->N) return LRD_ERR_INVALID_ARG;
    return LRD_OK;
}

lrd_status_t check_ws(const void* ws, size_t have, size_t need) {
    if (need == 0) return LRD_OK;
    if (!ws || have < need) return LRD_ERR_WORKSPACE;
    if ((uintptr_t)ws % 256) return LRD_ERR_ALIGNMENT;
    return LRD_OK;
}

lrd_status_t run_gemm(const GemmArgs& g, bool allow_split, float* partials, size_t partial_bytes, cudaStream_t s) {
    return lrd::run_gemm(g, g_path.load(), allow_split, partials, partial_bytes, s);
}
GemmArgs gemm(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, bool a_mn, const void* B, int64_t ldb,
              bool b_mn, void* C, int64_t ldc, const void* bias, lrd_dtype_t dt) {
    return make_gemm(M, N, K, A, lda, a_mn, B, ldb, b_mn, C, ldc, bias, dt);
}

// The fused chain for one layer, or for n layers of equal shape in one launch: on pairs of SMs where the shape
// allows, else (one layer only) on single blocks.  Returns LRD_ERR_UNSUPPORTED when no fused kernel takes it.
lrd_status_t launch_chain(const ChainArgs* c, int n, int path, cudaStream_t s, bool leave_room = false) {
    const int mode = g_chain_mma_blocks.load();
    const bool forced = path == LRD_PATH_FUSED;
    if (c[0].sm_share == 0 && mode != 1) {
        if (mode == 2 || forced ? chain_pair_eligible(c, n) : (chain_pair_preferred(c, n) || (leave_room && chain_pair_roomy(c, n))))
            return chain_pair_launch(c, n, s);
    }
    if (n != 1 || mode == 2) return LRD_ERR_UNSUPPORTED;
    if (forced ? chain_eligible(c[0]) : chain_preferred(c[0])) return chain_launch(c[0], s);
    return LRD_ERR_UNSUPPORTED;
}

ChainArgs fwd_chain_args(const Linear& L, const void* X, const void* V, const void* U, const void* bias, void* Y, void* Z_save,
                         int sm_share) {
    ChainArgs c;
    c.M = L.M; c.K1 = L.K; c.r = L.r; c.N2 = L.N;
    c.In = X; c.ld_in = L.ldx; c.P = V; c.ldp = L.ldv; c.Q = U; c.ldq = L.ldu; c.bias = bias;
    c.Out = Y; c.ld_out = L.ldy; c.T_save = Z_save; c.ldt = L.ldz; c.dtype = L.dt;
    c.sm_share = sm_share;
    return c;
}

ChainArgs bwd_chain_args(const Linear& L, const void* dY, const void* V, const void* U, void* dX, void* dZ_save, int sm_share) {
    ChainArgs c;
    c.M = L.M; c.K1 = L.N; c.r = L.r; c.N2 = L.K;
    c.In = dY; c.ld_in = L.ldy; c.P = U; c.ldp = L.ldu; c.Q = V; c.ldq = L.ldv; c.bias = nullptr;
    c.Out = dX; c.ld_out = L.ldx; c.T_save = dZ_save; c.ldt = L.r; c.dtype = L.dt;
    c.sm_share = sm_share;
    return c;
}

// A bf16 layer whose factors are stored with leading dimensions that are not multiples of 8 elements (an unquantized
// rank stored packed: rows start at addresses that are not multiples of 16 bytes) cannot feed TMA or the MMA
// descriptors directly.  Its factors are small -- r (K + N) elements -- so they are copied into the workspace with
// the rank rounded up to a multiple of 16 and zero columns, the layer runs on the tensor-core kernels at the padded
// rank (the zero columns add nothing), and Z / dU / dV are copied between the caller's packed layout and padded
// buffers.  The rank itself is unchanged: this is what an odd rank costs on this hardware beside a rounded one.
bool needs_repack(const Linear& L) { return L.dt == LRD_BF16 && L.r > 0 && (L.ldv % 8 || L.ldu % 8 || L.ldz % 8); }
int64_t padded_rank(const Linear& L) { return (L.r + 15) / 16 * 16; }
lrd_linear_desc_t padded_desc(const lrd_linear_desc_t& d, const Linear& L) {
    lrd_linear_desc_t q = d;
    q.r = padded_rank(L);
    q.ldv = q.ldu = q.ldz = q.r;
    q.ldx = L.ldx; q.ldy = L.ldy;
    return q;
}
struct RepackLayout {           // offsets into the workspace, behind the padded layer's own workspace
    size_t inner, Vp, Up, Zp, dUp, dVp, total;
};
RepackLayout repack_layout(const Linear& L, size_t inner_bytes) {
    const size_t rp = (size_t)padded_rank(L), e = 2;
    RepackLayout o;
    o.inner = 0;
    o.Vp = align_up(inner_bytes, 256);
    o.Up = o.Vp + align_up((size_t)L.K * rp * e, 256);
    o.Zp = o.Up + align_up((size_t)L.N * rp * e, 256);
    o.dUp = o.Zp + align_up((size_t)(L.M > 0 ? L.M : 1) * rp * e, 256);
    o.dVp = o.dUp + align_up((size_t)L.N * rp * e, 256);
    o.total = o.dVp + align_up((size_t)L.K * rp * e, 256);
    return o;
}

size_t linear_z_bytes(const Linear& L) { return align_up((size_t)(L.M > 0 ? L.M : 1) * L.r * elem_size(L.dt), 256); }

size_t linear_grad_scratch_bytes(const Linear& L) {     // dU, dV and dbias of one step, in the parameters' layouts
    const size_t e = elem_size(L.dt);
    return align_up((size_t)L.N * L.ldu * e, 256) + align_up((size_t)L.K * L.ldv * e, 256) + align_up((size_t)L.N * e, 256);
}

size_t linear_split_bytes(const Linear& L) {     // scratch after dZ: split partials of dU / dV, partial column sums
    if (L.M < 1) return 0;
    size_t need = colsum_scratch_bytes(L.M, L.N);
    if (L.dt == LRD_BF16) {
        const size_t a = tc_split_workspace_bytes(L.N, L.r, L.M), b = tc_split_workspace_bytes(L.K, L.r, L.M);
        need = need > a ? need : a;
        need = need > b ? need : b;
    }
    return need;
}

#define LRD_TRY(expr)                          \
    do {                                       \
        lrd_status_t st__ = (expr);            \
        if (st__ != LRD_OK) return st__;       \
    } while (0)

}  // namespace

namespace lrd {

void count_launch(int n) { g_launches.fetch_add((uint64_t)n); }

bool cuda_ok(cudaError_t e, const char* what) {
    if (e == cudaSuccess) return true;
    static const bool log = getenv("LRD_LOG_ERRORS") != nullptr;
    if (log) fprintf(stderr, "lrd: %s failed: %s\n", what, cudaGetErrorString(e));
    return false;
}

lrd_status_t run_gemm(const GemmArgs& g, int path, bool allow_split, float* partials, size_t partial_bytes,
                      cudaStream_t s) {
    if (g.M <= 0 || g.N <= 0) return LRD_OK;
    if (path != LRD_PATH_GENERAL && tc_gemm_eligible(g)) return tc_gemm(g, allow_split, partials, partial_bytes, s);
    return simt_gemm(g, s);
}

lrd_status_t zero_fill(void* p, int64_t rows, int64_t cols, int64_t ld, lrd_dtype_t dt, cudaStream_t s) {
    if (!p || rows <= 0 || cols <= 0) return LRD_OK;
    const size_t e = elem_size(dt);
    return cudaMemset2DAsync(p, (size_t)ld * e, 0, (size_t)cols * e, (size_t)rows, s) == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

namespace {
// dst[row][col] += src[row][col] (both with leading dimension ld): fp32 sum, one rounding to the storage type.
template <typename T>
__global__ void add_into_kernel(T* __restrict__ dst, const T* __restrict__ src, int64_t rows, int64_t cols, int64_t ld) {
    const int64_t n = rows * cols;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t at = (i / cols) * ld + i % cols;
        dst[at] = (T)((float)dst[at] + (float)src[at]);
    }
}
}  // namespace

namespace {
// dst[row][0 .. cols_dst) = src[row][0 .. min(cols_src, cols_dst)) followed by zeros, 2-byte elements, any
// leading dimensions: the copy between a packed factor (rows that start at odd multiples of 2 bytes) and its copy
// with rows padded to whole 16-byte groups.
__global__ void copy2d_bf16_kernel(__nv_bfloat16* __restrict__ dst, int64_t ldd, const __nv_bfloat16* __restrict__ src, int64_t lds,
                                   int64_t rows, int64_t cols_src, int64_t cols_dst) {
    const int64_t n = rows * cols_dst;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / cols_dst, c = i % cols_dst;
        dst[r * ldd + c] = c < cols_src ? src[r * lds + c] : __float2bfloat16_rn(0.f);
    }
}
}  // namespace

lrd_status_t copy2d_bf16(void* dst, int64_t ldd, const void* src, int64_t lds, int64_t rows, int64_t cols_src, int64_t cols_dst,
                         cudaStream_t s) {
    if (rows <= 0 || cols_dst <= 0) return LRD_OK;
    const int64_t n = rows * cols_dst;
    const unsigned blocks = (unsigned)std::min<int64_t>((n + 255) / 256, 148 * 16);
    copy2d_bf16_kernel<<<blocks, 256, 0, s>>>((__nv_bfloat16*)dst, ldd, (const __nv_bfloat16*)src, lds, rows, cols_src, cols_dst);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

lrd_status_t add_into(void* dst, const void* src, int64_t rows, int64_t cols, int64_t ld, lrd_dtype_t dt, cudaStream_t s) {
    if (!dst || rows <= 0 || cols <= 0) return LRD_OK;
    const int64_t n = rows * cols;
    const unsigned blocks = (unsigned)std::min<int64_t>((n + 255) / 256, 148 * 8);
    if (dt == LRD_BF16)
        add_into_kernel<<<blocks, 256, 0, s>>>((__nv_bfloat16*)dst, (const __nv_bfloat16*)src, rows, cols, ld);
    else
        add_into_kernel<<<blocks, 256, 0, s>>>((float*)dst, (const float*)src, rows, cols, ld);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

GemmArgs make_gemm(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, bool a_mn, const void* B, int64_t ldb,
                   bool b_mn, void* C, int64_t ldc, const void* bias, lrd_dtype_t dt) {
    GemmArgs g;
    g.M = M; g.N = N; g.K = K; g.A = A; g.lda = lda; g.a_mn_major = a_mn; g.B = B; g.ldb = ldb; g.b_mn_major = b_mn;
    g.C = C; g.ldc = ldc; g.bias = bias; g.dtype = dt;
    return g;
}

}  // namespace lrd

extern "C" {

int64_t lrd_rank_quantize(int64_t r, int64_t multiple, lrd_round_t mode, int64_t K, int64_t N) {
    if (r < 1 || multiple < 1 || K < 1 || N < 1) return -(int64_t)LRD_ERR_INVALID_ARG;
    const int64_t lim = K < N ? K : N;
    const int64_t cap = lim / multiple * multiple;
    if (cap == 0) return -(int64_t)LRD_ERR_BAD_RANK;
    int64_t q;
    switch (mode) {
        case LRD_ROUND_UP: q = (r + multiple - 1) / multiple * multiple; break;
        case LRD_ROUND_DOWN: q = r / multiple * multiple; break;
        case LRD_ROUND_NEAREST: q = (2 * r + multiple) / (2 * multiple) * multiple; break;
        default: return -(int64_t)LRD_ERR_INVALID_ARG;
    }
    if (q < multiple) q = multiple;
    if (q > cap) q = cap;
    return q;
}

lrd_freeze_t lrd_freeze_for_epoch(int64_t e) { return (e % 2 == 0) ? LRD_FREEZE_V : LRD_FREEZE_U; }

lrd_tucker_freeze_t lrd_tucker_freeze_for_epoch(int64_t e) {
    return (e % 2 == 0) ? LRD_TK_FREEZE_FACTORS : LRD_TK_FREEZE_CORE;
}

uint32_t lrd_linear_bwd_plan(lrd_freeze_t f) {
    if (f != LRD_FREEZE_NONE && f != LRD_FREEZE_U && f != LRD_FREEZE_V) return 0;
    uint32_t plan = LRD_PLAN_DZ | LRD_PLAN_DX;
    if (f != LRD_FREEZE_U) plan |= LRD_PLAN_DU | LRD_PLAN_DB | LRD_PLAN_NEEDS_Z;
    if (f != LRD_FREEZE_V) plan |= LRD_PLAN_DV | LRD_PLAN_NEEDS_X;
    return plan;
}

int64_t lrd_rank_search(const double* t, int64_t n, int64_t R_min, double T_orig, double min_rel_drop, int* use_decomposed) {
    if (!t || n < 1 || R_min < 1 || !(min_rel_drop >= 0.0)) return -(int64_t)LRD_ERR_INVALID_ARG;
    // delta[i] = t[i + 1] - t[i] belongs to rank R_min + i, i = 0 .. n-2; with a threshold only drops of at
    // least min_rel_drop * t[i] count
    auto counts = [&](int64_t i) {
        const double d = t[i + 1] - t[i];
        return d > 0.0 && (min_rel_drop == 0.0 || d >= min_rel_drop * t[i]);
    };
    int64_t best = -1;
    if (n == 1) {
        best = 0;
    } else {
        for (int64_t i = n - 2; i >= 0 && best < 0; --i) {
            const double d = t[i + 1] - t[i];
            const bool above_left = i == 0 || d > t[i] - t[i - 1];
            const bool above_right = i == n - 2 || d > t[i + 2] - t[i + 1];
            if (above_left && above_right && counts(i)) best = i;
        }
        if (best < 0 && min_rel_drop == 0.0) {            // no peak: the global maximum, largest rank on ties
            double mx = t[1] - t[0];
            best = 0;
            for (int64_t i = 1; i <= n - 2; ++i) {
                const double d = t[i + 1] - t[i];
                if (d >= mx) { mx = d; best = i; }
            }
        } else if (best < 0) {                            // the largest drop among those that count; none: stay at R
            double mx = 0.0;
            for (int64_t i = 0; i <= n - 2; ++i) {
                const double d = t[i + 1] - t[i];
                if (counts(i) && (best < 0 || d >= mx)) { mx = d; best = i; }
            }
            if (best < 0) best = n - 1;
        }
    }
    if (use_decomposed) *use_decomposed = t[best] < T_orig ? 1 : 0;
    return R_min + best;
}

int64_t lrd_rank_multiple(const double* t, int64_t n, int64_t R_min, double min_rel_drop) {
    if (!t || n < 1 || R_min < 1 || !(min_rel_drop >= 0.0)) return -(int64_t)LRD_ERR_INVALID_ARG;
    int64_t g = 0;
    for (int64_t i = 0; i + 1 < n; ++i) {
        const double d = t[i + 1] - t[i];
        if (!(d > 0.0 && d >= min_rel_drop * t[i])) continue;
        int64_t a = g, b = R_min + i;                     // gcd
        while (b) { const int64_t r = a % b; a = b; b = r; }
        g = a;
    }
    return g > 0 ? g : 1;
}

int64_t lrd_svd_rank(int64_t C, int64_t S, double alpha) {
    if (C < 1 || S < 1 || !(alpha > 0.0)) return -(int64_t)LRD_ERR_INVALID_ARG;
    return (int64_t)floor((double)C * (double)S / (alpha * (double)(C + S)));
}

int64_t lrd_tucker_rank(int64_t C, int64_t S, int64_t k, double alpha, double beta, int64_t* r2) {
    if (C < 1 || S < 1 || k < 1 || !(alpha > 0.0) || !(beta > 0.0)) return -(int64_t)LRD_ERR_INVALID_ARG;
    const double q = ((double)C + beta * (double)S) / (beta * (double)k * (double)k);
    const int64_t r1 = (int64_t)floor(0.5 * (-q + sqrt(q * q + 4.0 * (double)C * (double)S / (beta * alpha))));
    if (r2) *r2 = (int64_t)floor(beta * (double)r1);
    return r1;
}

int64_t lrd_tucker_rank_min(int64_t C, int64_t S, int64_t k, double alpha, double beta) {
    return lrd_tucker_rank(C, S, k, alpha + 1.0, beta, nullptr);
}

const char* lrd_status_string(lrd_status_t s) {
    switch (s) {
        case LRD_OK: return "ok";
        case LRD_ERR_INVALID_ARG: return "invalid argument";
        case LRD_ERR_BAD_RANK: return "rank out of range";
        case LRD_ERR_ALIGNMENT: return "pointer not aligned";
        case LRD_ERR_WORKSPACE: return "workspace missing or too small";
        case LRD_ERR_UNSUPPORTED: return "unsupported geometry";
        case LRD_ERR_ARCH: return "device is not sm_100";
        case LRD_ERR_CUDA: return "CUDA call failed";
        case LRD_ERR_TIMEOUT: return "device-side wait timed out";
        case LRD_ERR_TOO_LARGE: return "size exceeds the fixed limit of this entry point";
    }
    return "unknown status";
}

uint64_t lrd_launch_count(void) { return g_launches.load(); }

lrd_status_t lrd_set_path(lrd_path_t path) {
    if (path < LRD_PATH_AUTO || path > LRD_PATH_FUSED) return LRD_ERR_INVALID_ARG;
    g_path.store((int)path);
    return LRD_OK;
}

lrd_status_t lrd_chain_tuning(int cluster_blocks, int kblocks_per_stage, int chunk_columns) {
    if (cluster_blocks < 0 || cluster_blocks > 4) return LRD_ERR_INVALID_ARG;
    if (kblocks_per_stage < 0 || kblocks_per_stage > 4) return LRD_ERR_INVALID_ARG;
    if (chunk_columns != 0 && chunk_columns != 64 && chunk_columns != 128 && chunk_columns != 192 && chunk_columns != 256) return LRD_ERR_INVALID_ARG;
    chain_tuning(cluster_blocks, kblocks_per_stage, chunk_columns);
    return LRD_OK;
}

lrd_status_t lrd_chain_pair_tuning(int blocks_per_mma, int pairs_per_cluster, int kblocks_per_stage, int chunk_columns) {
    if (blocks_per_mma < 0 || blocks_per_mma > 2) return LRD_ERR_INVALID_ARG;
    if (pairs_per_cluster < 0 || pairs_per_cluster > 4) return LRD_ERR_INVALID_ARG;
    if (kblocks_per_stage < 0 || kblocks_per_stage > 4) return LRD_ERR_INVALID_ARG;
    if (chunk_columns != 0 && chunk_columns != 64 && chunk_columns != 128 && chunk_columns != 192 && chunk_columns != 256) return LRD_ERR_INVALID_ARG;
    g_chain_mma_blocks.store(blocks_per_mma);
    chain_pair_tuning(pairs_per_cluster, kblocks_per_stage, chunk_columns);
    return LRD_OK;
}

lrd_status_t lrd_gemm_tuning(int blocks_per_mma) {
    if (blocks_per_mma < 0 || blocks_per_mma > 2) return LRD_ERR_INVALID_ARG;
    tc_gemm_persistent_force_pairs(blocks_per_mma);
    return LRD_OK;
}

lrd_status_t lrd_tucker2_overlap(int on) {
    tucker2_overlap(on != 0);
    return LRD_OK;
}

lrd_status_t lrd_check_device_status(void) {
    if (cudaDeviceSynchronize() != cudaSuccess) return LRD_ERR_CUDA;
    bool raised = false;
    if (read_and_clear_device_timeout(&raised) != LRD_OK) return LRD_ERR_CUDA;
    return raised ? LRD_ERR_TIMEOUT : LRD_OK;
}

lrd_status_t lrd_selftest_wait_timeout(void* cuda_stream) {
    LRD_TRY(check_arch());
    return selftest_wait_runs_out((cudaStream_t)cuda_stream);
}

size_t lrd_linear_workspace_bytes(const lrd_linear_desc_t* desc, lrd_freeze_t freeze, int is_bwd) {
    Linear L;
    if (parse_linear(desc, &L, false) != LRD_OK) return 0;
    if (needs_repack(L)) {
        const lrd_linear_desc_t q = padded_desc(*desc, L);
        return repack_layout(L, lrd_linear_workspace_bytes(&q, freeze, is_bwd)).total;
    }
    (void)freeze;
    if (!is_bwd) return linear_z_bytes(L);
    const size_t bwd = linear_z_bytes(L) + linear_split_bytes(L);
    if (is_bwd != 2) return bwd;
    return align_up(bwd, 256) + linear_grad_scratch_bytes(L);      // + one gradient of every kind, for lrd_linear_bwd_accumulate
}

size_t lrd_dense_workspace_bytes(const lrd_linear_desc_t* desc, int is_bwd) {
    Linear L;
    if (parse_linear(desc, &L, true) != LRD_OK) return 0;
    if (!is_bwd || L.M < 1) return 256;
    size_t need = colsum_scratch_bytes(L.M, L.N);
    if (L.dt == LRD_BF16) {
        const size_t a = tc_split_workspace_bytes(L.N, L.K, L.M);
        need = need > a ? need : a;
    }
    return 256 + need;
}

// One layer's forward on stream s.  sm_share: SMs the launch can count on beside concurrent launches (0: all).
static lrd_status_t linear_fwd_on(const lrd_linear_desc_t* desc, const void* X, const void* V, const void* U,
                                  const void* bias, void* Y, void* Z_save, lrd_freeze_t freeze, void* workspace,
                                  size_t workspace_bytes, cudaStream_t s, int sm_share, bool check_only = false) {
    Linear L;
    LRD_TRY(parse_linear(desc, &L, false));
    if (freeze != LRD_FREEZE_NONE && freeze != LRD_FREEZE_U && freeze != LRD_FREEZE_V) return LRD_ERR_INVALID_ARG;
    if (!X || !V || !U || !Y) return LRD_ERR_INVALID_ARG;
    if ((freeze == LRD_FREEZE_U) != (Z_save == nullptr)) return LRD_ERR_INVALID_ARG;
    const void* ptrs[] = {X, V, U, bias, Y, Z_save};
    for (const void* p : ptrs)
        if (p && !elem_aligned(p, L.dt)) return LRD_ERR_ALIGNMENT;
    LRD_TRY(check_ws(workspace, workspace_bytes, lrd_linear_workspace_bytes(desc, freeze, 0)));
    LRD_TRY(check_arch());
    if (L.M == 0 || check_only) return LRD_OK;

    if (needs_repack(L) && g_path.load() != LRD_PATH_GENERAL && L.ldx % 8 == 0 && L.ldy % 8 == 0) {
        const lrd_linear_desc_t q = padded_desc(*desc, L);
        const size_t inner = lrd_linear_workspace_bytes(&q, freeze, 0);
        const RepackLayout o = repack_layout(L, inner);
        uint8_t* w = (uint8_t*)workspace;
        LRD_TRY(copy2d_bf16(w + o.Vp, q.r, V, L.ldv, L.K, L.r, q.r, s));
        LRD_TRY(copy2d_bf16(w + o.Up, q.r, U, L.ldu, L.N, L.r, q.r, s));
        LRD_TRY(linear_fwd_on(&q, X, w + o.Vp, w + o.Up, bias, Y, Z_save ? w + o.Zp : nullptr, freeze, w, inner, s, sm_share));
        if (Z_save) LRD_TRY(copy2d_bf16(Z_save, L.ldz, w + o.Zp, q.r, L.M, L.r, L.r, s));
        return LRD_OK;
    }

    const int path = g_path.load();
    if (path == LRD_PATH_AUTO || path == LRD_PATH_FUSED) {
        const ChainArgs c = fwd_chain_args(L, X, V, U, bias, Y, Z_save, sm_share);
        const lrd_status_t st = launch_chain(&c, 1, path, s);
        if (st != LRD_ERR_UNSUPPORTED) return st;
    }
    void* Z = Z_save ? Z_save : workspace;
    const int64_t ldz = Z_save ? L.ldz : L.r;
    LRD_TRY(run_gemm(gemm(L.M, L.r, L.K, X, L.ldx, false, V, L.ldv, true, Z, ldz, nullptr, L.dt), false, nullptr, 0, s));
    return run_gemm(gemm(L.M, L.N, L.r, Z, ldz, false, U, L.ldu, false, Y, L.ldy, bias, L.dt), false, nullptr, 0, s);
}

static lrd_status_t lrd_linear_fwd_impl(const lrd_linear_desc_t* desc, const void* X, const void* V, const void* U,
                            const void* bias, void* Y, void* Z_save, lrd_freeze_t freeze, void* workspace,
                            size_t workspace_bytes, void* cuda_stream) {
    return linear_fwd_on(desc, X, V, U, bias, Y, Z_save, freeze, workspace, workspace_bytes, (cudaStream_t)cuda_stream, 0);
}

// One layer's backward on stream s.  With a side stream, the dU (+ db) product, which needs nothing the data
// chain produces, runs there beside the chain; the caller has made `side` wait for s's earlier work and makes s
// wait for `side` afterwards.  dV follows the chain (it reads the dZ the chain spills) and, when dU is computed too,
// dU as well (the two may share the split-K scratch).
static lrd_status_t linear_bwd_on(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* V,
                                  const void* U, const void* Z_save, void* dX, void* dU, void* dV, void* dbias,
                                  lrd_freeze_t freeze, void* workspace, size_t workspace_bytes, cudaStream_t s,
                                  cudaStream_t side, cudaEvent_t side_done, int sm_share, bool check_only = false,
                                  int parts = 3) {
    // parts: 1 = the data half (dZ, dX), 2 = the weight-gradient half (it reads the dZ the data half left in the
    // workspace when V is unfrozen), 3 = both
    const bool do_data = (parts & 1) != 0, do_w = (parts & 2) != 0;
    // Weight gradients that run beside other launches (the weights-only call, which exists for that, and the layers of
    // a group, which run beside each other) split their reduction over clusters of 2, which find room next to a
    // chain kernel; alone on the GPU (lrd_linear_bwd) the larger clusters are faster.  Measured on the BERT-base-shaped
    // block: step 188.1 us with clusters of up to 8 everywhere, 184.1 with 4, 179.4 with 2 (attention backward alone: 16.8
    // against 19.2 us).
    const int wsplit = (parts == 2 || sm_share > 0) ? 2 : 0;
    Linear L;
    LRD_TRY(parse_linear(desc, &L, false));
    const uint32_t plan = lrd_linear_bwd_plan(freeze);
    if (!plan) return LRD_ERR_INVALID_ARG;
    if (!dY || (do_data && (!V || !U))) return LRD_ERR_INVALID_ARG;
    if (do_w && (plan & LRD_PLAN_NEEDS_Z) && (!Z_save || !dU)) return LRD_ERR_INVALID_ARG;
    if (do_w && (plan & LRD_PLAN_NEEDS_X) && (!X || !dV)) return LRD_ERR_INVALID_ARG;
    const void* ptrs[] = {dY, X, V, U, Z_save, dX, dU, dV, dbias};
    for (const void* p : ptrs)
        if (p && !elem_aligned(p, L.dt)) return LRD_ERR_ALIGNMENT;
    LRD_TRY(check_ws(workspace, workspace_bytes, lrd_linear_workspace_bytes(desc, freeze, 1)));
    LRD_TRY(check_arch());
    if (check_only) return LRD_OK;

    // frozen factor: no product is launched; a gradient buffer the caller passed reads as zero
    if (do_w && !(plan & LRD_PLAN_DU)) {
        LRD_TRY(zero_fill(dU, L.N, L.r, L.ldu, L.dt, s));
        LRD_TRY(zero_fill(dbias, 1, L.N, L.N, L.dt, s));
    }
    if (do_w && !(plan & LRD_PLAN_DV)) LRD_TRY(zero_fill(dV, L.K, L.r, L.ldv, L.dt, s));
    if (L.M == 0) {                      // no tokens: the unfrozen gradients are sums over nothing
        if (do_w && (plan & LRD_PLAN_DU)) { LRD_TRY(zero_fill(dU, L.N, L.r, L.ldu, L.dt, s)); LRD_TRY(zero_fill(dbias, 1, L.N, L.N, L.dt, s)); }
        if (do_w && (plan & LRD_PLAN_DV)) LRD_TRY(zero_fill(dV, L.K, L.r, L.ldv, L.dt, s));
        return LRD_OK;
    }

    if (needs_repack(L) && g_path.load() != LRD_PATH_GENERAL && L.ldx % 8 == 0 && L.ldy % 8 == 0) {
        const lrd_linear_desc_t q = padded_desc(*desc, L);
        const size_t inner = lrd_linear_workspace_bytes(&q, freeze, 1);
        const RepackLayout o = repack_layout(L, inner);
        uint8_t* w = (uint8_t*)workspace;
        const bool du = do_w && (plan & LRD_PLAN_DU) != 0, dv = do_w && (plan & LRD_PLAN_DV) != 0;
        if (do_data) {
            LRD_TRY(copy2d_bf16(w + o.Vp, q.r, V, L.ldv, L.K, L.r, q.r, s));
            LRD_TRY(copy2d_bf16(w + o.Up, q.r, U, L.ldu, L.N, L.r, q.r, s));
        }
        if (du) LRD_TRY(copy2d_bf16(w + o.Zp, q.r, Z_save, L.ldz, L.M, L.r, q.r, s));
        // the frozen factor's buffers were zero-filled above; the padded call gets none for them
        LRD_TRY(linear_bwd_on(&q, dY, X, w + o.Vp, w + o.Up, w + o.Zp, dX, w + o.dUp, w + o.dVp, du ? dbias : nullptr, freeze, w, inner, s,
                              nullptr, nullptr, sm_share, false, parts));
        if (du) LRD_TRY(copy2d_bf16(dU, L.ldu, w + o.dUp, q.r, L.N, L.r, L.r, s));
        if (dv) LRD_TRY(copy2d_bf16(dV, L.ldv, w + o.dVp, q.r, L.K, L.r, L.r, s));
        return LRD_OK;
    }

    void* dZ = workspace;
    float* partials = (float*)((uint8_t*)workspace + linear_z_bytes(L));
    const size_t partial_bytes = workspace_bytes - linear_z_bytes(L);
    const bool need_dz_in_memory = (plan & LRD_PLAN_DV) != 0;

    bool chained = !do_data;             // the data half (dX, and dZ where needed) has run already, or runs in a later call
    const int path = g_path.load();
    if (!chained && dX && (path == LRD_PATH_AUTO || path == LRD_PATH_FUSED)) {
        const ChainArgs c = bwd_chain_args(L, dY, V, U, dX, need_dz_in_memory ? dZ : nullptr, sm_share);
        // the data-only call exists so that weight gradients can run beside it: it takes the chain on pairs of SMs (96
        // blocks where the single-block chain has 128) although that kernel is slower alone (attention backward data
        // pass 11 against 9 us), because what it leaves free is worth more (step 178.9 -> 174.9 us)
        const lrd_status_t st = launch_chain(&c, 1, path, s, parts == 1);
        if (st == LRD_OK) chained = true;
        else if (st != LRD_ERR_UNSUPPORTED) return st;
    }
    if (!chained) {
        if (dX || need_dz_in_memory)
            LRD_TRY(run_gemm(gemm(L.M, L.r, L.N, dY, L.ldy, false, U, L.ldu, true, dZ, L.r, nullptr, L.dt), false, nullptr, 0, s));
        if (dX)
            LRD_TRY(run_gemm(gemm(L.M, L.K, L.r, dZ, L.r, false, V, L.ldv, false, dX, L.ldx, nullptr, L.dt), false, nullptr, 0, s));
    }
    if (do_w && (plan & LRD_PLAN_DU)) {
        GemmArgs gu = gemm(L.N, L.r, L.M, dY, L.ldy, true, Z_save, L.ldz, true, dU, L.ldu, nullptr, L.dt);
        gu.max_cluster_split = wsplit;
        bool db_done = false;
        if (dbias && g_path.load() != LRD_PATH_GENERAL) {      // db rides on the dU product (A = dY): no second pass over dY
            gu.a_colsum = dbias;
            if (tc_gemm_colsum_ok(gu)) db_done = true; else gu.a_colsum = nullptr;
        }
        cudaStream_t su = side ? side : s;
        LRD_TRY(run_gemm(gu, true, partials, partial_bytes, su));
        if (dbias && !db_done) LRD_TRY(colsum(dY, L.ldy, L.M, L.N, dbias, L.dt, partials, partial_bytes, su));
        if (side && (plan & LRD_PLAN_DV)) {
            if (cudaEventRecord(side_done, side) != cudaSuccess || cudaStreamWaitEvent(s, side_done, 0) != cudaSuccess) return LRD_ERR_CUDA;
        }
    }
    if (do_w && (plan & LRD_PLAN_DV)) {
        GemmArgs gv = gemm(L.K, L.r, L.M, X, L.ldx, true, dZ, L.r, true, dV, L.ldv, nullptr, L.dt);
        gv.max_cluster_split = wsplit;
        LRD_TRY(run_gemm(gv, true, partials, partial_bytes, s));
    }
    return LRD_OK;
}

static lrd_status_t lrd_linear_bwd_data_impl(const lrd_linear_desc_t* desc, const void* dY, const void* V, const void* U, void* dX,
                                 lrd_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return linear_bwd_on(desc, dY, nullptr, V, U, nullptr, dX, nullptr, nullptr, nullptr, freeze, workspace, workspace_bytes,
                         (cudaStream_t)cuda_stream, nullptr, nullptr, 0, false, 1);
}

static lrd_status_t lrd_linear_bwd_weights_impl(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* Z_save, void* dU,
                                    void* dV, void* dbias, lrd_freeze_t freeze, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream) {
    return linear_bwd_on(desc, dY, X, nullptr, nullptr, Z_save, nullptr, dU, dV, dbias, freeze, workspace, workspace_bytes,
                         (cudaStream_t)cuda_stream, nullptr, nullptr, 0, false, 2);
}

static lrd_status_t lrd_linear_bwd_impl(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* V,
                            const void* U, const void* Z_save, void* dX, void* dU, void* dV, void* dbias,
                            lrd_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return linear_bwd_on(desc, dY, X, V, U, Z_save, dX, dU, dV, dbias, freeze, workspace, workspace_bytes,
                         (cudaStream_t)cuda_stream, nullptr, nullptr, 0);
}

static lrd_status_t lrd_linear_bwd_accumulate_impl(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* V,
                                       const void* U, const void* Z_save, void* dX, void* dU, void* dV, void* dbias,
                                       lrd_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    Linear L;
    LRD_TRY(parse_linear(desc, &L, false));
    const uint32_t plan = lrd_linear_bwd_plan(freeze);
    if (!plan) return LRD_ERR_INVALID_ARG;
    LRD_TRY(check_ws(workspace, workspace_bytes, lrd_linear_workspace_bytes(desc, freeze, 2)));
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // this step's gradients go to scratch behind the ordinary backward workspace, then into the caller's buffers;
    // a frozen factor's buffers are not touched (its gradient is zero)
    const size_t bwd_bytes = align_up(lrd_linear_workspace_bytes(desc, freeze, 1), 256);
    const size_t e = elem_size(L.dt);
    uint8_t* g = (uint8_t*)workspace + bwd_bytes;
    void* gU = g;
    void* gV = g + align_up((size_t)L.N * L.ldu * e, 256);
    void* gb = g + align_up((size_t)L.N * L.ldu * e, 256) + align_up((size_t)L.K * L.ldv * e, 256);
    const bool du = (plan & LRD_PLAN_DU) != 0, dv = (plan & LRD_PLAN_DV) != 0;
    if ((du && !dU) || (dv && !dV)) return LRD_ERR_INVALID_ARG;
    const void* outs[] = {dU, dV, dbias};
    for (const void* p : outs)
        if (p && !elem_aligned(p, L.dt)) return LRD_ERR_ALIGNMENT;
    LRD_TRY(linear_bwd_on(desc, dY, X, V, U, Z_save, dX, du ? gU : nullptr, dv ? gV : nullptr, (du && dbias) ? gb : nullptr, freeze,
                          workspace, bwd_bytes, s, nullptr, nullptr, 0));
    if (L.M == 0) return LRD_OK;
    if (du) {
        LRD_TRY(add_into(dU, gU, L.N, L.r, L.ldu, L.dt, s));
        if (dbias) LRD_TRY(add_into(dbias, gb, 1, L.N, L.N, L.dt, s));
    }
    if (dv) LRD_TRY(add_into(dV, gV, L.K, L.r, L.ldv, L.dt, s));
    return LRD_OK;
}

// ---- groups of independent layers -------------------------------------------------------------------
// Layer 0 of a group runs on the caller's stream, layer i on side stream i - 1; the dU products of a backward
// group use the auxiliary set.
static lrd_status_t lrd_linear_group_fwd_impl(int n, const lrd_linear_desc_t* descs, const void* const* X, const void* const* V,
                                  const void* const* U, const void* const* bias, void* const* Y, void* const* Z_save,
                                  lrd_freeze_t freeze, void* const* workspace, const size_t* workspace_bytes,
                                  void* cuda_stream) {
    if (n < 0 || n > LRD_MAX_GROUP) return LRD_ERR_INVALID_ARG;
    if (n == 0) return LRD_OK;
    if (!descs || !X || !V || !U || !Y || !workspace || !workspace_bytes) return LRD_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    for (int i = 0; i < n; ++i)          // nothing is enqueued unless every layer's arguments are valid
        LRD_TRY(linear_fwd_on(&descs[i], X[i], V[i], U[i], bias ? bias[i] : nullptr, Y[i], Z_save ? Z_save[i] : nullptr, freeze,
                              workspace[i], workspace_bytes[i], s, 0, true));
    // layers of one shape: one launch of the fused chain on pairs of SMs, the layer picked by gridDim.z
    const int path = g_path.load();
    if (n > 1 && n <= kChainMaxLayers && (path == LRD_PATH_AUTO || path == LRD_PATH_FUSED) && g_chain_mma_blocks.load() != 1) {
        ChainArgs c[kChainMaxLayers];
        bool ok = true;
        for (int i = 0; i < n && ok; ++i) {
            Linear L;
            ok = parse_linear(&descs[i], &L, false) == LRD_OK && L.M > 0;
            if (ok) c[i] = fwd_chain_args(L, X[i], V[i], U[i], bias ? bias[i] : nullptr, Y[i], Z_save ? Z_save[i] : nullptr, 0);
        }
        if (ok && chain_pair_eligible(c, n)) return chain_pair_launch(c, n, s);
    }
    SideStreams* ss = n > 1 ? side_streams() : nullptr;
    if (n > 1 && !ss) return LRD_ERR_CUDA;
    if (n > 1 && cudaEventRecord(ss->fork, s) != cudaSuccess) return LRD_ERR_CUDA;
    const int share = n > 1 ? kNumSms / n : 0;
    lrd_status_t st = LRD_OK;
    for (int i = 0; i < n; ++i) {
        cudaStream_t si = i == 0 ? s : ss->layer[i - 1];
        if (i > 0 && cudaStreamWaitEvent(si, ss->fork, 0) != cudaSuccess) { st = LRD_ERR_CUDA; continue; }
        const lrd_status_t sti = linear_fwd_on(&descs[i], X[i], V[i], U[i], bias ? bias[i] : nullptr, Y[i],
                                               Z_save ? Z_save[i] : nullptr, freeze, workspace[i], workspace_bytes[i], si, share);
        if (sti != LRD_OK) st = sti;
        if (i > 0 && !stream_after(s, si, ss->join[i - 1])) st = LRD_ERR_CUDA;      // joined even after a failure
    }
    return st;
}

static lrd_status_t lrd_linear_group_bwd_impl(int n, const lrd_linear_desc_t* descs, const void* const* dY, const void* const* X,
                                  const void* const* V, const void* const* U, const void* const* Z_save, void* const* dX,
                                  void* const* dU, void* const* dV, void* const* dbias, lrd_freeze_t freeze,
                                  void* const* workspace, const size_t* workspace_bytes, void* cuda_stream) {
    if (n < 0 || n > LRD_MAX_GROUP) return LRD_ERR_INVALID_ARG;
    if (n == 0) return LRD_OK;
    if (!descs || !dY || !V || !U || !workspace || !workspace_bytes) return LRD_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    auto at = [](const void* const* a, int i) -> const void* { return a ? a[i] : nullptr; };
    auto at_w = [](void* const* a, int i) -> void* { return a ? a[i] : nullptr; };
    for (int i = 0; i < n; ++i)
        LRD_TRY(linear_bwd_on(&descs[i], dY[i], at(X, i), V[i], U[i], at(Z_save, i), at_w(dX, i), at_w(dU, i), at_w(dV, i),
                              at_w(dbias, i), freeze, workspace[i], workspace_bytes[i], s, nullptr, nullptr, 0, true));
    SideStreams* ss = side_streams();
    if (!ss) return LRD_ERR_CUDA;
    if (cudaEventRecord(ss->fork, s) != cudaSuccess) return LRD_ERR_CUDA;
    const bool du_aside = (lrd_linear_bwd_plan(freeze) & LRD_PLAN_DU) != 0;
    // layers of one shape: their data chains (dZ, dX) in one launch on pairs of SMs, the layer picked by gridDim.z;
    // the weight gradients then run side by side as below
    bool data_done = false;
    const int path = g_path.load();
    if (n > 1 && n <= kChainMaxLayers && dX && (path == LRD_PATH_AUTO || path == LRD_PATH_FUSED) && g_chain_mma_blocks.load() != 1) {
        ChainArgs c[kChainMaxLayers];
        bool ok = true;
        const bool need_dz = (lrd_linear_bwd_plan(freeze) & LRD_PLAN_DV) != 0;
        for (int i = 0; i < n && ok; ++i) {
            Linear L;
            ok = parse_linear(&descs[i], &L, false) == LRD_OK && L.M > 0 && dX[i] != nullptr;
            if (ok) c[i] = bwd_chain_args(L, dY[i], V[i], U[i], dX[i], need_dz ? workspace[i] : nullptr, 0);
        }
        if (ok && chain_pair_eligible(c, n)) {
            LRD_TRY(chain_pair_launch(c, n, s));
            data_done = true;
            if (!cuda_ok(cudaEventRecord(ss->mid, s), "cudaEventRecord(group mid)")) return LRD_ERR_CUDA;
        }
    }
    // The data chains are shaped for twice their even share: the weight-gradient launches that follow each of them
    // fill the machine anyway, and a chain of 2 blocks per row tile finishes sooner than one of 1 (three
    // 768 -> 768, r = 192 layers at 4096 tokens, U frozen: 32.9 us against 35.3 us).
    const int share = n > 1 ? 2 * kNumSms / n : 0;
    lrd_status_t st = LRD_OK;
    for (int i = 0; i < n; ++i) {
        cudaStream_t si = i == 0 ? s : ss->layer[i - 1];
        cudaStream_t sd = du_aside ? ss->aux[i] : nullptr;
        if (i > 0 && !cuda_ok(cudaStreamWaitEvent(si, data_done ? ss->mid : ss->fork, 0), "cudaStreamWaitEvent(group layer)")) { st = LRD_ERR_CUDA; continue; }
        if (sd && cudaStreamWaitEvent(sd, ss->fork, 0) != cudaSuccess) { st = LRD_ERR_CUDA; continue; }
        const lrd_status_t sti = linear_bwd_on(&descs[i], dY[i], at(X, i), V[i], U[i], at(Z_save, i), at_w(dX, i), at_w(dU, i),
                                               at_w(dV, i), at_w(dbias, i), freeze, workspace[i], workspace_bytes[i], si, sd,
                                               ss->aux_done[i], share, false, data_done ? 2 : 3);
        if (sti != LRD_OK) st = sti;
        if (sd && !stream_after(s, sd, ss->aux_done[i])) st = LRD_ERR_CUDA;
        if (i > 0 && !stream_after(s, si, ss->join[i - 1])) st = LRD_ERR_CUDA;
    }
    return st;
}

static lrd_status_t lrd_dense_fwd_impl(const lrd_linear_desc_t* desc, const void* X, const void* W, const void* bias, void* Y,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
    Linear L;
    LRD_TRY(parse_linear(desc, &L, true));
    if (!X || !W || !Y) return LRD_ERR_INVALID_ARG;
    (void)workspace; (void)workspace_bytes;
    for (const void* p : {X, W, bias, (const void*)Y})
        if (p && !elem_aligned(p, L.dt)) return LRD_ERR_ALIGNMENT;
    LRD_TRY(check_arch());
    return run_gemm(gemm(L.M, L.N, L.K, X, L.ldx, false, W, L.ldv, false, Y, L.ldy, bias, L.dt), false, nullptr, 0,
                    (cudaStream_t)cuda_stream);
}

static lrd_status_t lrd_dense_bwd_impl(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* W, void* dX,
                           void* dW, void* dbias, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    Linear L;
    LRD_TRY(parse_linear(desc, &L, true));
    if (!dY || !X || !W || !dW) return LRD_ERR_INVALID_ARG;
    for (const void* p : {dY, X, W, (const void*)dX, (const void*)dW, (const void*)dbias})
        if (p && !elem_aligned(p, L.dt)) return LRD_ERR_ALIGNMENT;
    LRD_TRY(check_ws(workspace, workspace_bytes, lrd_dense_workspace_bytes(desc, 1)));
    LRD_TRY(check_arch());
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (L.M == 0) {
        LRD_TRY(zero_fill(dW, L.N, L.K, L.ldv, L.dt, s));
        return zero_fill(dbias, 1, L.N, L.N, L.dt, s);
    }
    float* partials = (float*)((uint8_t*)workspace + 256);
    if (dX) LRD_TRY(run_gemm(gemm(L.M, L.K, L.N, dY, L.ldy, false, W, L.ldv, true, dX, L.ldx, nullptr, L.dt), false, nullptr, 0, s));
    GemmArgs gw = gemm(L.N, L.K, L.M, dY, L.ldy, true, X, L.ldx, true, dW, L.ldv, nullptr, L.dt);
    bool db_done = false;
    if (dbias && g_path.load() != LRD_PATH_GENERAL) {
        gw.a_colsum = dbias;
        if (tc_gemm_colsum_ok(gw)) db_done = true; else gw.a_colsum = nullptr;
    }
    LRD_TRY(run_gemm(gw, true, partials, workspace_bytes - 256, s));
    if (dbias && !db_done) LRD_TRY(colsum(dY, L.ldy, L.M, L.N, dbias, L.dt, partials, workspace_bytes - 256, s));
    return LRD_OK;
}

// ---- the undecomposed 3x3 convolution (the layer a Tucker-2 layer replaces) ---------------------------------------
static lrd_status_t conv3x3_check(int64_t B, int64_t H, int64_t W, int64_t C, int64_t S, int dtype) {
    if (B < 0 || H < 1 || W < 1 || C < 1 || S < 1) return LRD_ERR_INVALID_ARG;
    if (dtype != LRD_F32 && dtype != LRD_BF16) return LRD_ERR_INVALID_ARG;
    if (H > 32767 || W > 32767) return LRD_ERR_UNSUPPORTED;
    return LRD_OK;
}

size_t lrd_conv3x3_workspace_bytes(int64_t B, int64_t H, int64_t W, int64_t C, int64_t S, int dtype) {
    if (conv3x3_check(B, H, W, C, S, dtype) != LRD_OK) return 0;
    return align_up(dtype == LRD_BF16 ? tc_conv_filter_scratch_bytes(B, H, W, C, S) : 0, 256) + 256;
}

static lrd_status_t lrd_conv3x3_fwd_impl(int64_t B, int64_t H, int64_t W, int64_t C, int64_t S, int dtype, const void* X, const void* Wk,
                             void* Y, void* cuda_stream) {
    LRD_TRY(conv3x3_check(B, H, W, C, S, dtype));
    if (!X || !Wk || !Y) return LRD_ERR_INVALID_ARG;
    for (const void* p : {X, Wk, (const void*)Y})
        if (!elem_aligned(p, dtype)) return LRD_ERR_ALIGNMENT;
    LRD_TRY(check_arch());
    if (B == 0) return LRD_OK;
    return conv3x3_fwd(X, Wk, Y, B, H, W, C, S, (lrd_dtype_t)dtype, g_path.load(), (cudaStream_t)cuda_stream);
}

static lrd_status_t lrd_conv3x3_bwd_impl(int64_t B, int64_t H, int64_t W, int64_t C, int64_t S, int dtype, const void* dY, const void* X,
                             const void* Wk, void* dX, void* dW, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    LRD_TRY(conv3x3_check(B, H, W, C, S, dtype));
    if (!dY || !X || !Wk || !dW) return LRD_ERR_INVALID_ARG;
    for (const void* p : {dY, X, Wk, (const void*)dX, (const void*)dW})
        if (p && !elem_aligned(p, dtype)) return LRD_ERR_ALIGNMENT;
    LRD_TRY(check_ws(workspace, workspace_bytes, lrd_conv3x3_workspace_bytes(B, H, W, C, S, dtype)));
    LRD_TRY(check_arch());
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (B == 0) return zero_fill(dW, S, 9 * C, 9 * C, (lrd_dtype_t)dtype, s);
    if (dX) LRD_TRY(conv3x3_bwd_data(dY, Wk, dX, B, H, W, C, S, (lrd_dtype_t)dtype, g_path.load(), s));
    return conv3x3_bwd_filter(dY, X, dW, B, H, W, C, S, (lrd_dtype_t)dtype, g_path.load(), (float*)workspace, workspace_bytes - 256, s);
}

size_t lrd_tucker2_workspace_bytes(const lrd_tucker2_desc_t* desc, lrd_tucker_freeze_t freeze, int is_bwd) {
    return tucker2_workspace_bytes(desc, freeze, is_bwd);
}

static lrd_status_t lrd_tucker2_fwd_impl(const lrd_tucker2_desc_t* desc, const void* X, const void* A, const void* G,
                             const void* Bm, const void* bias, void* Y, void* Z1_save, void* Z2_save,
                             lrd_tucker_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    LRD_TRY(tucker2_check(desc, freeze));
    if (!X || !A || !G || !Bm || !Y) return LRD_ERR_INVALID_ARG;
    if ((freeze == LRD_TK_FREEZE_CORE) != (Z1_save == nullptr)) return LRD_ERR_INVALID_ARG;
    if ((freeze == LRD_TK_FREEZE_FACTORS) != (Z2_save == nullptr)) return LRD_ERR_INVALID_ARG;
    for (const void* p : {X, A, G, Bm, bias, (const void*)Y, (const void*)Z1_save, (const void*)Z2_save})
        if (p && !elem_aligned(p, desc->dtype)) return LRD_ERR_ALIGNMENT;
    LRD_TRY(check_ws(workspace, workspace_bytes, tucker2_workspace_bytes(desc, freeze, 0)));
    LRD_TRY(check_arch());
    return tucker2_fwd(desc, X, A, G, Bm, bias, Y, Z1_save, Z2_save, freeze, workspace, workspace_bytes,
                       g_path.load(), (cudaStream_t)cuda_stream);
}

static lrd_status_t lrd_tucker2_bwd_impl(const lrd_tucker2_desc_t* desc, const void* dY, const void* X, const void* A,
                             const void* G, const void* Bm, const void* Z1_save, const void* Z2_save, void* dX,
                             void* dA, void* dG, void* dB, void* dbias, lrd_tucker_freeze_t freeze, void* workspace,
                             size_t workspace_bytes, void* cuda_stream) {
    LRD_TRY(tucker2_check(desc, freeze));
    if (!dY || !A || !G || !Bm) return LRD_ERR_INVALID_ARG;
    if (freeze != LRD_TK_FREEZE_FACTORS && (!X || !Z2_save || !dA || !dB)) return LRD_ERR_INVALID_ARG;
    if (freeze != LRD_TK_FREEZE_CORE && (!Z1_save || !dG)) return LRD_ERR_INVALID_ARG;
    for (const void* p : {dY, X, A, G, Bm, Z1_save, Z2_save, (const void*)dX, (const void*)dA, (const void*)dG, (const void*)dB, (const void*)dbias})
        if (p && !elem_aligned(p, desc->dtype)) return LRD_ERR_ALIGNMENT;
    LRD_TRY(check_ws(workspace, workspace_bytes, tucker2_workspace_bytes(desc, freeze, 1)));
    LRD_TRY(check_arch());
    return tucker2_bwd(desc, dY, X, A, G, Bm, Z1_save, Z2_save, dX, dA, dG, dB, dbias, freeze, workspace,
                       workspace_bytes, g_path.load(), (cudaStream_t)cuda_stream);
}


// ---- debug mode ---------------------------------------------------------------------------------------------------
// With the environment variable LRD_DEBUG set (to anything but 0), every compute entry point waits for the work it has
// enqueued and reports what went wrong in it -- LRD_ERR_CUDA for a launch or execution error, LRD_ERR_TIMEOUT for a
// bounded device wait that ran out -- instead of leaving both to the next lrd_check_device_status().  A call made
// while its stream is being captured is left alone.  Off by default: the library otherwise never synchronises.
static bool debug_on() {
    static const bool on = [] { const char* e = getenv("LRD_DEBUG"); return e && *e && strcmp(e, "0") != 0; }();
    return on;
}
static lrd_status_t debug_checked(lrd_status_t st, void* cuda_stream) {
    if (st != LRD_OK || !debug_on()) return st;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing((cudaStream_t)cuda_stream, &cap) != cudaSuccess) { cudaGetLastError(); return st; }
    if (cap != cudaStreamCaptureStatusNone) return st;
    if (!cuda_ok(cudaStreamSynchronize((cudaStream_t)cuda_stream), "cudaStreamSynchronize(LRD_DEBUG)")) return LRD_ERR_CUDA;
    bool raised = false;
    if (read_and_clear_device_timeout(&raised) != LRD_OK) return LRD_ERR_CUDA;
    return raised ? LRD_ERR_TIMEOUT : LRD_OK;
}

lrd_status_t lrd_linear_fwd(const lrd_linear_desc_t* desc, const void* X, const void* V, const void* U,
                            const void* bias, void* Y, void* Z_save, lrd_freeze_t freeze, void* workspace,
                            size_t workspace_bytes, void* cuda_stream) {
    return debug_checked(lrd_linear_fwd_impl(desc, X, V, U, bias, Y, Z_save, freeze, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_linear_bwd_data(const lrd_linear_desc_t* desc, const void* dY, const void* V, const void* U, void* dX,
                                 lrd_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return debug_checked(lrd_linear_bwd_data_impl(desc, dY, V, U, dX, freeze, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_linear_bwd_weights(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* Z_save, void* dU,
                                    void* dV, void* dbias, lrd_freeze_t freeze, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream) {
    return debug_checked(lrd_linear_bwd_weights_impl(desc, dY, X, Z_save, dU, dV, dbias, freeze, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_linear_bwd(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* V,
                            const void* U, const void* Z_save, void* dX, void* dU, void* dV, void* dbias,
                            lrd_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return debug_checked(lrd_linear_bwd_impl(desc, dY, X, V, U, Z_save, dX, dU, dV, dbias, freeze, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_linear_bwd_accumulate(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* V,
                                       const void* U, const void* Z_save, void* dX, void* dU, void* dV, void* dbias,
                                       lrd_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return debug_checked(lrd_linear_bwd_accumulate_impl(desc, dY, X, V, U, Z_save, dX, dU, dV, dbias, freeze, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_linear_group_fwd(int n, const lrd_linear_desc_t* descs, const void* const* X, const void* const* V,
                                  const void* const* U, const void* const* bias, void* const* Y, void* const* Z_save,
                                  lrd_freeze_t freeze, void* const* workspace, const size_t* workspace_bytes,
                                  void* cuda_stream) {
    return debug_checked(lrd_linear_group_fwd_impl(n, descs, X, V, U, bias, Y, Z_save, freeze, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_linear_group_bwd(int n, const lrd_linear_desc_t* descs, const void* const* dY, const void* const* X,
                                  const void* const* V, const void* const* U, const void* const* Z_save, void* const* dX,
                                  void* const* dU, void* const* dV, void* const* dbias, lrd_freeze_t freeze,
                                  void* const* workspace, const size_t* workspace_bytes, void* cuda_stream) {
    return debug_checked(lrd_linear_group_bwd_impl(n, descs, dY, X, V, U, Z_save, dX, dU, dV, dbias, freeze, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_dense_fwd(const lrd_linear_desc_t* desc, const void* X, const void* W, const void* bias, void* Y,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return debug_checked(lrd_dense_fwd_impl(desc, X, W, bias, Y, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_dense_bwd(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* W, void* dX,
                           void* dW, void* dbias, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return debug_checked(lrd_dense_bwd_impl(desc, dY, X, W, dX, dW, dbias, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_conv3x3_fwd(int64_t B, int64_t H, int64_t W, int64_t C, int64_t S, int dtype, const void* X, const void* Wk,
                             void* Y, void* cuda_stream) {
    return debug_checked(lrd_conv3x3_fwd_impl(B, H, W, C, S, dtype, X, Wk, Y, cuda_stream), cuda_stream);
}

lrd_status_t lrd_conv3x3_bwd(int64_t B, int64_t H, int64_t W, int64_t C, int64_t S, int dtype, const void* dY, const void* X,
                             const void* Wk, void* dX, void* dW, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return debug_checked(lrd_conv3x3_bwd_impl(B, H, W, C, S, dtype, dY, X, Wk, dX, dW, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_tucker2_fwd(const lrd_tucker2_desc_t* desc, const void* X, const void* A, const void* G,
                             const void* Bm, const void* bias, void* Y, void* Z1_save, void* Z2_save,
                             lrd_tucker_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return debug_checked(lrd_tucker2_fwd_impl(desc, X, A, G, Bm, bias, Y, Z1_save, Z2_save, freeze, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

lrd_status_t lrd_tucker2_bwd(const lrd_tucker2_desc_t* desc, const void* dY, const void* X, const void* A,
                             const void* G, const void* Bm, const void* Z1_save, const void* Z2_save, void* dX,
                             void* dA, void* dG, void* dB, void* dbias, lrd_tucker_freeze_t freeze, void* workspace,
                             size_t workspace_bytes, void* cuda_stream) {
    return debug_checked(lrd_tucker2_bwd_impl(desc, dY, X, A, G, Bm, Z1_save, Z2_save, dX, dA, dG, dB, dbias, freeze, workspace, workspace_bytes, cuda_stream), cuda_stream);
}

}  // extern "C"
