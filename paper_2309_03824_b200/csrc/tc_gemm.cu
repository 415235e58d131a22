// Tensor-core matrix product for sm_100a: TMA -> shared memory (128-byte swizzle) ->
// tcgen05.mma with the accumulator in tensor memory -> tcgen05.ld epilogue.
//
//   C[M x N] = op(A) op(B) (+ bias), bf16 in, fp32 accumulate, bf16 out; or, with a split of the
//   reduction dimension over gridDim.z, fp32 partial tiles that a second kernel adds in a fixed
//   order (deterministic weight gradients, no floating-point atomics).
//
// One 128 x BN output tile per block.  Warp 0 issues TMA loads, warp 1 owns tensor memory and
// issues the MMAs, warps 2-5 read the accumulator (each its own quarter of the 128 lanes) and
// store.  The single-thread instructions are issued under elect.sync by a converged warp.  Both operands may be K-major (reduction index contiguous) or MN-major (row / column
// index contiguous), which covers every product of the forward and backward pass without a
// transposed copy.
#include "common.cuh"
#include "ptx.cuh"
#include "tc.cuh"
#include "tma.cuh"

namespace lrd {
namespace {

using namespace ptx;

constexpr int BM = 128, BK = 64;
constexpr int kThreads = 192;
constexpr uint32_t A_STAGE_BYTES = BM * BK * 2;

// ONES: every stage carries one more 64-wide MN-major block of B that holds 1.0 everywhere and is never
// overwritten; with N = BN + 16 the MMA then also forms sum_k A(m, k) in accumulator column BN (the bias
// gradient falls out of the dU product: its A operand is dY).
template <int BN, bool ONES = false> struct Cfg {
    static constexpr uint32_t B_STAGE_BYTES = BN * BK * 2 + (ONES ? 8192 : 0);
    static constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int STAGES_RAW = (200 * 1024) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
    static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + 1024;   // + slack for 1024-B alignment
    static constexpr uint32_t TMEM_COLS = (BN + (ONES ? 32 : 0)) <= 64 ? 64 : ((BN + (ONES ? 32 : 0)) <= 128 ? 128 : 256);
};

struct TcParams {
    int64_t M, N;
    int64_t ldp;        // leading dimension of the fp32 partial tiles (N rounded up to 4)
    int kb_total, kb_per_split;
    void* C;            // bf16 [M x N] (ldc) or fp32 partials [splits][M x N] packed
    int64_t ldc;
    const __nv_bfloat16* bias;
    int partial;        // 1: write fp32 partials
    float* colsum_partial;        // ONES, split: [splits][M] partial sums over k of A
    __nv_bfloat16* colsum_out;    // ONES, not split: [M]
    unsigned int* timeout_flag;
};

template <int BN, bool A_MN, bool B_MN, bool ONES = false>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const TcParams p) {
    static_assert(!ONES || (A_MN && B_MN && BN <= 192), "the ones block rides on an MN-major B of at most 192 columns");
    using C = Cfg<BN, ONES>;
    constexpr int STAGES = C::STAGES;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[STAGES], empty_bar[STAGES], acc_bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const AbortCtx ab{&abort_flag, p.timeout_flag};
    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0), lane = threadIdx.x % 32;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int kb_begin = blockIdx.z * p.kb_per_split;
    const int kb_end = min(kb_begin + p.kb_per_split, p.kb_total);

    if (threadIdx.x == 0) {
        abort_flag = 0;
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        mbar_init(smem_u32(&acc_bar), 1);
        fence_mbar_init();
    }
    if (ONES) {          // bf16 1.0 in every element of the extra block of each stage
        for (uint32_t off = threadIdx.x * 16u; off < STAGES * 8192u; off += kThreads * 16u)
            st_shared_v4(smem_base + (off / 8192u) * C::STAGE_BYTES + A_STAGE_BYTES + BN * 128u + (off % 8192u), 0x3F803F80u,
                         0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
        fence_proxy_async_smem();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), C::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0) {
        // TMA producer: the whole warp runs the loop, one elected lane issues (operands stay uniform)
        int it = 0;
        for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1;
            if (!mbar_wait_uniform(smem_u32(&empty_bar[s]), ph ^ 1, ab)) break;
            const uint32_t fb = smem_u32(&full_bar[s]);
            const uint32_t a_dst = smem_base + s * C::STAGE_BYTES;
            const uint32_t b_dst = a_dst + A_STAGE_BYTES;
            const int k0 = kb * BK;
            if (elect_one()) {
                mbar_expect_tx(fb, A_STAGE_BYTES + BN * BK * 2);
                if (A_MN) {
#pragma unroll
                    for (int j = 0; j < BM / 64; ++j) tma_load_2d(a_dst + j * 8192, &tmA, fb, m0 + 64 * j, k0);
                } else {
                    tma_load_2d(a_dst, &tmA, fb, k0, m0);
                }
                if (B_MN) {
#pragma unroll
                    for (int j = 0; j < BN / 64; ++j) tma_load_2d(b_dst + j * 8192, &tmB, fb, n0 + 64 * j, k0);
                } else {
                    tma_load_2d(b_dst, &tmB, fb, k0, n0);
                }
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        // MMA issuer: converged warp, elect.sync around the issue
        const uint32_t idesc = idesc_bf16(BN + ((ONES && blockIdx.x == 0) ? 16 : 0), A_MN, B_MN);
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int kb = kb_begin; kb < kb_end; ++kb) {
            ok = mbar_wait_uniform(smem_u32(&full_bar[s]), ph, ab);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_src = smem_base + s * C::STAGE_BYTES;
            const uint32_t b_src = a_src + A_STAGE_BYTES;
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk) {
                    const uint64_t ad = A_MN ? smem_desc_sw128(a_src + kk * 2048, 8192, 1024)
                                             : smem_desc_sw128(a_src + kk * 32, 0, 1024);
                    const uint64_t bd = B_MN ? smem_desc_sw128(b_src + kk * 2048, 8192, 1024)
                                             : smem_desc_sw128(b_src + kk * 32, 0, 1024);
                    mma_bf16_ss(tmem_base, ad, bd, idesc, (kb > kb_begin || kk > 0) ? 1u : 0u);
                }
                mma_commit(smem_u32(&empty_bar[s]));
            }
            __syncwarp();
            if (++s == STAGES) { s = 0; ph ^= 1; }
        }
        if (ok && elect_one()) mma_commit(smem_u32(&acc_bar));
        __syncwarp();
    } else {
        const int quarter = warp % 4;                      // lanes [32 q, 32 q + 32) of tensor memory
        const bool ready = mbar_wait_warp(smem_u32(&acc_bar), 0, ab);
        tc_fence_after();
        if (ready) {
            const int64_t row = (int64_t)m0 + quarter * 32 + lane;
            const bool row_ok = row < p.M;
            const bool bias_vec_ok = p.bias && (((uintptr_t)p.bias & 15u) == 0);
            if (ONES && blockIdx.x == 0) {                 // accumulator column BN = sum over k of A(row, k)
                uint32_t cs[16];
                tmem_ld_32x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + BN, cs);
                tmem_ld_wait();
                if (row_ok) {
                    if (p.partial) p.colsum_partial[(int64_t)blockIdx.z * p.M + row] = __uint_as_float(cs[0]);
                    else if (p.colsum_out) p.colsum_out[row] = __float2bfloat16_rn(__uint_as_float(cs[0]));
                }
            }
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + c * 32, v);
                tmem_ld_wait();
                const int64_t col0 = (int64_t)n0 + c * 32;
                if (!row_ok || col0 >= p.N) continue;
                if (p.partial) {
                    float* dst = (float*)p.C + ((int64_t)blockIdx.z * p.M + row) * p.ldp + col0;
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        if (col0 + g * 4 + 4 <= p.N) {
                            *reinterpret_cast<uint4*>(dst + g * 4) = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                        } else {
                            for (int e = 0; e < 4; ++e)
                                if (col0 + g * 4 + e < p.N) dst[g * 4 + e] = __uint_as_float(v[4 * g + e]);
                        }
                    }
                } else {
                    __nv_bfloat16* dst = (__nv_bfloat16*)p.C + row * p.ldc + col0;
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        float f[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[8 * g + e]);
                        if (p.bias) {
                            if (bias_vec_ok && col0 + g * 8 + 8 <= p.N) {       // one 16-byte load for 8 columns
                                const uint4 b4 = __ldg(reinterpret_cast<const uint4*>(p.bias + col0 + g * 8));
                                const uint32_t bw[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    f[2 * e] += __uint_as_float(bw[e] << 16);
                                    f[2 * e + 1] += __uint_as_float(bw[e] & 0xFFFF0000u);
                                }
                            } else {
                                for (int e = 0; e < 8; ++e)
                                    if (col0 + g * 8 + e < p.N) f[e] += __bfloat162float(p.bias[col0 + g * 8 + e]);
                            }
                        }
                        if (col0 + g * 8 + 8 <= p.N) {
                            *reinterpret_cast<uint4*>(dst + g * 8) = make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]),
                                                                                 pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
                        } else {
                            for (int e = 0; e < 8; ++e)
                                if (col0 + g * 8 + e < p.N) dst[g * 8 + e] = __float2bfloat16_rn(f[e]);
                        }
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (abort_flag) {            // give copies and MMAs still in flight time to land before freeing
            for (int i = 0; i < 256; ++i) __nanosleep(1000);
        }
        tc_fence_after();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

// out[m][n] = sum_z partial[z][m][n] (+ bias[n]), z ascending; 4 columns per thread.
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const float* __restrict__ partial, int splits, int64_t M,
                                                            int64_t N, int64_t ldp,
                                                            const __nv_bfloat16* __restrict__ bias,
                                                            __nv_bfloat16* __restrict__ C, int64_t ldc,
                                                            const float* __restrict__ colsum_partial,
                                                            __nv_bfloat16* __restrict__ colsum_out) {
    const int64_t n4 = (N + 3) / 4;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= M * n4) {                                // trailing threads: the column sums, one row each
        const int64_t m = idx - M * n4;
        if (colsum_out && m < M) {
            float t = 0.f;
            for (int z = 0; z < splits; ++z) t += colsum_partial[(int64_t)z * M + m];
            colsum_out[m] = __float2bfloat16_rn(t);
        }
        return;
    }
    const int64_t m = idx / n4, n = (idx % n4) * 4;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const bool full = n + 4 <= N;
    for (int z = 0; z < splits; ++z) {
        const float* src = partial + ((int64_t)z * M + m) * ldp + n;
        if (full) {
            const float4 v = *reinterpret_cast<const float4*>(src);
            acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
        } else {
            for (int e = 0; e < 4; ++e)
                if (n + e < N) acc[e] += src[e];
        }
    }
    for (int e = 0; e < 4; ++e)
        if (n + e < N) {
            float v = acc[e];
            if (bias) v += __bfloat162float(bias[n + e]);
            C[m * ldc + n + e] = __float2bfloat16_rn(v);
        }
}

template <int BN, bool A_MN, bool B_MN, bool ONES = false>
lrd_status_t launch(const CUtensorMap& tA, const CUtensorMap& tB, const TcParams& p, dim3 grid, cudaStream_t stream) {
    auto kern = tc_gemm_kernel<BN, A_MN, B_MN, ONES>;
    static bool configured = false;     // per instantiation; the attribute is sticky per function
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<BN, ONES>::SMEM_BYTES) != cudaSuccess)
            return LRD_ERR_CUDA;
        configured = true;
    }
    kern<<<grid, kThreads, Cfg<BN, ONES>::SMEM_BYTES, stream>>>(tA, tB, p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

template <int BN>
lrd_status_t launch_major(bool a_mn, bool b_mn, const CUtensorMap& tA, const CUtensorMap& tB, const TcParams& p,
                          dim3 grid, cudaStream_t s) {
    if (a_mn) return b_mn ? launch<BN, true, true>(tA, tB, p, grid, s) : launch<BN, true, false>(tA, tB, p, grid, s);
    return b_mn ? launch<BN, false, true>(tA, tB, p, grid, s) : launch<BN, false, false>(tA, tB, p, grid, s);
}

inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

}  // namespace

bool tc_gemm_eligible(const GemmArgs& g) {
    if (g.dtype != LRD_BF16 || g.M < 1 || g.N < 1 || g.K < 1) return false;
    if (g.M > (int64_t)65535 * BM || g.K > (int64_t)1 << 30 || g.N > (int64_t)1 << 30) return false;
    if (!aligned16(g.A) || !aligned16(g.B) || !aligned16(g.C)) return false;
    if (g.lda % 8 || g.ldb % 8 || g.ldc % 8) return false;
    return true;
}

// Tile width.  One k-block of a 128 x BN tile costs four MMAs of max(77, BN / 2) cycles each (an MMA
// narrower than 154 columns is issue-bound), so a 64-wide tile is as slow as a 128-wide one.
//   split = false: blocks run in waves over the SMs -> minimise waves x per-tile cost;
//   split = true:  the reduction is split until the machine is full -> minimise tiles x per-tile cost.
static int pick_bn(int64_t M, int64_t N, bool split) {
    const int cands[4] = {256, 192, 128, 64};
    const int64_t mt = (M + BM - 1) / BM;
    int best = 64;
    double best_cost = 1e300;
    for (int bn : cands) {
        if (bn == 64 && N > 64) continue;
        const int64_t tiles = mt * ((N + bn - 1) / bn);
        const double per_tile = bn < 154 ? 154.0 : (double)bn;
        const double cost = split ? (double)tiles * per_tile : (double)((tiles + kNumSms - 1) / kNumSms) * (per_tile + 32);
        if (cost < best_cost) { best_cost = cost; best = bn; }
    }
    return best;
}

int tc_pick_bn(int64_t M, int64_t N) { return pick_bn(M, N, false); }

int tc_pick_splits(int64_t M, int64_t N, int64_t K) {
    const int bn = pick_bn(M, N, true);
    const int64_t tiles = ((M + BM - 1) / BM) * ((N + bn - 1) / bn);
    const int64_t kb = (K + BK - 1) / BK;
    int64_t s = kNumSms / tiles;
    if (s < 1) s = 1;
    if (s > kb / 4) s = kb / 4;          // at least four k-blocks per split
    if (s < 1) s = 1;
    if (s > 64) s = 64;
    // no empty split: shrink until every z has work
    const int64_t per = (kb + s - 1) / s;
    s = (kb + per - 1) / per;
    return (int)s;
}

// fp32 partial tiles [splits][M][ldp], then (for the optional column sums) [splits][M]
size_t tc_split_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    const int s = tc_pick_splits(M, N, K);
    return s > 1 ? align_up((size_t)s * M * ((N + 3) / 4 * 4) * sizeof(float), 256) + align_up((size_t)s * M * sizeof(float), 256) : 0;
}

bool tc_gemm_colsum_ok(const GemmArgs& g) {
    return tc_gemm_eligible(g) && g.a_mn_major && g.b_mn_major && (((uintptr_t)g.a_colsum & 1u) == 0);
}

lrd_status_t tc_gemm(const GemmArgs& g, bool allow_split, float* partials, size_t partial_bytes,
                     cudaStream_t stream) {
    if (!tc_gemm_eligible(g)) return LRD_ERR_UNSUPPORTED;
    int splits = allow_split ? tc_pick_splits(g.M, g.N, g.K) : 1;
    int bn = pick_bn(g.M, g.N, splits > 1);
    const bool ones = g.a_colsum != nullptr;
    if (ones && !tc_gemm_colsum_ok(g)) return LRD_ERR_UNSUPPORTED;
    if (ones && bn > 192) bn = 192;                    // the ones block needs 16 accumulator columns beside the tile
    const int64_t ldp = (g.N + 3) / 4 * 4;
    const size_t tile_bytes = align_up((size_t)splits * g.M * ldp * sizeof(float), 256);
    if (splits > 1 && (!partials || partial_bytes < tile_bytes + (ones ? (size_t)splits * g.M * sizeof(float) : 0)))
        return LRD_ERR_WORKSPACE;
    const int kb_total = (int)((g.K + BK - 1) / BK);
    const int kb_per = (kb_total + splits - 1) / splits;

    CUtensorMap tA, tB;
    bool ok = g.a_mn_major ? make_tmap_2d_bf16(&tA, g.A, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.lda, BK, 64)
                           : make_tmap_2d_bf16(&tA, g.A, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)g.lda, BM, BK);
    ok = ok && (g.b_mn_major ? make_tmap_2d_bf16(&tB, g.B, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)g.ldb, BK, 64)
                             : make_tmap_2d_bf16(&tB, g.B, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.ldb, (uint32_t)bn, BK));
    if (!ok) return LRD_ERR_CUDA;

    TcParams p;
    p.M = g.M; p.N = g.N; p.ldp = ldp; p.kb_total = kb_total; p.kb_per_split = kb_per;
    p.partial = splits > 1 ? 1 : 0;
    p.timeout_flag = device_timeout_flag();
    p.C = splits > 1 ? (void*)partials : g.C;
    p.ldc = g.ldc;
    p.bias = splits > 1 ? nullptr : (const __nv_bfloat16*)g.bias;
    p.colsum_partial = (ones && splits > 1) ? (float*)((uint8_t*)partials + tile_bytes) : nullptr;
    p.colsum_out = (ones && splits == 1) ? (__nv_bfloat16*)g.a_colsum : nullptr;
    dim3 grid((unsigned)((g.N + bn - 1) / bn), (unsigned)((g.M + BM - 1) / BM), (unsigned)splits);
    lrd_status_t st;
    if (ones) {
        switch (bn) {
            case 192: st = launch<192, true, true, true>(tA, tB, p, grid, stream); break;
            case 128: st = launch<128, true, true, true>(tA, tB, p, grid, stream); break;
            default:  st = launch<64, true, true, true>(tA, tB, p, grid, stream); break;
        }
    } else
    switch (bn) {
        case 256: st = launch_major<256>(g.a_mn_major, g.b_mn_major, tA, tB, p, grid, stream); break;
        case 192: st = launch_major<192>(g.a_mn_major, g.b_mn_major, tA, tB, p, grid, stream); break;
        case 128: st = launch_major<128>(g.a_mn_major, g.b_mn_major, tA, tB, p, grid, stream); break;
        default:  st = launch_major<64>(g.a_mn_major, g.b_mn_major, tA, tB, p, grid, stream); break;
    }
    if (st != LRD_OK || splits == 1) return st;
    const int64_t work = g.M * ((g.N + 3) / 4) + (ones ? g.M : 0);
    splitk_reduce_kernel<<<(unsigned)((work + 255) / 256), 256, 0, stream>>>(
        partials, splits, g.M, g.N, ldp, (const __nv_bfloat16*)g.bias, (__nv_bfloat16*)g.C, g.ldc, p.colsum_partial,
        ones ? (__nv_bfloat16*)g.a_colsum : nullptr);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

}  // namespace lrd
