// Persistent tensor-core matrix product for sm_100a (unsplit products with a bf16 result):
//   C[M x N] = op(A) op(B) (+ bias)
// One block per SM walks over the 128 x BN output tiles (tile t -> row tile t % m_tiles, column tile
// t / m_tiles, so that blocks working at the same time share the B operand in L2).  The accumulator is
// double-buffered in tensor memory: while the four epilogue warps round tile i to bf16 and store it
// (each warp its own 32 rows, through [32 x 32] shared-memory slabs and TMA stores that clip the ragged
// edges), the MMA warp already accumulates tile i + 1.  A short reduction (K of a few hundred, as in the
// second product of an unfused decomposed layer) is otherwise all epilogue.
// Warp 0: TMA producer.  Warp 1: tensor memory + MMA issue.  Warps 2-5: epilogue.  Single-thread
// instructions are issued under elect.sync by a converged warp; every wait is bounded.
#include "common.cuh"
#include "ptx.cuh"
#include "tc.cuh"
#include "tma.cuh"

namespace lrd {
namespace {

using namespace ptx;

constexpr int BM = 128, BK = 64;
constexpr int kThreads = 192;
constexpr uint32_t kATile = BM * BK * 2;
constexpr uint32_t kSlabBytes = 32 * 32 * 2;                 // one warp's slab: 32 rows x 32 columns of bf16
constexpr uint32_t kStagingBytes = 4 * 2 * kSlabBytes;

template <int BN> struct PCfg {
    static constexpr uint32_t STAGE_BYTES = kATile + BN * BK * 2;
    static constexpr int STAGES_RAW = (200 * 1024) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
    static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + kStagingBytes + 1024;
    static constexpr uint32_t TMEM_COLS = 2 * BN <= 128 ? 128 : (2 * BN <= 256 ? 256 : 512);
    static constexpr uint32_t BUF_COLS = TMEM_COLS / 2;      // column offset of the second accumulator
};

struct PParams {
    int64_t M, N;
    int kb_total, m_tiles, n_tiles;
    const __nv_bfloat16* bias;
    unsigned int* timeout_flag;
};

template <int BN, bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_persistent_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                          const __grid_constant__ CUtensorMap tmC, const PParams p) {
    using C = PCfg<BN>;
    constexpr int STAGES = C::STAGES;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[STAGES], empty_bar[STAGES], out_full[2], out_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging_base = smem_base, ring_base = smem_base + kStagingBytes;
    const AbortCtx ab{&abort_flag, p.timeout_flag};
    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0), lane = threadIdx.x % 32;
    const int n_tiles_total = p.m_tiles * p.n_tiles;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        prefetch_tmap(&tmC);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&out_full[i]), 1);
            mbar_init(smem_u32(&out_empty[i]), 4);
        }
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), C::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // set-up above touched only this block's own shared and tensor memory: it may overlap the tail of the
    // previous kernel in the stream; global memory is first touched below this line
    griddep_launch_dependents();
    griddep_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        int s = 0;
        uint32_t ph = 1;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x) {
            const int m0 = (t % p.m_tiles) * BM, n0 = (t / p.m_tiles) * BN;
            for (int kb = 0; kb < p.kb_total; ++kb) {
                ok = mbar_wait_uniform(smem_u32(&empty_bar[s]), ph, ab);
                if (!ok) break;
                const uint32_t fb = smem_u32(&full_bar[s]);
                const uint32_t a_dst = ring_base + s * C::STAGE_BYTES, b_dst = a_dst + kATile;
                const int k0 = kb * BK;
                if (elect_one()) {
                    mbar_expect_tx(fb, C::STAGE_BYTES);
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
                if (++s == STAGES) { s = 0; ph ^= 1; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = idesc_bf16(BN, A_MN, B_MN);
        int s = 0, i = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x, ++i) {
            const int buf = i & 1;
            const uint32_t d_tmem = tmem_base + (uint32_t)buf * C::BUF_COLS;
            ok = mbar_wait_uniform(smem_u32(&out_empty[buf]), ((i >> 1) & 1) ^ 1, ab);      // accumulator buffer drained
            for (int kb = 0; kb < p.kb_total && ok; ++kb) {
                ok = mbar_wait_uniform(smem_u32(&full_bar[s]), ph, ab);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_src = ring_base + s * C::STAGE_BYTES, b_src = a_src + kATile;
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk) {
                        const uint64_t ad = A_MN ? smem_desc_sw128(a_src + kk * 2048, 8192, 1024)
                                                 : smem_desc_sw128(a_src + kk * 32, 0, 1024);
                        const uint64_t bd = B_MN ? smem_desc_sw128(b_src + kk * 2048, 8192, 1024)
                                                 : smem_desc_sw128(b_src + kk * 32, 0, 1024);
                        mma_bf16_ss(d_tmem, ad, bd, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&empty_bar[s]));
                    if (kb == p.kb_total - 1) mma_commit(smem_u32(&out_full[buf]));
                }
                __syncwarp();
                if (++s == STAGES) { s = 0; ph ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int q = warp % 4;                              // tensor-memory lanes [32 q, 32 q + 32)
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t slab0 = staging_base + (uint32_t)(warp - 2) * 2u * kSlabBytes;
        const uint32_t row_off = (uint32_t)lane * 64u, row_xor = ((uint32_t)lane >> 1) & 3u;
        const bool bias_ok = p.bias && (((uintptr_t)p.bias & 15u) == 0);
        int i = 0, sb = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x, ++i) {
            const int buf = i & 1;
            const int m0 = (t % p.m_tiles) * BM, n0 = (t / p.m_tiles) * BN;
            ok = mbar_wait_uniform(smem_u32(&out_full[buf]), (i >> 1) & 1, ab);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = lane_addr + (uint32_t)buf * C::BUF_COLS;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c, ++sb) {
                const int col0 = n0 + c * 32;
                if (col0 >= p.N) break;                      // (uniform) nothing of this piece is inside C
                uint4 bv[4] = {};
                const bool bvec = bias_ok && col0 + 32 <= p.N;
                if (bvec) {
                    const uint4* bp = reinterpret_cast<const uint4*>(p.bias + col0);
#pragma unroll
                    for (int e = 0; e < 4; ++e) bv[e] = __ldg(bp + e);
                }
                uint32_t v[32];
                tmem_ld_32x32(d_tmem + c * 32, v);
                const uint32_t slab = slab0 + (uint32_t)(sb & 1) * kSlabBytes;
                if (sb >= 2) {                               // the store that last read this slab has finished reading
                    tma_store_wait_read<1>();
                    __syncwarp();
                }
                tmem_ld_wait();
                if (bvec) {
                    const uint32_t* bw = reinterpret_cast<const uint32_t*>(bv);
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        v[2 * e] = __float_as_uint(__uint_as_float(v[2 * e]) + __uint_as_float(bw[e] << 16));
                        v[2 * e + 1] = __float_as_uint(__uint_as_float(v[2 * e + 1]) + __uint_as_float(bw[e] & 0xFFFF0000u));
                    }
                } else if (p.bias) {
                    for (int e = 0; e < 32; ++e)
                        if (col0 + e < p.N) v[e] = __float_as_uint(__uint_as_float(v[e]) + __bfloat162float(p.bias[col0 + e]));
                }
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
                    st_shared_v4(slab + row_off + ((((uint32_t)cc) ^ row_xor) << 4),
                                 pack_bf16(__uint_as_float(v[8 * cc]), __uint_as_float(v[8 * cc + 1])),
                                 pack_bf16(__uint_as_float(v[8 * cc + 2]), __uint_as_float(v[8 * cc + 3])),
                                 pack_bf16(__uint_as_float(v[8 * cc + 4]), __uint_as_float(v[8 * cc + 5])),
                                 pack_bf16(__uint_as_float(v[8 * cc + 6]), __uint_as_float(v[8 * cc + 7])));
                fence_proxy_async_smem();
                __syncwarp();
                if (elect_one()) {
                    tma_store_2d(&tmC, slab, col0, m0 + q * 32);
                    tma_store_commit();
                }
                __syncwarp();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&out_empty[buf]));
        }
        tma_store_wait_read<0>();                            // shared memory may go once the stores have read it
        __syncwarp();
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

template <int BN, bool A_MN, bool B_MN>
lrd_status_t launch_p(const CUtensorMap& tA, const CUtensorMap& tB, const CUtensorMap& tC, const PParams& p, unsigned blocks,
                      cudaStream_t stream) {
    auto kern = tc_gemm_persistent_kernel<BN, A_MN, B_MN>;
    static bool configured = false;     // per instantiation; the attribute is sticky per function
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, PCfg<BN>::SMEM_BYTES) != cudaSuccess)
            return LRD_ERR_CUDA;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = PCfg<BN>::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // the kernel waits (griddepcontrol.wait) before it touches global memory
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, tA, tB, tC, p) != cudaSuccess) return LRD_ERR_CUDA;
    count_launch();
    return LRD_OK;
}

template <int BN>
lrd_status_t launch_p_major(bool a_mn, bool b_mn, const CUtensorMap& tA, const CUtensorMap& tB, const CUtensorMap& tC,
                            const PParams& p, unsigned blocks, cudaStream_t s) {
    if (a_mn) return b_mn ? launch_p<BN, true, true>(tA, tB, tC, p, blocks, s) : launch_p<BN, true, false>(tA, tB, tC, p, blocks, s);
    return b_mn ? launch_p<BN, false, true>(tA, tB, tC, p, blocks, s) : launch_p<BN, false, false>(tA, tB, tC, p, blocks, s);
}

// Tile width: every block streams (A tile + B tile) per k-block and the slowest block walks over
// ceil(tiles / SMs) tiles, so minimise that product; wider tiles on ties (fewer re-reads of A).
int pick_bn_p(int64_t M, int64_t N) {
    if (N <= 64) return 64;
    const int64_t mt = (M + BM - 1) / BM;
    const int cands[4] = {256, 192, 128, 64};
    int best = 128;
    double best_cost = 1e300;
    for (int bn : cands) {
        const int64_t tiles = mt * ((N + bn - 1) / bn);
        const double cost = (double)((tiles + kNumSms - 1) / kNumSms) * (double)(kATile + bn * BK * 2);
        if (cost < best_cost) { best_cost = cost; best = bn; }
    }
    return best;
}

}  // namespace

lrd_status_t tc_gemm_persistent(const GemmArgs& g, cudaStream_t stream) {
    if (!tc_gemm_eligible(g) || g.a_colsum) return LRD_ERR_UNSUPPORTED;
    const int bn = pick_bn_p(g.M, g.N);
    CUtensorMap tA, tB, tC;
    bool ok = g.a_mn_major ? make_tmap_2d_bf16(&tA, g.A, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.lda, BK, 64)
                           : make_tmap_2d_bf16(&tA, g.A, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)g.lda, BM, BK);
    ok = ok && (g.b_mn_major ? make_tmap_2d_bf16(&tB, g.B, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)g.ldb, BK, 64)
                             : make_tmap_2d_bf16(&tB, g.B, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.ldb, (uint32_t)bn, BK));
    ok = ok && make_tmap_2d_bf16(&tC, g.C, (uint64_t)g.M, (uint64_t)g.N, (uint64_t)g.ldc, 32, 32);
    if (!ok) return LRD_ERR_CUDA;
    PParams p;
    p.M = g.M; p.N = g.N;
    p.kb_total = (int)((g.K + BK - 1) / BK);
    p.m_tiles = (int)((g.M + BM - 1) / BM);
    p.n_tiles = (int)((g.N + bn - 1) / bn);
    p.bias = (const __nv_bfloat16*)g.bias;
    p.timeout_flag = device_timeout_flag();
    const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
    // every block gets the same number of tiles (+-1): blocks = tiles / ceil(tiles / SMs), rounded up
    const int64_t waves = (tiles + kNumSms - 1) / kNumSms;
    const unsigned blocks = (unsigned)((tiles + waves - 1) / waves);
    switch (bn) {
        case 256: return launch_p_major<256>(g.a_mn_major, g.b_mn_major, tA, tB, tC, p, blocks, stream);
        case 192: return launch_p_major<192>(g.a_mn_major, g.b_mn_major, tA, tB, tC, p, blocks, stream);
        case 128: return launch_p_major<128>(g.a_mn_major, g.b_mn_major, tA, tB, tC, p, blocks, stream);
        default:  return launch_p_major<64>(g.a_mn_major, g.b_mn_major, tA, tB, tC, p, blocks, stream);
    }
}

}  // namespace lrd
