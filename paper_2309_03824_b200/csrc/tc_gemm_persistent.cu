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
//
// CG = 2 runs the same loop on pairs of blocks (a cluster of two SMs, tcgen05 cta_group::2): a pair owns a
// 256 x BN tile, each block loads its own 128 rows of A but only HALF of the B tile, and the even block
// issues MMAs of 256 rows that read both halves.  Per k-block a block then takes (16 KB + BN x 64 B)
// instead of (16 KB + BN x 128 B) through its L2 -> shared-memory path, which is what bounds the wide
// tiles: at BN = 256 the shared-memory port sees 64 KB (fill + operand reads) per 512 MMA cycles instead
// of 96 KB.
#include "common.cuh"
#include "ptx_pair.cuh"
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

template <int BN, int CG> struct PCfg {
    static constexpr int BNH = BN / CG;                      // columns of B this block loads
    static constexpr uint32_t STAGE_BYTES = kATile + BNH * BK * 2;
    static constexpr int STAGES_RAW = (200 * 1024) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
    static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + kStagingBytes + 1024;
    static constexpr uint32_t TMEM_COLS = 2 * BN <= 128 ? 128 : (2 * BN <= 256 ? 256 : 512);
    static constexpr uint32_t BUF_COLS = TMEM_COLS / 2;      // column offset of the second accumulator
};

template <int CG>
__device__ __forceinline__ void load2d(uint32_t dst, const CUtensorMap* m, uint32_t bar, int x, int y) {
    if (CG == 2) tma_load_2d_pair(dst, m, bar, x, y);        // bar: shared::cluster address (the even block's barrier)
    else tma_load_2d(dst, m, bar, x, y);
}

struct PParams {
    int64_t M, N;
    int kb_total, m_tiles, n_tiles;
    const __nv_bfloat16* bias;
    unsigned int* timeout_flag;
};

template <int BN, bool A_MN, bool B_MN, int CG>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_persistent_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                          const __grid_constant__ CUtensorMap tmC, const PParams p) {
    using C = PCfg<BN, CG>;
    constexpr int BNH = C::BNH;
    static_assert(CG == 1 || CG == 2, "blocks per MMA");
    static_assert(CG == 1 || !B_MN || BNH % 64 == 0, "an MN-major half of B is made of 64-column boxes");
    constexpr int STAGES = C::STAGES;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[STAGES], empty_bar[STAGES], out_full[2], out_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging_base = smem_base, ring_base = smem_base + kStagingBytes;
    const AbortCtx ab{&abort_flag, p.timeout_flag};
    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0), lane = threadIdx.x % 32;
    const int n_tiles_total = p.m_tiles * p.n_tiles;         // p.m_tiles counts row tiles of 128 CG rows
    const int h = CG == 2 ? (int)cluster_ctarank() : 0;      // this block's half of the pair
    const int unit = (int)blockIdx.x / CG, n_units = (int)gridDim.x / CG;

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
            mbar_init(smem_u32(&out_empty[i]), 4 * CG);       // the epilogue warps of every block of the pair
        }
        fence_mbar_init();
    }
    if (warp == 1) {
        if (CG == 2) {
            tmem_alloc_pair(smem_u32(&tmem_base_slot), C::TMEM_COLS);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(&tmem_base_slot), C::TMEM_COLS);
            tmem_relinquish();
        }
    }
    tc_fence_before();
    if (CG == 2) {                   // the other block's barriers exist before anything signals them
        cluster_arrive();
        cluster_wait();
    } else {
        __syncthreads();
    }
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
        for (int t = unit; t < n_tiles_total && ok; t += n_units) {
            const int m0 = (t % p.m_tiles) * (BM * CG) + h * BM, n0 = (t / p.m_tiles) * BN + h * BNH;
            for (int kb = 0; kb < p.kb_total; ++kb) {
                ok = mbar_wait_uniform(smem_u32(&empty_bar[s]), ph, ab);
                if (!ok) break;
                // a pair's loads all complete on the even block's barrier, which its MMA warp waits on
                const uint32_t fb_local = smem_u32(&full_bar[s]);
                const uint32_t fb = CG == 2 ? map_to_cta(fb_local, 0) : fb_local;
                const uint32_t a_dst = ring_base + s * C::STAGE_BYTES, b_dst = a_dst + kATile;
                const int k0 = kb * BK;
                if (elect_one()) {
                    if (h == 0) mbar_expect_tx(fb_local, CG * C::STAGE_BYTES);
                    if (A_MN) {
#pragma unroll
                        for (int j = 0; j < BM / 64; ++j) load2d<CG>(a_dst + j * 8192, &tmA, fb, m0 + 64 * j, k0);
                    } else {
                        load2d<CG>(a_dst, &tmA, fb, k0, m0);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int j = 0; j < BNH / 64; ++j) load2d<CG>(b_dst + j * 8192, &tmB, fb, n0 + 64 * j, k0);
                    } else {
                        load2d<CG>(b_dst, &tmB, fb, k0, n0);
                    }
                }
                __syncwarp();
                if (++s == STAGES) { s = 0; ph ^= 1; }
            }
        }
    } else if (warp == 1 && h == 0) {
        // ------------------------------------------------------------------ MMA issuer (the even block of a pair)
        constexpr uint32_t idesc = CG == 2 ? idesc_bf16_pair(BN, A_MN, B_MN) : idesc_bf16(BN, A_MN, B_MN);
        int s = 0, i = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int t = unit; t < n_tiles_total && ok; t += n_units, ++i) {
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
                        if (CG == 2) mma_bf16_ss_pair(d_tmem, ad, bd, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
                        else mma_bf16_ss(d_tmem, ad, bd, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
                    }
                    if (CG == 2) {       // both blocks' stages are free, both blocks' accumulators are ready
                        mma_commit_pair(smem_u32(&empty_bar[s]), 3);
                        if (kb == p.kb_total - 1) mma_commit_pair(smem_u32(&out_full[buf]), 3);
                    } else {
                        mma_commit(smem_u32(&empty_bar[s]));
                        if (kb == p.kb_total - 1) mma_commit(smem_u32(&out_full[buf]));
                    }
                }
                __syncwarp();
                if (++s == STAGES) { s = 0; ph ^= 1; }
            }
        }
    } else if (warp >= 2) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp % 4;                              // tensor-memory lanes [32 q, 32 q + 32)
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t slab0 = staging_base + (uint32_t)(warp - 2) * 2u * kSlabBytes;
        const uint32_t row_off = (uint32_t)lane * 64u, row_xor = ((uint32_t)lane >> 1) & 3u;
        const bool bias_ok = p.bias && (((uintptr_t)p.bias & 15u) == 0);
        int i = 0, sb = 0;
        bool ok = true;
        for (int t = unit; t < n_tiles_total && ok; t += n_units, ++i) {
            const int buf = i & 1;
            const int m0 = (t % p.m_tiles) * (BM * CG) + h * BM, n0 = (t / p.m_tiles) * BN;
            const bool rows_inside = m0 + q * 32 < p.M;      // (uniform) a pair's odd block may hang over the last row tile
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
                    if (rows_inside) tma_store_2d(&tmC, slab, col0, m0 + q * 32);
                    tma_store_commit();
                }
                __syncwarp();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CG == 2) mbar_arrive_remote(smem_u32(&out_empty[buf]), 0);
                else mbar_arrive(smem_u32(&out_empty[buf]));
            }
        }
        tma_store_wait_read<0>();                            // shared memory may go once the stores have read it
        __syncwarp();
    }

    tc_fence_before();
    if (CG == 2) {
        // neither block leaves (or frees tensor memory) while the other may still signal one of its barriers,
        // read its shared memory with an MMA or write its accumulators: every thread of the pair is past all of
        // that when it arrives here
        cluster_arrive();
        cluster_wait();
    } else {
        __syncthreads();
    }
    if (warp == 1) {
        if (abort_flag) {            // give copies and MMAs still in flight time to land before freeing
            for (int i = 0; i < 256; ++i) __nanosleep(1000);
        }
        tc_fence_after();
        if (CG == 2) tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
        else tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

template <int BN, bool A_MN, bool B_MN, int CG>
lrd_status_t launch_p(const CUtensorMap& tA, const CUtensorMap& tB, const CUtensorMap& tC, const PParams& p, unsigned blocks,
                      cudaStream_t stream) {
    auto kern = tc_gemm_persistent_kernel<BN, A_MN, B_MN, CG>;
    static bool configured_on[kMaxDevices] = {};     // per instantiation; the attribute is sticky per function
    bool& configured = configured_on[device_slot()];
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, PCfg<BN, CG>::SMEM_BYTES) != cudaSuccess)
            return LRD_ERR_CUDA;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = PCfg<BN, CG>::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // the kernel waits (griddepcontrol.wait) before it touches global memory
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = CG;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = CG == 2 ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kern, tA, tB, tC, p) != cudaSuccess) return LRD_ERR_CUDA;
    count_launch();
    return LRD_OK;
}

template <int BN, int CG>
lrd_status_t launch_p_major(bool a_mn, bool b_mn, const CUtensorMap& tA, const CUtensorMap& tB, const CUtensorMap& tC,
                            const PParams& p, unsigned blocks, cudaStream_t s) {
    if (a_mn) return b_mn ? launch_p<BN, true, true, CG>(tA, tB, tC, p, blocks, s) : launch_p<BN, true, false, CG>(tA, tB, tC, p, blocks, s);
    return b_mn ? launch_p<BN, false, true, CG>(tA, tB, tC, p, blocks, s) : launch_p<BN, false, false, CG>(tA, tB, tC, p, blocks, s);
}

// Tile shape.  Per k-block a block streams (A tile + its part of the B tile) from L2 at about 64 B/clk and
// its MMAs take 2 BN clocks; the slowest unit walks over ceil(tiles / units) tiles.  Minimise the product over
// the tile widths and over single blocks (148 units, 128-row tiles) and pairs (74 units, 256-row tiles);
// earlier candidates (wider, single) win ties.
struct PShape { int bn, cg; };
int g_force_cg = 0;                  // 0: by the cost above; 1 or 2: forced where possible (test hook)

PShape pick_shape_p(int64_t M, int64_t N) {
    if (N <= 64) return {64, 1};
    const int cands[4] = {256, 192, 128, 64};
    PShape best = {128, 1};
    double best_cost = 1e300;
    for (int cg = 1; cg <= 2; ++cg) {
        if (g_force_cg && cg != g_force_cg) continue;
        if (cg == 2 && M <= BM) continue;
        const int64_t mt = (M + BM * cg - 1) / (BM * cg);
        const int64_t units = kNumSms / cg;
        for (int bn : cands) {
            if (cg == 2 && bn != 256 && bn != 128) continue;
            const int64_t tiles = mt * ((N + bn - 1) / bn);
            const double fill = (double)(kATile + (bn / cg) * BK * 2) / 64.0, mma = 2.0 * bn;
            const double cost = (double)((tiles + units - 1) / units) * (fill > mma ? fill : mma);
            if (cost < best_cost) { best_cost = cost; best = {bn, cg}; }
        }
    }
    return best;
}

}  // namespace

void tc_gemm_persistent_force_pairs(int cg) { g_force_cg = (cg == 1 || cg == 2) ? cg : 0; }

lrd_status_t tc_gemm_persistent(const GemmArgs& g, cudaStream_t stream) {
    if (!tc_gemm_eligible(g) || g.a_colsum) return LRD_ERR_UNSUPPORTED;
    PShape sh = pick_shape_p(g.M, g.N);
    if (g_force_cg == 2 && sh.cg != 2) { g_force_cg = 0; sh = pick_shape_p(g.M, g.N); g_force_cg = 2; }
    const int bn = sh.bn, cg = sh.cg, bnh = bn / cg;
    CUtensorMap tA, tB, tC;
    bool ok = g.a_mn_major ? make_tmap_2d_bf16(&tA, g.A, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.lda, BK, 64)
                           : make_tmap_2d_bf16(&tA, g.A, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)g.lda, BM, BK);
    ok = ok && (g.b_mn_major ? make_tmap_2d_bf16(&tB, g.B, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)g.ldb, BK, 64)
                             : make_tmap_2d_bf16(&tB, g.B, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.ldb, (uint32_t)bnh, BK));
    ok = ok && make_tmap_2d_bf16(&tC, g.C, (uint64_t)g.M, (uint64_t)g.N, (uint64_t)g.ldc, 32, 32);
    if (!ok) return LRD_ERR_CUDA;
    PParams p;
    p.M = g.M; p.N = g.N;
    p.kb_total = (int)((g.K + BK - 1) / BK);
    p.m_tiles = (int)((g.M + BM * cg - 1) / (BM * cg));
    p.n_tiles = (int)((g.N + bn - 1) / bn);
    p.bias = (const __nv_bfloat16*)g.bias;
    p.timeout_flag = device_timeout_flag();
    const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles, units_max = kNumSms / cg;
    // every unit (block or pair) gets the same number of tiles (+-1): units = tiles / ceil(tiles / units_max), rounded up
    const int64_t waves = (tiles + units_max - 1) / units_max;
    const unsigned blocks = (unsigned)((tiles + waves - 1) / waves) * (unsigned)cg;
    if (cg == 2) {
        if (bn == 256) return launch_p_major<256, 2>(g.a_mn_major, g.b_mn_major, tA, tB, tC, p, blocks, stream);
        return launch_p_major<128, 2>(g.a_mn_major, g.b_mn_major, tA, tB, tC, p, blocks, stream);
    }
    switch (bn) {
        case 256: return launch_p_major<256, 1>(g.a_mn_major, g.b_mn_major, tA, tB, tC, p, blocks, stream);
        case 192: return launch_p_major<192, 1>(g.a_mn_major, g.b_mn_major, tA, tB, tC, p, blocks, stream);
        case 128: return launch_p_major<128, 1>(g.a_mn_major, g.b_mn_major, tA, tB, tC, p, blocks, stream);
        default:  return launch_p_major<64, 1>(g.a_mn_major, g.b_mn_major, tA, tB, tC, p, blocks, stream);
    }
}

}  // namespace lrd
