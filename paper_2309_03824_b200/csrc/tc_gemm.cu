// Tensor-core matrix product for sm_100a: TMA -> shared memory (128-byte swizzle) ->
// tcgen05.mma with the accumulator in tensor memory -> tcgen05.ld epilogue.
//
//   C[M x N] = op(A) op(B) (+ bias), bf16 in, fp32 accumulate, bf16 out.  The reduction dimension
//   may be split over gridDim.z (weight gradients reduce over all tokens but have few output tiles):
//     cluster split   the z blocks of a tile form a thread-block cluster; each block stages its fp32
//                     partial tile in shared memory, sends every peer the column slice that peer owns
//                     (bulk DSMEM copies) and adds the slices it receives in rank order -- one launch,
//                     no partials in global memory, a fixed order of additions;
//     global split    fp32 partial tiles in scratch memory that a second kernel adds in a fixed order
//                     (tiles wider than the cluster path supports, or more splits than a cluster holds).
//   No floating-point atomics anywhere: weight gradients are bit-reproducible.
//
// One 128 x BN output tile per block.  Warp 0 issues the TMA loads of the A operand and warp 6 those of the
// B operand (issuing a copy costs a thread about a hundred clocks, and an MN-major operand takes one copy per
// 64 columns: one warp alone issues a 40 KB stage in about 0.4 us, less than the memory system delivers),
// warp 1 owns tensor memory and issues the MMAs, warps 2-5 read the accumulator (each its own quarter of the
// 128 lanes) and store.  The single-thread instructions are issued under elect.sync by a converged warp.  Both
// operands may be K-major (reduction index contiguous) or MN-major (row / column index contiguous),
// which covers every product of the forward and backward pass without a transposed copy.
#include <algorithm>

#include "common.cuh"
#include "ptx.cuh"
#include "tc.cuh"
#include "tma.cuh"

namespace lrd {
namespace {

using namespace ptx;

constexpr int BM = 128, BK = 64;
constexpr int kThreads = 224;                         // warp 6: second TMA producer (the B operand)
constexpr uint32_t A_STAGE_BYTES = BM * BK * 2;
constexpr int kMaxClusterSplits = 8;                 // portable cluster size

// ONES: every stage carries one more 64-wide MN-major block of B that holds 1.0 everywhere and is never
// overwritten; with N = BN + 16 the MMA then also forms sum_k A(m, k) in accumulator column BN (the bias
// gradient falls out of the dU product: its A operand is dY).
template <int BN, bool ONES = false> struct Cfg {
    static constexpr uint32_t B_STAGE_BYTES = BN * BK * 2 + (ONES ? 8192 : 0);
    static constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int STAGES_RAW = (200 * 1024) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
    // cluster split: fp32 staging tile + receive slots of the same size (+ column-sum slots), over the dead ring
    static constexpr uint32_t REDUCE_BYTES = BN <= 192 ? 2u * 128u * BN * 4u + 512u * (kMaxClusterSplits + 1) : 0u;
    static constexpr uint32_t RING_BYTES = STAGES * STAGE_BYTES;
    static constexpr uint32_t SMEM_BYTES = (RING_BYTES > REDUCE_BYTES ? RING_BYTES : REDUCE_BYTES) + 1024;   // + slack for 1024-B alignment
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
    int cluster_splits; // > 1: the gridDim.z blocks of a tile are one cluster and reduce through shared memory
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
    __shared__ __align__(8) uint64_t full_bar[STAGES], empty_bar[STAGES], acc_bar, red_bar;
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
        mbar_init(smem_u32(&red_bar), 1);
        if (p.cluster_splits > 1) {                        // bytes the peers will send this block
            const uint32_t S = (uint32_t)p.cluster_splits;
            uint32_t tx = (S - 1u) * 128u * (BN / S) * 4u;
            if (ONES && blockIdx.x == 0 && cluster_ctarank() == 0) tx += (S - 1u) * 512u;
            mbar_expect_tx(smem_u32(&red_bar), tx);
        }
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
    // set-up above touched only this block's own shared and tensor memory: it may overlap the tail of the
    // previous kernel in the stream; global memory is first touched below this line
    griddep_launch_dependents();
    griddep_wait();

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
                mbar_expect_tx(fb, A_STAGE_BYTES + BN * BK * 2);       // the whole stage: warp 6's copies complete on the same barrier
                if (A_MN) {
#pragma unroll
                    for (int j = 0; j < BM / 64; ++j) tma_load_2d(a_dst + j * 8192, &tmA, fb, m0 + 64 * j, k0);
                } else {
                    tma_load_2d(a_dst, &tmA, fb, k0, m0);
                }
            }
            __syncwarp();
            (void)b_dst;
        }
        if (p.cluster_splits > 1) { cluster_arrive(); cluster_wait(); cluster_arrive_relaxed(); }   // barriers 1 and 2, see the epilogue
    } else if (warp == 6) {
        // second TMA producer: the B operand of every stage (its bytes are counted by warp 0's expect_tx; a copy that
        // lands before that arrival only makes the barrier's byte count negative for a moment)
        int it = 0;
        for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1;
            if (!mbar_wait_uniform(smem_u32(&empty_bar[s]), ph ^ 1, ab)) break;
            const uint32_t fb = smem_u32(&full_bar[s]);
            const uint32_t b_dst = smem_base + s * C::STAGE_BYTES + A_STAGE_BYTES;
            const int k0 = kb * BK;
            if (elect_one()) {
                if (B_MN) {
#pragma unroll
                    for (int j = 0; j < BN / 64; ++j) tma_load_2d(b_dst + j * 8192, &tmB, fb, n0 + 64 * j, k0);
                } else {
                    tma_load_2d(b_dst, &tmB, fb, k0, n0);
                }
            }
            __syncwarp();
        }
        if (p.cluster_splits > 1) { cluster_arrive(); cluster_wait(); cluster_arrive_relaxed(); }
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
        if (p.cluster_splits > 1) { cluster_arrive(); cluster_wait(); cluster_arrive_relaxed(); }
    } else if (p.cluster_splits > 1) {
        // ---- cluster split: reduce the partial tiles of the cluster's blocks through shared memory ----
        const int quarter = warp % 4;
        const int row = quarter * 32 + lane;
        const uint32_t S = (uint32_t)p.cluster_splits, self = cluster_ctarank();
        const uint32_t cs = BN / S;                        // columns this block owns (multiple of 8)
        const uint32_t chunk_bytes = 128u * cs * 4u, ngrp = cs / 4u;
        const uint32_t stage_base = smem_base, recv_base = smem_base + 128u * BN * 4u;
        const uint32_t cs_stage = recv_base + 128u * BN * 4u, cs_recv = cs_stage + 512u;
        const bool with_colsum = ONES && blockIdx.x == 0;
        bool ok = mbar_wait_warp(smem_u32(&acc_bar), 0, ab);
        tc_fence_after();
        // barrier 1: this block's pipeline ring is dead (all its MMAs have completed).  Progress only: what the peers
        // must see of this block (its initialised barriers) is released by the arrivals of warps 0 and 1.
        cluster_arrive_relaxed();
        if (ok) {
            // partial tile -> staging, laid out [owner][row][cs] so that each owner's slice is one contiguous range
            const bool has_work = kb_begin < kb_end;       // a block past the end of the reduction contributes zeros
            // within a row of a slice the 16-byte groups are rotated by the row index: rows a power of two
            // apart in bytes would otherwise all hit the same banks
            const uint32_t rot = (uint32_t)row % ngrp;
            uint32_t grp = 0, dst_row = stage_base + (uint32_t)row * cs * 4u;   // group within the slice, row of the current owner's slice
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                if (has_work) {
                    tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + c * 32, v);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = 0u;
                }
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    uint32_t rg = grp + rot;
                    if (rg >= ngrp) rg -= ngrp;
                    st_shared_v4(dst_row + rg * 16u, v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                    if (++grp == ngrp) { grp = 0; dst_row += chunk_bytes; }
                }
            }
            if (with_colsum) {
                uint32_t cv[16];
                if (has_work) {
                    tmem_ld_32x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + BN, cv);
                    tmem_ld_wait();
                } else {
                    cv[0] = 0u;
                }
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(cs_stage + (uint32_t)row * 4u), "r"(cv[0]) : "memory");
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        cluster_wait();        // barrier 1 complete: every peer's ring is dead, its receive slots may be written
        ok = named_bar_and(2, 128, ok);
        if (warp == 2) {
            if (ok && elect_one()) {
                for (uint32_t t = 1; t < S; ++t) {
                    const uint32_t peer = (self + t) % S;
                    dsmem_bulk_copy(recv_base + self * chunk_bytes, stage_base + peer * chunk_bytes, chunk_bytes, smem_u32(&red_bar), peer);
                }
                if (with_colsum && self != 0) dsmem_bulk_copy(cs_recv + self * 512u, cs_stage, 512u, smem_u32(&red_bar), 0);
            }
            __syncwarp();
        }
        if (ok) {
            bool got = false;
            if (lane == 0) got = mbar_wait_cluster(smem_u32(&red_bar), 0, ab);
            ok = __shfl_sync(0xffffffffu, got ? 1 : 0, 0) != 0;
            if (ok) { for (int i = 0; i < 64 && !mbar_try_wait_cluster(smem_u32(&red_bar), 0); ++i) {} }
        }
        cluster_arrive_relaxed();   // barrier 2: everything addressed to this block has landed (progress only, no data)
        if (ok) {
            // this block's column slice: add the S partials in rank order, round once, store
            const int64_t grow = (int64_t)m0 + row;
            const int64_t gcol0 = (int64_t)n0 + self * cs;
            const uint32_t rot = (uint32_t)row % ngrp;
            // 8 columns of this row: the S partials in rank order (+ bias), rounded once
            auto sum8 = [&](uint32_t c4, uint32_t (&w)[4], float (&acc)[8]) {
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = 0.f;
                uint32_t g0 = c4 / 4u + rot, g1 = c4 / 4u + 1u + rot;
                if (g0 >= ngrp) g0 -= ngrp;
                if (g1 >= ngrp) g1 -= ngrp;
#pragma unroll 2
                for (uint32_t k = 0; k < S; ++k) {
                    const uint32_t row_base = (k == self ? stage_base + self * chunk_bytes : recv_base + k * chunk_bytes) + (uint32_t)row * cs * 4u;
                    float4 x, y;
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w) : "r"(row_base + g0 * 16u));
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(y.x), "=f"(y.y), "=f"(y.z), "=f"(y.w) : "r"(row_base + g1 * 16u));
                    acc[0] += x.x; acc[1] += x.y; acc[2] += x.z; acc[3] += x.w;
                    acc[4] += y.x; acc[5] += y.y; acc[6] += y.z; acc[7] += y.w;
                }
                const int64_t col = gcol0 + c4;
                if (p.bias) {
                    for (int e = 0; e < 8; ++e)
                        if (col + e < p.N) acc[e] += __bfloat162float(p.bias[col + e]);
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) w[e] = pack_bf16(acc[2 * e], acc[2 * e + 1]);
            };
            auto store8 = [&](uint32_t c4, const uint32_t (&w)[4], const float (&acc)[8]) {
                const int64_t col = gcol0 + c4;
                if (grow >= p.M || col >= p.N) return;
                __nv_bfloat16* dst = (__nv_bfloat16*)p.C + grow * p.ldc + col;
                if (col + 8 <= p.N) {
                    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
                } else {
                    for (int e = 0; e < 8; ++e)
                        if (col + e < p.N) dst[e] = __float2bfloat16_rn(acc[e]);
                }
            };
            // 16 columns (one whole 32-byte sector) per store instruction where the layout allows, else two 16-byte stores
            const bool sectors = (p.ldc % 16 == 0) && (((uintptr_t)p.C & 31u) == 0) && (gcol0 % 16 == 0);
            for (uint32_t c4 = 0; c4 < cs; c4 += 16) {
                uint32_t w0[4], w1[4];
                float a0[8], a1[8];
                sum8(c4, w0, a0);
                const bool second = c4 + 8 < cs;
                if (second) sum8(c4 + 8, w1, a1);
                const int64_t col = gcol0 + c4;
                if (sectors && second && grow < p.M && col + 16 <= p.N) {
                    __nv_bfloat16* dst = (__nv_bfloat16*)p.C + grow * p.ldc + col;
                    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                                 ::"l"(dst), "r"(w0[0]), "r"(w0[1]), "r"(w0[2]), "r"(w0[3]), "r"(w1[0]), "r"(w1[1]), "r"(w1[2]), "r"(w1[3]) : "memory");
                } else {
                    store8(c4, w0, a0);
                    if (second) store8(c4 + 8, w1, a1);
                }
            }
            if (with_colsum && self == 0 && p.colsum_out && grow < p.M) {
                float t = 0.f;
                for (uint32_t k = 0; k < S; ++k) {
                    const uint32_t src = (k == 0 ? cs_stage : cs_recv + k * 512u) + (uint32_t)row * 4u;
                    float x;
                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x) : "r"(src));
                    t += x;
                }
                p.colsum_out[grow] = __float2bfloat16_rn(t);
            }
        }
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

    // cluster split, barrier 2: no block leaves while a peer may still be reading its slice out of this
    // block's shared memory
    if (p.cluster_splits > 1) cluster_wait();
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
    static bool configured_on[kMaxDevices] = {};     // per instantiation; the attribute is sticky per function
    bool& configured = configured_on[device_slot()];
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<BN, ONES>::SMEM_BYTES) != cudaSuccess)
            return LRD_ERR_CUDA;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = Cfg<BN, ONES>::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = p.cluster_splits > 1 ? (unsigned)p.cluster_splits : 1u;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // the kernel waits (griddepcontrol.wait) before it touches global memory
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, kern, tA, tB, p) != cudaSuccess) return LRD_ERR_CUDA;
    count_launch();
    return LRD_OK;
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

// Tile width.  Every MMA of a tile reads its 128 x 16 block of A from shared memory whatever its width, and
// every tile streams its own copy of A, so a narrow tile pays the same A traffic for fewer columns: below
// about 154 columns the cost of a k-block is taken as constant, above as proportional to the width.
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

static int global_splits(int64_t M, int64_t N, int64_t K, int bn) {
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

// Clusters of S blocks that can be resident at once (S blocks need S free SMs inside one GPC, so this is
// fewer than SMs / S).  All instantiations hold one block per SM, so one of them answers for all.
static int max_active_clusters(int S) {
    static int cache_on[kMaxDevices][kMaxClusterSplits + 1] = {};
    int* cache = cache_on[device_slot()];
    if (S < 2 || S > kMaxClusterSplits) return kNumSms;
    if (cache[S] == 0) {
        auto kern = tc_gemm_kernel<64, true, true, false>;
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(1, 1, (unsigned)S);
        cfg.blockDim = dim3(kThreads, 1, 1);
        cfg.dynamicSmemBytes = Cfg<64, false>::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 1;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = (unsigned)S;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<64, false>::SMEM_BYTES) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = (kNumSms - 20) / S;                     // no answer (no device yet): a cautious guess
        }
        cache[S] = n;
    }
    return cache[S];
}

// How a product whose reduction may be split is run.
struct SplitPlan {
    int bn;
    int cluster;     // > 1: cluster split (blocks per tile)
    int global;      // > 1: global split (partials in scratch memory + reduce kernel)
};

// Cluster split: the time of one block is its operand traffic (every block streams its share of A and
// B through one SM's memory port); all blocks together must not exceed what L2 delivers.  The
// candidates are tile widths that the reduction buffers fit (<= 192) and cluster sizes that divide
// the tile into slices of whole 16-byte groups.
static SplitPlan pick_split(int64_t M, int64_t N, int64_t K, bool ones, int max_cluster = 0) {
    const int top = max_cluster >= 2 && max_cluster < kMaxClusterSplits ? max_cluster : kMaxClusterSplits;
    const int64_t mt = (M + BM - 1) / BM, kb = (K + BK - 1) / BK;
    SplitPlan best{pick_bn(M, N, true), 1, 1};
    if (ones && best.bn > 192) best.bn = 192;
    best.global = global_splits(M, N, K, best.bn);
    double best_t = 1e300;
    const int bns[3] = {192, 128, 64};
    for (int bn : bns) {
        const int64_t nt = (N + bn - 1) / bn;
        if (nt * bn >= N + 64 && bn > 64) continue;              // a narrower width covers N with less waste
        const int64_t tiles = mt * nt;
        for (int S = top; S >= 2; --S) {
            if (bn % (8 * S)) continue;
            if (tiles > max_active_clusters(S) || S > kb) continue;    // one wave: a second wave would double the time
            const double per_block = (double)((kb + S - 1) / S) * (A_STAGE_BYTES + bn * BK * 2.0);
            const double t = std::max(per_block / 110e9, per_block * (double)(tiles * S) / 11.5e12) + 2e-6 * bn / 192.0;
            if (t < best_t) { best_t = t; best.bn = bn; best.cluster = S; best.global = 1; }
            break;                                                // the largest feasible cluster for this width
        }
    }
    return best;
}

int tc_pick_splits(int64_t M, int64_t N, int64_t K) { return pick_split(M, N, K, false).global; }

// fp32 partial tiles [splits][M][ldp], then (for the optional column sums) [splits][M]; nothing for a cluster split
size_t tc_split_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    size_t need = 0;
    for (int v = 0; v < 4; ++v) {                    // with and without the column sums, for either cluster limit
        const int ones = v & 1;
        const int s = pick_split(M, N, K, ones != 0, (v & 2) ? 2 : 0).global;
        const size_t n = s > 1 ? align_up((size_t)s * M * ((N + 3) / 4 * 4) * sizeof(float), 256) + align_up((size_t)s * M * sizeof(float), 256) : 0;
        need = need > n ? need : n;
    }
    return need;
}

bool tc_gemm_colsum_ok(const GemmArgs& g) {
    return tc_gemm_eligible(g) && g.a_mn_major && g.b_mn_major && (((uintptr_t)g.a_colsum & 1u) == 0);
}

lrd_status_t tc_gemm(const GemmArgs& g, bool allow_split, float* partials, size_t partial_bytes,
                     cudaStream_t stream) {
    if (!tc_gemm_eligible(g)) return LRD_ERR_UNSUPPORTED;
    const bool ones = g.a_colsum != nullptr;
    if (ones && !tc_gemm_colsum_ok(g)) return LRD_ERR_UNSUPPORTED;
    if (!allow_split && !ones) return tc_gemm_persistent(g, stream);   // data products: the persistent kernel
    int splits = 1, cluster = 1, bn;
    if (allow_split) {
        const SplitPlan sp = pick_split(g.M, g.N, g.K, ones, g.max_cluster_split);
        bn = sp.bn; cluster = sp.cluster; splits = sp.global;
    } else {
        bn = pick_bn(g.M, g.N, false);
        if (ones && bn > 192) bn = 192;                // the ones block needs 16 accumulator columns beside the tile
    }
    const int64_t ldp = (g.N + 3) / 4 * 4;
    const size_t tile_bytes = align_up((size_t)splits * g.M * ldp * sizeof(float), 256);
    if (splits > 1 && (!partials || partial_bytes < tile_bytes + (ones ? (size_t)splits * g.M * sizeof(float) : 0)))
        return LRD_ERR_WORKSPACE;
    const int kb_total = (int)((g.K + BK - 1) / BK);
    const int zdim = cluster > 1 ? cluster : splits;
    const int kb_per = (kb_total + zdim - 1) / zdim;

    CUtensorMap tA, tB;
    bool ok = g.a_mn_major ? make_tmap_2d_bf16(&tA, g.A, (uint64_t)g.K, (uint64_t)g.M, (uint64_t)g.lda, BK, 64)
                           : make_tmap_2d_bf16(&tA, g.A, (uint64_t)g.M, (uint64_t)g.K, (uint64_t)g.lda, BM, BK);
    ok = ok && (g.b_mn_major ? make_tmap_2d_bf16(&tB, g.B, (uint64_t)g.K, (uint64_t)g.N, (uint64_t)g.ldb, BK, 64)
                             : make_tmap_2d_bf16(&tB, g.B, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.ldb, (uint32_t)bn, BK));
    if (!ok) return LRD_ERR_CUDA;

    TcParams p;
    p.M = g.M; p.N = g.N; p.ldp = ldp; p.kb_total = kb_total; p.kb_per_split = kb_per;
    p.partial = splits > 1 ? 1 : 0;
    p.cluster_splits = cluster;
    p.timeout_flag = device_timeout_flag();
    p.C = splits > 1 ? (void*)partials : g.C;
    p.ldc = g.ldc;
    p.bias = splits > 1 ? nullptr : (const __nv_bfloat16*)g.bias;
    p.colsum_partial = (ones && splits > 1) ? (float*)((uint8_t*)partials + tile_bytes) : nullptr;
    p.colsum_out = (ones && splits == 1) ? (__nv_bfloat16*)g.a_colsum : nullptr;
    dim3 grid((unsigned)((g.N + bn - 1) / bn), (unsigned)((g.M + BM - 1) / BM), (unsigned)zdim);
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
