// Tensor-core 3x3 core convolution of the Tucker-2 layer (stride 1, zero pad 1, NHWC, bf16) as an
// implicit GEMM on sm_100a.  No im2col buffer exists anywhere: for every filter tap the A operand is a
// shifted window of the image fetched by one 4-D TMA box; the hardware's out-of-bounds zero fill is the
// padding.
//
//   conv_kernel<false>: forward        out[p][o] = sum_{tap,i} in [p + tap][i] G[o][tap][i]
//   conv_kernel<true> : data gradient  din[p][i] = sum_{tap,o} dout[p - tap][o] G[o][tap][i]
//   filter_kernel     : filter gradient dG[o][tap][i] = sum_p dout[p][o] in[p + tap][i]   (split over
//                       pixel chunks, fp32 partials added in a fixed order by filter_reduce_kernel)
//   conv_kernel<.., true> (fused): the 1x1 product that follows the core runs in the same kernel.  The
//                       tile of the core's result is rounded to bf16 into shared memory (K-major,
//                       128-byte swizzle; written to memory only if the caller needs it), the ring,
//                       dead by then, receives the 1x1 factor Q[N2 x n1], and a second set of MMAs forms
//                       out2[p][:] = core[p][:] Q^T (+ bias) in other tensor-memory columns:
//                       forward  Y = conv(Z1, G) Bm^T + b,  backward  dX = conv^T(dZ2, G) A^T.
//
// A tile is bh rows of one image (bh * W <= 128 pixels = the 128 MMA rows / the reduction chunk).
// Warp roles as in the matrix-product kernel: TMA producer, MMA issuer (both issue under elect.sync from a converged warp), 4 epilogue warps.
#include "common.cuh"
#include "conv.cuh"
#include "ptx.cuh"
#include "tc.cuh"
#include "tma.cuh"

namespace lrd {
namespace {

using namespace ptx;

constexpr int kThreads = 192;
constexpr int kStages = 6;                           // what a block streams is its stages in flight over a stage's turn-around
constexpr uint32_t kTile = 128 * 128;               // one operand tile slot: 128 rows x 64 channels of bf16
constexpr uint32_t kStageBytes = 2 * kTile;          // A slot + B slot (N = 128: one K-major tile or two 64-wide MN-major boxes)
constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024;

struct ConvParams {
    int B, H, W, bh, tiles_per_img;
    int ka;                 // channels of the A-side image (reduction per tap)
    int n_total;            // output channels of this product (columns of out)
    int g_ci;               // Ci of G[o][tap][i] (its row length is 9 * g_ci)
    int sign;               // +1 forward, -1 data gradient
    __nv_bfloat16* out;     // [B*H*W][n_total]; fused: nullable (the core's result is then never written to memory)
    unsigned int* timeout_flag;
    // fused 1x1 product
    int n2;                       // columns of out2 (<= 256)
    __nv_bfloat16* out2;          // [B*H*W][n2]
    const __nv_bfloat16* bias2;   // [n2] or nullptr
};

// grid: (ceil(n_total / 128), tiles_per_img, B); fused: gridDim.x = 1 and the block walks over the (one or two) column tiles
template <bool DGRAD, bool FUSE>
__global__ void __launch_bounds__(kThreads, 1)
conv_kernel(const __grid_constant__ CUtensorMap tmImg, const __grid_constant__ CUtensorMap tmG,
            const __grid_constant__ CUtensorMap tmQ, const ConvParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kStages], empty_bar[kStages], acc_bar, q_full, t_ready, out_full;
    constexpr uint32_t kTmemCols = FUSE ? 512 : 128;        // fused: the second product accumulates in columns [256, 512)
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const AbortCtx ab{&abort_flag, p.timeout_flag};
    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0), lane = threadIdx.x % 32;
    const int h0 = blockIdx.y * p.bh, img = blockIdx.z;
    // 128-column tiles of the core's result: one per block (gridDim.x), or, fused, all of them (up to two) in this block
    const int n_tiles = FUSE ? (p.n_total + 127) / 128 : 1;
    const int nkc = (p.ka + 63) / 64;                  // 64-channel blocks per tap
    const int iters = 9 * nkc;
    const uint32_t a_bytes = (uint32_t)(p.bh * p.W) * 128u;
    const uint32_t stage_tx = a_bytes + 2u * 64u * 128u;   // B: 128 x 64 (K-major) or 2 x [64 x 64] (MN-major)

    if (threadIdx.x == 0) {
        abort_flag = 0;
        prefetch_tmap(&tmImg);
        prefetch_tmap(&tmG);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        mbar_init(smem_u32(&acc_bar), 1);
        mbar_init(smem_u32(&q_full), 1);
        mbar_init(smem_u32(&t_ready), 4);
        mbar_init(smem_u32(&out_full), 1);
        if (FUSE) prefetch_tmap(&tmQ);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // set-up above touched only this block's own shared and tensor memory: under programmatic dependent launch it
    // overlaps the tail of the previous kernel in the stream; global memory is first touched below this line
    griddep_launch_dependents();
    griddep_wait();
    // fused: once the core's MMAs are done the ring is dead; it then holds [T: one atom of 128 rows x 64 columns per 64
    // columns of the core's result | Q: one [256 rows x 64 k] tile per 64 columns of the core's result]
    const int nq = (p.n_total + 63) / 64;
    const uint32_t t_base = smem_base, q_base = smem_base + (uint32_t)nq * kTile;

    if (warp == 0) {
        // TMA producer: the whole warp runs the loop, one elected lane issues
        int s = 0;
        uint32_t ph = 1;
        bool go = true;
        for (int nt = 0; nt < n_tiles && go; ++nt)
        for (int it = 0; it < iters; ++it) {
            const int n0 = FUSE ? nt * 128 : (int)blockIdx.x * 128;
            const int tap = it / nkc, cb = it % nkc;
            const int kh = tap / 3, kw = tap % 3;
            if (!mbar_wait_uniform(smem_u32(&empty_bar[s]), ph, ab)) { go = false; break; }
            const uint32_t fb = smem_u32(&full_bar[s]);
            const uint32_t a_dst = smem_base + s * kStageBytes, b_dst = a_dst + kTile;
            if (elect_one()) {
                mbar_expect_tx(fb, stage_tx);
                // image window of this tap: rows h0 + sign (kh - 1) ..., columns sign (kw - 1) ...; outside = zeros
                tma_load_4d(a_dst, &tmImg, fb, cb * 64, p.sign * (kw - 1), h0 + p.sign * (kh - 1), img);
                if (DGRAD) {           // B[n = i][k = o] = G[o][tap][i]: MN-major, rows o of this block, 64 columns of i per box
                    tma_load_2d(b_dst, &tmG, fb, tap * p.g_ci + n0, cb * 64);
                    tma_load_2d(b_dst + 8192, &tmG, fb, tap * p.g_ci + n0 + 64, cb * 64);
                } else {               // B[n = o][k = i] = G[o][tap][i]: K-major, 128 rows of o
                    tma_load_2d(b_dst, &tmG, fb, tap * p.g_ci + cb * 64, n0);
                }
            }
            __syncwarp();
            if (++s == kStages) { s = 0; ph ^= 1; }
        }
        if (FUSE) {                                          // the 1x1 factor, into the dead ring (rows past n2, columns past n1: zeros)
            if (mbar_wait_uniform(smem_u32(&acc_bar), 0, ab)) {
                if (elect_one()) {
                    mbar_expect_tx(smem_u32(&q_full), (uint32_t)nq * 2u * kTile);
                    for (int kb = 0; kb < nq; ++kb) tma_load_2d(q_base + kb * 2 * kTile, &tmQ, smem_u32(&q_full), kb * 64, 0);
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        // MMA issuer: converged warp, elect.sync around the issue
        constexpr uint32_t idesc = idesc_bf16(128, false, DGRAD);
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int nt = 0; nt < n_tiles && ok; ++nt)
        for (int it = 0; it < iters; ++it) {
            ok = mbar_wait_uniform(smem_u32(&full_bar[s]), ph, ab);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_src = smem_base + s * kStageBytes, b_src = a_src + kTile;
            const uint32_t acc = tmem_base + (uint32_t)nt * 128u;
            const int nks = min(4, (p.ka - (it % nkc) * 64 + 15) / 16);      // 16-channel steps past ka hold zeros: not issued
            if (elect_one()) {
                const uint64_t ad0 = smem_desc_sw128(a_src, 0, 1024);
                const uint64_t bd0 = DGRAD ? smem_desc_sw128(b_src, 8192, 1024) : smem_desc_sw128(b_src, 0, 1024);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)                               // the k-step moves the start address only
                    if (kk < nks) mma_bf16_ss(acc, ad0 + 2u * kk, bd0 + (DGRAD ? 128u : 2u) * kk, idesc, (it > 0 || kk > 0) ? 1u : 0u);
                mma_commit(smem_u32(&empty_bar[s]));
            }
            __syncwarp();
            if (++s == kStages) { s = 0; ph ^= 1; }
        }
        if (ok && elect_one()) mma_commit(smem_u32(&acc_bar));
        __syncwarp();
        if (FUSE) {                                          // out2 tile = T Q^T, reduction over the n_total columns of T
            if (ok) ok = mbar_wait_uniform(smem_u32(&t_ready), 0, ab);
            if (ok) ok = mbar_wait_uniform(smem_u32(&q_full), 0, ab);
            if (ok) {
                tc_fence_after();
                const uint32_t idesc2 = idesc_bf16((p.n2 + 15) / 16 * 16, false, false);
                if (elect_one()) {
                    for (int ks = 0; ks * 16 < p.n_total; ++ks) {
                        const uint64_t ad = smem_desc_sw128(t_base + (ks / 4) * kTile + (ks % 4) * 32, 0, 1024);
                        const uint64_t bd = smem_desc_sw128(q_base + (ks / 4) * 2 * kTile + (ks % 4) * 32, 0, 1024);
                        mma_bf16_ss(tmem_base + 256u, ad, bd, idesc2, ks > 0 ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&out_full));
                }
                __syncwarp();
            }
        }
    } else {
        const int q = warp % 4;
        const bool ready = mbar_wait_uniform(smem_u32(&acc_bar), 0, ab);
        tc_fence_after();
        const int row = q * 32 + lane;                           // pixel of the tile: (h0 + row / W, row % W)
        const bool row_ok = row < p.bh * p.W && h0 + row / p.W < p.H;
        if (ready) {
            __nv_bfloat16* dst_row = p.out + ((int64_t)(img * p.H + h0) * p.W + row) * p.n_total;
            const int n0 = FUSE ? 0 : (int)blockIdx.x * 128;
#pragma unroll 1
            for (int cchunk = 0; cchunk < 4 * n_tiles; ++cchunk) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + cchunk * 32, v);
                tmem_ld_wait();
                const int col0 = n0 + cchunk * 32;
                if (FUSE) {                                  // bf16 tile T for the second product (rows past the tile hold
                    if (col0 < p.n_total) {                  // garbage that only reaches output rows nobody stores)
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const uint32_t col = (uint32_t)(cchunk * 32 + g * 8);
                            st_shared_v4(t_base + (col / 64u) * kTile + (uint32_t)row * 128u + ((((col % 64u) / 8u) ^ ((uint32_t)row & 7u)) << 4),
                                         pack_bf16(__uint_as_float(v[8 * g]), __uint_as_float(v[8 * g + 1])),
                                         pack_bf16(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3])),
                                         pack_bf16(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5])),
                                         pack_bf16(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7])));
                        }
                    }
                    if (!p.out) continue;
                }
                if (!row_ok || col0 >= p.n_total) continue;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    if (col0 + g * 8 + 8 <= p.n_total) {
                        *reinterpret_cast<uint4*>(dst_row + col0 + g * 8) =
                            make_uint4(pack_bf16(__uint_as_float(v[8 * g]), __uint_as_float(v[8 * g + 1])),
                                       pack_bf16(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3])),
                                       pack_bf16(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5])),
                                       pack_bf16(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7])));
                    } else {
                        for (int e = 0; e < 8; ++e)
                            if (col0 + g * 8 + e < p.n_total) dst_row[col0 + g * 8 + e] = __float2bfloat16_rn(__uint_as_float(v[8 * g + e]));
                    }
                }
            }
        }
        if (FUSE) {
            fence_proxy_async_smem();                        // T was written by ordinary stores, the MMA reads it through the async proxy
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&t_ready));
            const bool done = ready && mbar_wait_uniform(smem_u32(&out_full), 0, ab);
            tc_fence_after();
            if (done) {
                __nv_bfloat16* dst_row = p.out2 + ((int64_t)(img * p.H + h0) * p.W + row) * p.n2;
                const bool bias_vec = p.bias2 && (((uintptr_t)p.bias2 & 15u) == 0);
#pragma unroll 1
                for (int cchunk = 0; cchunk * 32 < p.n2; ++cchunk) {
                    const int col0 = cchunk * 32;
                    uint4 bv[4] = {};
                    const bool bvec = bias_vec && col0 + 32 <= p.n2;
                    if (bvec) {
                        const uint4* bp = reinterpret_cast<const uint4*>(p.bias2 + col0);
#pragma unroll
                        for (int e = 0; e < 4; ++e) bv[e] = __ldg(bp + e);
                    }
                    uint32_t v[32];
                    tmem_ld_32x32(tmem_base + 256u + ((uint32_t)(q * 32) << 16) + cchunk * 32, v);
                    tmem_ld_wait();
                    if (!row_ok) continue;
                    if (bvec) {
                        const uint32_t* bw = reinterpret_cast<const uint32_t*>(bv);
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            v[2 * e] = __float_as_uint(__uint_as_float(v[2 * e]) + __uint_as_float(bw[e] << 16));
                            v[2 * e + 1] = __float_as_uint(__uint_as_float(v[2 * e + 1]) + __uint_as_float(bw[e] & 0xFFFF0000u));
                        }
                    } else if (p.bias2) {
                        for (int e = 0; e < 32; ++e)
                            if (col0 + e < p.n2) v[e] = __float_as_uint(__uint_as_float(v[e]) + __bfloat162float(p.bias2[col0 + e]));
                    }
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        if (col0 + g * 8 + 8 <= p.n2) {
                            *reinterpret_cast<uint4*>(dst_row + col0 + g * 8) =
                                make_uint4(pack_bf16(__uint_as_float(v[8 * g]), __uint_as_float(v[8 * g + 1])),
                                           pack_bf16(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3])),
                                           pack_bf16(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5])),
                                           pack_bf16(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7])));
                        } else {
                            for (int e = 0; e < 8; ++e)
                                if (col0 + g * 8 + e < p.n2) dst_row[col0 + g * 8 + e] = __float2bfloat16_rn(__uint_as_float(v[8 * g + e]));
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (abort_flag)
            for (int i = 0; i < 256; ++i) __nanosleep(1000);
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---- filter gradient ------------------------------------------------------------------------------
constexpr int kFStages = 3;
constexpr uint32_t kFStageBytes = 4 * kTile;         // two 64-wide slots of dout (M = o) + two of the shifted image (N = i)
constexpr uint32_t kFSmemBytes = kFStages * kFStageBytes + 1024;

struct FilterParams {
    int B, H, W, bh, tiles_per_img, co, ci, tiles_i;
    int chunks_total, chunks_per_split;     // a chunk = one tile of one image = bh * W pixels of the reduction
    int ldp;                                // leading dimension of a partial [co x ci] block (ci rounded up to 4)
    float* partial;                         // [splits][9][co][ldp]
    unsigned int* timeout_flag;
};

// grid: (9 taps, tiles_o * tiles_i, splits)
__global__ void __launch_bounds__(kThreads, 1)
filter_kernel(const __grid_constant__ CUtensorMap tmDout, const __grid_constant__ CUtensorMap tmIn, const FilterParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kFStages], empty_bar[kFStages], acc_bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const AbortCtx ab{&abort_flag, p.timeout_flag};
    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0), lane = threadIdx.x % 32;
    const int tap = blockIdx.x, kh = tap / 3, kw = tap % 3;
    const int m0 = (blockIdx.y / p.tiles_i) * 128, n0 = (blockIdx.y % p.tiles_i) * 128;
    const int c_begin = blockIdx.z * p.chunks_per_split;
    const int c_end = min(c_begin + p.chunks_per_split, p.chunks_total);
    const int rows = p.bh * p.W;                        // pixels per chunk (<= 128)
    const int ksteps = (rows + 15) / 16;
    const uint32_t box_bytes = (uint32_t)rows * 128u;

    // Rows of a slot past the box are never written by TMA; they must read as zero in the last 16-row
    // MMA step, so the whole ring starts out zeroed.
    for (uint32_t off = threadIdx.x * 16u; off < kFStages * kFStageBytes; off += kThreads * 16u)
        st_shared_v4(smem_base + off, 0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    if (threadIdx.x == 0) {
        abort_flag = 0;
        prefetch_tmap(&tmDout);
        prefetch_tmap(&tmIn);
        for (int s = 0; s < kFStages; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        mbar_init(smem_u32(&acc_bar), 1);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), 128);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // set-up above touched only this block's own shared and tensor memory: under programmatic dependent launch it
    // overlaps the tail of the previous kernel in the stream; global memory is first touched below this line
    griddep_launch_dependents();
    griddep_wait();

    if (warp == 0) {
        int s = 0;
        uint32_t ph = 1;
        for (int ch = c_begin; ch < c_end; ++ch) {
            const int img = ch / p.tiles_per_img, h0 = (ch % p.tiles_per_img) * p.bh;
            if (!mbar_wait_uniform(smem_u32(&empty_bar[s]), ph, ab)) break;
            const uint32_t fb = smem_u32(&full_bar[s]);
            const uint32_t dst = smem_base + s * kFStageBytes;
            if (elect_one()) {
                mbar_expect_tx(fb, 4u * box_bytes);
                tma_load_4d(dst, &tmDout, fb, m0, 0, h0, img);
                tma_load_4d(dst + kTile, &tmDout, fb, m0 + 64, 0, h0, img);
                tma_load_4d(dst + 2 * kTile, &tmIn, fb, n0, kw - 1, h0 + kh - 1, img);
                tma_load_4d(dst + 3 * kTile, &tmIn, fb, n0 + 64, kw - 1, h0 + kh - 1, img);
            }
            __syncwarp();
            if (++s == kFStages) { s = 0; ph ^= 1; }
        }
    } else if (warp == 1) {
        constexpr uint32_t idesc = idesc_bf16(128, true, true);
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int ch = c_begin; ch < c_end; ++ch) {
            ok = mbar_wait_uniform(smem_u32(&full_bar[s]), ph, ab);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_src = smem_base + s * kFStageBytes, b_src = a_src + 2 * kTile;
            if (elect_one()) {
                for (int kk = 0; kk < ksteps; ++kk) {
                    const uint64_t ad = smem_desc_sw128(a_src + kk * 2048, kTile, 1024);
                    const uint64_t bd = smem_desc_sw128(b_src + kk * 2048, kTile, 1024);
                    mma_bf16_ss(tmem_base, ad, bd, idesc, (ch > c_begin || kk > 0) ? 1u : 0u);
                }
                mma_commit(smem_u32(&empty_bar[s]));
            }
            __syncwarp();
            if (++s == kFStages) { s = 0; ph ^= 1; }
        }
        if (ok && elect_one()) mma_commit(smem_u32(&acc_bar));
        __syncwarp();
    } else {
        const int q = warp % 4;
        const bool ready = mbar_wait_warp(smem_u32(&acc_bar), 0, ab);
        tc_fence_after();
        if (ready) {
            const int o = m0 + q * 32 + lane;
            float* dst_row = p.partial + (((int64_t)blockIdx.z * 9 + tap) * p.co + o) * p.ldp;
#pragma unroll 1
            for (int cchunk = 0; cchunk < 4; ++cchunk) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + cchunk * 32, v);
                tmem_ld_wait();
                const int col0 = n0 + cchunk * 32;
                if (o >= p.co || col0 >= p.ci) continue;
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    if (col0 + g * 4 + 4 <= p.ci) {
                        *reinterpret_cast<uint4*>(dst_row + col0 + g * 4) = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                    } else {
                        for (int e = 0; e < 4; ++e)
                            if (col0 + g * 4 + e < p.ci) dst_row[col0 + g * 4 + e] = __uint_as_float(v[4 * g + e]);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (abort_flag)
            for (int i = 0; i < 256; ++i) __nanosleep(1000);
        tc_fence_after();
        tmem_dealloc(tmem_base, 128);
    }
}

// dG[o][tap][i] = sum_z partial[z][tap][o][i], z ascending.
__global__ void __launch_bounds__(256) filter_reduce_kernel(const float* __restrict__ partial, int splits, int co, int ci,
                                                            int ldp, __nv_bfloat16* __restrict__ dG) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)co * 9 * ci) return;
    const int i = (int)(idx % ci), t = (int)((idx / ci) % 9), o = (int)(idx / ((int64_t)9 * ci));
    float acc = 0.f;
    for (int z = 0; z < splits; ++z) acc += partial[(((int64_t)z * 9 + t) * co + o) * ldp + i];
    dG[idx] = __float2bfloat16_rn(acc);
}

}  // namespace

namespace {

struct Geo { int bh, tiles_per_img; };

inline bool a16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

bool geometry(int64_t B, int64_t H, int64_t W, int64_t ci, int64_t co, Geo* g) {
    if (W < 1 || W > 128 || H < 1 || B < 1 || B > 65535 || ci % 8 || co % 8) return false;
    int bh = (int)(128 / W);
    if (bh > H) bh = (int)H;
    if (bh > 256) bh = 256;
    g->bh = bh;
    g->tiles_per_img = (int)((H + bh - 1) / bh);
    return g->tiles_per_img <= 65535;
}

int filter_splits(int64_t B, const Geo& g, int64_t ci, int64_t co) {
    const int64_t blocks = 9 * ((co + 127) / 128) * ((ci + 127) / 128);
    const int64_t chunks = B * g.tiles_per_img;
    int64_t s = (kNumSms + blocks - 1) / blocks;
    if (s > chunks) s = chunks;
    if (s > 64) s = 64;
    if (s < 1) s = 1;
    const int64_t per = (chunks + s - 1) / s;
    return (int)((chunks + per - 1) / per);
}

// Launch with the programmatic-serialization attribute: the kernel waits (griddepcontrol.wait) before it
// touches global memory, so its set-up may overlap the previous kernel's tail.
template <typename K, typename... Args>
void launch_pdl(K kern, dim3 grid, uint32_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kern, args...);     // errors surface through cudaGetLastError() at the call site
}

template <typename K>
bool set_smem(K kern, uint32_t bytes) {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess;
}

}  // namespace

bool tc_conv_eligible(int64_t B, int64_t H, int64_t W, int64_t ci, int64_t co, lrd_dtype_t dt, const void* p0,
                      const void* p1, const void* p2) {
    Geo g;
    return dt == LRD_BF16 && a16(p0) && a16(p1) && a16(p2) && geometry(B, H, W, ci, co, &g);
}

size_t tc_conv_filter_scratch_bytes(int64_t B, int64_t H, int64_t W, int64_t ci, int64_t co) {
    Geo g;
    if (!geometry(B, H, W, ci, co, &g)) return 0;
    const int splits = filter_splits(B, g, ci, co);
    return align_up((size_t)splits * 9 * co * ((ci + 3) / 4 * 4) * sizeof(float), 256);
}

// forward (dgrad = false: img = in [..][ci], out [..][co]) or data gradient (dgrad = true: img = dout [..][co], out = din [..][ci])
lrd_status_t tc_conv3x3(bool dgrad, const void* img, const void* G, void* out, int64_t B, int64_t H, int64_t W, int64_t ci,
                        int64_t co, cudaStream_t s) {
    Geo g;
    if (!geometry(B, H, W, ci, co, &g)) return LRD_ERR_UNSUPPORTED;
    const int64_t ka = dgrad ? co : ci, n_total = dgrad ? ci : co;
    CUtensorMap tImg, tG;
    bool ok = make_tmap_nhwc_bf16(&tImg, img, (uint64_t)B, (uint64_t)H, (uint64_t)W, (uint64_t)ka, (uint32_t)g.bh, (uint32_t)W, 64);
    ok = ok && make_tmap_2d_bf16(&tG, G, (uint64_t)co, (uint64_t)(9 * ci), (uint64_t)(9 * ci), dgrad ? 64 : 128, 64);
    if (!ok) return LRD_ERR_CUDA;
    ConvParams p;
    p.B = (int)B; p.H = (int)H; p.W = (int)W; p.bh = g.bh; p.tiles_per_img = g.tiles_per_img;
    p.ka = (int)ka; p.n_total = (int)n_total; p.g_ci = (int)ci; p.sign = dgrad ? -1 : 1;
    p.out = (__nv_bfloat16*)out; p.timeout_flag = device_timeout_flag();
    p.n2 = 0; p.out2 = nullptr; p.bias2 = nullptr;
    static bool configured_on[kMaxDevices] = {};
    bool& configured = configured_on[device_slot()];
    if (!configured) {
        if (!set_smem(conv_kernel<false, false>, kSmemBytes) || !set_smem(conv_kernel<true, false>, kSmemBytes)) return LRD_ERR_CUDA;
        configured = true;
    }
    dim3 grid((unsigned)((n_total + 127) / 128), (unsigned)g.tiles_per_img, (unsigned)B);
    if (dgrad) launch_pdl(conv_kernel<true, false>, grid, kSmemBytes, s, tImg, tG, tG, p);
    else launch_pdl(conv_kernel<false, false>, grid, kSmemBytes, s, tImg, tG, tG, p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

bool tc_conv_chain_eligible(bool dgrad, int64_t B, int64_t H, int64_t W, int64_t ci, int64_t co, int64_t n2, lrd_dtype_t dt,
                            const void* img, const void* G, const void* Q, const void* out2, const void* core_out) {
    const int64_t n1 = dgrad ? ci : co;                  // channels of the core's result = reduction of the 1x1 product
    if (!tc_conv_eligible(B, H, W, ci, co, dt, img, G, Q)) return false;
    if (n1 > 256 || n1 % 16 || n2 < 8 || n2 > 256 || n2 % 8) return false;
    return a16(out2) && (!core_out || a16(core_out));
}

// The core followed by the 1x1 product out2[p][:] = core[p][:] Q^T (+ bias2) in one launch.  Q is [n2 x n1] with n1
// contiguous; core_out (nullable) receives the core's bf16 result when the caller needs it later.
lrd_status_t tc_conv3x3_chain(bool dgrad, const void* img, const void* G, const void* Q, const void* bias2, void* out2,
                              void* core_out, int64_t B, int64_t H, int64_t W, int64_t ci, int64_t co, int64_t n2,
                              cudaStream_t s) {
    Geo g;
    if (!geometry(B, H, W, ci, co, &g)) return LRD_ERR_UNSUPPORTED;
    const int64_t ka = dgrad ? co : ci, n1 = dgrad ? ci : co;
    CUtensorMap tImg, tG, tQ;
    bool ok = make_tmap_nhwc_bf16(&tImg, img, (uint64_t)B, (uint64_t)H, (uint64_t)W, (uint64_t)ka, (uint32_t)g.bh, (uint32_t)W, 64);
    ok = ok && make_tmap_2d_bf16(&tG, G, (uint64_t)co, (uint64_t)(9 * ci), (uint64_t)(9 * ci), dgrad ? 64 : 128, 64);
    ok = ok && make_tmap_2d_bf16(&tQ, Q, (uint64_t)n2, (uint64_t)n1, (uint64_t)n1, 256, 64);
    if (!ok) return LRD_ERR_CUDA;
    ConvParams p;
    p.B = (int)B; p.H = (int)H; p.W = (int)W; p.bh = g.bh; p.tiles_per_img = g.tiles_per_img;
    p.ka = (int)ka; p.n_total = (int)n1; p.g_ci = (int)ci; p.sign = dgrad ? -1 : 1;
    p.out = (__nv_bfloat16*)core_out; p.timeout_flag = device_timeout_flag();
    p.n2 = (int)n2; p.out2 = (__nv_bfloat16*)out2; p.bias2 = (const __nv_bfloat16*)bias2;
    static bool configured_on[kMaxDevices] = {};
    bool& configured = configured_on[device_slot()];
    if (!configured) {
        if (!set_smem(conv_kernel<false, true>, kSmemBytes) || !set_smem(conv_kernel<true, true>, kSmemBytes)) return LRD_ERR_CUDA;
        configured = true;
    }
    dim3 grid(1, (unsigned)g.tiles_per_img, (unsigned)B);
    if (dgrad) launch_pdl(conv_kernel<true, true>, grid, kSmemBytes, s, tImg, tG, tQ, p);
    else launch_pdl(conv_kernel<false, true>, grid, kSmemBytes, s, tImg, tG, tQ, p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

lrd_status_t tc_conv3x3_filter(const void* dout, const void* in, void* dG, int64_t B, int64_t H, int64_t W, int64_t ci,
                               int64_t co, float* scratch, size_t scratch_bytes, cudaStream_t s) {
    Geo g;
    if (!geometry(B, H, W, ci, co, &g)) return LRD_ERR_UNSUPPORTED;
    if (!scratch || scratch_bytes < tc_conv_filter_scratch_bytes(B, H, W, ci, co)) return LRD_ERR_WORKSPACE;
    CUtensorMap tD, tI;
    bool ok = make_tmap_nhwc_bf16(&tD, dout, (uint64_t)B, (uint64_t)H, (uint64_t)W, (uint64_t)co, (uint32_t)g.bh, (uint32_t)W, 64);
    ok = ok && make_tmap_nhwc_bf16(&tI, in, (uint64_t)B, (uint64_t)H, (uint64_t)W, (uint64_t)ci, (uint32_t)g.bh, (uint32_t)W, 64);
    if (!ok) return LRD_ERR_CUDA;
    const int splits = filter_splits(B, g, ci, co);
    FilterParams p;
    p.B = (int)B; p.H = (int)H; p.W = (int)W; p.bh = g.bh; p.tiles_per_img = g.tiles_per_img;
    p.co = (int)co; p.ci = (int)ci; p.tiles_i = (int)((ci + 127) / 128);
    p.chunks_total = (int)(B * g.tiles_per_img);
    p.chunks_per_split = (p.chunks_total + splits - 1) / splits;
    p.ldp = (int)((ci + 3) / 4 * 4);
    p.partial = scratch; p.timeout_flag = device_timeout_flag();
    static bool configured_on[kMaxDevices] = {};
    bool& configured = configured_on[device_slot()];
    if (!configured) {
        if (!set_smem(filter_kernel, kFSmemBytes)) return LRD_ERR_CUDA;
        configured = true;
    }
    dim3 grid(9, (unsigned)(((co + 127) / 128) * p.tiles_i), (unsigned)splits);
    launch_pdl(filter_kernel, grid, kFSmemBytes, s, tD, tI, p);
    const int64_t n = co * 9 * ci;
    filter_reduce_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(scratch, splits, (int)co, (int)ci, p.ldp, (__nv_bfloat16*)dG);
    count_launch(2);
    return cudaGetLastError() == cudaSuccess ? LRD_OK : LRD_ERR_CUDA;
}

}  // namespace lrd
