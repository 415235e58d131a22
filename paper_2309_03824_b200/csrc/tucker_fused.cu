// One launch for a whole data pass of the Tucker-2 layer (3 x 3 core, stride 1, zero pad 1, NHWC, bf16) on sm_100a:
//
//   forward   Y  = conv(X A, G) Bm^T + b        (In = X,  P1 = A [C x r1],  P3 = Bm [S x r2])
//   backward  dX = conv^T(dY Bm, G) A^T         (In = dY, P1 = Bm [S x r2], P3 = A [C x r1])
//
// A block owns bh rows of one image.  Three products follow each other on chip:
//   A  T1 = In_halo P1 on the tile WITH its halo rows (bh + 2 image rows of W pixels = the 128 MMA rows; one 4-D TMA
//      box per 64 input channels, rows outside the image arrive as zeros, so their T1 is zero = the core's
//      padding).  The accumulator is rounded to bf16 into shared memory as [8-channel slab][pixel slot][8 channels],
//      unswizzled, pixel slot = row * (W + 2) + column + 1: the columns left and right of the image are slots that
//      stay zero.
//   B  T2 = core(T1): for every tap the A operand is the SAME buffer read from a shifted start address (slot shift
//      kh (W + 2) + kw forward, (2 - kh)(W + 2) + (2 - kw) backward), which the unswizzled layout allows at 16-byte
//      granularity; B is the tap's slice of G (by TMA, one tap per stage).  Output rows are pixel slots of the bh
//      output rows, W + 2 wide (the two extra columns per row are computed and never stored).
//   C  Out = T2 P3^T (+ bias): T2 rounded to bf16 into shared memory (K-major, 128-byte swizzle), P3 by TMA into
//      the ring.
// T1 (its bh interior rows) and T2 go to global memory only where the caller needs them later (the saved
// activations Z1 / Z2 of the forward pass, dZ2 / dZ1 of the backward pass).
// Warp 0: TMA producer (one ring for all three phases).  Warp 1: tensor memory + MMA issue.  Warps 2-5: the three
// epilogues.  Every wait is bounded; a wait that runs out raises the device timeout flag and the block tears down.
#include "common.cuh"
#include "conv.cuh"
#include "ptx.cuh"
#include "tc.cuh"
#include "tma.cuh"

namespace lrd {
namespace {

using namespace ptx;

constexpr int kThreads = 192;
constexpr int kSlots = 4;
constexpr uint32_t kTile = 128 * 128;                // 128 rows x 64 channels of bf16
constexpr uint32_t kSlotBytes = 2 * kTile;           // a stage of any phase fits 32 KB
constexpr uint32_t kZ2Bytes = 2 * kTile;             // T2: up to 128 channels
constexpr uint32_t kAcc2Col = 128, kAcc3Col = 256;   // tensor-memory columns of the three accumulators: 0, 128, 256

struct FusedParams {
    int H, W, PW, bh;             // image, padded row width W + 2, output rows per tile
    int c_in, nA, nB, n3;         // channels: input, after the first 1x1, after the core, output
    int g_ci;                     // row length of G per tap (r1)
    int swb;                      // swizzle span of the P1 boxes (bytes); a box is 64 rows x swb / 2 columns
    int z1_slots;                 // pixel slots of the T1 buffer (a slab is z1_slots * 16 bytes)
    __nv_bfloat16* save1;         // [B H W][nA] or nullptr
    __nv_bfloat16* save2;         // [B H W][nB] or nullptr
    __nv_bfloat16* out3;          // [B H W][n3]
    const __nv_bfloat16* bias3;   // [n3] or nullptr
    unsigned int* timeout_flag;
};

// Shared-memory matrix descriptor without swizzle (K-major): 8 rows x 16 bytes are contiguous; sbo = bytes between
// 8-row groups, lbo = bytes between the two 8-element halves of a 16-deep k-step.
__device__ __forceinline__ uint64_t smem_desc_plain(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    return d;
}

// grid: (1, tiles per image, B)
template <bool DGRAD>
__global__ void __launch_bounds__(kThreads, 1)
tucker_fused_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmP1,
                    const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmP3, const FusedParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kSlots], empty_bar[kSlots], acc_bar[3], ready_bar[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const AbortCtx ab{&abort_flag, p.timeout_flag};
    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0), lane = threadIdx.x % 32;
    const int h0 = blockIdx.y * p.bh, img = blockIdx.z;
    const uint32_t slab_bytes = (uint32_t)p.z1_slots * 16u;
    const uint32_t z1_bytes = ((uint32_t)(p.nA / 8) * slab_bytes + 1023u) & ~1023u;
    const uint32_t z1_base = smem_base, z2_base = z1_base + z1_bytes, ring_base = z2_base + kZ2Bytes;
    const int HR = (p.bh + 2) * p.W;                     // rows of the haloed tile
    const int nkb1 = (p.c_in + 63) / 64;                 // stages of phase A
    const int ncbB = (p.nA + 63) / 64;                   // 64-deep k-blocks of a tap
    const int natC = (p.nB + 63) / 64;                   // stages of phase C (64-deep k-blocks of T2)
    const int atom_cols = p.swb / 2, n_pbox = p.nA / atom_cols;
    const uint32_t pbox_bytes = 64u * (uint32_t)p.swb;

    // the T1 buffer starts out zeroed: the slots left and right of the image rows, and past the tile, are the padding
    for (uint32_t off = threadIdx.x * 16u; off < z1_bytes; off += kThreads * 16u) st_shared_v4(z1_base + off, 0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    if (threadIdx.x == 0) {
        abort_flag = 0;
        prefetch_tmap(&tmIn);
        prefetch_tmap(&tmP1);
        prefetch_tmap(&tmG);
        prefetch_tmap(&tmP3);
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        for (int i = 0; i < 3; ++i) mbar_init(smem_u32(&acc_bar[i]), 1);
        for (int i = 0; i < 2; ++i) mbar_init(smem_u32(&ready_bar[i]), 4);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
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
        // ------------------------------------------------------------------ TMA producer: phases A, B, C through one ring
        int s = 0;
        uint32_t ph = 1;
        bool ok = true;
        const int stages = nkb1 + 9 + natC;
        for (int st = 0; st < stages && ok; ++st) {
            ok = mbar_wait_uniform(smem_u32(&empty_bar[s]), ph, ab);
            if (!ok) break;
            const uint32_t fb = smem_u32(&full_bar[s]);
            const uint32_t dst = ring_base + (uint32_t)s * kSlotBytes;
            if (elect_one()) {
                if (st < nkb1) {                             // In box (halo rows; outside the image: zeros) + the P1 boxes
                    mbar_expect_tx(fb, (uint32_t)HR * 128u + (uint32_t)n_pbox * pbox_bytes);
                    tma_load_4d(dst, &tmIn, fb, st * 64, 0, h0 - 1, img);
                    for (int i = 0; i < n_pbox; ++i) tma_load_2d(dst + kTile + (uint32_t)i * pbox_bytes, &tmP1, fb, i * atom_cols, st * 64);
                } else if (st < nkb1 + 9) {                  // one tap of G
                    const int tap = st - nkb1;
                    if (DGRAD) {       // B[n = i][k = o] = G[o][tap][i]: MN-major, 64 o-rows x 64 i-columns per box
                        const int nnb = (p.nB + 63) / 64;
                        mbar_expect_tx(fb, (uint32_t)(ncbB * nnb) * 8192u);
                        for (int cb = 0; cb < ncbB; ++cb)
                            for (int nb = 0; nb < nnb; ++nb)
                                tma_load_2d(dst + (uint32_t)cb * kTile + (uint32_t)nb * 8192u, &tmG, fb, tap * p.g_ci + nb * 64, cb * 64);
                    } else {           // B[n = o][k = i] = G[o][tap][i]: K-major, 128 o-rows x 64 i-columns per box
                        mbar_expect_tx(fb, (uint32_t)ncbB * kTile);
                        for (int cb = 0; cb < ncbB; ++cb) tma_load_2d(dst + (uint32_t)cb * kTile, &tmG, fb, tap * p.g_ci + cb * 64, 0);
                    }
                } else {                                     // 64 columns of P3 (256 rows)
                    mbar_expect_tx(fb, kSlotBytes);
                    tma_load_2d(dst, &tmP3, fb, (st - nkb1 - 9) * 64, 0);
                }
            }
            __syncwarp();
            if (++s == kSlots) { s = 0; ph ^= 1; }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        // phase A: T1 = In_halo P1
        const uint32_t idescA = idesc_bf16(p.nA, false, true);
        for (int st = 0; st < nkb1 && ok; ++st) {
            ok = mbar_wait_uniform(smem_u32(&full_bar[s]), ph, ab);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_src = ring_base + (uint32_t)s * kSlotBytes, b_src = a_src + kTile;
            const int nks = min(4, (p.c_in - st * 64 + 15) / 16);
            if (elect_one()) {
                const uint64_t ad0 = smem_desc_sw128(a_src, 0, 1024);
                const uint64_t bd0 = smem_desc(b_src, pbox_bytes, 8u * (uint32_t)p.swb, (uint32_t)p.swb);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    if (kk < nks) mma_bf16_ss(tmem_base, ad0 + 2u * kk, bd0 + (uint64_t)(kk * p.swb), idescA, (st > 0 || kk > 0) ? 1u : 0u);
                mma_commit(smem_u32(&empty_bar[s]));
            }
            __syncwarp();
            if (++s == kSlots) { s = 0; ph ^= 1; }
        }
        if (ok && elect_one()) mma_commit(smem_u32(&acc_bar[0]));
        __syncwarp();
        // phase B: T2 = core(T1), the A operand is the T1 buffer from a shifted start
        if (ok) ok = mbar_wait_uniform(smem_u32(&ready_bar[0]), 0, ab);
        const uint32_t idescB = idesc_bf16(p.nB, false, DGRAD);
        const uint64_t z1_desc0 = smem_desc_plain(z1_base, slab_bytes, 128);
        const uint32_t ks_units = 2u * (slab_bytes >> 4);        // a 16-deep k-step = two slabs
        for (int tap = 0; tap < 9 && ok; ++tap) {
            ok = mbar_wait_uniform(smem_u32(&full_bar[s]), ph, ab);
            if (!ok) break;
            tc_fence_after();
            const uint32_t b_src = ring_base + (uint32_t)s * kSlotBytes;
            const int kh = tap / 3, kw = tap % 3;
            const uint32_t shift = DGRAD ? (uint32_t)((2 - kh) * p.PW + (2 - kw)) : (uint32_t)(kh * p.PW + kw);
            if (elect_one()) {
                for (int cb = 0; cb < ncbB; ++cb) {
                    const int nks = min(4, (p.nA - cb * 64) / 16);
                    const uint64_t bd0 = DGRAD ? smem_desc_sw128(b_src + (uint32_t)cb * kTile, 8192, 1024)
                                               : smem_desc_sw128(b_src + (uint32_t)cb * kTile, 0, 1024);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        if (kk < nks)
                            mma_bf16_ss(tmem_base + kAcc2Col, z1_desc0 + shift + (uint32_t)(cb * 4 + kk) * ks_units,
                                        bd0 + (DGRAD ? 128u : 2u) * kk, idescB, (tap > 0 || cb > 0 || kk > 0) ? 1u : 0u);
                }
                mma_commit(smem_u32(&empty_bar[s]));
            }
            __syncwarp();
            if (++s == kSlots) { s = 0; ph ^= 1; }
        }
        if (ok && elect_one()) mma_commit(smem_u32(&acc_bar[1]));
        __syncwarp();
        // phase C: Out = T2 P3^T
        if (ok) ok = mbar_wait_uniform(smem_u32(&ready_bar[1]), 0, ab);
        const uint32_t idescC = idesc_bf16((p.n3 + 15) / 16 * 16, false, false);
        for (int kb = 0; kb < natC && ok; ++kb) {
            ok = mbar_wait_uniform(smem_u32(&full_bar[s]), ph, ab);
            if (!ok) break;
            tc_fence_after();
            const uint32_t b_src = ring_base + (uint32_t)s * kSlotBytes;
            const int nks = min(4, (p.nB - kb * 64) / 16);
            if (elect_one()) {
                const uint64_t ad0 = smem_desc_sw128(z2_base + (uint32_t)kb * kTile, 0, 1024);
                const uint64_t bd0 = smem_desc_sw128(b_src, 0, 1024);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    if (kk < nks) mma_bf16_ss(tmem_base + kAcc3Col, ad0 + 2u * kk, bd0 + 2u * kk, idescC, (kb > 0 || kk > 0) ? 1u : 0u);
                mma_commit(smem_u32(&empty_bar[s]));
            }
            __syncwarp();
            if (++s == kSlots) { s = 0; ph ^= 1; }
        }
        if (ok && elect_one()) mma_commit(smem_u32(&acc_bar[2]));
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ the three epilogues
        const int q = warp % 4;
        const int row = q * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        // T1: row = pixel of the haloed tile
        bool ok = mbar_wait_uniform(smem_u32(&acc_bar[0]), 0, ab);
        tc_fence_after();
        if (ok) {
            const int hr = row / p.W, w = row % p.W;
            const bool in_tile = row < HR;
            const int hi = h0 - 1 + hr;
            const bool keep = p.save1 && in_tile && hr >= 1 && hr <= p.bh && hi < p.H;
            const uint32_t slot_addr = z1_base + (uint32_t)(hr * p.PW + w + 1) * 16u;
            __nv_bfloat16* dst_row = p.save1 + ((int64_t)(img * p.H + hi) * p.W + w) * p.nA;
#pragma unroll 1
            for (int c0 = 0; c0 < p.nA; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32x32(lane_addr + c0, v);
                tmem_ld_wait();
                if (!in_tile) continue;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    if (c0 + g * 8 >= p.nA) break;
                    const uint32_t w0 = pack_bf16(__uint_as_float(v[8 * g]), __uint_as_float(v[8 * g + 1]));
                    const uint32_t w1 = pack_bf16(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3]));
                    const uint32_t w2 = pack_bf16(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5]));
                    const uint32_t w3 = pack_bf16(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7]));
                    st_shared_v4(slot_addr + (uint32_t)(c0 / 8 + g) * slab_bytes, w0, w1, w2, w3);
                    if (keep) *reinterpret_cast<uint4*>(dst_row + c0 + g * 8) = make_uint4(w0, w1, w2, w3);
                }
            }
        }
        fence_proxy_async_smem();                            // T1 was written by ordinary stores, the MMAs read it through the async proxy
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ready_bar[0]));
        // T2: row = pixel slot of the output rows, W + 2 wide
        const int ho = row / p.PW, wo = row % p.PW;
        const bool row_ok = ho < p.bh && wo < p.W && h0 + ho < p.H;
        const int64_t pix = (int64_t)(img * p.H + h0 + ho) * p.W + wo;
        if (ok) ok = mbar_wait_uniform(smem_u32(&acc_bar[1]), 0, ab);
        tc_fence_after();
        if (ok) {
            __nv_bfloat16* dst_row = p.save2 + pix * p.nB;
            const bool keep = p.save2 && row_ok;
#pragma unroll 1
            for (int c0 = 0; c0 < p.nB; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32x32(lane_addr + kAcc2Col + c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    if (c0 + g * 8 >= p.nB) break;
                    const uint32_t col = (uint32_t)(c0 + g * 8);
                    const uint32_t w0 = pack_bf16(__uint_as_float(v[8 * g]), __uint_as_float(v[8 * g + 1]));
                    const uint32_t w1 = pack_bf16(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3]));
                    const uint32_t w2 = pack_bf16(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5]));
                    const uint32_t w3 = pack_bf16(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7]));
                    st_shared_v4(z2_base + (col / 64u) * kTile + (uint32_t)row * 128u + ((((col % 64u) / 8u) ^ ((uint32_t)row & 7u)) << 4),
                                 w0, w1, w2, w3);
                    if (keep) *reinterpret_cast<uint4*>(dst_row + col) = make_uint4(w0, w1, w2, w3);
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ready_bar[1]));
        // Out
        if (ok) ok = mbar_wait_uniform(smem_u32(&acc_bar[2]), 0, ab);
        tc_fence_after();
        if (ok) {
            __nv_bfloat16* dst_row = p.out3 + pix * p.n3;
            const bool bias_vec = p.bias3 && (((uintptr_t)p.bias3 & 15u) == 0);
#pragma unroll 1
            for (int c0 = 0; c0 < p.n3; c0 += 32) {
                uint4 bv[4] = {};
                const bool bvec = bias_vec && c0 + 32 <= p.n3;
                if (bvec) {
                    const uint4* bp = reinterpret_cast<const uint4*>(p.bias3 + c0);
#pragma unroll
                    for (int e = 0; e < 4; ++e) bv[e] = __ldg(bp + e);
                }
                uint32_t v[32];
                tmem_ld_32x32(lane_addr + kAcc3Col + c0, v);
                tmem_ld_wait();
                if (!row_ok) continue;
                if (bvec) {
                    const uint32_t* bw = reinterpret_cast<const uint32_t*>(bv);
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        v[2 * e] = __float_as_uint(__uint_as_float(v[2 * e]) + __uint_as_float(bw[e] << 16));
                        v[2 * e + 1] = __float_as_uint(__uint_as_float(v[2 * e + 1]) + __uint_as_float(bw[e] & 0xFFFF0000u));
                    }
                } else if (p.bias3) {
                    for (int e = 0; e < 32; ++e)
                        if (c0 + e < p.n3) v[e] = __float_as_uint(__uint_as_float(v[e]) + __bfloat162float(p.bias3[c0 + e]));
                }
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    if (c0 + g * 8 + 8 <= p.n3)
                        *reinterpret_cast<uint4*>(dst_row + c0 + g * 8) =
                            make_uint4(pack_bf16(__uint_as_float(v[8 * g]), __uint_as_float(v[8 * g + 1])),
                                       pack_bf16(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3])),
                                       pack_bf16(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5])),
                                       pack_bf16(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7])));
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
        tmem_dealloc(tmem_base, 512);
    }
}

struct FusedGeo { int bh, tiles_per_img, PW, z1_slots; uint32_t smem_bytes; };

inline bool a16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

bool fused_geometry(int64_t B, int64_t H, int64_t W, int64_t c_in, int64_t nA, int64_t nB, int64_t n3, FusedGeo* g) {
    if (B < 1 || B > 65535 || H < 1 || W < 1 || W > 40) return false;
    if (c_in < 8 || c_in % 8 || nA < 16 || nA > 128 || nA % 16 || nB < 16 || nB > 128 || nB % 16 || n3 < 8 || n3 > 256 || n3 % 8) return false;
    const int PW = (int)W + 2;
    int bh = (int)(128 / W) - 2;                         // the haloed tile fits the 128 MMA rows of the first product
    if (bh > 128 / PW) bh = 128 / PW;                    // the padded output rows fit those of the core
    if (bh > H) bh = (int)H;
    if (bh < 1) return false;
    g->bh = bh;
    g->PW = PW;
    g->tiles_per_img = (int)((H + bh - 1) / bh);
    g->z1_slots = (130 + 2 * PW + 7) / 8 * 8;            // the last of 128 rows at the largest shift still reads inside the buffer
    const uint32_t z1_bytes = ((uint32_t)(nA / 8) * (uint32_t)g->z1_slots * 16u + 1023u) & ~1023u;
    g->smem_bytes = 1024u + z1_bytes + kZ2Bytes + kSlots * kSlotBytes;
    return g->tiles_per_img <= 65535 && g->smem_bytes <= 226u * 1024u;
}

}  // namespace

bool tucker_fused_eligible(int64_t B, int64_t H, int64_t W, int64_t c_in, int64_t nA, int64_t nB, int64_t n3, lrd_dtype_t dt,
                           const void* in, const void* P1, const void* G, const void* P3, const void* out3, const void* save1,
                           const void* save2) {
    FusedGeo g;
    return dt == LRD_BF16 && a16(in) && a16(P1) && a16(G) && a16(P3) && a16(out3) && (!save1 || a16(save1)) && (!save2 || a16(save2)) &&
           fused_geometry(B, H, W, c_in, nA, nB, n3, &g);
}

lrd_status_t tucker_fused(bool dgrad, const void* in, const void* P1, const void* G, const void* P3, const void* bias3, void* out3,
                          void* save1, void* save2, int64_t B, int64_t H, int64_t W, int64_t c_in, int64_t nA, int64_t nB,
                          int64_t n3, cudaStream_t s) {
    FusedGeo g;
    if (!fused_geometry(B, H, W, c_in, nA, nB, n3, &g)) return LRD_ERR_UNSUPPORTED;
    const int64_t r1 = dgrad ? nB : nA, r2 = dgrad ? nA : nB;     // G is [r2][9][r1]
    const int swb = nA % 64 == 0 ? 128 : (nA % 32 == 0 ? 64 : 32);
    CUtensorMap tIn, tP1, tG, tP3;
    bool ok = make_tmap_nhwc_bf16(&tIn, in, (uint64_t)B, (uint64_t)H, (uint64_t)W, (uint64_t)c_in, (uint32_t)(g.bh + 2), (uint32_t)W, 64);
    ok = ok && make_tmap_2d_bf16(&tP1, P1, (uint64_t)c_in, (uint64_t)nA, (uint64_t)nA, 64, (uint32_t)swb / 2);
    ok = ok && make_tmap_2d_bf16(&tG, G, (uint64_t)r2, (uint64_t)(9 * r1), (uint64_t)(9 * r1), dgrad ? 64 : 128, 64);
    ok = ok && make_tmap_2d_bf16(&tP3, P3, (uint64_t)n3, (uint64_t)nB, (uint64_t)nB, 256, 64);
    if (!ok) return LRD_ERR_CUDA;
    FusedParams p;
    p.H = (int)H; p.W = (int)W; p.PW = g.PW; p.bh = g.bh;
    p.c_in = (int)c_in; p.nA = (int)nA; p.nB = (int)nB; p.n3 = (int)n3;
    p.g_ci = (int)r1; p.swb = swb; p.z1_slots = g.z1_slots;
    p.save1 = (__nv_bfloat16*)save1; p.save2 = (__nv_bfloat16*)save2; p.out3 = (__nv_bfloat16*)out3;
    p.bias3 = (const __nv_bfloat16*)bias3;
    p.timeout_flag = device_timeout_flag();
    static bool configured_on[kMaxDevices] = {};
    bool& configured = configured_on[device_slot()];
    if (!configured) {
        const int lim = 226 * 1024;
        if (cudaFuncSetAttribute(tucker_fused_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim) != cudaSuccess ||
            cudaFuncSetAttribute(tucker_fused_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim) != cudaSuccess)
            return LRD_ERR_CUDA;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1, (unsigned)g.tiles_per_img, (unsigned)B);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = g.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = dgrad ? cudaLaunchKernelEx(&cfg, tucker_fused_kernel<true>, tIn, tP1, tG, tP3, p)
                                : cudaLaunchKernelEx(&cfg, tucker_fused_kernel<false>, tIn, tP1, tG, tP3, p);
    if (e != cudaSuccess) return LRD_ERR_CUDA;
    count_launch();
    return LRD_OK;
}

}  // namespace lrd
