// Fused chain  Out[M x N2] = (In[M x K1] P[K1 x r]) Q[N2 x r]^T (+ bias)  on sm_100a.
//
// A cluster of C blocks owns one 128-row tile.
//   Phase 1  block c forms its r/C-column slice of T = In P in tensor memory (TMA-fed tcgen05.mma:
//            In K-major, the slice of P MN-major).
//   Gather   four warps read the slice (tcgen05.ld), round it to bf16 and write it into this block's T
//            buffer (K-major, swizzled, slices are whole atoms = one contiguous range); one thread then
//            copies the range into every peer's T buffer with bulk DSMEM copies that complete on the
//            peer's barrier.  T never goes to global memory unless T_save asks.
//   Phase 2  block c forms every C-th column chunk of Out = T Q^T (T from shared memory, Q by TMA),
//            double-buffered in tensor memory; the epilogue adds the bias, rounds to bf16 and writes
//            through shared memory with TMA stores (which clip the ragged edges).
// A pipeline stage holds a GROUP of 64-deep k-blocks behind one barrier pair: the cost of a stage
// turn-around (barrier round trip, hand-over to the MMA thread, TMA issue) is per stage, not per byte,
// so stages are made as large as shared memory allows.  The two phases lay their stages out
// differently over the same ring.
// Warp 0: TMA producer.  Warp 1: tensor memory + MMA issue.  Warps 2-5: gather and epilogue.
// Warp 6: waits on the stage barriers for warp 1 and hands ready stages over by a named barrier (the
// issuing thread must not read shared memory behind a tcgen05.commit: that read waits for the MMAs).
#include "chain.cuh"

#include "ptx.cuh"
#include "tc.cuh"
#include "tma.cuh"

namespace lrd {
namespace {

using namespace ptx;

constexpr int kThreads = 224;
constexpr int kMaxStages = 8;
constexpr uint32_t kSmemLimit = 226 * 1024;         // dynamic shared memory; the rest is left for the barriers
constexpr uint32_t kInTileBytes = 128 * 64 * 2;     // In tile of one k-block: 128 rows x 64 k
constexpr uint32_t kSlabBytes = 32 * 64;            // epilogue slab: 32 rows x 32 columns of bf16
constexpr uint32_t kStagingBytes = 4 * 2 * kSlabBytes;

struct ChainParams {
    int C, RS, swb, BN2, n_chunks, kb1, ks2, kb2, N2;
    int G1, S1, G2, S2;       // k-blocks per stage and stage count of phase 1 / phase 2
    uint32_t stage1_bytes, stage2_bytes, t_bytes;
    int taw;                  // columns per atom of the T buffer (64, 32 or 16; swizzle span = 2 * taw bytes)
    const __nv_bfloat16* bias;
    int has_tsave;
    unsigned int* timeout_flag;
};

__global__ void __launch_bounds__(kThreads, 1)
chain_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmP,
             const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmOut,
             const __grid_constant__ CUtensorMap tmT, const ChainParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full1[kMaxStages], empty1[kMaxStages], full2[kMaxStages], empty2[kMaxStages],
        tacc_bar, tready_bar, out_full[2], out_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t t_base = smem_base;
    const uint32_t staging_base = t_base + p.t_bytes;
    const uint32_t ring_base = staging_base + kStagingBytes;
    const AbortCtx ab{&abort_flag, p.timeout_flag};
    const uint32_t t_sw = 2u * (uint32_t)p.taw, t_atom_bytes = 128u * t_sw;   // T: atoms of [128 rows x taw columns]
    const int t_steps = p.taw / 16;                                           // MMA k-steps per atom
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int c = (int)cluster_ctarank();
    const int m0 = blockIdx.y * 128;
    const int ng1 = (p.kb1 + p.G1 - 1) / p.G1, ng2 = (p.kb2 + p.G2 - 1) / p.G2;   // stage turns per phase / chunk
    // phase-1 stage: G1 In tiles, then the P boxes (one per column atom, 64 G1 rows tall)
    const uint32_t p_box_bytes = 64u * (uint32_t)p.G1 * (uint32_t)p.swb;
    const uint32_t q_tile_bytes = (uint32_t)p.BN2 * 128u;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        prefetch_tmap(&tmIn);
        prefetch_tmap(&tmP);
        prefetch_tmap(&tmQ);
        prefetch_tmap(&tmOut);
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&full1[s]), 1);
            mbar_init(smem_u32(&empty1[s]), 1);
            mbar_init(smem_u32(&full2[s]), 1);
            mbar_init(smem_u32(&empty2[s]), 1);
        }
        mbar_init(smem_u32(&tacc_bar), 1);
        // T complete = this block's own slice written (one arrival) + the peers' slices landed (bytes)
        mbar_init(smem_u32(&tready_bar), 2);
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&out_full[i]), 1);
            mbar_init(smem_u32(&out_empty[i]), 4);
        }
        mbar_expect_tx(smem_u32(&tready_bar), (uint32_t)(p.C - 1) * 256u * (uint32_t)p.RS);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_arrive();          // every block's barriers exist before any peer touches them
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // Lane 0 waits for the stage and arms its barrier; then lane l issues copy l of the stage.
        int s = 0;
        uint32_t ph = 1;                                     // parity to wait on for an empty stage
        bool ok = true;
        const int atom_cols = p.swb / 2;
        const int n_pbox = p.RS / atom_cols;
        for (int g = 0; g < ng1 && ok; ++g) {
            const uint32_t fb = smem_u32(&full1[s]);
            if (lane == 0) {
                ok = mbar_wait(smem_u32(&empty1[s]), ph, ab);
                if (ok) mbar_expect_tx(fb, p.stage1_bytes);
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            const uint32_t dst = ring_base + s * p.stage1_bytes;
            const int kb0 = g * p.G1;
            if (lane < p.G1)                                 // k-blocks past K1 read as zeros
                tma_load_2d(dst + lane * kInTileBytes, &tmIn, fb, (kb0 + lane) * 64, m0);
            else if (lane < p.G1 + n_pbox)
                tma_load_2d(dst + p.G1 * kInTileBytes + (lane - p.G1) * p_box_bytes, &tmP, fb,
                            c * p.RS + (lane - p.G1) * atom_cols, kb0 * 64);
            if (++s == p.S1) { s = 0; ph ^= 1; }
        }
        // the ring is laid out anew for phase 2: wait until every phase-1 MMA has read its operands
        if (lane == 0 && ok) ok = mbar_wait(smem_u32(&tacc_bar), 0, ab);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        s = 0;
        ph = 1;
        for (int j = c; j < p.n_chunks && ok; j += p.C) {
            for (int g = 0; g < ng2; ++g) {
                const uint32_t fb = smem_u32(&full2[s]);
                if (lane == 0) {
                    ok = mbar_wait(smem_u32(&empty2[s]), ph, ab);
                    if (ok) mbar_expect_tx(fb, p.stage2_bytes);
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                if (lane < p.G2)                             // k-blocks past r read as zeros
                    tma_load_2d(ring_base + s * p.stage2_bytes + lane * q_tile_bytes, &tmQ, fb, (g * p.G2 + lane) * 64,
                                j * p.BN2);
                if (++s == p.S2) { s = 0; ph ^= 1; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // Never waits on a barrier itself: warp 6 does the waiting and hands each ready stage over
        // through a named barrier.  Both warps run the same loops.
        int s = 0;
        bool ok = true;
        const uint32_t idesc1 = idesc_bf16(p.RS, false, true);
        const uint64_t a_desc0 = smem_desc_sw128(0, 0, 1024);
        const uint64_t b_desc0 = smem_desc(0, p_box_bytes, 8u * p.swb, p.swb);
        for (int g = 0; g < ng1; ++g) {
            ok = !pair_sync_or(false) && ok;
            if (lane == 0 && ok) {
                tc_fence_after();
                const uint32_t in_src = ring_base + s * p.stage1_bytes;
                const uint32_t p_src = in_src + p.G1 * kInTileBytes;
                const int nkb = min(p.G1, p.kb1 - g * p.G1);
                // descriptors differ only in the start-address field (bits 0-13, in 16-byte units): build one
                // per operand and add offsets
                uint64_t ad = a_desc0 + ((in_src >> 4) & 0x3FFFu);
                uint64_t bd = b_desc0 + ((p_src >> 4) & 0x3FFFu);
                for (int i = 0; i < nkb; ++i) {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_bf16_ss(tmem_base, ad + 2u * kk, bd + (uint64_t)(kk * p.swb), idesc1, (g > 0 || i > 0 || kk > 0) ? 1u : 0u);
                    ad += kInTileBytes >> 4;
                    bd += (uint64_t)(4 * p.swb);              // 64 rows of swb bytes
                }
                mma_commit(smem_u32(&empty1[s]));
            }
            if (++s == p.S1) s = 0;
        }
        if (lane == 0 && ok) mma_commit(smem_u32(&tacc_bar));
        const uint32_t idesc2 = idesc_bf16(p.BN2, false, false);
        const uint64_t t_desc0 = smem_desc(t_base, 0, 8u * t_sw, t_sw);
        s = 0;
        int i2 = 0;
        for (int j = c; j < p.n_chunks; j += p.C, ++i2) {
            const uint32_t d_tmem = tmem_base + (uint32_t)(i2 & 1) * 256u;
            for (int g = 0; g < ng2; ++g) {
                // (before a chunk's first stage warp 6 has also seen T complete and the accumulator buffer drained)
                ok = !pair_sync_or(false) && ok;
                if (lane == 0 && ok) {
                    tc_fence_after();
                    const uint32_t q_src = ring_base + s * p.stage2_bytes;
                    const int nkb = min(p.G2, p.kb2 - g * p.G2);
                    uint64_t bd = a_desc0 + ((q_src >> 4) & 0x3FFFu);
                    for (int i = 0; i < nkb; ++i) {
                        const int kb = g * p.G2 + i;
                        const int nks = min(4, p.ks2 - kb * 4);
                        for (int kk = 0; kk < nks; ++kk) {
                            const int ks = kb * 4 + kk;                       // 16-column step within T
                            const uint64_t ad = t_desc0 + (((uint32_t)(ks / t_steps) * t_atom_bytes + (uint32_t)(ks % t_steps) * 32u) >> 4);
                            mma_bf16_ss(d_tmem, ad, bd + 2u * kk, idesc2, (kb > 0 || kk > 0) ? 1u : 0u);
                        }
                        bd += q_tile_bytes >> 4;
                    }
                    mma_commit(smem_u32(&empty2[s]));
                    if (g == ng2 - 1) mma_commit(smem_u32(&out_full[i2 & 1]));
                }
                if (++s == p.S2) s = 0;
            }
        }
        __syncwarp();
    } else if (warp == 6) {
        // ------------------------------------------------------------------ waiter for the MMA issuer
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;                                      // lane 0's view; shared with warp 1 at every hand-over
        for (int g = 0; g < ng1; ++g) {
            if (lane == 0 && ok) ok = mbar_wait(smem_u32(&full1[s]), ph, ab);
            if (++s == p.S1) { s = 0; ph ^= 1; }
            __syncwarp();
            pair_sync_or(lane == 0 && !ok);
        }
        s = 0;
        ph = 0;
        int i2 = 0;
        for (int j = c; j < p.n_chunks; j += p.C, ++i2) {
            for (int g = 0; g < ng2; ++g) {
                if (lane == 0) {
                    if (g == 0) {
                        // every slice of T has landed in this block's buffer; the accumulator buffer is free again
                        if (ok && i2 == 0) ok = mbar_wait_cluster(smem_u32(&tready_bar), 0, ab);
                        if (ok) ok = mbar_wait(smem_u32(&out_empty[i2 & 1]), ((i2 >> 1) & 1) ^ 1, ab);
                    }
                    if (ok) ok = mbar_wait(smem_u32(&full2[s]), ph, ab);
                }
                if (++s == p.S2) { s = 0; ph ^= 1; }
                __syncwarp();
                pair_sync_or(lane == 0 && !ok);
            }
        }
    } else {
        // ------------------------------------------------------------------ gather + epilogue
        const int q = warp % 4;                              // tensor-memory lanes [32 q, 32 q + 32)
        const int row = q * 32 + lane;                       // row of the 128-row tile
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        bool ok = mbar_wait_warp(smem_u32(&tacc_bar), 0, ab);   // warp-uniform from here on
        tc_fence_after();
        if (ok) {
            for (int piece = 0; piece * 16 < p.RS; ++piece) {
                uint32_t v[16];
                tmem_ld_32x16(lane_addr + piece * 16, v);
                tmem_ld_wait();
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) w[e] = pack_bf16(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
                const int gc = c * p.RS + piece * 16;        // first column of this piece within T
                const uint32_t row_addr = t_base + (uint32_t)(gc / p.taw) * t_atom_bytes + (uint32_t)row * t_sw;
                const uint32_t chunk0 = (uint32_t)(gc % p.taw) / 8u;
                const uint32_t sw_xor = (((uint32_t)row * t_sw) >> 7) & (t_sw / 16u - 1u);
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    st_shared_v4(row_addr + (((chunk0 + h) ^ sw_xor) << 4), w[4 * h], w[4 * h + 1], w[4 * h + 2], w[4 * h + 3]);
            }
        }
        // The slice [c RS, (c+1) RS) is whole atoms, i.e. one contiguous range of this block's T buffer: after
        // the four warps have written it, one thread copies it into every peer's buffer (bulk DSMEM copy that
        // completes on the peer's barrier) and, if asked, stores it to T_save.  The accumulator columns of
        // the slice are free for phase 2 from here on.
        fence_proxy_async_smem();
        tc_fence_before();
        named_bar_sync(2, 128);
        if (q == 0 && lane == 0 && ok) {
            const uint32_t slice = t_base + (uint32_t)c * 256u * (uint32_t)p.RS;
            for (int t = 1; t < p.C; ++t) {
                const uint32_t peer = (uint32_t)((c + t) % p.C);
                dsmem_bulk_copy(slice, slice, 256u * (uint32_t)p.RS, smem_u32(&tready_bar), peer);
            }
            mbar_arrive(smem_u32(&tready_bar));
            if (p.has_tsave) {
                for (int a = 0; a * p.taw < p.RS; ++a)
                    tma_store_2d(&tmT, slice + (uint32_t)a * t_atom_bytes, c * p.RS + a * p.taw, m0);
                tma_store_commit();
            }
        }
        __syncwarp();
        // Epilogue: 32 columns at a time through a [32 rows x 64 B] slab of this warp (64-byte swizzle),
        // two slabs in rotation; each slab leaves by its own TMA store.
        const uint32_t slab_base = staging_base + q * 2 * kSlabBytes;
        const uint32_t slab_row = (uint32_t)lane * 64u;
        const uint32_t slab_xor = ((uint32_t)lane >> 1) & 3u;
        int i = 0, sb = 0;
        for (int j = c; j < p.n_chunks && ok; j += p.C, ++i) {
            const int buf = i & 1;
            ok = mbar_wait_warp(smem_u32(&out_full[buf]), (i >> 1) & 1, ab);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = lane_addr + (uint32_t)buf * 256u;
            for (int g = 0; g * 32 < p.BN2; ++g, ++sb) {
                const int colh = j * p.BN2 + g * 32;
                if (colh >= p.N2) continue;                  // (uniform) nothing of this piece is inside Out
                const uint32_t slab = slab_base + (sb & 1) * kSlabBytes;
                // the 32 bias values of this piece: four 16-byte loads (same address in every lane), issued
                // before the accumulator load so that both latencies overlap
                uint4 bv[4] = {};
                const bool bias_vec = p.bias && colh + 32 <= p.N2;
                if (bias_vec) {
                    const uint4* bp = reinterpret_cast<const uint4*>(p.bias + colh);
#pragma unroll
                    for (int e = 0; e < 4; ++e) bv[e] = __ldg(bp + e);
                }
                uint32_t v[32];
                tmem_ld_32x32(d_tmem + g * 32, v);
                if (sb >= 2) {                               // the store that last read this slab has finished reading
                    if (lane == 0) tma_store_wait_read<1>();
                    __syncwarp();
                }
                tmem_ld_wait();
                if (bias_vec) {
                    const uint32_t* bw = reinterpret_cast<const uint32_t*>(bv);
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        v[2 * e] = __float_as_uint(__uint_as_float(v[2 * e]) + __uint_as_float(bw[e] << 16));
                        v[2 * e + 1] = __float_as_uint(__uint_as_float(v[2 * e + 1]) + __uint_as_float(bw[e] & 0xFFFF0000u));
                    }
                } else if (p.bias) {                         // ragged last piece
                    for (int e = 0; e < 32; ++e)
                        if (colh + e < p.N2) v[e] = __float_as_uint(__uint_as_float(v[e]) + __bfloat162float(p.bias[colh + e]));
                }
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
                    st_shared_v4(slab + slab_row + (((uint32_t)cc ^ slab_xor) << 4),
                                 pack_bf16(__uint_as_float(v[8 * cc]), __uint_as_float(v[8 * cc + 1])),
                                 pack_bf16(__uint_as_float(v[8 * cc + 2]), __uint_as_float(v[8 * cc + 3])),
                                 pack_bf16(__uint_as_float(v[8 * cc + 4]), __uint_as_float(v[8 * cc + 5])),
                                 pack_bf16(__uint_as_float(v[8 * cc + 6]), __uint_as_float(v[8 * cc + 7])));
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&tmOut, slab, colh, m0 + q * 32);
                    tma_store_commit();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&out_empty[buf]));
        }
        if (lane == 0) tma_store_wait_all<0>();
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    cluster_arrive();          // no block leaves while a peer may still write into its shared memory
    cluster_wait();
    if (warp == 1) {
        if (abort_flag) {
            for (int i = 0; i < 256; ++i) __nanosleep(1000);
        }
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

struct Plan {
    int C, RS, swb, BN2, G1, S1, G2, S2;
    uint32_t stage1_bytes, stage2_bytes, t_bytes, smem_bytes;
};

inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

// Column chunk width of phase 2: the block with the most chunks sets the pace, so minimise
// (chunks of the busiest block) x width; wider chunks on ties (fewer, larger copies).
int pick_bn2(int64_t N2, int C) {
    const int cands[3] = {256, 192, 128};
    int best = 128;
    int64_t best_cost = -1;
    for (int bn : cands) {
        const int64_t chunks = (N2 + bn - 1) / bn;
        const int64_t cost = ((chunks + C - 1) / C) * bn;
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = bn; }
    }
    return best;
}

bool make_plan(const ChainArgs& a, Plan* out) {
    if (a.dtype != LRD_BF16 || a.M < 1 || a.K1 < 1 || a.N2 < 1) return false;
    if (a.r < 16 || a.r > 512 || a.r % 16) return false;
    if (a.M > (int64_t)65535 * 128 || a.K1 > (1 << 30) || a.N2 > (1 << 30)) return false;
    if (!aligned16(a.In) || !aligned16(a.P) || !aligned16(a.Q) || !aligned16(a.Out)) return false;
    if (a.ld_in % 8 || a.ldp % 8 || a.ldq % 8 || a.ld_out % 8) return false;
    if (a.T_save && (!aligned16(a.T_save) || a.ldt % 8)) return false;
    if (a.bias && !aligned16(a.bias)) return false;
    const int64_t tiles = (a.M + 127) / 128;
    const int t_bytes = (int)((a.r * 256 + 1023) / 1024 * 1024);      // 128 rows x r columns of bf16
    const int kb1 = (int)((a.K1 + 63) / 64), kb2 = (int)((a.r + 63) / 64);
    Plan best{};
    bool found = false;
    const int cands[3] = {4, 2, 1};
    for (int C : cands) {
        if (a.r % (16 * C)) continue;
        const int RS = (int)a.r / C;
        if (RS > 256) continue;
        const int swb = RS % 64 == 0 ? 128 : (RS % 32 == 0 ? 64 : 32);
        const int BN2 = pick_bn2(a.N2, C);
        const int64_t ring = (int64_t)kSmemLimit - 1024 - t_bytes - (int64_t)kStagingBytes;
        const uint32_t kb1_bytes = kInTileBytes + 128u * RS, kb2_bytes = (uint32_t)BN2 * 128u;
        // the most k-blocks per stage that still leave two stages (phase 1: a P box is at most 256 rows)
        int G1 = 0, G2 = 0;
        for (int g = 4; g >= 1; --g)
            if (ring / ((int64_t)g * kb1_bytes) >= 2) { G1 = g; break; }
        for (int g = 4; g >= 1; --g)
            if (ring / ((int64_t)g * kb2_bytes) >= 2) { G2 = g; break; }
        if (!G1 || !G2) continue;
        if (G1 > kb1) G1 = kb1;
        if (G2 > kb2) G2 = kb2;
        int S1 = (int)(ring / ((int64_t)G1 * kb1_bytes)), S2 = (int)(ring / ((int64_t)G2 * kb2_bytes));
        if (S1 > kMaxStages) S1 = kMaxStages;
        if (S2 > kMaxStages) S2 = kMaxStages;
        const uint32_t s1b = (uint32_t)G1 * kb1_bytes, s2b = (uint32_t)G2 * kb2_bytes;
        const uint32_t used = (uint32_t)S1 * s1b > (uint32_t)S2 * s2b ? (uint32_t)S1 * s1b : (uint32_t)S2 * s2b;
        Plan pl{C, RS, swb, BN2, G1, S1, G2, S2, s1b, s2b, (uint32_t)t_bytes, (uint32_t)(1024 + t_bytes + kStagingBytes + used)};
        // prefer the largest cluster whose blocks are all resident at once; else the smallest feasible
        if (!found) { best = pl; found = true; }
        if (tiles * C <= kNumSms) { best = pl; break; }
        best = pl;
    }
    if (!found) return false;
    *out = best;
    return true;
}

}  // namespace

bool chain_eligible(const ChainArgs& a) {
    Plan pl;
    return make_plan(a, &pl);
}

lrd_status_t chain_launch(const ChainArgs& a, cudaStream_t stream) {
    Plan pl;
    if (!make_plan(a, &pl)) return LRD_ERR_UNSUPPORTED;
    CUtensorMap tIn, tP, tQ, tOut, tT;
    bool ok = make_tmap_2d_bf16(&tIn, a.In, (uint64_t)a.M, (uint64_t)a.K1, (uint64_t)a.ld_in, 128, 64);
    ok = ok && make_tmap_2d_bf16(&tP, a.P, (uint64_t)a.K1, (uint64_t)a.r, (uint64_t)a.ldp, 64u * (uint32_t)pl.G1, (uint32_t)pl.swb / 2);
    ok = ok && make_tmap_2d_bf16(&tQ, a.Q, (uint64_t)a.N2, (uint64_t)a.r, (uint64_t)a.ldq, (uint32_t)pl.BN2, 64);
    ok = ok && make_tmap_2d_bf16(&tOut, a.Out, (uint64_t)a.M, (uint64_t)a.N2, (uint64_t)a.ld_out, 32, 32);
    if (a.T_save)
        ok = ok && make_tmap_2d_bf16(&tT, a.T_save, (uint64_t)a.M, (uint64_t)a.r, (uint64_t)a.ldt, 128, (uint32_t)pl.swb / 2);
    else
        tT = tOut;
    if (!ok) return LRD_ERR_CUDA;

    ChainParams p;
    p.C = pl.C; p.RS = pl.RS; p.swb = pl.swb; p.BN2 = pl.BN2;
    p.n_chunks = (int)((a.N2 + pl.BN2 - 1) / pl.BN2);
    p.kb1 = (int)((a.K1 + 63) / 64);
    p.ks2 = (int)a.r / 16;
    p.kb2 = (int)((a.r + 63) / 64);
    p.N2 = (int)a.N2;
    p.G1 = pl.G1; p.S1 = pl.S1; p.G2 = pl.G2; p.S2 = pl.S2;
    p.stage1_bytes = pl.stage1_bytes; p.stage2_bytes = pl.stage2_bytes; p.t_bytes = pl.t_bytes;
    p.taw = pl.swb / 2;
    p.bias = (const __nv_bfloat16*)a.bias;
    p.has_tsave = a.T_save ? 1 : 0;
    p.timeout_flag = device_timeout_flag();

    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess)
            return LRD_ERR_CUDA;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)pl.C, (unsigned)((a.M + 127) / 128), 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)pl.C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, chain_kernel, tIn, tP, tQ, tOut, tT, p) != cudaSuccess) return LRD_ERR_CUDA;
    count_launch();
    return LRD_OK;
}

}  // namespace lrd
