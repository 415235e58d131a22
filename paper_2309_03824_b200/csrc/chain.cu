// Fused chain  Out[M x N2] = (In[M x K1] P[K1 x r]) Q[N2 x r]^T (+ bias)  on sm_100a.
//
// A cluster of C blocks owns one 128-row tile.
//   Phase 1  block c forms its r/C-column slice of T = In P in tensor memory (TMA-fed tcgen05.mma:
//            In K-major, the slice of P MN-major).
//   Gather   four warps read the slice (tcgen05.ld), round to bf16 and write it into the T buffer of
//            every block of the cluster (distributed shared memory), in the 128-byte-swizzled
//            K-major layout the next MMA reads.  T never goes to global memory unless T_save asks.
//   Phase 2  block c forms every C-th column chunk of Out = T Q^T (T from shared memory, Q by TMA),
//            double-buffered in tensor memory; the epilogue adds the bias, rounds to bf16 and
//            writes through shared memory with TMA stores (which clip the ragged edges).
// Warp 0: TMA producer.  Warp 1: tensor memory + MMA issue.  Warps 2-5: gather and epilogue.
// Warp 6: waits on the stage barriers for warp 1 and hands ready stages over by a named barrier.
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
constexpr uint32_t kInTileBytes = 128 * 64 * 2;     // In tile: 128 rows x 64 k
constexpr uint32_t kStagingBytes = 4 * 2 * 4096;    // per epilogue warp: two [32 rows x 128 B] slabs

struct ChainParams {
    int C, RS, swb, BN2, n_chunks, kb1, ks2, kb2, stages, N2, G1, G2;
    uint32_t stage_bytes, t_bytes, tmem_out0, tmem_out1;
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
    __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], tacc_bar, tready_bar, out_full[2],
        out_empty[2];
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

    if (threadIdx.x == 0) {
        abort_flag = 0;
        prefetch_tmap(&tmIn);
        prefetch_tmap(&tmP);
        prefetch_tmap(&tmQ);
        prefetch_tmap(&tmOut);
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), 1);
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
        // Lane 0 waits for the slot and arms its barrier; then lane l issues box l of the stage
        // (one instruction for the warp instead of a serial chain of issues by one thread).
        int s = 0;
        uint32_t ph = 1;                                     // parity to wait on for an empty slot
        bool ok = true;
        const int atom_cols = p.swb / 2;
        const uint32_t p_box_bytes = 64u * p.swb;
        const int n_pbox = p.RS / atom_cols;
        for (int kb = 0; kb < p.kb1 && ok; ++kb) {
            const uint32_t fb = smem_u32(&full_bar[s]);
            if (lane == 0) {
                ok = mbar_wait(smem_u32(&empty_bar[s]), ph, ab);
                if (ok) mbar_expect_tx(fb, kInTileBytes + 64u * p.RS * 2u);
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            const uint32_t dst = ring_base + s * p.stage_bytes;
            if (lane == 0) tma_load_2d(dst, &tmIn, fb, kb * 64, m0);
            else if (lane <= n_pbox)
                tma_load_2d(dst + kInTileBytes + (lane - 1) * p_box_bytes, &tmP, fb, c * p.RS + (lane - 1) * atom_cols, kb * 64);
            if (++s == p.stages) { s = 0; ph ^= 1; }
        }
        if (lane == 0) {
            for (int j = c; j < p.n_chunks && ok; j += p.C) {
                for (int kb = 0; kb < p.kb2; ++kb) {
                    if (!mbar_wait(smem_u32(&empty_bar[s]), ph, ab)) { ok = false; break; }
                    const uint32_t fb = smem_u32(&full_bar[s]);
                    mbar_expect_tx(fb, (uint32_t)p.BN2 * 128u);
                    tma_load_2d(ring_base + s * p.stage_bytes, &tmQ, fb, kb * 64, j * p.BN2);
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // Never waits on a barrier itself: warp 6 does the waiting and hands each group of ready
        // stages over through a named barrier.  Both warps run the same group loops.
        int s = 0;
        bool ok = true;
        const uint32_t idesc1 = idesc_bf16(p.RS, false, true);
        for (int kb0 = 0; kb0 < p.kb1; kb0 += p.G1) {
            const int g = min(p.G1, p.kb1 - kb0);
            ok = !pair_sync_or(false) && ok;
            if (lane == 0 && ok) {
                tc_fence_after();
                int ss = s;
                for (int i = 0; i < g; ++i) {
                    const uint32_t a_src = ring_base + ss * p.stage_bytes;
                    const uint32_t b_src = a_src + kInTileBytes;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint64_t ad = smem_desc_sw128(a_src + kk * 32, 0, 1024);
                        const uint64_t bd = smem_desc(b_src + kk * 16 * p.swb, 64u * p.swb, 8u * p.swb, p.swb);
                        mma_bf16_ss(tmem_base, ad, bd, idesc1, (kb0 + i > 0 || kk > 0) ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&empty_bar[ss]));
                    if (++ss == p.stages) ss = 0;
                }
            }
            s = (s + g) % p.stages;
        }
        if (lane == 0 && ok) mma_commit(smem_u32(&tacc_bar));
        const uint32_t idesc2 = idesc_bf16(p.BN2, false, false);
        int i2 = 0;
        for (int j = c; j < p.n_chunks; j += p.C, ++i2) {
            const int buf = i2 & 1;
            const uint32_t d_tmem = tmem_base + (buf ? p.tmem_out1 : p.tmem_out0);
            for (int kb0 = 0; kb0 < p.kb2; kb0 += p.G2) {
                const int g = min(p.G2, p.kb2 - kb0);
                // (before a chunk's first group warp 6 has also seen T complete and the accumulator buffer drained)
                ok = !pair_sync_or(false) && ok;
                if (lane == 0 && ok) {
                    tc_fence_after();
                    int ss = s;
                    for (int i = 0; i < g; ++i) {
                        const int kb = kb0 + i;
                        const uint32_t b_src = ring_base + ss * p.stage_bytes;
                        const int nks = min(4, p.ks2 - kb * 4);
                        for (int kk = 0; kk < nks; ++kk) {
                            const int ks = kb * 4 + kk;                       // 16-column step within T
                            const uint64_t ad = smem_desc(t_base + (uint32_t)(ks / t_steps) * t_atom_bytes + (uint32_t)(ks % t_steps) * 32u,
                                                          0, 8u * t_sw, t_sw);
                            const uint64_t bd = smem_desc_sw128(b_src + kk * 32, 0, 1024);
                            mma_bf16_ss(d_tmem, ad, bd, idesc2, (kb > 0 || kk > 0) ? 1u : 0u);
                        }
                        mma_commit(smem_u32(&empty_bar[ss]));
                        if (++ss == p.stages) ss = 0;
                    }
                    if (kb0 + g >= p.kb2) mma_commit(smem_u32(&out_full[buf]));
                }
                s = (s + g) % p.stages;
            }
        }
        __syncwarp();
    } else if (warp == 6) {
        // ------------------------------------------------------------------ waiter for the MMA issuer
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;                                      // lane 0's view; shared with warp 1 at every hand-over
        for (int kb0 = 0; kb0 < p.kb1; kb0 += p.G1) {
            const int g = min(p.G1, p.kb1 - kb0);
            if (lane == 0) {
                for (int i = 0; i < g; ++i) {
                    if (ok) ok = mbar_wait(smem_u32(&full_bar[s]), ph, ab);
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
            }
            __syncwarp();
            pair_sync_or(lane == 0 && !ok);
        }
        int i2 = 0;
        for (int j = c; j < p.n_chunks; j += p.C, ++i2) {
            const int buf = i2 & 1;
            for (int kb0 = 0; kb0 < p.kb2; kb0 += p.G2) {
                const int g = min(p.G2, p.kb2 - kb0);
                if (lane == 0) {
                    if (kb0 == 0) {
                        // every slice of T has landed in this block's buffer; the accumulator buffer is free again
                        if (ok && i2 == 0) ok = mbar_wait_cluster(smem_u32(&tready_bar), 0, ab);
                        if (ok) ok = mbar_wait(smem_u32(&out_empty[buf]), ((i2 >> 1) & 1) ^ 1, ab);
                    }
                    for (int i = 0; i < g; ++i) {
                        if (ok) ok = mbar_wait(smem_u32(&full_bar[s]), ph, ab);
                        if (++s == p.stages) { s = 0; ph ^= 1; }
                    }
                }
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
        // completes on the peer's barrier) and, if asked, stores it to T_save.
        fence_proxy_async_smem();
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
        const uint32_t slab_base = staging_base + q * 8192;
        int i = 0, sb = 0;
        for (int j = c; j < p.n_chunks && ok; j += p.C, ++i) {
            const int buf = i & 1;
            ok = mbar_wait_warp(smem_u32(&out_full[buf]), (i >> 1) & 1, ab);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = lane_addr + (buf ? p.tmem_out1 : p.tmem_out0);
            for (int g = 0; g * 64 < p.BN2; ++g) {
                const int col0 = j * p.BN2 + g * 64;
                const uint32_t slab = slab_base + (sb & 1) * 4096;
                if (sb >= 2) {                               // the store that last read this slab has finished reading
                    if (lane == 0) tma_store_wait_read<1>();
                    __syncwarp();
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t v[32];
                    const int colh = col0 + h * 32;
                    // the 32 bias values of this piece: four 16-byte loads (same address in every lane),
                    // issued before the accumulator load so that both latencies overlap
                    uint4 bv[4] = {};
                    const bool bias_vec = p.bias && colh + 32 <= p.N2;
                    if (bias_vec) {
                        const uint4* bp = reinterpret_cast<const uint4*>(p.bias + colh);
#pragma unroll
                        for (int e = 0; e < 4; ++e) bv[e] = __ldg(bp + e);
                    }
                    tmem_ld_32x32(d_tmem + g * 64 + h * 32, v);
                    tmem_ld_wait();
                    if (bias_vec) {
                        const uint32_t* bw = reinterpret_cast<const uint32_t*>(bv);
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            v[2 * e] = __float_as_uint(__uint_as_float(v[2 * e]) + __uint_as_float(bw[e] << 16));
                            v[2 * e + 1] = __float_as_uint(__uint_as_float(v[2 * e + 1]) + __uint_as_float(bw[e] & 0xFFFF0000u));
                        }
                    } else if (p.bias) {                     // ragged last piece
                        for (int e = 0; e < 32; ++e)
                            if (colh + e < p.N2) v[e] = __float_as_uint(__uint_as_float(v[e]) + __bfloat162float(p.bias[colh + e]));
                    }
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc)
                        st_shared_v4(slab + (uint32_t)lane * 128u + ((uint32_t)((h * 4 + cc) ^ (lane & 7)) << 4),
                                     pack_bf16(__uint_as_float(v[8 * cc]), __uint_as_float(v[8 * cc + 1])),
                                     pack_bf16(__uint_as_float(v[8 * cc + 2]), __uint_as_float(v[8 * cc + 3])),
                                     pack_bf16(__uint_as_float(v[8 * cc + 4]), __uint_as_float(v[8 * cc + 5])),
                                     pack_bf16(__uint_as_float(v[8 * cc + 6]), __uint_as_float(v[8 * cc + 7])));
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && col0 < p.N2) {
                    tma_store_2d(&tmOut, slab, col0, m0 + q * 32);
                    tma_store_commit();
                }
                ++sb;
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
    int C, RS, swb, BN2, stages;
    uint32_t stage_bytes, t_bytes, smem_bytes;
};

inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

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
    Plan best{};
    bool found = false;
    const int cands[3] = {4, 2, 1};
    for (int C : cands) {
        if (a.r % (16 * C)) continue;
        const int RS = (int)a.r / C;
        if (RS > 256) continue;
        const int swb = RS % 64 == 0 ? 128 : (RS % 32 == 0 ? 64 : 32);
        const int BN2 = RS <= 128 ? 192 : 128;
        uint32_t stage = kInTileBytes + 64u * RS * 2u;
        if ((uint32_t)BN2 * 128u > stage) stage = (uint32_t)BN2 * 128u;
        stage = (stage + 1023u) & ~1023u;
        const int64_t room = (int64_t)kSmemLimit - 1024 - t_bytes - (int64_t)kStagingBytes;
        int stages = (int)(room / stage);
        if (stages > kMaxStages) stages = kMaxStages;
        if (stages < 2) continue;
        Plan pl{C, RS, swb, BN2, stages, stage, (uint32_t)t_bytes,
                (uint32_t)(1024 + t_bytes + kStagingBytes + stages * stage)};
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
    ok = ok && make_tmap_2d_bf16(&tP, a.P, (uint64_t)a.K1, (uint64_t)a.r, (uint64_t)a.ldp, 64, (uint32_t)pl.swb / 2);
    ok = ok && make_tmap_2d_bf16(&tQ, a.Q, (uint64_t)a.N2, (uint64_t)a.r, (uint64_t)a.ldq, (uint32_t)pl.BN2, 64);
    ok = ok && make_tmap_2d_bf16(&tOut, a.Out, (uint64_t)a.M, (uint64_t)a.N2, (uint64_t)a.ld_out, 32, 64);
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
    p.stages = pl.stages; p.N2 = (int)a.N2;
    // k-blocks handed over per rendezvous: enough MMA work to cover the hand-over's own latency
    p.G1 = pl.RS >= 176 ? 1 : 2;
    p.G2 = pl.BN2 >= 176 ? 1 : 2;
    if (p.G1 > pl.stages / 2) p.G1 = pl.stages / 2 > 0 ? pl.stages / 2 : 1;
    if (p.G2 > pl.stages / 2) p.G2 = pl.stages / 2 > 0 ? pl.stages / 2 : 1;
    p.stage_bytes = pl.stage_bytes; p.t_bytes = pl.t_bytes;
    p.taw = pl.swb / 2;
    p.tmem_out0 = pl.RS <= 128 ? 128 : 256;
    p.tmem_out1 = p.tmem_out0 + (pl.RS <= 128 ? 192 : 128);
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
