// Fused chain  Out[M x N2] = (In[M x K1] P[K1 x r]) Q[N2 x r]^T (+ bias)  on pairs of SMs (sm_100a).
//
// A cluster of 2 S blocks owns TWO 128-row tiles (256 rows).  Blocks 2 p and 2 p + 1 form MMA pair p
// (tcgen05 cta_group::2): block 2 p + h holds rows [128 h, 128 h + 128) of the cluster's rows, one thread
// of the even block (the leader) issues 256-row MMAs for both, and each block loads its own rows of In
// but only HALF of every B operand (its half of the pair's slice of P, its half of every chunk of Q).
// Per row of Out the weights then cross L2 -> shared memory half as often as with single blocks, and an
// MMA reads 8 KB instead of 12 KB of operands from each block's shared memory.
//   Phase 1  pair p forms the RS = r / S columns [p RS, (p + 1) RS) of T = In P in tensor memory.
//   Gather   each block rounds its 128 rows of the slice to bf16 into its own T buffer (K-major, swizzled,
//            a slice is whole atoms = one contiguous range) and copies the range into the T buffers of the
//            blocks that hold the same rows in the other pairs (bulk DSMEM copies completing on the
//            receiver's barrier).  T goes to global memory only when T_save asks.
//   Phase 2  pair p forms every S-th column chunk of Out = T Q^T (T from each block's shared memory, Q by
//            TMA), accumulators double-buffered in tensor memory; the epilogue warps of each block add the
//            bias, round to bf16 and store their 32 rows through per-warp slabs and TMA stores.
// Shared memory.  What bounds both products is the number of bytes in flight: a stage slot is held for about a
// microsecond (the load's latency from HBM or L2 under load, then its MMAs), so a block streams at most
// (bytes of slots) / 1 us.  Phase 1 therefore uses ALL of the block's shared memory as its ring, the region of
// the T buffer and of the epilogue slabs included (T is written only after the last MMA of phase 1); phase 2
// has the ring behind T and the slabs, in slots of exactly one Q tile.  Its first tiles are requested as soon as
// phase 1's MMAs are done and land while T is gathered.  Because a peer's slice lands in the region this block's
// phase-1 ring used, slices are pushed only after every block of the cluster has finished phase 1 (cluster
// barrier 1).
// gridDim.z selects one of up to kMaxLayers independent layers of equal shape (a group launch).
// Warp 0: TMA producer.  Warp 1: tensor memory; in the leader, MMA issue; in the odd block, forwarding
// "slice landed" to the leader.  Warps 2-5: gather and epilogue.  Every wait is bounded; a wait that runs
// out raises the device timeout flag and the cluster tears down in order.
#include <algorithm>

#include "chain.cuh"
#include "ptx_pair.cuh"
#include "tc.cuh"
#include "tma.cuh"

namespace lrd {
namespace {

using namespace ptx;

constexpr int kThreads = 192;
constexpr int kMaxSlots = 10;
constexpr int kMaxS = 4;             // pairs per cluster
constexpr uint32_t kSmemLimit = 224 * 1024;         // dynamic shared memory; the rest is left for the barriers and the bias
constexpr uint32_t kInTileBytes = 128 * 64 * 2;     // In tile of one k-block: 128 rows x 64 k
constexpr uint32_t kSlabBytes = 32 * 32 * 2;        // epilogue slab of one warp: 32 rows x 32 columns of bf16
constexpr uint32_t kStagingBytes = 4 * 2 * kSlabBytes;

struct LayerMaps {
    CUtensorMap in, p, q, out, t;
};
struct PairGroup {
    LayerMaps layer[kChainMaxLayers];
};

struct PairParams {
    int S, RS, swb, BN2, n_chunks, kb1, ks2, kb2, N2, M;
    int G1, NS1, NS2;         // k-blocks per phase-1 stage; slots of the two rings
    uint32_t stage1_bytes, stage2_bytes, t_bytes;
    int taw;                  // columns per atom of the T buffer (64, 32 or 16; swizzle span = 2 * taw bytes)
    int t_steps_lg;           // log2 of the MMA k-steps (16 columns) per atom
    const __nv_bfloat16* bias[kChainMaxLayers];
    int has_tsave[kChainMaxLayers];
    unsigned int* timeout_flag;
    // Phase 2 of pair p walks over the 64-column k-blocks of T in the order kb_order[p] (4 bits per position)
    // and needs the slices in kb_slices[p] (a 4-bit mask per position) for the k-block at that position.
    uint32_t kb_order[kMaxS], kb_slices[kMaxS];
};

__global__ void __launch_bounds__(kThreads, 1)
chain_pair_kernel(const __grid_constant__ PairGroup grp, const PairParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full1[kMaxSlots], empty1[kMaxSlots], full2[kMaxSlots], empty2[kMaxSlots], tacc_bar,
        tready_bar[kMaxS], pready_bar[kMaxS], out_full[2], out_empty[2];
    __shared__ __align__(16) float bias_s[2][256];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    // phase 1: [ring of NS1 slots];  afterwards: [T | epilogue slabs | ring of NS2 slots]
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t t_base = smem_base;
    const uint32_t ring1_base = smem_base;
    const uint32_t staging_base = t_base + p.t_bytes;
    const uint32_t ring2_base = staging_base + kStagingBytes;
    const AbortCtx ab{&abort_flag, p.timeout_flag};
    const uint32_t t_sw = 2u * (uint32_t)p.taw, t_atom_bytes = 128u * t_sw;   // T: atoms of [128 rows x taw columns]
    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0);
    const int lane = threadIdx.x % 32;
    const uint32_t crank = cluster_ctarank();
    const int pr = (int)(crank >> 1);                    // pair: which slice of r, which chunks of Out
    const int h = (int)(crank & 1u);                     // which row tile of the cluster; h = 0 leads the pair
    const uint32_t lead_rank = crank & ~1u;
    const uint16_t pair_mask = (uint16_t)(3u << lead_rank);
    const bool leader = h == 0;
    const LayerMaps& L = grp.layer[blockIdx.z];
    const __nv_bfloat16* bias = p.bias[blockIdx.z];
    const int has_tsave = p.has_tsave[blockIdx.z];
    const uint32_t my_order = pr == 0 ? p.kb_order[0] : (pr == 1 ? p.kb_order[1] : (pr == 2 ? p.kb_order[2] : p.kb_order[3]));
    const uint32_t my_slices = pr == 0 ? p.kb_slices[0] : (pr == 1 ? p.kb_slices[1] : (pr == 2 ? p.kb_slices[2] : p.kb_slices[3]));
    const int m0 = ((int)blockIdx.y * 2 + h) * 128;
    const int ng1 = (p.kb1 + p.G1 - 1) / p.G1;                                 // stage turns of phase 1
    const int RSL = p.RS / 2;                                                  // columns of the P slice this block loads
    const int QL = p.BN2 / 2;                                                  // rows of a Q chunk this block loads
    // phase-1 stage: G1 In tiles, then the P boxes (one per column atom, 64 G1 rows tall)
    const uint32_t p_box_bytes = 64u * (uint32_t)p.G1 * (uint32_t)p.swb;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        prefetch_tmap(&L.in);
        prefetch_tmap(&L.p);
        prefetch_tmap(&L.q);
        prefetch_tmap(&L.out);
        for (int s = 0; s < kMaxSlots; ++s) {
            mbar_init(smem_u32(&full1[s]), 1);
            mbar_init(smem_u32(&empty1[s]), 1);
            mbar_init(smem_u32(&full2[s]), 1);
            mbar_init(smem_u32(&empty2[s]), 1);
        }
        mbar_init(smem_u32(&tacc_bar), 1);
        // one barrier per slice of T: this block's own slice is ready after one arrival (written by its gather
        // warps), a peer's slice once its bytes have landed; pready: the same for the odd block's buffer, told to the leader
        for (int j = 0; j < p.S; ++j) {
            mbar_init(smem_u32(&tready_bar[j]), 1);
            mbar_init(smem_u32(&pready_bar[j]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&out_full[i]), 1);
            mbar_init(smem_u32(&out_empty[i]), 8);          // the epilogue warps of both blocks of the pair
        }
        for (int j = 0; j < p.S; ++j)
            if (j != pr) mbar_expect_tx(smem_u32(&tready_bar[j]), 256u * (uint32_t)p.RS);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(&tmem_base_slot), 512);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    // every block's barriers exist before a partner or a peer signals them
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // Everything above touched only shared and tensor memory, so it may overlap the tail of the previous kernel
    // in the stream; global memory is first read (and written) below this line.
    griddep_launch_dependents();
    griddep_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        int s = 0;
        uint32_t ph = 1;                                     // parity to wait on for an empty slot
        bool ok = true;
        const int atom_cols = p.swb / 2;
        const int n_pbox = RSL / atom_cols;
        const int p_col0 = pr * p.RS + h * RSL;              // first column of P this block loads
        cluster_arrive_relaxed();                            // barrier 1 (this warp has nothing to tell)
        for (int g = 0; g < ng1 && ok; ++g) {
            ok = mbar_wait_uniform(smem_u32(&empty1[s]), ph, ab);
            if (!ok) break;
            // the copies of both blocks of a pair complete on the leader's barrier
            const uint32_t fb = map_to_cta(smem_u32(&full1[s]), lead_rank);
            const uint32_t dst = ring1_base + s * p.stage1_bytes;
            const int kb0 = g * p.G1;
            if (elect_one()) {
                if (leader) mbar_expect_tx(smem_u32(&full1[s]), 2u * p.stage1_bytes);
                for (int i = 0; i < p.G1; ++i)               // k-blocks past K1 read as zeros
                    tma_load_2d_pair(dst + i * kInTileBytes, &L.in, fb, (kb0 + i) * 64, m0);
                for (int i = 0; i < n_pbox; ++i)
                    tma_load_2d_pair(dst + p.G1 * kInTileBytes + i * p_box_bytes, &L.p, fb, p_col0 + i * atom_cols, kb0 * 64);
            }
            __syncwarp();
            if (++s == p.NS1) { s = 0; ph ^= 1; }
        }
        // the ring is laid out anew for phase 2: wait until every phase-1 MMA has read its operands
        if (ok) ok = mbar_wait_uniform(smem_u32(&tacc_bar), 0, ab);
        s = 0;
        ph = 1;
        for (int j = pr; j < p.n_chunks && ok; j += p.S) {
            for (int i = 0; i < p.kb2; ++i) {                // columns past r read as zeros (never multiplied)
                const int kb = (int)((my_order >> (4 * i)) & 15u);
                ok = mbar_wait_uniform(smem_u32(&empty2[s]), ph, ab);
                if (!ok) break;
                const uint32_t fb = map_to_cta(smem_u32(&full2[s]), lead_rank);
                if (elect_one()) {
                    if (leader) mbar_expect_tx(smem_u32(&full2[s]), 2u * p.stage2_bytes);
                    tma_load_2d_pair(ring2_base + s * p.stage2_bytes, &L.q, fb, kb * 64, j * p.BN2 + h * QL);
                }
                __syncwarp();
                if (++s == p.NS2) { s = 0; ph ^= 1; }
            }
        }
        cluster_wait();                                      // barrier 1
    } else if (warp == 1 && !leader) {
        // ------------------------------------------------------------------ odd block: tell the leader which slices have landed here
        // (its MMAs read this block's T buffer, and the first of them overwrite this block's phase-1 accumulator,
        // which has been read out once this block's own slice is ready)
        bool ok = true;
        cluster_arrive_relaxed();                            // barrier 1
        for (int t = 0; t < p.S && ok; ++t) {
            const int j = (pr - t + p.S) % p.S;              // order of arrival: own slice first
            ok = mbar_wait_cluster_uniform(smem_u32(&tready_bar[j]), 0, ab);
            if (ok && elect_one()) mbar_arrive_remote(smem_u32(&pready_bar[j]), lead_rank);
            __syncwarp();
        }
        cluster_wait();                                      // barrier 1
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader)
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        const uint32_t idesc1 = idesc_bf16_pair(p.RS, false, true);
        const uint64_t a_desc0 = smem_desc_sw128(0, 0, 1024);
        const uint64_t b_desc0 = smem_desc(0, p_box_bytes, 8u * p.swb, p.swb);
        cluster_arrive_relaxed();                            // barrier 1
        for (int g = 0; g < ng1; ++g) {
            ok = mbar_wait_uniform(smem_u32(&full1[s]), ph, ab);
            if (!ok) break;
            tc_fence_after();
            const uint32_t in_src = ring1_base + s * p.stage1_bytes;
            const uint32_t p_src = in_src + p.G1 * kInTileBytes;
            const int nkb = min(p.G1, p.kb1 - g * p.G1);
            // descriptors differ only in the start-address field (bits 0-13, in 16-byte units)
            uint64_t ad = a_desc0 + ((in_src >> 4) & 0x3FFFu);
            uint64_t bd = b_desc0 + ((p_src >> 4) & 0x3FFFu);
            if (elect_one()) {
                for (int i = 0; i < nkb; ++i) {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_bf16_ss_pair(tmem_base, ad + 2u * kk, bd + (uint64_t)(kk * p.swb), idesc1, (g > 0 || i > 0 || kk > 0) ? 1u : 0u);
                    ad += kInTileBytes >> 4;
                    bd += (uint64_t)(4 * p.swb);              // 64 rows of swb bytes
                }
                mma_commit_pair(smem_u32(&empty1[s]), pair_mask);
            }
            __syncwarp();
            if (++s == p.NS1) { s = 0; ph ^= 1; }
        }
        if (ok && elect_one()) mma_commit_pair(smem_u32(&tacc_bar), pair_mask);
        __syncwarp();
        s = 0;
        ph = 0;
        // own slice in both blocks' T buffers (which also means that both blocks' phase-1 accumulator columns,
        // which the first chunk's accumulator overlaps, have been read out); the other slices are waited for where
        // the k-loop first touches them
        if (ok) ok = mbar_wait_uniform(smem_u32(&tready_bar[pr]), 0, ab);
        if (ok) ok = mbar_wait_cluster_uniform(smem_u32(&pready_bar[pr]), 0, ab);
        uint32_t slices_ready = 1u << pr;
        const uint32_t idesc2 = idesc_bf16_pair(p.BN2, false, false);
        const uint64_t t_desc0 = smem_desc(t_base, 0, 8u * t_sw, t_sw);
        int i2 = 0;
        for (int j = pr; j < p.n_chunks && ok; j += p.S, ++i2) {
            const uint32_t d_tmem = tmem_base + (uint32_t)(i2 & 1) * 256u;
            ok = mbar_wait_cluster_uniform(smem_u32(&out_empty[i2 & 1]), ((i2 >> 1) & 1) ^ 1, ab);   // accumulator buffer drained in both blocks
            for (int i = 0; i < p.kb2 && ok; ++i) {
                const int kb = (int)((my_order >> (4 * i)) & 15u);
                const int nks = min(4, p.ks2 - kb * 4);
                if (i2 == 0) {
                    uint32_t need = ((my_slices >> (4 * i)) & 15u) & ~slices_ready;
                    while (need && ok) {
                        const int jj = __ffs(need) - 1;
                        ok = mbar_wait_cluster_uniform(smem_u32(&tready_bar[jj]), 0, ab);
                        if (ok) ok = mbar_wait_cluster_uniform(smem_u32(&pready_bar[jj]), 0, ab);
                        need &= need - 1;
                        slices_ready |= 1u << jj;
                    }
                    if (!ok) break;
                }
                ok = mbar_wait_uniform(smem_u32(&full2[s]), ph, ab);
                if (!ok) break;
                tc_fence_after();
                const uint32_t q_src = ring2_base + s * p.stage2_bytes;
                const uint64_t bd = a_desc0 + ((q_src >> 4) & 0x3FFFu);
                if (elect_one()) {
                    for (int kk = 0; kk < nks; ++kk) {
                        const uint32_t ks = (uint32_t)(kb * 4 + kk);      // 16-column step within T
                        const uint64_t ad = t_desc0 + (((ks >> p.t_steps_lg) * t_atom_bytes + (ks & ((1u << p.t_steps_lg) - 1u)) * 32u) >> 4);
                        mma_bf16_ss_pair(d_tmem, ad, bd + 2u * kk, idesc2, (i > 0 || kk > 0) ? 1u : 0u);
                    }
                    mma_commit_pair(smem_u32(&empty2[s]), pair_mask);
                    if (i == p.kb2 - 1) mma_commit_pair(smem_u32(&out_full[i2 & 1]), pair_mask);
                }
                __syncwarp();
                if (++s == p.NS2) { s = 0; ph ^= 1; }
            }
        }
        // a pair without a chunk of its own still has to have received every slice before the cluster may leave
        for (int j = 0; j < p.S && ok; ++j)
            if (!((slices_ready >> j) & 1u)) ok = mbar_wait_cluster_uniform(smem_u32(&tready_bar[j]), 0, ab);
        cluster_wait();                                      // barrier 1
    } else {
        // ------------------------------------------------------------------ gather + epilogue
        const int q = warp % 4;                              // tensor-memory lanes [32 q, 32 q + 32)
        const int row = q * 32 + lane;                       // row of the 128-row tile
        const int et = (warp - 2) * 32 + lane;               // index among the 128 epilogue threads
        const bool lead_warp = (warp == 2);                  // issues this block's bulk copies and stores (elect.sync)
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const bool rows_inside = m0 + q * 32 < p.M;          // (uniform) the odd block may hang over the last row tile
        bool ok = mbar_wait_uniform(smem_u32(&tacc_bar), 0, ab);   // warp-uniform from here on
        tc_fence_after();
        // barrier 1: this block's phase-1 ring is dead (every MMA that read it has completed), peers may write
        // their slices into the T region (progress only: nothing this thread wrote has to be seen by a peer)
        cluster_arrive_relaxed();
        if (ok) {
            // 32 columns per step (two tensor-memory loads in flight, one wait), a 16-column tail if RS / 16 is odd
            for (int col = 0; col < p.RS; col += 32) {
                uint32_t v[32];
                const bool two = col + 32 <= p.RS;
                tmem_ld_32x16(lane_addr + col, *reinterpret_cast<uint32_t(*)[16]>(&v[0]));
                if (two) tmem_ld_32x16(lane_addr + col + 16, *reinterpret_cast<uint32_t(*)[16]>(&v[16]));
                tmem_ld_wait();
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (half == 1 && !two) break;
                    uint32_t w[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) w[e] = pack_bf16(__uint_as_float(v[16 * half + 2 * e]), __uint_as_float(v[16 * half + 2 * e + 1]));
                    const int gc = pr * p.RS + col + 16 * half;   // first column of this piece within T
                    const uint32_t row_addr = t_base + (uint32_t)(gc / p.taw) * t_atom_bytes + (uint32_t)row * t_sw;
                    const uint32_t chunk0 = (uint32_t)(gc % p.taw) / 8u;
                    const uint32_t sw_xor = (((uint32_t)row * t_sw) >> 7) & (t_sw / 16u - 1u);
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh)
                        st_shared_v4(row_addr + (((chunk0 + hh) ^ sw_xor) << 4), w[4 * hh], w[4 * hh + 1], w[4 * hh + 2], w[4 * hh + 3]);
                }
            }
        }
        // The slice [pr RS, (pr + 1) RS) is whole atoms, i.e. one contiguous range of this block's T buffer: after the
        // four warps have written it, one thread copies it into the buffers of the blocks with the same rows in the
        // other pairs and, if asked, stores it to T_save.
        fence_proxy_async_smem();
        tc_fence_before();
        cluster_wait();                                      // barrier 1 complete: every peer's ring is dead
        ok = named_bar_and(2, 128, ok);
        if (lead_warp) {
            if (ok && elect_one()) {
                const uint32_t slice = t_base + (uint32_t)pr * 256u * (uint32_t)p.RS;
                for (int t = 1; t < p.S; ++t) {
                    const uint32_t peer = (uint32_t)(((pr + t) % p.S) * 2 + h);
                    dsmem_bulk_copy(slice, slice, 256u * (uint32_t)p.RS, smem_u32(&tready_bar[pr]), peer);
                }
                mbar_arrive(smem_u32(&tready_bar[pr]));
                if (has_tsave && m0 < p.M) {                  // (the store clips rows past M inside a tile)
                    for (int a = 0; a * p.taw < p.RS; ++a)
                        tma_store_2d(&L.t, slice + (uint32_t)a * t_atom_bytes, pr * p.RS + a * p.taw, m0);
                    tma_store_commit();
                }
            }
            __syncwarp();
        }
        // Epilogue: each warp on its own.  32 columns of its 32 rows at a time go through a [32 rows x 64 B]
        // slab of the warp (64-byte swizzle, two slabs in rotation) and leave by one TMA store each.  The bias
        // of a chunk is staged in shared memory while its MMAs run.
        const uint32_t slab0 = staging_base + (uint32_t)(warp - 2) * 2u * kSlabBytes;
        const uint32_t row_off = (uint32_t)lane * 64u;
        const uint32_t row_xor = ((uint32_t)lane >> 1) & 3u;
        int i = 0, sb = 0;
        for (int j = pr; j < p.n_chunks && ok; j += p.S, ++i) {
            const int buf = i & 1;
            if (bias) {                                      // bias_s[buf] was last read two chunks ago, before a barrier
                for (int e = et; e < p.BN2; e += 128) {
                    const int col = j * p.BN2 + e;
                    bias_s[buf][e] = col < p.N2 ? __bfloat162float(bias[col]) : 0.f;
                }
            }
            ok = mbar_wait_uniform(smem_u32(&out_full[buf]), (i >> 1) & 1, ab);
            ok = named_bar_and(3, 128, ok);                  // the four warps go on, or give up, together (and see the bias)
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = lane_addr + (uint32_t)buf * 256u;
            for (int g = 0; g * 64 < p.BN2; ++g) {
                const int col0 = j * p.BN2 + g * 64;
                if (col0 >= p.N2) break;                     // (uniform) nothing of this piece is inside Out
                uint32_t v[64];                              // both halves are loaded before the first is converted
                tmem_ld_32x32(d_tmem + g * 64, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                tmem_ld_32x32(d_tmem + g * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                tmem_ld_wait();
#pragma unroll
                for (int hh = 0; hh < 2; ++hh, ++sb) {
                    if (col0 + 32 * hh >= p.N2) break;       // (uniform)
                    const uint32_t slab = slab0 + (uint32_t)(sb & 1) * kSlabBytes;
                    if (sb >= 2) {                           // the store that last read this slab has finished reading
                        tma_store_wait_read<1>();            // (only the lane that issued the stores has any to wait for)
                        __syncwarp();
                    }
                    if (bias) {
                        const float4* bp = reinterpret_cast<const float4*>(&bias_s[buf][g * 64 + hh * 32]);
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float4 b4 = bp[e];
                            v[32 * hh + 4 * e] = __float_as_uint(__uint_as_float(v[32 * hh + 4 * e]) + b4.x);
                            v[32 * hh + 4 * e + 1] = __float_as_uint(__uint_as_float(v[32 * hh + 4 * e + 1]) + b4.y);
                            v[32 * hh + 4 * e + 2] = __float_as_uint(__uint_as_float(v[32 * hh + 4 * e + 2]) + b4.z);
                            v[32 * hh + 4 * e + 3] = __float_as_uint(__uint_as_float(v[32 * hh + 4 * e + 3]) + b4.w);
                        }
                    }
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc)
                        st_shared_v4(slab + row_off + ((((uint32_t)cc) ^ row_xor) << 4),
                                     pack_bf16(__uint_as_float(v[32 * hh + 8 * cc]), __uint_as_float(v[32 * hh + 8 * cc + 1])),
                                     pack_bf16(__uint_as_float(v[32 * hh + 8 * cc + 2]), __uint_as_float(v[32 * hh + 8 * cc + 3])),
                                     pack_bf16(__uint_as_float(v[32 * hh + 8 * cc + 4]), __uint_as_float(v[32 * hh + 8 * cc + 5])),
                                     pack_bf16(__uint_as_float(v[32 * hh + 8 * cc + 6]), __uint_as_float(v[32 * hh + 8 * cc + 7])));
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (elect_one()) {
                        if (rows_inside) tma_store_2d(&L.out, slab, col0 + 32 * hh, m0 + q * 32);
                        tma_store_commit();
                    }
                    __syncwarp();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(smem_u32(&out_empty[buf]), lead_rank);
        }
        tma_store_wait_read<0>();                            // shared memory may go once the stores have read it
        __syncwarp();
    }

    // No block leaves (or frees tensor memory) while a partner or a peer may still signal one of its barriers, read
    // its shared memory with an MMA, write its accumulators or copy a slice into it: every thread of the cluster is
    // past all of that when it arrives here (the leader's MMA warp has seen every slice land; the odd block's warp 1
    // has seen the same for its buffer; every epilogue warp has made its last arrival).
    tc_fence_before();
    cluster_arrive();
    cluster_wait();
    if (warp == 1) {
        if (abort_flag) {            // give copies and MMAs still in flight time to land before freeing
            for (int i = 0; i < 256; ++i) __nanosleep(1000);
        }
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

struct Plan {
    int S, RS, swb, taw, BN2, G1, NS1, NS2;
    uint32_t stage1_bytes, stage2_bytes, t_bytes, smem_bytes;
};

int g_tune_S = 0, g_tune_G1 = 0, g_tune_BN2 = 0;    // 0 = automatic

inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

int pick_bn2(int64_t N2, int S) {
    if (g_tune_BN2) return g_tune_BN2;
    const int cands[3] = {256, 192, 128};
    int best = 128;
    int64_t best_cost = -1;
    for (int bn : cands) {
        const int64_t chunks = (N2 + bn - 1) / bn;
        const int64_t cost = ((chunks + S - 1) / S) * bn;
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = bn; }
    }
    return best;
}

// Clusters of n blocks that can be resident at once (a cluster needs n free SMs inside one GPC).
int max_active_clusters(int n) {
    static int cache_on[kMaxDevices][2 * kMaxS + 1] = {};
    int* cache = cache_on[device_slot()];
    if (n < 2 || n > 2 * kMaxS) return kNumSms;
    if (cache[n] == 0) {
        int cnt = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)n, 1, 1);
        cfg.blockDim = dim3(kThreads, 1, 1);
        cfg.dynamicSmemBytes = kSmemLimit;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)n;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(chain_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&cnt, chain_pair_kernel, &cfg) != cudaSuccess || cnt < 1) {
            cudaGetLastError();
            cnt = (kNumSms - 20) / n;                   // no answer (no device yet): a cautious guess
        }
        cache[n] = cnt;
    }
    return cache[n];
}

bool shape_ok(const ChainArgs& a) {
    if (a.dtype != LRD_BF16 || a.M < 129 || a.K1 < 1 || a.N2 < 1) return false;
    if (a.r < 32 || a.r > 512 || a.r % 32) return false;
    if (a.M > (int64_t)32767 * 256 || a.K1 > (1 << 30) || a.N2 > (1 << 30)) return false;
    if (!aligned16(a.In) || !aligned16(a.P) || !aligned16(a.Q) || !aligned16(a.Out)) return false;
    if (a.ld_in % 8 || a.ldp % 8 || a.ldq % 8 || a.ld_out % 8) return false;
    if (a.T_save && (!aligned16(a.T_save) || a.ldt % 8)) return false;
    if (a.bias && !aligned16(a.bias)) return false;
    return true;
}

// Estimated clocks of the slowest block: phase 1 at max(MMA, fill), phase 2 at the MMA rate, plus the serial
// latencies around them; clusters that are not all resident at once run in waves.
bool make_plan(const ChainArgs& a, int layers, Plan* out) {
    if (!shape_ok(a)) return false;
    const int64_t row_pairs = (a.M + 255) / 256;
    const int t_bytes = (int)((a.r * 256 + 1023) / 1024 * 1024);      // 128 rows x r columns of bf16
    const int kb1 = (int)((a.K1 + 63) / 64);
    Plan best{};
    double best_cost = 1e300;
    for (int S = kMaxS; S >= 1; --S) {
        if (g_tune_S && S != g_tune_S) continue;
        if (a.r % (32 * S)) continue;
        const int RS = (int)a.r / S, RSL = RS / 2;
        if (RS > 256) continue;
        const int swb = RSL % 64 == 0 ? 128 : (RSL % 32 == 0 ? 64 : 32);
        const int taw = RS % 64 == 0 ? 64 : (RS % 32 == 0 ? 32 : 16);
        const int BN2 = pick_bn2(a.N2, S);
        if (BN2 % 32) continue;
        const uint32_t kb1_bytes = kInTileBytes + 128u * (uint32_t)RSL, kb2_bytes = (uint32_t)(BN2 / 2) * 128u;
        // two k-blocks per phase-1 stage where they are small: the MMA warp's work per stage (a wait, a commit)
        // is then spread over eight MMAs
        int G1 = g_tune_G1 ? g_tune_G1 : (kb1_bytes <= 28 * 1024 ? 2 : 1);
        if (G1 > 4) G1 = 4;
        if (G1 > kb1) G1 = kb1;
        const int64_t all = (int64_t)kSmemLimit - 1024;
        const int64_t ring2 = all - t_bytes - (int64_t)kStagingBytes;
        const uint32_t s1b = (uint32_t)G1 * kb1_bytes;
        if (all < 2 * (int64_t)s1b || ring2 < 2 * (int64_t)kb2_bytes) continue;
        int NS1 = (int)(all / s1b), NS2 = (int)(ring2 / kb2_bytes);
        if (NS1 > kMaxSlots) NS1 = kMaxSlots;
        if (NS2 > kMaxSlots) NS2 = kMaxSlots;
        const int64_t clusters = row_pairs * layers;
        const int64_t room = max_active_clusters(2 * S);
        const int64_t waves = (clusters + room - 1) / room;
        const int64_t chunks = (a.N2 + BN2 - 1) / BN2, my_chunks = (chunks + S - 1) / S;
        const double fill1 = (double)kb1 * kb1_bytes / 90.0, mma1 = (double)kb1 * 4.0 * (RS / 2.0);
        const double ph2 = (double)my_chunks * ((a.r + 15) / 16) * (BN2 / 2.0);
        const double cost = (double)waves * (std::max(fill1, mma1) + ph2 + 6000.0);
        if (cost < best_cost) {
            best_cost = cost;
            const uint32_t used1 = (uint32_t)NS1 * s1b, used2 = (uint32_t)t_bytes + kStagingBytes + (uint32_t)NS2 * kb2_bytes;
            best = Plan{S, RS, swb, taw, BN2, G1, NS1, NS2, s1b, kb2_bytes, (uint32_t)t_bytes, 1024u + std::max(used1, used2)};
        }
    }
    if (best_cost >= 1e300) return false;
    *out = best;
    return true;
}

bool same_shape(const ChainArgs& a, const ChainArgs& b) {
    return a.M == b.M && a.K1 == b.K1 && a.r == b.r && a.N2 == b.N2 && a.dtype == b.dtype;
}

}  // namespace

void chain_pair_tuning(int S, int G1, int BN2) {
    g_tune_S = S;
    g_tune_G1 = G1;
    g_tune_BN2 = BN2;
}

bool chain_pair_eligible(const ChainArgs* layers, int n) {
    if (n < 1 || n > kChainMaxLayers) return false;
    for (int i = 0; i < n; ++i)
        if (!shape_ok(layers[i]) || !same_shape(layers[0], layers[i])) return false;
    Plan pl;
    return make_plan(layers[0], n, &pl);
}

// Eligible, the ring beside the T buffer holds at least three Q tiles, and the shape is one where pairs measured
// faster than single blocks: several layers in one launch, or a layer whose first product dominates (at 4096
// tokens, r = 384: 3072 -> 768 forward 21.2 us on pairs against 22.5 us, but 768 -> 3072 24.6 against 18.5 us --
// with few wide chunks per pair the epilogue of one chunk does not hide behind the MMAs of the next).
bool chain_pair_preferred(const ChainArgs* layers, int n) {
    if (!chain_pair_eligible(layers, n)) return false;
    Plan pl;
    if (!make_plan(layers[0], n, &pl) || pl.NS2 < 3) return false;
    // Measured against the chain on single blocks: pairs win for groups, where the first product dominates, where
    // the single blocks' T buffer leaves fewer than three weight tiles in flight (r = 512), and at r >= 384 once
    // there are more row tiles than clusters of four fit on the GPU (8192 tokens, 4096 x 4096: r = 384 59 against
    // 64 us forward, r = 512 62 against 85; r = 256 stays on single blocks, 50 against 54).
    const ChainArgs& a = layers[0];
    return n > 1 || a.K1 >= 2 * a.N2 || (a.r > 384 && !chain_preferred(a)) || (a.r >= 384 && (a.M + 127) / 128 > 37);
}

// Eligible, with at least three weight tiles of the second product in flight: the form to take where the launch should
// leave SMs free for others (16 clusters of 6 or fewer blocks against 32 clusters of 4).
bool chain_pair_roomy(const ChainArgs* layers, int n) {
    if (!chain_pair_eligible(layers, n)) return false;
    Plan pl;
    return make_plan(layers[0], n, &pl) && pl.NS2 >= 3;
}

lrd_status_t chain_pair_launch(const ChainArgs* layers, int n, cudaStream_t stream) {
    if (!chain_pair_eligible(layers, n)) return LRD_ERR_UNSUPPORTED;
    const ChainArgs& a = layers[0];
    Plan pl;
    if (!make_plan(a, n, &pl)) return LRD_ERR_UNSUPPORTED;
    PairGroup grp;
    PairParams p;
    for (int i = 0; i < kChainMaxLayers; ++i) {
        const ChainArgs& c = layers[i < n ? i : 0];
        LayerMaps& L = grp.layer[i];
        bool ok = make_tmap_2d_bf16(&L.in, c.In, (uint64_t)c.M, (uint64_t)c.K1, (uint64_t)c.ld_in, 128, 64);
        ok = ok && make_tmap_2d_bf16(&L.p, c.P, (uint64_t)c.K1, (uint64_t)c.r, (uint64_t)c.ldp, 64u * (uint32_t)pl.G1, (uint32_t)pl.swb / 2);
        ok = ok && make_tmap_2d_bf16(&L.q, c.Q, (uint64_t)c.N2, (uint64_t)c.r, (uint64_t)c.ldq, (uint32_t)(pl.BN2 / 2), 64);
        ok = ok && make_tmap_2d_bf16(&L.out, c.Out, (uint64_t)c.M, (uint64_t)c.N2, (uint64_t)c.ld_out, 32, 32);
        if (c.T_save)
            ok = ok && make_tmap_2d_bf16(&L.t, c.T_save, (uint64_t)c.M, (uint64_t)c.r, (uint64_t)c.ldt, 128, (uint32_t)pl.taw);
        else
            L.t = L.out;
        if (!ok) { cuda_ok(cudaErrorUnknown, "tensor map encode (pair chain)"); return LRD_ERR_CUDA; }
        p.bias[i] = (const __nv_bfloat16*)c.bias;
        p.has_tsave[i] = c.T_save ? 1 : 0;
    }
    p.S = pl.S; p.RS = pl.RS; p.swb = pl.swb; p.BN2 = pl.BN2;
    p.n_chunks = (int)((a.N2 + pl.BN2 - 1) / pl.BN2);
    p.kb1 = (int)((a.K1 + 63) / 64);
    p.ks2 = (int)a.r / 16;
    p.kb2 = (int)((a.r + 63) / 64);
    p.N2 = (int)a.N2;
    p.M = (int)a.M;
    p.G1 = pl.G1; p.NS1 = pl.NS1; p.NS2 = pl.NS2;
    p.stage1_bytes = pl.stage1_bytes; p.stage2_bytes = pl.stage2_bytes; p.t_bytes = pl.t_bytes;
    p.taw = pl.taw;
    p.t_steps_lg = p.taw == 64 ? 2 : (p.taw == 32 ? 1 : 0);
    // A block sends its slice of T to the pairs pr + 1, pr + 2, ... in turn, so slice j reaches pair c as the
    // ((c - j) mod S)-th arrival (0 = its own); phase 2 takes the k-blocks in the order in which the last slice
    // they touch arrives.  The order depends on the launch shape only, so results stay reproducible.
    for (int c = 0; c < kMaxS; ++c) {
        p.kb_order[c] = 0; p.kb_slices[c] = 0;
        if (c >= p.S) continue;
        int cnt = 0;
        for (int rank = 0; rank < p.S; ++rank)
            for (int kb = 0; kb < p.kb2; ++kb) {
                const int nks = std::min(4, p.ks2 - kb * 4);
                const int j_lo = kb * 64 / p.RS, j_hi = (kb * 64 + nks * 16 - 1) / p.RS;
                int worst = 0;
                uint32_t mask = 0;
                for (int j = j_lo; j <= j_hi; ++j) {
                    worst = std::max(worst, (c - j + p.S) % p.S);
                    mask |= 1u << j;
                }
                if (worst != rank) continue;
                p.kb_order[c] |= (uint32_t)kb << (4 * cnt);
                p.kb_slices[c] |= mask << (4 * cnt);
                ++cnt;
            }
    }
    p.timeout_flag = device_timeout_flag();

    static bool configured_on[kMaxDevices] = {};
    bool& configured = configured_on[device_slot()];
    if (!configured) {
        if (!cuda_ok(cudaFuncSetAttribute(chain_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit), "cudaFuncSetAttribute(pair chain)"))
            return LRD_ERR_CUDA;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pl.S), (unsigned)((a.M + 255) / 256), (unsigned)n);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)(2 * pl.S);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // the kernel waits (griddepcontrol.wait) before it touches global memory
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (!cuda_ok(cudaLaunchKernelEx(&cfg, chain_pair_kernel, grp, p), "cudaLaunchKernelEx(pair chain)")) return LRD_ERR_CUDA;
    count_launch();
    return LRD_OK;
}

}  // namespace lrd
