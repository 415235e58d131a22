// Fused chain  Out[M x N2] = (In[M x K1] P[K1 x r]) Q[N2 x r]^T (+ bias)  on sm_100a.
//
// A cluster of C blocks owns one 128-row tile.
//   Phase 1  block c forms its r/C-column slice of T = In P in tensor memory (TMA-fed tcgen05.mma:
//            In K-major, the slice of P MN-major), one or two 64-deep k-blocks per stage, as many
//            stages as the shared memory beside the T buffer holds.
//   Gather   four warps read the slice (tcgen05.ld), round it to bf16 and write it into this block's T
//            buffer (K-major, swizzled, slices are whole atoms = one contiguous range); one thread then
//            copies the range into every peer's T buffer with bulk DSMEM copies that complete on the
//            peer's barrier.  T never goes to global memory unless T_save asks.
//   Phase 2  block c forms every C-th column chunk of Out = T Q^T (T from shared memory, Q by TMA, one
//            64-deep tile per stage), double-buffered in tensor memory; each epilogue warp adds the
//            bias (staged in shared memory while the MMAs run), rounds to bf16 and stores its 32 rows
//            through its own [32 x 32] slabs by TMA stores (which clip the ragged edges).
// Warp 0: TMA producer.  Warp 1: tensor memory + MMA issue.  Warps 2-5: gather and epilogue.
// Two cluster barriers: the first (every block's barriers exist) is arrived at once and waited on only
// where the first remote copy is near; the second (every block has received all slices sent to it) lets
// no block leave while a peer may still be reading its shared memory.  The kernel's set-up runs before
// griddepcontrol.wait and so overlaps the tail of the previous kernel in the stream.
// Every wait is bounded; a wait that runs out raises the device timeout flag and the block tears
// down in order.
#include "chain.cuh"

#include "ptx.cuh"
#include "tc.cuh"
#include "tma.cuh"

namespace lrd {
namespace {

using namespace ptx;

constexpr int kThreads = 192;
constexpr int kMaxStages = 12;
constexpr int kMaxCluster = 4;       // blocks per row tile
constexpr int kMaxKb2 = 8;           // 64-column k-blocks of T (r <= 512)
constexpr uint32_t kSmemLimit = 224 * 1024;         // dynamic shared memory; the rest is left for the barriers and the bias
constexpr uint32_t kInTileBytes = 128 * 64 * 2;     // In tile of one k-block: 128 rows x 64 k
constexpr uint32_t kSlabBytes = 32 * 32 * 2;        // epilogue slab of one warp: 32 rows x 32 columns of bf16
constexpr uint32_t kStagingBytes = 4 * 2 * kSlabBytes;

struct ChainParams {
    int C, RS, swb, BN2, n_chunks, kb1, ks2, kb2, N2;
    int G1, S1, S2;           // k-blocks per phase-1 stage; stage counts of the two phases
    uint32_t stage1_bytes, stage2_bytes, t_bytes;
    int taw;                  // columns per atom of the T buffer (64, 32 or 16; swizzle span = 2 * taw bytes)
    int t_steps_lg;           // log2 of the MMA k-steps (16 columns) per atom
    const __nv_bfloat16* bias;
    int has_tsave;
    unsigned int* timeout_flag;
    // Phase 2 of block c walks over the 64-column k-blocks of T in the order kb_order[c] (4 bits per position)
    // and needs the slices in kb_slices[c] (a 4-bit mask per position) for the k-block at that position.
    uint32_t kb_order[kMaxCluster], kb_slices[kMaxCluster];
};

__global__ void __launch_bounds__(kThreads, 1)
chain_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmP,
             const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmOut,
             const __grid_constant__ CUtensorMap tmT, const ChainParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full1[kMaxStages], empty1[kMaxStages], full2[kMaxStages], empty2[kMaxStages],
        tacc_bar, tready_bar[kMaxCluster], out_full[2], out_empty[2];
    __shared__ __align__(16) float bias_s[2][256];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    // phase 1: [ring of S1 stages] over ALL of the shared memory (T is written only after the last MMA of phase 1 has
    // read its operands);  afterwards: [T | output slabs | ring of S2 stages].  What a block can stream is (bytes of
    // stages in flight) / (about a microsecond per stage turn: load latency under load, then its MMAs), so phase 1
    // gets every byte there is.
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t t_base = smem_base;
    const uint32_t ring1_base = smem_base;
    const uint32_t staging_base = t_base + p.t_bytes;
    const uint32_t ring2_base = staging_base + kStagingBytes;
    const AbortCtx ab{&abort_flag, p.timeout_flag};
    const uint32_t t_sw = 2u * (uint32_t)p.taw, t_atom_bytes = 128u * t_sw;   // T: atoms of [128 rows x taw columns]
    // The warp index is made provably warp-uniform, and the single-thread instructions (TMA, MMA, commit)
    // are issued under elect.sync by an otherwise converged warp: their operands then stay in uniform
    // registers.  (Issued from a lane-0 branch instead, every such instruction costs hundreds of cycles.)
    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0);
    const int lane = threadIdx.x % 32;
    const int c = (int)cluster_ctarank();
    const uint32_t my_order = c == 0 ? p.kb_order[0] : (c == 1 ? p.kb_order[1] : (c == 2 ? p.kb_order[2] : p.kb_order[3]));
    const uint32_t my_slices = c == 0 ? p.kb_slices[0] : (c == 1 ? p.kb_slices[1] : (c == 2 ? p.kb_slices[2] : p.kb_slices[3]));
    const int m0 = blockIdx.y * 128;
    const int ng1 = (p.kb1 + p.G1 - 1) / p.G1;                                 // stage turns of phase 1
    // phase-1 stage: G1 In tiles, then the P boxes (one per column atom, 64 G1 rows tall)
    const uint32_t p_box_bytes = 64u * (uint32_t)p.G1 * (uint32_t)p.swb;

    if (warp == 0 && lane >= 1 && lane <= kMaxStages) {      // the stage barriers, one stage per lane
        const int s = lane - 1;
        mbar_init(smem_u32(&full1[s]), 1);
        mbar_init(smem_u32(&empty1[s]), 1);
        mbar_init(smem_u32(&full2[s]), 1);
        mbar_init(smem_u32(&empty2[s]), 1);
        fence_mbar_init();
    }
    if (threadIdx.x == 0) {
        abort_flag = 0;
        prefetch_tmap(&tmIn);
        prefetch_tmap(&tmP);
        prefetch_tmap(&tmQ);
        prefetch_tmap(&tmOut);
        mbar_init(smem_u32(&tacc_bar), 1);
        // one barrier per slice of T: this block's own slice is ready after one arrival (written by its gather
        // warps), a peer's slice once its bytes have landed
        for (int j = 0; j < p.C; ++j) mbar_init(smem_u32(&tready_bar[j]), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&out_full[i]), 1);
            mbar_init(smem_u32(&out_empty[i]), 4);
        }
        for (int j = 0; j < p.C; ++j)
            if (j != c) mbar_expect_tx(smem_u32(&tready_bar[j]), 256u * (uint32_t)p.RS);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    // Cluster barrier 1 (every block's barriers exist, and its phase-1 ring -- which covers the region the peers'
    // slices of T land in -- is dead, before a peer pushes into it): the gather warps arrive once this block's
    // phase-1 MMAs have completed, the other warps now; waited on only where the first remote operation is near.
    if (warp < 2) cluster_arrive();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // Everything above touched only this block's own shared and tensor memory, so it may overlap the tail
    // of the previous kernel in the stream; global memory is first read (and written) below this line.
    griddep_launch_dependents();
    griddep_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        int s = 0;
        uint32_t ph = 1;                                     // parity to wait on for an empty stage
        bool ok = true;
        const int atom_cols = p.swb / 2;
        const int n_pbox = p.RS / atom_cols;
        for (int g = 0; g < ng1 && ok; ++g) {
            const uint32_t fb = smem_u32(&full1[s]);
            ok = mbar_wait_uniform(smem_u32(&empty1[s]), ph, ab);
            if (!ok) break;
            const uint32_t dst = ring1_base + s * p.stage1_bytes;
            const int kb0 = g * p.G1;
            if (elect_one()) {
                mbar_expect_tx(fb, p.stage1_bytes);
                for (int i = 0; i < p.G1; ++i)               // k-blocks past K1 read as zeros
                    tma_load_2d(dst + i * kInTileBytes, &tmIn, fb, (kb0 + i) * 64, m0);
                for (int i = 0; i < n_pbox; ++i)
                    tma_load_2d(dst + p.G1 * kInTileBytes + i * p_box_bytes, &tmP, fb, c * p.RS + i * atom_cols, kb0 * 64);
            }
            __syncwarp();
            if (++s == p.S1) { s = 0; ph ^= 1; }
        }
        // the ring is laid out anew for phase 2: wait until every phase-1 MMA has read its operands
        if (ok) ok = mbar_wait_uniform(smem_u32(&tacc_bar), 0, ab);
        s = 0;
        ph = 1;
        for (int j = c; j < p.n_chunks && ok; j += p.C) {
            for (int i = 0; i < p.kb2; ++i) {                // columns past r read as zeros (never multiplied)
                const int kb = (int)((my_order >> (4 * i)) & 15u);
                const uint32_t fb = smem_u32(&full2[s]);
                ok = mbar_wait_uniform(smem_u32(&empty2[s]), ph, ab);
                if (!ok) break;
                if (elect_one()) {
                    mbar_expect_tx(fb, p.stage2_bytes);
                    tma_load_2d(ring2_base + s * p.stage2_bytes, &tmQ, fb, kb * 64, j * p.BN2);
                }
                __syncwarp();
                if (++s == p.S2) { s = 0; ph ^= 1; }
            }
        }
        cluster_wait();        // barrier 1
        cluster_arrive_relaxed();   // barrier 2 (progress only)
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        const uint32_t idesc1 = idesc_bf16(p.RS, false, true);
        const uint64_t a_desc0 = smem_desc_sw128(0, 0, 1024);
        const uint64_t b_desc0 = smem_desc(0, p_box_bytes, 8u * p.swb, p.swb);
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
                        mma_bf16_ss(tmem_base, ad + 2u * kk, bd + (uint64_t)(kk * p.swb), idesc1, (g > 0 || i > 0 || kk > 0) ? 1u : 0u);
                    ad += kInTileBytes >> 4;
                    bd += (uint64_t)(4 * p.swb);              // 64 rows of swb bytes
                }
                mma_commit(smem_u32(&empty1[s]));
            }
            __syncwarp();
            if (++s == p.S1) { s = 0; ph ^= 1; }
        }
        if (ok && elect_one()) mma_commit(smem_u32(&tacc_bar));
        __syncwarp();
        // this block's own slice is in its T buffer, which also means that the phase-1 accumulator columns
        // (which the first chunk's accumulator overlaps) have been read out; the peers' slices are waited for
        // where the k-loop first touches them
        if (ok) ok = mbar_wait_uniform(smem_u32(&tready_bar[c]), 0, ab);
        uint32_t slices_ready = 1u << c;
        const uint32_t idesc2 = idesc_bf16(p.BN2, false, false);
        const uint64_t t_desc0 = smem_desc(t_base, 0, 8u * t_sw, t_sw);
        // T's descriptor for k-step kk of k-block kb is t_desc0 + kb * tk_stride + tk_off[kk] (16-byte units): what the
        // issuing thread computes per MMA is kept to one add (its instructions are what paces a stage of four MMAs)
        const uint32_t tk_stride = ((4u >> p.t_steps_lg) * t_atom_bytes) >> 4;
        uint32_t tk_off[4];
#pragma unroll
        for (uint32_t kk = 0; kk < 4; ++kk)
            tk_off[kk] = (((kk >> p.t_steps_lg) * t_atom_bytes) + (kk & ((1u << p.t_steps_lg) - 1u)) * 32u) >> 4;
        s = 0;
        ph = 0;
        int i2 = 0;
        for (int j = c; j < p.n_chunks && ok; j += p.C, ++i2) {
            const uint32_t d_tmem = tmem_base + (uint32_t)(i2 & 1) * 256u;
            ok = mbar_wait_uniform(smem_u32(&out_empty[i2 & 1]), ((i2 >> 1) & 1) ^ 1, ab);   // accumulator buffer drained
            for (int i = 0; i < p.kb2 && ok; ++i) {
                const int kb = (int)((my_order >> (4 * i)) & 15u);
                const int nks = min(4, p.ks2 - kb * 4);
                if (i2 == 0) {
                    uint32_t need = ((my_slices >> (4 * i)) & 15u) & ~slices_ready;
                    while (need && ok) {
                        const int j = __ffs(need) - 1;
                        ok = mbar_wait_cluster_uniform(smem_u32(&tready_bar[j]), 0, ab);
                        need &= need - 1;
                        slices_ready |= 1u << j;
                    }
                    if (!ok) break;
                }
                ok = mbar_wait_uniform(smem_u32(&full2[s]), ph, ab);
                if (!ok) break;
                tc_fence_after();
                const uint32_t q_src = ring2_base + s * p.stage2_bytes;
                const uint64_t bd = a_desc0 + ((q_src >> 4) & 0x3FFFu);
                if (elect_one()) {
                    const uint64_t adk = t_desc0 + (uint32_t)kb * tk_stride;
                    const uint32_t acc = i > 0 ? 1u : 0u;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)                        // 16-column steps within T
                        if (kk < nks) mma_bf16_ss(d_tmem, adk + tk_off[kk], bd + 2u * kk, idesc2, kk > 0 ? 1u : acc);
                    mma_commit(smem_u32(&empty2[s]));
                    if (i == p.kb2 - 1) mma_commit(smem_u32(&out_full[i2 & 1]));
                }
                __syncwarp();
                if (++s == p.S2) { s = 0; ph ^= 1; }
            }
        }
        // a block without a chunk of its own still has to have received every slice before it passes barrier 2
        for (int j = 0; j < p.C && ok; ++j)
            if (!((slices_ready >> j) & 1u)) ok = mbar_wait_cluster_uniform(smem_u32(&tready_bar[j]), 0, ab);
        cluster_wait();        // barrier 1 (long complete: every peer has pushed into this block)
        cluster_arrive_relaxed();   // barrier 2: this block has received everything its peers send
    } else {
        // ------------------------------------------------------------------ gather + epilogue
        const int q = warp % 4;                              // tensor-memory lanes [32 q, 32 q + 32)
        const int row = q * 32 + lane;                       // row of the 128-row tile
        const int et = (warp - 2) * 32 + lane;               // index among the 128 epilogue threads
        const bool lead_warp = (warp == 2);                  // issues this block's bulk copies and stores (elect.sync)
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        bool ok = mbar_wait_uniform(smem_u32(&tacc_bar), 0, ab);   // warp-uniform from here on
        tc_fence_after();
        cluster_arrive_relaxed();   // barrier 1: this block's phase-1 ring is dead (progress only, no data)
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
                    const int gc = c * p.RS + col + 16 * half;   // first column of this piece within T
                    const uint32_t row_addr = t_base + (uint32_t)(gc / p.taw) * t_atom_bytes + (uint32_t)row * t_sw;
                    const uint32_t chunk0 = (uint32_t)(gc % p.taw) / 8u;
                    const uint32_t sw_xor = (((uint32_t)row * t_sw) >> 7) & (t_sw / 16u - 1u);
#pragma unroll
                    for (int h = 0; h < 2; ++h)
                        st_shared_v4(row_addr + (((chunk0 + h) ^ sw_xor) << 4), w[4 * h], w[4 * h + 1], w[4 * h + 2], w[4 * h + 3]);
                }
            }
        }
        // The slice [c RS, (c+1) RS) is whole atoms, i.e. one contiguous range of this block's T buffer: after
        // the four warps have written it, one thread copies it into every peer's buffer (bulk DSMEM copy that
        // completes on the peer's barrier) and, if asked, stores it to T_save.  The accumulator columns of
        // the slice are free for phase 2 from here on.
        fence_proxy_async_smem();
        tc_fence_before();
        cluster_wait();        // barrier 1: the peers' barriers exist
        ok = named_bar_and(2, 128, ok);    // the four warps go on, or give up, together
        if (lead_warp) {
            if (ok && elect_one()) {
                const uint32_t slice = t_base + (uint32_t)c * 256u * (uint32_t)p.RS;
                for (int t = 1; t < p.C; ++t) {
                    const uint32_t peer = (uint32_t)((c + t) % p.C);
                    dsmem_bulk_copy(slice, slice, 256u * (uint32_t)p.RS, smem_u32(&tready_bar[c]), peer);
                }
                mbar_arrive(smem_u32(&tready_bar[c]));
                if (p.has_tsave) {
                    for (int a = 0; a * p.taw < p.RS; ++a)
                        tma_store_2d(&tmT, slice + (uint32_t)a * t_atom_bytes, c * p.RS + a * p.taw, m0);
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
        bool arrived2 = false;
        for (int j = c; j < p.n_chunks && ok; j += p.C, ++i) {
            const int buf = i & 1;
            if (p.bias) {                                    // bias_s[buf] was last read two chunks ago, before a barrier
                for (int e = et; e < p.BN2; e += 128) {
                    const int col = j * p.BN2 + e;
                    bias_s[buf][e] = col < p.N2 ? __bfloat162float(p.bias[col]) : 0.f;
                }
            }
            ok = mbar_wait_uniform(smem_u32(&out_full[buf]), (i >> 1) & 1, ab);
            ok = named_bar_and(3, 128, ok);                  // the four warps go on, or give up, together (and see the bias)
            if (!ok) break;
            if (!arrived2) { cluster_arrive_relaxed(); arrived2 = true; }   // barrier 2 (T was complete before these MMAs)
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
                for (int h = 0; h < 2; ++h, ++sb) {
                    if (col0 + 32 * h >= p.N2) break;        // (uniform)
                    const uint32_t slab = slab0 + (uint32_t)(sb & 1) * kSlabBytes;
                    if (sb >= 2) {                           // the store that last read this slab has finished reading
                        tma_store_wait_read<1>();            // (only the lane that issued the stores has any to wait for)
                        __syncwarp();
                    }
                    if (p.bias) {
                        const float4* bp = reinterpret_cast<const float4*>(&bias_s[buf][g * 64 + h * 32]);
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float4 b4 = bp[e];
                            v[32 * h + 4 * e] = __float_as_uint(__uint_as_float(v[32 * h + 4 * e]) + b4.x);
                            v[32 * h + 4 * e + 1] = __float_as_uint(__uint_as_float(v[32 * h + 4 * e + 1]) + b4.y);
                            v[32 * h + 4 * e + 2] = __float_as_uint(__uint_as_float(v[32 * h + 4 * e + 2]) + b4.z);
                            v[32 * h + 4 * e + 3] = __float_as_uint(__uint_as_float(v[32 * h + 4 * e + 3]) + b4.w);
                        }
                    }
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc)
                        st_shared_v4(slab + row_off + ((((uint32_t)cc) ^ row_xor) << 4),
                                     pack_bf16(__uint_as_float(v[32 * h + 8 * cc]), __uint_as_float(v[32 * h + 8 * cc + 1])),
                                     pack_bf16(__uint_as_float(v[32 * h + 8 * cc + 2]), __uint_as_float(v[32 * h + 8 * cc + 3])),
                                     pack_bf16(__uint_as_float(v[32 * h + 8 * cc + 4]), __uint_as_float(v[32 * h + 8 * cc + 5])),
                                     pack_bf16(__uint_as_float(v[32 * h + 8 * cc + 6]), __uint_as_float(v[32 * h + 8 * cc + 7])));
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (elect_one()) {
                        tma_store_2d(&tmOut, slab, col0 + 32 * h, m0 + q * 32);
                        tma_store_commit();
                    }
                    __syncwarp();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&out_empty[buf]));
        }
        if (!arrived2) cluster_arrive_relaxed();
        tma_store_wait_read<0>();                            // shared memory may go once the stores have read it
        __syncwarp();
    }

    // Cluster barrier 2: no block leaves while a peer may still be reading its slice out of this block's
    // shared memory (each block arrived once all slices addressed to it had landed).
    cluster_wait();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (abort_flag) {
            for (int i = 0; i < 256; ++i) __nanosleep(1000);
        }
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

struct Plan {
    int C, RS, swb, BN2, G1, S1, S2;
    uint32_t stage1_bytes, stage2_bytes, t_bytes, smem_bytes;
};

int g_tune_C = 0, g_tune_G1 = 0, g_tune_BN2 = 0;    // 0 = automatic

inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

// Column chunk width of phase 2: the block with the most chunks sets the pace, so minimise
// (chunks of the busiest block) x width; wider chunks on ties (fewer, larger copies).
int pick_bn2(int64_t N2, int C) {
    if (g_tune_BN2) return g_tune_BN2;
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

// Clusters of C blocks that can be resident at once (a cluster needs C free SMs inside one GPC).
int max_active_clusters(int C) {
    static int cache_on[kMaxDevices][5] = {};
    int* cache = cache_on[device_slot()];
    if (C < 2 || C > 4) return kNumSms;
    if (cache[C] == 0) {
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)C, 1, 1);
        cfg.blockDim = dim3(kThreads, 1, 1);
        cfg.dynamicSmemBytes = kSmemLimit;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)C;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, chain_kernel, &cfg) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = (kNumSms - 20) / C;                     // no answer (no device yet): a cautious guess
        }
        cache[C] = n;
    }
    return cache[C];
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
    const int kb1 = (int)((a.K1 + 63) / 64);
    Plan best{};
    bool found = false;
    const int cands[4] = {4, 3, 2, 1};
    for (int C : cands) {
        if (g_tune_C && C != g_tune_C) continue;
        if (a.r % (16 * C)) continue;
        const int RS = (int)a.r / C;
        if (RS > 256) continue;
        const int swb = RS % 64 == 0 ? 128 : (RS % 32 == 0 ? 64 : 32);
        const int BN2 = pick_bn2(a.N2, C);
        const int64_t ring1 = (int64_t)kSmemLimit - 1024;                         // phase 1 has all of it
        const int64_t ring2 = ring1 - t_bytes - (int64_t)kStagingBytes;
        const uint32_t kb1_bytes = kInTileBytes + 128u * RS, kb2_bytes = (uint32_t)BN2 * 128u;
        if (ring2 < 2 * (int64_t)kb2_bytes) continue;
        // phase 1: two k-blocks per stage: what a stage costs the issuing threads beside its copies and MMAs (a wait,
        // an election, a commit: some 250 cycles) is then spread over eight MMAs of r / C columns, which by
        // themselves take 40-60 cycles each (measured: one per stage 21.9, two 20.2, three 22.0 us on 3072 -> 768)
        int G1 = g_tune_G1 ? g_tune_G1 : 2;
        if (G1 > 4) G1 = 4;
        if (G1 > kb1) G1 = kb1;
        while (!g_tune_G1 && G1 > 1 && ring1 < 2 * (int64_t)G1 * kb1_bytes) --G1;   // a wide T buffer leaves room for single k-blocks only
        if (ring1 < 2 * (int64_t)G1 * kb1_bytes) continue;
        int S1 = (int)(ring1 / ((int64_t)G1 * kb1_bytes)), S2 = (int)(ring2 / (int64_t)kb2_bytes);
        if (S1 > kMaxStages) S1 = kMaxStages;
        if (S2 > kMaxStages) S2 = kMaxStages;
        const uint32_t s1b = (uint32_t)G1 * kb1_bytes;
        const uint32_t used1 = (uint32_t)S1 * s1b, used2 = kStagingBytes + (uint32_t)S2 * kb2_bytes;
        const uint32_t after1 = (uint32_t)t_bytes + used2;
        Plan pl{C, RS, swb, BN2, G1, S1, S2, s1b, kb2_bytes, (uint32_t)t_bytes, 1024u + (used1 > after1 ? used1 : after1)};
        // prefer the largest cluster whose blocks are all resident at once (within this launch's share of the
        // SMs, when it runs beside other launches); else the smallest feasible
        if (!found) { best = pl; found = true; }
        const int64_t room = a.sm_share > 0 && !g_tune_C ? (int64_t)a.sm_share / C : (int64_t)max_active_clusters(C);
        if (tiles <= room && tiles <= max_active_clusters(C)) { best = pl; break; }
        best = pl;
    }
    if (!found) return false;
    *out = best;
    return true;
}

}  // namespace

void chain_tuning(int C, int G1, int BN2) {
    g_tune_C = C;
    g_tune_G1 = G1;
    g_tune_BN2 = BN2;
}

bool chain_eligible(const ChainArgs& a) {
    Plan pl;
    return make_plan(a, &pl);
}

// The fused kernel loses to two separate products where the T buffer (128 rows x r) leaves room for only two
// Q tiles of phase 2 in flight, i.e. at r = 512 (measured at 8192 tokens: 1024 -> 4096 forward 65 us fused against 49 us on two
// persistent products, 4096 -> 1024 99 against 46 us; at r <= 384 the chain wins everywhere measured).  The
// automatic path then takes the separate products; LRD_PATH_FUSED still forces the chain.
bool chain_preferred(const ChainArgs& a) {
    Plan pl;
    if (!make_plan(a, &pl)) return false;
    return pl.S2 >= 3;                 // Q tiles of phase 2 in flight
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
    p.G1 = pl.G1; p.S1 = pl.S1; p.S2 = pl.S2;
    p.stage1_bytes = pl.stage1_bytes; p.stage2_bytes = pl.stage2_bytes; p.t_bytes = pl.t_bytes;
    p.taw = pl.swb / 2;
    p.t_steps_lg = p.taw == 64 ? 2 : (p.taw == 32 ? 1 : 0);
    p.bias = (const __nv_bfloat16*)a.bias;
    p.has_tsave = a.T_save ? 1 : 0;
    // A block sends its slice of T to the peers c + 1, c + 2, ... in turn, so slice j reaches block c as the
    // ((c - j) mod C)-th arrival (0 = its own); phase 2 takes the k-blocks in the order in which the last slice
    // they touch arrives.  The order depends on the launch shape only, so results stay reproducible.
    for (int c = 0; c < kMaxCluster; ++c) {
        p.kb_order[c] = 0; p.kb_slices[c] = 0;
        if (c >= p.C) continue;
        int n = 0;
        for (int rank = 0; rank < p.C; ++rank)
            for (int kb = 0; kb < p.kb2; ++kb) {
                const int nks = std::min(4, p.ks2 - kb * 4);
                const int j_lo = kb * 64 / p.RS, j_hi = (kb * 64 + nks * 16 - 1) / p.RS;
                int worst = 0;
                uint32_t mask = 0;
                for (int j = j_lo; j <= j_hi; ++j) {
                    worst = std::max(worst, (c - j + p.C) % p.C);
                    mask |= 1u << j;
                }
                if (worst != rank) continue;
                p.kb_order[c] |= (uint32_t)kb << (4 * n);
                p.kb_slices[c] |= mask << (4 * n);
                ++n;
            }
    }
    p.timeout_flag = device_timeout_flag();

    static bool configured_on[kMaxDevices] = {};
    bool& configured = configured_on[device_slot()];
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
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)pl.C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // the kernel waits (griddepcontrol.wait) before it touches global memory
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, chain_kernel, tIn, tP, tQ, tOut, tT, p) != cudaSuccess) return LRD_ERR_CUDA;
    count_launch();
    return LRD_OK;
}

}  // namespace lrd
