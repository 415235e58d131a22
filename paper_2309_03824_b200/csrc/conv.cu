// Tucker-2 decomposed k x k convolution (NHWC): 1x1 product, k x k core (which carries the layer's stride), 1x1
// product, and the backward pass through them under a freeze mask.  The 3 x 3, stride-1 core runs on the
// tensor-core kernels where the shape allows; every other geometry runs the core on the general kernels.
#include "conv.cuh"

#include "streams.cuh"
#include "tc.cuh"

namespace lrd {
namespace {

struct Tk {
    int64_t B, H, W, C, S, r1, r2;
    int64_t P;              // input pixels B H W (rows of X, Z1, dZ1, dX)
    int64_t Po;             // output pixels B Ho Wo (rows of Z2, Y, dY, dZ2)
    int64_t taps;           // k * k
    ConvGeom g;
    bool plain;             // 3 x 3, stride 1: the geometry the tensor-core core kernels take
    lrd_dtype_t dt;
};

Tk parse(const lrd_tucker2_desc_t* d) {
    Tk t;
    t.B = d->B; t.H = d->H; t.W = d->W; t.C = d->C; t.S = d->S; t.r1 = d->r1; t.r2 = d->r2;
    t.g = conv_geom(d->H, d->W, d->k, d->stride);
    t.P = d->B * d->H * d->W;
    t.Po = d->B * t.g.Ho * t.g.Wo;
    t.taps = d->k * d->k;
    t.plain = d->k == 3 && d->stride == 1;
    t.dt = (lrd_dtype_t)d->dtype;
    return t;
}

size_t act_bytes(const Tk& t, int64_t pixels, int64_t ch) { return align_up((size_t)(pixels > 0 ? pixels : 1) * ch * elem_size(t.dt), 256); }

// Scratch of the three weight-gradient launches of the backward pass, one region each: they may run side by side.
struct Scratch { size_t dB, dA, filter; };

Scratch split_regions(const Tk& t) {
    Scratch r{0, 0, 0};
    if (t.P < 1) return r;
    r.dB = colsum_scratch_bytes(t.Po, t.S);
    if (t.dt == LRD_BF16) {
        const size_t a = tc_split_workspace_bytes(t.S, t.r2, t.Po);
        r.dB = r.dB > a ? r.dB : a;
        r.dA = tc_split_workspace_bytes(t.C, t.r1, t.P);
        if (t.plain) r.filter = tc_conv_filter_scratch_bytes(t.B, t.H, t.W, t.r1, t.r2);
    }
    r.dB = align_up(r.dB, 256); r.dA = align_up(r.dA, 256); r.filter = align_up(r.filter, 256);
    return r;
}

size_t split_bytes(const Tk& t) {
    const Scratch r = split_regions(t);
    return r.dB + r.dA + r.filter;
}

bool g_tucker_overlap = true;

// Ranks that are not multiples of 8 (rows of A, Bm, G, Z1, Z2 then start off 16-byte boundaries): as for the linear
// layer, the factors -- small -- are copied into the workspace with the ranks rounded up to multiples of 16 and
// zeros in the padding, the layer runs on the tensor-core kernels at the padded ranks, and Z1 / Z2 / dA / dG / dB
// are copied between the caller's packed layout and padded buffers.
bool needs_repack(const Tk& t) { return t.plain && t.dt == LRD_BF16 && (t.r1 % 8 || t.r2 % 8) && t.C % 8 == 0 && t.S % 8 == 0; }
int64_t pad16(int64_t r) { return (r + 15) / 16 * 16; }
lrd_tucker2_desc_t padded_desc(const lrd_tucker2_desc_t& d) {
    lrd_tucker2_desc_t q = d;
    q.r1 = pad16(d.r1); q.r2 = pad16(d.r2);
    return q;
}
struct Repack { size_t A, G, Bm, Z1, Z2, dA, dG, dB, total; };
Repack repack_layout(const Tk& t, size_t inner) {
    const size_t r1 = (size_t)pad16(t.r1), r2 = (size_t)pad16(t.r2), P = (size_t)(t.P > 0 ? t.P : 1), e = 2;
    Repack o;
    size_t at = align_up(inner, 256);
    auto take = [&at](size_t bytes) { const size_t here = at; at += align_up(bytes, 256); return here; };
    o.A = take((size_t)t.C * r1 * e); o.G = take(r2 * 9 * r1 * e); o.Bm = take((size_t)t.S * r2 * e);
    o.Z1 = take(P * r1 * e); o.Z2 = take(P * r2 * e);
    o.dA = take((size_t)t.C * r1 * e); o.dG = take(r2 * 9 * r1 * e); o.dB = take((size_t)t.S * r2 * e);
    o.total = at;
    return o;
}

#define LRD_TRY(expr)                          \
    do {                                       \
        lrd_status_t st__ = (expr);            \
        if (st__ != LRD_OK) return st__;       \
    } while (0)

}  // namespace

lrd_status_t tucker2_check(const lrd_tucker2_desc_t* d, lrd_tucker_freeze_t freeze) {
    if (!d) return LRD_ERR_INVALID_ARG;
    if (freeze != LRD_TK_FREEZE_NONE && freeze != LRD_TK_FREEZE_FACTORS && freeze != LRD_TK_FREEZE_CORE)
        return LRD_ERR_INVALID_ARG;
    if (d->B < 0 || d->H < 1 || d->W < 1 || d->C < 1 || d->S < 1) return LRD_ERR_INVALID_ARG;
    if (d->dtype != LRD_F32 && d->dtype != LRD_BF16) return LRD_ERR_INVALID_ARG;
    if (d->r1 < 1 || d->r2 < 1 || d->r1 > d->C || d->r2 > d->S) return LRD_ERR_BAD_RANK;
    if (d->k < 1 || d->stride < 1 || d->pad < 0) return LRD_ERR_INVALID_ARG;
    if (d->k > 7 || d->k % 2 == 0 || d->stride > 2 || d->pad != (d->k - 1) / 2) return LRD_ERR_UNSUPPORTED;
    if (d->H > 32767 || d->W > 32767) return LRD_ERR_UNSUPPORTED;
    return LRD_OK;
}

size_t tucker2_workspace_bytes(const lrd_tucker2_desc_t* d, lrd_tucker_freeze_t freeze, int is_bwd) {
    if (tucker2_check(d, freeze) != LRD_OK) return 0;
    const Tk t = parse(d);
    if (needs_repack(t)) {
        const lrd_tucker2_desc_t q = padded_desc(*d);
        return repack_layout(t, tucker2_workspace_bytes(&q, freeze, is_bwd)).total;
    }
    return act_bytes(t, t.P, t.r1) + act_bytes(t, t.Po, t.r2) + (is_bwd ? split_bytes(t) : 0);
}

lrd_status_t tucker2_fwd(const lrd_tucker2_desc_t* d, const void* X, const void* A, const void* G, const void* Bm,
                         const void* bias, void* Y, void* Z1_save, void* Z2_save, lrd_tucker_freeze_t freeze,
                         void* ws, size_t ws_bytes, int path, cudaStream_t s) {
    (void)ws_bytes;
    const Tk t = parse(d);
    if (t.P == 0) return LRD_OK;
    if (needs_repack(t) && path != LRD_PATH_GENERAL) {
        const lrd_tucker2_desc_t q = padded_desc(*d);
        const size_t inner = tucker2_workspace_bytes(&q, freeze, 0);
        const Repack o = repack_layout(t, inner);
        uint8_t* w = (uint8_t*)ws;
        LRD_TRY(copy2d_bf16(w + o.A, q.r1, A, t.r1, t.C, t.r1, q.r1, s));
        LRD_TRY(copy2d_bf16(w + o.G, q.r1, G, t.r1, t.r2 * 9, t.r1, q.r1, s));
        LRD_TRY(zero_fill(w + o.G + (size_t)t.r2 * 9 * q.r1 * 2, (q.r2 - t.r2) * 9, q.r1, q.r1, LRD_BF16, s));
        LRD_TRY(copy2d_bf16(w + o.Bm, q.r2, Bm, t.r2, t.S, t.r2, q.r2, s));
        LRD_TRY(tucker2_fwd(&q, X, w + o.A, w + o.G, w + o.Bm, bias, Y, Z1_save ? w + o.Z1 : nullptr, Z2_save ? w + o.Z2 : nullptr, freeze,
                            w, inner, path, s));
        if (Z1_save) LRD_TRY(copy2d_bf16(Z1_save, t.r1, w + o.Z1, q.r1, t.P, q.r1, t.r1, s));
        if (Z2_save) LRD_TRY(copy2d_bf16(Z2_save, t.r2, w + o.Z2, q.r2, t.Po, q.r2, t.r2, s));
        return LRD_OK;
    }
    // the whole forward in one launch where the shape allows: Z1 and Z2 stay on chip unless the caller saves them
    if (t.plain && (path == LRD_PATH_AUTO || path == LRD_PATH_FUSED) && (!bias || ((uintptr_t)bias % 2) == 0) &&
        tucker_fused_eligible(t.B, t.H, t.W, t.C, t.r1, t.r2, t.S, t.dt, X, A, G, Bm, Y, Z1_save, Z2_save))
        return tucker_fused(false, X, A, G, Bm, bias, Y, Z1_save, Z2_save, t.B, t.H, t.W, t.C, t.r1, t.r2, t.S, s);
    void* Z1 = Z1_save ? Z1_save : ws;
    void* Z2 = Z2_save ? Z2_save : (void*)((uint8_t*)ws + act_bytes(t, t.P, t.r1));
    LRD_TRY(run_gemm(make_gemm(t.P, t.r1, t.C, X, t.C, false, A, t.r1, true, Z1, t.r1, nullptr, t.dt), path, false, nullptr, 0, s));
    // core + last 1x1 in one launch where the shape allows: Z2 then stays on chip unless the caller saves it
    if (t.plain && (path == LRD_PATH_AUTO || path == LRD_PATH_FUSED) &&
        tc_conv_chain_eligible(false, t.B, t.H, t.W, t.r1, t.r2, t.S, t.dt, Z1, G, Bm, Y, Z2_save) &&
        (!bias || ((uintptr_t)bias % 2) == 0))
        return tc_conv3x3_chain(false, Z1, G, Bm, bias, Y, Z2_save, t.B, t.H, t.W, t.r1, t.r2, t.S, s);
    if (t.plain) LRD_TRY(conv3x3_fwd(Z1, G, Z2, t.B, t.H, t.W, t.r1, t.r2, t.dt, path, s));
    else LRD_TRY(simt_conv_fwd(Z1, G, Z2, t.B, t.g, t.r1, t.r2, t.dt, s));
    return run_gemm(make_gemm(t.Po, t.S, t.r2, Z2, t.r2, false, Bm, t.r2, false, Y, t.S, bias, t.dt), path, false, nullptr, 0, s);
}

lrd_status_t tucker2_bwd(const lrd_tucker2_desc_t* d, const void* dY, const void* X, const void* A, const void* G,
                         const void* Bm, const void* Z1_save, const void* Z2_save, void* dX, void* dA, void* dG,
                         void* dB, void* dbias, lrd_tucker_freeze_t freeze, void* ws, size_t ws_bytes, int path,
                         cudaStream_t s) {
    const Tk t = parse(d);
    const bool factors = freeze != LRD_TK_FREEZE_FACTORS, core = freeze != LRD_TK_FREEZE_CORE;
    // frozen group: no product is launched; gradient buffers the caller passed read as zero
    if (!factors || t.P == 0) {
        LRD_TRY(zero_fill(dA, t.C, t.r1, t.r1, t.dt, s));
        LRD_TRY(zero_fill(dB, t.S, t.r2, t.r2, t.dt, s));
        LRD_TRY(zero_fill(dbias, 1, t.S, t.S, t.dt, s));
    }
    if (!core || t.P == 0) LRD_TRY(zero_fill(dG, t.r2, t.taps * t.r1, t.taps * t.r1, t.dt, s));
    if (t.P == 0) return LRD_OK;
    if (needs_repack(t) && path != LRD_PATH_GENERAL) {
        const lrd_tucker2_desc_t q = padded_desc(*d);
        const size_t inner = tucker2_workspace_bytes(&q, freeze, 1);
        const Repack o = repack_layout(t, inner);
        uint8_t* w = (uint8_t*)ws;
        LRD_TRY(copy2d_bf16(w + o.A, q.r1, A, t.r1, t.C, t.r1, q.r1, s));
        LRD_TRY(copy2d_bf16(w + o.G, q.r1, G, t.r1, t.r2 * 9, t.r1, q.r1, s));
        LRD_TRY(zero_fill(w + o.G + (size_t)t.r2 * 9 * q.r1 * 2, (q.r2 - t.r2) * 9, q.r1, q.r1, LRD_BF16, s));
        LRD_TRY(copy2d_bf16(w + o.Bm, q.r2, Bm, t.r2, t.S, t.r2, q.r2, s));
        if (core) LRD_TRY(copy2d_bf16(w + o.Z1, q.r1, Z1_save, t.r1, t.P, t.r1, q.r1, s));
        if (factors) LRD_TRY(copy2d_bf16(w + o.Z2, q.r2, Z2_save, t.r2, t.Po, t.r2, q.r2, s));
        // the frozen group's buffers were zero-filled above; the padded call gets none for them
        LRD_TRY(tucker2_bwd(&q, dY, X, w + o.A, w + o.G, w + o.Bm, core ? w + o.Z1 : nullptr, factors ? w + o.Z2 : nullptr, dX,
                            factors ? w + o.dA : nullptr, core ? w + o.dG : nullptr, factors ? w + o.dB : nullptr, factors ? dbias : nullptr,
                            freeze, w, inner, path, s));
        if (factors) {
            LRD_TRY(copy2d_bf16(dA, t.r1, w + o.dA, q.r1, t.C, q.r1, t.r1, s));
            LRD_TRY(copy2d_bf16(dB, t.r2, w + o.dB, q.r2, t.S, q.r2, t.r2, s));
        }
        if (core) LRD_TRY(copy2d_bf16(dG, t.r1, w + o.dG, q.r1, t.r2 * 9, q.r1, t.r1, s));
        return LRD_OK;
    }

    void* dZ1 = ws;
    void* dZ2 = (uint8_t*)ws + act_bytes(t, t.P, t.r1);
    const Scratch reg = split_regions(t);
    uint8_t* scratch0 = (uint8_t*)ws + act_bytes(t, t.P, t.r1) + act_bytes(t, t.Po, t.r2);
    float* pB = (float*)scratch0;
    float* pA = (float*)(scratch0 + reg.dB);
    float* pF = (float*)(scratch0 + reg.dB + reg.dA);
    (void)ws_bytes;

    // What depends on what: dZ2 = dY Bm first; the transposed core (+ dX) and the filter gradient both need dZ2 and
    // nothing of each other; dB (+ db) needs only dY and Z2_save; dA needs the dZ1 the transposed core writes.  Every
    // launch here is a few microseconds of latency around little work, so the independent ones run side by side:
    // dB from the start and the filter gradient after dZ2 on library-owned streams, the data path and dA on the
    // caller's stream, which waits for the other two before this function returns.
    SideStreams* ss = g_tucker_overlap && (factors || core) ? side_streams() : nullptr;
    cudaStream_t sB = ss && factors ? ss->aux[0] : s, sF = ss && core ? ss->aux[1] : s;
    lrd_status_t st = LRD_OK;
    auto keep = [&st](lrd_status_t x) { if (st == LRD_OK) st = x; };
    if (sB != s) {
        if (!stream_after(sB, s, ss->fork)) return LRD_ERR_CUDA;
    }
    auto launch_dB = [&]() {
        GemmArgs gb = make_gemm(t.S, t.r2, t.Po, dY, t.S, true, Z2_save, t.r2, true, dB, t.r2, nullptr, t.dt);
        bool db_done = false;
        if (dbias && path != LRD_PATH_GENERAL) {          // the bias gradient rides on the dB product (A = dY)
            gb.a_colsum = dbias;
            if (tc_gemm_colsum_ok(gb)) db_done = true; else gb.a_colsum = nullptr;
        }
        keep(run_gemm(gb, path, true, pB, reg.dB, sB));
        if (dbias && !db_done) keep(colsum(dY, t.S, t.Po, t.S, dbias, t.dt, pB, reg.dB, sB));
    };
    if (factors && sB != s) launch_dB();

    auto launch_filter = [&](cudaStream_t st_f) {
        if (t.plain) keep(conv3x3_bwd_filter(dZ2, Z1_save, dG, t.B, t.H, t.W, t.r1, t.r2, t.dt, path, pF, reg.filter, st_f));
        else keep(simt_conv_bwd_filter(dZ2, Z1_save, dG, t.B, t.g, t.r1, t.r2, t.dt, st_f));
    };
    // the whole data path (dZ2 = dY Bm, transposed core, dX = dZ1 A^T) in one launch where the shape allows; dZ2 is
    // written only for the filter gradient, dZ1 only for dA.  (Giving the filter gradient a dZ2 product of its own
    // beside the pass, so that it need not wait for it, was slower: 44.5 against 41.2 us per step with the core
    // unfrozen -- the extra launch takes SMs from the pass.)
    const bool one_launch = dX && t.plain && (path == LRD_PATH_AUTO || path == LRD_PATH_FUSED) &&
                            tucker_fused_eligible(t.B, t.H, t.W, t.S, t.r2, t.r1, t.C, t.dt, dY, Bm, G, A, dX, core ? dZ2 : nullptr,
                                                  factors ? dZ1 : nullptr);
    if (one_launch)
        keep(tucker_fused(true, dY, Bm, G, A, nullptr, dX, core ? dZ2 : nullptr, factors ? dZ1 : nullptr, t.B, t.H, t.W, t.S, t.r2,
                          t.r1, t.C, s));
    else
        keep(run_gemm(make_gemm(t.Po, t.r2, t.S, dY, t.S, false, Bm, t.r2, true, dZ2, t.r2, nullptr, t.dt), path, false, nullptr, 0, s));
    if (core && sF != s) {
        if (!stream_after(sF, s, ss->mid)) keep(LRD_ERR_CUDA);
        else launch_filter(sF);
    }
    // transposed core + first 1x1 (dX = dZ1 A^T) in one launch where the shape allows; dZ1 is written only for dA
    const bool fuse_dx = !one_launch && dX && t.plain && (path == LRD_PATH_AUTO || path == LRD_PATH_FUSED) &&
                         tc_conv_chain_eligible(true, t.B, t.H, t.W, t.r1, t.r2, t.C, t.dt, dZ2, G, A, dX, factors ? dZ1 : nullptr);
    if (one_launch) {
    } else if (fuse_dx) keep(tc_conv3x3_chain(true, dZ2, G, A, nullptr, dX, factors ? dZ1 : nullptr, t.B, t.H, t.W, t.r1, t.r2, t.C, s));
    else if ((dX || factors) && t.plain) keep(conv3x3_bwd_data(dZ2, G, dZ1, t.B, t.H, t.W, t.r1, t.r2, t.dt, path, s));
    else if (dX || factors) keep(simt_conv_bwd_data(dZ2, G, dZ1, t.B, t.g, t.r1, t.r2, t.dt, s));
    if (dX && !fuse_dx && !one_launch) keep(run_gemm(make_gemm(t.P, t.C, t.r1, dZ1, t.r1, false, A, t.r1, false, dX, t.C, nullptr, t.dt), path, false, nullptr, 0, s));
    if (factors) {
        if (sB == s) launch_dB();
        keep(run_gemm(make_gemm(t.C, t.r1, t.P, X, t.C, true, dZ1, t.r1, true, dA, t.r1, nullptr, t.dt), path, true, pA, reg.dA, s));
    }
    if (core && sF == s) launch_filter(s);
    // join even after a failed launch, so that a capture in progress is left whole
    if (sB != s && !stream_after(s, sB, ss->aux_done[0])) keep(LRD_ERR_CUDA);
    if (sF != s && !stream_after(s, sF, ss->aux_done[1])) keep(LRD_ERR_CUDA);
    return st;
}

void tucker2_overlap(bool on) { g_tucker_overlap = on; }

// Core convolution dispatch: tensor-core implicit GEMM where the geometry qualifies, else the general kernels.
lrd_status_t conv3x3_fwd(const void* in, const void* G, void* out, int64_t B, int64_t H, int64_t W, int64_t ci,
                         int64_t co, lrd_dtype_t dt, int path, cudaStream_t s) {
    if (path != LRD_PATH_GENERAL && tc_conv_eligible(B, H, W, ci, co, dt, in, G, out))
        return tc_conv3x3(false, in, G, out, B, H, W, ci, co, s);
    return simt_conv_fwd(in, G, out, B, conv_geom(H, W, 3, 1), ci, co, dt, s);
}
lrd_status_t conv3x3_bwd_data(const void* dout, const void* G, void* din, int64_t B, int64_t H, int64_t W, int64_t ci,
                              int64_t co, lrd_dtype_t dt, int path, cudaStream_t s) {
    if (path != LRD_PATH_GENERAL && tc_conv_eligible(B, H, W, ci, co, dt, dout, G, din))
        return tc_conv3x3(true, dout, G, din, B, H, W, ci, co, s);
    return simt_conv_bwd_data(dout, G, din, B, conv_geom(H, W, 3, 1), ci, co, dt, s);
}
lrd_status_t conv3x3_bwd_filter(const void* dout, const void* in, void* dG, int64_t B, int64_t H, int64_t W,
                                int64_t ci, int64_t co, lrd_dtype_t dt, int path, float* scratch, size_t scratch_bytes,
                                cudaStream_t s) {
    if (path != LRD_PATH_GENERAL && tc_conv_eligible(B, H, W, ci, co, dt, dout, in, dG) &&
        scratch_bytes >= tc_conv_filter_scratch_bytes(B, H, W, ci, co))
        return tc_conv3x3_filter(dout, in, dG, B, H, W, ci, co, scratch, scratch_bytes, s);
    return simt_conv_bwd_filter(dout, in, dG, B, conv_geom(H, W, 3, 1), ci, co, dt, s);
}

}  // namespace lrd
