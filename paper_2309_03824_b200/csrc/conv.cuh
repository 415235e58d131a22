// Tucker-2 decomposed 3x3 convolution: composition of 1x1 products and the r1 -> r2 core.
#pragma once
#include "common.cuh"

namespace lrd {

lrd_status_t tucker2_check(const lrd_tucker2_desc_t* d, lrd_tucker_freeze_t freeze);
size_t tucker2_workspace_bytes(const lrd_tucker2_desc_t* d, lrd_tucker_freeze_t freeze, int is_bwd);
lrd_status_t tucker2_fwd(const lrd_tucker2_desc_t* d, const void* X, const void* A, const void* G, const void* Bm,
                         const void* bias, void* Y, void* Z1_save, void* Z2_save, lrd_tucker_freeze_t freeze,
                         void* ws, size_t ws_bytes, int path, cudaStream_t s);
lrd_status_t tucker2_bwd(const lrd_tucker2_desc_t* d, const void* dY, const void* X, const void* A, const void* G,
                         const void* Bm, const void* Z1_save, const void* Z2_save, void* dX, void* dA, void* dG,
                         void* dB, void* dbias, lrd_tucker_freeze_t freeze, void* ws, size_t ws_bytes, int path,
                         cudaStream_t s);

// Whether the independent launches of tucker2_bwd run side by side on library-owned streams (default) or one
// after the other on the caller's stream.
void tucker2_overlap(bool on);

// Geometry of the k x k core: input H x W, output Ho x Wo = ((H - 1) / stride + 1) x ((W - 1) / stride + 1),
// zero pad (k - 1) / 2.
struct ConvGeom {
    int H, W, Ho, Wo, k, stride, pad;
};
inline ConvGeom conv_geom(int64_t H, int64_t W, int64_t k, int64_t stride) {
    return ConvGeom{(int)H, (int)W, (int)((H - 1) / stride + 1), (int)((W - 1) / stride + 1), (int)k, (int)stride, (int)((k - 1) / 2)};
}

// General-path k x k core, NHWC, any channel counts, any geometry above.  With p an output pixel and
// p * stride + (kh, kw) - pad the input pixel its tap (kh, kw) looks at:
//   fwd:        out[p][o] = sum_{kh,kw,i} in[p * stride + (kh, kw) - pad][i] G[o][kh][kw][i]
//   bwd_data:   din[q][i] = sum over (p, kh, kw) with p * stride + (kh, kw) - pad = q, and o, of dout[p][o] G[o][kh][kw][i]
//   bwd_filter: dG[o][kh][kw][i] = sum_p dout[p][o] in[p * stride + (kh, kw) - pad][i]
lrd_status_t simt_conv_fwd(const void* in, const void* G, void* out, int64_t B, const ConvGeom& g, int64_t ci, int64_t co,
                           lrd_dtype_t dt, cudaStream_t s);
lrd_status_t simt_conv_bwd_data(const void* dout, const void* G, void* din, int64_t B, const ConvGeom& g, int64_t ci,
                                int64_t co, lrd_dtype_t dt, cudaStream_t s);
lrd_status_t simt_conv_bwd_filter(const void* dout, const void* in, void* dG, int64_t B, const ConvGeom& g, int64_t ci,
                                  int64_t co, lrd_dtype_t dt, cudaStream_t s);

// Tensor-core 3x3 core (bf16, W <= 128, channel counts multiples of 8, 16-byte aligned bases).
bool tc_conv_eligible(int64_t B, int64_t H, int64_t W, int64_t ci, int64_t co, lrd_dtype_t dt, const void* p0,
                      const void* p1, const void* p2);
size_t tc_conv_filter_scratch_bytes(int64_t B, int64_t H, int64_t W, int64_t ci, int64_t co);
lrd_status_t tc_conv3x3(bool dgrad, const void* img, const void* G, void* out, int64_t B, int64_t H, int64_t W, int64_t ci,
                        int64_t co, cudaStream_t s);
// The core followed by the 1x1 product that consumes it, in one launch (the core's result stays on chip unless
// core_out asks for it): forward (dgrad = false) out2 = conv(img, G) Q^T + bias2 with Q = Bm [S x r2]; backward
// (dgrad = true) out2 = conv^T(img, G) Q^T with Q = A [C x r1].  n2 = rows of Q = columns of out2 (<= 256).
bool tc_conv_chain_eligible(bool dgrad, int64_t B, int64_t H, int64_t W, int64_t ci, int64_t co, int64_t n2, lrd_dtype_t dt,
                            const void* img, const void* G, const void* Q, const void* out2, const void* core_out);
lrd_status_t tc_conv3x3_chain(bool dgrad, const void* img, const void* G, const void* Q, const void* bias2, void* out2,
                              void* core_out, int64_t B, int64_t H, int64_t W, int64_t ci, int64_t co, int64_t n2,
                              cudaStream_t s);
lrd_status_t tc_conv3x3_filter(const void* dout, const void* in, void* dG, int64_t B, int64_t H, int64_t W, int64_t ci,
                               int64_t co, float* scratch, size_t scratch_bytes, cudaStream_t s);

// A whole data pass of the layer in one launch (3 x 3 core, stride 1; ranks <= 128 and multiples of 16, at most 256 output
// channels, images at most 40 pixels wide): forward (dgrad = false) out3 = conv(in P1, G) P3^T + bias3 with P1 = A [C x r1],
// P3 = Bm [S x r2]; backward (dgrad = true) out3 = conv^T(in P1, G) P3^T with in = dY, P1 = Bm [S x r2], P3 = A [C x r1].
// c_in = channels of `in`, nA = columns of P1, nB = channels after the core, n3 = rows of P3 = columns of out3.  save1
// [pixels x nA] / save2 [pixels x nB] (nullable) receive the two intermediates where the caller needs them later.
bool tucker_fused_eligible(int64_t B, int64_t H, int64_t W, int64_t c_in, int64_t nA, int64_t nB, int64_t n3, lrd_dtype_t dt,
                           const void* in, const void* P1, const void* G, const void* P3, const void* out3, const void* save1,
                           const void* save2);
lrd_status_t tucker_fused(bool dgrad, const void* in, const void* P1, const void* G, const void* P3, const void* bias3, void* out3,
                          void* save1, void* save2, int64_t B, int64_t H, int64_t W, int64_t c_in, int64_t nA, int64_t nB,
                          int64_t n3, cudaStream_t s);

// Path dispatch for the 3x3, stride-1 core (tensor-core kernel where the shape qualifies, else general).
lrd_status_t conv3x3_fwd(const void* in, const void* G, void* out, int64_t B, int64_t H, int64_t W, int64_t ci,
                         int64_t co, lrd_dtype_t dt, int path, cudaStream_t s);
lrd_status_t conv3x3_bwd_data(const void* dout, const void* G, void* din, int64_t B, int64_t H, int64_t W, int64_t ci,
                              int64_t co, lrd_dtype_t dt, int path, cudaStream_t s);
lrd_status_t conv3x3_bwd_filter(const void* dout, const void* in, void* dG, int64_t B, int64_t H, int64_t W,
                                int64_t ci, int64_t co, lrd_dtype_t dt, int path, float* scratch, size_t scratch_bytes,
                                cudaStream_t s);

}  // namespace lrd
