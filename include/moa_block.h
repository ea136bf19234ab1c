/*
 * moa_block.h -- C ABI of the token-wise pieces of the transformer block for NVIDIA B200
 * (sm_100a): RMSNorm and the gated MLP, each forward and backward, and the GEMM of the projections.
 *
 * These are the pieces the paper's block section puts around attention ("RMSNorm, gated MLP",
 * hidden width d_ff, with the gated-MLP backward the dominant kernel of its block profile).
 * The paper names them and counts the block's traffic but prints no formula for either; the
 * definitions taken here are the usual ones and are stated with each call.
 *
 * Conventions (the same as moa_attn.h): every tensor argument is a DEVICE pointer to a
 * contiguous row-major array, 16-byte aligned; the caller owns every buffer, workspace
 * included; calls enqueue kernels on `stream` (a cudaStream_t passed as void*) and return
 * without synchronising; outputs are overwritten; errors come back only as moa_status and
 * nothing has been enqueued when one is returned.  bf16 storage, fp32 arithmetic.
 */
#ifndef MOA_BLOCK_H
#define MOA_BLOCK_H

#include "moa_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/* ------------------------------------------------------------------------- RMSNorm
 *   r_i  = 1 / sqrt( (1/d) sum_k x_ik^2 + eps )          y_ik = x_ik r_i g_k
 *   dg_k = sum_i dy_ik x_ik r_i
 *   dx_ik = r_i g_k dy_ik - x_ik r_i^3 (1/d) sum_m x_im g_m dy_im
 * x, y, dy, dx: [n,d]; g, dg: [d]; r: [n] fp32.  n >= 1; d a multiple of 8, 8 <= d <= 8192;
 * dtype MOA_BF16 (others: MOA_ERR_UNSUPPORTED).  HBM-bound: the forward reads x and writes y
 * once, the backward reads x and dy and writes dx once. */
typedef struct {
    int32_t n, d;
    float   eps;
    int32_t dtype;       /* moa_dtype of x, g, y, dy, dx, dg */
} moa_rmsnorm_desc;

/* Workspace of the backward: per-CTA partial sums of dg, reduced in a fixed order (so the
 * result does not depend on timing).  0 for an invalid desc. */
size_t moa_rmsnorm_workspace_bytes(const moa_rmsnorm_desc *desc);

/* Reads x, g; writes y and, when r != NULL, r (which the backward wants). */
moa_status moa_rmsnorm_fwd(const moa_rmsnorm_desc *desc, const void *x, const void *g,
                           void *y, float *r, void *stream);

/* Reads x, g, dy and r (as written by the forward for the same x; NULL: recomputed from x);
 * writes dx and dg.  dx_add (NULL or [n,d]) is added to dx: the gradient that reaches x past the
 * norm, along a residual connection. */
moa_status moa_rmsnorm_bwd(const moa_rmsnorm_desc *desc, const void *x, const void *g, const float *r,
                           const void *dy, const void *dx_add, void *dx, void *dg,
                           void *ws, size_t ws_bytes, void *stream);

/* ----------------------------------------------------------------------- gated MLP
 * SiLU-gated MLP without biases, weights stored [out, in]:
 *   a = x W1^T, u = x W3^T   [n,d_ff]      h = silu(a) * u,  silu(a) = a / (1 + exp(-a))
 *   y = h W2^T               [n,d]
 *   dh = dy W2,  da = dh u s (1 + a (1 - s)) with s = 1/(1+exp(-a)),  du = dh a s
 *   dW2 = dy^T h,  dW1 = da^T x,  dW3 = du^T x,  dx = da W1 + du W3
 * x, y, dy, dx: [n,d]; W1, W3, dW1, dW3: [d_ff,d]; W2, dW2: [d,d_ff]; a, u, h: [n,d_ff].
 * The contractions run on the tensor cores (tcgen05, fp32 accumulation in TMEM) with the
 * gate arithmetic fused into the epilogues of the GEMMs that produce a|u and dh, so dh is
 * never written to memory.  n >= 1; d and d_ff multiples of 8 (rows stay 16-byte aligned);
 * d_ff >= 8, d >= 8; dtype MOA_BF16. */
typedef struct {
    int32_t n, d, d_ff;
    int32_t dtype;
} moa_mlp_desc;

/* Forward.  Reads x, W1, W3, W2; writes a, u, h (kept for the backward, bf16) and y.  res (NULL or
 * [n,d]) is added to y in the epilogue of the last GEMM: the block's residual connection. */
moa_status moa_gated_mlp_fwd(const moa_mlp_desc *desc, const void *x, const void *W1, const void *W3,
                             const void *W2, const void *res, void *a, void *u, void *h, void *y, void *stream);

/* Workspace of the backward: da and du, [n,d_ff] each in the storage type.  0 for an invalid desc. */
size_t moa_gated_mlp_workspace_bytes(const moa_mlp_desc *desc);

/* Backward.  Reads x, the weights, a, u, h (as written by the forward) and dy; writes dx, dW1,
 * dW3, dW2.  Weight gradients are overwritten (not accumulated into). */
moa_status moa_gated_mlp_bwd(const moa_mlp_desc *desc, const void *x, const void *W1, const void *W3,
                             const void *W2, const void *a, const void *u, const void *h, const void *dy,
                             void *dx, void *dW1, void *dW3, void *dW2,
                             void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------------ GEMM
 * The product the block's projections and their backward passes need, on the same tensor-core
 * kernel as the gated MLP:   C[M,N] = A B^T (+ R)
 * A is given as [M,K] row-major (a_layout = 0) or as [K,M] row-major (a_layout = 1); B as [N,K]
 * row-major (b_layout = 0) or as [K,N] row-major (b_layout = 1); C and the optional R are [M,N].
 * With weights stored [out,in]:  y = x W^T is (0,0);  dx = dy W is (0,1);  dW = dy^T x is (1,1) with
 * M = out, N = in, K = tokens.  R (NULL or [M,N]) is added in the epilogue: a residual connection, or
 * the running sum of a chain of products.  M, N, K >= 1; the row length of every array a multiple of
 * 8 (rows stay 16-byte aligned); dtype MOA_BF16; fp32 accumulation.
 * Tiling: 256 x 256 tiles on pairs of CTAs (one cluster of two, UMMAs of M = 256 reading half of B from each CTA's
 * shared memory), or 128 x 256 output tiles on single CTAs where M is so small that pairs would need more waves.  The environment variable MOA_GEMM_PAIR, read once per process, overrides the choice for
 * tests and measurements: 0 = never pairs, 2 = always pairs; the results do not depend on it beyond rounding order
 * (they are the same bits: every output element is one fp32 accumulation over K in the same order). */
typedef struct {
    int32_t M, N, K;
    int32_t a_layout, b_layout;
    int32_t dtype;
} moa_gemm_desc;
moa_status moa_gemm(const moa_gemm_desc *desc, const void *A, const void *B, const void *R, void *C, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MOA_BLOCK_H */
