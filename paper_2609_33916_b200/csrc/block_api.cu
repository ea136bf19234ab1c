// C-ABI entry points of the block pieces (include/moa_block.h): argument checks and the sequence
// of kernel launches of each operation.  No arithmetic here.
#include "common.cuh"
#include "moa_block.h"

using namespace moa;

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool finite(float v) { return v == v && v - v == 0.f; }

moa_status check_rmsnorm(const moa_rmsnorm_desc *d)
{
    if (!d) return MOA_ERR_INVALID_ARG;
    if (d->n <= 0 || d->d <= 0) return MOA_ERR_INVALID_ARG;
    if (!finite(d->eps) || d->eps < 0.f) return MOA_ERR_INVALID_ARG;
    if (d->dtype != MOA_BF16 && d->dtype != MOA_F32) return MOA_ERR_INVALID_ARG;
    if (d->dtype != MOA_BF16) return MOA_ERR_UNSUPPORTED;
    if (d->d % 8 != 0 || d->d > 8192) return MOA_ERR_UNSUPPORTED;
    return MOA_OK;
}

moa_status check_mlp(const moa_mlp_desc *d)
{
    if (!d) return MOA_ERR_INVALID_ARG;
    if (d->n <= 0 || d->d <= 0 || d->d_ff <= 0) return MOA_ERR_INVALID_ARG;
    if (d->dtype != MOA_BF16 && d->dtype != MOA_F32) return MOA_ERR_INVALID_ARG;
    if (d->dtype != MOA_BF16) return MOA_ERR_UNSUPPORTED;
    if (d->d % 8 != 0 || d->d_ff % 8 != 0) return MOA_ERR_UNSUPPORTED;       // rows of every array stay 16-byte aligned
    if ((long long)d->n * d->d_ff >= (1LL << 40)) return MOA_ERR_UNSUPPORTED;
    return MOA_OK;
}

size_t mlp_half_ws(const moa_mlp_desc *d) { return ((size_t)d->n * d->d_ff * 2 + 255) / 256 * 256; }

}  // namespace

extern "C" {

size_t moa_rmsnorm_workspace_bytes(const moa_rmsnorm_desc *desc)
{
    if (check_rmsnorm(desc) != MOA_OK) return 0;
    return rmsnorm_workspace_bytes(desc->n, desc->d);
}

moa_status moa_rmsnorm_fwd(const moa_rmsnorm_desc *desc, const void *x, const void *g, void *y, float *r, void *stream)
{
    moa_status s = check_rmsnorm(desc);
    if (s != MOA_OK) return s;
    if (!x || !g || !y) return MOA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(g) || !aligned16(y) || (r && !aligned16(r))) return MOA_ERR_INVALID_ARG;
    if ((s = check_device_arch()) != MOA_OK) return s;
    return rmsnorm_fwd(desc->n, desc->d, desc->eps, x, g, y, r, (cudaStream_t)stream) == cudaSuccess ? MOA_OK : MOA_ERR_CUDA;
}

moa_status moa_rmsnorm_bwd(const moa_rmsnorm_desc *desc, const void *x, const void *g, const float *r,
                           const void *dy, const void *dx_add, void *dx, void *dg, void *ws, size_t ws_bytes, void *stream)
{
    moa_status s = check_rmsnorm(desc);
    if (s != MOA_OK) return s;
    if (!x || !g || !dy || !dx || !dg) return MOA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(g) || !aligned16(dy) || !aligned16(dx) || !aligned16(dg) || (r && !aligned16(r)) ||
        (dx_add && !aligned16(dx_add)))
        return MOA_ERR_INVALID_ARG;
    if (!ws || ws_bytes < rmsnorm_workspace_bytes(desc->n, desc->d)) return MOA_ERR_WORKSPACE;
    if (!aligned16(ws)) return MOA_ERR_INVALID_ARG;
    if ((s = check_device_arch()) != MOA_OK) return s;
    return rmsnorm_bwd(desc->n, desc->d, desc->eps, x, g, r, dy, dx_add, dx, dg, ws, (cudaStream_t)stream) == cudaSuccess
               ? MOA_OK : MOA_ERR_CUDA;
}

size_t moa_gated_mlp_workspace_bytes(const moa_mlp_desc *desc)
{
    if (check_mlp(desc) != MOA_OK) return 0;
    return 2 * mlp_half_ws(desc);
}

moa_status moa_gated_mlp_fwd(const moa_mlp_desc *desc, const void *x, const void *W1, const void *W3, const void *W2,
                             const void *res, void *a, void *u, void *h, void *y, void *stream)
{
    moa_status s = check_mlp(desc);
    if (s != MOA_OK) return s;
    if (!x || !W1 || !W3 || !W2 || !a || !u || !h || !y) return MOA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(W1) || !aligned16(W3) || !aligned16(W2) || !aligned16(a) || !aligned16(u) ||
        !aligned16(h) || !aligned16(y) || (res && !aligned16(res)))
        return MOA_ERR_INVALID_ARG;
    if ((s = check_device_arch()) != MOA_OK) return s;
    return gated_mlp_fwd(desc->n, desc->d, desc->d_ff, x, W1, W3, W2, res, a, u, h, y, (cudaStream_t)stream) == cudaSuccess
               ? MOA_OK : MOA_ERR_CUDA;
}

moa_status moa_gated_mlp_bwd(const moa_mlp_desc *desc, const void *x, const void *W1, const void *W3, const void *W2,
                             const void *a, const void *u, const void *h, const void *dy,
                             void *dx, void *dW1, void *dW3, void *dW2, void *ws, size_t ws_bytes, void *stream)
{
    moa_status s = check_mlp(desc);
    if (s != MOA_OK) return s;
    if (!x || !W1 || !W3 || !W2 || !a || !u || !h || !dy || !dx || !dW1 || !dW3 || !dW2) return MOA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(W1) || !aligned16(W3) || !aligned16(W2) || !aligned16(a) || !aligned16(u) ||
        !aligned16(h) || !aligned16(dy) || !aligned16(dx) || !aligned16(dW1) || !aligned16(dW3) || !aligned16(dW2))
        return MOA_ERR_INVALID_ARG;
    if (!ws || ws_bytes < 2 * mlp_half_ws(desc)) return MOA_ERR_WORKSPACE;
    if (!aligned16(ws)) return MOA_ERR_INVALID_ARG;
    if ((s = check_device_arch()) != MOA_OK) return s;
    void *da = ws, *du = (char *)ws + mlp_half_ws(desc);
    return gated_mlp_bwd(desc->n, desc->d, desc->d_ff, x, W1, W3, W2, a, u, h, dy, da, du, dx, dW1, dW3, dW2,
                         (cudaStream_t)stream) == cudaSuccess ? MOA_OK : MOA_ERR_CUDA;
}

moa_status moa_gemm(const moa_gemm_desc *desc, const void *A, const void *B, const void *R, void *C, void *stream)
{
    if (!desc) return MOA_ERR_INVALID_ARG;
    if (desc->M <= 0 || desc->N <= 0 || desc->K <= 0) return MOA_ERR_INVALID_ARG;
    if ((desc->a_layout != 0 && desc->a_layout != 1) || (desc->b_layout != 0 && desc->b_layout != 1)) return MOA_ERR_INVALID_ARG;
    if (desc->dtype != MOA_BF16 && desc->dtype != MOA_F32) return MOA_ERR_INVALID_ARG;
    if (desc->dtype != MOA_BF16) return MOA_ERR_UNSUPPORTED;
    // row lengths: A [M,K] or [K,M]; B [N,K] or [K,N]; C, R [M,N]
    const int a_cols = desc->a_layout ? desc->M : desc->K, b_cols = desc->b_layout ? desc->N : desc->K;
    if (a_cols % 8 != 0 || b_cols % 8 != 0 || desc->N % 8 != 0) return MOA_ERR_UNSUPPORTED;
    if (!A || !B || !C) return MOA_ERR_INVALID_ARG;
    if (!aligned16(A) || !aligned16(B) || !aligned16(C) || (R && !aligned16(R))) return MOA_ERR_INVALID_ARG;
    moa_status s = check_device_arch();
    if (s != MOA_OK) return s;
    return gemm_bf16(desc->a_layout, desc->b_layout, desc->M, desc->N, desc->K, A, B, R, C, (cudaStream_t)stream) == cudaSuccess
               ? MOA_OK : MOA_ERR_CUDA;
}

}  // extern "C"
