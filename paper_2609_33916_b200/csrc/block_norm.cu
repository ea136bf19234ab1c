// RMSNorm forward and backward (bf16 storage, fp32 arithmetic).  HBM-bound: x is read once and y
// written once by the forward; the backward reads x and dy once and writes dx once.
//
// Thread layout (both kernels): a row is covered by `tpr` threads (a power of two, 1..256), each
// owning the 16-byte vectors v = c, c + tpr, ... of the row (kV of them at most), so a thread always
// touches the same columns and keeps the gain -- and, in the backward, its share of the dg sums --
// in registers.  The 256 threads of a CTA form 256/tpr row lanes, and a lane takes R rows per
// iteration.  Row sums are reduced by shuffles inside a warp and, for tpr > 32, through shared
// memory across the warps of the lane.  Two iterations are kept in registers (see below).
#include "common.cuh"
#include "moa_block.h"

namespace moa {
namespace {

constexpr int kNormThreads = 256;

__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8])
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 p = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&w[i]));
        f[2 * i] = p.x;
        f[2 * i + 1] = p.y;
    }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        w[i] = *reinterpret_cast<const uint32_t *>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Sum of v[0..R) over the tpr threads of a row lane; every thread of the lane gets the totals.
// `red` is [8 warps][R] floats of shared memory; the call contains block-wide barriers when tpr > 32,
// so every thread of the CTA must make it.
template <int R>
__device__ __forceinline__ void lane_sum(float (&v)[R], int tpr, float *red)
{
    const int width = tpr < 32 ? tpr : 32;
#pragma unroll
    for (int i = 0; i < R; ++i)
        for (int o = width / 2; o >= 1; o >>= 1) v[i] += __shfl_xor_sync(0xffffffffu, v[i], o);
    if (tpr > 32) {
        const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
        const int wpl = tpr / 32;                       // warps per row lane
        const int w0 = (warp / wpl) * wpl;
        if (lane == 0)
#pragma unroll
            for (int i = 0; i < R; ++i) red[warp * R + i] = v[i];
        __syncthreads();
#pragma unroll
        for (int i = 0; i < R; ++i) {
            float s = 0.f;
            for (int w = 0; w < wpl; ++w) s += red[(w0 + w) * R + i];     // fixed order
            v[i] = s;
        }
        __syncthreads();
    }
}

// Rows of one iteration of one row lane, as the raw 16-byte vectors this thread owns.
template <int kV, int R>
struct RowRegs {
    uint4 v[R][kV];
};

template <int kV, int R>
__device__ __forceinline__ void load_rows(RowRegs<kV, R> &dst, const __nv_bfloat16 *__restrict__ src, long long row0,
                                          int n, int d, int c, int tpr)
{
    const int nvec = d / 8;
#pragma unroll
    for (int i = 0; i < R; ++i)
#pragma unroll
        for (int j = 0; j < kV; ++j) {
            const int v = c + j * tpr;
            dst.v[i][j] = make_uint4(0u, 0u, 0u, 0u);
            if (row0 + i < n && v < nvec) dst.v[i][j] = __ldcs(reinterpret_cast<const uint4 *>(src + (size_t)(row0 + i) * d) + v);
        }
}

// Both kernels keep two iterations in registers: the loads of iteration it + 1 are issued before
// iteration it is reduced and written, so a CTA always has requests in flight (a load-reduce-store
// sequence per iteration, with its two block barriers, left HBM idle about 40 % of the time).
template <int kV, int R>
__global__ void __launch_bounds__(kNormThreads)
rmsnorm_fwd_kernel(const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ g,
                   __nv_bfloat16 *__restrict__ y, float *__restrict__ r_out, int n, int d, float eps, int tpr)
{
    __shared__ float red[8 * R];
    const int c = threadIdx.x % tpr, rl = threadIdx.x / tpr, lanes = kNormThreads / tpr;
    const int nvec = d / 8;
    float gf[kV][8];
#pragma unroll
    for (int j = 0; j < kV; ++j) {
        const int v = c + j * tpr;
        uint4 gv = make_uint4(0u, 0u, 0u, 0u);
        if (v < nvec) gv = __ldg(reinterpret_cast<const uint4 *>(g) + v);
        unpack8(gv, gf[j]);
    }
    const long long rows_per_iter = (long long)gridDim.x * lanes * R;
    const int iters = (int)((n + rows_per_iter - 1) / rows_per_iter);
    const long long first = ((long long)blockIdx.x * lanes + rl) * R;
    const float inv_d = 1.f / (float)d;
    RowRegs<kV, R> cur, nxt;
    load_rows<kV, R>(cur, x, first, n, d, c, tpr);
    for (int it = 0; it < iters; ++it) {
        const long long row0 = it * rows_per_iter + first;
        if (it + 1 < iters) load_rows<kV, R>(nxt, x, row0 + rows_per_iter, n, d, c, tpr);
        float ss[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            ss[i] = 0.f;
#pragma unroll
            for (int j = 0; j < kV; ++j) {
                float f[8];
                unpack8(cur.v[i][j], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) ss[i] = fmaf(f[e], f[e], ss[i]);
            }
        }
        lane_sum<R>(ss, tpr, red);
#pragma unroll
        for (int i = 0; i < R; ++i) {
            if (row0 + i >= n) continue;
            const float r = rsqrtf(ss[i] * inv_d + eps);
            if (c == 0 && r_out != nullptr) r_out[row0 + i] = r;
#pragma unroll
            for (int j = 0; j < kV; ++j) {
                const int v = c + j * tpr;
                if (v >= nvec) continue;
                float f[8];
                unpack8(cur.v[i][j], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) f[e] = f[e] * r * gf[j][e];
                __stcs(reinterpret_cast<uint4 *>(y + (size_t)(row0 + i) * d) + v, pack8(f));
            }
        }
        cur = nxt;
    }
}

// Backward.  Besides dx, every CTA leaves its partial dg (summed over its rows in a fixed order) in
// part[blockIdx.x][d]; rmsnorm_dg_kernel adds the partials up.
template <int kV, int R>
__global__ void __launch_bounds__(kNormThreads)
rmsnorm_bwd_kernel(const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ g,
                   const float *__restrict__ r_in, const __nv_bfloat16 *__restrict__ dy,
                   __nv_bfloat16 *__restrict__ dx, float *__restrict__ part, int n, int d, float eps, int tpr)
{
    __shared__ float red[8 * R];
    __shared__ float acc[kNormThreads * 8];              // [row lane][tpr*8] for one j at a time
    const int c = threadIdx.x % tpr, rl = threadIdx.x / tpr, lanes = kNormThreads / tpr;
    const int nvec = d / 8;
    float gf[kV][8], dgacc[kV][8];
#pragma unroll
    for (int j = 0; j < kV; ++j) {
        const int v = c + j * tpr;
        uint4 gv = make_uint4(0u, 0u, 0u, 0u);
        if (v < nvec) gv = __ldg(reinterpret_cast<const uint4 *>(g) + v);
        unpack8(gv, gf[j]);
#pragma unroll
        for (int e = 0; e < 8; ++e) dgacc[j][e] = 0.f;
    }
    const long long rows_per_iter = (long long)gridDim.x * lanes * R;
    const int iters = (int)((n + rows_per_iter - 1) / rows_per_iter);
    const long long first = ((long long)blockIdx.x * lanes + rl) * R;
    const float inv_d = 1.f / (float)d;
    RowRegs<kV, R> xc, dc, xn, dn;
    load_rows<kV, R>(xc, x, first, n, d, c, tpr);
    load_rows<kV, R>(dc, dy, first, n, d, c, tpr);
    for (int it = 0; it < iters; ++it) {
        const long long row0 = it * rows_per_iter + first;
        if (it + 1 < iters) {
            load_rows<kV, R>(xn, x, row0 + rows_per_iter, n, d, c, tpr);
            load_rows<kV, R>(dn, dy, row0 + rows_per_iter, n, d, c, tpr);
        }
        // the stored r of this iteration's rows: requested here, ahead of the reductions and their barriers
        float rr[R];
#pragma unroll
        for (int i = 0; i < R; ++i) rr[i] = (r_in != nullptr && row0 + i < n) ? __ldg(r_in + row0 + i) : 0.f;
        // per row: t = sum_k x_k g_k dy_k, and sum_k x_k^2 when r is not given
        float t[R], ss[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            t[i] = ss[i] = 0.f;
#pragma unroll
            for (int j = 0; j < kV; ++j) {
                float fx[8], fd[8];
                unpack8(xc.v[i][j], fx);
                unpack8(dc.v[i][j], fd);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    t[i] = fmaf(fx[e] * gf[j][e], fd[e], t[i]);
                    ss[i] = fmaf(fx[e], fx[e], ss[i]);
                }
            }
        }
        lane_sum<R>(t, tpr, red);
        if (r_in == nullptr) lane_sum<R>(ss, tpr, red);          // uniform over the grid
#pragma unroll
        for (int i = 0; i < R; ++i) {
            if (row0 + i >= n) continue;
            const float r = r_in != nullptr ? rr[i] : rsqrtf(ss[i] * inv_d + eps);
            const float coef = r * r * r * t[i] * inv_d;
#pragma unroll
            for (int j = 0; j < kV; ++j) {
                const int v = c + j * tpr;
                if (v >= nvec) continue;
                float fx[8], fd[8], o[8];
                unpack8(xc.v[i][j], fx);
                unpack8(dc.v[i][j], fd);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    o[e] = r * gf[j][e] * fd[e] - fx[e] * coef;
                    dgacc[j][e] = fmaf(fd[e] * fx[e], r, dgacc[j][e]);
                }
                __stcs(reinterpret_cast<uint4 *>(dx + (size_t)(row0 + i) * d) + v, pack8(o));
            }
        }
        xc = xn;
        dc = dn;
    }
    // CTA partial of dg: the row lanes' sums added in lane order
    float *mine = part + (size_t)blockIdx.x * d;
#pragma unroll
    for (int j = 0; j < kV; ++j) {
        __syncthreads();
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[(rl * tpr + c) * 8 + e] = dgacc[j][e];
        __syncthreads();
        for (int q = threadIdx.x; q < tpr * 8; q += kNormThreads) {
            const int col = (j * tpr + q / 8) * 8 + q % 8;
            if (col >= d) continue;
            float s = 0.f;
            for (int l = 0; l < lanes; ++l) s += acc[l * tpr * 8 + q];
            mine[col] = s;
        }
    }
}

// dg[col] = sum over the CTA partials, in a fixed order: a CTA owns 32 columns, its 16 warps take the
// partial rows w, w + 16, ... (four independent running sums each, so that the loads overlap) and the
// sums are added in a fixed order.
constexpr int kDgWarps = 16;
__global__ void __launch_bounds__(32 * kDgWarps)
rmsnorm_dg_kernel(const float *__restrict__ part, __nv_bfloat16 *__restrict__ dg, int parts, int d)
{
    __shared__ float s[kDgWarps][32];
    const int cx = threadIdx.x % 32, cy = threadIdx.x / 32;
    const int col = blockIdx.x * 32 + cx;
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    if (col < d) {
        int p = cy;
        for (; p + 3 * kDgWarps < parts; p += 4 * kDgWarps) {
            a0 += part[(size_t)p * d + col];
            a1 += part[(size_t)(p + kDgWarps) * d + col];
            a2 += part[(size_t)(p + 2 * kDgWarps) * d + col];
            a3 += part[(size_t)(p + 3 * kDgWarps) * d + col];
        }
        for (; p < parts; p += kDgWarps) a0 += part[(size_t)p * d + col];
    }
    s[cy][cx] = (a0 + a1) + (a2 + a3);
    __syncthreads();
    if (cy == 0 && col < d) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < kDgWarps; ++w) t += s[w][cx];
        dg[col] = __float2bfloat16_rn(t);
    }
}

struct NormPlan {
    int tpr, kV, R, grid;
};
// Threads per row: the smallest power of two (at least a warp, at most the CTA) that leaves a thread
// no more than max_kv vectors of a row.  Measured on B200 (n*d = 2^27): a few vectors per thread and
// one row per lane and iteration beat wider rows of threads (fewer CTA barriers per byte moved).
NormPlan norm_plan(int n, int d, bool bwd)
{
    NormPlan p{};
    const int nvec = d / 8;
    const int max_kv = bwd ? (d > 4096 ? 4 : 2) : 4;
    p.tpr = 1;
    while (p.tpr < nvec && p.tpr < 32) p.tpr *= 2;
    while ((nvec + p.tpr - 1) / p.tpr > max_kv && p.tpr < kNormThreads) p.tpr *= 2;
    const int need = (nvec + p.tpr - 1) / p.tpr;           // vectors per thread per row
    p.kV = need <= 1 ? 1 : need <= 2 ? 2 : 4;
    p.R = p.kV == 1 ? 2 : (bwd && p.kV == 4) ? 2 : 1;
    const int lanes = kNormThreads / p.tpr;
    const long long blocks = ((long long)n + (long long)lanes * p.R - 1) / ((long long)lanes * p.R);
    p.grid = (int)(blocks < 148 * 4 ? blocks : 148 * 4);
    if (p.grid < 1) p.grid = 1;
    return p;
}

}  // namespace

size_t rmsnorm_workspace_bytes(int n, int d) { return (size_t)norm_plan(n, d, true).grid * d * sizeof(float); }

cudaError_t rmsnorm_fwd(int n, int d, float eps, const void *x, const void *g, void *y, float *r, cudaStream_t st)
{
    const NormPlan p = norm_plan(n, d, false);
    const auto *xb = (const __nv_bfloat16 *)x;
    const auto *gb = (const __nv_bfloat16 *)g;
    auto *yb = (__nv_bfloat16 *)y;
    LaunchScope scope(MOA_KERNEL_OTHER, st);
    if (p.kV == 1) rmsnorm_fwd_kernel<1, 2><<<p.grid, kNormThreads, 0, st>>>(xb, gb, yb, r, n, d, eps, p.tpr);
    else if (p.kV == 2) rmsnorm_fwd_kernel<2, 1><<<p.grid, kNormThreads, 0, st>>>(xb, gb, yb, r, n, d, eps, p.tpr);
    else rmsnorm_fwd_kernel<4, 1><<<p.grid, kNormThreads, 0, st>>>(xb, gb, yb, r, n, d, eps, p.tpr);
    return cudaGetLastError();
}

cudaError_t rmsnorm_bwd(int n, int d, float eps, const void *x, const void *g, const float *r, const void *dy,
                        void *dx, void *dg, void *ws, cudaStream_t st)
{
    const NormPlan p = norm_plan(n, d, true);
    const auto *xb = (const __nv_bfloat16 *)x;
    const auto *gb = (const __nv_bfloat16 *)g;
    const auto *db = (const __nv_bfloat16 *)dy;
    auto *ob = (__nv_bfloat16 *)dx;
    float *part = (float *)ws;
    {
        LaunchScope scope(MOA_KERNEL_OTHER, st);
        if (p.kV == 1) rmsnorm_bwd_kernel<1, 2><<<p.grid, kNormThreads, 0, st>>>(xb, gb, r, db, ob, part, n, d, eps, p.tpr);
        else if (p.kV == 2) rmsnorm_bwd_kernel<2, 1><<<p.grid, kNormThreads, 0, st>>>(xb, gb, r, db, ob, part, n, d, eps, p.tpr);
        else rmsnorm_bwd_kernel<4, 2><<<p.grid, kNormThreads, 0, st>>>(xb, gb, r, db, ob, part, n, d, eps, p.tpr);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    LaunchScope scope(MOA_KERNEL_OTHER, st);
    rmsnorm_dg_kernel<<<(d + 31) / 32, 32 * kDgWarps, 0, st>>>(part, (__nv_bfloat16 *)dg, p.grid, d);
    return cudaGetLastError();
}

}  // namespace moa
