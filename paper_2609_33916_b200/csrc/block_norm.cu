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
#include "ptx.cuh"

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
                   const __nv_bfloat16 *__restrict__ dx_add, __nv_bfloat16 *__restrict__ dx, float *__restrict__ part, int n,
                   int d, float eps, int tpr)
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
                float fx[8], fd[8], o[8], fa[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                unpack8(xc.v[i][j], fx);
                unpack8(dc.v[i][j], fd);
                if (dx_add != nullptr) unpack8(__ldcs(reinterpret_cast<const uint4 *>(dx_add + (size_t)(row0 + i) * d) + v), fa);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    o[e] = r * gf[j][e] * fd[e] - fx[e] * coef + fa[e];
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

// ---------------------------------------------------------------------------------------------
// Ring variant (d <= 2048): the rows come through a shared-memory ring filled by bulk copies, so the
// bytes in flight no longer depend on what the computing warps hold in registers.  One producer
// thread keeps kRingStages stages of kRingWarps * m consecutive rows requested (x, and dy in the
// backward; a stage is one contiguous block of memory per array: one bulk copy each); two groups of
// eight consumer warps compute alternate stages (all of them follow every stage's barriers), a warp one row at a time (32 lanes x up to 8 vectors of
// 16 bytes), reduce with shuffles only -- no block barrier in the loop -- and write their results
// straight to global memory in whole 512-byte runs.  A row is read from shared memory twice (sums,
// then results) rather than held in registers, and the gain sits in shared memory as floats, which
// keeps the kernel near 100 registers.  Every wait is bounded.
constexpr int kRingWarps = 8;                 // consumer warps per group = rows per stage / m
constexpr int kRingGroups = 2;                // consumer groups; group q takes the CTA's stages q, q + 2, ...
constexpr int kRingThreads = 32 * (kRingGroups * kRingWarps + 1), kRingStages = 3;
enum { NERR_EMPTY = 0x401, NERR_FULL = 0x402 };

template <int kV, bool kBwd>
__global__ void __launch_bounds__(kRingThreads, 1)
rmsnorm_ring_kernel(const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ g, const float *__restrict__ r_in,
                    float *__restrict__ r_out, const __nv_bfloat16 *__restrict__ dy, const __nv_bfloat16 *__restrict__ dx_add,
                    __nv_bfloat16 *__restrict__ out, float *__restrict__ part, int n, int d, float eps, int m,
                    unsigned int *status)
{
    using namespace ptx;
    extern __shared__ __align__(128) uint8_t nring[];
    const int rows_stage = kRingWarps * m;
    const size_t row_bytes = (size_t)d * 2, arr_bytes = (size_t)rows_stage * row_bytes;
    const size_t stage_bytes = arr_bytes * (kBwd ? 2 : 1);
    float *gs = reinterpret_cast<float *>(nring + kRingStages * stage_bytes);          // gain as floats [d]
    uint64_t *full = reinterpret_cast<uint64_t *>(gs + d);
    uint64_t *empty = full + kRingStages;
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(empty + kRingStages);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int nvec = d / 8;
    const long long total_stages = ((long long)n + rows_stage - 1) / rows_stage;
    const int my_stages = (int)((total_stages - blockIdx.x + gridDim.x - 1) / gridDim.x);   // stages b, b + grid, ...
    if (threadIdx.x == 0) {
        for (int s = 0; s < kRingStages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, kRingGroups * kRingWarps); }
        *abortp = 0;
        fence_mbar_init();
    }
    for (int i = threadIdx.x; i < d; i += kRingThreads) gs[i] = __bfloat162float(g[i]);
    __syncthreads();
    float dgacc[kV][8];          // backward only (dead otherwise)
#pragma unroll
    for (int j = 0; j < kV; ++j)
#pragma unroll
        for (int e = 0; e < 8; ++e) dgacc[j][e] = 0.f;

    if (warp == kRingGroups * kRingWarps) {
        if (lane == 0) {
            ArmCounts<kRingStages> armed;     // stages armed for copies into the ring
            for (int i = 0; i < my_stages; ++i) {
                const int s = i % kRingStages;
                if (!mbar_wait(empty + s, ((i / kRingStages) & 1) ^ 1, abortp, status, NERR_EMPTY)) break;
                const long long row0 = ((long long)blockIdx.x + (long long)i * gridDim.x) * rows_stage;
                const int rows = (int)min((long long)rows_stage, (long long)n - row0);
                const uint32_t bytes = (uint32_t)(rows * row_bytes);
                mbar_arm(full, s, kBwd ? 2 * bytes : bytes, armed);
                bulk_load_1d(nring + s * stage_bytes, x + row0 * d, bytes, full + s);
                if (kBwd) bulk_load_1d(nring + s * stage_bytes + arr_bytes, dy + row0 * d, bytes, full + s);
            }
            mbar_drain(full, armed);      // copies still on their way land before the CTA leaves (bounded)
        }
    } else {
        const float inv_d = 1.f / (float)d;
        const int grp = warp / kRingWarps, gw = warp % kRingWarps;
        // Every consumer warp waits for every stage and releases it, in order, although it computes only its
        // group's: a warp that skipped stages could find a slot's barrier still in the phase of an older stage
        // of the same parity and take it for the one it is waiting for.
        for (int i = 0; i < my_stages; ++i) {
            const int s = i % kRingStages;
            if (!mbar_wait(full + s, (i / kRingStages) & 1, abortp, status, NERR_FULL)) break;
            if (i % kRingGroups != grp) {
                if (lane == 0) mbar_arrive(empty + s);
                continue;
            }
            const long long row0 = ((long long)blockIdx.x + (long long)i * gridDim.x) * rows_stage;
            const uint8_t *sx = nring + s * stage_bytes, *sd = sx + arr_bytes;
            for (int q = 0; q < m; ++q) {
                const int lr = gw * m + q;                    // row of the stage
                const long long row = row0 + lr;
                if (row >= n) break;                          // warp-uniform
                float rr = 0.f;
                if (kBwd && r_in != nullptr) rr = __ldg(r_in + row);
                float ss = 0.f, t = 0.f;
#pragma unroll
                for (int j = 0; j < kV; ++j) {
                    const int v = lane + 32 * j;
                    if (v >= nvec) continue;
                    float fx[8], fd[8];
                    unpack8(*reinterpret_cast<const uint4 *>(sx + lr * row_bytes + 16 * v), fx);
                    if (kBwd) unpack8(*reinterpret_cast<const uint4 *>(sd + lr * row_bytes + 16 * v), fd);
                    const float4 g0 = *reinterpret_cast<const float4 *>(gs + 8 * v), g1 = *reinterpret_cast<const float4 *>(gs + 8 * v + 4);
                    const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        ss = fmaf(fx[e], fx[e], ss);
                        if (kBwd) t = fmaf(fx[e] * gg[e], fd[e], t);
                    }
                }
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) {
                    ss += __shfl_xor_sync(0xffffffffu, ss, o);
                    if (kBwd) t += __shfl_xor_sync(0xffffffffu, t, o);
                }
                const float r = (kBwd && r_in != nullptr) ? rr : rsqrtf(ss * inv_d + eps);
                if (!kBwd && r_out != nullptr && lane == 0) r_out[row] = r;
                const float coef = r * r * r * t * inv_d;
                asm volatile("" ::: "memory");      // second pass reads the row again instead of keeping it in registers
#pragma unroll
                for (int j = 0; j < kV; ++j) {
                    const int v = lane + 32 * j;
                    if (v >= nvec) continue;
                    float fx[8], fd[8], o8[8], fa[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                    unpack8(*reinterpret_cast<const uint4 *>(sx + lr * row_bytes + 16 * v), fx);
                    if (kBwd) unpack8(*reinterpret_cast<const uint4 *>(sd + lr * row_bytes + 16 * v), fd);
                    if (kBwd && dx_add != nullptr) unpack8(__ldcs(reinterpret_cast<const uint4 *>(dx_add + (size_t)row * d) + v), fa);
                    const float4 g0 = *reinterpret_cast<const float4 *>(gs + 8 * v), g1 = *reinterpret_cast<const float4 *>(gs + 8 * v + 4);
                    const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        if (kBwd) {
                            o8[e] = r * gg[e] * fd[e] - fx[e] * coef + fa[e];
                            dgacc[j][e] = fmaf(fd[e] * fx[e], r, dgacc[j][e]);
                        } else {
                            o8[e] = fx[e] * r * gg[e];
                        }
                    }
                    __stcs(reinterpret_cast<uint4 *>(out + (size_t)row * d) + v, pack8(o8));
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty + s);
        }
    }
    if (kBwd) {
        // CTA partial of dg: the eight warps' sums, added in warp order (the ring is free: every consumer is done)
        __syncthreads();
        float *accs = reinterpret_cast<float *>(nring);                     // [consumer warps][d]
        if (warp < kRingGroups * kRingWarps) {
#pragma unroll
            for (int j = 0; j < kV; ++j) {
                const int v = lane + 32 * j;
                if (v < nvec)
#pragma unroll
                    for (int e = 0; e < 8; ++e) accs[(size_t)warp * d + 8 * v + e] = dgacc[j][e];
            }
        }
        __syncthreads();
        float *mine = part + (size_t)blockIdx.x * d;
        for (int col = threadIdx.x; col < d; col += kRingThreads) {
            float a = 0.f;
#pragma unroll
            for (int w = 0; w < kRingGroups * kRingWarps; ++w) a += accs[(size_t)w * d + col];
            mine[col] = a;
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
    const long long cap = 4LL * device_info().sms;
    p.grid = (int)(blocks < cap ? blocks : cap);
    if (p.grid < 1) p.grid = 1;
    return p;
}


// The ring variant serves rows of 256 .. 2048 elements (a warp per row, at most 8 vectors per lane).
bool norm_uses_ring(int d) { return d >= 256 && d <= 2048; }
struct RingPlan {
    int kV, m, grid;
    size_t smem;
};
RingPlan ring_plan(int n, int d, bool bwd)
{
    RingPlan p{};
    const int nvec = d / 8, need = (nvec + 31) / 32;
    p.kV = need <= 1 ? 1 : need <= 2 ? 2 : need <= 4 ? 4 : 8;
    p.m = 2048 / d < 1 ? 1 : 2048 / d;                                  // 32 KB per array and stage
    const long long rows_stage = (long long)kRingWarps * p.m;
    const long long stages = ((long long)n + rows_stage - 1) / rows_stage;
    const long long sms = device_info().sms;
    p.grid = (int)(stages < sms ? stages : sms);
    p.smem = (size_t)kRingStages * rows_stage * d * 2 * (bwd ? 2 : 1) + (size_t)d * 4 + 2 * kRingStages * 8 + 16;
    return p;
}

template <int kV, bool kBwd>
cudaError_t launch_ring(const RingPlan &p, const __nv_bfloat16 *x, const __nv_bfloat16 *g, const float *r_in, float *r_out,
                        const __nv_bfloat16 *dy, const __nv_bfloat16 *dx_add, __nv_bfloat16 *out, float *part, int n, int d,
                        float eps, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(rmsnorm_ring_kernel<kV, kBwd>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
    if (e != cudaSuccess) return e;
    rmsnorm_ring_kernel<kV, kBwd><<<p.grid, kRingThreads, p.smem, st>>>(x, g, r_in, r_out, dy, dx_add, out, part, n, d, eps,
                                                                        p.m, device_status_ptr());
    return cudaGetLastError();
}
template <bool kBwd>
cudaError_t launch_ring_kv(const RingPlan &p, const __nv_bfloat16 *x, const __nv_bfloat16 *g, const float *r_in, float *r_out,
                           const __nv_bfloat16 *dy, const __nv_bfloat16 *dx_add, __nv_bfloat16 *out, float *part, int n, int d,
                           float eps, cudaStream_t st)
{
    if (p.kV == 1) return launch_ring<1, kBwd>(p, x, g, r_in, r_out, dy, dx_add, out, part, n, d, eps, st);
    if (p.kV == 2) return launch_ring<2, kBwd>(p, x, g, r_in, r_out, dy, dx_add, out, part, n, d, eps, st);
    if (p.kV == 4) return launch_ring<4, kBwd>(p, x, g, r_in, r_out, dy, dx_add, out, part, n, d, eps, st);
    return launch_ring<8, kBwd>(p, x, g, r_in, r_out, dy, dx_add, out, part, n, d, eps, st);
}

}  // namespace

// per-CTA partial sums of dg: at most four CTAs per SM in either variant
size_t rmsnorm_workspace_bytes(int n, int d) { (void)n; return (size_t)device_info().sms * 4 * d * sizeof(float); }

cudaError_t rmsnorm_fwd(int n, int d, float eps, const void *x, const void *g, void *y, float *r, cudaStream_t st)
{
    const NormPlan p = norm_plan(n, d, false);
    const auto *xb = (const __nv_bfloat16 *)x;
    const auto *gb = (const __nv_bfloat16 *)g;
    auto *yb = (__nv_bfloat16 *)y;
    LaunchScope scope(MOA_KERNEL_OTHER, st);
    if (norm_uses_ring(d)) return launch_ring_kv<false>(ring_plan(n, d, false), xb, gb, nullptr, r, nullptr, nullptr, yb, nullptr, n, d, eps, st);
    if (p.kV == 1) rmsnorm_fwd_kernel<1, 2><<<p.grid, kNormThreads, 0, st>>>(xb, gb, yb, r, n, d, eps, p.tpr);
    else if (p.kV == 2) rmsnorm_fwd_kernel<2, 1><<<p.grid, kNormThreads, 0, st>>>(xb, gb, yb, r, n, d, eps, p.tpr);
    else rmsnorm_fwd_kernel<4, 1><<<p.grid, kNormThreads, 0, st>>>(xb, gb, yb, r, n, d, eps, p.tpr);
    return cudaGetLastError();
}

cudaError_t rmsnorm_bwd(int n, int d, float eps, const void *x, const void *g, const float *r, const void *dy,
                        const void *dx_add, void *dx, void *dg, void *ws, cudaStream_t st)
{
    const auto *ab = (const __nv_bfloat16 *)dx_add;
    const NormPlan p = norm_plan(n, d, true);
    const auto *xb = (const __nv_bfloat16 *)x;
    const auto *gb = (const __nv_bfloat16 *)g;
    const auto *db = (const __nv_bfloat16 *)dy;
    auto *ob = (__nv_bfloat16 *)dx;
    float *part = (float *)ws;
    int parts = p.grid;
    if (norm_uses_ring(d)) {
        const RingPlan rp = ring_plan(n, d, true);
        parts = rp.grid;
        LaunchScope scope(MOA_KERNEL_OTHER, st);
        const cudaError_t e = launch_ring_kv<true>(rp, xb, gb, r, nullptr, db, ab, ob, part, n, d, eps, st);
        if (e != cudaSuccess) return e;
    } else {
        LaunchScope scope(MOA_KERNEL_OTHER, st);
        if (p.kV == 1) rmsnorm_bwd_kernel<1, 2><<<p.grid, kNormThreads, 0, st>>>(xb, gb, r, db, ab, ob, part, n, d, eps, p.tpr);
        else if (p.kV == 2) rmsnorm_bwd_kernel<2, 1><<<p.grid, kNormThreads, 0, st>>>(xb, gb, r, db, ab, ob, part, n, d, eps, p.tpr);
        else rmsnorm_bwd_kernel<4, 2><<<p.grid, kNormThreads, 0, st>>>(xb, gb, r, db, ab, ob, part, n, d, eps, p.tpr);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    LaunchScope scope(MOA_KERNEL_OTHER, st);
    rmsnorm_dg_kernel<<<(d + 31) / 32, 32 * kDgWarps, 0, st>>>(part, (__nv_bfloat16 *)dg, parts, d);
    return cudaGetLastError();
}

}  // namespace moa
