// fp32 SIMT kernels: the MOA_F32 path, and a generic path for any dtype/shape.
//
// Tiles of 64 query rows x 64 keys, 256 threads as a 16 x 16 grid; thread (ty,tx)
// owns score rows ty*4..ty*4+3 and score columns tx, tx+16, tx+32, tx+48, and the
// output columns tx+16c.  Online softmax in the forward; the backward recomputes P
// from the stored logsumexp, one CTA per key tile (each dK/dV element has exactly
// one writer), dQ either by fp32 atomics or by a separate query-parallel kernel.
#include "common.cuh"
#include <math.h>

namespace moa {
namespace {

constexpr int BM = 64;       // query rows per tile
constexpr int BN = 64;       // keys per tile
constexpr int NTHREADS = 256;
constexpr int SLD = BN + 1;  // leading dimension of the 64x64 score tiles in shared memory

template <typename T, int D>
__device__ __forceinline__ void load_tile(float *dst, const T *src, int row0, int n)
{
    constexpr int LD = D + 1;
    for (int idx = threadIdx.x; idx < BM * D; idx += NTHREADS) {
        const int r = idx / D, c = idx % D;
        const int row = row0 + r;
        dst[r * LD + c] = row < n ? to_float<T>(src[(size_t)row * D + c]) : 0.f;
    }
}

__device__ __forceinline__ float group16_max(float v)
{
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float group16_sum(float v)
{
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ------------------------------------------------------------------------- forward
template <typename T, int D>
__global__ void __launch_bounds__(NTHREADS)
simt_fwd_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                T *__restrict__ O, float *__restrict__ L, int n, int causal, float scale, int nqt)
{
    constexpr int LD = D + 1;
    constexpr int NC = D / 16;
    extern __shared__ float smem[];
    float *Qs = smem, *Ks = Qs + BM * LD, *Vs = Ks + BN * LD, *Ss = Vs + BN * LD;

    int qt = blockIdx.x % nqt;
    const int bh = blockIdx.x / nqt;
    if (causal) qt = nqt - 1 - qt;  // longest rows first
    const int q0 = qt * BM;
    const size_t base = (size_t)bh * n * D;
    Q += base; K += base; V += base; O += base; L += (size_t)bh * n;

    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    load_tile<T, D>(Qs, Q, q0, n);

    float m[4], l[4], o[4][NC];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        m[a] = -INFINITY; l[a] = 0.f;
#pragma unroll
        for (int c = 0; c < NC; ++c) o[a][c] = 0.f;
    }
    const int kend = causal ? min(n, q0 + BM) : n;
    for (int k0 = 0; k0 < kend; k0 += BN) {
        __syncthreads();
        load_tile<T, D>(Ks, K, k0, n);
        load_tile<T, D>(Vs, V, k0, n);
        __syncthreads();
        float s[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) s[a][b] = 0.f;
#pragma unroll 4
        for (int k = 0; k < D; ++k) {
            float qv[4], kv[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) qv[a] = Qs[(ty * 4 + a) * LD + k];
#pragma unroll
            for (int b = 0; b < 4; ++b) kv[b] = Ks[(tx + 16 * b) * LD + k];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) s[a][b] = fmaf(qv[a], kv[b], s[a][b]);
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int row = q0 + ty * 4 + a;
            float mx = -INFINITY;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int col = k0 + tx + 16 * b;
                float v = s[a][b] * scale;
                if (col >= n || (causal && col > row)) v = -INFINITY;
                s[a][b] = v;
                mx = fmaxf(mx, v);
            }
            mx = group16_max(mx);
            float mn = fmaxf(m[a], mx);
            if (mn == -INFINITY) mn = 0.f;  // whole row masked so far (padding rows only)
            const float alpha = expf(m[a] - mn);
            float sum = 0.f;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const float pv = expf(s[a][b] - mn);
                sum += pv;
                Ss[(ty * 4 + a) * SLD + tx + 16 * b] = pv;
            }
            sum = group16_sum(sum);
            l[a] = l[a] * alpha + sum;
            m[a] = mn;
#pragma unroll
            for (int c = 0; c < NC; ++c) o[a][c] *= alpha;
        }
        __syncthreads();
#pragma unroll 4
        for (int j = 0; j < BN; ++j) {
            float pv[4], vv[NC];
#pragma unroll
            for (int a = 0; a < 4; ++a) pv[a] = Ss[(ty * 4 + a) * SLD + j];
#pragma unroll
            for (int c = 0; c < NC; ++c) vv[c] = Vs[j * LD + tx + 16 * c];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < NC; ++c) o[a][c] = fmaf(pv[a], vv[c], o[a][c]);
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int row = q0 + ty * 4 + a;
        if (row >= n) continue;
        const float inv = 1.f / l[a];
#pragma unroll
        for (int c = 0; c < NC; ++c) O[(size_t)row * D + tx + 16 * c] = from_float<T>(o[a][c] * inv);
        if (tx == 0) L[row] = m[a] + logf(l[a]);
    }
}

// ---------------------------------------------------- rowsum(dO o O), one warp per row
template <typename T>
__global__ void row_dot_kernel(const T *__restrict__ dO, const T *__restrict__ O,
                               float *__restrict__ Dv, size_t rows, int d)
{
    const size_t row = (size_t)blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    if (row >= rows) return;
    const int lane = threadIdx.x % 32;
    float acc = 0.f;
    for (int c = lane; c < d; c += 32)
        acc = fmaf(to_float<T>(dO[row * d + c]), to_float<T>(O[row * d + c]), acc);
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) Dv[row] = acc;
}

// --------------------------------------------- shared by the two backward kernels
// scores and dP of a 64x64 tile -> P and scale*dS in shared memory
template <int D>
__device__ __forceinline__ void bwd_tile_p_ds(const float *Qs, const float *dOs, const float *Ks,
                                              const float *Vs, const float *Ls, const float *Ds,
                                              float *Ps, float *dSs, int q0, int k0, int n,
                                              int causal, float scale, int tx, int ty)
{
    constexpr int LD = D + 1;
    float s[4][4], dp[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) { s[a][b] = 0.f; dp[a][b] = 0.f; }
#pragma unroll 2
    for (int k = 0; k < D; ++k) {
        float qv[4], gv[4], kv[4], vv[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) { qv[a] = Qs[(ty * 4 + a) * LD + k]; gv[a] = dOs[(ty * 4 + a) * LD + k]; }
#pragma unroll
        for (int b = 0; b < 4; ++b) { kv[b] = Ks[(tx + 16 * b) * LD + k]; vv[b] = Vs[(tx + 16 * b) * LD + k]; }
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                s[a][b] = fmaf(qv[a], kv[b], s[a][b]);
                dp[a][b] = fmaf(gv[a], vv[b], dp[a][b]);
            }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int r = ty * 4 + a, row = q0 + r;
        const float Li = Ls[r], Di = Ds[r];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int cidx = tx + 16 * b, col = k0 + cidx;
            const bool live = row < n && col < n && !(causal && col > row);
            const float pv = live ? expf(s[a][b] * scale - Li) : 0.f;
            Ps[r * SLD + cidx] = pv;
            if (dSs) dSs[r * SLD + cidx] = pv * (dp[a][b] - Di) * scale;
        }
    }
}

__device__ __forceinline__ void load_rowvec(float *dst, const float *src, int row0, int n)
{
    for (int r = threadIdx.x; r < BM; r += NTHREADS) dst[r] = (row0 + r) < n ? src[row0 + r] : 0.f;
}

// ----------------------------------------- backward, one CTA per key tile: dK, dV (+dQ red)
template <typename T, int D>
__global__ void __launch_bounds__(NTHREADS)
simt_bwd_kv_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                   const T *__restrict__ dO, const float *__restrict__ L, const float *__restrict__ Dv,
                   T *__restrict__ dK, T *__restrict__ dV, float *__restrict__ dQacc,
                   int n, int causal, float scale, int nkt)
{
    constexpr int LD = D + 1;
    constexpr int NC = D / 16;
    extern __shared__ float smem[];
    float *Ks = smem, *Vs = Ks + BN * LD, *Qs = Vs + BN * LD, *dOs = Qs + BM * LD;
    float *Ps = dOs + BM * LD, *dSs = Ps + BM * SLD, *Ls = dSs + BM * SLD, *Ds = Ls + BM;

    const int kt = blockIdx.x % nkt;   // causal: key tile 0 has the most work and comes first
    const int bh = blockIdx.x / nkt;
    const int k0 = kt * BN;
    const size_t base = (size_t)bh * n * D;
    Q += base; K += base; V += base; dO += base; dV += base;
    if (dK) dK += base;
    L += (size_t)bh * n; Dv += (size_t)bh * n;
    if (dQacc) dQacc += base;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;

    load_tile<T, D>(Ks, K, k0, n);
    load_tile<T, D>(Vs, V, k0, n);
    float dk[4][NC], dv[4][NC];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < NC; ++c) { dk[a][c] = 0.f; dv[a][c] = 0.f; }

    const int qstart = causal ? (k0 / BM) * BM : 0;
    for (int q0 = qstart; q0 < n; q0 += BM) {
        __syncthreads();
        load_tile<T, D>(Qs, Q, q0, n);
        load_tile<T, D>(dOs, dO, q0, n);
        load_rowvec(Ls, L, q0, n);
        load_rowvec(Ds, Dv, q0, n);
        __syncthreads();
        bwd_tile_p_ds<D>(Qs, dOs, Ks, Vs, Ls, Ds, Ps, dSs, q0, k0, n, causal, scale, tx, ty);
        __syncthreads();
        // dV[key][c] += sum_q P[q][key] dO[q][c] ; dK[key][c] += sum_q (scale dS)[q][key] Q[q][c]
#pragma unroll 2
        for (int q = 0; q < BM; ++q) {
            float pv[4], gv[4], gq[NC], qq[NC];
#pragma unroll
            for (int a = 0; a < 4; ++a) { pv[a] = Ps[q * SLD + ty * 4 + a]; gv[a] = dSs[q * SLD + ty * 4 + a]; }
#pragma unroll
            for (int c = 0; c < NC; ++c) { gq[c] = dOs[q * LD + tx + 16 * c]; qq[c] = Qs[q * LD + tx + 16 * c]; }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    dv[a][c] = fmaf(pv[a], gq[c], dv[a][c]);
                    dk[a][c] = fmaf(gv[a], qq[c], dk[a][c]);
                }
        }
        if (dQacc) {
            // dQ[q][c] += sum_key (scale dS)[q][key] K[key][c]
            float dq[4][NC];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < NC; ++c) dq[a][c] = 0.f;
#pragma unroll 2
            for (int j = 0; j < BN; ++j) {
                float gv[4], kk[NC];
#pragma unroll
                for (int a = 0; a < 4; ++a) gv[a] = dSs[(ty * 4 + a) * SLD + j];
#pragma unroll
                for (int c = 0; c < NC; ++c) kk[c] = Ks[j * LD + tx + 16 * c];
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int c = 0; c < NC; ++c) dq[a][c] = fmaf(gv[a], kk[c], dq[a][c]);
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int row = q0 + ty * 4 + a;
                if (row >= n) continue;
#pragma unroll
                for (int c = 0; c < NC; ++c) atomicAdd(&dQacc[(size_t)row * D + tx + 16 * c], dq[a][c]);
            }
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int row = k0 + ty * 4 + a;
        if (row >= n) continue;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            if (dK) dK[(size_t)row * D + tx + 16 * c] = from_float<T>(dk[a][c]);   // nullptr: dV only
            dV[(size_t)row * D + tx + 16 * c] = from_float<T>(dv[a][c]);
        }
    }
}

// ----------------------------------------- backward, one CTA per query tile: dQ, no atomics
template <typename T, int D>
__global__ void __launch_bounds__(NTHREADS)
simt_bwd_dq_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                   const T *__restrict__ dO, const float *__restrict__ L, const float *__restrict__ Dv,
                   T *__restrict__ dQ, int n, int causal, float scale, int nqt)
{
    constexpr int LD = D + 1;
    constexpr int NC = D / 16;
    extern __shared__ float smem[];
    float *Ks = smem, *Vs = Ks + BN * LD, *Qs = Vs + BN * LD, *dOs = Qs + BM * LD;
    float *Ps = dOs + BM * LD, *dSs = Ps + BM * SLD, *Ls = dSs + BM * SLD, *Ds = Ls + BM;

    int qt = blockIdx.x % nqt;
    const int bh = blockIdx.x / nqt;
    if (causal) qt = nqt - 1 - qt;
    const int q0 = qt * BM;
    const size_t base = (size_t)bh * n * D;
    Q += base; K += base; V += base; dO += base; dQ += base;
    L += (size_t)bh * n; Dv += (size_t)bh * n;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;

    load_tile<T, D>(Qs, Q, q0, n);
    load_tile<T, D>(dOs, dO, q0, n);
    load_rowvec(Ls, L, q0, n);
    load_rowvec(Ds, Dv, q0, n);
    float dq[4][NC];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < NC; ++c) dq[a][c] = 0.f;
    const int kend = causal ? min(n, q0 + BM) : n;
    for (int k0 = 0; k0 < kend; k0 += BN) {
        __syncthreads();
        load_tile<T, D>(Ks, K, k0, n);
        load_tile<T, D>(Vs, V, k0, n);
        __syncthreads();
        bwd_tile_p_ds<D>(Qs, dOs, Ks, Vs, Ls, Ds, Ps, dSs, q0, k0, n, causal, scale, tx, ty);
        __syncthreads();
#pragma unroll 2
        for (int j = 0; j < BN; ++j) {
            float gv[4], kk[NC];
#pragma unroll
            for (int a = 0; a < 4; ++a) gv[a] = dSs[(ty * 4 + a) * SLD + j];
#pragma unroll
            for (int c = 0; c < NC; ++c) kk[c] = Ks[j * LD + tx + 16 * c];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < NC; ++c) dq[a][c] = fmaf(gv[a], kk[c], dq[a][c]);
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int row = q0 + ty * 4 + a;
        if (row >= n) continue;
#pragma unroll
        for (int c = 0; c < NC; ++c) dQ[(size_t)row * D + tx + 16 * c] = from_float<T>(dq[a][c]);
    }
}

// ------------------ row-parallel fused forward+backward in one kernel, dK/dV by atomics
// The paper's own fused design (Sec. 4, its first GPU version): one kernel, parallel over query
// rows.  A CTA runs the forward of its 64 query rows (online softmax; O, L), takes D = rowsum(dO o O)
// from the O it holds, and runs the backward of the same rows straight away: every row statistic it
// needs is its own, so no other CTA is waited for.  dQ stays local; the dV and dK contributions of
// every (query tile, key tile) pair are added into global fp32 accumulators with atomics -- the
// paper's GV and GK atomic sites.  kSites = 2: both sites (the paper's v1).  kSites = 1: only dK;
// dV then comes from an atomic-free key-parallel kernel of its own, as in the paper's v3.
template <typename T, int D, int kSites>
__global__ void __launch_bounds__(NTHREADS)
simt_rowpar_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                   const T *__restrict__ dO, T *__restrict__ O, float *__restrict__ L, float *__restrict__ Dv,
                   T *__restrict__ dQ, float *__restrict__ dKacc, float *__restrict__ dVacc,
                   int n, int causal, float scale, int nqt)
{
    constexpr int LD = D + 1;
    constexpr int NC = D / 16;
    extern __shared__ float smem[];
    float *Ks = smem, *Vs = Ks + BN * LD, *Qs = Vs + BN * LD, *dOs = Qs + BM * LD;
    float *Ps = dOs + BM * LD, *dSs = Ps + BM * SLD, *Ls = dSs + BM * SLD, *Ds = Ls + BM;

    int qt = blockIdx.x % nqt;
    const int bh = blockIdx.x / nqt;
    if (causal) qt = nqt - 1 - qt;  // longest rows first
    const int q0 = qt * BM;
    const size_t base = (size_t)bh * n * D;
    Q += base; K += base; V += base; dO += base; O += base; dQ += base; dKacc += base;
    if (kSites == 2) dVacc += base;
    L += (size_t)bh * n; Dv += (size_t)bh * n;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    load_tile<T, D>(Qs, Q, q0, n);
    load_tile<T, D>(dOs, dO, q0, n);
    const int kend = causal ? min(n, q0 + BM) : n;

    // ---- forward of these rows (as simt_fwd_kernel; the P tile goes through Ps)
    {
        float m[4], l[4], o[4][NC];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            m[a] = -INFINITY; l[a] = 0.f;
#pragma unroll
            for (int c = 0; c < NC; ++c) o[a][c] = 0.f;
        }
        for (int k0 = 0; k0 < kend; k0 += BN) {
            __syncthreads();
            load_tile<T, D>(Ks, K, k0, n);
            load_tile<T, D>(Vs, V, k0, n);
            __syncthreads();
            float s[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) s[a][b] = 0.f;
#pragma unroll 4
            for (int k = 0; k < D; ++k) {
                float qv[4], kv[4];
#pragma unroll
                for (int a = 0; a < 4; ++a) qv[a] = Qs[(ty * 4 + a) * LD + k];
#pragma unroll
                for (int b = 0; b < 4; ++b) kv[b] = Ks[(tx + 16 * b) * LD + k];
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) s[a][b] = fmaf(qv[a], kv[b], s[a][b]);
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int row = q0 + ty * 4 + a;
                float mx = -INFINITY;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const int col = k0 + tx + 16 * b;
                    float v = s[a][b] * scale;
                    if (col >= n || (causal && col > row)) v = -INFINITY;
                    s[a][b] = v;
                    mx = fmaxf(mx, v);
                }
                mx = group16_max(mx);
                float mn = fmaxf(m[a], mx);
                if (mn == -INFINITY) mn = 0.f;  // whole row masked so far (padding rows only)
                const float alpha = expf(m[a] - mn);
                float sum = 0.f;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const float pv = expf(s[a][b] - mn);
                    sum += pv;
                    Ps[(ty * 4 + a) * SLD + tx + 16 * b] = pv;
                }
                sum = group16_sum(sum);
                l[a] = l[a] * alpha + sum;
                m[a] = mn;
#pragma unroll
                for (int c = 0; c < NC; ++c) o[a][c] *= alpha;
            }
            __syncthreads();
#pragma unroll 4
            for (int j = 0; j < BN; ++j) {
                float pv[4], vv[NC];
#pragma unroll
                for (int a = 0; a < 4; ++a) pv[a] = Ps[(ty * 4 + a) * SLD + j];
#pragma unroll
                for (int c = 0; c < NC; ++c) vv[c] = Vs[j * LD + tx + 16 * c];
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int c = 0; c < NC; ++c) o[a][c] = fmaf(pv[a], vv[c], o[a][c]);
            }
        }
        // O, L, and D = rowsum(dO o O) from the fp32 O held here (the paper's precompute pass)
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int r = ty * 4 + a, row = q0 + r;
            const float inv = row < n ? 1.f / l[a] : 0.f;
            float dsum = 0.f;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                const float ov = o[a][c] * inv;
                dsum = fmaf(ov, dOs[r * LD + tx + 16 * c], dsum);
                if (row < n) O[(size_t)row * D + tx + 16 * c] = from_float<T>(ov);
            }
            dsum = group16_sum(dsum);
            if (tx == 0) {
                const float lse = row < n ? m[a] + logf(l[a]) : 0.f;
                Ls[r] = lse;
                Ds[r] = row < n ? dsum : 0.f;
                if (row < n) { L[row] = lse; Dv[row] = dsum; }
            }
        }
    }

    // ---- backward of the same rows
    float dq[4][NC];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < NC; ++c) dq[a][c] = 0.f;
    for (int k0 = 0; k0 < kend; k0 += BN) {
        __syncthreads();
        load_tile<T, D>(Ks, K, k0, n);
        load_tile<T, D>(Vs, V, k0, n);
        __syncthreads();
        bwd_tile_p_ds<D>(Qs, dOs, Ks, Vs, Ls, Ds, Ps, dSs, q0, k0, n, causal, scale, tx, ty);
        __syncthreads();
#pragma unroll 2
        for (int j = 0; j < BN; ++j) {
            float gv[4], kk[NC];
#pragma unroll
            for (int a = 0; a < 4; ++a) gv[a] = dSs[(ty * 4 + a) * SLD + j];
#pragma unroll
            for (int c = 0; c < NC; ++c) kk[c] = Ks[j * LD + tx + 16 * c];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < NC; ++c) dq[a][c] = fmaf(gv[a], kk[c], dq[a][c]);
        }
        // this tile pair's dK (and dV) contribution: [keys][d], thread (ty,tx) owns keys ty*4+a
        float dk[4][NC], dv[4][NC];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int c = 0; c < NC; ++c) { dk[a][c] = 0.f; dv[a][c] = 0.f; }
#pragma unroll 2
        for (int q = 0; q < BM; ++q) {
            float pv[4], gv[4], gq[NC], qq[NC];
#pragma unroll
            for (int a = 0; a < 4; ++a) { pv[a] = Ps[q * SLD + ty * 4 + a]; gv[a] = dSs[q * SLD + ty * 4 + a]; }
#pragma unroll
            for (int c = 0; c < NC; ++c) { gq[c] = dOs[q * LD + tx + 16 * c]; qq[c] = Qs[q * LD + tx + 16 * c]; }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    if (kSites == 2) dv[a][c] = fmaf(pv[a], gq[c], dv[a][c]);
                    dk[a][c] = fmaf(gv[a], qq[c], dk[a][c]);
                }
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int row = k0 + ty * 4 + a;
            if (row >= n) continue;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                atomicAdd(&dKacc[(size_t)row * D + tx + 16 * c], dk[a][c]);                     // atomic site GK
                if (kSites == 2) atomicAdd(&dVacc[(size_t)row * D + tx + 16 * c], dv[a][c]);    // atomic site GV
            }
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int row = q0 + ty * 4 + a;
        if (row >= n) continue;
#pragma unroll
        for (int c = 0; c < NC; ++c) dQ[(size_t)row * D + tx + 16 * c] = from_float<T>(dq[a][c]);
    }
}

// HBM-bound (4 bytes read, 2 written per element): grid-stride over float4 groups, four
// independent loads in flight per thread, streaming loads (the accumulator is not read again).
__global__ void __launch_bounds__(256)
convert_kernel(const float *__restrict__ src, __nv_bfloat16 *__restrict__ dst, size_t count, float mul)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");      // launched as a programmatic dependent of the kernel that fills src
    const size_t quads = count / 4;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    auto put = [&](size_t at, const float4 v) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v.x * mul, v.y * mul), b = __floats2bfloat162_rn(v.z * mul, v.w * mul);
        uint2 u;
        u.x = *reinterpret_cast<uint32_t *>(&a);
        u.y = *reinterpret_cast<uint32_t *>(&b);
        *reinterpret_cast<uint2 *>(dst + 4 * at) = u;
    };
    const float4 *s4 = reinterpret_cast<const float4 *>(src);
    for (; q + 3 * stride < quads; q += 4 * stride) {
        const float4 v0 = __ldcs(s4 + q), v1 = __ldcs(s4 + q + stride), v2 = __ldcs(s4 + q + 2 * stride),
                     v3 = __ldcs(s4 + q + 3 * stride);
        put(q, v0); put(q + stride, v1); put(q + 2 * stride, v2); put(q + 3 * stride, v3);
    }
    for (; q < quads; q += stride) put(q, __ldcs(s4 + q));
    if (blockIdx.x == 0 && threadIdx.x == 0)
        for (size_t i = quads * 4; i < count; ++i) dst[i] = __float2bfloat16_rn(src[i] * mul);
}

// The same conversion row by row, for an accumulator [B*H, n, src_ld] whose rows are wider than d
// and / or a [B,n,H,d] destination; one thread converts four consecutive elements of a row.
__global__ void __launch_bounds__(256)
convert_rows_kernel(const float *__restrict__ src, int src_ld, __nv_bfloat16 *__restrict__ dst, size_t rows, int n, int H,
                    int d, Strides ds, float mul)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int quads_per_row = d / 4;
    const size_t total = rows * (size_t)quads_per_row;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x; q < total; q += stride) {
        const size_t row = q / quads_per_row;             // flat (b*H + h)*n + r
        const int c4 = (int)(q - row * quads_per_row);
        const size_t bh = row / (size_t)n;
        const size_t r = row - bh * (size_t)n, bb = bh / (size_t)H, h = bh - bb * (size_t)H;
        const size_t doff = ds.at((long long)bb, (long long)h, (long long)r);
        const float4 v = __ldcs(reinterpret_cast<const float4 *>(src + row * (size_t)src_ld) + c4);
        __nv_bfloat162 a = __floats2bfloat162_rn(v.x * mul, v.y * mul), b = __floats2bfloat162_rn(v.z * mul, v.w * mul);
        uint2 u;
        u.x = *reinterpret_cast<uint32_t *>(&a);
        u.y = *reinterpret_cast<uint32_t *>(&b);
        *reinterpret_cast<uint2 *>(dst + doff + 4 * c4) = u;
    }
}

constexpr size_t fwd_smem(int D) { return (size_t)(3 * BM * (D + 1) + BM * SLD) * sizeof(float); }
constexpr size_t bwd_smem(int D) { return (size_t)(4 * BM * (D + 1) + 2 * BM * SLD + 2 * BM) * sizeof(float); }

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes)
{
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

template <typename T, int D>
cudaError_t fwd_t(const Problem &p, const void *Q, const void *K, const void *V, void *O, float *L, cudaStream_t st)
{
    const int nqt = (p.n + BM - 1) / BM;
    cudaError_t e = set_smem(simt_fwd_kernel<T, D>, fwd_smem(D));
    if (e != cudaSuccess) return e;
    LaunchScope scope(MOA_KERNEL_FWD, st);
    simt_fwd_kernel<T, D><<<(unsigned)(nqt * p.BH()), NTHREADS, fwd_smem(D), st>>>(
        (const T *)Q, (const T *)K, (const T *)V, (T *)O, L, p.n, p.causal, p.scale, nqt);
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t bwd_kv_t(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                     const float *L, const float *Dv, void *dK, void *dV, float *dQacc, cudaStream_t st)
{
    const int nkt = (p.n + BN - 1) / BN;
    cudaError_t e = set_smem(simt_bwd_kv_kernel<T, D>, bwd_smem(D));
    if (e != cudaSuccess) return e;
    LaunchScope scope(MOA_KERNEL_BWD_KV, st);
    simt_bwd_kv_kernel<T, D><<<(unsigned)(nkt * p.BH()), NTHREADS, bwd_smem(D), st>>>(
        (const T *)Q, (const T *)K, (const T *)V, (const T *)dO, L, Dv, (T *)dK, (T *)dV, dQacc,
        p.n, p.causal, p.scale, nkt);
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t bwd_dq_t(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                     const float *L, const float *Dv, void *dQ, cudaStream_t st)
{
    const int nqt = (p.n + BM - 1) / BM;
    cudaError_t e = set_smem(simt_bwd_dq_kernel<T, D>, bwd_smem(D));
    if (e != cudaSuccess) return e;
    LaunchScope scope(MOA_KERNEL_BWD_DQ, st);
    simt_bwd_dq_kernel<T, D><<<(unsigned)(nqt * p.BH()), NTHREADS, bwd_smem(D), st>>>(
        (const T *)Q, (const T *)K, (const T *)V, (const T *)dO, L, Dv, (T *)dQ, p.n, p.causal, p.scale, nqt);
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t rowpar_t(const Problem &p, const void *Q, const void *K, const void *V, const void *dO, void *O, float *L,
                     float *Dv, void *dQ, float *dKacc, float *dVacc, int sites, cudaStream_t st)
{
    const int nqt = (p.n + BM - 1) / BM;
    cudaError_t e = set_smem(simt_rowpar_kernel<T, D, 1>, bwd_smem(D));
    if (e == cudaSuccess) e = set_smem(simt_rowpar_kernel<T, D, 2>, bwd_smem(D));
    if (e != cudaSuccess) return e;
    LaunchScope scope(MOA_KERNEL_OTHER, st);
    if (sites == 2)
        simt_rowpar_kernel<T, D, 2><<<(unsigned)(nqt * p.BH()), NTHREADS, bwd_smem(D), st>>>(
            (const T *)Q, (const T *)K, (const T *)V, (const T *)dO, (T *)O, L, Dv, (T *)dQ, dKacc, dVacc,
            p.n, p.causal, p.scale, nqt);
    else
        simt_rowpar_kernel<T, D, 1><<<(unsigned)(nqt * p.BH()), NTHREADS, bwd_smem(D), st>>>(
            (const T *)Q, (const T *)K, (const T *)V, (const T *)dO, (T *)O, L, Dv, (T *)dQ, dKacc, dVacc,
            p.n, p.causal, p.scale, nqt);
    return cudaGetLastError();
}

#define MOA_DISPATCH(FN, ...)                                                         \
    do {                                                                              \
        if (dtype == MOA_F32) {                                                       \
            if (p.d == 64) return FN<float, 64>(__VA_ARGS__);                         \
            if (p.d == 128) return FN<float, 128>(__VA_ARGS__);                       \
        } else {                                                                      \
            if (p.d == 64) return FN<__nv_bfloat16, 64>(__VA_ARGS__);                 \
            if (p.d == 128) return FN<__nv_bfloat16, 128>(__VA_ARGS__);               \
        }                                                                             \
        return cudaErrorInvalidValue;                                                 \
    } while (0)

}  // namespace

cudaError_t simt_fwd(const Problem &p, int dtype, const void *Q, const void *K, const void *V,
                     void *O, float *L, cudaStream_t st)
{
    MOA_DISPATCH(fwd_t, p, Q, K, V, O, L, st);
}

cudaError_t simt_bwd_kv(const Problem &p, int dtype, const void *Q, const void *K, const void *V,
                        const void *dO, const float *L, const float *Dv,
                        void *dK, void *dV, float *dQacc, cudaStream_t st)
{
    MOA_DISPATCH(bwd_kv_t, p, Q, K, V, dO, L, Dv, dK, dV, dQacc, st);
}

cudaError_t simt_rowpar(const Problem &p, int dtype, const void *Q, const void *K, const void *V, const void *dO,
                        void *O, float *L, float *Dv, void *dQ, float *dKacc, float *dVacc, int sites, cudaStream_t st)
{
    MOA_DISPATCH(rowpar_t, p, Q, K, V, dO, O, L, Dv, dQ, dKacc, dVacc, sites, st);
}

cudaError_t simt_bwd_dq(const Problem &p, int dtype, const void *Q, const void *K, const void *V,
                        const void *dO, const float *L, const float *Dv, void *dQ, cudaStream_t st)
{
    MOA_DISPATCH(bwd_dq_t, p, Q, K, V, dO, L, Dv, dQ, st);
}

cudaError_t row_dot(const Problem &p, int dtype, const void *dO, const void *O, float *Dv, cudaStream_t st)
{
    const size_t rows = (size_t)p.BH() * p.n;
    const int wpb = 8;
    const unsigned grid = (unsigned)((rows + wpb - 1) / wpb);
    LaunchScope scope(MOA_KERNEL_PREPROCESS, st);
    if (dtype == MOA_F32)
        row_dot_kernel<float><<<grid, wpb * 32, 0, st>>>((const float *)dO, (const float *)O, Dv, rows, p.d);
    else
        row_dot_kernel<__nv_bfloat16><<<grid, wpb * 32, 0, st>>>((const __nv_bfloat16 *)dO,
                                                                 (const __nv_bfloat16 *)O, Dv, rows, p.d);
    return cudaGetLastError();
}

cudaError_t convert_f32_to_bf16(const float *src, void *dst, size_t count, float mul, cudaStream_t st)
{
    const size_t quads = (count + 3) / 4;
    size_t blocks = (quads + 4 * 256 - 1) / (4 * 256);
    if (blocks < 1) blocks = 1;
    if (blocks > 16LL * device_info().sms) blocks = 16LL * device_info().sms;     // grid-stride beyond 16 blocks per SM
    const unsigned grid = (unsigned)blocks;
    LaunchScope scope(MOA_KERNEL_CONVERT, st);
    return launch_dependent(convert_kernel, dim3(grid), dim3(256), (size_t)0, st, src, (__nv_bfloat16 *)dst, count, mul);
}

cudaError_t convert_f32_to_bf16_rows(const float *src, int src_ld, void *dst, int B, int H, int n, int d, Strides ds,
                                     float mul, cudaStream_t st)
{
    const size_t rows = (size_t)B * H * n, quads = rows * (size_t)(d / 4);
    size_t blocks = (quads + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > 16LL * device_info().sms) blocks = 16LL * device_info().sms;
    LaunchScope scope(MOA_KERNEL_CONVERT, st);
    return launch_dependent(convert_rows_kernel, dim3((unsigned)blocks), dim3(256), (size_t)0, st, src, src_ld, (__nv_bfloat16 *)dst, rows, n, H, d,
                            ds, mul);
}

}  // namespace moa
