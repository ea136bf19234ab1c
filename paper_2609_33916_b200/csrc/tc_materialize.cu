// The n x n-materialising comparison variant (desc.materialize = 1), bf16, tensor cores.
//
// This is the paper's "left" realisation (Sec. 1.1): the probability array A = P and the
// gradient array GS = dS are written to device memory and read back, and dQ is computed
// atomic-free by a standalone pass that re-reads the persisted GS (Sec. 4, the GK-atomic
// removal).  It exists only to be measured against the fused path.  Both arrays are stored
// transposed, [key][query] per head with a row stride of n_pad = ceil(n/128)*128, because
// the key-parallel backward reads them by key row.
//
//   mat_fwd_kernel   query-parallel, two passes over the key tiles: pass 1 row max / row sum
//                    (-> L), pass 2 P = exp(S - L) written to HBM (as P^T) and O += P V.
//   mat_bwd_kernel   key-parallel: reads P^T rows from HBM (no recomputation), dP^T = V dO^T,
//                    dS^T = P^T o (dP^T - D) written to HBM, dV += P^T dO, dK += dS^T Q.
//   mat_dq_kernel    query-parallel GEMM dQ = scale * dS K reading dS^T tiles from HBM by TMA.
//
// n^2 traffic per head: P^T written once and read once, dS^T written once and read once
// (8 n_pad^2 bytes), against none for the fused path.
#include "common.cuh"
#include "ptx.cuh"
#include "tensormap.cuh"

namespace moa {
namespace {

using namespace ptx;

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kBoxBytes = 128 * 128;

__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

struct DescParts {
    uint32_t km_lo, km_hi, mn_lo, mn_hi;
};
__device__ __forceinline__ DescParts desc_parts()
{
    const uint64_t km = smem_desc_sw128(0, 16, 1024), mn = smem_desc_sw128(0, kBoxBytes, 1024);
    return DescParts{(uint32_t)km, (uint32_t)(km >> 32), (uint32_t)mn, (uint32_t)(mn >> 32)};
}
__device__ __forceinline__ uint32_t addr_field(const void *p) { return (smem_u32(p) >> 4) & 0x3FFFu; }
__device__ __forceinline__ uint32_t koff(int ks) { return (uint32_t)(((ks / 4) * kBoxBytes + (ks % 4) * 32) >> 4); }
__device__ __forceinline__ uint32_t moff(int ks) { return (uint32_t)((ks * 2048) >> 4); }

// ================================================================== forward, materialising
enum : uint32_t { FERR = 0x400 };

template <int D>
__global__ void __launch_bounds__(192, 1)
mat_fwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
               const __grid_constant__ CUtensorMap mapV, __nv_bfloat16 *__restrict__ O, float *__restrict__ L,
               __nv_bfloat16 *__restrict__ PT, int n, int n_pad, int causal, float scale_log2, int nqt, int hpg,
               unsigned int *status)
{
    constexpr int kTile = 128 * D * 2;
    constexpr int kBoxes = D / 64;
    constexpr uint32_t colS = 0, colO = 128;
    extern __shared__ __align__(1024) uint8_t sm[];
    uint8_t *sQ = sm, *sK = sm + kTile, *sV = sm + 2 * kTile;
    uint64_t *bars = reinterpret_cast<uint64_t *>(sm + 3 * kTile);
    uint64_t *bar_q = bars, *bar_k = bars + 1, *bar_v = bars + 2, *bar_s = bars + 3, *bar_p = bars + 4, *bar_o = bars + 5;
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bars + 6);
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(bars + 7);

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    int bh, t;
    job_from_block((int)blockIdx.x, nqt, (int)gridDim.x / nqt, hpg, bh, t);
    const int qt = causal ? nqt - 1 - t : t;
    const int q0 = qt * 128;
    const int nkt_all = n_pad / 128;
    const int nkt_want = causal ? min(qt + 1, nkt_all) : nkt_all;

    if (tid == 0) {
        mbar_init(bar_q, 1); mbar_init(bar_k, 1); mbar_init(bar_v, 1);
        mbar_init(bar_s, 1); mbar_init(bar_p, 128); mbar_init(bar_o, 1);
        *abortp = (smem_u32(sm) & 1023u) ? 1u : 0u;
        if (*abortp && status) atomicCAS(status, 0u, FERR + 8u);
        fence_mbar_init();
    }
    if (warp == 5) { tmem_alloc(tmem_base_s, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_base_s;
    const int nkt = (*abortp == 0) ? nkt_want : 0;
    const int total = 2 * nkt;   // pass 1: statistics; pass 2: P out, O += P V

    if (warp == 4) {
        ArmCounts<6> armed;     // barriers armed for copies into shared memory
        if (lane == 0 && nkt > 0) {
            mbar_arm(bars, bar_q, kTile, armed);
            for (int b = 0; b < kBoxes; ++b) tma_load_3d(sQ + b * kBoxBytes, &mapQ, bar_q, 64 * b, q0, bh);
        }
        for (int jj = 0; jj < total; ++jj) {
            const int pass2 = jj >= nkt, j = jj - pass2 * nkt;
            if (jj > 0 && !mbar_wait(bar_s, (jj - 1) & 1, abortp, status, FERR + 1)) break;   // K buffer free
            if (lane == 0) {
                mbar_arm(bars, bar_k, kTile, armed);
                for (int b = 0; b < kBoxes; ++b) tma_load_3d(sK + b * kBoxBytes, &mapK, bar_k, 64 * b, j * 128, bh);
            }
            if (pass2) {
                if (j > 0 && !mbar_wait(bar_o, (j - 1) & 1, abortp, status, FERR + 2)) break;  // V buffer free
                if (lane == 0) {
                    mbar_arm(bars, bar_v, kTile, armed);
                    for (int b = 0; b < kBoxes; ++b) tma_load_3d(sV + b * kBoxBytes, &mapV, bar_v, 64 * b, j * 128, bh);
                }
            }
            __syncwarp();
        }
        if (lane == 0) mbar_drain(bars, armed);     // copies still on their way land before the CTA leaves (bounded)
    } else if (warp == 5 && lane == 0) {
        constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);
        constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, 0, 1);
        const DescParts dp = desc_parts();
        const uint32_t q_lo = dp.km_lo + addr_field(sQ), k_lo = dp.km_lo + addr_field(sK), v_lo = dp.mn_lo + addr_field(sV);
        bool ok = nkt > 0 && mbar_wait(bar_q, 0, abortp, status, FERR + 3);
        for (int jj = 0; ok && jj < total; ++jj) {
            const int pass2 = jj >= nkt, j = jj - pass2 * nkt;
            if (!mbar_wait(bar_k, jj & 1, abortp, status, FERR + 4)) break;
            tc_fence_after();
            umma_ss2<false>(tbase + colS, q_lo, dp.km_hi, k_lo, dp.km_hi, idesc_s);
#pragma unroll
            for (int ks = 1; ks < D / 16; ++ks)
                umma_ss2<true>(tbase + colS, q_lo + koff(ks), dp.km_hi, k_lo + koff(ks), dp.km_hi, idesc_s);
            umma_commit(bar_s);
            if (pass2 && !mbar_wait(bar_v, j & 1, abortp, status, FERR + 5)) break;
            if (!mbar_wait(bar_p, jj & 1, abortp, status, FERR + 6)) break;   // threads are done with S
            tc_fence_after();
            if (pass2) {
                if (j > 0) umma_ts2<true>(tbase + colO, tbase + colS, v_lo, dp.mn_hi, idesc_pv);
                else       umma_ts2<false>(tbase + colO, tbase + colS, v_lo, dp.mn_hi, idesc_pv);
#pragma unroll
                for (int ks = 1; ks < 8; ++ks)
                    umma_ts2<true>(tbase + colO, tbase + colS + ks * 8, v_lo + moff(ks), dp.mn_hi, idesc_pv);
                umma_commit(bar_o);
            }
        }
    } else if (warp < 4) {
        const int row = q0 + tid;
        const uint32_t lane_addr = tbase + ((uint32_t)(warp * 32) << 16);
        float m = -INFINITY, l = 0.f, L2 = 0.f;
        bool ok = nkt > 0;
        for (int jj = 0; ok && jj < total; ++jj) {
            const int pass2 = jj >= nkt, j = jj - pass2 * nkt;
            if (jj == nkt) L2 = ((m == -INFINITY) ? 0.f : m) + log2f(l);
            if (!mbar_wait(bar_s, jj & 1, abortp, status, FERR + 7)) { ok = false; break; }
            tc_fence_after();
            const int k0 = j * 128;
            const bool need_mask = (k0 + 128 > n) || (causal && k0 + 127 > q0);
            uint32_t r[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld(lane_addr + colS + 32 * c, r[c]);
            tc_wait_ld();
            if (need_mask) {
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int col = k0 + 32 * c + i;
                        if (col >= n || (causal && col > row)) r[c][i] = 0xff800000u;   // -inf
                    }
            }
            if (!pass2) {
                float mx = -INFINITY;
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(r[c][i]));
                mx *= scale_log2;
                const float mn = fmaxf(m, mx);
                const float mref = (mn == -INFINITY) ? 0.f : mn;
                float sum = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i) sum += ex2(fmaf(__uint_as_float(r[c][i]), scale_log2, -mref));
                l = l * ex2(m - mref) + sum;
                m = mn;
            } else {
                __nv_bfloat16 *pt = PT + ((size_t)bh * n_pad + k0) * n_pad + row;   // P^T[key][query]
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const float p0 = ex2(fmaf(__uint_as_float(r[c][i]), scale_log2, -L2));
                        const float p1 = ex2(fmaf(__uint_as_float(r[c][i + 1]), scale_log2, -L2));
                        pk[i / 2] = pack_bf16(p0, p1);
                        // one probability per store; a warp covers 32 consecutive queries of one key row
                        reinterpret_cast<unsigned short *>(pt)[(size_t)(32 * c + i) * n_pad] = (unsigned short)(pk[i / 2] & 0xffffu);
                        reinterpret_cast<unsigned short *>(pt)[(size_t)(32 * c + i + 1) * n_pad] = (unsigned short)(pk[i / 2] >> 16);
                    }
                    tmem_st(lane_addr + colS + 16 * c, pk);
                }
                tc_wait_st();
            }
            tc_fence_before();
            mbar_arrive(bar_p);
        }
        if (ok && mbar_wait(bar_o, (nkt - 1) & 1, abortp, status, FERR + 9)) {
            tc_fence_after();
            __nv_bfloat16 *orow = O + ((size_t)bh * n + row) * D;
#pragma unroll
            for (int c = 0; c < D; c += 32) {
                uint32_t o[32];
                tmem_ld(lane_addr + colO + c, o);
                tc_wait_ld();
                if (row < n) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(o[i + 0]), __uint_as_float(o[i + 1]));
                        v.y = pack_bf16(__uint_as_float(o[i + 2]), __uint_as_float(o[i + 3]));
                        v.z = pack_bf16(__uint_as_float(o[i + 4]), __uint_as_float(o[i + 5]));
                        v.w = pack_bf16(__uint_as_float(o[i + 6]), __uint_as_float(o[i + 7]));
                        *reinterpret_cast<uint4 *>(orow + c + i) = v;
                    }
                }
            }
            if (row < n) L[(size_t)bh * n + row] = L2 * kLn2;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) tmem_dealloc(tbase, 256);
}

// ================================================================= backward, materialising
enum : uint32_t { BERR = 0x500 };
enum { MB_KV = 0, MB_QFULL = 1 /*2*/, MB_QEMPTY = 3 /*2*/, MB_DOFULL = 5 /*2*/, MB_DOEMPTY = 7 /*2*/, MB_P = 9, MB_DP = 10,
       MB_DS = 11, MB_ITER = 12, MB_COUNT = 13 };

template <int D>
struct MatBwdSmem {
    static constexpr int kTile = 128 * D * 2;
    static constexpr int offK = 0, offV = kTile, offQ = 2 * kTile, offdO = 4 * kTile, offD = 6 * kTile /*2 x 512 B*/;
    static constexpr int offBar = offD + 1024;
    static constexpr int kTotal = offBar + 128;
};

template <int D>
__global__ void __launch_bounds__(320, 1)
mat_bwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
               const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapdO,
               const float *__restrict__ Dp, const __nv_bfloat16 *__restrict__ PT, __nv_bfloat16 *__restrict__ GST,
               __nv_bfloat16 *__restrict__ dK, __nv_bfloat16 *__restrict__ dV,
               int n, int n_pad, int causal, float scale, int nkt, int hpg, unsigned int *status)
{
    using SM = MatBwdSmem<D>;
    constexpr int kBoxes = D / 64;
    constexpr uint32_t colP = 0, colDP = 128, colDV = 256, colDK = 256 + D;
    extern __shared__ __align__(1024) uint8_t sm[];
    float *sD = reinterpret_cast<float *>(sm + SM::offD);
    uint64_t *bars = reinterpret_cast<uint64_t *>(sm + SM::offBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bars + MB_COUNT);
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(bars + MB_COUNT + 1);

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    int bh, kt;
    job_from_block((int)blockIdx.x, nkt, (int)gridDim.x / nkt, hpg, bh, kt);
    const int k0 = kt * 128;
    const int nqt = n_pad / 128;
    const int i_begin = causal ? kt : 0;

    if (tid == 0) {
        for (int b = 0; b < MB_COUNT; ++b) mbar_init(bars + b, (b == MB_P || b == MB_DS) ? 256u : 1u);
        *abortp = (smem_u32(sm) & 1023u) ? 1u : 0u;
        if (*abortp && status) atomicCAS(status, 0u, BERR + 8u);
        fence_mbar_init();
    }
    if (warp == 9) { tmem_alloc(tmem_base_s, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_base_s;
    const int niter = (*abortp == 0) ? (nqt - i_begin) : 0;

    if (warp == 8) {
        ArmCounts<MB_COUNT> armed;     // barriers armed for copies into shared memory
        if (lane == 0 && niter > 0) {
            mbar_arm(bars, bars + MB_KV, 2 * SM::kTile, armed);
            for (int b = 0; b < kBoxes; ++b) {
                tma_load_3d(sm + SM::offK + b * kBoxBytes, &mapK, bars + MB_KV, 64 * b, k0, bh);
                tma_load_3d(sm + SM::offV + b * kBoxBytes, &mapV, bars + MB_KV, 64 * b, k0, bh);
            }
        }
        for (int it = 0; it < niter; ++it) {
            const int s = it & 1, q0 = (i_begin + it) * 128;
            if (it >= 2 && !mbar_wait(bars + MB_DOEMPTY + s, ((it >> 1) - 1) & 1, abortp, status, BERR + 1)) break;
            if (lane == 0) {
                mbar_arm(bars, bars + MB_DOFULL + s, SM::kTile, armed);
                for (int b = 0; b < kBoxes; ++b)
                    tma_load_3d(sm + SM::offdO + s * SM::kTile + b * kBoxBytes, &mapdO, bars + MB_DOFULL + s, 64 * b, q0, bh);
            }
            if (it >= 2 && !mbar_wait(bars + MB_QEMPTY + s, ((it >> 1) - 1) & 1, abortp, status, BERR + 2)) break;
            if (lane == 0) {
                mbar_arm(bars, bars + MB_QFULL + s, SM::kTile + 512, armed);
                for (int b = 0; b < kBoxes; ++b)
                    tma_load_3d(sm + SM::offQ + s * SM::kTile + b * kBoxBytes, &mapQ, bars + MB_QFULL + s, 64 * b, q0, bh);
                bulk_load_1d(sD + s * 128, Dp + (size_t)bh * n_pad + q0, 512, bars + MB_QFULL + s);
            }
            __syncwarp();
        }
        if (lane == 0) mbar_drain(bars, armed);     // copies still on their way land before the CTA leaves (bounded)
    } else if (warp == 9 && lane == 0) {
        constexpr uint32_t idesc_st = idesc_bf16_f32(128, 128, 0, 0);
        constexpr uint32_t idesc_acc = idesc_bf16_f32(128, D, 0, 1);
        const DescParts dp = desc_parts();
        const uint32_t v_km = dp.km_lo + addr_field(sm + SM::offV);
        const uint32_t q_mn0 = dp.mn_lo + addr_field(sm + SM::offQ);
        const uint32_t do_km0 = dp.km_lo + addr_field(sm + SM::offdO), do_mn0 = dp.mn_lo + addr_field(sm + SM::offdO);
        constexpr uint32_t kSlot = (uint32_t)(SM::kTile >> 4);
        bool ok = niter > 0 && mbar_wait(bars + MB_KV, 0, abortp, status, BERR + 3);
        for (int it = 0; ok && it < niter; ++it) {
            const int s = it & 1;
            const uint32_t q_mn = q_mn0 + s * kSlot, do_km = do_km0 + s * kSlot, do_mn = do_mn0 + s * kSlot;
            if (!mbar_wait(bars + MB_DOFULL + s, (it >> 1) & 1, abortp, status, BERR + 4)) break;
            tc_fence_after();
            // dP^T(it): its columns still hold dS^T(it-1), read by dK(it-1), issued earlier
            umma_ss2<false>(tbase + colDP, v_km, dp.km_hi, do_km, dp.km_hi, idesc_st);
#pragma unroll
            for (int ks = 1; ks < D / 16; ++ks)
                umma_ss2<true>(tbase + colDP, v_km + koff(ks), dp.km_hi, do_km + koff(ks), dp.km_hi, idesc_st);
            umma_commit(bars + MB_DP);
            if (!mbar_wait(bars + MB_P, it & 1, abortp, status, BERR + 5)) break;
            tc_fence_after();
            if (it > 0) umma_ts2<true>(tbase + colDV, tbase + colP, do_mn, dp.mn_hi, idesc_acc);
            else        umma_ts2<false>(tbase + colDV, tbase + colP, do_mn, dp.mn_hi, idesc_acc);
#pragma unroll
            for (int ks = 1; ks < 8; ++ks)
                umma_ts2<true>(tbase + colDV, tbase + colP + 64 * (ks / 4) + 8 * (ks % 4), do_mn + moff(ks), dp.mn_hi, idesc_acc);
            umma_commit(bars + MB_DOEMPTY + s);
            if (!mbar_wait(bars + MB_QFULL + s, (it >> 1) & 1, abortp, status, BERR + 6)) break;
            if (!mbar_wait(bars + MB_DS, it & 1, abortp, status, BERR + 7)) break;
            tc_fence_after();
            if (it > 0) umma_ts2<true>(tbase + colDK, tbase + colDP, q_mn, dp.mn_hi, idesc_acc);
            else        umma_ts2<false>(tbase + colDK, tbase + colDP, q_mn, dp.mn_hi, idesc_acc);
#pragma unroll
            for (int ks = 1; ks < 8; ++ks)
                umma_ts2<true>(tbase + colDK, tbase + colDP + 64 * (ks / 4) + 8 * (ks % 4), q_mn + moff(ks), dp.mn_hi, idesc_acc);
            umma_commit(bars + MB_QEMPTY + s);
            umma_commit(bars + MB_ITER);
        }
    } else if (warp < 8) {
        const int wg = warp / 4;
        const int lane_row = 32 * (warp % 4) + lane;   // key inside the tile
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        const size_t arr_row = ((size_t)bh * n_pad + k0 + lane_row) * n_pad;   // this key's row of P^T / dS^T
        bool ok = niter > 0;
        for (int it = 0; ok && it < niter; ++it) {
            const int s = it & 1, q0 = (i_begin + it) * 128;
            // P^T(it) from HBM: 64 probabilities (128 bytes) of this key row, already packed as the UMMA wants them
            uint32_t pk[2][16];
            const uint4 *src = reinterpret_cast<const uint4 *>(PT + arr_row + q0 + 64 * wg);
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                const uint4 x = src[v];
                pk[v / 4][4 * (v % 4)] = x.x; pk[v / 4][4 * (v % 4) + 1] = x.y;
                pk[v / 4][4 * (v % 4) + 2] = x.z; pk[v / 4][4 * (v % 4) + 3] = x.w;
            }
            // the TMEM columns of P^T(it-1) are free once dV(it-1) and dK(it-1) have completed
            if (it > 0 && !mbar_wait(bars + MB_ITER, (it - 1) & 1, abortp, status, BERR + 9)) { ok = false; break; }
            tc_fence_after();
            tmem_st(lane_addr + colP + 64 * wg, pk[0]);
            tmem_st(lane_addr + colP + 64 * wg + 16, pk[1]);
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bars + MB_P);

            if (!mbar_wait(bars + MB_DP, it & 1, abortp, status, BERR + 10)) { ok = false; break; }
            if (!mbar_wait(bars + MB_QFULL + s, (it >> 1) & 1, abortp, status, BERR + 11)) { ok = false; break; }   // D_i is there
            tc_fence_after();
            const float *Ds = sD + s * 128;
            uint4 *dst = reinterpret_cast<uint4 *>(GST + arr_row + q0 + 64 * wg);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t rd[32], gk[16];
                tmem_ld(lane_addr + colDP + 64 * wg + 32 * c, rd);
                tc_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const uint32_t pp = pk[c][e / 2];
                    const float p0 = __uint_as_float(pp << 16), p1 = __uint_as_float(pp & 0xffff0000u);
                    const float2 d2 = *reinterpret_cast<const float2 *>(Ds + 64 * wg + 32 * c + e);
                    gk[e / 2] = pack_bf16(p0 * (__uint_as_float(rd[e]) + d2.x), p1 * (__uint_as_float(rd[e + 1]) + d2.y));   // Dp holds -D
                }
                tmem_st(lane_addr + colDP + 64 * wg + 16 * c, gk);
#pragma unroll
                for (int v = 0; v < 4; ++v) dst[4 * c + v] = make_uint4(gk[4 * v], gk[4 * v + 1], gk[4 * v + 2], gk[4 * v + 3]);
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bars + MB_DS);
        }
        if (ok && mbar_wait(bars + MB_ITER, (niter - 1) & 1, abortp, status, BERR + 12)) {
            tc_fence_after();
            const int krow = k0 + lane_row;
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const uint32_t col = (which == 0 ? colDV : colDK) + (D / 2) * wg;
                const float mul = which == 0 ? 1.f : scale;
                __nv_bfloat16 *outp = (which == 0 ? dV : dK) + ((size_t)bh * n + krow) * D + (D / 2) * wg;
#pragma unroll
                for (int c = 0; c < D / 2; c += 32) {
                    uint32_t r[32];
                    tmem_ld(lane_addr + col + c, r);
                    tc_wait_ld();
                    if (krow < n) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            uint4 v;
                            v.x = pack_bf16(__uint_as_float(r[e + 0]) * mul, __uint_as_float(r[e + 1]) * mul);
                            v.y = pack_bf16(__uint_as_float(r[e + 2]) * mul, __uint_as_float(r[e + 3]) * mul);
                            v.z = pack_bf16(__uint_as_float(r[e + 4]) * mul, __uint_as_float(r[e + 5]) * mul);
                            v.w = pack_bf16(__uint_as_float(r[e + 6]) * mul, __uint_as_float(r[e + 7]) * mul);
                            *reinterpret_cast<uint4 *>(outp + c + e) = v;
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tbase, 512);
}

// ======================================================== dQ = scale * dS K from the persisted dS^T
enum : uint32_t { QERR = 0x600 };

template <int D>
__global__ void __launch_bounds__(192, 1)
mat_dq_kernel(const __grid_constant__ CUtensorMap mapGST, const __grid_constant__ CUtensorMap mapK,
              __nv_bfloat16 *__restrict__ dQ, int n, int n_pad, int causal, float scale, int nqt, int hpg, unsigned int *status)
{
    constexpr int kTileK = 128 * D * 2, kTileG = 128 * 128 * 2;
    constexpr int kBoxes = D / 64;
    extern __shared__ __align__(1024) uint8_t sm[];
    uint8_t *sG = sm /*2 slots*/, *sK = sm + 2 * kTileG /*2 slots*/;
    uint64_t *bars = reinterpret_cast<uint64_t *>(sm + 2 * kTileG + 2 * kTileK);
    uint64_t *bar_full = bars /*2*/, *bar_empty = bars + 2 /*2*/, *bar_done = bars + 4;
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bars + 5);
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(bars + 6);

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    int bh, t;
    job_from_block((int)blockIdx.x, nqt, (int)gridDim.x / nqt, hpg, bh, t);
    const int qt = causal ? nqt - 1 - t : t;
    const int q0 = qt * 128;
    const int nkt_all = n_pad / 128;
    const int nkt_want = causal ? min(qt + 1, nkt_all) : nkt_all;

    if (tid == 0) {
        for (int b = 0; b < 5; ++b) mbar_init(bars + b, 1);
        *abortp = (smem_u32(sm) & 1023u) ? 1u : 0u;
        if (*abortp && status) atomicCAS(status, 0u, QERR + 8u);
        fence_mbar_init();
    }
    if (warp == 5) { tmem_alloc(tmem_base_s, 128); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_base_s;
    const int nkt = (*abortp == 0) ? nkt_want : 0;

    if (warp == 4) {
        ArmCounts<5> armed;     // barriers armed for copies into shared memory
        for (int j = 0; j < nkt; ++j) {
            const int s = j & 1;
            if (j >= 2 && !mbar_wait(bar_empty + s, ((j >> 1) - 1) & 1, abortp, status, QERR + 1)) break;
            if (lane == 0) {
                mbar_arm(bars, bar_full + s, kTileG + kTileK, armed);
                // dS^T tile: rows = keys j*128.., columns = queries q0.. (two 64-column boxes)
                for (int b = 0; b < 2; ++b)
                    tma_load_3d(sG + s * kTileG + b * kBoxBytes, &mapGST, bar_full + s, q0 + 64 * b, j * 128, bh);
                for (int b = 0; b < kBoxes; ++b)
                    tma_load_3d(sK + s * kTileK + b * kBoxBytes, &mapK, bar_full + s, 64 * b, j * 128, bh);
            }
            __syncwarp();
        }
        if (lane == 0) mbar_drain(bars, armed);     // copies still on their way land before the CTA leaves (bounded)
    } else if (warp == 5 && lane == 0) {
        constexpr uint32_t idesc = idesc_bf16_f32(128, D, 1, 1);   // A = dS^T tile (MN-major), B = K (MN-major)
        const DescParts dp = desc_parts();
        const uint32_t g_mn0 = dp.mn_lo + addr_field(sG), k_mn0 = dp.mn_lo + addr_field(sK);
        for (int j = 0; j < nkt; ++j) {
            const int s = j & 1;
            const uint32_t g_mn = g_mn0 + s * (uint32_t)(kTileG >> 4), k_mn = k_mn0 + s * (uint32_t)(kTileK >> 4);
            if (!mbar_wait(bar_full + s, (j >> 1) & 1, abortp, status, QERR + 2)) break;
            tc_fence_after();
            if (j > 0) umma_ss2<true>(tbase, g_mn, dp.mn_hi, k_mn, dp.mn_hi, idesc);
            else       umma_ss2<false>(tbase, g_mn, dp.mn_hi, k_mn, dp.mn_hi, idesc);
#pragma unroll
            for (int ks = 1; ks < 8; ++ks) umma_ss2<true>(tbase, g_mn + moff(ks), dp.mn_hi, k_mn + moff(ks), dp.mn_hi, idesc);
            umma_commit(bar_empty + s);
            if (j == nkt - 1) umma_commit(bar_done);
        }
    } else if (warp < 4) {
        if (nkt > 0 && mbar_wait(bar_done, 0, abortp, status, QERR + 3)) {
            tc_fence_after();
            const int qrow = q0 + tid;
            const uint32_t lane_addr = tbase + ((uint32_t)(warp * 32) << 16);
            __nv_bfloat16 *outp = dQ + ((size_t)bh * n + qrow) * D;
#pragma unroll
            for (int c = 0; c < D; c += 32) {
                uint32_t r[32];
                tmem_ld(lane_addr + c, r);
                tc_wait_ld();
                if (qrow < n) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(r[e + 0]) * scale, __uint_as_float(r[e + 1]) * scale);
                        v.y = pack_bf16(__uint_as_float(r[e + 2]) * scale, __uint_as_float(r[e + 3]) * scale);
                        v.z = pack_bf16(__uint_as_float(r[e + 4]) * scale, __uint_as_float(r[e + 5]) * scale);
                        v.w = pack_bf16(__uint_as_float(r[e + 6]) * scale, __uint_as_float(r[e + 7]) * scale);
                        *reinterpret_cast<uint4 *>(outp + c + e) = v;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) tmem_dealloc(tbase, 128);
}

template <int D>
cudaError_t run_group(const Problem &p, const void *Q, const void *K, const void *V, const void *dO, void *O, float *L,
                      const float *Dp_group, void *PT, void *GST, void *dQ, void *dK, void *dV, int stage, cudaStream_t st)
{
    // stage 0: forward (P^T out); stage 1: backward (needs Dp of this head group)
    const uint64_t heads = (uint64_t)p.BH();
    const int nt = (p.n + 127) / 128, n_pad = nt * 128;
    CUtensorMap mq, mk, mv, mdo, mg;
    if (!make_tensor_map_3d(&mq, Q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64) ||
        !make_tensor_map_3d(&mk, K, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64) ||
        !make_tensor_map_3d(&mv, V, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64))
        return cudaErrorInvalidValue;
    cudaError_t e;
    if (stage == 0) {
        constexpr int kSmem = 3 * 128 * D * 2 + 128;
        if ((e = cudaFuncSetAttribute(mat_fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem)) != cudaSuccess) return e;
        LaunchScope scope(MOA_KERNEL_FWD, st);
        mat_fwd_kernel<D><<<(unsigned)(nt * p.BH()), 192, kSmem, st>>>(mq, mk, mv, (__nv_bfloat16 *)O, L, (__nv_bfloat16 *)PT,
                                                                      p.n, n_pad, p.causal, p.scale * kLog2e, nt,
                                                                      heads_per_group(p, nt), device_status_ptr());
        return cudaGetLastError();
    }
    if (!make_tensor_map_3d(&mdo, dO, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64) ||
        !make_tensor_map_3d(&mg, GST, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, n_pad, n_pad, 128, 64))
        return cudaErrorInvalidValue;
    {
        constexpr int kSmem = MatBwdSmem<D>::kTotal;
        if ((e = cudaFuncSetAttribute(mat_bwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem)) != cudaSuccess) return e;
        LaunchScope scope(MOA_KERNEL_BWD_KV, st);
        mat_bwd_kernel<D><<<(unsigned)(nt * p.BH()), 320, kSmem, st>>>(mq, mk, mv, mdo, Dp_group, (const __nv_bfloat16 *)PT,
                                                                      (__nv_bfloat16 *)GST, (__nv_bfloat16 *)dK,
                                                                      (__nv_bfloat16 *)dV, p.n, n_pad, p.causal, p.scale, nt,
                                                                      heads_per_group(p, nt), device_status_ptr());
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    {
        constexpr int kSmem = 2 * 128 * 128 * 2 + 2 * 128 * D * 2 + 128;
        if ((e = cudaFuncSetAttribute(mat_dq_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem)) != cudaSuccess) return e;
        LaunchScope scope(MOA_KERNEL_BWD_DQ, st);
        mat_dq_kernel<D><<<(unsigned)(nt * p.BH()), 192, kSmem, st>>>(mg, mk, (__nv_bfloat16 *)dQ, p.n, n_pad, p.causal, p.scale,
                                                                     nt, heads_per_group(p, nt), device_status_ptr());
        return cudaGetLastError();
    }
}

}  // namespace

// Forward of `p` (a group of heads): O, L and P^T[heads][n_pad][n_pad].
cudaError_t mat_fwd(const Problem &p, const void *Q, const void *K, const void *V, void *O, float *L, void *PT, cudaStream_t st)
{
    if (p.d == 64) return run_group<64>(p, Q, K, V, nullptr, O, L, nullptr, PT, nullptr, nullptr, nullptr, nullptr, 0, st);
    if (p.d == 128) return run_group<128>(p, Q, K, V, nullptr, O, L, nullptr, PT, nullptr, nullptr, nullptr, nullptr, 0, st);
    return cudaErrorInvalidValue;
}

// Backward of `p` (a group of heads) from the persisted P^T; dS^T goes to GST and is read back for dQ.
cudaError_t mat_bwd(const Problem &p, const void *Q, const void *K, const void *V, const void *dO, const float *Dp,
                    const void *PT, void *GST, void *dQ, void *dK, void *dV, cudaStream_t st)
{
    if (p.d == 64)
        return run_group<64>(p, Q, K, V, dO, nullptr, nullptr, Dp, const_cast<void *>(PT), GST, dQ, dK, dV, 1, st);
    if (p.d == 128)
        return run_group<128>(p, Q, K, V, dO, nullptr, nullptr, Dp, const_cast<void *>(PT), GST, dQ, dK, dV, 1, st);
    return cudaErrorInvalidValue;
}

}  // namespace moa
