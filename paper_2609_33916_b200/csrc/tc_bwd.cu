// Backward attention on the sm_100a tensor cores, bf16 in, fp32 accumulate.
//
// One CTA owns 128 keys (one K/V tile) of one (batch, head) and walks the query tiles
// of 128 rows; dK and dV of those keys accumulate in TMEM and are written once, by this
// CTA only (no atomics: the paper's (b,ic)-parallel GV pass, applied to GK as well).
// Per query tile i, with everything transposed so that TMEM lanes are keys:
//     S^T  = K Q_i^T                 (SS-UMMA, both operands K-major)
//     dP^T = V dO_i^T                (SS-UMMA)
//     P^T  = exp2(S^T scale log2e - L_i log2e)         (registers; L from the forward)
//     dS^T = scale * P^T o (dP^T - D_i)                (D = rowsum(dO o O))
//     dV  += P^T dO_i                (TS-UMMA: P^T bf16 in TMEM, dO_i MN-major in smem)
//     dK  += dS^T Q_i                (TS-UMMA: dS^T bf16 in TMEM, Q_i MN-major in smem)
//     dQ_i = dS K                    (SS-UMMA: dS^T tile in smem as MN-major A, K MN-major)
// dQ_i is one key tile's contribution; it is added into an fp32 [B,H,n,d] accumulator
// with vector red.global.add (the contended step the dq_mode knob is about).
//
// Roles (320 threads): warps 0-7 elementwise work (thread = TMEM lane, the two
// warpgroups split the columns), warp 8 TMA producer (K,V once; Q_i, dO_i, L_i, D_i in a
// two-stage ring), warp 9 UMMA issuer and TMEM owner.
//
// TMEM columns (512): S^T [0,128), dP^T [128,256), dV [256,256+D), dK [256+D,256+2D);
// P^T / dS^T (bf16) overwrite the front of their fp32 source columns; for D = 128 the dQ
// tile reuses the dP^T columns (the UMMAs that read dS^T there are issued before it).
//
// Rows past n need no masking: TMA zero-fills K, V, Q, dO there, the preprocess kernel
// pads L with +inf (so P = 0) and D with 0, and stores are row-guarded.
#include "common.cuh"
#include "ptx.cuh"
#include "tensormap.cuh"

namespace moa {
namespace {

using namespace ptx;

constexpr int kThreads = 320;
constexpr int kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;

enum : uint32_t {
    ERR_KV = 0x201, ERR_FULL = 0x202, ERR_EMPTY = 0x203, ERR_SDP = 0x204, ERR_PDS = 0x205, ERR_DQ = 0x206,
    ERR_DQR = 0x207, ERR_ALIGN = 0x208
};

__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void red_add_v4(float *addr, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

// Lp = L log2(e) and D = rowsum(dO o O), both padded per head to n_pad rows
// (+inf and 0 past n).  One warp per padded row.
template <int D>
__global__ void bwd_preprocess_kernel(const __nv_bfloat16 *__restrict__ dO, const __nv_bfloat16 *__restrict__ O,
                                      const float *__restrict__ L, float *__restrict__ Lp, float *__restrict__ Dp,
                                      int n, int n_pad, size_t padded_rows)
{
    const size_t prow = (size_t)blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    if (prow >= padded_rows) return;
    const int lane = threadIdx.x % 32;
    const size_t bh = prow / n_pad;
    const int r = (int)(prow % n_pad);
    if (r >= n) {
        if (lane == 0) { Lp[prow] = INFINITY; Dp[prow] = 0.f; }
        return;
    }
    const size_t row = bh * n + r;
    float acc = 0.f;
    constexpr int kPerLane = D / 32;   // 2 or 4 consecutive elements
    const __nv_bfloat16 *a = dO + row * D + lane * kPerLane;
    const __nv_bfloat16 *b = O + row * D + lane * kPerLane;
#pragma unroll
    for (int i = 0; i < kPerLane; i += 2) {
        const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(a + i));
        const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(b + i));
        acc = fmaf(x.x, y.x, acc);
        acc = fmaf(x.y, y.y, acc);
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) { Dp[prow] = acc; Lp[prow] = L[row] * kLog2e; }
}

template <int D>
struct BwdSmem {
    static constexpr int kTile = 128 * D * 2;        // K, V, Q_i, dO_i tiles
    static constexpr int kdS = 128 * 128 * 2;        // dS^T tile, [128 keys][128 queries] bf16
    static constexpr int offK = 0;
    static constexpr int offV = offK + kTile;
    static constexpr int offQ = offV + kTile;        // 2 stages
    static constexpr int offdO = offQ + 2 * kTile;   // 2 stages
    static constexpr int offdS = offdO + 2 * kTile;
    static constexpr int offL = offdS + kdS;         // 2 x 128 floats
    static constexpr int offD = offL + 2 * 512;      // 2 x 128 floats
    static constexpr int offBar = offD + 2 * 512;    // 8 mbarriers + tmem base + abort flag
    static constexpr int kTotal = offBar + 128;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
tc_bwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
              const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapdO,
              const float *__restrict__ Lp, const float *__restrict__ Dp,
              __nv_bfloat16 *__restrict__ dK, __nv_bfloat16 *__restrict__ dV, float *__restrict__ dQacc,
              int n, int n_pad, int causal, float scale, float scale_log2, int nkt, unsigned int *status)
{
    using SM = BwdSmem<D>;
    constexpr int kBoxes = D / 64;
    constexpr int kBoxBytes = 128 * 128;
    constexpr uint32_t colS = 0, colDP = 128, colDV = 256, colDK = 256 + D, colDQ = (D == 128) ? 128 : 384;
    extern __shared__ __align__(1024) uint8_t sm[];
    uint8_t *sK = sm + SM::offK, *sV = sm + SM::offV, *sdS = sm + SM::offdS;
    float *sL = reinterpret_cast<float *>(sm + SM::offL);
    float *sD = reinterpret_cast<float *>(sm + SM::offD);
    uint64_t *bars = reinterpret_cast<uint64_t *>(sm + SM::offBar);
    uint64_t *bar_kv = bars + 0, *bar_full = bars + 1 /*[2]*/, *bar_empty = bars + 3 /*[2]*/;
    uint64_t *bar_sdp = bars + 5, *bar_pds = bars + 6, *bar_dq = bars + 7, *bar_dqr = bars + 8;
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bars + 9);
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(bars + 10);

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int bh = blockIdx.x / nkt;
    const int kt = blockIdx.x % nkt;          // causal: key tile 0 has the most query tiles and goes first
    const int k0 = kt * 128;
    const int nqt = n_pad / 128;
    const int i_begin = causal ? kt : 0;
    const int niter = nqt - i_begin;

    if (tid == 0) {
        mbar_init(bar_kv, 1);
        mbar_init(bar_full + 0, 1); mbar_init(bar_full + 1, 1);
        mbar_init(bar_empty + 0, 1); mbar_init(bar_empty + 1, 1);
        mbar_init(bar_sdp, 1); mbar_init(bar_pds, 256); mbar_init(bar_dq, 1); mbar_init(bar_dqr, 256);
        *abortp = (smem_u32(sm) & 1023u) ? 1u : 0u;
        if (*abortp && status) atomicCAS(status, 0u, (unsigned)ERR_ALIGN);
        fence_mbar_init();
        prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV); prefetch_tensormap(&mapdO);
    }
    if (warp == 9) { tmem_alloc(tmem_base_s, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_base_s;
    const bool aligned_ok = (*abortp == 0);

    if (!aligned_ok) {
        // shared memory base is not 1024-byte aligned: swizzled tiles would be misplaced
    } else if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_arrive_expect_tx(bar_kv, 2 * SM::kTile);
            for (int b = 0; b < kBoxes; ++b) {
                tma_load_3d(sK + b * kBoxBytes, &mapK, bar_kv, 64 * b, k0, bh);
                tma_load_3d(sV + b * kBoxBytes, &mapV, bar_kv, 64 * b, k0, bh);
            }
        }
        for (int it = 0; it < niter; ++it) {
            const int s = it & 1;
            const int q0 = (i_begin + it) * 128;
            if (it >= 2 && !mbar_wait(bar_empty + s, ((it >> 1) - 1) & 1, abortp, status, ERR_EMPTY)) break;
            if (lane == 0) {
                uint8_t *sQ = sm + SM::offQ + s * SM::kTile, *sdO = sm + SM::offdO + s * SM::kTile;
                mbar_arrive_expect_tx(bar_full + s, 2 * SM::kTile + 1024);
                for (int b = 0; b < kBoxes; ++b) {
                    tma_load_3d(sQ + b * kBoxBytes, &mapQ, bar_full + s, 64 * b, q0, bh);
                    tma_load_3d(sdO + b * kBoxBytes, &mapdO, bar_full + s, 64 * b, q0, bh);
                }
                bulk_load_1d(sL + s * 128, Lp + (size_t)bh * n_pad + q0, 512, bar_full + s);
                bulk_load_1d(sD + s * 128, Dp + (size_t)bh * n_pad + q0, 512, bar_full + s);
            }
            __syncwarp();
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------- UMMA issuer
        constexpr uint32_t idesc_st = idesc_bf16_f32(128, 128, 0, 0);   // S^T, dP^T
        constexpr uint32_t idesc_acc = idesc_bf16_f32(128, D, 0, 1);    // dV, dK: A in TMEM, B MN-major
        constexpr uint32_t idesc_dq = idesc_bf16_f32(128, D, 1, 1);     // dQ: A and B MN-major
        const uint32_t k_addr = smem_u32(sK), v_addr = smem_u32(sV), ds_addr = smem_u32(sdS);
        bool ok = mbar_wait(bar_kv, 0, abortp, status, ERR_KV);
        for (int it = 0; ok && it < niter; ++it) {
            const int s = it & 1;
            const uint32_t q_addr = smem_u32(sm + SM::offQ + s * SM::kTile);
            const uint32_t do_addr = smem_u32(sm + SM::offdO + s * SM::kTile);
            if (!mbar_wait(bar_full + s, (it >> 1) & 1, abortp, status, ERR_FULL)) break;
            if (it > 0 && !mbar_wait(bar_dqr, (it - 1) & 1, abortp, status, ERR_DQR)) break;   // dQ tile read out
            tc_fence_after();
            if (lane == 0) {
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks / 4) * kBoxBytes + (ks % 4) * 32;
                    umma_ss(tbase + colS, smem_desc_sw128(k_addr + off, 16, 1024),
                            smem_desc_sw128(q_addr + off, 16, 1024), idesc_st, ks > 0);
                }
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks / 4) * kBoxBytes + (ks % 4) * 32;
                    umma_ss(tbase + colDP, smem_desc_sw128(v_addr + off, 16, 1024),
                            smem_desc_sw128(do_addr + off, 16, 1024), idesc_st, ks > 0);
                }
                umma_commit(bar_sdp);
            }
            __syncwarp();
            if (!mbar_wait(bar_pds, it & 1, abortp, status, ERR_PDS)) break;
            tc_fence_after();
            if (lane == 0) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // 16 queries per step
                    const uint32_t a_col = 64 * (ks / 4) + 8 * (ks % 4);
                    umma_ts(tbase + colDV, tbase + colS + a_col,
                            smem_desc_sw128(do_addr + ks * 2048, kBoxBytes, 1024), idesc_acc, (it > 0 || ks > 0));
                }
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t a_col = 64 * (ks / 4) + 8 * (ks % 4);
                    umma_ts(tbase + colDK, tbase + colDP + a_col,
                            smem_desc_sw128(q_addr + ks * 2048, kBoxBytes, 1024), idesc_acc, (it > 0 || ks > 0));
                }
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // 16 keys per step
                    umma_ss(tbase + colDQ, smem_desc_sw128(ds_addr + ks * 2048, kBoxBytes, 1024),
                            smem_desc_sw128(k_addr + ks * 2048, kBoxBytes, 1024), idesc_dq, ks > 0);
                }
                umma_commit(bar_empty + s);
                umma_commit(bar_dq);
            }
            __syncwarp();
        }
    } else {
        // ----------------------------------------------------------- elementwise warps 0-7
        const int wg = warp / 4;                          // which half of the columns
        const int lane_row = 32 * (warp % 4) + lane;      // TMEM lane of this thread
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        bool ok = true;
        for (int it = 0; it < niter; ++it) {
            const int s = it & 1;
            const int i = i_begin + it;
            const int q0 = i * 128;
            const bool diag = causal && (i == kt);
            if (!mbar_wait(bar_sdp, it & 1, abortp, status, ERR_SDP)) { ok = false; break; }
            tc_fence_after();
            const float *Ls = sL + s * 128, *Ds = sD + s * 128;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int qc0 = 64 * wg + 32 * c;         // first query column of this chunk
                uint32_t rs[32], rd[32];
                tmem_ld(lane_addr + colS + qc0, rs);
                tmem_ld(lane_addr + colDP + qc0, rd);
                tc_wait_ld();
                uint32_t pk[16], gk[16];
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const float4 l4 = *reinterpret_cast<const float4 *>(Ls + qc0 + e);
                    const float4 d4 = *reinterpret_cast<const float4 *>(Ds + qc0 + e);
                    const float lv[4] = {l4.x, l4.y, l4.z, l4.w}, dv[4] = {d4.x, d4.y, d4.z, d4.w};
                    float p[4], g[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        float pv = ex2(fmaf(__uint_as_float(rs[e + u]), scale_log2, -lv[u]));
                        if (diag && (qc0 + e + u) < lane_row) pv = 0.f;   // query index < key index: masked
                        p[u] = pv;
                        g[u] = pv * (__uint_as_float(rd[e + u]) - dv[u]) * scale;
                    }
                    pk[e / 2] = pack_bf16(p[0], p[1]); pk[e / 2 + 1] = pack_bf16(p[2], p[3]);
                    gk[e / 2] = pack_bf16(g[0], g[1]); gk[e / 2 + 1] = pack_bf16(g[2], g[3]);
                }
                tmem_st(lane_addr + colS + 64 * wg + 16 * c, pk);
                tmem_st(lane_addr + colDP + 64 * wg + 16 * c, gk);
                // dS^T row (this key) into the MN-major smem tile: box wg, 128-byte row, swizzled 16-byte chunks
                uint8_t *rowp = sdS + wg * kBoxBytes + lane_row * 128;
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int chunk = (4 * c + jj) ^ (lane_row & 7);
                    *reinterpret_cast<uint4 *>(rowp + chunk * 16) =
                        make_uint4(gk[4 * jj], gk[4 * jj + 1], gk[4 * jj + 2], gk[4 * jj + 3]);
                }
            }
            tc_wait_st();
            tc_fence_before();
            fence_proxy_async_smem();
            mbar_arrive(bar_pds);

            if (!mbar_wait(bar_dq, it & 1, abortp, status, ERR_DQ)) { ok = false; break; }
            tc_fence_after();
            // dQ tile: lanes are query rows now; this warpgroup takes D/2 columns
            const int qrow = q0 + lane_row;
            float *dst = dQacc + ((size_t)bh * n + qrow) * D + (D / 2) * wg;
#pragma unroll
            for (int c = 0; c < D / 2; c += 32) {
                uint32_t r[32];
                tmem_ld(lane_addr + colDQ + (D / 2) * wg + c, r);
                tc_wait_ld();
                if (qrow < n) {
#pragma unroll
                    for (int e = 0; e < 32; e += 4)
                        red_add_v4(dst + c + e, __uint_as_float(r[e]), __uint_as_float(r[e + 1]),
                                   __uint_as_float(r[e + 2]), __uint_as_float(r[e + 3]));
                }
            }
            tc_fence_before();
            mbar_arrive(bar_dqr);
        }
        if (ok) {
            // all UMMAs have completed (the last bar_dq wait): write dV and dK rows of this key
            const int krow = k0 + lane_row;
            __nv_bfloat16 *dvp = dV + ((size_t)bh * n + krow) * D + (D / 2) * wg;
            __nv_bfloat16 *dkp = dK + ((size_t)bh * n + krow) * D + (D / 2) * wg;
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const uint32_t col = (which == 0 ? colDV : colDK) + (D / 2) * wg;
                __nv_bfloat16 *outp = which == 0 ? dvp : dkp;
#pragma unroll
                for (int c = 0; c < D / 2; c += 32) {
                    uint32_t r[32];
                    tmem_ld(lane_addr + col + c, r);
                    tc_wait_ld();
                    if (krow < n) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            uint4 v;
                            v.x = pack_bf16(__uint_as_float(r[e + 0]), __uint_as_float(r[e + 1]));
                            v.y = pack_bf16(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3]));
                            v.z = pack_bf16(__uint_as_float(r[e + 4]), __uint_as_float(r[e + 5]));
                            v.w = pack_bf16(__uint_as_float(r[e + 6]), __uint_as_float(r[e + 7]));
                            *reinterpret_cast<uint4 *>(outp + c + e) = v;
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tbase, kTmemCols);
}

template <int D>
cudaError_t launch_bwd(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                       const float *Lp, const float *Dp, void *dK, void *dV, float *dQacc, cudaStream_t st)
{
    CUtensorMap mq, mk, mv, mdo;
    const uint64_t heads = (uint64_t)p.BH();
    if (!make_tensor_map_3d(&mq, Q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64) ||
        !make_tensor_map_3d(&mk, K, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64) ||
        !make_tensor_map_3d(&mv, V, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64) ||
        !make_tensor_map_3d(&mdo, dO, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64))
        return cudaErrorInvalidValue;
    constexpr int kSmem = BwdSmem<D>::kTotal;
    cudaError_t e = cudaFuncSetAttribute(tc_bwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const int nkt = (p.n + 127) / 128;
    LaunchScope scope(MOA_KERNEL_BWD_KV, st);
    tc_bwd_kernel<D><<<(unsigned)(nkt * p.BH()), kThreads, kSmem, st>>>(
        mq, mk, mv, mdo, Lp, Dp, (__nv_bfloat16 *)dK, (__nv_bfloat16 *)dV, dQacc, p.n, nkt * 128, p.causal,
        p.scale, p.scale * kLog2e, nkt, device_status_ptr());
    return cudaGetLastError();
}

}  // namespace

cudaError_t tc_bwd_preprocess(const Problem &p, const void *dO, const void *O, const float *L, float *Lp, float *Dp,
                              cudaStream_t st)
{
    const int n_pad = (p.n + 127) / 128 * 128;
    const size_t rows = (size_t)p.BH() * n_pad;
    const int wpb = 8;
    const unsigned grid = (unsigned)((rows + wpb - 1) / wpb);
    LaunchScope scope(MOA_KERNEL_PREPROCESS, st);
    if (p.d == 64)
        bwd_preprocess_kernel<64><<<grid, wpb * 32, 0, st>>>((const __nv_bfloat16 *)dO, (const __nv_bfloat16 *)O, L,
                                                             Lp, Dp, p.n, n_pad, rows);
    else
        bwd_preprocess_kernel<128><<<grid, wpb * 32, 0, st>>>((const __nv_bfloat16 *)dO, (const __nv_bfloat16 *)O, L,
                                                              Lp, Dp, p.n, n_pad, rows);
    return cudaGetLastError();
}

cudaError_t tc_bwd_kv(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                      const float *Lp, const float *Dp, void *dK, void *dV, float *dQacc, cudaStream_t st)
{
    if (p.d == 64) return launch_bwd<64>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
    if (p.d == 128) return launch_bwd<128>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
    return cudaErrorInvalidValue;
}

}  // namespace moa
