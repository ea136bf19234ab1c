// Atomic-free dQ pass on the sm_100a tensor cores (dq_mode = MOA_DQ_SEPARATE_PASS).
//
// One CTA owns 128 query rows of one (batch, head) and walks the key tiles, so every dQ
// element has exactly one writer and the result is bitwise reproducible.  The price is
// recomputation: per key tile j
//     S  = Q K_j^T,  dP = dO V_j^T          (SS-UMMA)
//     dS = exp2(S scale log2e - L log2e) o (dP - D)   (registers, bf16 back into TMEM)
//     dQ += dS K_j                          (TS-UMMA: dS in TMEM, K_j MN-major in smem)
// i.e. three GEMMs where the key-parallel backward needs one for dQ.  This is the B200
// counterpart of the paper's choice between an atomic and an extra pass; there the extra
// pass re-read a persisted n x n array from DRAM, here it recomputes it on chip.
//
// Roles (320 threads): warps 0-7 elementwise (thread = TMEM lane = query row, the two
// warpgroups split the key columns), warp 8 TMA producer (Q, dO once; K_j, V_j in a
// two-slot ring), warp 9 (one thread) UMMA issuer and TMEM owner.
// TMEM: S [0,128), dP [128,256) (dS bf16 over its front), dQ [256,256+D).
#include "common.cuh"
#include "ptx.cuh"
#include "tensormap.cuh"

namespace moa {
namespace {

using namespace ptx;

constexpr int kThreads = 320;
constexpr int kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
enum : uint32_t { ERR_Q = 0x301, ERR_KV = 0x302, ERR_EMPTY = 0x303, ERR_SDP = 0x304, ERR_DS = 0x305, ERR_DONE = 0x306,
                  ERR_ALIGN = 0x308 };
enum { B_Q = 0, B_KVFULL = 1 /*2*/, B_KVEMPTY = 3 /*2*/, B_SDP = 5, B_DS = 6, B_DONE = 7, B_COUNT = 8 };

template <int D>
struct DqSmem {
    static constexpr int kTile = 128 * D * 2;
    static constexpr int offQ = 0, offdO = kTile, offK = 2 * kTile /*2 slots*/, offV = 4 * kTile /*2 slots*/;
    static constexpr int offBar = 6 * kTile;
    static constexpr int kTotal = offBar + 128;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
tc_dq_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
             const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapdO,
             const float *__restrict__ Lp, const float *__restrict__ Dp, __nv_bfloat16 *__restrict__ dQ,
             int n, int n_pad, int causal, float scale, float scale_log2, int nqt, int hpg,
             int group, int H, Strides sq, int d, unsigned int *status)
{
    using SM = DqSmem<D>;
    constexpr int kBoxes = D / 64;
    constexpr int kBoxBytes = 128 * 128;
    constexpr uint32_t colS = 0, colDP = 128, colDQ = 256;
    extern __shared__ __align__(1024) uint8_t sm[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(sm + SM::offBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bars + B_COUNT);
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(bars + B_COUNT + 1);

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    int bh, t;
    job_from_block((int)blockIdx.x, nqt, (int)gridDim.x / nqt, hpg, bh, t);
    const int bb = bh / H, hq = bh - bb * H;    // batch and query head: coordinates of the 4-D tensor maps
    const int hk = hq / group;                  // the K/V head this query head reads
    const int qt = causal ? nqt - 1 - t : t;   // causal: longest rows first
    const int q0 = qt * 128;
    const int nkt_all = n_pad / 128;
    const int nkt_want = causal ? min(qt + 1, nkt_all) : nkt_all;

    if (tid == 0) {
        for (int b = 0; b < B_COUNT; ++b) mbar_init(bars + b, b == B_DS ? 256u : 1u);
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
    const int nkt = (*abortp == 0) ? nkt_want : 0;   // misaligned shared memory: every role is a no-op

    if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        ArmCounts<B_COUNT> armed;     // barriers armed for copies into shared memory
        if (lane == 0 && nkt > 0) {
            mbar_arm(bars, bars + B_Q, 2 * SM::kTile, armed);
            for (int b = 0; b < kBoxes; ++b) {
                tma_load_4d(sm + SM::offQ + b * kBoxBytes, &mapQ, bars + B_Q, 64 * b, q0, hq, bb);
                tma_load_4d(sm + SM::offdO + b * kBoxBytes, &mapdO, bars + B_Q, 64 * b, q0, hq, bb);
            }
        }
        for (int j = 0; j < nkt; ++j) {
            const int s = j & 1;
            if (j >= 2 && !mbar_wait(bars + B_KVEMPTY + s, ((j >> 1) - 1) & 1, abortp, status, ERR_EMPTY)) break;
            if (lane == 0) {
                mbar_arm(bars, bars + B_KVFULL + s, 2 * SM::kTile, armed);
                for (int b = 0; b < kBoxes; ++b) {
                    tma_load_4d(sm + SM::offK + s * SM::kTile + b * kBoxBytes, &mapK, bars + B_KVFULL + s, 64 * b, j * 128, hk, bb);
                    tma_load_4d(sm + SM::offV + s * SM::kTile + b * kBoxBytes, &mapV, bars + B_KVFULL + s, 64 * b, j * 128, hk, bb);
                }
            }
            __syncwarp();
        }
        if (lane == 0) mbar_drain(bars, armed);     // copies of this CTA still on their way land before it leaves (bounded)
    } else if (warp == 9 && lane == 0) {
        // ------------------------------------------------------- UMMA issuer (one thread)
        constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);
        constexpr uint32_t idesc_dq = idesc_bf16_f32(128, D, 0, 1);
        const uint64_t km_proto = smem_desc_sw128(0, 16, 1024), mn_proto = smem_desc_sw128(0, kBoxBytes, 1024);
        const uint32_t km_hi = (uint32_t)(km_proto >> 32), mn_hi = (uint32_t)(mn_proto >> 32);
        auto field = [](const void *ptr) { return (smem_u32(ptr) >> 4) & 0x3FFFu; };
        const uint32_t q_km = (uint32_t)km_proto + field(sm + SM::offQ), do_km = (uint32_t)km_proto + field(sm + SM::offdO);
        const uint32_t k_km0 = (uint32_t)km_proto + field(sm + SM::offK), v_km0 = (uint32_t)km_proto + field(sm + SM::offV);
        const uint32_t k_mn0 = (uint32_t)mn_proto + field(sm + SM::offK);
        constexpr uint32_t kSlot = (uint32_t)(SM::kTile >> 4);
        auto koff = [](int ks) { return (uint32_t)(((ks / 4) * kBoxBytes + (ks % 4) * 32) >> 4); };
        bool ok = nkt > 0 && mbar_wait(bars + B_Q, 0, abortp, status, ERR_Q);
        for (int j = 0; ok && j < nkt; ++j) {
            const int s = j & 1;
            const uint32_t k_km = k_km0 + s * kSlot, v_km = v_km0 + s * kSlot, k_mn = k_mn0 + s * kSlot;
            if (!mbar_wait(bars + B_KVFULL + s, (j >> 1) & 1, abortp, status, ERR_KV)) break;
            tc_fence_after();
            // S(j) and dP(j): the previous tile's dS (over the dP columns) is read by dQ(j-1),
            // which was issued before these and executes before them
            umma_ss2<false>(tbase + colS, q_km, km_hi, k_km, km_hi, idesc_s);
#pragma unroll
            for (int ks = 1; ks < D / 16; ++ks)
                umma_ss2<true>(tbase + colS, q_km + koff(ks), km_hi, k_km + koff(ks), km_hi, idesc_s);
            umma_ss2<false>(tbase + colDP, do_km, km_hi, v_km, km_hi, idesc_s);
#pragma unroll
            for (int ks = 1; ks < D / 16; ++ks)
                umma_ss2<true>(tbase + colDP, do_km + koff(ks), km_hi, v_km + koff(ks), km_hi, idesc_s);
            umma_commit(bars + B_SDP);
            if (!mbar_wait(bars + B_DS, j & 1, abortp, status, ERR_DS)) break;
            tc_fence_after();
            if (j > 0) umma_ts2<true>(tbase + colDQ, tbase + colDP, k_mn, mn_hi, idesc_dq);
            else       umma_ts2<false>(tbase + colDQ, tbase + colDP, k_mn, mn_hi, idesc_dq);
#pragma unroll
            for (int ks = 1; ks < 8; ++ks)
                umma_ts2<true>(tbase + colDQ, tbase + colDP + 64 * (ks / 4) + 8 * (ks % 4),
                               k_mn + (uint32_t)((ks * 2048) >> 4), mn_hi, idesc_dq);
            umma_commit(bars + B_KVEMPTY + s);
            if (j == nkt - 1) umma_commit(bars + B_DONE);
        }
    } else if (warp < 8) {
        // ----------------------------------------------------------- elementwise warps 0-7
        const int wg = warp / 4;
        const int lane_row = 32 * (warp % 4) + lane;              // query row inside the tile
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        const float Lrow = Lp[(size_t)bh * n_pad + q0 + lane_row];   // -L log2e; -inf past n: P = 0
        const float Drow = Dp[(size_t)bh * n_pad + q0 + lane_row];   // -D
        bool ok = nkt > 0;
        for (int j = 0; ok && j < nkt; ++j) {
            if (!mbar_wait(bars + B_SDP, j & 1, abortp, status, ERR_SDP)) { ok = false; break; }
            tc_fence_after();
            const bool diag = causal && (j == qt);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int kc0 = 64 * wg + 32 * c;                 // first key column of this chunk
                uint32_t rs[32], rd[32];
                tmem_ld(lane_addr + colS + kc0, rs);
                tmem_ld(lane_addr + colDP + kc0, rd);
                tc_wait_ld();
                uint32_t gk[16];
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    float p0 = ex2(fmaf(__uint_as_float(rs[e]), scale_log2, Lrow));
                    float p1 = ex2(fmaf(__uint_as_float(rs[e + 1]), scale_log2, Lrow));
                    if (diag) {                                   // key index > query index: masked
                        if (kc0 + e > lane_row) p0 = 0.f;
                        if (kc0 + e + 1 > lane_row) p1 = 0.f;
                    }
                    gk[e / 2] = pack_bf16(p0 * (__uint_as_float(rd[e]) + Drow), p1 * (__uint_as_float(rd[e + 1]) + Drow));
                }
                tmem_st(lane_addr + colDP + 64 * wg + 16 * c, gk);
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bars + B_DS);
        }
        if (ok && mbar_wait(bars + B_DONE, 0, abortp, status, ERR_DONE)) {
            tc_fence_after();
            const int qrow = q0 + lane_row;
            __nv_bfloat16 *outp = dQ + sq.at(bb, hq, qrow) + (D / 2) * wg;   // row of dQ in the caller's layout; d <= D columns exist in memory
#pragma unroll
            for (int c = 0; c < D / 2; c += 32) {
                uint32_t r[32];
                tmem_ld(lane_addr + colDQ + (D / 2) * wg + c, r);
                tc_wait_ld();
                if (qrow < n) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(r[e + 0]) * scale, __uint_as_float(r[e + 1]) * scale);
                        v.y = pack_bf16(__uint_as_float(r[e + 2]) * scale, __uint_as_float(r[e + 3]) * scale);
                        v.z = pack_bf16(__uint_as_float(r[e + 4]) * scale, __uint_as_float(r[e + 5]) * scale);
                        v.w = pack_bf16(__uint_as_float(r[e + 6]) * scale, __uint_as_float(r[e + 7]) * scale);
                        if ((D / 2) * wg + c + e < d) *reinterpret_cast<uint4 *>(outp + c + e) = v;
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
cudaError_t launch_dq(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                      const float *Lp, const float *Dp, void *dQ, cudaStream_t st)
{
    CUtensorMap mq, mk, mv, mdo;
    const auto bf = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    if (!make_tensor_map_4d_strided(&mq, Q, bf, 2, p.B, p.H, p.n, p.d, p.sq.row, p.sq.head, p.sq.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mk, K, bf, 2, p.B, p.kv_heads(), p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mv, V, bf, 2, p.B, p.kv_heads(), p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mdo, dO, bf, 2, p.B, p.H, p.n, p.d, p.so.row, p.so.head, p.so.batch, 128, 64))
        return cudaErrorInvalidValue;
    constexpr int kSmem = DqSmem<D>::kTotal;
    cudaError_t e = cudaFuncSetAttribute(tc_dq_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const int nqt = (p.n + 127) / 128;
    LaunchScope scope(MOA_KERNEL_BWD_DQ, st);
    tc_dq_kernel<D><<<(unsigned)(nqt * p.BH()), kThreads, kSmem, st>>>(
        mq, mk, mv, mdo, Lp, Dp, (__nv_bfloat16 *)dQ, p.n, nqt * 128, p.causal, p.scale, p.scale * kLog2e, nqt,
        heads_per_group(p, nqt), p.group(), p.H, p.sq, p.d, device_status_ptr());
    return cudaGetLastError();
}

}  // namespace

cudaError_t tc_bwd_dq(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                      const float *Lp, const float *Dp, void *dQ, cudaStream_t st)
{
    if (p.d < 8 || p.d > 128 || p.d % 8) return cudaErrorInvalidValue;
    return kernel_d(p.d) == 64 ? launch_dq<64>(p, Q, K, V, dO, Lp, Dp, dQ, st) : launch_dq<128>(p, Q, K, V, dO, Lp, Dp, dQ, st);
}

}  // namespace moa
