// Backward attention for head dimensions 136..256 on the sm_100a tensor cores, bf16 in, fp32 accumulate.
//
// Same mathematics, the same key-tile-parallel structure and the same one-writer rule for dK and dV as tc_bwd.cu
// (the paper's (b,ic)-parallel GV pass, applied to GK as well).  What changes is the tiling, because neither TMEM
// nor shared memory holds the 128 x 128 plan at 256 columns: the accumulators dV, dK of 256 columns would fill TMEM
// alone, and K, V, Q_i, dO_i at 256 columns are 256 KB.
//   * two passes over the halves of d: the grid has two CTAs per (head, key tile), CTA p accumulates dV[:, p],
//     dK[:, p] and the dQ contribution [:, p] (128 columns each); the scores S^T = K Q_i^T and dP^T = V dO_i^T need the
//     whole head dimension and are computed by both (K-dimension 256: sixteen UMMAs each);
//   * query tiles of 64 rows: S^T, dP^T are 128 keys x 64 queries (UMMA N = 64), so Q_i and dO_i are 32 KB each,
//     the dS^T tile 16 KB, and TMEM holds S^T 64 + dP^T 64 + dQ^T 64 + dV 128 + dK 128 = 448 columns with nothing aliased;
//   * Q_i lives in three half-slots of 16 KB: the d-half this pass does not own is read by S(i) only and has one slot,
//     the half it owns is read again by dK(i) at the end of the tile and alternates between two.
// Shared memory: K 64 KB + V 64 KB + Q 48 KB + dO 32 KB + dS^T 16 KB = 224 KB; dQ leaves as red.global.add.f32 from
// registers (one warp-wide instruction = 32 consecutive floats of one dQ row), there is no room for a staging tile.
// Per query tile i: dP(i), dV(i), S(i+1), dK(i), dQ(i), issued by one thread; roles as in tc_bwd.cu.
// Head dimensions below 256 (192, ...) run with the missing columns zero-filled by the loads and dropped by the stores.
#include "common.cuh"
#include "ptx.cuh"
#include "tensormap.cuh"

namespace moa {
namespace {

using namespace ptx;

constexpr int kThreads = 512;   // warps 0-7 elementwise, 8-11 dQ read-out and reds, 12 TMA, 13 UMMA, 14-15 idle
constexpr int kReduceWarp0 = 8, kLoadWarp = 12, kMmaWarp = 13;
constexpr int kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr int BQ = 64;          // query rows per tile
constexpr int DW = 256;         // head dimension of the kernel

enum : uint32_t {
    WERR_KV = 0x241, WERR_FULL = 0x242, WERR_EMPTY = 0x243, WERR_SDP = 0x244, WERR_PDS = 0x245, WERR_DQ = 0x246,
    WERR_DQR = 0x247, WERR_ALIGN = 0x248
};

struct WideSmem {
    static constexpr int kBoxK = 128 * 128;          // [128 keys][64 columns] bf16, 128-byte rows
    static constexpr int kBoxQ = 64 * 128;           // [64 queries][64 columns]
    static constexpr int kHalf = 2 * kBoxQ;          // one d-half of a query tile: two boxes
    static constexpr int offK = 0;                   // four boxes
    static constexpr int offV = offK + 4 * kBoxK;
    static constexpr int offQ = offV + 4 * kBoxK;    // half-slot 0: the other d-half; 1, 2: this pass's half (tile parity)
    static constexpr int offdO = offQ + 3 * kHalf;   // four boxes
    static constexpr int offdS = offdO + 4 * kBoxQ;  // dS^T tile, [128 keys][64 queries]
    static constexpr int offL = offdS + 128 * 128;   // 2 x 64 floats, travels with the owned Q half
    static constexpr int offDd = offL + 2 * 256;
    static constexpr int offBar = offDd + 2 * 256;
    static constexpr int kTotal = offBar + 256;
};
static_assert(WideSmem::kTotal <= 232448, "shared memory of one CTA");

enum {
    W_KV = 0, W_QOWN = 1 /*2*/, W_QOTH = 3, W_QEMPTY = 4 /*2*/, W_DOFULL = 6, W_DOEMPTY = 7, W_S = 8, W_P = 9, W_DP = 10,
    W_DS = 11, W_DQ = 12, W_DQR = 13, W_EPI = 14, W_COUNT = 15
};

__device__ __forceinline__ void red_add_f32(float *addr, float a)
{
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(addr), "f"(a) : "memory");
}

template <bool kGrouped>
__global__ void __launch_bounds__(kThreads, 1)
tc_bwd_wide_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                   const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapdO,
                   const __grid_constant__ CUtensorMap mapdK, const __grid_constant__ CUtensorMap mapdV,
                   const float *__restrict__ Lp, const float *__restrict__ Dp, float *__restrict__ dQacc,
                   int n, int n_pad, int d, int causal, float scale, float scale_log2, int nkt, int hpg, int group,
                   int Hkv, unsigned int *status)
{
    using SM = WideSmem;
    constexpr uint32_t colS = 0, colDP = 64, colDQ = 128, colDV = 192, colDK = 320;
    extern __shared__ __align__(1024) uint8_t sm[];
    uint8_t *sK = sm + SM::offK, *sV = sm + SM::offV, *sQ = sm + SM::offQ, *sdO = sm + SM::offdO, *sdS = sm + SM::offdS;
    float *sL = reinterpret_cast<float *>(sm + SM::offL);
    float *sD = reinterpret_cast<float *>(sm + SM::offDd);
    uint64_t *bars = reinterpret_cast<uint64_t *>(sm + SM::offBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bars + W_COUNT);
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(bars + W_COUNT + 1);

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int pass = (int)(blockIdx.x & 1u);             // the d-half whose dV, dK, dQ columns this CTA accumulates
    int bh, kt;                                           // causal: key tile 0 has the most query tiles and goes first
    job_from_block((int)(blockIdx.x >> 1), nkt, (int)(gridDim.x >> 1) / nkt, hpg, bh, kt);
    const int k0 = kt * 128;
    const int nqt = n_pad / BQ;                           // query tiles of 64 rows
    const int i_begin = causal ? 2 * kt : 0;
    const int bb = bh / Hkv, hk = bh - bb * Hkv;
    const int hq0 = hk * (kGrouped ? group : 1) - bh * (kGrouped ? group : 1);   // query head in batch = flat index + hq0
    const int niter_all = (kGrouped ? group : 1) * (nqt - i_begin);
    struct TileWalk {
        int qh, qi, first, end;
        __device__ void next()
        {
            ++qi;
            if (kGrouped && qi == end) { qi = first; ++qh; }
        }
    };
    const TileWalk walk0{kGrouped ? bh * group : bh, i_begin, i_begin, nqt};

    if (tid == 0) {
        for (int b = 0; b < W_COUNT; ++b)
            mbar_init(bars + b, (b == W_P || b == W_DS || b == W_EPI) ? 256u : (b == W_DQR) ? 128u : 1u);
        *abortp = (smem_u32(sm) & 1023u) ? 1u : 0u;
        if (*abortp && status) atomicCAS(status, 0u, (unsigned)WERR_ALIGN);
        fence_mbar_init();
        prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV); prefetch_tensormap(&mapdO);
        prefetch_tensormap(&mapdK); prefetch_tensormap(&mapdV);
    }
    if (warp == kMmaWarp) { tmem_alloc(tmem_base_s, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_base_s;
    const int niter = (*abortp == 0) ? niter_all : 0;

    if (warp >= kLoadWarp) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
      if (warp == kLoadWarp) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && niter > 0) {
            mbar_arrive_expect_tx(bars + W_KV, 8 * SM::kBoxK);
            for (int b = 0; b < 4; ++b) {
                tma_load_4d(sK + b * SM::kBoxK, &mapK, bars + W_KV, 64 * b, k0, hk, bb);
                tma_load_4d(sV + b * SM::kBoxK, &mapV, bars + W_KV, 64 * b, k0, hk, bb);
            }
        }
        const int nq_per = nqt - i_begin;
        auto tile_of = [&](int it, int &qh, int &q0) {
            const int hh = kGrouped ? it / nq_per : 0;
            qh = (kGrouped ? bh * group : bh) + hh;
            q0 = (i_begin + it - hh * nq_per) * BQ;
        };
        auto load_qown = [&](int it) {        // this pass's d-half of Q_it, with -L log2e and -D of its 64 queries
            int qh, q0;
            tile_of(it, qh, q0);
            const int s = it & 1;
            uint8_t *dst = sQ + (1 + s) * SM::kHalf;
            mbar_arrive_expect_tx(bars + W_QOWN + s, SM::kHalf + 512);
            for (int b = 0; b < 2; ++b) tma_load_4d(dst + b * SM::kBoxQ, &mapQ, bars + W_QOWN + s, 128 * pass + 64 * b, q0, qh + hq0, bb);
            bulk_load_1d(sL + s * 64, Lp + (size_t)qh * n_pad + q0, 256, bars + W_QOWN + s);
            bulk_load_1d(sD + s * 64, Dp + (size_t)qh * n_pad + q0, 256, bars + W_QOWN + s);
        };
        auto load_qoth = [&](int it) {        // the other d-half of Q_it (read by S(it) only)
            int qh, q0;
            tile_of(it, qh, q0);
            mbar_arrive_expect_tx(bars + W_QOTH, SM::kHalf);
            for (int b = 0; b < 2; ++b) tma_load_4d(sQ + b * SM::kBoxQ, &mapQ, bars + W_QOTH, 128 * (1 - pass) + 64 * b, q0, qh + hq0, bb);
        };
        auto load_do = [&](int it) {          // dO_it, all 256 columns
            int qh, q0;
            tile_of(it, qh, q0);
            mbar_arrive_expect_tx(bars + W_DOFULL, 4 * SM::kBoxQ);
            for (int b = 0; b < 4; ++b) tma_load_4d(sdO + b * SM::kBoxQ, &mapdO, bars + W_DOFULL, 64 * b, q0, qh + hq0, bb);
        };
        if (lane == 0 && niter > 0) {
            load_qown(0);
            load_qoth(0);
            load_do(0);
            if (niter > 1) load_qown(1);
        }
        // Refills, in the order in which the commits they wait for happen: the other half of Q_{it+1} when S(it) has
        // completed, dO_{it+1} when dV(it) has, the owned half of Q_{it+2} when dK(it) has.  The next phase of each of
        // these barriers needs the refill that follows the wait, so a parity wait here is never a phase behind.
        for (int it = 0; it < niter; ++it) {
            if (it + 1 < niter) {
                if (!mbar_wait(bars + W_S, it & 1, abortp, status, WERR_EMPTY)) break;
                if (lane == 0) load_qoth(it + 1);
                if (!mbar_wait(bars + W_DOEMPTY, it & 1, abortp, status, WERR_EMPTY)) break;
                if (lane == 0) load_do(it + 1);
            }
            if (it + 2 < niter) {
                if (!mbar_wait(bars + W_QEMPTY + (it & 1), (it >> 1) & 1, abortp, status, WERR_EMPTY)) break;
                if (lane == 0) load_qown(it + 2);
            }
            __syncwarp();
        }
      } else if (warp == kMmaWarp && lane == 0) {
        // ------------------------------------------------------------------- UMMA issuer (one thread)
        constexpr uint32_t idesc_st = idesc_bf16_f32(128, 64, 0, 0);     // S^T, dP^T: 128 keys x 64 queries
        constexpr uint32_t idesc_acc = idesc_bf16_f32(128, 128, 0, 1);   // dV, dK: A in TMEM, B MN-major, 128 columns of d
        constexpr uint32_t idesc_dq = idesc_bf16_f32(128, 64, 1, 1);     // dQ^T: 128 columns of d x 64 queries
        const uint64_t km_proto = smem_desc_sw128(0, 16, 1024);
        const uint64_t mnq_proto = smem_desc_sw128(0, SM::kBoxQ, 1024);  // MN-major over boxes of 64 rows (Q, dO, dS^T)
        const uint64_t mnk_proto = smem_desc_sw128(0, SM::kBoxK, 1024);  // MN-major over boxes of 128 rows (K)
        const uint32_t km_hi = (uint32_t)(km_proto >> 32), mnq_hi = (uint32_t)(mnq_proto >> 32), mnk_hi = (uint32_t)(mnk_proto >> 32);
        const uint32_t km_lo = (uint32_t)km_proto, mnq_lo = (uint32_t)mnq_proto, mnk_lo = (uint32_t)mnk_proto;
        auto field = [](const void *ptr) { return (smem_u32(ptr) >> 4) & 0x3FFFu; };
        const uint32_t k_km = km_lo + field(sK), v_km = km_lo + field(sV);
        const uint32_t qoth_km = km_lo + field(sQ), qown_km0 = km_lo + field(sQ + SM::kHalf);
        const uint32_t qown_mn0 = mnq_lo + field(sQ + SM::kHalf);
        const uint32_t do_km = km_lo + field(sdO), do_mn = mnq_lo + field(sdO + 2 * pass * SM::kBoxQ);
        const uint32_t kp_mn = mnk_lo + field(sK + 2 * pass * SM::kBoxK), ds_mn = mnq_lo + field(sdS);
        constexpr uint32_t kHalfF = (uint32_t)(SM::kHalf >> 4);
        auto moff = [](int ks) { return (uint32_t)((ks * 2048) >> 4); };
        // S^T(it): sixteen k-steps over the four 64-column boxes of d; box bx of K against box bx of Q_it, which sits in
        // the owned half-slot (tile parity) or in the other one
        auto issue_S = [&](int it) {
            const uint32_t qown_km = qown_km0 + (uint32_t)(it & 1) * kHalfF;
#pragma unroll
            for (int bx = 0; bx < 4; ++bx) {
                const uint32_t a = k_km + (uint32_t)((bx * SM::kBoxK) >> 4);
                const uint32_t b = ((bx >> 1) == pass ? qown_km : qoth_km) + (uint32_t)(((bx & 1) * SM::kBoxQ) >> 4);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (bx == 0 && q == 0) umma_ss2<false>(tbase + colS, a, km_hi, b, km_hi, idesc_st);
                    else umma_ss2<true>(tbase + colS, a + (uint32_t)((q * 32) >> 4), km_hi, b + (uint32_t)((q * 32) >> 4), km_hi, idesc_st);
                }
            }
            umma_commit(bars + W_S);
        };
        bool ok = niter > 0 && mbar_wait(bars + W_KV, 0, abortp, status, WERR_KV);
        ok = ok && mbar_wait(bars + W_QOWN + 0, 0, abortp, status, WERR_FULL) && mbar_wait(bars + W_QOTH, 0, abortp, status, WERR_FULL);
        if (ok) {
            tc_fence_after();
            issue_S(0);
        }
        for (int it = 0; ok && it < niter; ++it) {
            const int s = it & 1;
            if (!mbar_wait(bars + W_DOFULL, it & 1, abortp, status, WERR_FULL)) break;
            tc_fence_after();
#pragma unroll
            for (int bx = 0; bx < 4; ++bx) {       // dP^T(it) = V dO_it^T over all 256 columns
                const uint32_t a = v_km + (uint32_t)((bx * SM::kBoxK) >> 4), b = do_km + (uint32_t)((bx * SM::kBoxQ) >> 4);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (bx == 0 && q == 0) umma_ss2<false>(tbase + colDP, a, km_hi, b, km_hi, idesc_st);
                    else umma_ss2<true>(tbase + colDP, a + (uint32_t)((q * 32) >> 4), km_hi, b + (uint32_t)((q * 32) >> 4), km_hi, idesc_st);
                }
            }
            umma_commit(bars + W_DP);
            if (!mbar_wait(bars + W_P, it & 1, abortp, status, WERR_PDS)) break;
            if (it + 1 < niter) {       // S(it+1)'s operands, probed here so that dV and S are issued back to back
                if (!mbar_wait(bars + W_QOWN + ((it + 1) & 1), ((it + 1) >> 1) & 1, abortp, status, WERR_FULL)) break;
                if (!mbar_wait(bars + W_QOTH, (it + 1) & 1, abortp, status, WERR_FULL)) break;
            }
            tc_fence_after();
            // dV[:, pass] += P^T dO_it[:, pass]: 64 queries = four k-steps; P^T bf16 at columns 0-15 (queries 0-31) and
            // 32-47 (queries 32-63) of the S^T region
            if (it > 0) umma_ts2<true>(tbase + colDV, tbase + colS, do_mn, mnq_hi, idesc_acc);
            else        umma_ts2<false>(tbase + colDV, tbase + colS, do_mn, mnq_hi, idesc_acc);
#pragma unroll
            for (int ks = 1; ks < 4; ++ks)
                umma_ts2<true>(tbase + colDV, tbase + colS + 32 * (ks >> 1) + 8 * (ks & 1), do_mn + moff(ks), mnq_hi, idesc_acc);
            umma_commit(bars + W_DOEMPTY);
            if (it + 1 < niter) issue_S(it + 1);
            if (!mbar_wait(bars + W_DS, it & 1, abortp, status, WERR_PDS)) break;
            if (it > 0 && !mbar_wait(bars + W_DQR, (it - 1) & 1, abortp, status, WERR_DQR)) break;   // dQ(it-1) read out
            tc_fence_after();
            const uint32_t q_mn = qown_mn0 + (uint32_t)s * kHalfF;
            if (it > 0) umma_ts2<true>(tbase + colDK, tbase + colDP, q_mn, mnq_hi, idesc_acc);
            else        umma_ts2<false>(tbase + colDK, tbase + colDP, q_mn, mnq_hi, idesc_acc);
#pragma unroll
            for (int ks = 1; ks < 4; ++ks)
                umma_ts2<true>(tbase + colDK, tbase + colDP + 32 * (ks >> 1) + 8 * (ks & 1), q_mn + moff(ks), mnq_hi, idesc_acc);
            umma_commit(bars + W_QEMPTY + s);
            // dQ_it^T[:, pass] = K[:, pass]^T dS^T: 128 keys = eight k-steps
            umma_ss2<false>(tbase + colDQ, kp_mn, mnk_hi, ds_mn, mnq_hi, idesc_dq);
#pragma unroll
            for (int ks = 1; ks < 8; ++ks)
                umma_ss2<true>(tbase + colDQ, kp_mn + moff(ks), mnk_hi, ds_mn + moff(ks), mnq_hi, idesc_dq);
            umma_commit(bars + W_DQ);
        }
      }
    } else if (warp >= kReduceWarp0) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 144;");
        // ------------------------------------------------- dQ warps: lanes are the 128 columns of this pass's d-half
        const int lane_row = 32 * (warp % 4) + lane;
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        const bool col_exists = 128 * pass + lane_row < d;      // (the accumulator row is 256 wide; columns past d stay zero)
        TileWalk wr = walk0;
        for (int it = 0; it < niter; ++it) {
            const int q0 = wr.qi * BQ, qh = wr.qh;
            wr.next();
            if (!mbar_wait(bars + W_DQ, it & 1, abortp, status, WERR_DQ)) break;
            tc_fence_after();
            uint32_t r[2][32];
            tmem_ld(lane_addr + colDQ, r[0]);
            tmem_ld(lane_addr + colDQ + 32, r[1]);
            tc_wait_ld();
            tc_fence_before();
            mbar_arrive(bars + W_DQR);      // the columns are free again; the reds go out from registers
            float *dst = dQacc + ((size_t)qh * n + q0) * DW + 128 * pass + lane_row;
            const int valid = col_exists ? min(BQ, n - q0) : 0;
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    if (32 * t + e < valid) red_add_f32(dst + (size_t)(32 * t + e) * DW, __uint_as_float(r[t][e]));
        }
    } else {
        // ----------------------------------------------------------- elementwise warps 0-7
        asm volatile("setmaxnreg.inc.sync.aligned.u32 144;");
        const int wg = warp / 4;                          // query columns [32 wg, 32 wg + 32) of the 64-query tile
        const int lane_row = 32 * (warp % 4) + lane;      // TMEM lane of this thread = key index in the tile
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        uint64_t p2[16];                                  // this thread's 32 probabilities of the current tile, as fp32 pairs
        const uint64_t sl2 = pack_f32x2(scale_log2, scale_log2);
        const int qc0 = 32 * wg;
        bool ok = true;

        TileWalk wp = walk0;
        auto p_phase = [&](int it) -> bool {
            const int s = it & 1;
            // causal: query (tile qi of 64, column q) sees key (tile kt of 128, row lane_row) iff qi*64 + q >= kt*128 + lane_row
            const int rel = wp.qi * BQ - k0;
            const bool masked = causal && rel < 128;        // p_phase runs for it = 0, 1, 2, ... in order
            wp.next();
            if (!mbar_wait(bars + W_S, it & 1, abortp, status, WERR_SDP)) return false;
            tc_fence_after();
            const float *Ls = sL + s * 64;     // -L log2e
            uint32_t rs[32];
            tmem_ld(lane_addr + colS + qc0, rs);
            tc_wait_ld();
            uint32_t pk[16];
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
                const ulonglong2 l4 = *reinterpret_cast<const ulonglong2 *>(Ls + qc0 + e);   // two pairs
                const uint64_t t0 = fma_f32x2(pack_f32x2(__uint_as_float(rs[e]), __uint_as_float(rs[e + 1])), sl2, l4.x);
                const uint64_t t1 = fma_f32x2(pack_f32x2(__uint_as_float(rs[e + 2]), __uint_as_float(rs[e + 3])), sl2, l4.y);
                float a0, a1, a2, a3;
                unpack_f32x2(t0, a0, a1);
                unpack_f32x2(t1, a2, a3);
                a0 = ex2(a0); a1 = ex2(a1); a2 = ex2(a2); a3 = ex2(a3);
                if (masked) {
                    const int q = qc0 + e + rel;
                    if (q < lane_row) a0 = 0.f;
                    if (q + 1 < lane_row) a1 = 0.f;
                    if (q + 2 < lane_row) a2 = 0.f;
                    if (q + 3 < lane_row) a3 = 0.f;
                }
                p2[e / 2] = pack_f32x2(a0, a1);
                p2[e / 2 + 1] = pack_f32x2(a2, a3);
                pk[e / 2] = pack_bf16(a0, a1);
                pk[e / 2 + 1] = pack_bf16(a2, a3);
            }
            tmem_st(lane_addr + colS + qc0, pk);          // over the first 16 of the 32 columns just read
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bars + W_P);
            return true;
        };

        // (one loop, entered a step early, so that the P phase is inlined once: the roles' hot code is what the
        // schedulers keep fetching, and the kernel measurably runs faster the smaller it is)
        ok = niter > 0;
        for (int it = -1; ok && it < niter; ++it) {
          if (it >= 0) {
            const int s = it & 1;
            // dS-phase: dS^T = P^T o (dP^T - D)   (the factor `scale` is applied to dK and dQ at the end).
            // dP(it) complete also means dQ(it-1), issued before it, has read the dS^T tile.
            if (!mbar_wait(bars + W_DP, it & 1, abortp, status, WERR_SDP)) { ok = false; break; }
            tc_fence_after();
            const float *Ds = sD + s * 64;     // -D
            uint32_t rd[32];
            tmem_ld(lane_addr + colDP + qc0, rd);
            tc_wait_ld();
            uint32_t gk[16];
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
                const ulonglong2 d4 = *reinterpret_cast<const ulonglong2 *>(Ds + qc0 + e);
                const uint64_t u0 = add_f32x2(pack_f32x2(__uint_as_float(rd[e]), __uint_as_float(rd[e + 1])), d4.x);
                const uint64_t u1 = add_f32x2(pack_f32x2(__uint_as_float(rd[e + 2]), __uint_as_float(rd[e + 3])), d4.y);
                float g0, g1, g2, g3;
                unpack_f32x2(mul_f32x2(p2[e / 2], u0), g0, g1);
                unpack_f32x2(mul_f32x2(p2[e / 2 + 1], u1), g2, g3);
                gk[e / 2] = pack_bf16(g0, g1);
                gk[e / 2 + 1] = pack_bf16(g2, g3);
            }
            tmem_st(lane_addr + colDP + qc0, gk);
            // dS^T row (this key) into the MN-major tile: 128-byte row of 64 queries, 16-byte chunks 4 wg .. 4 wg + 3, swizzled
            uint8_t *rowp = sdS + lane_row * 128;
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int chunk = (4 * wg + jj) ^ (lane_row & 7);
                *reinterpret_cast<uint4 *>(rowp + chunk * 16) = make_uint4(gk[4 * jj], gk[4 * jj + 1], gk[4 * jj + 2], gk[4 * jj + 3]);
            }
            tc_wait_st();
            tc_fence_before();
            fence_proxy_async_smem();
            mbar_arrive(bars + W_DS);
          }
            if (it + 1 < niter) ok = p_phase(it + 1);
        }
        if (ok && mbar_wait(bars + W_DQ, (niter - 1) & 1, abortp, status, WERR_DQ)) {
            // All UMMAs have completed (one issuing thread; dQ is its last product).  dV[:, pass] and scale*dK[:, pass] go
            // out as bf16 through the first two boxes of the V and K tiles (no longer read) and TMA stores; rows past n and
            // columns past d are clipped by the tensor map.
            tc_fence_after();
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const uint32_t col = (which == 0 ? colDV : colDK) + 64 * wg;
                const float mul = which == 0 ? 1.f : scale;
                uint8_t *stage = which == 0 ? sV : sK;
#pragma unroll
                for (int c = 0; c < 64; c += 32) {
                    uint32_t r[32];
                    tmem_ld(lane_addr + col + c, r);
                    tc_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(r[e + 0]) * mul, __uint_as_float(r[e + 1]) * mul);
                        v.y = pack_bf16(__uint_as_float(r[e + 2]) * mul, __uint_as_float(r[e + 3]) * mul);
                        v.z = pack_bf16(__uint_as_float(r[e + 4]) * mul, __uint_as_float(r[e + 5]) * mul);
                        v.w = pack_bf16(__uint_as_float(r[e + 6]) * mul, __uint_as_float(r[e + 7]) * mul);
                        const int cabs = 64 * wg + c + e;          // first of 8 columns of the 128-column half
                        const int chunk = ((cabs & 63) >> 3) ^ (lane_row & 7);   // 128-byte swizzle, as the maps expect
                        *reinterpret_cast<uint4 *>(stage + (cabs >> 6) * SM::kBoxK + lane_row * 128 + chunk * 16) = v;
                    }
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(bars + W_EPI);
            if (tid == 0 && mbar_wait(bars + W_EPI, 0, abortp, status, WERR_DQ)) {
                for (int b = 0; b < 2; ++b) {
                    if (128 * pass + 64 * b < d) {       // (a box wholly past the head dimension has nothing to store)
                        tma_store_4d(&mapdV, sV + b * SM::kBoxK, 128 * pass + 64 * b, k0, hk, bb);
                        tma_store_4d(&mapdK, sK + b * SM::kBoxK, 128 * pass + 64 * b, k0, hk, bb);
                    }
                }
                bulk_commit();
                bulk_wait_read<0>();      // shared memory is read before the CTA may exit
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tbase, kTmemCols);
    if (*abortp && tid == kLoadWarp * 32) {
        // A wait expired: copies this thread asked for may still be on their way into the CTA's shared memory.  It
        // stays for a fixed 400,000 cycles (hundreds of times a copy's latency) before the CTA can leave.
        const long long t0 = clock64();
        while (clock64() - t0 < 400000LL) { }
    }
}

template <bool kGrouped>
cudaError_t launch_wide(const Problem &p, const void *Q, const void *K, const void *V, const void *dO, const float *Lp,
                        const float *Dp, void *dK, void *dV, float *dQacc, cudaStream_t st)
{
    CUtensorMap mq, mk, mv, mdo, mdk, mdv;
    const auto bf = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const int hkv = p.kv_heads();
    // p.d <= 256 columns exist in memory: loads fill the rest of a box with zeros, stores drop it
    if (!make_tensor_map_4d_strided(&mq, Q, bf, 2, p.B, p.H, p.n, p.d, p.sq.row, p.sq.head, p.sq.batch, 64, 64) ||
        !make_tensor_map_4d_strided(&mdo, dO, bf, 2, p.B, p.H, p.n, p.d, p.so.row, p.so.head, p.so.batch, 64, 64) ||
        !make_tensor_map_4d_strided(&mk, K, bf, 2, p.B, hkv, p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mv, V, bf, 2, p.B, hkv, p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mdk, dK, bf, 2, p.B, hkv, p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mdv, dV, bf, 2, p.B, hkv, p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64))
        return cudaErrorInvalidValue;
    auto kernel = tc_bwd_wide_kernel<kGrouped>;
    constexpr int kSmem = WideSmem::kTotal;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const int nkt = (p.n + 127) / 128;
    LaunchScope scope(MOA_KERNEL_BWD_KV, st);
    Problem pkv = p;
    pkv.H = hkv;
    pkv.Hkv = 0;
    // two CTAs (the two halves of d) per (K/V head, key tile), adjacent in the grid: they share every load in L2
    kernel<<<(unsigned)(2 * nkt * p.BHkv()), kThreads, kSmem, st>>>(
        mq, mk, mv, mdo, mdk, mdv, Lp, Dp, dQacc, p.n, nkt * 128, p.d, p.causal, p.scale, p.scale * kLog2e, nkt,
        heads_per_group(pkv, nkt), p.group(), hkv, device_status_ptr());
    return cudaGetLastError();
}

}  // namespace

cudaError_t tc_bwd_kv_wide(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                           const float *Lp, const float *Dp, void *dK, void *dV, float *dQacc, cudaStream_t st)
{
    if (p.d <= 128 || p.d > 256 || p.d % 8 || dQacc == nullptr) return cudaErrorInvalidValue;
    return p.group() > 1 ? launch_wide<true>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st)
                         : launch_wide<false>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
}

}  // namespace moa
