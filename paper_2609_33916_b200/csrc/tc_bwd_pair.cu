// Backward attention on pairs of CTAs (tcgen05.mma.cta_group::2), head dimension up to 128, bf16 in,
// fp32 accumulate.  Same mathematics and the same one-writer rule for dK and dV as tc_bwd.cu (the
// paper's (b,ic)-parallel GV pass, applied to GK as well); what changes is who holds which operand.
//
// The two CTAs of a cluster own two adjacent key tiles (128 keys each) of one (batch, head) and walk
// the query tiles together.  The CTA of rank 0 issues every UMMA for both:
//     S^T  = K Q_i^T, dP^T = V dO_i^T   M = 256 keys (128 per CTA), N = 128 queries: each CTA stages
//                                       its own K, V tile and only HALF of the query rows of Q_i, dO_i
//     dV  += P^T dO_i, dK += dS^T Q_i   M = 256, N = 128 (d): P^T, dS^T come from each CTA's TMEM,
//                                       each CTA stages only HALF of the d columns of dO_i, Q_i
//     dQ_i^T = K^T dS^T                 M = 128 (d: 64 rows per CTA), N = 128 queries, contraction over
//                                       all 256 keys of the pair: each CTA holds its d-column half of
//                                       both K tiles, and the dS^T values of its query half from both
//                                       CTAs -- every CTA writes half of its dS^T tile into the other
//                                       CTA's shared memory (plain stores through the cluster window)
// Per query tile and CTA the tensor cores read 192 KB of operands from shared memory instead of 256 KB,
// TMA writes the same 64 KB, and the dQ tile that leaves the CTA is 128 queries x 64 columns that
// already holds the sum over 256 keys: half the staging traffic and half the fp32 adds into the
// accumulator.
// Issue order per query tile i:  dP(i), dV(i), S(i+1), dK(i), dQ(i).
//
// What it measured (B1 H8 n8192 d128, one launch): 0.97 ms against 0.69 ms on single CTAs; without the
// dQ product 0.56 against 0.52 ms.  dK and dV are the same bits as on single CTAs.  Clock stamps of the
// roles (MOA_PAIR_TRACE builds) show why: the loop is bound by its dependency chain -- P phase (1500-1800
// cycles) -> dV -> S -> next P phase, and dS phase -> dK/dQ -> read-out -> dP -> next dS phase, with one
// S^T and one dP^T buffer in a full TMEM -- and not by shared-memory bandwidth: with 40 % less operand
// traffic an UMMA still takes ~100 cycles inside the loop.  A pair adds a cross-SM hop to every hand-off
// on that chain, and the dS^T exchange (16 KB by bulk copy: ~1100 cycles from staged to landed) sits
// between dS(i) and dQ(i) with only dK(i) to hide behind.  The kernel is kept as a selectable form
// (moa_bwd_pair_mode / MOA_BWD_PAIR=1) with its own parity tests; single CTAs stay the default.
//
// TMEM (512 columns per CTA): S^T [0,128), dP^T [128,256), dV [256,384), dK [384,512).  P^T and dS^T
// (bf16) go over the LAST 64 columns of their fp32 sources; the dQ^T tile (an M = 128 pair product puts
// 64 rows x 128 columns on 128 lanes x 64 columns: lanes 64-127 hold columns 64-127) takes the first 64
// columns of dP^T, which are free as soon as dS^T is written.  For that a warpgroup w handles query
// columns [64+32w, 96+32w) first and [32w, 32w+32) second: its two 32-column reads and its two 16-column
// bf16 writes (into [64+32w, 96+32w)) touch only columns it has consumed itself, and step u of every
// thread belongs to query half 1-u, i.e. to the dS^T buffer of CTA 1-u.
//
// Hand-offs.  Copies of both CTAs complete on barriers of rank 0 (armed there for the bytes of both);
// commits arrive on the barrier at the same offset in both CTAs; the elementwise and reduce threads of
// both CTAs arrive on barriers of rank 0, where the issuing thread waits -- rank 1's with relaxed
// cluster arrivals (what they announce, TMEM contents after tcgen05.wait and shared memory after a
// proxy fence, is complete when the instruction issues; a cluster-scope release arrival measured
// ~1200 cycles on the critical path and the kernel ran 50 % slower with it).  The half of a dS^T tile
// that belongs to the other CTA is written to a 16 KB staging tile of the sender and crosses as ONE bulk
// copy (shared memory to the other CTA's shared memory, bytes counted on an mbarrier of the receiver:
// asynchronous proxy end to end, nobody waits for an acknowledgement), issued by a helper thread per CTA
// once the 256 elementwise threads have staged their part; the same helper waits for its own CTA's
// incoming half and tells the issuing thread.  (Per-thread st.async stores were tried first: a thousand
// of them per tile took the dS phase from 500 to 2800 cycles and delayed the TMA loads behind them.)
// CTA 0 sends in the first half of its dS phase, CTA 1 in the second, and dK(i), which needs dS^T only
// in TMEM, is issued before dQ(i): the exchange runs under it.
// A hardware cluster barrier after set-up and before tear-down keeps either CTA from touching the other
// outside its lifetime.  Every mbarrier wait is bounded.  No copy is multicast.
#include "common.cuh"
#include "ptx.cuh"
#include "tensormap.cuh"

#include <atomic>
#include <cstdlib>

namespace moa {
namespace {

using namespace ptx;

constexpr int kThreads = 512;   // warps 0-7 elementwise, 8-11 dQ reduce, 12 TMA, 13 UMMA, 14 dS^T exchange helper, 15 idle
constexpr int kReduceWarp0 = 8, kLoadWarp = 12, kMmaWarp = 13, kHelpWarp = 14;
constexpr int kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr int D = 128;

enum : uint32_t {
    PERR_KV = 0x221, PERR_FULL = 0x222, PERR_EMPTY = 0x223, PERR_SDP = 0x224, PERR_PDS = 0x225, PERR_DQ = 0x226,
    PERR_DQR = 0x227, PERR_ALIGN = 0x228, PERR_STAGE = 0x229, PERR_LD = 0x22A, PERR_DONE = 0x22B, PERR_DSRX = 0x22C
};

// Shared memory of one CTA (bytes).  Every tile sits at the same offset in both CTAs: an UMMA names an
// operand by one address that each CTA applies to its own shared memory.
struct PairSmem {
    static constexpr int offK = 0;                      // K tile, [128 keys][128 d] as two 64-column boxes
    static constexpr int offV = offK + 32768;           // V tile, the same
    static constexpr int offKd = offV + 32768;          // [256 keys of the pair][this CTA's 64 d columns]
    static constexpr int offQr = offKd + 32768;         // [this CTA's 64 query rows][128 d] as two 64-column boxes
    static constexpr int offQc = offQr + 16384;         // [128 query rows][this CTA's 64 d columns]
    static constexpr int offdOr = offQc + 16384;        // dO_i, the row half
    static constexpr int offdOc = offdOr + 16384;       // dO_i, the column half
    static constexpr int offdS = offdOc + 16384;        // dS^T: [256 keys of the pair][this CTA's 64 queries]
    static constexpr int offStage = offdS + 32768;      // 2 x ([32 queries][64 floats]): dQ on its way out
    static constexpr int kStage = 32 * 64 * 4;
    static constexpr int offXs = offStage + 2 * kStage;  // dS^T half on its way to the other CTA: [128 keys][64 queries]
    static constexpr int offL = offXs + 16384;          // 2 x 128 floats, travels with the query tile
    static constexpr int offDd = offL + 2 * 512;        // 2 x 128 floats
    static constexpr int offBar = offDd + 2 * 512;
    static constexpr int kTotal = offBar + 256;
};
static_assert(PairSmem::kTotal <= 232448, "shared memory of one CTA");

enum {
    P_KV = 0, P_QRFULL = 1, P_QCFULL = 3, P_DORFULL = 4, P_DOCFULL = 5, P_LD = 6 /*2*/, P_S = 8, P_DP = 9,
    P_DOCEMPTY = 10, P_QCEMPTY = 11, P_P = 12, P_DS = 13, P_DQ = 14, P_DQR = 15, P_DONE = 16, P_STGFREE = 17,
    P_STGFULL = 18, P_EPI = 19, P_DSRX = 20 /*this CTA's incoming dS^T half*/, P_DSX = 21 /*both halves in place*/,
    P_XS = 22 /*outgoing dS^T half staged*/, P_COUNT = 23
};

#ifdef MOA_PAIR_TRACE
// Debug build only: clock stamps of the first cluster's roles, tile by tile (read back by moa_debug_pair_trace).
__device__ long long g_pair_trace[2][64][32];
#define PT(rank_, it_, slot_) do { if (blockIdx.x < 2 && (it_) < 64) g_pair_trace[rank_][it_][slot_] = clock64(); } while (0)
#else
#define PT(rank_, it_, slot_) do { } while (0)
#endif

__device__ __forceinline__ void red_add_f32(float *addr, float a)
{
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(addr), "f"(a) : "memory");
}

template <bool kBulk, bool kGrouped>
__global__ void __launch_bounds__(kThreads, 1)
tc_bwd_pair_kernel(const __grid_constant__ CUtensorMap mapQr, const __grid_constant__ CUtensorMap mapQc,
                   const __grid_constant__ CUtensorMap mapdOr, const __grid_constant__ CUtensorMap mapdOc,
                   const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                   const __grid_constant__ CUtensorMap mapKd, const __grid_constant__ CUtensorMap mapdQ,
                   const __grid_constant__ CUtensorMap mapdK, const __grid_constant__ CUtensorMap mapdV,
                   const float *__restrict__ Lp, const float *__restrict__ Dp, float *__restrict__ dQacc,
                   int n, int n_pad, int causal, float scale, float scale_log2, int npt, int hpg, int group,
                   int Hkv, int skip_dq, unsigned int *status)
{
    using SM = PairSmem;
    constexpr uint32_t colS = 0, colDP = 128, colDV = 256, colDK = 384, colDQ = 128, kBf = 64 /*bf16 copies: last 64 columns*/;
    extern __shared__ __align__(1024) uint8_t sm[];
    uint8_t *sK = sm + SM::offK, *sV = sm + SM::offV, *sKd = sm + SM::offKd, *sdS = sm + SM::offdS;
    float *sL = reinterpret_cast<float *>(sm + SM::offL);
    float *sD = reinterpret_cast<float *>(sm + SM::offDd);
    uint64_t *bars = reinterpret_cast<uint64_t *>(sm + SM::offBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bars + P_COUNT);
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(bars + P_COUNT + 1);

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const uint32_t rank = cluster_ctarank();
    int bh, pt;                               // causal: pair 0 has the most query tiles and goes first
    job_from_block((int)(blockIdx.x >> 1), npt, (int)(gridDim.x >> 1) / npt, hpg, bh, pt);
    const int kt = 2 * pt + (int)rank;        // this CTA's key tile (may lie past the last one: all zeros, nothing stored)
    const int k0 = kt * 128;
    const int nqt = n_pad / 128;
    const int i_begin = causal ? 2 * pt : 0;  // first query tile either CTA of the pair needs
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
        for (int b = 0; b < P_COUNT; ++b) {
            // P_P, P_DS, P_DQR: this CTA's own threads arrive on its own barrier; rank 1's are forwarded to rank 0's by
            // one thread each (one more arrival there)
            const uint32_t fwd = rank == 0 ? 1u : 0u;
            const uint32_t cnt = (b == P_P || b == P_DS) ? 256u + fwd : (b == P_DQR) ? 128u + fwd
                               : (b == P_EPI || b == P_XS) ? 256u : (b == P_STGFULL) ? 128u : (b == P_DSX) ? 2u : 1u;
            mbar_init(bars + b, cnt);
        }
        *abortp = (smem_u32(sm) & 1023u) ? 1u : 0u;
        if (*abortp && status) atomicCAS(status, 0u, (unsigned)PERR_ALIGN);
        fence_mbar_init();
        prefetch_tensormap(&mapQr); prefetch_tensormap(&mapQc); prefetch_tensormap(&mapdOr); prefetch_tensormap(&mapdOc);
        prefetch_tensormap(&mapK); prefetch_tensormap(&mapV); prefetch_tensormap(&mapKd);
        if (kBulk) prefetch_tensormap(&mapdQ);
        prefetch_tensormap(&mapdK); prefetch_tensormap(&mapdV);
    }
    if (warp == kMmaWarp) { tmem_alloc_pair(tmem_base_s, kTmemCols); tmem_relinquish_pair(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();        // the other CTA's barriers are initialised before anything arrives on them
    tc_fence_after();
    const uint32_t tbase = *tmem_base_s;
    const int niter = (*abortp == 0) ? niter_all : 0;
    // barriers of rank 0 that both CTAs' threads arrive on or both CTAs' copies complete on
    auto lead = [&](int b) { return mapa_u32(smem_u32(bars + b), 0); };

    if (warp >= kLoadWarp) {
      // 512 threads start with 128 registers each; the elementwise warps take 144, paid for by the reduce warps
      // (120: they hold a 64-value tile) and this warpgroup (104)
      asm volatile("setmaxnreg.dec.sync.aligned.u32 104;");
      if (warp == kLoadWarp) {
        // ------------------------------------------------------------------ TMA producer (one per CTA)
        const int kc = 64 * (int)rank;        // this CTA's d-column half
        const int qr = 64 * (int)rank;        // this CTA's query-row half inside a tile
        if (lane == 0 && niter > 0) {
            const uint32_t kvbytes = skip_dq ? 65536u : 98304u;
            if (rank == 0) mbar_arrive_expect_tx(bars + P_KV, 2 * kvbytes);
            const uint32_t bar = lead(P_KV);
            for (int b = 0; b < 2; ++b) {
                tma_load_4d_pair(sK + b * 16384, &mapK, bar, 64 * b, k0, hk, bb);
                tma_load_4d_pair(sV + b * 16384, &mapV, bar, 64 * b, k0, hk, bb);
            }
            if (!skip_dq) tma_load_4d_pair(sKd, &mapKd, bar, kc, 2 * pt * 128, hk, bb);
        }
        // (query head, first query row) of iteration `it`; with shared K/V heads the iterations run over the
        // query tiles of one query head after the other
        const int nq_per = nqt - i_begin;
        auto tile_of = [&](int it, int &qh, int &q0) {
            const int hh = kGrouped ? it / nq_per : 0;
            qh = (kGrouped ? bh * group : bh) + hh;
            q0 = (i_begin + it - hh * nq_per) * 128;
        };
        auto load_qr = [&](int it) {          // the row half of Q: B operand of S^T
            int qh, q0;
            tile_of(it, qh, q0);
            uint8_t *dst = sm + SM::offQr;
            if (rank == 0) mbar_arrive_expect_tx(bars + P_QRFULL, 2 * 16384);
            const uint32_t bar = lead(P_QRFULL);
            tma_load_4d_pair(dst, &mapQr, bar, 0, q0 + qr, qh + hq0, bb);
            tma_load_4d_pair(dst + 8192, &mapQr, bar, 64, q0 + qr, qh + hq0, bb);
        };
        auto load_qc = [&](int it) {          // the column half of Q: B operand of dK
            int qh, q0;
            tile_of(it, qh, q0);
            if (rank == 0) mbar_arrive_expect_tx(bars + P_QCFULL, 2 * 16384);
            tma_load_4d_pair(sm + SM::offQc, &mapQc, lead(P_QCFULL), kc, q0, qh + hq0, bb);
        };
        auto load_ld = [&](int it) {          // -L log2e and -D of the tile's 128 queries (this CTA's own barrier)
            int qh, q0;
            tile_of(it, qh, q0);
            const int s = it & 1;
            mbar_arrive_expect_tx(bars + P_LD + s, 1024);
            bulk_load_1d(sL + s * 128, Lp + (size_t)qh * n_pad + q0, 512, bars + P_LD + s);
            bulk_load_1d(sD + s * 128, Dp + (size_t)qh * n_pad + q0, 512, bars + P_LD + s);
        };
        auto load_dor = [&](int it) {         // the row half of dO: B operand of dP^T
            int qh, q0;
            tile_of(it, qh, q0);
            if (rank == 0) mbar_arrive_expect_tx(bars + P_DORFULL, 2 * 16384);
            const uint32_t bar = lead(P_DORFULL);
            tma_load_4d_pair(sm + SM::offdOr, &mapdOr, bar, 0, q0 + qr, qh + hq0, bb);
            tma_load_4d_pair(sm + SM::offdOr + 8192, &mapdOr, bar, 64, q0 + qr, qh + hq0, bb);
        };
        auto load_doc = [&](int it) {         // the column half of dO: B operand of dV
            int qh, q0;
            tile_of(it, qh, q0);
            if (rank == 0) mbar_arrive_expect_tx(bars + P_DOCFULL, 2 * 16384);
            tma_load_4d_pair(sm + SM::offdOc, &mapdOc, lead(P_DOCFULL), kc, q0, qh + hq0, bb);
        };
        if (lane == 0 && niter > 0) {
            load_qr(0); load_ld(0); load_dor(0); load_doc(0); load_qc(0);
            if (niter > 1) load_ld(1);
        }
        // Every tile half has ONE slot, refilled as soon as the UMMAs that read it have completed (their commits arrive
        // in both CTAs) and wanted again about one tile time later: Q rows of tile it+2 after S(it+1), dO rows of it+1
        // after dP(it), dO columns of it+1 after dV(it), Q columns of it+1 after dK(it); L, D (two slots) of it+2 after
        // dK(it) as well, when the elementwise threads have read tile it's.  The waits below are in the order in which
        // those commits happen, and each next phase of a barrier needs the refill that follows the wait for the one
        // before, so a parity wait here is never a phase behind.
        bool live = niter > 1;
        if (live) {
            live = mbar_wait(bars + P_S, 0, abortp, status, PERR_EMPTY);
            if (live && lane == 0) load_qr(1);
        }
        for (int it = 0; live && it < niter; ++it) {
            if (it + 1 < niter) {
                if (!mbar_wait(bars + P_DP, it & 1, abortp, status, PERR_EMPTY)) break;
                if (lane == 0) load_dor(it + 1);
                if (!mbar_wait(bars + P_DOCEMPTY, it & 1, abortp, status, PERR_EMPTY)) break;
                if (lane == 0) load_doc(it + 1);
                if (it + 2 < niter) {
                    if (!mbar_wait(bars + P_S, (it + 1) & 1, abortp, status, PERR_EMPTY)) break;
                    if (lane == 0) load_qr(it + 2);
                }
                if (!mbar_wait(bars + P_QCEMPTY, it & 1, abortp, status, PERR_EMPTY)) break;
                if (lane == 0) {
                    load_qc(it + 1);
                    if (it + 2 < niter) load_ld(it + 2);
                }
            }
            __syncwarp();
        }
      } else if (warp == kMmaWarp && lane == 0 && rank == 0) {
        // ------------------------------------------------------------------- UMMA issuer (rank 0 only)
        // Issue order per query tile i:  dP(i), dV(i), S(i+1), dK(i), dQ(i).
        constexpr uint32_t idesc_st = idesc_bf16_f32(256, 128, 0, 0);    // S^T, dP^T
        constexpr uint32_t idesc_acc = idesc_bf16_f32(256, 128, 0, 1);   // dV, dK: A in TMEM, B MN-major
        constexpr uint32_t idesc_dq = idesc_bf16_f32(128, 128, 1, 1);    // dQ^T: A and B MN-major, 64 rows per CTA
        const uint64_t km_proto = smem_desc_sw128(0, 16, 1024), mn_proto = smem_desc_sw128(0, 16384, 1024);
        const uint32_t km_hi = (uint32_t)(km_proto >> 32), mn_hi = (uint32_t)(mn_proto >> 32);
        const uint32_t km_lo = (uint32_t)km_proto, mn_lo = (uint32_t)mn_proto;
        auto field = [](const void *ptr) { return (smem_u32(ptr) >> 4) & 0x3FFFu; };
        const uint32_t k_km = km_lo + field(sK), v_km = km_lo + field(sV);
        const uint32_t kd_mn = mn_lo + field(sKd), ds_mn = mn_lo + field(sdS);
        const uint32_t qr_km = km_lo + field(sm + SM::offQr), qc_mn = mn_lo + field(sm + SM::offQc);
        const uint32_t dor_km = km_lo + field(sm + SM::offdOr), doc_mn = mn_lo + field(sm + SM::offdOc);
        // k-steps of 16: K-major operands advance 32 bytes inside a 64-column box (A: boxes of 128 rows, B halves: of
        // 64 rows); MN-major operands advance 16 rows of 128 bytes
        auto koffA = [](int ks) { return (uint32_t)(((ks / 4) * 16384 + (ks % 4) * 32) >> 4); };
        auto koffB = [](int ks) { return (uint32_t)(((ks / 4) * 8192 + (ks % 4) * 32) >> 4); };
        auto moff = [](int ks) { return (uint32_t)((ks * 2048) >> 4); };
        // P^T / dS^T in TMEM: the eight columns that hold queries [16 j, 16 j + 16) (see the column plan at the top).
        // The k-steps go in query order, so dV and dK add up in the same order as on single CTAs.
        auto acol = [](int j) { return (uint32_t)(64 + 32 * ((j >> 1) & 1) + 16 * (1 - (j >> 2)) + 8 * (j & 1)); };
        auto issue_S = [&]() {
            umma_ss2_pair<false>(tbase + colS, k_km, km_hi, qr_km, km_hi, idesc_st);
#pragma unroll
            for (int ks = 1; ks < 8; ++ks)
                umma_ss2_pair<true>(tbase + colS, k_km + koffA(ks), km_hi, qr_km + koffB(ks), km_hi, idesc_st);
            umma_commit_pair(bars + P_S);
        };
        bool ok = niter > 0 && mbar_wait(bars + P_KV, 0, abortp, status, PERR_KV);
        ok = ok && mbar_wait(bars + P_QRFULL, 0, abortp, status, PERR_FULL);
        if (ok) {
            tc_fence_after();
            issue_S();
        }
        for (int it = 0; ok && it < niter; ++it) {
            PT(0, it, 0);
            if (!mbar_wait(bars + P_DORFULL, it & 1, abortp, status, PERR_FULL)) break;
            PT(0, it, 1);
            // dP(it) overwrites the columns that hold dQ(it-1): read out by the reduce warps of both CTAs
            if (!skip_dq && it > 0 && !mbar_wait(bars + P_DQR, (it - 1) & 1, abortp, status, PERR_DQR)) break;
            PT(0, it, 2);
            tc_fence_after();
            umma_ss2_pair<false>(tbase + colDP, v_km, km_hi, dor_km, km_hi, idesc_st);
#pragma unroll
            for (int ks = 1; ks < 8; ++ks)
                umma_ss2_pair<true>(tbase + colDP, v_km + koffA(ks), km_hi, dor_km + koffB(ks), km_hi, idesc_st);
            umma_commit_pair(bars + P_DP);
            PT(0, it, 3);
            if (!mbar_wait(bars + P_P, it & 1, abortp, status, PERR_PDS)) break;
            PT(0, it, 4);
            if (!mbar_wait(bars + P_DOCFULL, it & 1, abortp, status, PERR_FULL)) break;
            PT(0, it, 5);
            tc_fence_after();
            if (it > 0) umma_ts2_pair<true>(tbase + colDV, tbase + colS + acol(0), doc_mn, mn_hi, idesc_acc);
            else        umma_ts2_pair<false>(tbase + colDV, tbase + colS + acol(0), doc_mn, mn_hi, idesc_acc);
#pragma unroll
            for (int j = 1; j < 8; ++j)
                umma_ts2_pair<true>(tbase + colDV, tbase + colS + acol(j), doc_mn + moff(j), mn_hi, idesc_acc);
            umma_commit_pair(bars + P_DOCEMPTY);
            PT(0, it, 6);
            if (it + 1 < niter) {
                if (!mbar_wait(bars + P_QRFULL, (it + 1) & 1, abortp, status, PERR_FULL)) break;
                PT(0, it, 7);
                tc_fence_after();
                issue_S();
            }
            PT(0, it, 8);
            if (!mbar_wait(bars + P_DS, it & 1, abortp, status, PERR_PDS)) break;
            PT(0, it, 9);
            if (!mbar_wait(bars + P_QCFULL, it & 1, abortp, status, PERR_FULL)) break;
            PT(0, it, 10);
            tc_fence_after();
            if (it > 0) umma_ts2_pair<true>(tbase + colDK, tbase + colDP + acol(0), qc_mn, mn_hi, idesc_acc);
            else        umma_ts2_pair<false>(tbase + colDK, tbase + colDP + acol(0), qc_mn, mn_hi, idesc_acc);
#pragma unroll
            for (int j = 1; j < 8; ++j)
                umma_ts2_pair<true>(tbase + colDK, tbase + colDP + acol(j), qc_mn + moff(j), mn_hi, idesc_acc);
            umma_commit_pair(bars + P_QCEMPTY);
            PT(0, it, 11);
            if (!skip_dq) {       // (the atomic-free mode computes dQ in its own query-parallel kernel)
                // both CTAs' dS^T buffers are complete: own halves (P_DS above) and the halves that crossed
                if (!mbar_wait(bars + P_DSX, it & 1, abortp, status, PERR_DSRX)) break;
                tc_fence_after();
                umma_ss2_pair<false>(tbase + colDQ, kd_mn, mn_hi, ds_mn, mn_hi, idesc_dq);
#pragma unroll
                for (int ks = 1; ks < 16; ++ks)
                    umma_ss2_pair<true>(tbase + colDQ, kd_mn + moff(ks), mn_hi, ds_mn + moff(ks), mn_hi, idesc_dq);
                umma_commit_pair(bars + P_DQ);
            }
            PT(0, it, 12);
            if (it == niter - 1) umma_commit_pair(bars + P_DONE);     // once, after the last product
        }
      } else if ((warp == kMmaWarp || warp == kMmaWarp + 2) && lane == 0 && rank == 1) {
        // ------------------------------------------------------- rank 1: arrival forwarders
        // 256 arrivals from another SM on one barrier are slow to add up; rank 1's threads meet on their own CTA's
        // barrier and one thread passes each completed phase on to the issuing CTA (P^T written: warp 13, dS^T: warp 15).
        const int b = warp == kMmaWarp ? P_P : P_DS;
        const uint32_t to = lead(b);
        for (int it = 0; it < niter; ++it) {
            if (!mbar_wait(bars + b, it & 1, abortp, status, PERR_PDS)) break;
            mbar_arrive_relaxed_cluster(to);
        }
      } else if (warp == kHelpWarp && lane == 0 && !skip_dq) {
        // ------------------------------------------------------- dS^T exchange helper (one per CTA)
        // Per tile: sends this CTA's staged half (one bulk copy into the other CTA's dS^T buffer, rows of this CTA's
        // keys), waits until the other CTA's half has landed here, and tells the issuing thread.
        const uint32_t dsx = lead(P_DSX), dqr_fwd = lead(P_DQR);
        const uint32_t dst = mapa_u32(smem_u32(sdS + 16384 * (int)rank), rank ^ 1u);
        const uint32_t dst_bar = mapa_u32(smem_u32(bars + P_DSRX), rank ^ 1u);
        for (int it = 0; it < niter; ++it) {
            mbar_arrive_expect_tx(bars + P_DSRX, 16384);
            if (!mbar_wait(bars + P_XS, it & 1, abortp, status, PERR_DSRX)) break;
            PT(rank, it, 26);
            bulk_copy_to_cluster(dst, sm + SM::offXs, 16384, dst_bar);
            PT(rank, it, 27);
            if (!mbar_wait_cluster(bars + P_DSRX, it & 1, abortp, status, PERR_DSRX)) break;
            PT(rank, it, 28);
            if (rank == 0) mbar_arrive(bars + P_DSX);
            else mbar_arrive_relaxed_cluster(dsx);
            if (rank == 1) {          // and forwards "dQ(it) has been read out of TMEM" of rank 1's reduce warps
                if (!mbar_wait(bars + P_DQR, it & 1, abortp, status, PERR_DQR)) break;
                mbar_arrive_relaxed_cluster(dqr_fwd);
            }
        }
      }
    } else if (warp >= kReduceWarp0) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 120;");
        // ------------------------------------------------- dQ reduce warps
        // The dQ^T tile of this CTA: lane l holds column d = 64 rank + (l % 64) of the 64 query rows
        // 64 (l / 64) + [0, 64) of the tile, already summed over the pair's 256 keys.
        const int lane_row = 32 * (warp % 4) + lane;
        const int half = lane_row >> 6, dcol = lane_row & 63;
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        const bool leader = (tid == kReduceWarp0 * 32);
        TileWalk wr = walk0;
        for (int it = 0; it < (skip_dq ? 0 : niter); ++it) {
            const int q0 = wr.qi * 128, qh = wr.qh;
            wr.next();
            if (!mbar_wait(bars + P_DQ, it & 1, abortp, status, PERR_DQ)) break;
            tc_fence_after();
            uint32_t r[2][32];
            tmem_ld(lane_addr + colDQ, r[0]);
            tmem_ld(lane_addr + colDQ + 32, r[1]);
            tc_wait_ld();
            tc_fence_before();
            mbar_arrive(bars + P_DQR);                 // the columns are free again; the adds go out from registers
            if (kBulk) {
                // Two steps of 32 + 32 query rows: the threads of each lane half fill their [32 rows][64 floats]
                // buffer (a thread writes one column: conflict-free), and the leader hands both buffers to the TMA
                // engine as add-reduces into the fp32 accumulator; rows past n are clipped by the map.
                float *stage = reinterpret_cast<float *>(sm + SM::offStage + half * SM::kStage);
                bool stage_ok = true;
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int g = it * 2 + t;       // running step count
                    if (g >= 1) {
                        if (leader) { bulk_wait_read<0>(); mbar_arrive(bars + P_STGFREE); }   // TMA has read both buffers
                        if (stage_ok && !mbar_wait(bars + P_STGFREE, (g - 1) & 1, abortp, status, PERR_STAGE)) stage_ok = false;
                    }
                    if (stage_ok) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) stage[e * 64 + dcol] = __uint_as_float(r[t][e]);
                        fence_proxy_async_smem();
                    }
                    mbar_arrive(bars + P_STGFULL);
                    if (leader && stage_ok && mbar_wait(bars + P_STGFULL, g & 1, abortp, status, PERR_STAGE)) {
                        tma_reduce_add_3d(&mapdQ, sm + SM::offStage, 64 * (int)rank, q0 + 32 * t, qh);
                        tma_reduce_add_3d(&mapdQ, sm + SM::offStage + SM::kStage, 64 * (int)rank, q0 + 64 + 32 * t, qh);
                        bulk_commit();
                    }
                }
                if (!stage_ok) break;
            } else {
                // one warp-wide red covers 32 consecutive floats of one dQ row: a full 128-byte line
                const int qb = q0 + 64 * half;
                float *dst = dQacc + ((size_t)qh * n + qb) * D + 64 * (int)rank + dcol;
                const int valid = min(64, n - qb);
#pragma unroll
                for (int t = 0; t < 2; ++t)
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (32 * t + e < valid) red_add_f32(dst + (size_t)(32 * t + e) * D, __uint_as_float(r[t][e]));
            }
        }
        if (kBulk && leader) bulk_wait<0>();   // all reduces done before exit
    } else {
        // ----------------------------------------------------------- elementwise warps 0-7
        asm volatile("setmaxnreg.inc.sync.aligned.u32 144;");
        const int wg = warp / 4;                          // query columns [64 + 32 wg, 96 + 32 wg) first, then [32 wg, 32 wg + 32)
        const int lane_row = 32 * (warp % 4) + lane;      // TMEM lane of this thread = key index in this CTA's tile
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        uint64_t p2[32];                                  // this thread's 64 probabilities of the current tile, as fp32 pairs
        const uint64_t sl2 = pack_f32x2(scale_log2, scale_log2);
        // row of this thread's key in the dS^T buffers of both CTAs: [256 keys][64 queries], 128-byte rows, swizzled
        uint8_t *ds_row_own = sdS + (128 * (int)rank + lane_row) * 128;
        uint8_t *ds_row_out = sm + SM::offXs + lane_row * 128;      // staged for the other CTA (same row swizzle)
        bool ok = true;

        TileWalk wp = walk0;
        auto p_phase = [&](int it) -> bool {
            const int s = it & 1;
            // causal: query (tile qi, column q) sees key (tile kt, row lane_row) iff qi*128 + q >= kt*128 + lane_row
            const int rel = (wp.qi - kt) * 128;
            const bool masked = causal && rel < 128;        // p_phase runs for it = 0, 1, 2, ... in order
            wp.next();
            if (tid == 0) PT(rank, it, 16);
            if (!mbar_wait(bars + P_LD + s, (it >> 1) & 1, abortp, status, PERR_LD)) return false;
            if (!mbar_wait(bars + P_S, it & 1, abortp, status, PERR_SDP)) return false;
            if (tid == 0) PT(rank, it, 17);
            tc_fence_after();
            const float *Ls = sL + s * 128;    // -L log2e
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int qc0 = 64 * (1 - u) + 32 * wg;
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
                    p2[16 * u + e / 2] = pack_f32x2(a0, a1);
                    p2[16 * u + e / 2 + 1] = pack_f32x2(a2, a3);
                    pk[e / 2] = pack_bf16(a0, a1);
                    pk[e / 2 + 1] = pack_bf16(a2, a3);
                }
                tmem_st(lane_addr + colS + kBf + 32 * wg + 16 * u, pk);
            }
            tc_wait_st();
            tc_fence_before();
            if (tid == 0) PT(rank, it, 18);
            mbar_arrive(bars + P_P);
            if (tid == 0) PT(rank, it, 19);
            return true;
        };

        ok = niter > 0 && p_phase(0);
        for (int it = 0; ok && it < niter; ++it) {
            const int s = it & 1;
            // dS-phase: dS^T = P^T o (dP^T - D)   (the factor `scale` is applied to dK and dQ at the end).
            // dP(it) complete also means dQ(it-1) has read the dS^T buffers of both CTAs.
            if (tid == 0) PT(rank, it, 20);
            if (!mbar_wait(bars + P_DP, it & 1, abortp, status, PERR_SDP)) { ok = false; break; }
            if (tid == 0) PT(rank, it, 21);
            tc_fence_after();
            const float *Ds = sD + s * 128;    // -D
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int qc0 = 64 * (1 - u) + 32 * wg;
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
                    unpack_f32x2(mul_f32x2(p2[16 * u + e / 2], u0), g0, g1);
                    unpack_f32x2(mul_f32x2(p2[16 * u + e / 2 + 1], u1), g2, g3);
                    gk[e / 2] = pack_bf16(g0, g1);
                    gk[e / 2 + 1] = pack_bf16(g2, g3);
                }
                tmem_st(lane_addr + colDP + kBf + 32 * wg + 16 * u, gk);
                // The 32 values belong to query half 1-u, i.e. to the dS^T buffer of CTA 1-u: row = this key, 16-byte
                // chunks 4 wg .. 4 wg + 3 of the 128-byte row, swizzled.  This CTA's half goes straight into its buffer,
                // the other CTA's into the staging tile that the helper sends (rank 0 stages in its first step, rank 1
                // in its second).
                if (!skip_dq) {
                    const bool own = (uint32_t)(1 - u) == rank;
                    uint8_t *rowp = own ? ds_row_own : ds_row_out;
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        const uint32_t chunk = (uint32_t)((4 * wg + jj) ^ (lane_row & 7));
                        *reinterpret_cast<uint4 *>(rowp + chunk * 16) = make_uint4(gk[4 * jj], gk[4 * jj + 1], gk[4 * jj + 2], gk[4 * jj + 3]);
                    }
                    if (!own) {
                        fence_proxy_async_smem();
                        mbar_arrive(bars + P_XS);
                    }
                }
            }
            tc_wait_st();
            tc_fence_before();
            if (tid == 0) PT(rank, it, 22);
            fence_proxy_async_smem();
            if (tid == 0) PT(rank, it, 23);
            mbar_arrive(bars + P_DS);
            if (tid == 0) PT(rank, it, 24);
            if (it + 1 < niter) ok = p_phase(it + 1);
        }
        if (ok && mbar_wait(bars + P_DONE, 0, abortp, status, PERR_DONE)) {
            // All UMMAs have completed.  dV and scale*dK of this CTA's keys go out as bf16 through the K and V
            // tiles (no longer read) and TMA stores; rows past n are clipped by the tensor map.
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
                        const int cabs = 64 * wg + c + e;          // first of 8 columns
                        const int chunk = ((cabs & 63) >> 3) ^ (lane_row & 7);   // 128-byte swizzle, as the maps expect
                        *reinterpret_cast<uint4 *>(stage + (cabs >> 6) * 16384 + lane_row * 128 + chunk * 16) = v;
                    }
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(bars + P_EPI);
            if (tid == 0 && mbar_wait(bars + P_EPI, 0, abortp, status, PERR_DONE)) {
                if (k0 < n) {
                    for (int b = 0; b < 2; ++b) {
                        tma_store_4d(&mapdV, sV + b * 16384, 64 * b, k0, hk, bb);
                        tma_store_4d(&mapdK, sK + b * 16384, 64 * b, k0, hk, bb);
                    }
                    bulk_commit();
                    bulk_wait_read<0>();      // shared memory is read before the CTA may exit
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abortp && tid == kLoadWarp * 32) {
        // A wait expired: copies this thread asked for may still be on their way into shared memory.  It stays for a
        // fixed 400,000 cycles (hundreds of times a copy's latency) before the pair can leave.
        const long long t0 = clock64();
        while (clock64() - t0 < 400000LL) { }
    }
    // neither CTA leaves, or frees its TMEM, while the other may still read its shared memory, write into it,
    // write its accumulators or arrive on its barriers
    __syncwarp();
    cluster_sync_all();
    if (warp == kMmaWarp) tmem_dealloc_pair(tbase, kTmemCols);
}

template <bool kBulk, bool kGrouped>
cudaError_t launch_pair(const Problem &p, const void *Q, const void *K, const void *V, const void *dO, const float *Lp,
                        const float *Dp, void *dK, void *dV, float *dQacc, cudaStream_t st)
{
    CUtensorMap mqr, mqc, mdor, mdoc, mk, mv, mkd, mdq, mdk, mdv;
    const uint64_t heads = (uint64_t)p.BH();
    const auto bf = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const int hkv = p.kv_heads();
    // p.d <= 128 columns exist in memory: loads fill the rest of a box with zeros, stores drop it
    if (!make_tensor_map_4d_strided(&mqr, Q, bf, 2, p.B, p.H, p.n, p.d, p.sq.row, p.sq.head, p.sq.batch, 64, 64) ||
        !make_tensor_map_4d_strided(&mqc, Q, bf, 2, p.B, p.H, p.n, p.d, p.sq.row, p.sq.head, p.sq.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mdor, dO, bf, 2, p.B, p.H, p.n, p.d, p.so.row, p.so.head, p.so.batch, 64, 64) ||
        !make_tensor_map_4d_strided(&mdoc, dO, bf, 2, p.B, p.H, p.n, p.d, p.so.row, p.so.head, p.so.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mk, K, bf, 2, p.B, hkv, p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mv, V, bf, 2, p.B, hkv, p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mkd, K, bf, 2, p.B, hkv, p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 256, 64) ||
        !make_tensor_map_4d_strided(&mdk, dK, bf, 2, p.B, hkv, p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mdv, dV, bf, 2, p.B, hkv, p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64))
        return cudaErrorInvalidValue;
    // fp32 accumulator as [heads, n, 128] with boxes of 32 rows x 64 floats (no swizzle); also encoded when unused
    if (!make_tensor_map_3d(&mdq, dQacc ? (const void *)dQacc : Q, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, heads, p.n, D, 32, 64))
        return cudaErrorInvalidValue;
    auto kernel = tc_bwd_pair_kernel<kBulk, kGrouped>;
    constexpr int kSmem = PairSmem::kTotal;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const int nkt = (p.n + 127) / 128, npt = (nkt + 1) / 2;
    LaunchScope scope(MOA_KERNEL_BWD_KV, st);
    // one pair of CTAs per (K/V head, pair of key tiles); the block order groups K/V heads
    Problem pkv = p;
    pkv.H = hkv;
    pkv.Hkv = 0;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3((unsigned)(2 * npt * p.BHkv()));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, mqr, mqc, mdor, mdoc, mk, mv, mkd, mdq, mdk, mdv, Lp, Dp, dQacc, p.n, nkt * 128,
                              p.causal, p.scale, p.scale * kLog2e, npt, heads_per_group(pkv, npt), p.group(), hkv,
                              dQacc == nullptr ? 1 : 0, device_status_ptr());
}

}  // namespace

// Whether the 128-column backward runs on CTA pairs: the environment variable MOA_BWD_PAIR (read once per process;
// unset or 0: single CTAs, the faster form; anything else: pairs) unless moa_bwd_pair_mode has set it since.
static std::atomic<int> g_pair_mode{-1};
int bwd_pair_mode(int set)
{
    int cur = g_pair_mode.load(std::memory_order_relaxed);
    if (cur < 0) {
        const char *e = getenv("MOA_BWD_PAIR");
        cur = (e && atoi(e) != 0) ? 1 : 0;
        g_pair_mode.store(cur, std::memory_order_relaxed);
    }
    if (set >= 0) g_pair_mode.store(set ? 1 : 0, std::memory_order_relaxed);
    return cur;
}
bool bwd_pair_enabled() { return bwd_pair_mode(-1) != 0; }

#ifdef MOA_PAIR_TRACE
extern "C" int moa_debug_pair_trace(long long *out)
{
    return (int)cudaMemcpyFromSymbol(out, g_pair_trace, sizeof(long long) * 2 * 64 * 32);
}
#endif

cudaError_t tc_bwd_kv_pair(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                           const float *Lp, const float *Dp, void *dK, void *dV, float *dQacc, int dq_bulk,
                           cudaStream_t st)
{
    if (p.d < 8 || p.d > 128 || p.d % 8 || kernel_d(p.d) != 128) return cudaErrorInvalidValue;
    const bool grouped = p.group() > 1;
    if (dq_bulk) return grouped ? launch_pair<true, true>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st)
                                : launch_pair<true, false>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
    return grouped ? launch_pair<false, true>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st)
                   : launch_pair<false, false>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
}

}  // namespace moa
