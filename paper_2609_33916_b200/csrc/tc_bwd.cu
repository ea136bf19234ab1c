// Backward attention on the sm_100a tensor cores, bf16 in, fp32 accumulate.
//
// One CTA owns 128 keys (one K/V tile) of one (batch, head) and walks the query tiles
// of 128 rows; dK and dV of those keys accumulate in TMEM and are written once, by this
// CTA only (no atomics: the paper's (b,ic)-parallel GV pass, applied to GK as well).
// Per query tile i, with everything transposed so that TMEM lanes are keys:
//     S^T  = K Q_i^T                 (SS-UMMA, both operands K-major)
//     dP^T = V dO_i^T                (SS-UMMA)
//     P^T  = exp2(S^T scale log2e - L_i log2e)         (registers; L from the forward)
//     dS^T = P^T o (dP^T - D_i)                        (D = rowsum(dO o O); the factor
//                                                       `scale` of dK and dQ is applied at the end)
//     dV  += P^T dO_i                (TS-UMMA: P^T bf16 in TMEM, dO_i MN-major in smem)
//     dK  += dS^T Q_i                (D = 128: SS-UMMA, the dS^T tile in smem as K-major A, Q_i MN-major;
//                                     D = 64: TS-UMMA, dS^T bf16 in TMEM)
//     dQ_i = dS K                    (SS-UMMA: dS^T tile in smem as MN-major A, K MN-major)
// dQ_i is one key tile's contribution; it is added into an fp32 [B,H,n,d] accumulator (the contended step the
// dq_mode knob is about): for D = 128 the tile is produced transposed (dQ_i^T = K^T dS^T, lanes = d) and leaves
// either as warp-wide red.global.add.f32 (one full 128-byte line per instruction) or, by default, staged 32 rows
// at a time in shared memory and handed to the TMA engine as cp.reduce.async.bulk.tensor add.f32; D = 64 keeps the
// untransposed tile (UMMA needs M = 128, so lanes stay queries): each reduce warp stages its own 32 rows as two swizzled boxes
// and sends them by the same instruction (default), or the rows leave as red.global.add.v4.f32 (half a sector per lane).
//
// Roles (512 threads; registers are re-split per warpgroup with setmaxnreg: 144 / 144 / 144 / 80): warps 0-7
// elementwise work (thread = TMEM lane = key, the two warpgroups split the query columns), warps 8-11 read each
// finished dQ tile out of TMEM and send it to the accumulator, warp 12 TMA producer (K,V once; Q_i with L_i, D_i
// two tiles ahead in a two-slot ring; dO_i in two slots, or one when the staging buffers of the bulk reduce take
// the other), warp 13 (one thread) UMMA issuer and TMEM owner.
// UMMA issue order per query tile: dP(i), dV(i), S(i+1), then dQ(i), dK(i) (D = 128; dK(i), dQ(i) for D = 64), so that
// the exp2 work of tile i+1 overlaps the dK/dQ UMMAs of tile i, the dS work of tile i overlaps dV(i) and S(i+1), and
// the read-out of dQ(i), which dP(i+1) waits for because the tile sits on the dP^T columns, runs under dK(i).  One thread issues everything: two splits of the issue over two threads
// ({S, dV} | {dP, dK, dQ} and {S, dP, dV} | {dK, dQ}) were correct and 18-22 % slower, because the second thread's
// products then share the in-order pipe with the products at the head of the dependency chain
// dS(i) -> dK(i), dQ(i) -> read-out -> dP(i+1) -> dS(i+1), which is what paces the loop.
//
// TMEM columns (512): S^T [0,128), dP^T [128,256), dV [256,256+D), dK [256+D,256+2D);
// P^T (bf16) overwrites the front of its fp32 source columns (for D = 64 so does dS^T); for D = 128 the dQ
// tile reuses the dP^T columns, which are free once the elementwise threads have read dP^T.
//
// Rows past n need no masking: TMA zero-fills K, V, Q, dO there, the preprocess kernel
// pads L with +inf (so P = 0) and D with 0, and stores are row-guarded.
#include "common.cuh"
#include "ptx.cuh"
#include "tensormap.cuh"

namespace moa {
namespace {

using namespace ptx;

constexpr int kThreads = 512;   // warps 0-7 elementwise, 8-11 dQ reduce, 12 TMA, 13 UMMA, 14-15 idle
constexpr int kReduceWarp0 = 8, kLoadWarp = 12, kMmaWarp = 13;
constexpr int kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;

enum : uint32_t {
    ERR_KV = 0x201, ERR_FULL = 0x202, ERR_EMPTY = 0x203, ERR_SDP = 0x204, ERR_PDS = 0x205, ERR_DQ = 0x206,
    ERR_DQR = 0x207, ERR_ALIGN = 0x208, ERR_STAGE = 0x209
};

__device__ __forceinline__ void red_add_f32(float *addr, float a)
{
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(addr), "f"(a) : "memory");
}

__device__ __forceinline__ void red_add_v4(float *addr, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

// Lp = -L log2(e) and Dp = -rowsum(dO o O), both padded per head to n_pad rows (-inf and 0
// past n).  Stored negated so that the kernels can use them as fma / add operands directly.
// HBM-bound (reads 2 * D * 2 bytes per row): every lane fetches 16 bytes of dO and of O, a row
// takes D/8 lanes, and a warp has kPasses independent row groups in flight before it reduces.
template <int D>
__global__ void __launch_bounds__(256)
bwd_preprocess_kernel(const __nv_bfloat16 *__restrict__ dO, const __nv_bfloat16 *__restrict__ O,
                      const float *__restrict__ L, float *__restrict__ Lp, float *__restrict__ Dp,
                      int n, int n_pad, size_t padded_rows, int H, Strides so, int d)
{
    // d <= D: the head dimension in memory (lanes past it contribute zeros)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");      // the backward kernel behind this one may set itself up
    constexpr int kLanesPerRow = D / 8;
    constexpr int kRowsPerPass = 32 / kLanesPerRow;
    constexpr int kPasses = 4;
    const int lane = threadIdx.x % 32;
    const int sub = lane / kLanesPerRow, l = lane % kLanesPerRow;
    const size_t warp_global = (size_t)blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    const size_t prow0 = warp_global * (kRowsPerPass * kPasses) + sub;
    uint4 a[kPasses], b[kPasses];
    float lv[kPasses];
    bool real[kPasses];
#pragma unroll
    for (int p = 0; p < kPasses; ++p) {
        const size_t prow = prow0 + (size_t)p * kRowsPerPass;
        const size_t bh = prow / (size_t)n_pad;
        const int r = (int)(prow - bh * (size_t)n_pad);
        real[p] = prow < padded_rows && r < n;
        a[p] = b[p] = make_uint4(0u, 0u, 0u, 0u);
        lv[p] = 0.f;
        if (real[p]) {
            const size_t row = bh * (size_t)n + r;                      // row of L: always [B,H,n]
            const size_t bb = bh / (size_t)H;
            const size_t toff = so.at((long long)bb, (long long)(bh - bb * (size_t)H), r);      // first element of the row of dO, O
            if (8 * l < d) {
                a[p] = __ldcs(reinterpret_cast<const uint4 *>(dO + toff) + l);
                b[p] = __ldcs(reinterpret_cast<const uint4 *>(O + toff) + l);
            }
            if (l == 0) lv[p] = L[row];
        }
    }
#pragma unroll
    for (int p = 0; p < kPasses; ++p) {
        const uint32_t x[4] = {a[p].x, a[p].y, a[p].z, a[p].w}, y[4] = {b[p].x, b[p].y, b[p].z, b[p].w};
        float acc = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 u = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&x[i]));
            const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&y[i]));
            acc = fmaf(u.x, v.x, acc);
            acc = fmaf(u.y, v.y, acc);
        }
#pragma unroll
        for (int o = kLanesPerRow / 2; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        const size_t prow = prow0 + (size_t)p * kRowsPerPass;
        if (l == 0 && prow < padded_rows) {
            Dp[prow] = real[p] ? -acc : 0.f;
            Lp[prow] = real[p] ? -lv[p] * kLog2e : -INFINITY;
        }
    }
}

// kBulk: the dQ tile goes out through the TMA add-reduce; at D = 128 that needs 32 KB of staging, which is
// taken from the second dO slot (dO_i is only read early in tile i, by dP and dV, so one slot
// works, at the price of a later refill).  Without it dO has two slots like Q.
template <int D, bool kBulk>
struct BwdSmem {
    static constexpr int kTile = 128 * D * 2;        // K, V, Q_i, dO_i tiles
    static constexpr int kdS = 128 * 128 * 2;        // dS^T tile, [128 keys][128 queries] bf16
    static constexpr int offK = 0;
    static constexpr int offV = offK + kTile;
    static constexpr int offQ = offV + kTile;        // 2 slots
    static constexpr int kDoSlots = (kBulk && D == 128) ? 1 : 2;      // (D = 64 has the room for both)
    static constexpr int offdO = offQ + 2 * kTile;
    static constexpr int offStage = offdO + kDoSlots * kTile;   // 2 x [32 rows][D] fp32 staging (kBulk only)
    static constexpr int kStage = kBulk ? 32 * D * 4 : 0;
    // D = 128: two stages of 32 rows, filled by all four reduce warps in turn; D = 64: a stage per reduce warp (its own 32 rows)
    static constexpr int offdS = offStage + (D == 128 ? 2 : 4) * kStage;
    static constexpr int offL = offdS + kdS;         // 2 x 128 floats, travels with the Q slot
    static constexpr int offD = offL + 2 * 512;      // 2 x 128 floats, travels with the Q slot
    static constexpr int offBar = offD + 2 * 512;    // mbarriers + tmem base + abort flag
    static constexpr int kTotal = offBar + 192;
};

// Barrier slots inside the shared-memory barrier block
enum {
    B_KV = 0, B_QFULL = 1 /*2*/, B_QEMPTY = 3 /*2*/, B_DOFULL = 5 /*2*/, B_DOEMPTY = 7 /*2*/,
    B_S = 9, B_P = 10, B_DP = 11, B_DS = 12, B_DQ = 13, B_DQR = 14, B_STGFREE = 15 /*2*/, B_STGFULL = 17 /*2*/,
    B_EPI = 19 /*dK, dV tiles staged in shared memory*/, B_COUNT = 20
};

template <int D, bool kBulk, bool kGrouped>
__global__ void __launch_bounds__(kThreads, 1)
tc_bwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
              const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapdO,
              const __grid_constant__ CUtensorMap mapdQ, const __grid_constant__ CUtensorMap mapdK,
              const __grid_constant__ CUtensorMap mapdV, const float *__restrict__ Lp, const float *__restrict__ Dp,
              float *__restrict__ dQacc,
              int n, int n_pad, int causal, float scale, float scale_log2, int nkt, int hpg, int group,
              int Hkv, int skip_dq, unsigned int *status)
{
    using SM = BwdSmem<D, kBulk>;
    constexpr int kDoSlots = SM::kDoSlots;
    constexpr bool dq_bulk = kBulk;
    constexpr int kBoxes = D / 64;
    constexpr int kBoxBytes = 128 * 128;
    constexpr bool kAliasDQ = (D == 128);   // dQ tile shares the dP^T columns
    // For D = 128 the tile is produced transposed (lanes = d) so that one warp-wide red covers
    // 32 consecutive floats of one dQ row: a full 128-byte line per request instead of 32
    // half-used sectors.  (UMMA needs M = 128, so D = 64 keeps lanes = queries.)
    constexpr bool kTransposeDQ = (D == 128);
    // D = 128: dK(i) reads dS^T from the shared-memory tile (as dQ(i) does) instead of a bf16 copy in TMEM, so that
    // dQ(i), which lands on the dP^T columns, can be issued FIRST and its read-out runs under dK(i) instead of between
    // dQ(i) and dP(i+1), on the chain dS(i) -> dQ(i) -> read-out -> dP(i+1) -> dS(i+1) that paces the loop.
    constexpr bool kDKfromSmem = (D == 128);
    constexpr uint32_t colS = 0, colDP = 128, colDV = 256, colDK = 256 + D, colDQ = kAliasDQ ? 128 : 384;
    extern __shared__ __align__(1024) uint8_t sm[];
    uint8_t *sK = sm + SM::offK, *sV = sm + SM::offV, *sdS = sm + SM::offdS;
    float *sL = reinterpret_cast<float *>(sm + SM::offL);
    float *sD = reinterpret_cast<float *>(sm + SM::offD);
    uint64_t *bars = reinterpret_cast<uint64_t *>(sm + SM::offBar);
    uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bars + B_COUNT);
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(bars + B_COUNT + 1);

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    int bh, kt;                               // causal: key tile 0 has the most query tiles and goes first
    job_from_block((int)blockIdx.x, nkt, (int)gridDim.x / nkt, hpg, bh, kt);
    const int k0 = kt * 128;
    const int nqt = n_pad / 128;
    const int i_begin = causal ? kt : 0;
    // With shared K/V heads (group > 1) `bh` counts K/V heads and the CTA walks the query tiles of
    // all `group` query heads that read this K/V tile: dK and dV accumulate over the whole group in
    // TMEM, still written once by one CTA, with no atomics.
    // coordinates of the 4-D tensor maps of the caller's tensors: batch, K/V head, and the first
    // query head of the group; the flat query-head index (walkers below) addresses the internal
    // [B*H, ...] arrays (L', D, the dQ accumulator)
    const int bb = bh / Hkv, hk = bh - bb * Hkv;
    const int hq0 = hk * (kGrouped ? group : 1) - bh * (kGrouped ? group : 1);   // query head in batch = flat index + hq0
    const int niter_all = (kGrouped ? group : 1) * (nqt - i_begin);
    // (query head, query tile) of consecutive iterations, advanced without a division: each role
    // keeps a walker of its own, in step with the iterations it handles.  kGrouped = false (one K/V
    // head per query head) compiles to the plain tile counter.
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
        for (int b = 0; b < B_COUNT; ++b) {
            const uint32_t cnt = (b == B_P || b == B_DS || b == B_EPI) ? 256u
                               : (b == B_DQR || b == B_STGFULL || b == B_STGFULL + 1) ? 128u : 1u;
            mbar_init(bars + b, cnt);
        }
        *abortp = (smem_u32(sm) & 1023u) ? 1u : 0u;
        if (*abortp && status) atomicCAS(status, 0u, (unsigned)ERR_ALIGN);
        fence_mbar_init();
        prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV); prefetch_tensormap(&mapdO);
        if (dq_bulk) prefetch_tensormap(&mapdQ);
        prefetch_tensormap(&mapdK); prefetch_tensormap(&mapdV);
    }
    if (warp == kMmaWarp) { tmem_alloc(tmem_base_s, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    grid_launch_dependents();      // the dQ conversion that follows may be set up while this grid drains
    const uint32_t tbase = *tmem_base_s;
    // a misaligned shared-memory base (swizzled tiles would be misplaced) turns every role into a no-op
    const int niter = (*abortp == 0) ? niter_all : 0;

    // 512 threads start with 128 registers each (the whole register file); the last
    // warpgroup (TMA, UMMA, two idle warps) gives most of its share to the others
    // (setmaxnreg at the top of each role's branch).
    if (warp >= kLoadWarp) {
      // one instruction for the whole last warpgroup (TMA warp, UMMA warp, two idle warps)
      asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
      if (warp == kLoadWarp) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && niter > 0) {
            mbar_arrive_expect_tx(bars + B_KV, 2 * SM::kTile);
            for (int b = 0; b < kBoxes; ++b) {
                tma_load_4d(sK + b * kBoxBytes, &mapK, bars + B_KV, 64 * b, k0, hk, bb);
                tma_load_4d(sV + b * kBoxBytes, &mapV, bars + B_KV, 64 * b, k0, hk, bb);
            }
        }
        // Q tiles (with L, D) go through a two-slot ring and are fetched two tiles ahead: S(i+1) is
        // issued in the middle of tile i.  dO has one slot: it is read only by dP(i) and dV(i),
        // early in tile i, and is refilled as soon as dV(i) has completed.
        // K, V, Q and dO are the caller's tensors; L', D and the cleared dQ accumulator were written by the kernel in front of
        // this one in the stream (the forward or the preprocess kernel), which may still be running: the first tiles are
        // requested, then this warp waits for that kernel before it asks for L' and D.
        TileWalk wq = walk0, wdo = walk0;     // load_q and load_do are each called for it = 0, 1, 2, ... in order
        auto load_q = [&](int it, bool wait_first) {
            const int s = it & 1, q0 = wq.qi * 128, qh = wq.qh;
            wq.next();
            uint8_t *sQ = sm + SM::offQ + s * SM::kTile;
            mbar_arrive_expect_tx(bars + B_QFULL + s, SM::kTile + 1024);
            for (int b = 0; b < kBoxes; ++b) tma_load_4d(sQ + b * kBoxBytes, &mapQ, bars + B_QFULL + s, 64 * b, q0, qh + hq0, bb);
            if (wait_first) grid_dependency_wait();
            bulk_load_1d(sL + s * 128, Lp + (size_t)qh * n_pad + q0, 512, bars + B_QFULL + s);
            bulk_load_1d(sD + s * 128, Dp + (size_t)qh * n_pad + q0, 512, bars + B_QFULL + s);
        };
        auto load_do = [&](int it) {
            const int s = it % kDoSlots, q0 = wdo.qi * 128, qh = wdo.qh;
            wdo.next();
            uint8_t *sdO = sm + SM::offdO + s * SM::kTile;
            mbar_arrive_expect_tx(bars + B_DOFULL + s, SM::kTile);
            for (int b = 0; b < kBoxes; ++b) tma_load_4d(sdO + b * kBoxBytes, &mapdO, bars + B_DOFULL + s, 64 * b, q0, qh + hq0, bb);
        };
        if (lane == 0 && niter > 0) {
            load_do(0);
            if (kDoSlots == 2 && niter > 1) load_do(1);
            load_q(0, true);
            if (niter > 1) load_q(1, false);
        }
        grid_dependency_wait();     // (the lanes that issued nothing, and a CTA without tiles)
        for (int it = 0; it < niter; ++it) {
            if (it + kDoSlots < niter) {     // dV(it) done: its dO slot takes tile it + kDoSlots
                if (!mbar_wait(bars + B_DOEMPTY + it % kDoSlots, (it / kDoSlots) & 1, abortp, status, ERR_EMPTY)) break;
                if (lane == 0) load_do(it + kDoSlots);
            }
            if (it + 2 < niter) {     // dK(it) done: its Q slot takes tile it+2
                if (!mbar_wait(bars + B_QEMPTY + (it & 1), (it >> 1) & 1, abortp, status, ERR_EMPTY)) break;
                if (lane == 0) load_q(it + 2, false);
            }
            __syncwarp();
        }
      } else if (warp == kMmaWarp && lane == 0) {
        // the whole role runs in one thread: no warp re-convergence between waits and issues
        // ------------------------------------------------------------------- UMMA issuer
        // Issue order per query tile i:  dP(i), dV(i), S(i+1), dQ(i), dK(i)  (D = 64: dK(i), dQ(i)).
        constexpr uint32_t idesc_st = idesc_bf16_f32(128, 128, 0, 0);   // S^T, dP^T
        constexpr uint32_t idesc_acc = idesc_bf16_f32(128, D, 0, 1);    // dV, dK: A in TMEM, B MN-major
        constexpr uint32_t idesc_dq = idesc_bf16_f32(128, D, 1, 1);     // dQ: A and B MN-major
        constexpr uint32_t idesc_dqt = idesc_bf16_f32(128, 128, 1, 1);  // dQ^T (D = 128 only)
        // Descriptors are built once and kept as 32-bit halves.  Only the low half (address field)
        // changes between k-steps and slots, so an UMMA costs the issuing thread one or two
        // integer adds, a setp and the tcgen05.mma itself.  This matters: the issuing warp shares
        // its scheduler with three busy warps, and at a dozen instructions per UMMA it could not
        // keep the 64-cycle UMMAs fed.
        const uint64_t km_proto = smem_desc_sw128(0, 16, 1024), mn_proto = smem_desc_sw128(0, kBoxBytes, 1024);
        const uint32_t km_hi = (uint32_t)(km_proto >> 32), mn_hi = (uint32_t)(mn_proto >> 32);
        const uint32_t km_lo = (uint32_t)km_proto, mn_lo = (uint32_t)mn_proto;
        auto field = [](const void *ptr) { return (smem_u32(ptr) >> 4) & 0x3FFFu; };
        const uint32_t k_km = km_lo + field(sK), v_km = km_lo + field(sV);            // A of S^T, dP^T
        const uint32_t k_mn = mn_lo + field(sK), ds_mn = mn_lo + field(sdS);          // dQ operands
        const uint32_t ds_km = km_lo + field(sdS);                                    // dS^T as the K-major A of dK
        const uint32_t q_km0 = km_lo + field(sm + SM::offQ), q_mn0 = mn_lo + field(sm + SM::offQ);
        const uint32_t do_km0 = km_lo + field(sm + SM::offdO), do_mn0 = mn_lo + field(sm + SM::offdO);
        constexpr uint32_t kSlot = (uint32_t)(SM::kTile >> 4);   // address-field step between the two slots
        auto koff = [](int ks) { return (uint32_t)(((ks / 4) * kBoxBytes + (ks % 4) * 32) >> 4); };
        auto moff = [](int ks) { return (uint32_t)((ks * 2048) >> 4); };
        auto issue_S = [&](uint32_t q_km) {
            umma_ss2<false>(tbase + colS, k_km, km_hi, q_km, km_hi, idesc_st);
#pragma unroll
            for (int ks = 1; ks < D / 16; ++ks)
                umma_ss2<true>(tbase + colS, k_km + koff(ks), km_hi, q_km + koff(ks), km_hi, idesc_st);
            umma_commit(bars + B_S);
        };
        bool ok = niter > 0 && mbar_wait(bars + B_KV, 0, abortp, status, ERR_KV);
        ok = ok && mbar_wait(bars + B_QFULL + 0, 0, abortp, status, ERR_FULL);
        if (ok) {
            tc_fence_after();
            if (lane == 0) issue_S(q_km0);
        }
        for (int it = 0; ok && it < niter; ++it) {
            const int s = it & 1;
            const int sdo = it % kDoSlots;
            const uint32_t q_mn = q_mn0 + s * kSlot, do_km = do_km0 + sdo * kSlot, do_mn = do_mn0 + sdo * kSlot;
            if (!mbar_wait(bars + B_DOFULL + sdo, (it / kDoSlots) & 1, abortp, status, ERR_FULL)) break;
            if (kAliasDQ && !skip_dq && it > 0 && !mbar_wait(bars + B_DQR, (it - 1) & 1, abortp, status, ERR_DQR)) break;
            tc_fence_after();
            if (lane == 0) {
                umma_ss2<false>(tbase + colDP, v_km, km_hi, do_km, km_hi, idesc_st);
#pragma unroll
                for (int ks = 1; ks < D / 16; ++ks)
                    umma_ss2<true>(tbase + colDP, v_km + koff(ks), km_hi, do_km + koff(ks), km_hi, idesc_st);
                umma_commit(bars + B_DP);
            }
            if (!mbar_wait(bars + B_P, it & 1, abortp, status, ERR_PDS)) break;
            // (the probe for S(i+1)'s operand sits here, not between dV and S: a thread that reads shared memory between
            // two UMMAs first waits for the ones it issued to complete, and the pipe then idles until the next one
            // arrives -- 150-185 cycles per such point in a replay of this loop's issue pattern)
            if (it + 1 < niter && !mbar_wait(bars + B_QFULL + ((it + 1) & 1), ((it + 1) >> 1) & 1, abortp, status, ERR_FULL)) break;
            tc_fence_after();
            if (lane == 0) {
                // 16 queries per step; the very first UMMA of the CTA overwrites the accumulator
                if (it > 0) umma_ts2<true>(tbase + colDV, tbase + colS, do_mn, mn_hi, idesc_acc);
                else        umma_ts2<false>(tbase + colDV, tbase + colS, do_mn, mn_hi, idesc_acc);
#pragma unroll
                for (int ks = 1; ks < 8; ++ks) {
                    const uint32_t a_col = 64 * (ks / 4) + 8 * (ks % 4);
                    umma_ts2<true>(tbase + colDV, tbase + colS + a_col, do_mn + moff(ks), mn_hi, idesc_acc);
                }
                umma_commit(bars + B_DOEMPTY + sdo);
            }
            if (it + 1 < niter) issue_S(q_km0 + ((it + 1) & 1) * kSlot);
            if (!mbar_wait(bars + B_DS, it & 1, abortp, status, ERR_PDS)) break;
            if (!kAliasDQ && !skip_dq && it > 0 && !mbar_wait(bars + B_DQR, (it - 1) & 1, abortp, status, ERR_DQR)) break;
            tc_fence_after();
            if (lane == 0 && kDKfromSmem) {
                // dQ^T first (16 keys per step), then dK += dS^T Q_i with dS^T from shared memory (16 queries per step)
                if (!skip_dq) {
                    umma_ss2<false>(tbase + colDQ, k_mn, mn_hi, ds_mn, mn_hi, idesc_dqt);
#pragma unroll
                    for (int ks = 1; ks < 8; ++ks)
                        umma_ss2<true>(tbase + colDQ, k_mn + moff(ks), mn_hi, ds_mn + moff(ks), mn_hi, idesc_dqt);
                }
                umma_commit(bars + B_DQ);
                if (it > 0) umma_ss2<true>(tbase + colDK, ds_km, km_hi, q_mn, mn_hi, idesc_acc);
                else        umma_ss2<false>(tbase + colDK, ds_km, km_hi, q_mn, mn_hi, idesc_acc);
#pragma unroll
                for (int ks = 1; ks < 8; ++ks)
                    umma_ss2<true>(tbase + colDK, ds_km + koff(ks), km_hi, q_mn + moff(ks), mn_hi, idesc_acc);
                umma_commit(bars + B_QEMPTY + s);   // Q slot (and, on the last tile, everything issued) is done
            }
            if (lane == 0 && !kDKfromSmem) {
                if (it > 0) umma_ts2<true>(tbase + colDK, tbase + colDP, q_mn, mn_hi, idesc_acc);
                else        umma_ts2<false>(tbase + colDK, tbase + colDP, q_mn, mn_hi, idesc_acc);
#pragma unroll
                for (int ks = 1; ks < 8; ++ks) {
                    const uint32_t a_col = 64 * (ks / 4) + 8 * (ks % 4);
                    umma_ts2<true>(tbase + colDK, tbase + colDP + a_col, q_mn + moff(ks), mn_hi, idesc_acc);
                }
                umma_commit(bars + B_QEMPTY + s);   // Q slot is free once dK is done (dQ does not read it)
                // 16 keys per step.  D = 128: dQ^T = K^T dS^T (lanes are d, columns are queries);
                // D = 64: dQ = dS K (lanes are queries, columns are d)
                if (!skip_dq) {   // (the atomic-free mode computes dQ in its own query-parallel kernel)
                    if (kTransposeDQ) umma_ss2<false>(tbase + colDQ, k_mn, mn_hi, ds_mn, mn_hi, idesc_dqt);
                    else              umma_ss2<false>(tbase + colDQ, ds_mn, mn_hi, k_mn, mn_hi, idesc_dq);
#pragma unroll
                    for (int ks = 1; ks < 8; ++ks) {
                        if (kTransposeDQ) umma_ss2<true>(tbase + colDQ, k_mn + moff(ks), mn_hi, ds_mn + moff(ks), mn_hi, idesc_dqt);
                        else              umma_ss2<true>(tbase + colDQ, ds_mn + moff(ks), mn_hi, k_mn + moff(ks), mn_hi, idesc_dq);
                    }
                }
                umma_commit(bars + B_DQ);
            }
        }
      }
    } else if (warp >= kReduceWarp0) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 144;");
        // ------------------------------------------------- dQ reduce warps: lanes are query rows
        grid_dependency_wait();      // the accumulator these warps add into was cleared by the kernel in front
        const int lane_row = 32 * (warp % 4) + lane;
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        TileWalk wr = walk0;
        for (int it = 0; it < (skip_dq ? 0 : niter); ++it) {
            const int qtile = wr.qi, qh = wr.qh, qrow = qtile * 128 + lane_row;
            wr.next();
            if (!mbar_wait(bars + B_DQ, it & 1, abortp, status, ERR_DQ)) break;
            tc_fence_after();
            uint32_t r[D / 32][32];
            if (kTransposeDQ) {
                // lanes are d (this thread: column lane_row of every dQ row), TMEM columns are queries
                const int q0 = qtile * 128;
                float *dst = dQacc + ((size_t)qh * n + q0) * D + lane_row;
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld(lane_addr + colDQ + 32 * c, r[c]);
                tc_wait_ld();
                tc_fence_before();
                mbar_arrive(bars + B_DQR);      // TMEM columns are free again; the reds go out from registers
                if (dq_bulk) {
                    // Stage 32 query rows x 128 floats at a time in shared memory (this thread writes
                    // column lane_row of each row: conflict-free) and hand each stage to the TMA engine
                    // as one add-reduce into the fp32 accumulator; rows past n are clipped by the map.
                    // All hand-offs inside the reduce group go through bounded mbarrier waits
                    // (no named barriers), so a timed-out CTA can still drain.
                    const bool leader = (tid == kReduceWarp0 * 32);
                    bool stage_ok = true;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int g = it * 4 + c, st = c & 1;       // g: running chunk count, two stages
                        float *stage = reinterpret_cast<float *>(sm + SM::offStage + st * SM::kStage);
                        if (g >= 2) {
                            if (leader) { bulk_wait_read<1>(); mbar_arrive(bars + B_STGFREE + st); }   // TMA has read the stage
                            if (stage_ok && !mbar_wait(bars + B_STGFREE + st, ((g >> 1) - 1) & 1, abortp, status, ERR_STAGE))
                                stage_ok = false;
                        }
                        if (stage_ok) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) stage[e * D + lane_row] = __uint_as_float(r[c][e]);
                            fence_proxy_async_smem();
                        }
                        mbar_arrive(bars + B_STGFULL + st);
                        if (leader && stage_ok && mbar_wait(bars + B_STGFULL + st, (g >> 1) & 1, abortp, status, ERR_STAGE)) {
                            // (query head, tile) of this iteration: recomputed here, by the one thread that
                            // needs them, rather than kept live beside the 128 registers of the tile
                            const int nq_per = nqt - i_begin;
                            const int hh = kGrouped ? it / nq_per : 0;
                            tma_reduce_add_3d(&mapdQ, stage, 0, (i_begin + it - hh * nq_per) * 128 + 32 * c,
                                              (kGrouped ? bh * group : bh) + hh);
                            bulk_commit();
                        }
                    }
                    if (!stage_ok) break;
                } else {
                    const int valid = min(128, n - q0);
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (32 * c + e < valid) red_add_f32(dst + (size_t)(32 * c + e) * D, __uint_as_float(r[c][e]));
                }
            } else {
                float *dst = dQacc + ((size_t)qh * n + qrow) * D;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) tmem_ld(lane_addr + colDQ + 32 * c, r[c]);
                tc_wait_ld();
                tc_fence_before();
                mbar_arrive(bars + B_DQR);
                if (dq_bulk) {
                    // D = 64, bulk reduce: a thread holds the 64 floats of its query row, a warp 32 consecutive rows -- one
                    // box pair of the accumulator's tensor map (32 rows x 32 floats each, 128-byte swizzle), staged and sent
                    // by the warp alone: no hand-off between the warps.  `red.global.add.v4` from here fills half a sector
                    // per lane and instruction; the staged rows leave as whole lines.
                    uint8_t *wstage = sm + SM::offStage + (warp % 4) * SM::kStage;
                    if (it > 0) {       // the reduces of the tile before have read the boxes
                        if (lane == 0) bulk_wait_read<0>();
                        __syncwarp();
                    }
#pragma unroll
                    for (int c = 0; c < D / 32; ++c)
#pragma unroll
                        for (int jj = 0; jj < 8; ++jj) {
                            const int chunk = jj ^ (lane & 7);
                            *reinterpret_cast<uint4 *>(wstage + c * 4096 + lane * 128 + chunk * 16) =
                                make_uint4(r[c][4 * jj], r[c][4 * jj + 1], r[c][4 * jj + 2], r[c][4 * jj + 3]);
                        }
                    fence_proxy_async_smem();
                    __syncwarp();
                    const int row0 = qtile * 128 + 32 * (warp % 4);
                    if (lane == 0 && row0 < n) {        // (rows past n inside the box are clipped by the map)
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) tma_reduce_add_3d(&mapdQ, wstage + c * 4096, 32 * c, row0, qh);
                        bulk_commit();
                    }
                } else if (qrow < n) {
#pragma unroll
                    for (int c = 0; c < D / 32; ++c)
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            red_add_v4(dst + 32 * c + e, __uint_as_float(r[c][e]), __uint_as_float(r[c][e + 1]),
                                       __uint_as_float(r[c][e + 2]), __uint_as_float(r[c][e + 3]));
                }
            }
        }
        if (kTransposeDQ && dq_bulk && tid == kReduceWarp0 * 32) bulk_wait<0>();   // all reduces done before exit
        if (!kTransposeDQ && dq_bulk && lane == 0) bulk_wait<0>();                 // (D = 64: every reduce warp sent its own)
    } else {
        // ----------------------------------------------------------- elementwise warps 0-7
        asm volatile("setmaxnreg.inc.sync.aligned.u32 144;");
        const int wg = warp / 4;                          // which half of the query columns
        const int lane_row = 32 * (warp % 4) + lane;      // TMEM lane of this thread = key index in the tile
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        uint64_t p2[32];                                  // this thread's 64 probabilities of the current tile, as fp32 pairs
        const uint64_t sl2 = pack_f32x2(scale_log2, scale_log2);
        bool ok = true;

        // P-phase of tile `it`: P^T = exp2(S^T scale log2e - L log2e), kept in registers and
        // written as bf16 over the first half of this warpgroup's S^T columns.  Arithmetic is
        // on fp32 pairs (f32x2) to halve the instruction count: the UMMA-issuing warp shares
        // its scheduler with these warps.
        TileWalk wp = walk0;
        auto p_phase = [&](int it) -> bool {
            const int s = it & 1;
            const bool diag = causal && (wp.qi == kt);     // p_phase runs for it = 0, 1, 2, ... in order
            wp.next();
            if (!mbar_wait(bars + B_S, it & 1, abortp, status, ERR_SDP)) return false;
            tc_fence_after();
            const float *Ls = sL + s * 128;    // -L log2e
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int qc0 = 64 * wg + 32 * c;
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
                    if (diag) {   // query index < key index: masked
                        if (qc0 + e < lane_row) a0 = 0.f;
                        if (qc0 + e + 1 < lane_row) a1 = 0.f;
                        if (qc0 + e + 2 < lane_row) a2 = 0.f;
                        if (qc0 + e + 3 < lane_row) a3 = 0.f;
                    }
                    p2[16 * c + e / 2] = pack_f32x2(a0, a1);
                    p2[16 * c + e / 2 + 1] = pack_f32x2(a2, a3);
                    pk[e / 2] = pack_bf16(a0, a1);
                    pk[e / 2 + 1] = pack_bf16(a2, a3);
                }
                tmem_st(lane_addr + colS + 64 * wg + 16 * c, pk);
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bars + B_P);
            return true;
        };

        // (one loop, entered a step early, so that the P phase is inlined once: the roles' hot code is what the
        // schedulers keep fetching, and the kernel measurably runs faster the smaller it is)
        ok = niter > 0;
        for (int it = -1; ok && it < niter; ++it) {
          if (it >= 0) {
            const int s = it & 1;
            // dS-phase: dS^T = P^T o (dP^T - D)   (the factor `scale` is applied to dK and dQ at the end)
            if (!mbar_wait(bars + B_DP, it & 1, abortp, status, ERR_SDP)) { ok = false; break; }
            tc_fence_after();
            const float *Ds = sD + s * 128;    // -D
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int qc0 = 64 * wg + 32 * c;
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
                    unpack_f32x2(mul_f32x2(p2[16 * c + e / 2], u0), g0, g1);
                    unpack_f32x2(mul_f32x2(p2[16 * c + e / 2 + 1], u1), g2, g3);
                    gk[e / 2] = pack_bf16(g0, g1);
                    gk[e / 2 + 1] = pack_bf16(g2, g3);
                }
                if (!kDKfromSmem) tmem_st(lane_addr + colDP + 64 * wg + 16 * c, gk);
                // dS^T row (this key) into the MN-major smem tile: box wg, 128-byte row, swizzled 16-byte chunks
                uint8_t *rowp = sdS + wg * kBoxBytes + lane_row * 128;
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int chunk = (4 * c + jj) ^ (lane_row & 7);
                    *reinterpret_cast<uint4 *>(rowp + chunk * 16) =
                        make_uint4(gk[4 * jj], gk[4 * jj + 1], gk[4 * jj + 2], gk[4 * jj + 3]);
                }
            }
            if (!kDKfromSmem) tc_wait_st();
            tc_fence_before();
            fence_proxy_async_smem();
            mbar_arrive(bars + B_DS);
          }
            if (it + 1 < niter) ok = p_phase(it + 1);
        }
        if (ok && mbar_wait(bars + B_DQ, (niter - 1) & 1, abortp, status, ERR_DQ) &&
            (!kDKfromSmem || mbar_wait(bars + B_QEMPTY + ((niter - 1) & 1), ((niter - 1) >> 1) & 1, abortp, status, ERR_DQ))) {
            // All UMMAs have completed.  dV and scale*dK go out as bf16 through shared memory (the K and V
            // tiles are no longer read) and TMA stores: a thread owns a row, so direct stores would be 16
            // bytes at a 2D-byte stride, one 128-byte line per lane and instruction -- 4096 line requests
            // per CTA, which kept the load/store unit busy for ~3 us; staged, the tile leaves as
            // full lines, and rows past n are clipped by the tensor map.
            tc_fence_after();
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const uint32_t col = (which == 0 ? colDV : colDK) + (D / 2) * wg;
                const float mul = which == 0 ? 1.f : scale;
                uint8_t *stage = which == 0 ? sV : sK;
#pragma unroll
                for (int c = 0; c < D / 2; c += 32) {
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
                        const int cabs = (D / 2) * wg + c + e;          // first of 8 columns
                        const int chunk = ((cabs & 63) >> 3) ^ (lane_row & 7);   // 128-byte swizzle, as the maps expect
                        *reinterpret_cast<uint4 *>(stage + (cabs >> 6) * kBoxBytes + lane_row * 128 + chunk * 16) = v;
                    }
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(bars + B_EPI);
            if (tid == 0 && mbar_wait(bars + B_EPI, 0, abortp, status, ERR_DQ)) {
                for (int b = 0; b < kBoxes; ++b) {
                    tma_store_4d(&mapdV, sV + b * kBoxBytes, 64 * b, k0, hk, bb);
                    tma_store_4d(&mapdK, sK + b * kBoxBytes, 64 * b, k0, hk, bb);
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
        // stays for a fixed 400,000 cycles (hundreds of times a copy's latency) before the CTA can leave.  (The other
        // kernels wait on the barriers they armed; here that bookkeeping cost 1.5-3 % under the role's register cap.)
        const long long t0 = clock64();
        while (clock64() - t0 < 400000LL) { }
    }
}

template <int D, bool kBulk, bool kGrouped>
cudaError_t launch_bwd_g(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                       const float *Lp, const float *Dp, void *dK, void *dV, float *dQacc, cudaStream_t st)
{
    CUtensorMap mq, mk, mv, mdo, mdq, mdk, mdv;
    const uint64_t heads = (uint64_t)p.BH();
    const auto bf = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    // p.d <= D columns exist in memory: loads fill the rest of a box with zeros, stores drop it
    if (!make_tensor_map_4d_strided(&mq, Q, bf, 2, p.B, p.H, p.n, p.d, p.sq.row, p.sq.head, p.sq.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mk, K, bf, 2, p.B, p.kv_heads(), p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mv, V, bf, 2, p.B, p.kv_heads(), p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mdo, dO, bf, 2, p.B, p.H, p.n, p.d, p.so.row, p.so.head, p.so.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mdk, dK, bf, 2, p.B, p.kv_heads(), p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mdv, dV, bf, 2, p.B, p.kv_heads(), p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64))
        return cudaErrorInvalidValue;
    // fp32 accumulator as [heads, n, D] with boxes of 32 rows x D floats (no swizzle); also encoded when unused
    // (D = 64: boxes of 32 rows x 32 floats with the 128-byte swizzle, two per warp and tile)
    if (!make_tensor_map_3d(&mdq, dQacc ? (const void *)dQacc : Q, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, heads, p.n, D, 32, D == 64 ? 32 : D))
        return cudaErrorInvalidValue;
    constexpr int kSmem = BwdSmem<D, kBulk>::kTotal;
    cudaError_t e = cudaFuncSetAttribute(tc_bwd_kernel<D, kBulk, kGrouped>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const int nkt = (p.n + 127) / 128;
    LaunchScope scope(MOA_KERNEL_BWD_KV, st);
    // one CTA per (K/V head, key tile); the block order groups K/V heads
    Problem pkv = p;
    pkv.H = p.kv_heads();
    pkv.Hkv = 0;
    return launch_dependent(tc_bwd_kernel<D, kBulk, kGrouped>, dim3((unsigned)(nkt * p.BHkv())), dim3(kThreads), (size_t)kSmem, st,
                            mq, mk, mv, mdo, mdq, mdk, mdv, Lp, Dp, dQacc, p.n, nkt * 128, p.causal, p.scale, p.scale * kLog2e, nkt,
                            heads_per_group(pkv, nkt), p.group(), p.kv_heads(), dQacc == nullptr ? 1 : 0, device_status_ptr());
}

template <int D, bool kBulk>
cudaError_t launch_bwd(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                       const float *Lp, const float *Dp, void *dK, void *dV, float *dQacc, cudaStream_t st)
{
    return p.group() > 1 ? launch_bwd_g<D, kBulk, true>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st)
                         : launch_bwd_g<D, kBulk, false>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
}

}  // namespace

cudaError_t tc_bwd_preprocess(const Problem &p, const void *dO, const void *O, const float *L, float *Lp, float *Dp,
                              cudaStream_t st)
{
    const int n_pad = (p.n + 127) / 128 * 128;
    const size_t rows = (size_t)p.BH() * n_pad;
    const int wpb = 8;
    const int D = kernel_d(p.d);
    const size_t rows_per_block = (size_t)wpb * (32 / (D / 8)) * 4;   // warps x rows per pass x passes
    const unsigned grid = (unsigned)((rows + rows_per_block - 1) / rows_per_block);
    LaunchScope scope(MOA_KERNEL_PREPROCESS, st);
    if (D == 256)
        bwd_preprocess_kernel<256><<<grid, wpb * 32, 0, st>>>((const __nv_bfloat16 *)dO, (const __nv_bfloat16 *)O, L,
                                                              Lp, Dp, p.n, n_pad, rows, p.H, p.so, p.d);
    else if (D == 64)
        bwd_preprocess_kernel<64><<<grid, wpb * 32, 0, st>>>((const __nv_bfloat16 *)dO, (const __nv_bfloat16 *)O, L,
                                                             Lp, Dp, p.n, n_pad, rows, p.H, p.so, p.d);
    else
        bwd_preprocess_kernel<128><<<grid, wpb * 32, 0, st>>>((const __nv_bfloat16 *)dO, (const __nv_bfloat16 *)O, L,
                                                              Lp, Dp, p.n, n_pad, rows, p.H, p.so, p.d);
    return cudaGetLastError();
}

cudaError_t tc_bwd_kv(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                      const float *Lp, const float *Dp, void *dK, void *dV, float *dQacc, int dq_bulk, cudaStream_t st)
{
    if (p.d < 8 || p.d > 256 || p.d % 8) return cudaErrorInvalidValue;
    const int D = kernel_d(p.d);     // dQacc rows are D floats wide
    if (D == 256) return dq_bulk ? cudaErrorInvalidValue : tc_bwd_kv_wide(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
    if (D == 128 && bwd_pair_enabled()) return tc_bwd_kv_pair(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, dq_bulk, st);
    if (D == 64 && !dq_bulk) return launch_bwd<64, false>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
    if (D == 64 && dq_bulk) return launch_bwd<64, true>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
    if (D == 128 && !dq_bulk) return launch_bwd<128, false>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
    if (D == 128 && dq_bulk) return launch_bwd<128, true>(p, Q, K, V, dO, Lp, Dp, dK, dV, dQacc, st);
    return cudaErrorInvalidValue;
}

}  // namespace moa
