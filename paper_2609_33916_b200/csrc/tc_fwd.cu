// Forward attention on the sm_100a tensor cores (tcgen05 + TMEM + TMA), bf16 in,
// fp32 accumulate.
//
// One CTA (one per SM) owns 128 query rows of one (batch, head) and walks the key/value
// tiles of 128 keys.  Roles (384 threads; registers re-split with setmaxnreg: 208 for the softmax
// warpgroups, 88 for the rest):
//   warps 0-7  softmax: thread = query row = TMEM lane.  Warpgroup h = warp / 4 takes the key tiles
//              j = h, h + 2, ... whole -- 128 fp32 scores from TMEM into registers, max (3-input,
//              independent chains), exp2 + row sum on packed fp32 pairs, bf16 P into the stream's own
//              64 TMEM columns -- with its own running max, row sum and O accumulator: two independent
//              online-softmax streams, merged only in the epilogue; O_h in TMEM is rescaled only when
//              the max has grown by more than 8 (log2 domain).
//   warp 8     TMA producer of Q (once) and of the K ring; warp 11 of the V ring (a thread each: the K
//              ring follows the score products, the V ring the P V products, and a single producer made
//              the next K tile wait for a V slot, i.e. for a P V product).
//   warp 9     UMMA issuer (one thread) for S = Q K^T (SS, both operands K-major) into the ONE score
//              buffer: S(j+1) is issued as soon as the warpgroup of tile j holds that tile's scores in
//              registers, and runs under tile j's exponentials.
//   warp 10    UMMA issuer (one thread) for O_h += P V (TS: P from TMEM, V MN-major in smem).  It lets
//              S(j+2) through the pipe before it issues P V(j): the warpgroup that waits for those scores
//              has nothing else to do, and UMMAs of two threads issued together interleave, so that both
//              products take twice as long.
// The two warpgroups take turns on the score buffer, so one is in its exp2 loop while the other waits,
// loads and takes its maxima; with both working on halves of the same tile (the earlier form of this
// kernel) the two exp2 loops ran together, the MUFU unit was saturated during them and idle otherwise.
// UMMAs of different threads are unordered; every hazard between them goes through an mbarrier.
// TMEM (512 columns): scores [0,128), P of stream 0 / 1 [128,192) / [192,256), O_0 [256,256+D),
// O_1 [256+D,256+2D).  S, P and the O accumulators never leave the SM: nothing of size n x n reaches HBM.
//
// What bounds it (config 4, d = 128): per 128 x 128 tile the UMMAs need 1024 cycles and the one exp2 per
// score 1024 cycles of the MUFU unit; a warpgroup is busy about 2650 cycles per tile of its own (load 220,
// maxima 620, exp2 loop 1750 when the other warpgroup's loop overlaps it, hand-off 65), i.e. 1330 per tile
// with two of them, and the tile takes about 1550.
// The O tile leaves through the Q tile's shared memory and a TMA store.
//
// Head dimensions 136..256 (KC = 2): the scores need the whole head dimension, the output does not.  S = Q K^T is
// accumulated over KC chunks of 128 columns -- Q holds all of them, the K ring carries one chunk per slot, so a key
// tile passes through it KC times -- and the grid has KC CTAs per (head, query tile), each with the V columns and the
// O columns of one 128-column half (the scores and the softmax are computed KC times; O(n d) memory as before).
// The backward's per-row inputs are then not prepared here (a CTA holds half of an O row).
#include "common.cuh"
#include "ptx.cuh"
#include "tensormap.cuh"

namespace moa {
namespace {

using namespace ptx;

constexpr int BM = 128;            // query rows per CTA
constexpr int BN = 128;            // keys per tile
constexpr int kThreads = 384;      // warps 0-7 softmax, 8 TMA, 9 UMMA issuer for S, 10 UMMA issuer for PV, 11 idle
constexpr int kTmemCols = 512;     // scores [0,128); bf16 P of the two streams [128,192), [192,256); two O accumulators from 256
constexpr uint32_t kColS = 0, kColP = 128, kColO = 256;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;

enum : uint32_t { ERR_Q = 0x101, ERR_K = 0x102, ERR_V = 0x103, ERR_S = 0x104, ERR_P = 0x105, ERR_O = 0x106 };

enum { F_Q = 0, F_KFULL = 1 /*2*/, F_KEMPTY = 3 /*2*/, F_VFULL = 5 /*2*/, F_VEMPTY = 7 /*2*/, F_S_UNUSED = 9 /*2*/,
       F_P = 11 /*2: per stream*/, F_SFREE = 13 /*2: per stream, the tile's scores are in registers*/, F_O = 15 /*unused*/,
       F_X = 16 /*epilogue exchange*/, F_OB = 17 /*2: per stream, P V of the stream's tile has completed*/,
       F_E = 19 /*O tile staged in shared memory*/, F_DONE = 20 /*last P V of the job has completed*/, 
       F_S = 21 /*[stream][tile count of the stream & 1]: 4.  Two barriers per stream, taken in turn: the P V issuer, which
                  lets S(j+2) pass before it issues P V(j), may be stalled on the V ring while the scores run two tiles of
                  the stream ahead of it, and a parity wait must never fall two phases of one barrier behind*/,
       F_COUNT = 25 };

// Split use of the kernel (decode: few query rows, a long cache): the key tiles are divided among
// `splits` CTAs per (head, query tile); each writes the attention over its tiles alone (normalised O
// and its logsumexp, batch coordinate split * B + b), to be merged by the caller.  n_q: valid query
// rows of a head (the main path: n_q = n, splits = 1, tiles_per_split = all tiles).
struct FwdSplit {
    int n_q, splits, tiles_per_split;
};

// Fused call only (dO == nullptr otherwise): the backward's per-row inputs, written by the forward
// epilogue: Lp = -(logsumexp in the log2 domain), Dp = -rowsum(dO o O), [B*H, n_pad] each.
struct FwdPrep {
    const __nv_bfloat16 *dO;
    float *Lp, *Dp;
    int n_pad;
    Strides so;          // where the rows of dO live
    int d;               // columns of a dO row in memory (<= D)
};

template <int D, int KC>
__global__ void __launch_bounds__(kThreads, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
              const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO,
              float *__restrict__ L,
              int n, int causal, float scale_log2, int nqt, int hpg, int group, int H, FwdSplit sp,
              float *__restrict__ zero_acc, FwdPrep prep, unsigned int *status)
{
    constexpr int kTileBytes = 128 * D * 2;
    constexpr int kBoxes = D / 64;         // 64-column (128-byte) swizzled boxes per tile
    constexpr int kBoxBytes = 128 * 128;   // 128 rows x 128 bytes
    extern __shared__ __align__(1024) uint8_t sm[];
    uint8_t *sQ = sm /*KC chunks*/, *sK = sm + KC * kTileBytes /*2 slots of one chunk*/, *sV = sm + (KC + 2) * kTileBytes /*2 slots*/;
    uint64_t *bars = reinterpret_cast<uint64_t *>(sm + (KC + 4) * kTileBytes);
    uint32_t *tmem_base_p = reinterpret_cast<uint32_t *>(bars + F_COUNT);
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(bars + F_COUNT + 1);

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    int bh, t;
    // KC > 1: KC consecutive CTAs share a job, CTA `pass` computes output columns [D pass, D pass + D)
    const int pass = KC > 1 ? (int)blockIdx.x % KC : 0;
    const int blk = KC > 1 ? (int)blockIdx.x / KC : (int)blockIdx.x;
    const int split = sp.splits > 1 ? blk % sp.splits : 0;
    const int heads_all = (int)gridDim.x / KC / sp.splits / nqt;
    job_from_block(sp.splits > 1 ? blk / sp.splits : blk, nqt, heads_all, hpg, bh, t);
    const int bb = bh / H, hq = bh - bb * H;    // batch and query head: coordinates of the 4-D tensor maps
    const int hk = hq / group;                  // the K/V head this query head reads (group > 1: shared heads)
    const int qt = causal ? nqt - 1 - t : t;   // causal: longest rows first
    const int q0 = qt * BM;
    const int nkt_all = (n + BN - 1) / BN;
    const int kt0 = split * sp.tiles_per_split;                       // first key tile of this CTA
    const int nkt_want = causal ? min(qt + 1, nkt_all) : min(sp.tiles_per_split, nkt_all - kt0);

    // The two producer threads initialise the barriers of their own loads and send the job's first loads off at once:
    // Q, the first two K chunks and the first two V tiles are on their way while the rest of the set-up (the other
    // barriers, the TMEM allocation, the CTA-wide barrier) still runs, instead of starting behind it.
    const bool aligned = (smem_u32(sm) & 1023u) == 0;      // (swizzled tiles need the 1024-byte alignment)
    const int early_k = aligned ? min(nkt_want * KC, 2) : 0, early_v = aligned ? min(nkt_want, 2) : 0;
    if (warp == 8 && lane == 0) {
        mbar_init(bars + F_Q, 1u);
        mbar_init(bars + F_KFULL, 1u);
        mbar_init(bars + F_KFULL + 1, 1u);
        fence_mbar_init();
        if (early_k > 0) {
            mbar_arrive_expect_tx(bars + F_Q, KC * kTileBytes);
            for (int b = 0; b < KC * kBoxes; ++b) tma_load_4d(sQ + b * kBoxBytes, &mapQ, bars + F_Q, 64 * b, q0, hq, bb);
            for (int g = 0; g < early_k; ++g) {       // chunk g: columns [D c, D c + D) of key tile j, g = j KC + c
                const int j = g / KC, c = g % KC;
                mbar_arrive_expect_tx(bars + F_KFULL + g, kTileBytes);
                for (int b = 0; b < kBoxes; ++b)
                    tma_load_4d(sK + g * kTileBytes + b * kBoxBytes, &mapK, bars + F_KFULL + g, D * c + 64 * b, (kt0 + j) * BN, hk, bb);
            }
        }
    }
    if (warp == 11 && lane == 0) {
        mbar_init(bars + F_VFULL, 1u);
        mbar_init(bars + F_VFULL + 1, 1u);
        fence_mbar_init();
        for (int j = 0; j < early_v; ++j) {
            mbar_arrive_expect_tx(bars + F_VFULL + j, kTileBytes);
            for (int b = 0; b < kBoxes; ++b)
                tma_load_4d(sV + j * kTileBytes + b * kBoxBytes, &mapV, bars + F_VFULL + j, D * pass + 64 * b, (kt0 + j) * BN, hk, bb);
        }
    }
    if (tid == 0) {
        for (int b = 0; b < F_COUNT; ++b) {
            if (b == F_Q || b == F_KFULL || b == F_KFULL + 1 || b == F_VFULL || b == F_VFULL + 1) continue;   // (the producers' own)
            mbar_init(bars + b, ((b >= F_P && b < F_P + 2) || (b >= F_SFREE && b < F_SFREE + 2)) ? 128u : ((b == F_X || b == F_E) ? 256u : 1u));
        }
        *abortp = aligned ? 0u : 1u;
        if (!aligned && status) atomicCAS(status, 0u, 0x108u);
        fence_mbar_init();
        prefetch_tensormap(&mapO);
    }
    if (warp == 9) { tmem_alloc(tmem_base_p, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_base_p;
    const int nkt = (*abortp == 0) ? nkt_want : 0;   // misaligned shared memory: every role is a no-op

    // 384 threads start with 168 registers each; the last warpgroup (TMA, the two issuers, an idle warp) gives most of its
    // share to the softmax warpgroups, whose threads hold the 128 scores of a row.  The two counts must add up to what the
    // CTA was launched with (128 x 88 + 256 x 208 = 384 x 168): an increase that asks for more than the decrease frees
    // waits for registers forever.
    if (warp >= 8) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
      if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        int nk = early_k;       // K chunks requested so far (slot = count & 1): Q and the first two went out before the set-up
        // chunk g of the K stream: 128 columns [D c, D c + D) of key tile j, g = j KC + c, ring slot g & 1
        auto load_k = [&](int g) {
            const int s = g & 1, j = g / KC, c = g % KC;
            mbar_arrive_expect_tx(bars + F_KFULL + s, kTileBytes);
            ++nk;
            for (int b = 0; b < kBoxes; ++b)
                tma_load_4d(sK + s * kTileBytes + b * kBoxBytes, &mapK, bars + F_KFULL + s, D * c + 64 * b, (kt0 + j) * BN, hk, bb);
        };
        if (zero_acc != nullptr) {
            // Fused forward+backward (KC = 1): this CTA's 128 rows of the fp32 dQ accumulator ([B*H, n, D]) are
            // cleared here, by the producer warp while its first loads are in flight (the next slot
            // frees two tiles from now), so that the step needs no separate clearing pass.
            const int rows = min(BM, n - q0);
            float4 *dst = reinterpret_cast<float4 *>(zero_acc + ((size_t)bh * n + q0) * D);
            for (int i = lane; i < rows * (D / 4); i += 32) dst[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        bool live = true;
        for (int j = early_k / KC; live && j < nkt; ++j) {
            for (int c = (j == early_k / KC ? early_k % KC : 0); c < KC; ++c) {
                const int g = j * KC + c;
                if (g >= 2 && !mbar_wait(bars + F_KEMPTY + (g & 1), ((g >> 1) - 1) & 1, abortp, status, ERR_K)) { live = false; break; }
                if (lane == 0) load_k(g);
            }
            if (!live) break;
            __syncwarp();
        }
        if (lane == 0 && *abortp) {
            // a wait expired somewhere in the CTA: copies still on their way land before it leaves (bounded)
            mbar_drain_one(bars + F_Q, nkt > 0 ? 1 : 0);
            for (int s = 0; s < 2; ++s) mbar_drain_one(bars + F_KFULL + s, nk > s ? (nk - s + 1) / 2 : 0);
        }
      } else if (warp == 11) {
        // ------------------------------------------------------------------ TMA producer of the V stream
        // (a thread of its own: the V ring follows the P V products, the K ring the score products, and neither waits
        // for the other's slots)
        int nv = early_v;       // (the first two tiles went out before the set-up)
        for (int j = early_v; j < nkt; ++j) {
            if (j >= 2 && !mbar_wait(bars + F_VEMPTY + (j & 1), ((j >> 1) - 1) & 1, abortp, status, ERR_V)) break;
            if (lane == 0) {
                const int s = j & 1;
                mbar_arrive_expect_tx(bars + F_VFULL + s, kTileBytes);
                ++nv;
                for (int b = 0; b < kBoxes; ++b)
                    tma_load_4d(sV + s * kTileBytes + b * kBoxBytes, &mapV, bars + F_VFULL + s, D * pass + 64 * b, (kt0 + j) * BN, hk, bb);
            }
            __syncwarp();
        }
        if (lane == 0 && *abortp)
            for (int s = 0; s < 2; ++s) mbar_drain_one(bars + F_VFULL + s, nv > s ? (nv - s + 1) / 2 : 0);
      } else if (warp == 9 && lane == 0) {
        // ------------------------------------------- UMMA issuer for the score GEMMs (one thread)
        // Two issuing threads (this one for S = Q K^T, warp 10 for O += P V): a successful barrier
        // probe or a commit costs an issuing thread ~100 cycles during which it feeds nothing, and
        // the tensor pipe only queues a few UMMAs, so with a single issuer the pipe idled for a
        // third of every tile.  UMMAs of different threads are not ordered, so every hazard between
        // the two streams goes through an mbarrier: S(j) may overwrite score buffer j&1 only after
        // PV(j-2), which read P(j-2) there, has completed (F_OB).
        constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);
        const uint64_t km_proto = smem_desc_sw128(0, 16, 1024);
        const uint32_t km_hi = (uint32_t)(km_proto >> 32);
        auto field = [](const void *ptr) { return (smem_u32(ptr) >> 4) & 0x3FFFu; };
        const uint32_t q_lo = (uint32_t)km_proto + field(sQ), k_lo0 = (uint32_t)km_proto + field(sK);
        constexpr uint32_t kSlot = (uint32_t)(kTileBytes >> 4);
        bool ok = nkt > 0 && mbar_wait(bars + F_Q, 0, abortp, status, ERR_Q);
        for (int j = 0; ok && j < nkt; ++j) {
            const uint32_t dcol = tbase + kColS;
#pragma unroll
            for (int c = 0; c < KC; ++c) {          // the contraction over the head dimension, 128 columns per K chunk
                const int g = j * KC + c, sl = g & 1;
                const uint32_t k_lo = k_lo0 + sl * kSlot, q_c = q_lo + c * kSlot;
                if (!mbar_wait(bars + F_KFULL + sl, (g >> 1) & 1, abortp, status, ERR_K)) { ok = false; break; }
                // the one score buffer is free once the warpgroup of tile j-1 holds that tile's scores in registers
                if (c == 0 && j >= 1 && !mbar_wait(bars + F_SFREE + ((j - 1) & 1), ((j - 1) >> 1) & 1, abortp, status, ERR_O)) { ok = false; break; }
                tc_fence_after();
                if (c == 0) umma_ss2<false>(dcol, q_c, km_hi, k_lo, km_hi, idesc_s);
                else        umma_ss2<true>(dcol, q_c, km_hi, k_lo, km_hi, idesc_s);
#pragma unroll
                for (int ks = 1; ks < D / 16; ++ks) {
                    const uint32_t off = (uint32_t)(((ks / 4) * kBoxBytes + (ks % 4) * 32) >> 4);
                    umma_ss2<true>(dcol, q_c + off, km_hi, k_lo + off, km_hi, idesc_s);
                }
                umma_commit(bars + F_KEMPTY + sl);
            }
            if (!ok) break;
            umma_commit(bars + F_S + 2 * (j & 1) + ((j >> 1) & 1));
        }
      } else if (warp == 10 && lane == 0) {
        // ------------------------------------------------ UMMA issuer for O += P V (one thread)
        constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, 0, 1);
        const uint64_t mn_proto = smem_desc_sw128(0, kBoxBytes, 1024);
        const uint32_t mn_hi = (uint32_t)(mn_proto >> 32);
        const uint32_t v_lo0 = (uint32_t)mn_proto + ((smem_u32(sV) >> 4) & 0x3FFFu);
        constexpr uint32_t kSlot = (uint32_t)(kTileBytes >> 4);
        for (int j = 0; j < nkt; ++j) {
            const int b = j & 1;        // V ring slot and stream of tile j
            const uint32_t v_lo = v_lo0 + b * kSlot, acol = tbase + kColP + 64 * b, ocol = tbase + kColO + b * D;
            if (!mbar_wait(bars + F_VFULL + b, (j >> 1) & 1, abortp, status, ERR_V)) break;
            if (!mbar_wait(bars + F_P + b, (j >> 1) & 1, abortp, status, ERR_P)) break;
            // The scores come first: this product waits until S(j+2), which is issued the moment tile j+1's scores are in
            // registers, is through the pipe (two issuing threads' UMMAs interleave and both products take twice as long).
            if (j + 2 < nkt && !mbar_wait(bars + F_S + 2 * (j & 1) + (((j + 2) >> 1) & 1), ((j + 2) >> 2) & 1, abortp, status, ERR_S)) break;
            tc_fence_after();
            // O_b (+)= P(j) V(j): 128 keys = eight k-steps; P (bf16) is 64 TMEM columns, V rows 16 ks .. 16 ks + 15
            if (j > 1) umma_ts2<true>(ocol, acol, v_lo, mn_hi, idesc_pv);
            else       umma_ts2<false>(ocol, acol, v_lo, mn_hi, idesc_pv);      // the stream's first tile
#pragma unroll
            for (int ks = 1; ks < 8; ++ks)
                umma_ts2<true>(ocol, acol + ks * 8, v_lo + (uint32_t)((ks * 2048) >> 4), mn_hi, idesc_pv);
            umma_commit(bars + F_OB + b);
            umma_commit(bars + F_VEMPTY + b);
            if (j == nkt - 1) umma_commit(bars + F_DONE);
        }
      }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        // ---------------------------------------------------------------- softmax warps
        // Thread = query row (TMEM lane).  Warpgroup h = warp / 4 takes the key tiles j = h, h + 2, ... whole (128 scores
        // per thread), with its own running max, row sum, P buffer and O accumulator: two independent online-softmax
        // streams, merged only in the epilogue.  The two warpgroups take turns on the one score buffer -- S(j+1) is issued
        // as soon as the warpgroup of tile j holds its scores in registers -- so one of them is in its exp2 loop while the
        // other waits, loads and takes its maxima: the MUFU unit, which two warps per scheduler saturate when they run
        // their exp2 loops together, is busy through both.
        const int h = warp / 4;
        const int lane_row = 32 * (warp % 4) + lane;
        const int row = q0 + lane_row;
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        const uint32_t ocol = kColO + h * D, pcol = kColP + 64 * h;
        float m_used = -1e30f, l = 0.f;      // (a stream without tiles contributes nothing to the merge)
        bool ok = nkt > 0;
        if (prep.dO != nullptr && row < n) {
            // fused call: the epilogue reads this thread's 128 bytes (D = 128) of its dO row; ask L2 for
            // them now so that the read at the end of the job does not wait on HBM
            const size_t doff = prep.so.at(bb, hq, row);
            if ((D / 2) * h < prep.d) asm volatile("prefetch.global.L2 [%0];" ::"l"(prep.dO + doff + (D / 2) * h));
        }
        for (int j = h; ok && j < nkt; j += 2) {
            const int t = j >> 1;                                      // this stream's tile count
            if (!mbar_wait(bars + F_S + 2 * h + (t & 1), (t >> 1) & 1, abortp, status, ERR_S)) { ok = false; break; }
            tc_fence_after();
            const int k0 = (kt0 + j) * BN;
            const bool need_mask = (k0 + BN > n) || (causal && k0 + BN - 1 > q0);
            uint32_t r[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld(lane_addr + kColS + 32 * c, r[c]);
            tc_wait_ld();
            tc_fence_before();
            mbar_arrive(bars + F_SFREE + h);      // the score columns are free: S(j+1) runs under this tile's exponentials
            if (need_mask) {
                // columns of this tile the row may see: keys below n and, causal, not past the row itself
                const int lim = min(n, causal ? row + 1 : n) - k0;
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (32 * c + i >= lim) r[c][i] = 0xff800000u;   // -inf
            }
            // max of the raw scores (scale_log2 > 0, so scaling commutes with max): 3-input max, sixteen
            // independent chains so that the dependent-issue latency does not add up
            float mx16[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                const int c = q >> 2, i0 = 8 * (q & 3);
                float a = fmax3(__uint_as_float(r[c][i0]), __uint_as_float(r[c][i0 + 1]), __uint_as_float(r[c][i0 + 2]));
                a = fmax3(a, __uint_as_float(r[c][i0 + 3]), __uint_as_float(r[c][i0 + 4]));
                a = fmax3(a, __uint_as_float(r[c][i0 + 5]), __uint_as_float(r[c][i0 + 6]));
                mx16[q] = fmaxf(a, __uint_as_float(r[c][i0 + 7]));
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) mx16[q] = fmaxf(mx16[q], mx16[q + 8]);
            const float mx = fmax3(fmax3(mx16[0], mx16[1], mx16[2]), fmax3(mx16[3], mx16[4], mx16[5]), fmaxf(mx16[6], mx16[7])) * scale_log2;
            if (t == 0) {
                m_used = (mx == -INFINITY) ? -1e30f : mx;     // a stream with no visible key yet: any finite reference
            } else {
                const bool grow = mx > m_used + kRescaleThreshold;
                if (__any_sync(0xffffffffu, grow)) {
                    // O_h must be stable for a rescale: P V(j-2) has completed
                    if (!mbar_wait(bars + F_OB + h, (t - 1) & 1, abortp, status, ERR_O)) { ok = false; break; }
                    tc_fence_after();
                    const float alpha = grow ? ex2(m_used - mx) : 1.f;
                    if (grow) m_used = mx;
                    l *= alpha;
#pragma unroll 1
                    for (int c = 0; c < D; c += 16) {   // rare path
                        uint32_t o[16];
                        tmem_ld(lane_addr + ocol + c, o);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st(lane_addr + ocol + c, o);
                    }
                }
            }
            // P = 2^(s scale_log2 - m_used), row sum, bf16 P into the stream's own 64 TMEM columns.
            // Arithmetic runs on fp32 pairs (f32x2) to halve the instruction count.
            const uint64_t sl2 = pack_f32x2(scale_log2, scale_log2);
            const uint64_t negm2 = pack_f32x2(-m_used, -m_used);
            uint64_t ls2[2] = {0ull, 0ull};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const uint64_t tt = fma_f32x2(pack_f32x2(__uint_as_float(r[c][i]), __uint_as_float(r[c][i + 1])), sl2, negm2);
                    float p0, p1;
                    unpack_f32x2(tt, p0, p1);
                    p0 = ex2(p0);
                    p1 = ex2(p1);
                    ls2[(i >> 1) & 1] = add_f32x2(ls2[(i >> 1) & 1], pack_f32x2(p0, p1));
                    pk[i / 2] = pack_bf16(p0, p1);
                }
                // P(j) goes where P(j-2) was: P V(j-2), which gave way to S(j) in the pipe, has read it by now (the first
                // 32 exponentials of the tile ran under the rest of that product)
                if (c == 0 && t > 0 && !mbar_wait(bars + F_OB + h, (t - 1) & 1, abortp, status, ERR_O)) { ok = false; break; }
                tmem_st(lane_addr + pcol + 16 * c, pk);
            }
            {
                float s0, s1, s2, s3;
                unpack_f32x2(ls2[0], s0, s1);
                unpack_f32x2(ls2[1], s2, s3);
                l += (s0 + s1) + (s2 + s3);
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bars + F_P + h);
        }
        // ---- epilogue: merge the two streams.  Each thread publishes (m, l) of its stream, then
        // writes D/2 output columns of its row from both accumulators.
        float2 *xch = reinterpret_cast<float2 *>(bars + F_COUNT + 2);   // [2][128] (m, l)
        float *xd = reinterpret_cast<float *>(xch + 256);               // [2][128] partial rowsum(dO o O)
        // fused call: this thread's D/2 elements of its dO row, requested before the waits below
        uint4 dov[D / 16];
        const bool want_d = prep.dO != nullptr && row < n;
        if (want_d) {
            const uint4 *src = reinterpret_cast<const uint4 *>(prep.dO + prep.so.at(bb, hq, row) + (D / 2) * h);
#pragma unroll
            for (int k = 0; k < D / 16; ++k)      // columns past the head dimension count as zeros
                dov[k] = (D / 2) * h + 8 * k < prep.d ? __ldg(src + k) : make_uint4(0u, 0u, 0u, 0u);
        }
        float dpart = 0.f;
        xch[h * 128 + lane_row] = make_float2(m_used, l);
        mbar_arrive(bars + F_X);
        if (ok && mbar_wait(bars + F_X, 0, abortp, status, ERR_P) &&
            mbar_wait(bars + F_DONE, 0, abortp, status, ERR_O)) {
            // (F_DONE, not the per-tile F_O with the last tile's parity: the softmax threads can finish the last
            // tile while the P V products of the last TWO tiles are still pending -- the S and P V issuers are
            // different threads -- and a wait on F_O's parity would then be satisfied by the tile before those,
            // which has the same parity.  Seen in decode through this kernel, where tiles arrive at HBM pace:
            // about one CTA in a hundred wrote an O that missed its last tiles.)
            tc_fence_after();
            const float2 other = xch[(h ^ 1) * 128 + lane_row];
            const float m_all = fmaxf(m_used, other.x);
            const float a_me = ex2(m_used - m_all), a_ot = ex2(other.x - m_all);
            const float l_all = l * a_me + other.y * a_ot;
            const float inv = 1.f / l_all;
            const float w0 = (h == 0 ? a_me : a_ot) * inv, w1 = (h == 0 ? a_ot : a_me) * inv;   // weights of O_0, O_1
            const bool has1 = nkt > 1;      // (one key tile: the second stream's accumulator was never written)
            // O leaves as bf16 through shared memory (the Q tile is no longer read) and a TMA store: a
            // thread owns a row, so direct stores would be 16 bytes at a 2D-byte stride, one 128-byte line
            // per lane and instruction.  Rows past n are clipped by the tensor map.
#pragma unroll
            for (int c = 0; c < D / 2; c += 32) {
                uint32_t o0[32], o1[32];
                tmem_ld(lane_addr + kColO + (D / 2) * h + c, o0);
                if (has1) tmem_ld(lane_addr + kColO + D + (D / 2) * h + c, o1);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    float v[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) v[u] = __uint_as_float(o0[i + u]) * w0 + (has1 ? __uint_as_float(o1[i + u]) * w1 : 0.f);
                    if (want_d) {
                        const uint4 g = dov[(c + i) / 8];
                        const uint32_t gw[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const float2 gg = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gw[u]));
                            dpart = fmaf(v[2 * u], gg.x, dpart);
                            dpart = fmaf(v[2 * u + 1], gg.y, dpart);
                        }
                    }
                    uint4 q;
                    q.x = pack_bf16(v[0], v[1]); q.y = pack_bf16(v[2], v[3]);
                    q.z = pack_bf16(v[4], v[5]); q.w = pack_bf16(v[6], v[7]);
                    const int cabs = (D / 2) * h + c + i;                        // first of 8 columns
                    const int chunk = ((cabs & 63) >> 3) ^ (lane_row & 7);       // 128-byte swizzle, as the map expects
                    *reinterpret_cast<uint4 *>(sQ + (cabs >> 6) * kBoxBytes + lane_row * 128 + chunk * 16) = q;
                }
            }
            xd[h * 128 + lane_row] = dpart;
            fence_proxy_async_smem();
            mbar_arrive(bars + F_E);
            if (prep.dO != nullptr && h == 0 && mbar_wait(bars + F_E, 0, abortp, status, ERR_O)) {
                // both halves of the row are in: the backward's per-row inputs, in its padded layout
                const size_t prow = (size_t)bh * prep.n_pad + row;
                prep.Dp[prow] = row < n ? -(dpart + xd[128 + lane_row]) : 0.f;
                prep.Lp[prow] = row < n ? -(m_all + log2f(l_all)) : -INFINITY;
            }
            if (tid == 0 && mbar_wait(bars + F_E, 0, abortp, status, ERR_O)) {
                for (int b = 0; b < kBoxes; ++b)
                    if (D * pass + 64 * b < prep.d)       // (a box wholly past the head dimension has nothing to store)
                        tma_store_4d(&mapO, sQ + b * kBoxBytes, D * pass + 64 * b, q0, hq, split * (heads_all / H) + bb);
                bulk_commit();
                bulk_wait_read<0>();      // shared memory is read before the CTA may exit
            }
            if (row < sp.n_q && h == 0 && pass == 0) L[((size_t)split * heads_all + bh) * sp.n_q + row] = m_all * kLn2 + logf(l_all);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tbase, kTmemCols);
}

template <int D, int KC>
cudaError_t launch_fwd(const Problem &p, const void *Q, const void *K, const void *V, void *O, float *L,
                       const FwdForBwd &fb, cudaStream_t st)
{
    constexpr int kSmem = (KC + 4) * 128 * D * 2 + 8 * (F_COUNT + 2) + 2 * 128 * 8 + 2 * 128 * 4;
    if (KC > 1 && (fb.dO != nullptr || fb.zero_acc != nullptr)) return cudaErrorInvalidValue;   // no fused preparation with KC > 1
    CUtensorMap mq, mk, mv, mo;
    const auto bf = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    // p.d <= D columns exist in memory: loads fill the rest of a box with zeros, the store drops it
    if (!make_tensor_map_4d_strided(&mq, Q, bf, 2, p.B, p.H, p.n, p.d, p.sq.row, p.sq.head, p.sq.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mk, K, bf, 2, p.B, p.kv_heads(), p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mv, V, bf, 2, p.B, p.kv_heads(), p.n, p.d, p.skv.row, p.skv.head, p.skv.batch, 128, 64) ||
        !make_tensor_map_4d_strided(&mo, O, bf, 2, p.B, p.H, p.n, p.d, p.so.row, p.so.head, p.so.batch, 128, 64))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(tc_fwd_kernel<D, KC>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const int nqt = (p.n + BM - 1) / BM;
    LaunchScope scope(MOA_KERNEL_FWD, st);
    tc_fwd_kernel<D, KC><<<(unsigned)(nqt * p.BH() * KC), kThreads, kSmem, st>>>(
        mq, mk, mv, mo, L, p.n, p.causal, p.scale * kLog2e, nqt, heads_per_group(p, nqt), p.group(), p.H,
        FwdSplit{p.n, 1, (p.n + BN - 1) / BN}, fb.zero_acc,
        FwdPrep{(const __nv_bfloat16 *)fb.dO, fb.Lp, fb.Dp, nqt * BM, p.so, p.d}, device_status_ptr());
    return cudaGetLastError();
}

// Decode through the forward kernel: the G query heads that share a K/V head are the query rows of
// one tile (q [B,H,d] read as [B,Hkv,G,d]; rows G..127 are zero fill and are never written), the
// cache is divided among `splits` CTAs per K/V head.  O_part [splits*B, Hkv, G, d] bf16, L_part
// [splits, B*Hkv, G] fp32.
template <int D>
cudaError_t launch_fwd_decode(int B, int Hkv, int G, int n, float scale, const void *q, const void *K, const void *V,
                              void *O_part, float *L_part, int splits, int tiles_per_split, cudaStream_t st)
{
    constexpr int kSmem = 5 * 128 * D * 2 + 8 * (F_COUNT + 2) + 2 * 128 * 8 + 2 * 128 * 4;
    CUtensorMap mq, mk, mv, mo;
    const auto bf = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    if (!make_tensor_map_4d(&mq, q, bf, 2, B, Hkv, G, D, false, 128, 64) ||
        !make_tensor_map_4d(&mk, K, bf, 2, B, Hkv, n, D, false, 128, 64) ||
        !make_tensor_map_4d(&mv, V, bf, 2, B, Hkv, n, D, false, 128, 64) ||
        !make_tensor_map_4d(&mo, O_part, bf, 2, (uint64_t)splits * B, Hkv, G, D, false, 128, 64))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(tc_fwd_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    LaunchScope scope(MOA_KERNEL_FWD, st);
    tc_fwd_kernel<D, 1><<<(unsigned)(B * Hkv * splits), kThreads, kSmem, st>>>(
        mq, mk, mv, mo, L_part, n, 0, scale * kLog2e, 1, 1, 1, Hkv, FwdSplit{G, splits, tiles_per_split},
        nullptr, FwdPrep{nullptr, nullptr, nullptr, 0, Strides{0, 0, 0}, D}, device_status_ptr());
    return cudaGetLastError();
}

}  // namespace

cudaError_t tc_fwd_decode(int B, int Hkv, int G, int n, int d, float scale, const void *q, const void *K, const void *V,
                          void *O_part, float *L_part, int splits, int tiles_per_split, cudaStream_t st)
{
    if (d == 64) return launch_fwd_decode<64>(B, Hkv, G, n, scale, q, K, V, O_part, L_part, splits, tiles_per_split, st);
    if (d == 128) return launch_fwd_decode<128>(B, Hkv, G, n, scale, q, K, V, O_part, L_part, splits, tiles_per_split, st);
    return cudaErrorInvalidValue;
}

cudaError_t tc_fwd(const Problem &p, const void *Q, const void *K, const void *V, void *O, float *L,
                   const FwdForBwd &fb, cudaStream_t st)
{
    if (p.d < 8 || p.d > 256 || p.d % 8) return cudaErrorInvalidValue;
    if (p.d > 128) return launch_fwd<128, 2>(p, Q, K, V, O, L, fb, st);      // two 128-column passes, scores over both chunks
    return kernel_d(p.d) == 64 ? launch_fwd<64, 1>(p, Q, K, V, O, L, fb, st) : launch_fwd<128, 1>(p, Q, K, V, O, L, fb, st);
}

}  // namespace moa
