// bf16 GEMMs of the gated MLP on the tensor cores (tcgen05, fp32 accumulators in TMEM, operands
// staged by TMA), with the gate arithmetic fused into the epilogues.
//
//   C[M,N] = sum over operand pairs p of  A_p[M,K] * B_p[N,K]^T
//
// One persistent CTA per SM walks output tiles of 128 x 256.  Warp 0 is the TMA producer (a ring of
// stages of 64 K-elements: 16 KB of A, 32 KB of B), warp 1 allocates TMEM and issues the
// UMMAs (M = 128, N = 256, K = 16 each, four per stage), warps 2-9 are the epilogue (two warps per
// 32-lane group of TMEM, one column half each).  The two
// 256-column halves of TMEM alternate between tiles, so the epilogue of a tile runs under the main
// loop of the next one.  Every wait is bounded (ptx::mbar_wait).
//
// kPair: the same roles in each of the two CTAs of a cluster, on tiles of 256 x 256: the CTA of rank 0
// issues UMMAs of M = 256 (tcgen05.mma.cta_group::2) that read 128 rows of A and HALF of the B rows
// from each CTA's shared memory and write 128 x 256 accumulators in each CTA's TMEM.  Per SM and
// unit of work the B traffic (L2 -> shared memory, shared memory -> tensor core) halves; a stage holds
// two 64-element K blocks (64 KB) and the ring has three.  Both producers' copies complete on the full barrier of rank 0; its
// commits arrive on the empty and accumulator-full barriers of both CTAs; both epilogues hand the
// accumulator back on the barrier of rank 0; a cluster-wide barrier at both ends keeps either CTA
// from touching the other before it is set up or after it has left.  Measured: products of every
// operand layout 1240-1340 -> 1350-1530 TFLOP/s; launches of a few tiles, and shapes whose M is so
// small that pairs would need more waves, stay on single CTAs.
//
// Operand storage is a template choice per operand, because the backward's GEMMs read the same
// arrays transposed:
//   K-major  : the array is [rows = M or N, K] row-major; one TMA box of 64 K-elements x rows.
//   MN-major : the array is [K, cols = M or N] row-major; boxes of 64 columns x 64 K-rows.
// Tails in M, N and K are handled by the TMA zero fill on loads and by guards on stores.
//
// Epilogues:
//   EPI_STORE       C -> bf16; with a residual R (map C2) C + R -> bf16 (residual connections, sums of products)
//   EPI_SWIGLU_FWD  the tile's B rows are 128 rows of W1 and the same 128 rows of W3 (two maps), so
//                   its accumulator holds a | u for 128 hidden units; writes a, u and
//                   h = silu(a) * u (all from the fp32 values).
//   EPI_SWIGLU_BWD  C = dh; reads the stored a, u; writes da = dh u s (1 + a (1 - s)) and
//                   du = dh a s, s = sigmoid(a).  dh itself never reaches memory.
#include "common.cuh"
#include "ptx.cuh"
#include "tensormap.cuh"
#include "moa_block.h"

namespace moa {
namespace {

using namespace ptx;

constexpr int GM = 128, GN = 256, GK = 64;
constexpr int kGemmThreads = 320;                      // producer, issuer, eight epilogue warps
constexpr int kABytes = GM * GK * 2, kBBytes = GN * GK * 2;
// A CTA on its own stages 16 KB of A and 32 KB of B per 64 K-elements, four stages (three measured 7-16 % slower: the
// ring has to cover the L2 latency).  A CTA of a pair stages 16 KB of A and its half of B, 16 KB: six stages.
// In a pair a stage holds two such blocks (128 K-elements, 64 KB) and the ring has three: one wait and one commit of
// the issuing thread per eight UMMAs instead of per four (that thread's time per stage is on the critical path: a
// second commit per stage cost 3-4 %).
constexpr int kMaxStages = 6;
__host__ __device__ constexpr int gemm_sub(bool pair) { return pair ? 2 : 1; }                 // 64-element K blocks per stage
__host__ __device__ constexpr int gemm_stages(bool pair) { return pair ? 3 : 4; }
__host__ __device__ constexpr int gemm_sub_bytes(bool pair) { return kABytes + (pair ? kBBytes / 2 : kBBytes); }
__host__ __device__ constexpr int gemm_stage_bytes(bool pair) { return gemm_sub(pair) * gemm_sub_bytes(pair); }
constexpr int kMnBox = 64 * GK * 2;                    // one MN-major box: 64 columns x 64 K-rows
constexpr int kOutBox = 128 * 64 * 2;                  // one staged output chunk: 128 rows x 64 columns, bf16
__host__ __device__ constexpr int gemm_smem(bool pair)
{
    return gemm_stages(pair) * gemm_stage_bytes(pair) + 2 * kOutBox + 1024 /* alignment */ + 256 /* barriers */;
}
constexpr int kStages = kMaxStages;                    // barrier slots (the ring uses gemm_stages(pair) of them)

enum { EPI_STORE = 0, EPI_SWIGLU_FWD = 1, EPI_SWIGLU_BWD = 2 };
enum { G_FULL = 0, G_EMPTY = kStages, G_ACCFULL = 2 * kStages, G_ACCEMPTY = 2 * kStages + 2, G_EPI = 2 * kStages + 4,
       G_IN = 2 * kStages + 5, G_RES = 2 * kStages + 6 /* two */, G_COUNT = 2 * kStages + 8 };
enum { GERR_EMPTY = 0x301, GERR_FULL = 0x302, GERR_ACCFULL = 0x303, GERR_ACCEMPTY = 0x304, GERR_EPI = 0x305, GERR_IN = 0x306, GERR_RES = 0x307 };

// Outputs leave through TMA stores (tensor maps C0..C3: STORE: C (and the second product's C); FWD gate: a, u, h;
// BWD gate: da, du, and the stored a, u as C2, C3, which its epilogue brings in by TMA loads).

__device__ __forceinline__ void unpack8(const uint4 &v, float *f)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 t = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&w[i]));
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}
// 1 / (1 + exp(-a)) on the two fast special-function instructions (ex2.approx, rcp.approx).  (__frcp_rn, the
// correctly rounded reciprocal, is a multi-instruction sequence: with it the backward gate epilogue took 17,000
// cycles per tile instead of 6,800 and held its GEMM 25 % below the others.)
__device__ __forceinline__ float sigmoidf_fast(float a)
{
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-1.4426950408889634f * a));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.f + e));
    return r;
}

// Tile order: groups of `kGroup` tile rows, column-major inside a group, so that the CTAs running at the same time
// share a few A row blocks and a few B column blocks.  B is swept once per group: the launcher picks taller groups
// when B is too large to survive in L2 between sweeps (with groups of 8 a [8192 x 2048] x [16384 x 2048]^T product
// read its 67 MB of B eight times from DRAM: the outputs streaming through L2 evict it in between).
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int kGroup, int &tm, int &tn)
{
    const int per_group = kGroup * tiles_n;
    const int g = t / per_group, r = t - g * per_group;
    const int rows = min(kGroup, tiles_m - g * kGroup);
    tn = r / rows;
    tm = g * kGroup + (r - tn * rows);
}

template <bool kAMn, bool kBMn, int kEpi, bool kPair>
__global__ void __launch_bounds__(kGemmThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap mapA0, const __grid_constant__ CUtensorMap mapB0,
               const __grid_constant__ CUtensorMap mapA1, const __grid_constant__ CUtensorMap mapB1,
               const __grid_constant__ CUtensorMap mapC0, const __grid_constant__ CUtensorMap mapC1,
               const __grid_constant__ CUtensorMap mapC2, const __grid_constant__ CUtensorMap mapC3, int M, int N, int K, int nparts, int nbatch, int a_blocked, int b_blocked, int has_res, int group_rows, unsigned int *status)
{
    constexpr bool kDualN = kEpi == EPI_SWIGLU_FWD;         // B tile = 128 rows of map B0 + 128 rows of map B1
    constexpr int kTileN = kDualN ? 128 : GN;                // output columns a tile covers
    // Epilogue warps: two per 32-lane group of TMEM; together they fill one 64-column output chunk at a time
    constexpr int kEpiWarps = 8;
    // kPair: the two CTAs of a cluster share tiles of 256 rows: UMMAs of M = 256 issued by the CTA of rank 0 read the
    // A rows and the B half staged in each CTA (this CTA: rows rank*128.. of the tile, B rows rank*128.. of its 256)
    // and write each CTA's accumulator; every CTA runs its own producer and epilogue.
    constexpr int kSt = gemm_stages(kPair), kStageBytes = gemm_stage_bytes(kPair), kTileM = kPair ? 2 * GM : GM;
    constexpr int kSub = gemm_sub(kPair), kSubBytes = gemm_sub_bytes(kPair);
    const uint32_t rank = kPair ? cluster_ctarank() : 0u;
    const int cta = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, ncta = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *sout = sm + kSt * kStageBytes;               // two staged output chunks (128-byte swizzle)
    uint64_t *bars = reinterpret_cast<uint64_t *>(sout + 2 * kOutBox);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + G_COUNT);
    volatile uint32_t *abortp = tmem_slot + 1;
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;

    const int tiles_m = (M + kTileM - 1) / kTileM, tiles_n = (N + kTileN - 1) / kTileN;
    // nbatch = 2: two independent products of one shape in one launch (A1 B1^T -> map C1 after A0 B0^T ->
    // map C0), so that their tiles share the waves of the persistent grid
    const int tiles_one = tiles_m * tiles_n, tiles = tiles_one * nbatch;
    const int nk = (K + GK * kSub - 1) / (GK * kSub), nk_total = nk * nparts;     // stages per operand pair

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(bars + G_FULL + i, 1);
            mbar_init(bars + G_EMPTY + i, 1);
        }
        mbar_init(bars + G_ACCFULL + 0, 1);
        mbar_init(bars + G_ACCFULL + 1, 1);
        mbar_init(bars + G_ACCEMPTY + 0, (kPair ? 2 : 1) * 32 * kEpiWarps);   // a pair: the epilogue threads of both CTAs
        mbar_init(bars + G_ACCEMPTY + 1, (kPair ? 2 : 1) * 32 * kEpiWarps);
        mbar_init(bars + G_EPI, 32 * kEpiWarps);
        mbar_init(bars + G_IN, 1);
        mbar_init(bars + G_RES + 0, 1);
        mbar_init(bars + G_RES + 1, 1);
        *abortp = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        if (kPair) {
            tmem_alloc_pair(tmem_slot, 512);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(tmem_slot, 512);
            tmem_relinquish();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (kPair) cluster_sync_all();       // the other CTA's barriers are initialised before anything arrives on them
    tc_fence_after();
    const uint32_t tbase = *tmem_slot;

    if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------------ TMA producer
        prefetch_tensormap(&mapA0);
        prefetch_tensormap(&mapB0);
        ArmCounts<G_COUNT> armed;     // barriers armed for copies into shared memory
        int it = 0;
        bool ok = true;
        for (int t = cta; ok && t < tiles; t += ncta) {
            int tm, tn;
            const int second = t >= tiles_one ? 1 : 0;
            tile_coords(t - second * tiles_one, tiles_m, tiles_n, group_rows, tm, tn);
            const int m0 = tm * kTileM + (int)rank * GM, n0 = tn * kTileN;
            const int nb0 = n0 + ((kPair && !kDualN) ? (int)rank * (GN / 2) : 0);    // first B row this CTA stages
            for (int ks = 0; ks < nk_total; ++ks, ++it) {
                const int s = it % kSt;
                if (!mbar_wait(bars + G_EMPTY + s, ((it / kSt) & 1) ^ 1, abortp, status, GERR_EMPTY)) { ok = false; break; }
                const int part = ks / nk;
                const CUtensorMap *ma = (part || second) ? &mapA1 : &mapA0;
                const CUtensorMap *mb = ((part || second) && !kDualN) ? &mapB1 : &mapB0;
                uint64_t *full = bars + G_FULL + s;
                // a pair: the copies of both CTAs complete on the barrier of rank 0, which its producer arms for both
                const uint32_t full_pair = kPair ? mapa_u32(smem_u32(full), 0) : 0u;
                if (!kPair || rank == 0) mbar_arm(bars, G_FULL + s, (kPair ? 2 : 1) * kStageBytes, armed);
                auto load = [&](void *dst, const CUtensorMap *m, int x, int y, int z) {
                    if (kPair) tma_load_3d_pair(dst, m, full_pair, x, y, z);
                    else tma_load_3d(dst, m, full, x, y, z);
                };
#pragma unroll
              for (int sub = 0; sub < kSub; ++sub) {          // (a block past K is filled with zeros by the copy)
                const int k0 = ((ks - part * nk) * kSub + sub) * GK;
                uint8_t *sa = sm + s * kStageBytes + sub * kSubBytes, *sb = sa + kABytes;
                if (kAMn) {
                    if (a_blocked) {                          // one copy: (64 columns, K rows, column blocks)
                        load(sa, ma, 0, k0, m0 / 64);
                    } else {
                        load(sa, ma, m0, k0, 0);
                        load(sa + kMnBox, ma, m0 + 64, k0, 0);
                    }
                } else {
                    load(sa, ma, k0, m0, 0);
                }
                if (kBMn) {
                    if (b_blocked) {
                        load(sb, mb, 0, k0, nb0 / 64);
                    } else {
#pragma unroll
                        for (int b = 0; b < (kPair ? 2 : 4); ++b) load(sb + b * kMnBox, mb, nb0 + 64 * b, k0, 0);
                    }
                } else if (kDualN) {
                    if (kPair) {                              // rank 0 stages the W1 rows, rank 1 the W3 rows
                        load(sb, rank ? &mapB1 : &mapB0, k0, n0, 0);
                    } else {
                        load(sb, &mapB0, k0, n0, 0);
                        load(sb + kBBytes / 2, &mapB1, k0, n0, 0);
                    }
                } else {
                    load(sb, mb, k0, nb0, 0);
                }
              }
            }
        }
        mbar_drain(bars, armed);      // copies of this CTA still on their way land before it leaves (bounded)
    } else if (warp == 1 && lane == 0 && rank == 0) {
        // ------------------------------------------------------------------- UMMA issuer
        constexpr uint32_t idesc = idesc_bf16_f32(kTileM, GN, kAMn ? 1 : 0, kBMn ? 1 : 0);
        const uint64_t km_proto = smem_desc_sw128(0, 16, 1024), mn_proto = smem_desc_sw128(0, kMnBox, 1024);
        const uint32_t a_hi = (uint32_t)((kAMn ? mn_proto : km_proto) >> 32), b_hi = (uint32_t)((kBMn ? mn_proto : km_proto) >> 32);
        const uint32_t a_lo0 = (uint32_t)(kAMn ? mn_proto : km_proto), b_lo0 = (uint32_t)(kBMn ? mn_proto : km_proto);
        constexpr uint32_t a_step = (kAMn ? 2048 : 32) >> 4, b_step = (kBMn ? 2048 : 32) >> 4;   // per 16 K-elements
        int it = 0, ti = 0;
        bool ok = true;
        for (int t = cta; ok && t < tiles; t += ncta, ++ti) {
            const int buf = ti & 1;
            if (!mbar_wait(bars + G_ACCEMPTY + buf, ((ti >> 1) & 1) ^ 1, abortp, status, GERR_ACCEMPTY)) break;
            tc_fence_after();
            const uint32_t acc = tbase + (uint32_t)(buf * GN);
            for (int ks = 0; ks < nk_total; ++ks, ++it) {
                const int s = it % kSt;
                if (!mbar_wait(bars + G_FULL + s, (it / kSt) & 1, abortp, status, GERR_FULL)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_lo = a_lo0 + ((smem_u32(sm + s * kStageBytes) >> 4) & 0x3FFFu);
                const uint32_t b_lo = b_lo0 + ((smem_u32(sm + s * kStageBytes + kABytes) >> 4) & 0x3FFFu);
                if (kPair) {
#pragma unroll
                    for (int sub = 0; sub < kSub; ++sub) {
                        const uint32_t a_s = a_lo + (uint32_t)(sub * (kSubBytes >> 4)), b_s = b_lo + (uint32_t)(sub * (kSubBytes >> 4));
                        if (ks == 0 && sub == 0) umma_ss2_pair<false>(acc, a_s, a_hi, b_s, b_hi, idesc);
                        else                     umma_ss2_pair<true>(acc, a_s, a_hi, b_s, b_hi, idesc);
#pragma unroll
                        for (int q = 1; q < GK / 16; ++q)
                            umma_ss2_pair<true>(acc, a_s + q * a_step, a_hi, b_s + q * b_step, b_hi, idesc);
                    }
                    umma_commit_pair(bars + G_EMPTY + s);     // frees the stage in both CTAs
                } else {
                    if (ks == 0) umma_ss2<false>(acc, a_lo, a_hi, b_lo, b_hi, idesc);
                    else         umma_ss2<true>(acc, a_lo, a_hi, b_lo, b_hi, idesc);
#pragma unroll
                    for (int q = 1; q < GK / 16; ++q)
                        umma_ss2<true>(acc, a_lo + q * a_step, a_hi, b_lo + q * b_step, b_hi, idesc);
                    umma_commit(bars + G_EMPTY + s);          // the stage is free once these UMMAs have read it
                }
            }
            if (ok) {
                if (kPair) umma_commit_pair(bars + G_ACCFULL + buf);
                else umma_commit(bars + G_ACCFULL + buf);
            }
        }
    } else if (warp >= 2 && warp < 2 + kEpiWarps) {
        // ---------------------------------------------------------------------- epilogue
        // A thread owns one row of the tile (its TMEM lane) and 32 of the 64 columns of the current chunk.  Results go
        // to a shared-memory chunk in the 128-byte-swizzle layout and leave as one TMA store per chunk (whole 128-byte
        // lines; rows and columns past the array are clipped by the tensor map): row-owner 16-byte stores to global
        // memory cost one L2 request each, and at 6000 requests per tile they slowed the operand loads of the next tile.
        const int lane_row = 32 * (warp % 4) + lane;               // TMEM lane = row of the tile
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        const int half = (warp - 2) / 4;                           // which 32 columns of a 64-column chunk
        const bool leader = tid == 64;
        uint32_t epi_phase = 0, chunk_q = 0, in_q = 0;
        ArmCounts<G_COUNT> armed;     // barriers the leader armed for copies into the staging buffers
        bool ok = true;
        // hands an accumulator back to the issuer (a pair: to the issuer in the CTA of rank 0)
        const uint32_t accempty_pair = kPair ? mapa_u32(smem_u32(bars + G_ACCEMPTY), 0) : 0u;
        auto acc_release = [&](int b) {
            tc_fence_before();
            if (kPair) mbar_arrive_cluster(accempty_pair + 8u * (uint32_t)b);
            else mbar_arrive(bars + G_ACCEMPTY + b);
        };
        // all epilogue threads meet (bounded wait)
        auto epi_sync = [&]() -> bool {
            mbar_arrive(bars + G_EPI);
            const bool r = mbar_wait(bars + G_EPI, epi_phase & 1, abortp, status, GERR_EPI);
            ++epi_phase;
            return r;
        };
        // the 32 values of this thread (as 16 bf16 pairs) -> staged chunk -> TMA store at (row0, col0)
        auto stage_store = [&](const CUtensorMap *map, const uint32_t (&v)[16], int col0, int row0) -> bool {
            uint8_t *buf = sout + (chunk_q & 1) * kOutBox;
            if (leader) bulk_wait_read<1>();                       // the store issued two chunks ago has left this buffer
            if (!epi_sync()) return false;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                *reinterpret_cast<uint4 *>(buf + lane_row * 128 + (((half * 4 + j) ^ (lane_row & 7)) << 4)) =
                    make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            fence_proxy_async_smem();
            if (!epi_sync()) return false;
            if (leader) {
                if (row0 < M) tma_store_3d(map, buf, col0, row0, 0);   // (a pair's second half can lie past the last row)
                bulk_commit();
            }
            ++chunk_q;
            return true;
        };
        // the same with a residual: the chunk of R comes into the staging buffer by TMA, every thread adds its 32
        // values in place, and the buffer leaves by a TMA store
        auto stage_store_res = [&](const CUtensorMap *map, const uint32_t (&racc)[32], int col0, int row0) -> bool {
            const uint32_t b = chunk_q & 1;
            uint8_t *buf = sout + b * kOutBox;
            if (leader) {
                bulk_wait_read<1>();                                   // the store issued two chunks ago has left this buffer
                mbar_arm(bars, G_RES + (int)b, kOutBox, armed);
                tma_load_3d(buf, &mapC2, bars + G_RES + b, col0, row0, 0);
            }
            if (!mbar_wait(bars + G_RES + b, (chunk_q >> 1) & 1, abortp, status, GERR_RES)) return false;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 *pr = reinterpret_cast<uint4 *>(buf + lane_row * 128 + (((half * 4 + j) ^ (lane_row & 7)) << 4));
                float r8[8];
                unpack8(*pr, r8);
#pragma unroll
                for (int i = 0; i < 8; ++i) r8[i] += __uint_as_float(racc[8 * j + i]);
                *pr = make_uint4(pack_bf16(r8[0], r8[1]), pack_bf16(r8[2], r8[3]), pack_bf16(r8[4], r8[5]), pack_bf16(r8[6], r8[7]));
            }
            fence_proxy_async_smem();
            if (!epi_sync()) return false;
            if (leader) {
                if (row0 < M) tma_store_3d(map, buf, col0, row0, 0);   // (a pair's second half can lie past the last row)
                bulk_commit();
            }
            ++chunk_q;
            return true;
        };
        int ti = 0;
        for (int t = cta; ok && t < tiles; t += ncta, ++ti) {
            int tm, tn;
            const int second = t >= tiles_one ? 1 : 0;
            tile_coords(t - second * tiles_one, tiles_m, tiles_n, group_rows, tm, tn);
            const int buf = ti & 1;
            const int m0 = tm * kTileM + (int)rank * GM, n0 = tn * kTileN;
            if (kEpi == EPI_STORE && has_res && leader) {     // the tile's residual: into L2 while its main loop runs
#pragma unroll
                for (int c0 = 0; c0 < GN; c0 += 64) tma_prefetch_3d(&mapC2, n0 + c0, m0, 0);
            }
            if (kEpi == EPI_SWIGLU_BWD && leader) {       // the tile's stored a, u: into L2 while its main loop runs
#pragma unroll
                for (int c0 = 0; c0 < GN; c0 += 64) {
                    tma_prefetch_3d(&mapC2, n0 + c0, m0, 0);
                    tma_prefetch_3d(&mapC3, n0 + c0, m0, 0);
                }
            }
            if (!mbar_wait(bars + G_ACCFULL + buf, (ti >> 1) & 1, abortp, status, GERR_ACCFULL)) break;
            tc_fence_after();
            const uint32_t acc = lane_addr + (uint32_t)(buf * GN);
            if (kEpi == EPI_SWIGLU_FWD) {
#pragma unroll 1
                for (int c0 = 0; ok && c0 < 128; c0 += 64) {
                    const int c = c0 + 32 * half;
                    uint32_t ra[32], ru[32];
                    tmem_ld(acc + c, ra);
                    tmem_ld(acc + 128 + c, ru);
                    tc_wait_ld();
                    if (c0 == 64) {                       // last read of this accumulator: hand it back early
                        acc_release(buf);
                    }
                    uint32_t pa[16], pu[16], ph[16];
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const float a0 = __uint_as_float(ra[e]), a1 = __uint_as_float(ra[e + 1]);
                        const float u0 = __uint_as_float(ru[e]), u1 = __uint_as_float(ru[e + 1]);
                        pa[e / 2] = pack_bf16(a0, a1);
                        pu[e / 2] = pack_bf16(u0, u1);
                        ph[e / 2] = pack_bf16(a0 * sigmoidf_fast(a0) * u0, a1 * sigmoidf_fast(a1) * u1);
                    }
                    ok = stage_store(&mapC0, pa, n0 + c0, m0) && stage_store(&mapC1, pu, n0 + c0, m0) &&
                         stage_store(&mapC2, ph, n0 + c0, m0);
                }
            } else if (kEpi == EPI_STORE) {
#pragma unroll 1
                for (int c0 = 0; ok && c0 < GN; c0 += 64) {
                    uint32_t r[32];
                    tmem_ld(acc + c0 + 32 * half, r);
                    tc_wait_ld();
                    if (c0 == GN - 64) {                  // last read of this accumulator: hand it back early
                        acc_release(buf);
                    }
                    if (has_res) {
                        ok = stage_store_res(&mapC0, r, n0 + c0, m0);
                    } else {
                        uint32_t pc[16];
#pragma unroll
                        for (int e = 0; e < 32; e += 2) pc[e / 2] = pack_bf16(__uint_as_float(r[e]), __uint_as_float(r[e + 1]));
                        ok = stage_store(second ? &mapC1 : &mapC0, pc, n0 + c0, m0);
                    }
                }
            } else {
                // Backward gate: per 64-column chunk the stored a and u come into the two staging buffers by TMA, every
                // thread turns its 32 + 32 values into da, du in place, and the buffers leave by TMA stores.
#pragma unroll 1
                for (int c0 = 0; ok && c0 < GN; c0 += 64, ++in_q) {
                    if (leader) {
                        bulk_wait_read<0>();              // the previous chunk's stores have left both buffers
                        mbar_arm(bars, G_IN, 2 * kOutBox, armed);
                        tma_load_3d(sout, &mapC2, bars + G_IN, n0 + c0, m0, 0);
                        tma_load_3d(sout + kOutBox, &mapC3, bars + G_IN, n0 + c0, m0, 0);
                    }
                    uint32_t r[32];
                    tmem_ld(acc + c0 + 32 * half, r);
                    tc_wait_ld();
                    if (c0 == GN - 64) {
                        acc_release(buf);
                    }
                    if (!mbar_wait(bars + G_IN, in_q & 1, abortp, status, GERR_IN)) { ok = false; break; }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint32_t off = lane_row * 128 + (((half * 4 + q) ^ (lane_row & 7)) << 4);
                        uint4 *pa = reinterpret_cast<uint4 *>(sout + off), *pu = reinterpret_cast<uint4 *>(sout + kOutBox + off);
                        float fa[8], fu[8], da[8], du[8];
                        unpack8(*pa, fa);
                        unpack8(*pu, fu);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float f = __uint_as_float(r[8 * q + i]);
                            const float sg = sigmoidf_fast(fa[i]);
                            da[i] = f * fu[i] * sg * (1.f + fa[i] * (1.f - sg));
                            du[i] = f * fa[i] * sg;
                        }
                        *pa = make_uint4(pack_bf16(da[0], da[1]), pack_bf16(da[2], da[3]), pack_bf16(da[4], da[5]), pack_bf16(da[6], da[7]));
                        *pu = make_uint4(pack_bf16(du[0], du[1]), pack_bf16(du[2], du[3]), pack_bf16(du[4], du[5]), pack_bf16(du[6], du[7]));
                    }
                    fence_proxy_async_smem();
                    if (!epi_sync()) { ok = false; break; }
                    if (leader) {
                        if (m0 < M) {
                            tma_store_3d(&mapC0, sout, n0 + c0, m0, 0);
                            tma_store_3d(&mapC1, sout + kOutBox, n0 + c0, m0, 0);
                        }
                        bulk_commit();
                    }
                }
            }
        }
        if (leader) {
            bulk_wait<0>();               // every store has completed before the CTA gives up its shared memory
            mbar_drain(bars, armed);      // and so has every copy into the staging buffers (bounded)
        }
    }
    tc_fence_before();
    __syncthreads();
    if (kPair) {
        // neither CTA leaves, or frees its TMEM, while the other may still read its shared memory, write its
        // accumulator or arrive on its barriers
        __syncwarp();
        cluster_sync_all();
        if (warp == 1) tmem_dealloc_pair(tbase, 512);
    } else if (warp == 1) {
        tmem_dealloc(tbase, 512);
    }
}

struct Operand {
    const void *p;
    int rows, cols;          // the array as stored: [rows, cols] row-major
};

// K-major: stored [MN, K], box of `box_rows` rows x 64 K-elements.  MN-major: stored [K, MN]: one blocked box of
// box_rows / 64 column blocks x 64 K-rows when `blocked`, else boxes of 64 x 64.
bool operand_map(CUtensorMap *m, const Operand &o, bool mn_major, int box_rows, bool blocked = false)
{
    if (mn_major && blocked)
        return make_tensor_map_blocked(m, o.p, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)o.rows, (uint64_t)o.cols, 64,
                                       (uint32_t)box_rows / 64);
    return make_tensor_map_3d(m, o.p, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 1, (uint64_t)o.rows, (uint64_t)o.cols,
                              mn_major ? 64 : (uint32_t)box_rows, 64);
}

// Clusters of two CTAs of `kernel` that can be resident at once (cudaOccupancyMaxActiveClusters; cached per kernel
// and device); half the SM count if the query fails.
template <typename K>
int max_active_pairs(K kernel, int smem)
{
    constexpr int kMaxDev = 64;
    static int cache[kMaxDev] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return device_info().sms / 2;
    if (cache[dev] > 0) return cache[dev];
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3((unsigned)device_info().sms / 2 * 2);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = smem;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        n = device_info().sms / 2;
    }
    if (n > device_info().sms / 2) n = device_info().sms / 2;
    return cache[dev] = n;
}

template <bool kAMn, bool kBMn, int kEpi, bool kPair>
// C0..C2: output arrays (row length ldc); unused ones may repeat C0.
cudaError_t launch_gemm_as(const Operand &A0, const Operand &B0, const Operand *A1, const Operand *B1, void *C0, void *C1,
                        const void *C2, const void *C3, int c_rows, int ldc, int M, int N, int K, cudaStream_t st,
                        int nbatch = 1, bool has_res = false)
{
    constexpr bool kDualN = kEpi == EPI_SWIGLU_FWD;
    CUtensorMap ma0, mb0, ma1, mb1;
    const int b_rows = (kDualN || kPair) ? 128 : GN;     // B rows one CTA stages per copy
    // MN-major operands whose width is a multiple of 64 come in by one blocked copy per stage (try the encode; if the
    // driver refuses the map, or a width has a tail, use one copy per 64-column block)
    const Operand &a1 = A1 ? *A1 : A0, &b1 = B1 ? *B1 : B0;
    bool a_blocked = kAMn && A0.cols % 64 == 0 && a1.cols % 64 == 0;
    bool b_blocked = kBMn && B0.cols % 64 == 0 && b1.cols % 64 == 0;
    if (a_blocked && !(operand_map(&ma0, A0, true, GM, true) && operand_map(&ma1, a1, true, GM, true))) a_blocked = false;
    if (b_blocked && !(operand_map(&mb0, B0, true, b_rows, true) && operand_map(&mb1, b1, true, b_rows, true))) b_blocked = false;
    if (!a_blocked && (!operand_map(&ma0, A0, kAMn, GM) || !operand_map(&ma1, a1, kAMn, GM))) return cudaErrorInvalidValue;
    if (!b_blocked && (!operand_map(&mb0, B0, kBMn, b_rows) || !operand_map(&mb1, b1, kBMn, b_rows))) return cudaErrorInvalidValue;
    CUtensorMap mc[4];
    const void *cs[4] = {C0, C1 ? C1 : C0, C2 ? C2 : C0, C3 ? C3 : C0};
    for (int i = 0; i < 4; ++i)     // [c_rows, ldc] bf16, boxes of 128 rows x 64 columns, 128-byte swizzle
        if (!make_tensor_map_3d(&mc[i], cs[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 1, (uint64_t)c_rows, (uint64_t)ldc, 128, 64))
            return cudaErrorInvalidValue;
    auto kernel = tc_gemm_kernel<kAMn, kBMn, kEpi, kPair>;
    constexpr int kSmem = gemm_smem(kPair), kTileM = kPair ? 2 * GM : GM;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const int tiles = ((M + kTileM - 1) / kTileM) * ((N + (kDualN ? 128 : GN) - 1) / (kDualN ? 128 : GN)) * nbatch;
    const int nparts = (A1 && !kDualN && nbatch == 1) ? 2 : 1;
    // Groups of 8 tile rows, unless B is too large to stay in L2 between groups (above 48 MB): then groups as tall as
    // keeps their A rows within 32 MB, so that B is swept fewer times (measured: taller groups cost the products with
    // a small B 2-5 %, and save the forward gate GEMM, whose B is W1 and W3 together, 3 % and 70 % of its DRAM reads)
    const long long b_bytes = (long long)B0.rows * B0.cols * 2 * ((kDualN || nparts == 2) ? 2 : 1);
    long long group_rows = 8;
    if (b_bytes > (48LL << 20)) {
        group_rows = (32LL << 20) / ((long long)GM * K * nparts * 2);
        group_rows = group_rows < 8 ? 8 : group_rows > 64 ? 64 : group_rows;
    }
    if (kPair) group_rows = group_rows / 2 < 2 ? 2 : group_rows / 2;     // tile rows of 256
    LaunchScope scope(MOA_KERNEL_OTHER, st);
    // persistent grid: one CTA per SM, or as many clusters of two as the device can hold at once
    const int sms = device_info().sms, pairs = kPair ? max_active_pairs(kernel, kSmem) : 0;
    const int ctas = kPair ? 2 * (tiles < pairs ? tiles : pairs) : (tiles < sms ? tiles : sms);
    if (!kPair) {
        kernel<<<ctas, kGemmThreads, kSmem, st>>>(ma0, mb0, ma1, mb1, mc[0], mc[1], mc[2], mc[3], M, N, K, nparts, nbatch,
                                                  a_blocked ? 1 : 0, b_blocked ? 1 : 0, has_res ? 1 : 0, (int)group_rows,
                                                  device_status_ptr());
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = st;
    if (kPair) {
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    return cudaLaunchKernelEx(&cfg, kernel, ma0, mb0, ma1, mb1, mc[0], mc[1], mc[2], mc[3], M, N, K, nparts, nbatch,
                              a_blocked ? 1 : 0, b_blocked ? 1 : 0, has_res ? 1 : 0, (int)group_rows, device_status_ptr());
}

// Pairs of CTAs (tiles of 256 rows, half the B traffic per SM) by default; single CTAs where pairs would need more
// waves.  MOA_GEMM_PAIR (read once): 0 never pairs, 2 always.
int gemm_pair_mode()
{
    static int mode = -1;
    if (mode < 0) {
        const char *e = getenv("MOA_GEMM_PAIR");
        mode = e ? atoi(e) : 1;
    }
    return mode;
}
template <bool kAMn, bool kBMn, int kEpi>
cudaError_t launch_gemm(const Operand &A0, const Operand &B0, const Operand *A1, const Operand *B1, void *C0, void *C1,
                        const void *C2, const void *C3, int c_rows, int ldc, int M, int N, int K, cudaStream_t st,
                        int nbatch = 1, bool has_res = false)
{
    const int tn = kEpi == EPI_SWIGLU_FWD ? 128 : GN;
    const long long cols = (N + tn - 1) / tn;
    const long long pair_tiles = (long long)((M + 2 * GM - 1) / (2 * GM)) * cols * nbatch;
    const long long single_tiles = (long long)((M + GM - 1) / GM) * cols * nbatch;
    // pairs unless they would need more waves than single CTAs (tiny M); the two gate GEMMs only when the main loop
    // outlasts their epilogue
    const long long sms = device_info().sms, pairs = sms / 2;
    const bool fits = pair_tiles >= 8 && (pair_tiles + pairs - 1) / pairs <= (single_tiles + sms - 1) / sms;   // (a few tiles: launch-bound)
    if (gemm_pair_mode() == 2 || (gemm_pair_mode() && fits && (kEpi == EPI_STORE || K >= 1024)))
        return launch_gemm_as<kAMn, kBMn, kEpi, true>(A0, B0, A1, B1, C0, C1, C2, C3, c_rows, ldc, M, N, K, st, nbatch, has_res);
    return launch_gemm_as<kAMn, kBMn, kEpi, false>(A0, B0, A1, B1, C0, C1, C2, C3, c_rows, ldc, M, N, K, st, nbatch, has_res);
}

}  // namespace

// C[M,N] = A B^T (+ R): A given as [M,K] (a_mn = 0) or [K,M] (a_mn = 1), B as [N,K] (b_mn = 0) or [K,N] (b_mn = 1)
cudaError_t gemm_bf16(int a_mn, int b_mn, int M, int N, int K, const void *A, const void *B, const void *R, void *C,
                      cudaStream_t st)
{
    const Operand a{A, a_mn ? K : M, a_mn ? M : K}, b{B, b_mn ? K : N, b_mn ? N : K};
    const bool res = R != nullptr;
    if (!a_mn && !b_mn) return launch_gemm<false, false, EPI_STORE>(a, b, nullptr, nullptr, C, nullptr, R, nullptr, M, N, M, N, K, st, 1, res);
    if (!a_mn && b_mn) return launch_gemm<false, true, EPI_STORE>(a, b, nullptr, nullptr, C, nullptr, R, nullptr, M, N, M, N, K, st, 1, res);
    if (a_mn && b_mn) return launch_gemm<true, true, EPI_STORE>(a, b, nullptr, nullptr, C, nullptr, R, nullptr, M, N, M, N, K, st, 1, res);
    return launch_gemm<true, false, EPI_STORE>(a, b, nullptr, nullptr, C, nullptr, R, nullptr, M, N, M, N, K, st, 1, res);
}

cudaError_t gated_mlp_fwd(int n, int d, int dff, const void *x, const void *W1, const void *W3, const void *W2,
                          const void *res, void *a, void *u, void *h, void *y, cudaStream_t st)
{
    // a | u = x [W1; W3]^T with the gate in the epilogue, then y = h W2^T
    const Operand X{x, n, d}, w1{W1, dff, d}, w3{W3, dff, d}, Hh{h, n, dff}, w2{W2, d, dff};
    cudaError_t e = launch_gemm<false, false, EPI_SWIGLU_FWD>(X, w1, nullptr, &w3, a, u, h, nullptr, n, dff, n, dff, d, st);
    if (e != cudaSuccess) return e;
    return launch_gemm<false, false, EPI_STORE>(Hh, w2, nullptr, nullptr, y, nullptr, res, nullptr, n, d, n, d, dff, st, 1, res != nullptr);
}

cudaError_t gated_mlp_bwd(int n, int d, int dff, const void *x, const void *W1, const void *W3, const void *W2,
                          const void *a, const void *u, const void *h, const void *dy, void *da, void *du,
                          void *dx, void *dW1, void *dW3, void *dW2, cudaStream_t st)
{
    const Operand X{x, n, d}, w1{W1, dff, d}, w3{W3, dff, d}, w2{W2, d, dff}, Hh{h, n, dff}, DY{dy, n, d};
    const Operand DA{da, n, dff}, DU{du, n, dff};
    // dh = dy W2 (W2 [d,d_ff] read as the MN-major B operand), gate backward in the epilogue -> da, du
    cudaError_t e = launch_gemm<false, true, EPI_SWIGLU_BWD>(DY, w2, nullptr, nullptr, da, du, a, u, n, dff, n, dff, d, st);
    if (e != cudaSuccess) return e;
    // dW2 [d,d_ff] = dy^T h: both operands read transposed (K = tokens)
    if ((e = launch_gemm<true, true, EPI_STORE>(DY, Hh, nullptr, nullptr, dW2, nullptr, nullptr, nullptr, d, dff, d, dff, n, st)) !=
        cudaSuccess)
        return e;
    // dW1 = da^T x, dW3 = du^T x   [d_ff,d]: one launch, so that the two tile sets fill the waves together
    if ((e = launch_gemm<true, true, EPI_STORE>(DA, X, &DU, &X, dW1, dW3, nullptr, nullptr, dff, d, dff, d, n, st, 2)) != cudaSuccess)
        return e;
    // dx = da W1 + du W3: two operand pairs accumulate into one tile (W1, W3 [d_ff,d] as MN-major B)
    return launch_gemm<false, true, EPI_STORE>(DA, w1, &DU, &w3, dx, nullptr, nullptr, nullptr, n, d, n, d, dff, st);
}

}  // namespace moa
