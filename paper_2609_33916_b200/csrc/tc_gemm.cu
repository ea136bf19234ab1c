// bf16 GEMMs of the gated MLP on the tensor cores (tcgen05, fp32 accumulators in TMEM, operands
// staged by TMA), with the gate arithmetic fused into the epilogues.
//
//   C[M,N] = sum over operand pairs p of  A_p[M,K] * B_p[N,K]^T
//
// One persistent CTA per SM walks output tiles of 128 x 256.  Warp 0 is the TMA producer (a ring of
// kStages stages of 64 K-elements: 16 KB of A, 32 KB of B), warp 1 allocates TMEM and issues the
// UMMAs (M = 128, N = 256, K = 16 each, four per stage), warps 2-9 are the epilogue (two warps per
// 32-lane group of TMEM, one column half each).  The two
// 256-column halves of TMEM alternate between tiles, so the epilogue of a tile runs under the main
// loop of the next one.  Every wait is bounded (ptx::mbar_wait).
//
// Operand storage is a template choice per operand, because the backward's GEMMs read the same
// arrays transposed:
//   K-major  : the array is [rows = M or N, K] row-major; one TMA box of 64 K-elements x rows.
//   MN-major : the array is [K, cols = M or N] row-major; boxes of 64 columns x 64 K-rows.
// Tails in M, N and K are handled by the TMA zero fill on loads and by guards on stores.
//
// Epilogues:
//   EPI_STORE       C -> bf16
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
constexpr int kStages = 4;   // three stages measured 7-16 % slower: the ring has to cover the L2 latency
constexpr int kGemmThreads = 320;                      // producer, issuer, eight epilogue warps
constexpr int kABytes = GM * GK * 2, kBBytes = GN * GK * 2, kStageBytes = kABytes + kBBytes;
constexpr int kMnBox = 64 * GK * 2;                    // one MN-major box: 64 columns x 64 K-rows
constexpr int kGemmSmem = kStages * kStageBytes + 1024 /* alignment */ + 256 /* barriers */;

enum { EPI_STORE = 0, EPI_SWIGLU_FWD = 1, EPI_SWIGLU_BWD = 2 };
enum { G_FULL = 0, G_EMPTY = kStages, G_ACCFULL = 2 * kStages, G_ACCEMPTY = 2 * kStages + 2, G_COUNT = 2 * kStages + 4 };
enum { GERR_EMPTY = 0x301, GERR_FULL = 0x302, GERR_ACCFULL = 0x303, GERR_ACCEMPTY = 0x304 };

struct GemmEpi {
    __nv_bfloat16 *c0;          // STORE: C.  FWD: a.  BWD: da
    __nv_bfloat16 *c1;          // FWD: u.  BWD: du
    __nv_bfloat16 *c2;          // FWD: h
    const __nv_bfloat16 *a;     // BWD: stored a
    const __nv_bfloat16 *u;     // BWD: stored u
    int ldc;                    // row length of every array above
};

__device__ __forceinline__ void store8(__nv_bfloat16 *p, const float *f)
{
    uint4 v;
    v.x = pack_bf16(f[0], f[1]);
    v.y = pack_bf16(f[2], f[3]);
    v.z = pack_bf16(f[4], f[5]);
    v.w = pack_bf16(f[6], f[7]);
    *reinterpret_cast<uint4 *>(p) = v;
}
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
__device__ __forceinline__ float sigmoidf_fast(float a) { return __frcp_rn(1.f + __expf(-a)); }

// Tile order: groups of 8 tile rows, column-major inside a group, so that the CTAs running at the
// same time share a few A row blocks and a few B column blocks.
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int &tm, int &tn)
{
    constexpr int kGroup = 8;
    const int per_group = kGroup * tiles_n;
    const int g = t / per_group, r = t - g * per_group;
    const int rows = min(kGroup, tiles_m - g * kGroup);
    tn = r / rows;
    tm = g * kGroup + (r - tn * rows);
}

template <bool kAMn, bool kBMn, int kEpi>
__global__ void __launch_bounds__(kGemmThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap mapA0, const __grid_constant__ CUtensorMap mapB0,
               const __grid_constant__ CUtensorMap mapA1, const __grid_constant__ CUtensorMap mapB1,
               GemmEpi epi, int M, int N, int K, int nparts, int nbatch, unsigned int *status)
{
    constexpr bool kDualN = kEpi == EPI_SWIGLU_FWD;         // B tile = 128 rows of map B0 + 128 rows of map B1
    constexpr int kTileN = kDualN ? 128 : GN;                // output columns a tile covers
    // Epilogue warps: two per 32-lane group (one column half each), except in the forward gate epilogue,
    // where eight warps of stores and exponentials measured 13 % slower than four
    constexpr int kEpiWarps = kEpi == EPI_SWIGLU_FWD ? 4 : 8;
    constexpr int kHalfCols = (kDualN ? 128 : GN) / (kEpiWarps / 4);
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(sm + kStages * kStageBytes);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + G_COUNT);
    volatile uint32_t *abortp = tmem_slot + 1;
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;

    const int tiles_m = (M + GM - 1) / GM, tiles_n = (N + kTileN - 1) / kTileN;
    // nbatch = 2: two independent products of one shape in one launch (A1 B1^T -> epi.c1 after A0 B0^T ->
    // epi.c0), so that their tiles share the waves of the persistent grid
    const int tiles_one = tiles_m * tiles_n, tiles = tiles_one * nbatch;
    const int nk = (K + GK - 1) / GK, nk_total = nk * nparts;

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(bars + G_FULL + i, 1);
            mbar_init(bars + G_EMPTY + i, 1);
        }
        mbar_init(bars + G_ACCFULL + 0, 1);
        mbar_init(bars + G_ACCFULL + 1, 1);
        mbar_init(bars + G_ACCEMPTY + 0, 32 * kEpiWarps);
        mbar_init(bars + G_ACCEMPTY + 1, 32 * kEpiWarps);
        *abortp = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_slot;

    if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------------ TMA producer
        prefetch_tensormap(&mapA0);
        prefetch_tensormap(&mapB0);
        int it = 0;
        bool ok = true;
        for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x) {
            int tm, tn;
            const int second = t >= tiles_one ? 1 : 0;
            tile_coords(t - second * tiles_one, tiles_m, tiles_n, tm, tn);
            const int m0 = tm * GM, n0 = tn * kTileN;
            for (int ks = 0; ks < nk_total; ++ks, ++it) {
                const int s = it % kStages;
                if (!mbar_wait(bars + G_EMPTY + s, ((it / kStages) & 1) ^ 1, abortp, status, GERR_EMPTY)) { ok = false; break; }
                const int part = ks / nk, k0 = (ks - part * nk) * GK;
                const CUtensorMap *ma = (part || second) ? &mapA1 : &mapA0;
                const CUtensorMap *mb = ((part || second) && !kDualN) ? &mapB1 : &mapB0;
                uint8_t *sa = sm + s * kStageBytes, *sb = sa + kABytes;
                uint64_t *full = bars + G_FULL + s;
                mbar_arrive_expect_tx(full, kStageBytes);
                if (kAMn) {
                    tma_load_3d(sa, ma, full, m0, k0, 0);
                    tma_load_3d(sa + kMnBox, ma, full, m0 + 64, k0, 0);
                } else {
                    tma_load_3d(sa, ma, full, k0, m0, 0);
                }
                if (kBMn) {
#pragma unroll
                    for (int b = 0; b < 4; ++b) tma_load_3d(sb + b * kMnBox, mb, full, n0 + 64 * b, k0, 0);
                } else if (kDualN) {
                    tma_load_3d(sb, &mapB0, full, k0, n0, 0);
                    tma_load_3d(sb + kBBytes / 2, &mapB1, full, k0, n0, 0);
                } else {
                    tma_load_3d(sb, mb, full, k0, n0, 0);
                }
            }
        }
    } else if (warp == 1 && lane == 0) {
        // ------------------------------------------------------------------- UMMA issuer
        constexpr uint32_t idesc = idesc_bf16_f32(GM, GN, kAMn ? 1 : 0, kBMn ? 1 : 0);
        const uint64_t km_proto = smem_desc_sw128(0, 16, 1024), mn_proto = smem_desc_sw128(0, kMnBox, 1024);
        const uint32_t a_hi = (uint32_t)((kAMn ? mn_proto : km_proto) >> 32), b_hi = (uint32_t)((kBMn ? mn_proto : km_proto) >> 32);
        const uint32_t a_lo0 = (uint32_t)(kAMn ? mn_proto : km_proto), b_lo0 = (uint32_t)(kBMn ? mn_proto : km_proto);
        constexpr uint32_t a_step = (kAMn ? 2048 : 32) >> 4, b_step = (kBMn ? 2048 : 32) >> 4;   // per 16 K-elements
        int it = 0, ti = 0;
        bool ok = true;
        for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++ti) {
            const int buf = ti & 1;
            if (!mbar_wait(bars + G_ACCEMPTY + buf, ((ti >> 1) & 1) ^ 1, abortp, status, GERR_ACCEMPTY)) break;
            tc_fence_after();
            const uint32_t acc = tbase + (uint32_t)(buf * GN);
            for (int ks = 0; ks < nk_total; ++ks, ++it) {
                const int s = it % kStages;
                if (!mbar_wait(bars + G_FULL + s, (it / kStages) & 1, abortp, status, GERR_FULL)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_lo = a_lo0 + ((smem_u32(sm + s * kStageBytes) >> 4) & 0x3FFFu);
                const uint32_t b_lo = b_lo0 + ((smem_u32(sm + s * kStageBytes + kABytes) >> 4) & 0x3FFFu);
                if (ks == 0) umma_ss2<false>(acc, a_lo, a_hi, b_lo, b_hi, idesc);
                else         umma_ss2<true>(acc, a_lo, a_hi, b_lo, b_hi, idesc);
#pragma unroll
                for (int q = 1; q < GK / 16; ++q)
                    umma_ss2<true>(acc, a_lo + q * a_step, a_hi, b_lo + q * b_step, b_hi, idesc);
                umma_commit(bars + G_EMPTY + s);          // the stage is free once these UMMAs have read it
            }
            if (ok) umma_commit(bars + G_ACCFULL + buf);
        }
    } else if (warp >= 2 && warp < 2 + kEpiWarps) {
        // ---------------------------------------------------------------------- epilogue
        const int lane_row = 32 * (warp % 4) + lane;               // TMEM lane = row of the tile
        const uint32_t lane_addr = tbase + ((uint32_t)(32 * (warp % 4)) << 16);
        const int half = (warp - 2) / 4;                           // which half of the tile's columns
        int ti = 0;
        for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++ti) {
            int tm, tn;
            const int second = t >= tiles_one ? 1 : 0;
            tile_coords(t - second * tiles_one, tiles_m, tiles_n, tm, tn);
            const int buf = ti & 1;
            const int row = tm * GM + lane_row, n0 = tn * kTileN;
            if (!mbar_wait(bars + G_ACCFULL + buf, (ti >> 1) & 1, abortp, status, GERR_ACCFULL)) break;
            tc_fence_after();
            const uint32_t acc = lane_addr + (uint32_t)(buf * GN);
            const size_t rbase = (size_t)row * epi.ldc;
            if (kEpi == EPI_SWIGLU_FWD) {
#pragma unroll 1
                for (int c = kHalfCols * half; c < kHalfCols * half + kHalfCols; c += 32) {
                    uint32_t ra[32], ru[32];
                    tmem_ld(acc + c, ra);
                    tmem_ld(acc + 128 + c, ru);
                    tc_wait_ld();
                    if (row < M) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            const int col = n0 + c + e;
                            if (col >= N) break;
                            float fa[8], fu[8], fh[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                fa[i] = __uint_as_float(ra[e + i]);
                                fu[i] = __uint_as_float(ru[e + i]);
                                fh[i] = fa[i] * sigmoidf_fast(fa[i]) * fu[i];
                            }
                            store8(epi.c0 + rbase + col, fa);
                            store8(epi.c1 + rbase + col, fu);
                            store8(epi.c2 + rbase + col, fh);
                        }
                    }
                }
            } else {
#pragma unroll 1
                for (int c = kHalfCols * half; c < kHalfCols * half + kHalfCols; c += 32) {
                    // the stored a, u of this chunk are requested before the accumulator is read
                    uint4 va[4], vu[4];
                    if (kEpi == EPI_SWIGLU_BWD && row < M) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int col = n0 + c + 8 * q;
                            if (col < N) {
                                va[q] = __ldg(reinterpret_cast<const uint4 *>(epi.a + rbase + col));
                                vu[q] = __ldg(reinterpret_cast<const uint4 *>(epi.u + rbase + col));
                            }
                        }
                    }
                    uint32_t r[32];
                    tmem_ld(acc + c, r);
                    tc_wait_ld();
                    if (row < M) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            const int col = n0 + c + e;
                            if (col >= N) break;
                            float f[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(r[e + i]);
                            if (kEpi == EPI_STORE) {
                                store8((second ? epi.c1 : epi.c0) + rbase + col, f);
                            } else {
                                float fa[8], fu[8], da[8], du[8];
                                unpack8(va[e / 8], fa);
                                unpack8(vu[e / 8], fu);
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const float sg = sigmoidf_fast(fa[i]);
                                    da[i] = f[i] * fu[i] * sg * (1.f + fa[i] * (1.f - sg));
                                    du[i] = f[i] * fa[i] * sg;
                                }
                                store8(epi.c0 + rbase + col, da);
                                store8(epi.c1 + rbase + col, du);
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bars + G_ACCEMPTY + buf);       // this thread has read its lanes of the accumulator
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tbase, 512);
}

struct Operand {
    const void *p;
    int rows, cols;          // the array as stored: [rows, cols] row-major
};

// K-major: stored [MN, K], box of `box_rows` rows x 64 K-elements.  MN-major: stored [K, MN], box of 64 x 64.
bool operand_map(CUtensorMap *m, const Operand &o, bool mn_major, int box_rows)
{
    return make_tensor_map_3d(m, o.p, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 1, (uint64_t)o.rows, (uint64_t)o.cols,
                              mn_major ? 64 : (uint32_t)box_rows, 64);
}

template <bool kAMn, bool kBMn, int kEpi>
cudaError_t launch_gemm(const Operand &A0, const Operand &B0, const Operand *A1, const Operand *B1, const GemmEpi &epi,
                        int M, int N, int K, cudaStream_t st, int nbatch = 1)
{
    constexpr bool kDualN = kEpi == EPI_SWIGLU_FWD;
    CUtensorMap ma0, mb0, ma1, mb1;
    const int b_rows = kDualN ? 128 : GN;
    if (!operand_map(&ma0, A0, kAMn, GM) || !operand_map(&mb0, B0, kBMn, b_rows)) return cudaErrorInvalidValue;
    if (!operand_map(&ma1, A1 ? *A1 : A0, kAMn, GM) || !operand_map(&mb1, B1 ? *B1 : B0, kBMn, b_rows))
        return cudaErrorInvalidValue;
    auto kernel = tc_gemm_kernel<kAMn, kBMn, kEpi>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
    if (e != cudaSuccess) return e;
    const int tiles = ((M + GM - 1) / GM) * ((N + (kDualN ? 128 : GN) - 1) / (kDualN ? 128 : GN)) * nbatch;
    const int nparts = (A1 && !kDualN && nbatch == 1) ? 2 : 1;
    LaunchScope scope(MOA_KERNEL_OTHER, st);
    kernel<<<tiles < 148 ? tiles : 148, kGemmThreads, kGemmSmem, st>>>(ma0, mb0, ma1, mb1, epi, M, N, K, nparts,
                                                                      nbatch, device_status_ptr());
    return cudaGetLastError();
}

}  // namespace

cudaError_t gated_mlp_fwd(int n, int d, int dff, const void *x, const void *W1, const void *W3, const void *W2,
                          void *a, void *u, void *h, void *y, cudaStream_t st)
{
    // a | u = x [W1; W3]^T with the gate in the epilogue, then y = h W2^T
    const Operand X{x, n, d}, w1{W1, dff, d}, w3{W3, dff, d}, Hh{h, n, dff}, w2{W2, d, dff};
    GemmEpi e1{(__nv_bfloat16 *)a, (__nv_bfloat16 *)u, (__nv_bfloat16 *)h, nullptr, nullptr, dff};
    cudaError_t e = launch_gemm<false, false, EPI_SWIGLU_FWD>(X, w1, nullptr, &w3, e1, n, dff, d, st);
    if (e != cudaSuccess) return e;
    GemmEpi e2{(__nv_bfloat16 *)y, nullptr, nullptr, nullptr, nullptr, d};
    return launch_gemm<false, false, EPI_STORE>(Hh, w2, nullptr, nullptr, e2, n, d, dff, st);
}

cudaError_t gated_mlp_bwd(int n, int d, int dff, const void *x, const void *W1, const void *W3, const void *W2,
                          const void *a, const void *u, const void *h, const void *dy, void *da, void *du,
                          void *dx, void *dW1, void *dW3, void *dW2, cudaStream_t st)
{
    const Operand X{x, n, d}, w1{W1, dff, d}, w3{W3, dff, d}, w2{W2, d, dff}, Hh{h, n, dff}, DY{dy, n, d};
    const Operand DA{da, n, dff}, DU{du, n, dff};
    // dh = dy W2 (W2 [d,d_ff] read as the MN-major B operand), gate backward in the epilogue -> da, du
    GemmEpi e3{(__nv_bfloat16 *)da, (__nv_bfloat16 *)du, nullptr, (const __nv_bfloat16 *)a, (const __nv_bfloat16 *)u, dff};
    cudaError_t e = launch_gemm<false, true, EPI_SWIGLU_BWD>(DY, w2, nullptr, nullptr, e3, n, dff, d, st);
    if (e != cudaSuccess) return e;
    // dW2 [d,d_ff] = dy^T h: both operands read transposed (K = tokens)
    GemmEpi e4{(__nv_bfloat16 *)dW2, nullptr, nullptr, nullptr, nullptr, dff};
    if ((e = launch_gemm<true, true, EPI_STORE>(DY, Hh, nullptr, nullptr, e4, d, dff, n, st)) != cudaSuccess) return e;
    // dW1 = da^T x, dW3 = du^T x   [d_ff,d]: one launch, so that the two tile sets fill the waves together
    GemmEpi e5{(__nv_bfloat16 *)dW1, (__nv_bfloat16 *)dW3, nullptr, nullptr, nullptr, d};
    if ((e = launch_gemm<true, true, EPI_STORE>(DA, X, &DU, &X, e5, dff, d, n, st, 2)) != cudaSuccess) return e;
    // dx = da W1 + du W3: two operand pairs accumulate into one tile (W1, W3 [d_ff,d] as MN-major B)
    GemmEpi e7{(__nv_bfloat16 *)dx, nullptr, nullptr, nullptr, nullptr, d};
    return launch_gemm<false, true, EPI_STORE>(DA, w1, &DU, &w3, e7, n, d, dff, st);
}

}  // namespace moa
