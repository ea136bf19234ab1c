// Forward attention on the sm_100a tensor cores (tcgen05 + TMEM + TMA), bf16 in,
// fp32 accumulate.
//
// One CTA owns 128 query rows of one (batch, head) and walks the key/value tiles of
// 128 keys.  Roles (192 threads):
//   warps 0-3  softmax: thread t owns query row t = TMEM lane t.  Reads the fp32 score
//              tile S from TMEM, keeps the running row max / row sum, writes the bf16
//              probabilities P back into TMEM (over the first half of S), rescales the
//              O accumulator in TMEM when the row max has grown, and writes O and the
//              logsumexp L at the end.
//   warp 4     TMA producer: Q once, then K and V tiles into single buffers that are
//              refilled as soon as the UMMA that read them has completed.
//   warp 5     UMMA issuer: S = Q K^T (both operands K-major in shared memory), then
//              O += P V (P from TMEM, V MN-major in shared memory).  Owns the TMEM
//              allocation.
// S, P and the O accumulator never leave the SM: nothing of size n x n reaches HBM.
// Two CTAs fit on one SM (256 TMEM columns and at most 97 KB shared memory each), so
// one CTA's softmax overlaps the other's UMMAs.
//
// The running max is lazy: O and the row sum are rescaled only when the new tile's max
// exceeds the max in use by more than 8 (a factor 256 in P), which leaves the result
// unchanged mathematically and keeps P well inside bf16/fp32 range.
#include "common.cuh"
#include "ptx.cuh"
#include "tensormap.cuh"

namespace moa {
namespace {

using namespace ptx;

constexpr int BM = 128;            // query rows per CTA
constexpr int BN = 128;            // keys per tile
constexpr int kThreads = 192;
constexpr int kTmemCols = 256;     // S: columns [0,128), O: [128,128+D)
constexpr uint32_t kColS = 0, kColP = 0, kColO = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;

enum : uint32_t { ERR_Q = 0x101, ERR_K = 0x102, ERR_V = 0x103, ERR_S = 0x104, ERR_P = 0x105, ERR_O = 0x106 };

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
tc_fwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
              const __grid_constant__ CUtensorMap mapV, __nv_bfloat16 *__restrict__ O, float *__restrict__ L,
              int n, int causal, float scale_log2, int nqt, unsigned int *status)
{
    constexpr int kTileBytes = 128 * D * 2;
    constexpr int kBoxes = D / 64;         // 64-column (128-byte) swizzled boxes per tile
    constexpr int kBoxBytes = 128 * 128;   // 128 rows x 128 bytes
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sQ = sm, *sK = sm + kTileBytes, *sV = sm + 2 * kTileBytes;
    __shared__ uint64_t bar_q, bar_k, bar_v, bar_s, bar_p, bar_o;
    __shared__ uint32_t tmem_base_s;
    __shared__ uint32_t abort_flag;

    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int bh = blockIdx.x / nqt;
    const int t = blockIdx.x % nqt;
    const int qt = causal ? nqt - 1 - t : t;   // causal: longest rows first
    const int q0 = qt * BM;
    const int nkt_all = (n + BN - 1) / BN;
    const int nkt = causal ? min(qt + 1, nkt_all) : nkt_all;

    if (tid == 0) {
        mbar_init(&bar_q, 1); mbar_init(&bar_k, 1); mbar_init(&bar_v, 1);
        mbar_init(&bar_s, 1); mbar_init(&bar_p, 128); mbar_init(&bar_o, 1);
        abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV);
    }
    if (warp == 5) { tmem_alloc(&tmem_base_s, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = tmem_base_s;
    volatile uint32_t *abortp = &abort_flag;

    if (warp == 4) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_arrive_expect_tx(&bar_q, kTileBytes);
            for (int b = 0; b < kBoxes; ++b) tma_load_3d(sQ + b * kBoxBytes, &mapQ, &bar_q, 64 * b, q0, bh);
        }
        for (int j = 0; j < nkt; ++j) {
            if (j > 0 && !mbar_wait(&bar_s, (j - 1) & 1, abortp, status, ERR_S)) break;   // K buffer free
            if (lane == 0) {
                mbar_arrive_expect_tx(&bar_k, kTileBytes);
                for (int b = 0; b < kBoxes; ++b) tma_load_3d(sK + b * kBoxBytes, &mapK, &bar_k, 64 * b, j * BN, bh);
            }
            if (j > 0 && !mbar_wait(&bar_o, (j - 1) & 1, abortp, status, ERR_O)) break;   // V buffer free
            if (lane == 0) {
                mbar_arrive_expect_tx(&bar_v, kTileBytes);
                for (int b = 0; b < kBoxes; ++b) tma_load_3d(sV + b * kBoxBytes, &mapV, &bar_v, 64 * b, j * BN, bh);
            }
            __syncwarp();
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------- UMMA issuer
        constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);
        constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, 0, 1);
        // Descriptors are built once; inside the loops only a constant is added to the address
        // field (the issuing thread's instruction stream must stay far shorter than the 64 cycles
        // one 128x128x16 UMMA takes, or the tensor pipe starves).
        const uint64_t q_desc = smem_desc_sw128(smem_u32(sQ), 16, 1024);
        const uint64_t k_desc = smem_desc_sw128(smem_u32(sK), 16, 1024);
        const uint64_t v_desc = smem_desc_sw128(smem_u32(sV), kBoxBytes, 1024);   // MN-major
        const uint32_t q_lo = (uint32_t)q_desc, k_lo = (uint32_t)k_desc, v_lo = (uint32_t)v_desc;
        const uint32_t km_hi = (uint32_t)(q_desc >> 32), mn_hi = (uint32_t)(v_desc >> 32);
        bool ok = mbar_wait(&bar_q, 0, abortp, status, ERR_Q);
        for (int j = 0; ok && j < nkt; ++j) {
            if (!mbar_wait(&bar_k, j & 1, abortp, status, ERR_K)) break;
            tc_fence_after();
            if (lane == 0) {
                umma_ss2<false>(tbase + kColS, q_lo, km_hi, k_lo, km_hi, idesc_s);
#pragma unroll
                for (int ks = 1; ks < D / 16; ++ks) {
                    const uint32_t off = (uint32_t)(((ks / 4) * kBoxBytes + (ks % 4) * 32) >> 4);
                    umma_ss2<true>(tbase + kColS, q_lo + off, km_hi, k_lo + off, km_hi, idesc_s);
                }
                umma_commit(&bar_s);
            }
            __syncwarp();
            if (!mbar_wait(&bar_v, j & 1, abortp, status, ERR_V)) break;
            if (!mbar_wait(&bar_p, j & 1, abortp, status, ERR_P)) break;
            tc_fence_after();
            if (lane == 0) {
                if (j > 0) umma_ts2<true>(tbase + kColO, tbase + kColP, v_lo, mn_hi, idesc_pv);
                else       umma_ts2<false>(tbase + kColO, tbase + kColP, v_lo, mn_hi, idesc_pv);
#pragma unroll
                for (int ks = 1; ks < BN / 16; ++ks)
                    umma_ts2<true>(tbase + kColO, tbase + kColP + ks * 8, v_lo + (uint32_t)((ks * 2048) >> 4), mn_hi, idesc_pv);
                umma_commit(&bar_o);
            }
            __syncwarp();
        }
    } else {
        // ---------------------------------------------------------------- softmax warps
        const int row = q0 + tid;
        const uint32_t lane_addr = tbase + ((uint32_t)(warp * 32) << 16);
        float m_used = 0.f, l = 0.f;
        bool ok = true;
        for (int j = 0; j < nkt; ++j) {
            if (!mbar_wait(&bar_s, j & 1, abortp, status, ERR_S)) { ok = false; break; }
            tc_fence_after();
            const int k0 = j * BN;
            const bool need_mask = (k0 + BN > n) || (causal && k0 + BN - 1 > q0);
            // The whole score row (128 fp32) comes into registers with one round trip to TMEM.
            uint32_t r[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld(lane_addr + kColS + 32 * c, r[c]);
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
            // row max of the raw scores (scale_log2 > 0, so scaling commutes with max); 3-input max
            float mx4[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float a = fmaxf(__uint_as_float(r[c][0]), __uint_as_float(r[c][1]));
#pragma unroll
                for (int i = 2; i < 32; i += 2) a = fmax3(a, __uint_as_float(r[c][i]), __uint_as_float(r[c][i + 1]));
                mx4[c] = a;
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2;
            if (j == 0) {
                m_used = (mx == -INFINITY) ? 0.f : mx;
            } else {
                const bool grow = mx > m_used + kRescaleThreshold;
                if (__any_sync(0xffffffffu, grow)) {
                    // all UMMAs issued before S(j), PV(j-1) included, have completed: O is stable
                    const float alpha = grow ? ex2(m_used - mx) : 1.f;
                    if (grow) m_used = mx;
                    l *= alpha;
                    // rare path, kept small: the 128 score registers stay live across it
#pragma unroll 1
                    for (int c = 0; c < D; c += 8) {
                        uint32_t o[8];
                        tmem_ld(lane_addr + kColO + c, o);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 8; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st(lane_addr + kColO + c, o);
                    }
                }
            }
            // P = 2^(s scale_log2 - m_used), row sum, bf16 P into TMEM over the first 64 of the S
            // columns.  Arithmetic runs on fp32 pairs (f32x2) to halve the instruction count.
            const uint64_t sl2 = pack_f32x2(scale_log2, scale_log2);
            const uint64_t negm2 = pack_f32x2(-m_used, -m_used);
            uint64_t ls2[2] = {0ull, 0ull};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const uint64_t t = fma_f32x2(pack_f32x2(__uint_as_float(r[c][i]), __uint_as_float(r[c][i + 1])), sl2, negm2);
                    float p0, p1;
                    unpack_f32x2(t, p0, p1);
                    p0 = ex2(p0);
                    p1 = ex2(p1);
                    ls2[(i >> 1) & 1] = add_f32x2(ls2[(i >> 1) & 1], pack_f32x2(p0, p1));
                    pk[i / 2] = pack_bf16(p0, p1);
                }
                tmem_st(lane_addr + kColP + 16 * c, pk);
            }
            {
                float s0, s1, s2, s3;
                unpack_f32x2(ls2[0], s0, s1);
                unpack_f32x2(ls2[1], s2, s3);
                l += (s0 + s1) + (s2 + s3);
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(&bar_p);
        }
        if (ok && mbar_wait(&bar_o, (nkt - 1) & 1, abortp, status, ERR_O)) {
            tc_fence_after();
            const float inv = 1.f / l;
            __nv_bfloat16 *orow = O + ((size_t)bh * n + row) * D;
#pragma unroll
            for (int c = 0; c < D; c += 32) {
                uint32_t r[32];
                tmem_ld(lane_addr + kColO + c, r);
                tc_wait_ld();
                if (row < n) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(r[i + 0]) * inv, __uint_as_float(r[i + 1]) * inv);
                        v.y = pack_bf16(__uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
                        v.z = pack_bf16(__uint_as_float(r[i + 4]) * inv, __uint_as_float(r[i + 5]) * inv);
                        v.w = pack_bf16(__uint_as_float(r[i + 6]) * inv, __uint_as_float(r[i + 7]) * inv);
                        *reinterpret_cast<uint4 *>(orow + c + i) = v;
                    }
                }
            }
            if (row < n) L[(size_t)bh * n + row] = m_used * kLn2 + logf(l);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) tmem_dealloc(tbase, kTmemCols);
}

template <int D>
cudaError_t launch_fwd(const Problem &p, const void *Q, const void *K, const void *V, void *O, float *L,
                       cudaStream_t st)
{
    constexpr int kSmem = 3 * 128 * D * 2 + 1024;
    CUtensorMap mq, mk, mv;
    const uint64_t heads = (uint64_t)p.BH();
    if (!make_tensor_map_3d(&mq, Q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64) ||
        !make_tensor_map_3d(&mk, K, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64) ||
        !make_tensor_map_3d(&mv, V, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads, p.n, D, 128, 64))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(tc_fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const int nqt = (p.n + BM - 1) / BM;
    LaunchScope scope(MOA_KERNEL_FWD, st);
    tc_fwd_kernel<D><<<(unsigned)(nqt * p.BH()), kThreads, kSmem, st>>>(
        mq, mk, mv, (__nv_bfloat16 *)O, L, p.n, p.causal, p.scale * kLog2e, nqt, device_status_ptr());
    return cudaGetLastError();
}

}  // namespace

cudaError_t tc_fwd(const Problem &p, const void *Q, const void *K, const void *V, void *O, float *L, cudaStream_t st)
{
    if (p.d == 64) return launch_fwd<64>(p, Q, K, V, O, L, st);
    if (p.d == 128) return launch_fwd<128>(p, Q, K, V, O, L, st);
    return cudaErrorInvalidValue;
}

}  // namespace moa
