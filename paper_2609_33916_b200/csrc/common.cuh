// Shared declarations of the CUDA library's translation units (internal; the
// public interface is include/moa_attn.h).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "moa_attn.h"

namespace moa {

// Where element (b, h, row, 0) of one of the caller's tensors lives: b * batch + h * head + row * row elements past
// its base pointer (the d elements of a row are contiguous).
struct Strides {
    long long row, head, batch;
    __host__ __device__ size_t at(long long b, long long h, long long r) const { return (size_t)(b * batch + h * head + r * row); }
};

struct Problem {
    int B, H, n, d;
    int causal;
    float scale;
    int Hkv = 0;                                   // key/value heads; 0: same as H
    int bnhd = 0;                                  // 1: the caller's tensors are [B,n,H,d] in memory (L stays [B,H,n])
    // strides of the three tensor classes: Q, dQ | K, V, dK, dV | O, dO.  Filled by with_layout() from the fixed
    // layouts, or taken from the descriptor (MOA_LAYOUT_STRIDED).
    Strides sq{0, 0, 0}, skv{0, 0, 0}, so{0, 0, 0};
    Problem &with_layout()
    {
        const long long hk = kv_heads();
        if (bnhd) {
            sq = so = Strides{(long long)H * d, d, (long long)n * H * d};
            skv = Strides{hk * d, d, (long long)n * hk * d};
        } else {
            sq = so = Strides{d, (long long)n * d, (long long)H * n * d};
            skv = Strides{d, (long long)n * d, hk * n * d};
        }
        return *this;
    }
    bool contiguous_bhnd() const     // every tensor is a plain [B,heads,n,d] array
    {
        return sq.row == d && sq.head == (long long)n * d && sq.batch == (long long)H * n * d && so.row == sq.row &&
               so.head == sq.head && so.batch == sq.batch;
    }
    int BH() const { return B * H; }
    int kv_heads() const { return Hkv > 0 ? Hkv : H; }
    int group() const { return H / kv_heads(); }    // query heads per key/value head
    int BHkv() const { return B * kv_heads(); }
};

// Head dimension the tensor-core kernels are compiled for: a head of d columns (a multiple of 8, so
// that rows stay 16-byte aligned) runs in the 64-, 128- or 256-column kernels; the TMA loads fill the
// columns past d with zeros and the TMA stores drop them, which leaves every result unchanged.
// 256: the two-pass kernels for head dimensions 136..256 (tc_fwd.cu with KC = 2, tc_bwd_wide.cu).
inline int kernel_d(int d) { return d <= 64 ? 64 : d <= 128 ? 128 : 256; }

// Block order of the tile-parallel kernels.  Heads are taken in groups of `hpg`; inside a group
// the blocks go tile-major (every head's tile 0, then every head's tile 1, ...).  With causal
// masking tile t is the t-th longest job, so the hardware's in-order block dispatch becomes
// longest-job-first inside a group and the last blocks to start are the shortest: head-major
// order left SMs idle for ~12 % of a causal backward, waiting for long jobs that started late.
// hpg = 1 is head-major order (best L2 locality), used whenever all jobs have the same length.
__device__ __forceinline__ void job_from_block(int block, int tiles, int heads, int hpg, int &bh, int &t)
{
    const int per_group = hpg * tiles;
    const int group = block / per_group, r = block - group * per_group;
    const int cur = min(hpg, heads - group * hpg);
    t = r / cur;
    bh = group * hpg + (r - t * cur);
}

// What the launch arithmetic needs to know about the current device, read once per device
// (cudaDevAttrMultiProcessorCount, cudaDevAttrL2CacheSize); a B200 gives 148 SMs and 126 MB.
struct DeviceInfo {
    int sms;             // streaming multiprocessors
    long long l2_bytes;  // L2 cache
};
const DeviceInfo &device_info();

// Heads per group: enough jobs per group that its longest job (tiles iterations) is shorter than
// the group's share of the SMs, and as many heads as keep Q, K, V, dO of a group within half of L2.
inline int heads_per_group(const Problem &p, int tiles)
{
    if (!p.causal) return 1;
    const DeviceInfo &dev = device_info();
    const long long per_head = 4LL * p.n * p.d * 2;
    const long long fit = (dev.l2_bytes / 2 + per_head / 2) / (per_head > 0 ? per_head : 1);     // to the nearest head
    long long g = (2 * dev.sms + tiles) / (tiles + 1);
    if (fit > g) g = fit;
    if (g < 1) g = 1;
    if (g > p.BH()) g = p.BH();
    const long long groups = (p.BH() + g - 1) / g;      // groups of equal size (to within one head)
    g = (p.BH() + groups - 1) / groups;
    return (int)g;
}

// Decode through the tensor-core forward kernel (tc_fwd.cu): the G query heads of a K/V head are
// the rows of one query tile, the cache is split among CTAs; partial results to be merged.
cudaError_t tc_fwd_decode(int B, int Hkv, int G, int n, int d, float scale, const void *q, const void *K, const void *V,
                          void *O_part, float *L_part, int splits, int tiles_per_split, cudaStream_t st);

// ---- decode attention (decode.cu) ----------------------------------------------------
struct DecodeProblem {
    int B, H, Hkv, n, d;     // Hkv resolved (never 0)
    float scale;
};
int decode_splits(const DecodeProblem &p);                            // cache segments per K/V head (CUDA-core route)
size_t decode_workspace_bytes(const DecodeProblem &p, int dtype);    // partial results of all segments
// q [B,H,d], K, V [B,Hkv,n,d] -> out [B,H,d] (dtype of the inputs), lse [B,H] fp32 (may be null)
cudaError_t decode_attn(const DecodeProblem &p, int dtype, const void *q, const void *K, const void *V, void *out,
                        float *lse, void *ws, cudaStream_t st);

// Host-side launch counter (moa_launch_count).
void count_launch(int k = 1);

// Brackets one kernel launch with an event pair when profiling is enabled
// (moa_profile_enable); also counts the launch.
struct LaunchScope {
    LaunchScope(int kind, cudaStream_t st);
    ~LaunchScope();
    int slot;
    cudaStream_t st;
};

// Launch `kernel` so that it may start before the kernel in front of it in the stream has finished (programmatic
// dependent launch): the kernel itself calls ptx::grid_dependency_wait() before it touches anything that kernel
// wrote.  MOA_PDL=0 in the environment turns the attribute off (plain stream order).
bool pdl_enabled();
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Device address of the status word kernels write when a bounded wait expires.
unsigned int *device_status_ptr();

// MOA_OK when the current device is compute capability 10.x, MOA_ERR_ARCH otherwise (cached per device).
moa_status check_device_arch();

// ---- block pieces (block_norm.cu, tc_gemm.cu), bf16 ------------------------------------
size_t rmsnorm_workspace_bytes(int n, int d);          // per-CTA partial sums of dg
cudaError_t rmsnorm_fwd(int n, int d, float eps, const void *x, const void *g, void *y, float *r, cudaStream_t st);
// dx_add (may be null): dx = (RMSNorm backward) + dx_add
cudaError_t rmsnorm_bwd(int n, int d, float eps, const void *x, const void *g, const float *r, const void *dy,
                        const void *dx_add, void *dx, void *dg, void *ws, cudaStream_t st);
// gated MLP (tc_gemm.cu): x, y, dy, dx [n,d]; W1, W3 [d_ff,d]; W2 [d,d_ff]; a, u, h, da, du [n,d_ff]
// res (may be null): y = h W2^T + res
cudaError_t gated_mlp_fwd(int n, int d, int dff, const void *x, const void *W1, const void *W3, const void *W2,
                          const void *res, void *a, void *u, void *h, void *y, cudaStream_t st);
// C[M,N] = A B^T (+ R): A given as [M,K] (a_mn = 0) or [K,M] (a_mn = 1), B as [N,K] (b_mn = 0) or [K,N] (b_mn = 1); bf16
cudaError_t gemm_bf16(int a_mn, int b_mn, int M, int N, int K, const void *A, const void *B, const void *R, void *C,
                      cudaStream_t st);
cudaError_t gated_mlp_bwd(int n, int d, int dff, const void *x, const void *W1, const void *W3, const void *W2,
                          const void *a, const void *u, const void *h, const void *dy, void *da, void *du,
                          void *dx, void *dW1, void *dW3, void *dW2, cudaStream_t st);

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ---- tensor-core path (tc_fwd.cu), bf16 only ---------------------------------------------
// What the forward of a fused call does for its backward (all null for a plain forward): it clears the fp32
// dQ accumulator [B*H, n, kernel_d(d)], and writes the backward's per-row inputs -L log2 e and -D = -rowsum(dO o O)
// (from the fp32 O it holds), padded to n_pad rows per head with -inf / 0.
struct FwdForBwd {
    float *zero_acc = nullptr;
    const void *dO = nullptr;
    float *Lp = nullptr, *Dp = nullptr;
};
cudaError_t tc_fwd(const Problem &p, const void *Q, const void *K, const void *V, void *O, float *L,
                   const FwdForBwd &fb, cudaStream_t st);

// Lp = -L*log2(e) and Dp = -rowsum(dO o O) (negated: fma/add operands), each padded per head to a
// multiple of 128 rows (-inf / 0 past n)
cudaError_t tc_bwd_preprocess(const Problem &p, const void *dO, const void *O, const float *L, float *Lp, float *Dp,
                              cudaStream_t st);
// dK, dV; UNSCALED dQ contributions (dS K, without the factor scale) red-added into dQacc
// (fp32 [B,H,n,kernel_d(d)], pre-zeroed); dQacc == nullptr skips the dQ contraction altogether
cudaError_t tc_bwd_kv(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                      const float *Lp, const float *Dp, void *dK, void *dV, float *dQacc, int dq_bulk,
                      cudaStream_t st);   // dq_bulk: TMA bulk add-reduce instead of red.global (d = 128 only)

// The same on pairs of CTAs (tc_bwd_pair.cu; the 128-column kernel only), and whether tc_bwd_kv hands such
// problems to it (moa_bwd_pair_mode; environment variable MOA_BWD_PAIR=1 for the initial mode; default: no)
cudaError_t tc_bwd_kv_pair(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                           const float *Lp, const float *Dp, void *dK, void *dV, float *dQacc, int dq_bulk,
                           cudaStream_t st);
bool bwd_pair_enabled();
int bwd_pair_mode(int set);      // set < 0: query; returns the mode in force before the call

// Head dimensions 136..256 (tc_bwd_wide.cu): tiles of 128 keys x 64 queries, two passes over the halves of d; dQ by
// red.global into dQacc (fp32 [B,H,n,256], pre-zeroed)
cudaError_t tc_bwd_kv_wide(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                           const float *Lp, const float *Dp, void *dK, void *dV, float *dQacc, cudaStream_t st);

// atomic-free query-parallel dQ pass on the tensor cores (tc_dq.cu); writes dQ (bf16) directly
cudaError_t tc_bwd_dq(const Problem &p, const void *Q, const void *K, const void *V, const void *dO,
                      const float *Lp, const float *Dp, void *dQ, cudaStream_t st);

// ---- n x n-materialising comparison variant (tc_materialize.cu), bf16 --------------------
// P^T and dS^T are [heads][n_pad][n_pad] bf16 arrays in the caller's workspace.
cudaError_t mat_fwd(const Problem &p, const void *Q, const void *K, const void *V, void *O, float *L, void *PT,
                    cudaStream_t st);
cudaError_t mat_bwd(const Problem &p, const void *Q, const void *K, const void *V, const void *dO, const float *Dp,
                    const void *PT, void *GST, void *dQ, void *dK, void *dV, cudaStream_t st);

// ---- SIMT fp32 path (simt_kernels.cu) -------------------------------------------------
// dtype: MOA_BF16 or MOA_F32 storage; arithmetic is fp32 FMA throughout.
cudaError_t simt_fwd(const Problem &p, int dtype, const void *Q, const void *K, const void *V,
                     void *O, float *L, cudaStream_t st);
// D_i = sum_k dO_ik O_ik
cudaError_t row_dot(const Problem &p, int dtype, const void *dO, const void *O, float *Dv, cudaStream_t st);
// dK, dV always; dQ contributions are atomically added into dQacc (fp32 [B,H,n,d], pre-zeroed)
// when dQacc != nullptr.
cudaError_t simt_bwd_kv(const Problem &p, int dtype, const void *Q, const void *K, const void *V,
                        const void *dO, const float *L, const float *Dv,
                        void *dK, void *dV, float *dQacc, cudaStream_t st);
// atomic-free query-parallel dQ pass
// Row-parallel fused forward+backward in one kernel with dK (sites = 1) or dK and dV (sites = 2)
// accumulated by fp32 atomics into dKacc / dVacc [B*H, n, d]; writes O, L, D, dQ.
cudaError_t simt_rowpar(const Problem &p, int dtype, const void *Q, const void *K, const void *V, const void *dO,
                        void *O, float *L, float *Dv, void *dQ, float *dKacc, float *dVacc, int sites, cudaStream_t st);
cudaError_t simt_bwd_dq(const Problem &p, int dtype, const void *Q, const void *K, const void *V,
                        const void *dO, const float *L, const float *Dv, void *dQ, cudaStream_t st);
// dst[i] = (bf16)(mul * src[i])
cudaError_t convert_f32_to_bf16(const float *src, void *dst, size_t count, float mul, cudaStream_t st);
// the same row by row: the accumulator is [B*H, n, src_ld] (src_ld >= d: the kernels' padded head
// dimension), the destination addressed through the strides `ds` of the caller's dQ
cudaError_t convert_f32_to_bf16_rows(const float *src, int src_ld, void *dst, int B, int H, int n, int d, Strides ds,
                                     float mul, cudaStream_t st);

}  // namespace moa
