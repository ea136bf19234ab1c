/*
 * moa_attn.h -- C ABI of the B200 (sm_100a) fused attention forward+backward library.
 *
 * The operation.  For every (batch b, head h) pair independently, with
 * Q, K, V, dO in R^{n x d} and a scalar `scale`:
 *
 *     S = scale * Q K^T            (causal: S_ij = -inf for j > i; the diagonal is visible)
 *     P = rowsoftmax(S)            L_i = log sum_j exp(S_ij)      (natural log)
 *     O = P V
 *     dV = P^T dO      dP = dO V^T      D_i = sum_k dO_ik O_ik
 *     dS = P o (dP - D 1^T)        dQ = scale * dS K       dK = scale * dS^T Q
 *
 * These are the arrays the paper calls Q, K, V, Out, A (= P), GS (= dS), GQ, GK,
 * GV (Sec. 3 traffic table; Sec. 4 backward and fused kernels).  The paper's
 * point, and this library's contract, is that the fused path never stores the
 * n x n arrays A and GS in device memory (Sec. 1.1, the two-ONF figure): extra
 * memory is O(n d).  The paper's four-pass restructuring (Sec. 4, "the fix"),
 * one-writer-per-element passes instead of one monolithic kernel with atomics
 * on GV and GK, is kept: dK and dV are written without atomics by the CTA that
 * owns the key tile.  How dQ is accumulated is selectable (`dq_mode`), because
 * that step is where the paper's own regression (atomic contention) sat.
 *
 * Conventions common to every call
 *  - All tensor arguments are DEVICE pointers to contiguous [B,H,n,d] arrays,
 *    d fastest, 16-byte aligned; element type bfloat16 (MOA_BF16) or float
 *    (MOA_F32) per desc->dtype.  L is a DEVICE pointer to float [B,H,n].
 *  - The caller owns every buffer, workspace included.  The library never
 *    allocates or frees device memory.  What it keeps between calls is small and
 *    per process: a device status word (moa_last_device_status), the event records
 *    of moa_profile_*, a launch counter and per-device attribute caches.
 *  - Calls enqueue kernels on `stream` (a cudaStream_t passed as void*; NULL is
 *    the legacy default stream) and return without synchronising the host.
 *  - Outputs are overwritten, never accumulated into.
 *  - A call is one to four kernels in stream order.  The tensor-core backward kernel and the dQ conversion are
 *    launched as programmatic dependents of the kernel in front of them (they set themselves up while it drains and
 *    wait for its completion before reading or adding to anything it wrote); the first kernel of every call is an
 *    ordinary launch, so a call never starts before work the caller enqueued earlier has finished.  MOA_PDL=0 in the
 *    environment (read once per process) launches everything in plain stream order.
 *  - Errors are reported only through the returned moa_status; the library does
 *    not abort or throw.  Argument, workspace, scratch-limit and architecture errors
 *    are found before anything is enqueued.  MOA_ERR_CUDA can come from a later
 *    launch, clear or descriptor encode of a call that consists of several: kernels
 *    enqueued before it still run, and the outputs and the workspace are undefined.
 *  - Supported: d in {64, 128} everywhere; on the bf16 tensor-core kernels also every
 *    other multiple of 8 up to 256 (d = 96, 80, 32, 192, ...: the head runs in the 64-,
 *    128- or 256-column kernel, TMA zero-fills the missing columns on load and drops
 *    them on store; not with materialize = 1).  Above 128 the forward accumulates the
 *    scores over two 128-column chunks and the backward works on 128 x 64 tiles in two
 *    passes over the halves of d; there dq_mode is MOA_DQ_AUTO or MOA_DQ_RED
 *    (BULK_REDUCE and SEPARATE_PASS give MOA_ERR_UNSUPPORTED).  Any n >= 1 and B, H >= 1 (B*H <= 2^20 and
 *    ceil(n/64)*B*H < 2^31, else MOA_ERR_UNSUPPORTED); n need not be a multiple
 *    of the tile size.
 *    A device that is not compute capability 10.x gives MOA_ERR_ARCH.
 */
#ifndef MOA_ATTN_H
#define MOA_ATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MOA_OK = 0,
    MOA_ERR_INVALID_ARG = 1, /* NULL pointer, misaligned pointer, non-positive size, bad enum  */
    MOA_ERR_UNSUPPORTED = 2, /* well-formed request this build cannot run (e.g. d = 320)      */
    MOA_ERR_WORKSPACE = 3,   /* ws == NULL or ws_bytes < moa_attn_workspace_bytes(...)         */
    MOA_ERR_ARCH = 4,        /* current device is not sm_100                                   */
    MOA_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed (launch, descriptor encode)  */
    MOA_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (reported by moa_last_device_status) */
    MOA_ERR_SCRATCH_LIMIT = 7 /* moa_attn_bwd_static_scratch: the problem needs more scratch than
                                 MOA_STATIC_SCRATCH_BYTES                                        */
} moa_status;

typedef enum { MOA_BF16 = 0, MOA_F32 = 1 } moa_dtype;

/* How dQ_i = scale * sum_j dS_ij K_j is accumulated across key tiles (Sec. 4: the
 * paper's GK/GV atomic sites and their removal, transposed here onto dQ because
 * the backward kernel is parallel over key tiles). */
typedef enum {
    MOA_DQ_AUTO = 0,          /* library's choice: BULK_REDUCE for bf16 d <= 128, else RED     */
    MOA_DQ_RED = 1,           /* fp32 red.global.add into a [B,H,n,d] fp32 accumulator        */
    MOA_DQ_BULK_REDUCE = 2,   /* shared-memory tile + cp.reduce.async.bulk add.f32 (bf16 d <= 128) */
    MOA_DQ_SEPARATE_PASS = 3  /* no atomics: a second, query-parallel kernel recomputes dS     */
} moa_dq_mode;

/* Which kernels run the contractions. */
typedef enum {
    MOA_PATH_AUTO = 0,  /* tensor cores when dtype is bf16, SIMT fp32 otherwise                */
    MOA_PATH_SIMT = 1,  /* fp32 FMA kernels (any dtype); the only path for MOA_F32             */
    MOA_PATH_TC = 2     /* tcgen05/TMEM/TMA kernels (bf16 only)                                */
} moa_path;

typedef enum { MOA_OP_FWD = 0, MOA_OP_BWD = 1, MOA_OP_FUSED = 2, MOA_OP_ROWPARALLEL = 3 } moa_op;

/* Memory layout of Q, K, V, dO, O, dQ, dK, dV (all eight; L is always [B,H,n]).
 * BHND: [B,H,n,d] contiguous (the layout of every named configuration).
 * BNHD: [B,n,H,d] contiguous (token-major, as projection GEMMs produce it); the tensor
 * maps take the strides, the arithmetic and the results are the same.  Tensor-core bf16
 * path only; other paths return MOA_ERR_UNSUPPORTED.
 * STRIDED: every tensor is addressed through explicit strides (desc->q_stride, kv_stride, o_stride: elements
 * between consecutive rows, heads and batches; the d elements of a row stay contiguous), e.g. the three
 * thirds of a packed [B,n,3,H,d] projection output handed over as Q, K, V with row stride 3*H*d, so that one
 * projection GEMM can feed the attention without a copy (the block composition the paper's full-block
 * section times).  Every stride must be a multiple of 8 elements and at least d.  Same restriction
 * to the tensor-core bf16 path. */
typedef enum { MOA_LAYOUT_BHND = 0, MOA_LAYOUT_BNHD = 1, MOA_LAYOUT_STRIDED = 2 } moa_layout;

typedef struct {
    int32_t B, H, n, d;
    int32_t causal;      /* 0 or 1                                                            */
    float   scale;       /* multiplies Q K^T inside the softmax (the configs use 1/sqrt(d))    */
    int32_t dtype;       /* moa_dtype of Q,K,V,dO,O,dQ,dK,dV                                   */
    int32_t dq_mode;     /* moa_dq_mode                                                        */
    int32_t materialize; /* 0: fused (no n x n array in memory).  1: comparison variant that
                            writes P and dS to the workspace and reads them back (the paper's
                            "left" ONF, Sec. 1.1); needs an O(n^2) workspace.                  */
    int32_t path;        /* moa_path                                                           */
    int32_t H_kv;        /* key/value heads.  0 or H: one K/V head per query head.  Otherwise
                            H_kv must divide H, and query head h reads K/V head h / (H / H_kv):
                            grouped-query attention (H_kv = 1: multi-query), the head sharing the
                            paper's decode section treats.  K, V, dK, dV are then [B,H_kv,n,d];
                            dK, dV sum the contributions of the H / H_kv query heads of a group.
                            Tensor-core bf16 path only; other paths return MOA_ERR_UNSUPPORTED. */
    int32_t layout;      /* moa_layout                                                         */
    int32_t reserved;    /* 0 (keeps the 64-bit fields below aligned)                          */
    /* MOA_LAYOUT_STRIDED only (ignored otherwise): {row, head, batch} strides in elements of
     * Q and dQ | K, V, dK and dV | O and dO.  L stays [B,H,n]. */
    int64_t q_stride[3];
    int64_t kv_stride[3];
    int64_t o_stride[3];
} moa_attn_desc;

/* Bytes of caller-provided workspace `op` (a moa_op) needs for `desc`.  Returns 0
 * when none is needed and also when desc is invalid (the call itself reports why).
 * Fused path: D [B,H,n] fp32 plus, for bf16 with an atomic dq_mode, an fp32
 * [B,H,n,d] dQ accumulator: O(n d), never O(n^2). */
size_t moa_attn_workspace_bytes(const moa_attn_desc *desc, int op);

/* Forward: O = softmax(scale Q K^T) V and the per-row logsumexp L (needed by the
 * backward).  Reads Q,K,V; writes O [B,H,n,d] and L [B,H,n].  (Paper: forward
 * kernel, Sec. 3; fused ONF, Sec. 1.1.) */
moa_status moa_attn_fwd(const moa_attn_desc *desc,
                        const void *Q, const void *K, const void *V,
                        void *O, float *L,
                        void *ws, size_t ws_bytes, void *stream);

/* Backward: dQ, dK, dV from dO, recomputing P tile by tile from L (written by
 * moa_attn_fwd for the same Q,K,V,desc) and D = rowsum(dO o O) (the paper's
 * "precompute pass", Sec. 4).  Reads Q,K,V,O,L,dO; writes dQ,dK,dV. */
moa_status moa_attn_bwd(const moa_attn_desc *desc,
                        const void *Q, const void *K, const void *V,
                        const void *O, const float *L, const void *dO,
                        void *dQ, void *dK, void *dV,
                        void *ws, size_t ws_bytes, void *stream);

/* Backward for callers that cannot allocate device memory.  (The paper has no
 * counterpart: its benchmarks allocate everything up front on the host.)
 *
 * Some callers of this library have no way to hand it a workspace: code running
 * inside a memory pool whose allocator they do not control, plugins invoked with a
 * fixed argument list of inputs and outputs, or hosts where cudaMalloc is forbidden
 * after start-up.  For them this entry point computes exactly what moa_attn_bwd
 * computes, same arguments minus ws/ws_bytes, but takes its scratch (D, the padded
 * logsumexp and the fp32 dQ accumulator) from an array of MOA_STATIC_SCRATCH_BYTES
 * bytes that is part of the library image itself.  Every GPU that loads the library
 * carries that array until the process exits, which is why it is kept modest.
 *
 *  - It calls no cudaMalloc, cudaFree or any other allocating routine.
 *  - If moa_attn_workspace_bytes(desc, MOA_OP_BWD) exceeds MOA_STATIC_SCRATCH_BYTES the
 *    call returns MOA_ERR_SCRATCH_LIMIT and enqueues nothing; use moa_attn_bwd then.
 *  - The first call on each device looks up the array's device address (a one-time,
 *    per-device set-up done with that device current).  Make that first call before
 *    any stream capture begins.
 *  - All calls on a device share the one array, and it keeps whatever the previous
 *    call left in it; the parts that must start from zero are cleared on the stream at
 *    the start of every call.  Two calls that can overlap on the GPU (different
 *    streams, or different host threads) therefore race on it: serialise them.
 *  - Device ordinals 0..63 are supported (the per-device address cache); beyond that the
 *    call returns MOA_ERR_CUDA. */
#define MOA_STATIC_SCRATCH_BYTES (16u << 20)
moa_status moa_attn_bwd_static_scratch(const moa_attn_desc *desc,
                                       const void *Q, const void *K, const void *V,
                                       const void *O, const float *L, const void *dO,
                                       void *dQ, void *dK, void *dV, void *stream);

/* Which form of the bf16 tensor-core backward runs for head dimensions 72..128: mode 0 (the default) one CTA
 * per key tile; mode 1 pairs of CTAs (two adjacent key tiles per cluster, tcgen05 cta_group::2, the dS tile
 * halves exchanged through the cluster's shared memory); mode < 0 only queries.  Returns the mode in force
 * before the call.  Process-wide; the environment variable MOA_BWD_PAIR=1 sets the initial mode to 1.
 * Both forms compute the same dK and dV bit for bit (one writer per element, the paper's Sec. 4 fix, same
 * summation order); dQ differs by the order of its fp32 additions.  The paired form halves the operand
 * traffic per SM but measured slower (its hand-offs cross SMs); it is kept for that comparison.  No passage
 * of the paper corresponds to the switch. */
int moa_bwd_pair_mode(int mode);

/* Fused forward+backward (the paper's Algorithm 2 as one library call): several
 * launches on one stream, no n x n array in memory.  Reads Q,K,V,dO; writes O, L,
 * dQ, dK, dV. */
moa_status moa_attn_fused_fwd_bwd(const moa_attn_desc *desc,
                                  const void *Q, const void *K, const void *V, const void *dO,
                                  void *O, float *L, void *dQ, void *dK, void *dV,
                                  void *ws, size_t ws_bytes, void *stream);

/* The paper's own fused design, kept as a comparison variant (Sec. 4, "fused v1" and "v3"):
 * ONE kernel, parallel over query rows, does the forward of its rows and then their backward;
 * dQ stays local and the dK (atomic_sites = 1) or dK and dV (atomic_sites = 2) contributions of
 * every (query tile, key tile) pair are added into fp32 accumulators with atomics -- the paper's
 * GK and GV atomic sites, whose count it found to set the device time (2 sites = 2.0000x the
 * atomic instructions = 1.97x the time).  With atomic_sites = 1, dV comes from an atomic-free
 * key-parallel kernel of its own, as in the paper's v3.  fp32 CUDA-core arithmetic (bf16 or fp32
 * tensors, [B,H,n,d], one K/V head per query head); same results as moa_attn_fused_fwd_bwd up
 * to rounding.  Workspace: moa_attn_workspace_bytes(desc, MOA_OP_ROWPARALLEL) (D plus, for bf16,
 * two fp32 [B,H,n,d] accumulators).  desc->dq_mode, path and materialize are ignored. */
moa_status moa_attn_fused_rowparallel(const moa_attn_desc *desc,
                                      const void *Q, const void *K, const void *V, const void *dO,
                                      void *O, float *L, void *dQ, void *dK, void *dV,
                                      int atomic_sites, void *ws, size_t ws_bytes, void *stream);

/* Decode attention (the paper's inference section): one new query per head over a cache of n
 * keys and values, O(n) work, every cached element read once:
 *     out[b,h,:] = softmax_j(scale * q[b,h,:] . K[b,kv,j,:]) V[b,kv,:,:],   kv = h / (H / H_kv).
 * q, out: [B,H,d]; K, V: [B,H_kv,n,d] (H_kv = 0 means H; grouped-query heads share one pass over
 * their K/V head); lse: [B,H] fp32 natural-log logsumexp of the scaled scores, may be NULL.
 * dtype: MOA_BF16 or MOA_F32 (fp32 accumulation either way); d in {64, 128}.  All device
 * pointers, 16-byte aligned; the caller owns every buffer; asynchronous on `stream`.
 * Workspace: moa_decode_workspace_bytes(desc) (partial results of the cache segments). */
typedef struct {
    int32_t B, H, H_kv, n, d;
    float   scale;
    int32_t dtype;       /* moa_dtype */
} moa_decode_desc;
size_t moa_decode_workspace_bytes(const moa_decode_desc *desc);
moa_status moa_decode_attn(const moa_decode_desc *desc, const void *q, const void *K, const void *V,
                           void *out, float *lse, void *ws, size_t ws_bytes, void *stream);

/* Synchronises `stream` and returns MOA_ERR_TIMEOUT if any kernel launched by this
 * library on the current device gave up a bounded wait since the last call of this
 * function (the flag is then cleared), MOA_ERR_CUDA if the stream reports an error,
 * else MOA_OK.  Outputs of a timed-out kernel are undefined. */
moa_status moa_last_device_status(void *stream);

/* Self-test of that mechanism: enqueues one warp that waits on a barrier nothing will ever
 * complete, with a limit of about `limit_cycles` SM cycles (clamped to 1,000 .. 2,000,000,000; the
 * kernels count parked waits of up to 20 us each, so a limit below a few million cycles means
 * one or two milliseconds) instead of the kernels' two seconds.  The wait expires,
 * the warp records the expiry and returns; the next moa_last_device_status on the stream then
 * reports MOA_ERR_TIMEOUT (once) and the device stays usable.  Nothing faults and nothing hangs:
 * this is the path a real kernel takes when a copy or a partner never arrives. */
moa_status moa_selftest_expired_wait(long long limit_cycles, void *stream);

/* Per-kernel device timing, for benchmarks.  The paper's lesson that device time and
 * wall time differ (Sec. 3, device-timer vs wall clock) is why this exists: while
 * enabled, the library records a CUDA event pair on the caller's stream around each
 * kernel it launches (at most MOA_PROFILE_MAX_RECORDS launches between two reads; later
 * ones go untimed).  moa_profile_read synchronises on the recorded events, adds up
 * elapsed milliseconds and launch counts per kernel kind into out (arrays of
 * MOA_KERNEL_KINDS entries), and clears the records.  Not thread-safe; one device at a
 * time.  Returns MOA_ERR_CUDA if an event call fails. */
enum { MOA_KERNEL_FWD = 0, MOA_KERNEL_PREPROCESS = 1, MOA_KERNEL_BWD_KV = 2, MOA_KERNEL_BWD_DQ = 3,
       MOA_KERNEL_CONVERT = 4, MOA_KERNEL_OTHER = 5, MOA_KERNEL_KINDS = 6 };
enum { MOA_PROFILE_MAX_RECORDS = 4096 };
typedef struct { float ms[MOA_KERNEL_KINDS]; uint32_t launches[MOA_KERNEL_KINDS]; } moa_profile;
moa_status moa_profile_enable(int on);
moa_status moa_profile_read(moa_profile *out);

/* Number of kernel launches the library has enqueued in this process since it was
 * loaded (all devices, all streams).  Host-side counter; for benchmarks. */
uint64_t moa_launch_count(void);

const char *moa_status_string(moa_status s);
int moa_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MOA_ATTN_H */
