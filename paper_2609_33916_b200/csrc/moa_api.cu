// C-ABI entry points (include/moa_attn.h): argument checks, workspace carving and
// the sequence of kernel launches of each operation.  No arithmetic here.
#include "common.cuh"
#include "ptx.cuh"
#include <atomic>
#include <mutex>
#include <vector>

#include <cstddef>

// the layout the Python binding mirrors
static_assert(sizeof(moa_attn_desc) == 128 && offsetof(moa_attn_desc, scale) == 20 && offsetof(moa_attn_desc, layout) == 44 &&
              offsetof(moa_attn_desc, q_stride) == 56 && offsetof(moa_attn_desc, o_stride) == 104, "moa_attn_desc layout");

namespace moa {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int k) { g_launches.fetch_add((uint64_t)k, std::memory_order_relaxed); }

// ---- optional per-kernel event timing -------------------------------------------------
namespace {
struct ProfRecord { cudaEvent_t a, b; int kind; };
bool g_prof_on = false;
std::vector<ProfRecord> g_prof_records;   // in use
std::vector<ProfRecord> g_prof_pool;      // created, idle
}  // namespace

LaunchScope::LaunchScope(int kind, cudaStream_t s) : slot(-1), st(s)
{
    count_launch();
    if (!g_prof_on || g_prof_records.size() >= MOA_PROFILE_MAX_RECORDS) return;
    ProfRecord r;
    if (!g_prof_pool.empty()) {
        r = g_prof_pool.back();
        g_prof_pool.pop_back();
    } else if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) {
        return;
    }
    r.kind = kind;
    if (cudaEventRecord(r.a, st) != cudaSuccess) { g_prof_pool.push_back(r); return; }
    g_prof_records.push_back(r);
    slot = (int)g_prof_records.size() - 1;
}

LaunchScope::~LaunchScope()
{
    if (slot >= 0) cudaEventRecord(g_prof_records[slot].b, st);
}

// One status word per device image of this library; kernels with bounded waits set
// it to a non-zero code when a wait expires.
__device__ unsigned int g_device_status[4];

unsigned int *device_status_ptr()
{
    constexpr int kMaxDev = 64;
    static unsigned int *cache[kMaxDev] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return nullptr;
    std::lock_guard<std::mutex> lk(mu);
    if (!cache[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
        cache[dev] = (unsigned int *)p;
    }
    return cache[dev];
}

bool pdl_enabled()
{
    static const bool on = [] { const char *e = getenv("MOA_PDL"); return !(e && e[0] == '0'); }();
    return on;
}

const DeviceInfo &device_info()
{
    constexpr int kMaxDev = 64;
    static DeviceInfo cache[kMaxDev];
    static std::atomic<int> known[kMaxDev];
    static const DeviceInfo fallback{148, 126LL << 20};      // B200, if the attributes cannot be read
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return fallback;
    if (!known[dev].load(std::memory_order_acquire)) {
        int sms = 0, l2 = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return fallback;
        if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess || l2 <= 0) return fallback;
        cache[dev] = DeviceInfo{sms, (long long)l2};
        known[dev].store(1, std::memory_order_release);
    }
    return cache[dev];
}

namespace {

constexpr size_t kAlign = 256;
size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

moa_status check_arch()
{
    constexpr int kMaxDev = 64;
    static std::atomic<int> cache[kMaxDev];  // 0 unknown, 1 ok, 2 wrong arch
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MOA_ERR_CUDA;
    if (dev >= 0 && dev < kMaxDev && cache[dev].load() != 0)
        return cache[dev].load() == 1 ? MOA_OK : MOA_ERR_ARCH;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return MOA_ERR_CUDA;
    const bool ok = major == 10;
    if (dev >= 0 && dev < kMaxDev) cache[dev].store(ok ? 1 : 2);
    return ok ? MOA_OK : MOA_ERR_ARCH;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Shape/enum checks that need no device.
moa_status check_desc(const moa_attn_desc *d)
{
    if (!d) return MOA_ERR_INVALID_ARG;
    if (d->B <= 0 || d->H <= 0 || d->n <= 0 || d->d <= 0) return MOA_ERR_INVALID_ARG;
    if (d->causal != 0 && d->causal != 1) return MOA_ERR_INVALID_ARG;
    if (d->dtype != MOA_BF16 && d->dtype != MOA_F32) return MOA_ERR_INVALID_ARG;
    if (d->dq_mode < MOA_DQ_AUTO || d->dq_mode > MOA_DQ_SEPARATE_PASS) return MOA_ERR_INVALID_ARG;
    if (d->materialize != 0 && d->materialize != 1) return MOA_ERR_INVALID_ARG;
    if (d->path < MOA_PATH_AUTO || d->path > MOA_PATH_TC) return MOA_ERR_INVALID_ARG;
    if (!(d->scale == d->scale) || d->scale - d->scale != 0.f) return MOA_ERR_INVALID_ARG;  // NaN / inf
    // head dimensions other than 64 and 128: multiples of 8 up to 256, on the tensor-core kernels only
    // (they run in the 64-, 128- or 256-column kernels with the missing columns filled with zeros)
    if (d->d != 64 && d->d != 128 &&
        !(d->d % 8 == 0 && d->d <= 256 && d->dtype == MOA_BF16 && d->path != MOA_PATH_SIMT && d->scale > 0.f &&
          !d->materialize))
        return MOA_ERR_UNSUPPORTED;
    // above 128 the backward exists with plain reds only (no bulk reduce, no separate dQ pass)
    if (d->d > 128 && (d->dq_mode == MOA_DQ_BULK_REDUCE || d->dq_mode == MOA_DQ_SEPARATE_PASS)) return MOA_ERR_UNSUPPORTED;
    if ((long long)d->B * d->H > (1 << 20)) return MOA_ERR_UNSUPPORTED;
    // one CTA per (tile, head) in grid.x
    const long long tiles = ((long long)d->n + 63) / 64;
    if (tiles * d->B * d->H >= (1LL << 31)) return MOA_ERR_UNSUPPORTED;
    if (d->path == MOA_PATH_TC && d->dtype != MOA_BF16) return MOA_ERR_UNSUPPORTED;
    // the materialising comparison variant runs on the tensor-core path only
    if (d->materialize && !(d->dtype == MOA_BF16 && d->path != MOA_PATH_SIMT && d->scale > 0.f)) return MOA_ERR_UNSUPPORTED;
    // the bulk-reduce strategy exists in the 64- and 128-column tensor-core backward only
    if (d->dq_mode == MOA_DQ_BULK_REDUCE &&
        !(d->dtype == MOA_BF16 && d->path != MOA_PATH_SIMT && kernel_d(d->d) <= 128 && d->scale > 0.f))
        return MOA_ERR_UNSUPPORTED;
    if (d->path == MOA_PATH_TC && !(d->scale > 0.f)) return MOA_ERR_UNSUPPORTED;   // non-positive scale: SIMT path only
    if (d->layout != MOA_LAYOUT_BHND && d->layout != MOA_LAYOUT_BNHD && d->layout != MOA_LAYOUT_STRIDED) return MOA_ERR_INVALID_ARG;
    if (d->layout == MOA_LAYOUT_STRIDED) {
        // rows of d contiguous elements; every stride positive, a multiple of 8 elements (16 bytes: what the
        // tensor maps and the 16-byte row accesses need) and at least one row long
        const int64_t *cls[3] = {d->q_stride, d->kv_stride, d->o_stride};
        for (int c = 0; c < 3; ++c)
            for (int k = 0; k < 3; ++k)
                if (cls[c][k] < d->d || cls[c][k] % 8 != 0) return MOA_ERR_INVALID_ARG;
    }
    // token-major and strided tensors: tensor-core kernels only
    if (d->layout != MOA_LAYOUT_BHND &&
        !(d->dtype == MOA_BF16 && d->path != MOA_PATH_SIMT && d->scale > 0.f && !d->materialize))
        return MOA_ERR_UNSUPPORTED;
    if (d->H_kv < 0 || d->H_kv > d->H) return MOA_ERR_INVALID_ARG;
    if (d->H_kv > 0 && d->H % d->H_kv != 0) return MOA_ERR_INVALID_ARG;
    // shared K/V heads: tensor-core kernels only
    if (d->H_kv > 0 && d->H_kv != d->H &&
        !(d->dtype == MOA_BF16 && d->path != MOA_PATH_SIMT && d->scale > 0.f && !d->materialize))
        return MOA_ERR_UNSUPPORTED;
    return MOA_OK;
}

// AUTO: the TMA bulk add-reduce where it exists (tensor-core path, 64- and 128-column kernels: measured slightly ahead of
// plain reds at every size at 128 columns, 15-25 % ahead at 64, where the reds fill half a sector each), plain reds otherwise.
int resolved_dq_mode(const moa_attn_desc *d)
{
    if (d->dq_mode != MOA_DQ_AUTO) return d->dq_mode;
    const bool tc = d->dtype == MOA_BF16 && d->path != MOA_PATH_SIMT && d->scale > 0.f;
    return (tc && kernel_d(d->d) <= 128) ? MOA_DQ_BULK_REDUCE : MOA_DQ_RED;
}

// the tensor-core kernels take the row max before scaling, which needs scale > 0
bool use_tc_fwd(const moa_attn_desc *d) { return d->dtype == MOA_BF16 && d->path != MOA_PATH_SIMT && d->scale > 0.f; }
bool use_tc_bwd(const moa_attn_desc *d)
{
    const int mode = resolved_dq_mode(d);
    return d->dtype == MOA_BF16 && d->path != MOA_PATH_SIMT && d->scale > 0.f &&
           (mode == MOA_DQ_RED || mode == MOA_DQ_BULK_REDUCE || mode == MOA_DQ_SEPARATE_PASS);
}

// Workspace of the backward: [ D | Lp (tensor-core path only) | dQacc (bf16 with an atomic mode) ]
struct BwdWorkspace {
    size_t d_bytes, lp_bytes, dqacc_bytes, total;
};
BwdWorkspace bwd_workspace(const moa_attn_desc *d)
{
    BwdWorkspace w{};
    const size_t rows = (size_t)d->B * d->H * d->n;
    if (use_tc_bwd(d)) {
        const size_t prows = (size_t)d->B * d->H * (((size_t)d->n + 127) / 128 * 128);
        w.d_bytes = align_up(prows * sizeof(float));
        w.lp_bytes = align_up(prows * sizeof(float));
    } else {
        w.d_bytes = align_up(rows * sizeof(float));
    }
    const bool need_acc = d->dtype == MOA_BF16 && resolved_dq_mode(d) != MOA_DQ_SEPARATE_PASS;
    // the tensor-core backward accumulates rows of its own (64 or 128) columns
    const size_t acc_cols = use_tc_bwd(d) ? (size_t)kernel_d(d->d) : (size_t)d->d;
    w.dqacc_bytes = need_acc ? align_up(rows * acc_cols * sizeof(float)) : 0;
    w.total = w.d_bytes + w.lp_bytes + w.dqacc_bytes;
    return w;
}

// Materialising variant: heads are processed in groups so that the two n x n arrays (P^T, dS^T,
// bf16, row stride n_pad) of one group stay under kMatCapBytes.
constexpr size_t kMatCapBytes = (size_t)16 << 30;
struct MatWorkspace {
    int group;            // heads per group
    size_t npad, arr_bytes /* one array, one group */, lp_bytes, d_bytes, total;
};
MatWorkspace mat_workspace(const moa_attn_desc *d, int op)
{
    MatWorkspace w{};
    const size_t heads = (size_t)d->B * d->H;
    w.npad = ((size_t)d->n + 127) / 128 * 128;
    const size_t per_head = w.npad * w.npad * 2;
    size_t g = kMatCapBytes / (2 * per_head);
    if (g < 1) g = 1;
    if (g > heads) g = heads;
    w.group = (int)g;
    w.arr_bytes = align_up(g * per_head);
    w.lp_bytes = align_up(g * w.npad * sizeof(float));
    w.d_bytes = w.lp_bytes;
    w.total = op == MOA_OP_FWD ? w.arr_bytes : 2 * w.arr_bytes + w.lp_bytes + w.d_bytes;
    return w;
}

Problem to_problem(const moa_attn_desc *d)
{
    Problem p{d->B, d->H, d->n, d->d, d->causal, d->scale, d->H_kv, d->layout == MOA_LAYOUT_BNHD ? 1 : 0};
    p.with_layout();
    if (d->layout == MOA_LAYOUT_STRIDED) {
        p.sq = Strides{d->q_stride[0], d->q_stride[1], d->q_stride[2]};
        p.skv = Strides{d->kv_stride[0], d->kv_stride[1], d->kv_stride[2]};
        p.so = Strides{d->o_stride[0], d->o_stride[1], d->o_stride[2]};
    }
    return p;
}

// Materialising variant.  with_bwd = false: forward only (P^T is written and dropped).
moa_status run_materialized(const moa_attn_desc *d, const void *Q, const void *K, const void *V, const void *dO,
                            void *O, float *L, void *dQ, void *dK, void *dV, void *ws, bool with_bwd, cudaStream_t st)
{
    const MatWorkspace w = mat_workspace(d, with_bwd ? MOA_OP_FUSED : MOA_OP_FWD);
    char *base = (char *)ws;
    void *PT = base;
    void *GST = base + w.arr_bytes;
    float *Lp = (float *)(base + 2 * w.arr_bytes);
    float *Dp = (float *)(base + 2 * w.arr_bytes + w.lp_bytes);
    const int heads = d->B * d->H;
    const size_t esz = 2, hs = (size_t)d->n * d->d * esz;
    for (int g0 = 0; g0 < heads; g0 += w.group) {
        const int g = heads - g0 < w.group ? heads - g0 : w.group;
        Problem p{1, g, d->n, d->d, d->causal, d->scale, 0};
        p.with_layout();
        const char *q = (const char *)Q + g0 * hs, *k = (const char *)K + g0 * hs, *v = (const char *)V + g0 * hs;
        char *o = (char *)O + g0 * hs;
        float *l = L + (size_t)g0 * d->n;
        if (mat_fwd(p, q, k, v, o, l, PT, st) != cudaSuccess) return MOA_ERR_CUDA;
        if (!with_bwd) continue;
        const char *g_do = (const char *)dO + g0 * hs;
        if (tc_bwd_preprocess(p, g_do, o, l, Lp, Dp, st) != cudaSuccess) return MOA_ERR_CUDA;
        if (mat_bwd(p, q, k, v, g_do, Dp, PT, GST, (char *)dQ + g0 * hs, (char *)dK + g0 * hs, (char *)dV + g0 * hs, st) !=
            cudaSuccess)
            return MOA_ERR_CUDA;
    }
    return MOA_OK;
}

moa_status run_fwd(const moa_attn_desc *d, const void *Q, const void *K, const void *V, void *O, float *L,
                   const FwdForBwd &fb, cudaStream_t st)
{
    // fb: what the tensor-core forward of a fused call prepares for its backward (empty otherwise)
    const cudaError_t e = use_tc_fwd(d) ? tc_fwd(to_problem(d), Q, K, V, O, L, fb, st)
                             : simt_fwd(to_problem(d), d->dtype, Q, K, V, O, L, st);
    return e == cudaSuccess ? MOA_OK : MOA_ERR_CUDA;
}

moa_status run_bwd(const moa_attn_desc *d, const void *Q, const void *K, const void *V, const void *O,
                   const float *L, const void *dO, void *dQ, void *dK, void *dV, void *ws, bool prepared,
                   cudaStream_t st)
{
    // prepared: the forward of the same fused call has cleared the dQ accumulator and written -L log2e and -D
    const Problem p = to_problem(d);
    const BwdWorkspace w = bwd_workspace(d);
    float *Dv = (float *)ws;
    float *Lp = (float *)((char *)ws + w.d_bytes);
    float *dQacc = w.dqacc_bytes ? (float *)((char *)ws + w.d_bytes + w.lp_bytes) : nullptr;
    const size_t elems = (size_t)p.BH() * p.n * p.d;
    const int mode = resolved_dq_mode(d);
#define MOA_TRY(x) do { if ((x) != cudaSuccess) return MOA_ERR_CUDA; } while (0)
    if (use_tc_bwd(d)) {
        if (!prepared) MOA_TRY(tc_bwd_preprocess(p, dO, O, L, Lp, Dv, st));
        if (mode == MOA_DQ_SEPARATE_PASS) {
            MOA_TRY(tc_bwd_kv(p, Q, K, V, dO, Lp, Dv, dK, dV, nullptr, 0, st));
            MOA_TRY(tc_bwd_dq(p, Q, K, V, dO, Lp, Dv, dQ, st));
            return MOA_OK;
        }
        const int acc_ld = kernel_d(p.d);
        if (!prepared) MOA_TRY(cudaMemsetAsync(dQacc, 0, (size_t)p.BH() * p.n * acc_ld * sizeof(float), st));
        MOA_TRY(tc_bwd_kv(p, Q, K, V, dO, Lp, Dv, dK, dV, dQacc, mode == MOA_DQ_BULK_REDUCE, st));
        if (!p.contiguous_bhnd() || acc_ld != p.d) MOA_TRY(convert_f32_to_bf16_rows(dQacc, acc_ld, dQ, p.B, p.H, p.n, p.d, p.sq, p.scale, st));
        else MOA_TRY(convert_f32_to_bf16(dQacc, dQ, elems, p.scale, st));
        return MOA_OK;
    }
    MOA_TRY(row_dot(p, d->dtype, dO, O, Dv, st));
    if (mode == MOA_DQ_SEPARATE_PASS) {
        MOA_TRY(simt_bwd_kv(p, d->dtype, Q, K, V, dO, L, Dv, dK, dV, nullptr, st));
        MOA_TRY(simt_bwd_dq(p, d->dtype, Q, K, V, dO, L, Dv, dQ, st));
    } else {
        float *acc = d->dtype == MOA_F32 ? (float *)dQ : dQacc;   // fp32 output accumulates in place
        MOA_TRY(cudaMemsetAsync(acc, 0, elems * sizeof(float), st));
        MOA_TRY(simt_bwd_kv(p, d->dtype, Q, K, V, dO, L, Dv, dK, dV, acc, st));
        if (d->dtype == MOA_BF16) MOA_TRY(convert_f32_to_bf16(dQacc, dQ, elems, 1.f, st));
    }
#undef MOA_TRY
    return MOA_OK;
}

// Built-in scratch of moa_attn_bwd_static_scratch.  In host code this name is only a
// handle for the symbol, not a device address: the address each device gives it is
// looked up once per device below and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[MOA_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device (nullptr on failure).
void *static_scratch_ptr()
{
    constexpr int kMaxDev = 64;
    static void *cache[kMaxDev] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return nullptr;
    std::lock_guard<std::mutex> lk(mu);
    if (!cache[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess) return nullptr;
        cache[dev] = p;
    }
    return cache[dev];
}

}  // namespace

moa_status check_device_arch() { return check_arch(); }

}  // namespace moa

using namespace moa;

// Workspace of the row-parallel comparison variant: [ D | dKacc | dVacc ] (accumulators for bf16 only;
// fp32 tensors accumulate in place)
static size_t rowpar_workspace(const moa_attn_desc *d)
{
    const size_t rows = (size_t)d->B * d->H * d->n;
    const size_t acc = d->dtype == MOA_BF16 ? align_up(rows * d->d * sizeof(float)) : 0;
    return align_up(rows * sizeof(float)) + 2 * acc;
}

extern "C" {

size_t moa_attn_workspace_bytes(const moa_attn_desc *desc, int op)
{
    if (check_desc(desc) != MOA_OK) return 0;
    if (desc->materialize) return (op == MOA_OP_FWD || op == MOA_OP_FUSED) ? mat_workspace(desc, op).total : 0;
    if (op == MOA_OP_FWD) return 0;
    if (op == MOA_OP_BWD || op == MOA_OP_FUSED) return bwd_workspace(desc).total;
    if (op == MOA_OP_ROWPARALLEL) return rowpar_workspace(desc);
    return 0;
}

moa_status moa_attn_fwd(const moa_attn_desc *desc, const void *Q, const void *K, const void *V,
                        void *O, float *L, void *ws, size_t ws_bytes, void *stream)
{
    moa_status s = check_desc(desc);
    if (s != MOA_OK) return s;
    if (!Q || !K || !V || !O || !L) return MOA_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(L)) return MOA_ERR_INVALID_ARG;
    if (desc->materialize) {
        if (!ws || ws_bytes < mat_workspace(desc, MOA_OP_FWD).total) return MOA_ERR_WORKSPACE;
        if (!aligned16(ws)) return MOA_ERR_INVALID_ARG;
    }
    if ((s = check_arch()) != MOA_OK) return s;
    if (desc->materialize)
        return run_materialized(desc, Q, K, V, nullptr, O, L, nullptr, nullptr, nullptr, ws, false, (cudaStream_t)stream);
    return run_fwd(desc, Q, K, V, O, L, FwdForBwd{}, (cudaStream_t)stream);
}

moa_status moa_attn_bwd(const moa_attn_desc *desc, const void *Q, const void *K, const void *V,
                        const void *O, const float *L, const void *dO,
                        void *dQ, void *dK, void *dV, void *ws, size_t ws_bytes, void *stream)
{
    moa_status s = check_desc(desc);
    if (s != MOA_OK) return s;
    // the materialising variant's backward consumes the P array its own forward wrote: fused call only
    if (desc->materialize) return MOA_ERR_UNSUPPORTED;
    if (!Q || !K || !V || !O || !L || !dO || !dQ || !dK || !dV) return MOA_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(L) || !aligned16(dO) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV))
        return MOA_ERR_INVALID_ARG;
    const size_t need = bwd_workspace(desc).total;
    if (!ws || ws_bytes < need) return MOA_ERR_WORKSPACE;
    if (!aligned16(ws)) return MOA_ERR_INVALID_ARG;
    if ((s = check_arch()) != MOA_OK) return s;
    return run_bwd(desc, Q, K, V, O, L, dO, dQ, dK, dV, ws, false, (cudaStream_t)stream);
}

moa_status moa_attn_bwd_static_scratch(const moa_attn_desc *desc, const void *Q, const void *K, const void *V,
                                       const void *O, const float *L, const void *dO,
                                       void *dQ, void *dK, void *dV, void *stream)
{
    moa_status s = check_desc(desc);
    if (s != MOA_OK) return s;
    if (!Q || !K || !V || !O || !L || !dO || !dQ || !dK || !dV) return MOA_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(L) || !aligned16(dO) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV))
        return MOA_ERR_INVALID_ARG;
    if (desc->materialize) return MOA_ERR_UNSUPPORTED;
    if (bwd_workspace(desc).total > (size_t)MOA_STATIC_SCRATCH_BYTES) return MOA_ERR_SCRATCH_LIMIT;
    if ((s = check_arch()) != MOA_OK) return s;
    void *scratch = static_scratch_ptr();   // first call on this device resolves the symbol's address
    if (!scratch) return MOA_ERR_CUDA;
    // run_bwd clears the dQ accumulator on the stream and overwrites D / Lp before use
    return run_bwd(desc, Q, K, V, O, L, dO, dQ, dK, dV, scratch, false, (cudaStream_t)stream);
}

moa_status moa_attn_fused_fwd_bwd(const moa_attn_desc *desc, const void *Q, const void *K, const void *V,
                                  const void *dO, void *O, float *L, void *dQ, void *dK, void *dV,
                                  void *ws, size_t ws_bytes, void *stream)
{
    moa_status s = check_desc(desc);
    if (s != MOA_OK) return s;
    if (!Q || !K || !V || !O || !L || !dO || !dQ || !dK || !dV) return MOA_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(L) || !aligned16(dO) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV))
        return MOA_ERR_INVALID_ARG;
    const size_t need = desc->materialize ? mat_workspace(desc, MOA_OP_FUSED).total : bwd_workspace(desc).total;
    if (!ws || ws_bytes < need) return MOA_ERR_WORKSPACE;
    if (!aligned16(ws)) return MOA_ERR_INVALID_ARG;
    if ((s = check_arch()) != MOA_OK) return s;
    if (desc->materialize) return run_materialized(desc, Q, K, V, dO, O, L, dQ, dK, dV, ws, true, (cudaStream_t)stream);
    // tensor-core path with an atomic dQ mode: the forward clears the accumulator its backward adds into
    // and writes the backward's per-row inputs (-L log2e, -D) from the fp32 O it holds
    FwdForBwd fb;
    // (head dimensions above 128: a forward CTA holds half of an O row, so the backward prepares its own inputs)
    const bool both_tc = use_tc_fwd(desc) && use_tc_bwd(desc) && kernel_d(desc->d) <= 128;
    if (both_tc) {
        const BwdWorkspace w = bwd_workspace(desc);
        fb.Dp = (float *)ws;
        fb.Lp = (float *)((char *)ws + w.d_bytes);
        fb.dO = dO;
        if (w.dqacc_bytes) fb.zero_acc = (float *)((char *)ws + w.d_bytes + w.lp_bytes);
    }
    if ((s = run_fwd(desc, Q, K, V, O, L, fb, (cudaStream_t)stream)) != MOA_OK) return s;
    return run_bwd(desc, Q, K, V, O, L, dO, dQ, dK, dV, ws, both_tc, (cudaStream_t)stream);
}

moa_status moa_attn_fused_rowparallel(const moa_attn_desc *desc, const void *Q, const void *K, const void *V,
                                      const void *dO, void *O, float *L, void *dQ, void *dK, void *dV,
                                      int atomic_sites, void *ws, size_t ws_bytes, void *stream)
{
    moa_status s = check_desc(desc);
    if (s != MOA_OK) return s;
    if (atomic_sites != 1 && atomic_sites != 2) return MOA_ERR_INVALID_ARG;
    if ((desc->H_kv > 0 && desc->H_kv != desc->H) || desc->layout != MOA_LAYOUT_BHND) return MOA_ERR_UNSUPPORTED;
    if (desc->d != 64 && desc->d != 128) return MOA_ERR_UNSUPPORTED;          // CUDA-core kernels: d in {64, 128}
    if (!Q || !K || !V || !O || !L || !dO || !dQ || !dK || !dV) return MOA_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(L) || !aligned16(dO) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV))
        return MOA_ERR_INVALID_ARG;
    if (!ws || ws_bytes < rowpar_workspace(desc)) return MOA_ERR_WORKSPACE;
    if (!aligned16(ws)) return MOA_ERR_INVALID_ARG;
    if ((s = check_arch()) != MOA_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    Problem p = to_problem(desc);
    p.Hkv = 0;
    const size_t rows = (size_t)p.BH() * p.n, elems = rows * p.d;
    float *Dv = (float *)ws;
    const bool bf = desc->dtype == MOA_BF16;
    float *dKacc = bf ? (float *)((char *)ws + align_up(rows * sizeof(float))) : (float *)dK;
    float *dVacc = bf ? dKacc + align_up(elems * sizeof(float)) / sizeof(float) : (float *)dV;
#define MOA_TRY(x) do { if ((x) != cudaSuccess) return MOA_ERR_CUDA; } while (0)
    MOA_TRY(cudaMemsetAsync(dKacc, 0, elems * sizeof(float), st));
    if (atomic_sites == 2) MOA_TRY(cudaMemsetAsync(dVacc, 0, elems * sizeof(float), st));
    MOA_TRY(simt_rowpar(p, desc->dtype, Q, K, V, dO, O, L, Dv, dQ, dKacc, dVacc, atomic_sites, st));
    if (atomic_sites == 1)   // dV by the atomic-free key-parallel kernel (no dK, no dQ from it)
        MOA_TRY(simt_bwd_kv(p, desc->dtype, Q, K, V, dO, L, Dv, nullptr, dV, nullptr, st));
    if (bf) {
        MOA_TRY(convert_f32_to_bf16(dKacc, dK, elems, 1.f, st));
        if (atomic_sites == 2) MOA_TRY(convert_f32_to_bf16(dVacc, dV, elems, 1.f, st));
    }
#undef MOA_TRY
    return MOA_OK;
}

static moa_status check_decode_desc(const moa_decode_desc *d, DecodeProblem *p)
{
    if (!d) return MOA_ERR_INVALID_ARG;
    if (d->B <= 0 || d->H <= 0 || d->n <= 0 || d->d <= 0 || d->H_kv < 0 || d->H_kv > d->H) return MOA_ERR_INVALID_ARG;
    const int hkv = d->H_kv > 0 ? d->H_kv : d->H;
    if (d->H % hkv != 0) return MOA_ERR_INVALID_ARG;
    if (d->dtype != MOA_BF16 && d->dtype != MOA_F32) return MOA_ERR_INVALID_ARG;
    if (!(d->scale == d->scale) || d->scale - d->scale != 0.f) return MOA_ERR_INVALID_ARG;
    if (d->d != 64 && d->d != 128) return MOA_ERR_UNSUPPORTED;
    if ((long long)d->B * d->H > (1 << 24)) return MOA_ERR_UNSUPPORTED;
    *p = DecodeProblem{d->B, d->H, hkv, d->n, d->d, d->scale};
    return MOA_OK;
}

size_t moa_decode_workspace_bytes(const moa_decode_desc *desc)
{
    DecodeProblem p;
    if (check_decode_desc(desc, &p) != MOA_OK) return 0;
    return decode_workspace_bytes(p, desc->dtype);
}

moa_status moa_decode_attn(const moa_decode_desc *desc, const void *q, const void *K, const void *V,
                           void *out, float *lse, void *ws, size_t ws_bytes, void *stream)
{
    DecodeProblem p;
    moa_status s = check_decode_desc(desc, &p);
    if (s != MOA_OK) return s;
    if (!q || !K || !V || !out) return MOA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(K) || !aligned16(V) || !aligned16(out) || (lse && !aligned16(lse))) return MOA_ERR_INVALID_ARG;
    if (!ws || ws_bytes < decode_workspace_bytes(p, desc->dtype)) return MOA_ERR_WORKSPACE;
    if (!aligned16(ws)) return MOA_ERR_INVALID_ARG;
    if ((s = check_arch()) != MOA_OK) return s;
    return decode_attn(p, desc->dtype, q, K, V, out, lse, ws, (cudaStream_t)stream) == cudaSuccess ? MOA_OK
                                                                                                             : MOA_ERR_CUDA;
}

moa_status moa_last_device_status(void *stream)
{
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return MOA_ERR_CUDA;
    unsigned int *p = device_status_ptr();
    if (!p) return MOA_ERR_CUDA;
    unsigned int h[4] = {0, 0, 0, 0};
    if (cudaMemcpy(h, p, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return MOA_ERR_CUDA;
    if (h[0] != 0) {
        cudaMemset(p, 0, sizeof(h));
        return MOA_ERR_TIMEOUT;
    }
    return MOA_OK;
}

// One warp waits on a barrier that nothing completes; the bounded wait expires and records it.
__global__ void selftest_expired_wait_kernel(unsigned int *status, long long limit)
{
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        moa::ptx::mbar_init(&bar, 1);
        abort_flag = 0;
        moa::ptx::fence_mbar_init();
    }
    __syncthreads();
    moa::ptx::mbar_wait(&bar, 0, &abort_flag, status, 0x7F1u, limit);
}

moa_status moa_selftest_expired_wait(long long limit_cycles, void *stream)
{
    moa_status s = check_device_arch();
    if (s != MOA_OK) return s;
    if (limit_cycles < 1000) limit_cycles = 1000;
    if (limit_cycles > 2000000000LL) limit_cycles = 2000000000LL;
    unsigned int *p = device_status_ptr();
    if (!p) return MOA_ERR_CUDA;
    count_launch();
    selftest_expired_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(p, limit_cycles);
    return cudaGetLastError() == cudaSuccess ? MOA_OK : MOA_ERR_CUDA;
}

moa_status moa_profile_enable(int on)
{
    g_prof_on = on != 0;
    return MOA_OK;
}

moa_status moa_profile_read(moa_profile *out)
{
    if (!out) return MOA_ERR_INVALID_ARG;
    for (int k = 0; k < MOA_KERNEL_KINDS; ++k) { out->ms[k] = 0.f; out->launches[k] = 0; }
    moa_status rc = MOA_OK;
    for (auto &r : g_prof_records) {
        float ms = 0.f;
        if (cudaEventSynchronize(r.b) != cudaSuccess || cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess) {
            rc = MOA_ERR_CUDA;
        } else if (r.kind >= 0 && r.kind < MOA_KERNEL_KINDS) {
            out->ms[r.kind] += ms;
            out->launches[r.kind] += 1;
        }
        g_prof_pool.push_back(r);
    }
    g_prof_records.clear();
    return rc;
}

int moa_bwd_pair_mode(int mode) { return bwd_pair_mode(mode); }


uint64_t moa_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char *moa_status_string(moa_status s)
{
    switch (s) {
        case MOA_OK: return "ok";
        case MOA_ERR_INVALID_ARG: return "invalid argument";
        case MOA_ERR_UNSUPPORTED: return "unsupported configuration";
        case MOA_ERR_WORKSPACE: return "workspace missing or too small";
        case MOA_ERR_ARCH: return "device is not sm_100";
        case MOA_ERR_CUDA: return "CUDA call failed";
        case MOA_ERR_TIMEOUT: return "bounded device wait expired";
        case MOA_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the built-in static array holds";
    }
    return "unknown status";
}

int moa_version(void) { return 100; }

}  // extern "C"
