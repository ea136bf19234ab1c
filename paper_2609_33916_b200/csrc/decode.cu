// Decode attention: one new query per head over a cache of n keys and values (the paper's
// decode section: O(n) work per token, every cached element read exactly once).
//
// HBM-bound: 2 n d elements of cache per K/V head against 4 n d flop per query head, so the
// kernel is organised around keeping reads in flight, not around the tensor cores (a tile of
// 1..8 query rows would fill 1-6 % of a 128-row UMMA).  One CTA streams a segment of the cache
// of one K/V head and serves all query heads that share it (grouped-query attention: the cache
// is read once per group, not once per query head):
//   * a row of d elements is fetched by d*sizeof(T)/16 lanes with one 16-byte streaming load
//     each, so every warp instruction reads whole rows, fully coalesced; a warp keeps kUnroll
//     row groups of K and of V in flight;
//   * score = q . k: per-lane partial dot (the lane's 16 bytes of the row against the same
//     elements of q, kept in registers, pre-multiplied by scale*log2 e), then an xor-shuffle
//     butterfly over the lanes of the row;
//   * online softmax per lane group (exp2, running max and sum), out += p * v on the lane's own
//     elements of the V row: no further exchange inside the loop;
//   * at the end the lane groups of a warp, the warps of the CTA (through shared memory) and,
//     in a second tiny kernel, the CTAs of a head are merged by their running maxima.
#include "common.cuh"
#include "ptx.cuh"

namespace moa {
namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kUnroll = 4;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <typename T> struct Vec16;
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static void unpack(const uint4 &v, float *f)
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 p = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&w[i]));
            f[2 * i] = p.x;
            f[2 * i + 1] = p.y;
        }
    }
};
template <> struct Vec16<float> {
    static constexpr int kElems = 4;
    __device__ static void unpack(const uint4 &v, float *f)
    {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
};

// The running state of one lane group (the lanes that share rows): per query head of the group the
// maximum m (log2 domain), the sum l of 2^(s - m) and this lane's E elements of sum_j 2^(s_j - m) v_j.
template <typename T, int D, int GC>
struct DecodeState {
    static constexpr int E = Vec16<T>::kElems;      // elements per lane
    static constexpr int LPR = D / E;               // lanes per row
    static constexpr int RPW = 32 / LPR;            // rows per warp-wide access
    static_assert(LPR >= 1 && LPR <= 32 && 32 % LPR == 0, "row must map onto a warp");
    float qv[GC][E], m[GC], lsum[GC], acc[GC][E];

    // this lane's elements of every query of the group, pre-multiplied by scale * log2 e
    __device__ void init(const T *q_first, int gcount, int l, float scale_log2)
    {
#pragma unroll
        for (int g = 0; g < GC; ++g) {
            float f[E];
            if (g < gcount) {
                Vec16<T>::unpack(*reinterpret_cast<const uint4 *>(q_first + (size_t)g * D + l * E), f);
            } else {
#pragma unroll
                for (int e = 0; e < E; ++e) f[e] = 0.f;
            }
#pragma unroll
            for (int e = 0; e < E; ++e) { qv[g][e] = f[e] * scale_log2; acc[g][e] = 0.f; }
            m[g] = -INFINITY;
            lsum[g] = 0.f;
        }
    }

    // U rows (one per lane group each): scores by per-lane partial dots and a butterfly over the lanes of
    // the row, one online-softmax step over the U rows, then out += p * v on the lane's own elements
    template <int U>
    __device__ void consume(const uint4 (&kraw)[U], const uint4 (&vraw)[U], const bool (&live)[U])
    {
        float s[U][GC];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            float kf[E];
            Vec16<T>::unpack(kraw[u], kf);
#pragma unroll
            for (int g = 0; g < GC; ++g) {
                float d0 = 0.f;
#pragma unroll
                for (int e = 0; e < E; ++e) d0 = fmaf(qv[g][e], kf[e], d0);
#pragma unroll
                for (int o = LPR / 2; o >= 1; o >>= 1) d0 += __shfl_xor_sync(0xffffffffu, d0, o);
                s[u][g] = live[u] ? d0 : -INFINITY;
            }
        }
#pragma unroll
        for (int g = 0; g < GC; ++g) {
            float mx = m[g];
#pragma unroll
            for (int u = 0; u < U; ++u) mx = fmaxf(mx, s[u][g]);
            const float ref = (mx == -INFINITY) ? 0.f : mx;      // nothing visible yet: any finite reference
            const float alpha = exp2f(m[g] - ref);
            m[g] = mx;
            lsum[g] *= alpha;
#pragma unroll
            for (int e = 0; e < E; ++e) acc[g][e] *= alpha;
#pragma unroll
            for (int u = 0; u < U; ++u) s[u][g] = exp2f(s[u][g] - ref);     // now the weight p
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            float vf[E];
            Vec16<T>::unpack(vraw[u], vf);
#pragma unroll
            for (int g = 0; g < GC; ++g) {
                lsum[g] += s[u][g];
#pragma unroll
                for (int e = 0; e < E; ++e) acc[g][e] = fmaf(s[u][g], vf[e], acc[g][e]);
            }
        }
    }

    // Merge the lane groups of the warp, then the warps of the CTA through `sm` ([warp][g][D + 2]
    // floats), and write this segment's partial result: part_o [splits][B*H][D], part_ml [splits][B*H][2].
    __device__ void finish(float *sm, int warp, int lane, int nwarps, int gcount, size_t head0, int split, size_t BH,
                           float *part_o, float *part_ml, int nthreads)
    {
        const int sub = lane / LPR, l = lane % LPR;
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
            for (int g = 0; g < GC; ++g) {
                const float mo = __shfl_xor_sync(0xffffffffu, m[g], o);
                const float lo = __shfl_xor_sync(0xffffffffu, lsum[g], o);
                const float mx = fmaxf(m[g], mo);
                const float ref = (mx == -INFINITY) ? 0.f : mx;
                const float a = exp2f(m[g] - ref), bo = exp2f(mo - ref);
                lsum[g] = lsum[g] * a + lo * bo;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const float ao = __shfl_xor_sync(0xffffffffu, acc[g][e], o);
                    acc[g][e] = acc[g][e] * a + ao * bo;
                }
                m[g] = mx;
            }
        }
        constexpr int kStride = D + 2;
        if (warp < nwarps && sub == 0) {
#pragma unroll
            for (int g = 0; g < GC; ++g) {
                float *dst = sm + (warp * GC + g) * kStride;
#pragma unroll
                for (int e = 0; e < E; ++e) dst[l * E + e] = acc[g][e];
                if (l == 0) { dst[D] = m[g]; dst[D + 1] = lsum[g]; }
            }
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < gcount * D; idx += nthreads) {
            const int g = idx / D, c = idx - g * D;
            float mx = -INFINITY;
            for (int w = 0; w < nwarps; ++w) mx = fmaxf(mx, sm[(w * GC + g) * kStride + D]);
            const float ref = (mx == -INFINITY) ? 0.f : mx;
            float o = 0.f, ls = 0.f;
            for (int w = 0; w < nwarps; ++w) {
                const float *src = sm + (w * GC + g) * kStride;
                const float a = exp2f(src[D] - ref);
                o = fmaf(src[c], a, o);
                ls = fmaf(src[D + 1], a, ls);
            }
            const size_t at = (size_t)split * BH + head0 + g;
            part_o[at * D + c] = o;
            if (c == 0) { part_ml[at * 2] = mx; part_ml[at * 2 + 1] = ls; }
        }
    }
};

// Where a CTA works: K/V head, the query heads of its group it serves, its segment of the cache.
struct DecodeJob {
    int split, bkv, g0, gcount, b, kvh, k_begin, k_end;
    size_t head0;      // flat index b * H + first query head
    __device__ DecodeJob(int splits, int GC, int group, int H, int Hkv, int n, int keys_per_split)
    {
        split = blockIdx.x % splits;
        bkv = blockIdx.x / splits;
        g0 = blockIdx.y * GC;
        gcount = min(GC, group - g0);
        b = bkv / Hkv;
        kvh = bkv - b * Hkv;
        head0 = (size_t)b * H + kvh * group + g0;
        k_begin = split * keys_per_split;
        k_end = min(n, k_begin + keys_per_split);
    }
};

// Merge of one query head's segments (thread = (stripe of segments, output column), the stripes merged through
// `sh`: kStripes * (D + 2) floats), normalise, write out (and the natural-log lse).  Called by every thread of a CTA
// of at least 256 threads; threads past 256 only take part in the barriers.  The partial results are read with
// ld.global.cg: other CTAs wrote them.
template <typename T, int D>
__device__ __forceinline__ void merge_head(const float *__restrict__ part_o, const float *__restrict__ part_ml,
                                           T *__restrict__ out, float *__restrict__ lse, int splits, size_t BH, size_t head,
                                           float *sh)
{
    constexpr int kStripes = 256 / D;
    float *sh_o = sh, *sh_m = sh + kStripes * D, *sh_l = sh_m + kStripes;
    const bool active = threadIdx.x < 256;
    const int c = threadIdx.x % D, stripe = (threadIdx.x / D) % kStripes;
    // two passes, so that the loads of a pass do not wait on the running maximum: first the maximum
    // of the stripe, then the weighted sums
    float mx = -INFINITY, o = 0.f, ls = 0.f;
    if (active) {
#pragma unroll 8
        for (int s = stripe; s < splits; s += kStripes) mx = fmaxf(mx, __ldcg(part_ml + ((size_t)s * BH + head) * 2));
        const float ref = (mx == -INFINITY) ? 0.f : mx;
#pragma unroll 8
        for (int s = stripe; s < splits; s += kStripes) {
            const size_t at = (size_t)s * BH + head;
            const float w = exp2f(__ldcg(part_ml + at * 2) - ref);
            o = fmaf(__ldcg(part_o + at * D + c), w, o);
            ls = fmaf(__ldcg(part_ml + at * 2 + 1), w, ls);
        }
        sh_o[stripe * D + c] = o;
        if (c == 0) { sh_m[stripe] = mx; sh_l[stripe] = ls; }
    }
    __syncthreads();
    if (active && stripe == 0) {
        float mt = -INFINITY;
#pragma unroll
        for (int k = 0; k < kStripes; ++k) mt = fmaxf(mt, sh_m[k]);
        float ot = 0.f, lt = 0.f;
#pragma unroll
        for (int k = 0; k < kStripes; ++k) {
            const float a = exp2f(sh_m[k] - mt);
            ot = fmaf(sh_o[k * D + c], a, ot);
            lt = fmaf(sh_l[k], a, lt);
        }
        out[head * D + c] = from_float<T>(ot / lt);
        if (lse && c == 0) lse[head] = (mt + log2f(lt)) * kLn2;
    }
    __syncthreads();
}

// The CTA that finishes last among the `splits` CTAs of a group of query heads merges their partial results, so
// the merge needs no launch of its own and runs while other heads are still streaming.  No CTA waits for another:
// each one publishes its partials (fence), then adds one to the group's counter (zeroed by the host before the
// launch); whoever reads splits - 1 is the last.
template <typename T, int D>
__device__ __forceinline__ void merge_if_last(unsigned int *counters, const DecodeJob &job, int splits, size_t BH,
                                              const float *part_o, const float *part_ml, T *out, float *lse, float *sh)
{
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int old = atomicAdd(counters + (size_t)job.bkv * gridDim.y + blockIdx.y, 1u);
        s_last = old == (unsigned int)(splits - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int g = 0; g < job.gcount; ++g) merge_head<T, D>(part_o, part_ml, out, lse, splits, BH, job.head0 + g, sh);
}

// ---- variant 1: rows straight from global memory into registers (16-byte streaming loads, kUnroll row
// groups of K and of V in flight per warp).  Few registers when the group is small, so several CTAs
// per SM keep enough bytes in flight: used for one or two query heads per K/V head.
template <typename T, int D, int GC>
__global__ void __launch_bounds__(kThreads)
decode_split_kernel(const T *__restrict__ q, const T *__restrict__ K, const T *__restrict__ V,
                    float *__restrict__ part_o, float *__restrict__ part_ml, T *__restrict__ out, float *__restrict__ lse,
                    unsigned int *__restrict__ counters,
                    int n, int H, int Hkv, int group, int splits, int keys_per_split, size_t BH, float scale_log2)
{
    using State = DecodeState<T, D, GC>;
    constexpr int E = State::E, LPR = State::LPR, RPW = State::RPW;
    const DecodeJob job(splits, GC, group, H, Hkv, n, keys_per_split);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int sub = lane / LPR, l = lane % LPR;          // row of the group, lane of the row
    const T *Kh = K + (size_t)job.bkv * n * D;
    const T *Vh = V + (size_t)job.bkv * n * D;
    State st;
    st.init(q + job.head0 * D, job.gcount, l, scale_log2);
    constexpr int kRowsPerIter = kUnroll * RPW;          // rows one warp consumes per iteration
    for (int base = job.k_begin + warp * kRowsPerIter; base < job.k_end; base += kWarps * kRowsPerIter) {
        uint4 kraw[kUnroll], vraw[kUnroll];
        bool live[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int row = base + u * RPW + sub;
            live[u] = row < job.k_end;
            const size_t off = (size_t)(live[u] ? row : job.k_begin) * D + l * E;
            kraw[u] = __ldcs(reinterpret_cast<const uint4 *>(Kh + off));
            vraw[u] = __ldcs(reinterpret_cast<const uint4 *>(Vh + off));
        }
        st.template consume<kUnroll>(kraw, vraw, live);
    }
    extern __shared__ float sm[];
    st.finish(sm, warp, lane, kWarps, job.gcount, job.head0, job.split, BH, part_o, part_ml, kThreads);
    merge_if_last<T, D>(counters, job, splits, BH, part_o, part_ml, out, lse, sm);
}

// ---- variant 2: the cache segment streams through a shared-memory ring filled by bulk copies (a tile
// of 64 rows of one head is contiguous in memory: one copy per tile and tensor), so the bytes in
// flight are the whole ring whatever the register budget of the consumers: used for groups of four or
// more query heads, whose state (GC x E accumulators and queries per lane) leaves one or two CTAs per SM.
// Warp 8 produces; warps 0-7 each consume 8 rows of every tile.  Every wait is bounded.
constexpr int kRingThreads = kThreads + 32;
constexpr int kTileRows = 64;
// K and V tile per stage; about 190 KB of ring, eight stages at most
template <typename T, int D>
struct Ring {
    static constexpr int kFit = (190 * 1024) / (2 * kTileRows * D * (int)sizeof(T));
    static constexpr int kStages = kFit > 8 ? 8 : kFit;
};

template <typename T, int D, int GC>
__global__ void __launch_bounds__(kRingThreads, 1)
decode_ring_kernel(const T *__restrict__ q, const T *__restrict__ K, const T *__restrict__ V,
                   float *__restrict__ part_o, float *__restrict__ part_ml, T *__restrict__ out, float *__restrict__ lse,
                   unsigned int *__restrict__ counters,
                   int n, int H, int Hkv, int group, int splits, int keys_per_split, size_t BH, float scale_log2,
                   unsigned int *status)
{
    using namespace ptx;
    using State = DecodeState<T, D, GC>;
    constexpr int E = State::E, LPR = State::LPR, RPW = State::RPW;
    constexpr int kStages = Ring<T, D>::kStages;
    constexpr int kRowBytes = D * (int)sizeof(T), kTileBytes = kTileRows * kRowBytes;
    constexpr int U = (kTileRows / kWarps) / RPW;         // row groups per warp and tile
    static_assert(U >= 1, "a warp consumes at least one row group per tile");
    extern __shared__ __align__(128) uint8_t ring[];
    uint64_t *full = reinterpret_cast<uint64_t *>(ring + (size_t)kStages * 2 * kTileBytes);
    uint64_t *empty = full + kStages;
    volatile uint32_t *abortp = reinterpret_cast<uint32_t *>(empty + kStages);

    const DecodeJob job(splits, GC, group, H, Hkv, n, keys_per_split);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int ntiles = job.k_end > job.k_begin ? (job.k_end - job.k_begin + kTileRows - 1) / kTileRows : 0;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, kWarps); }
        *abortp = 0;
        fence_mbar_init();
    }
    __syncthreads();
    State st;
    if (warp == kWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const uint8_t *Kh = reinterpret_cast<const uint8_t *>(K) + ((size_t)job.bkv * n + job.k_begin) * kRowBytes;
            const uint8_t *Vh = reinterpret_cast<const uint8_t *>(V) + ((size_t)job.bkv * n + job.k_begin) * kRowBytes;
            ArmCounts<kStages> armed;     // stages armed for copies into the ring
            for (int t = 0; t < ntiles; ++t) {
                const int s = t % kStages;
                if (t >= kStages && !mbar_wait(empty + s, (t / kStages - 1) & 1, abortp, status, 0x301u)) break;
                const int rows = min(kTileRows, job.k_end - job.k_begin - t * kTileRows);
                const uint32_t bytes = (uint32_t)rows * kRowBytes;
                mbar_arm(full, s, 2 * bytes, armed);
                bulk_load_1d(ring + (size_t)s * 2 * kTileBytes, Kh + (size_t)t * kTileBytes, bytes, full + s);
                bulk_load_1d(ring + (size_t)s * 2 * kTileBytes + kTileBytes, Vh + (size_t)t * kTileBytes, bytes, full + s);
            }
            mbar_drain(full, armed);      // copies still on their way land before the CTA leaves (bounded)
        }
    } else {
        // ----------------------------------------------------------------- consumers
        const int sub = lane / LPR, l = lane % LPR;
        st.init(q + job.head0 * D, job.gcount, l, scale_log2);
        for (int t = 0; t < ntiles; ++t) {
            const int s = t % kStages;
            if (!mbar_wait(full + s, (t / kStages) & 1, abortp, status, 0x302u)) break;
            const uint8_t *tk = ring + (size_t)s * 2 * kTileBytes, *tv = tk + kTileBytes;
            const int row0 = job.k_begin + t * kTileRows;
            uint4 kraw[U], vraw[U];
            bool live[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int r = warp * (kTileRows / kWarps) + u * RPW + sub;      // row of the tile
                live[u] = row0 + r < job.k_end;
                // rows past the segment were not copied: read row 0 of the tile instead (always present)
                const int rr = live[u] ? r : 0;
                kraw[u] = *reinterpret_cast<const uint4 *>(tk + rr * kRowBytes + l * 16);
                vraw[u] = *reinterpret_cast<const uint4 *>(tv + rr * kRowBytes + l * 16);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty + s);      // the tile is in registers: the stage may be refilled
            st.template consume<U>(kraw, vraw, live);
        }
    }
    __syncthreads();       // every consumer is done with the ring: reuse its start for the merge
    if (warp == kWarps) st.init(q + job.head0 * D, 0, 0, 0.f);     // the producer warp holds no state
    st.finish(reinterpret_cast<float *>(ring), warp, lane, kWarps, job.gcount, job.head0, job.split, BH, part_o,
              part_ml, kRingThreads);
    merge_if_last<T, D>(counters, job, splits, BH, part_o, part_ml, out, lse, reinterpret_cast<float *>(ring));
}

// Merge for the tensor-core route: O_part [splits*B, Hkv, G, D] bf16 (each normalised over its own
// segment), L_part [splits, B*Hkv, G] natural-log logsumexp of the segment.  One block per query head.
template <int D>
__global__ void __launch_bounds__(256)
decode_merge_tc_kernel(const __nv_bfloat16 *__restrict__ O_part, const float *__restrict__ L_part,
                       __nv_bfloat16 *__restrict__ out, float *__restrict__ lse, int splits, int B, int Hkv, int G)
{
    constexpr int kStripes = 256 / D;
    __shared__ float sh_o[kStripes][D], sh_m[kStripes], sh_l[kStripes];
    const int head = blockIdx.x;                      // b * H + kvh * G + g
    const int H = Hkv * G;
    const int b = head / H, hq = head - b * H, kvh = hq / G, g = hq - kvh * G;
    const int c = threadIdx.x % D, stripe = threadIdx.x / D;
    float mx = -INFINITY, o = 0.f, ls = 0.f;          // running max of L, sum of weights, weighted output
    for (int s = stripe; s < splits; s += kStripes) {
        const float Ls = L_part[((size_t)s * B * Hkv + (size_t)b * Hkv + kvh) * G + g];
        const float mn = fmaxf(mx, Ls);
        const float a = __expf(mx - mn), w = __expf(Ls - mn);
        const float ov = __bfloat162float(O_part[((((size_t)s * B + b) * Hkv + kvh) * G + g) * D + c]);
        o = o * a + ov * w;
        ls = ls * a + w;
        mx = mn;
    }
    sh_o[stripe][c] = o;
    if (c == 0) { sh_m[stripe] = mx; sh_l[stripe] = ls; }
    __syncthreads();
    if (stripe == 0) {
        float mt = -INFINITY;
#pragma unroll
        for (int k = 0; k < kStripes; ++k) mt = fmaxf(mt, sh_m[k]);
        float ot = 0.f, lt = 0.f;
#pragma unroll
        for (int k = 0; k < kStripes; ++k) {
            const float a = __expf(sh_m[k] - mt);
            ot = fmaf(sh_o[k][c], a, ot);
            lt = fmaf(sh_l[k], a, lt);
        }
        out[(size_t)head * D + c] = __float2bfloat16_rn(ot / lt);
        if (lse && c == 0) lse[head] = mt + __logf(lt);
    }
}

int group_chunk(int group) { return group >= 8 ? 8 : group >= 4 ? 4 : group >= 2 ? 2 : 1; }

template <typename T, int D, int GC>
cudaError_t launch_split(const DecodeProblem &p, const void *q, const void *K, const void *V, float *part_o,
                         float *part_ml, void *out, float *lse, unsigned int *counters, int splits, int keys_per_split,
                         cudaStream_t st)
{
    const int group = p.H / p.Hkv;
    dim3 grid((unsigned)(p.B * p.Hkv * splits), (unsigned)((group + GC - 1) / GC));
    size_t merge_smem = (size_t)kWarps * GC * (D + 2) * sizeof(float);       // warps' states; then the stripes of merge_head
    if (merge_smem < (size_t)(256 / D) * (D + 2) * sizeof(float)) merge_smem = (size_t)(256 / D) * (D + 2) * sizeof(float);
    // one counter per (K/V head, chunk of query heads): the last of its CTAs to finish merges
    cudaError_t ce = cudaMemsetAsync(counters, 0, (size_t)p.B * p.Hkv * grid.y * sizeof(unsigned int), st);
    if (ce != cudaSuccess) return ce;
    LaunchScope scope(MOA_KERNEL_OTHER, st);
    if (GC >= 4) {
        constexpr int kStages = Ring<T, D>::kStages;
        const size_t smem = (size_t)kStages * 2 * kTileRows * D * sizeof(T) + 2 * kStages * sizeof(uint64_t) + 16;
        cudaError_t e = cudaFuncSetAttribute(decode_ring_kernel<T, D, GC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(smem > merge_smem ? smem : merge_smem));
        if (e != cudaSuccess) return e;
        decode_ring_kernel<T, D, GC><<<grid, kRingThreads, smem > merge_smem ? smem : merge_smem, st>>>(
            (const T *)q, (const T *)K, (const T *)V, part_o, part_ml, (T *)out, lse, counters, p.n, p.H, p.Hkv, group, splits,
            keys_per_split, (size_t)p.B * p.H, p.scale * kLog2e, device_status_ptr());
        return cudaGetLastError();
    }
    cudaError_t e = cudaFuncSetAttribute(decode_split_kernel<T, D, GC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)merge_smem);
    if (e != cudaSuccess) return e;
    decode_split_kernel<T, D, GC><<<grid, kThreads, merge_smem, st>>>((const T *)q, (const T *)K, (const T *)V, part_o,
                                                                      part_ml, (T *)out, lse, counters, p.n, p.H, p.Hkv,
                                                                      group, splits, keys_per_split, (size_t)p.B * p.H,
                                                                      p.scale * kLog2e);
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch_decode(const DecodeProblem &p, const void *q, const void *K, const void *V, void *out, float *lse,
                          float *ws, cudaStream_t st)
{
    const int splits = decode_splits(p);
    const int keys_per_split = (p.n + splits - 1) / splits;
    const size_t BH = (size_t)p.B * p.H;
    float *part_o = ws, *part_ml = ws + (size_t)splits * BH * D;
    unsigned int *counters = reinterpret_cast<unsigned int *>(part_ml + (size_t)splits * BH * 2);
    const int gc = group_chunk(p.H / p.Hkv);
    // the merge of a head's segments is done by the last of its CTAs to finish (no merge launch)
    return gc == 8 ? launch_split<T, D, 8>(p, q, K, V, part_o, part_ml, out, lse, counters, splits, keys_per_split, st)
         : gc == 4 ? launch_split<T, D, 4>(p, q, K, V, part_o, part_ml, out, lse, counters, splits, keys_per_split, st)
         : gc == 2 ? launch_split<T, D, 2>(p, q, K, V, part_o, part_ml, out, lse, counters, splits, keys_per_split, st)
                   : launch_split<T, D, 1>(p, q, K, V, part_o, part_ml, out, lse, counters, splits, keys_per_split, st);
}

}  // namespace

// Groups of 4 to 128 query heads over a bf16 cache go through the tensor-core forward kernel (the
// group is its query tile); everything else through the CUDA-core streaming kernels above.
static bool decode_uses_tc(const DecodeProblem &p, int dtype)
{
    const int group = p.H / p.Hkv;
    return dtype == MOA_BF16 && group >= 4 && group <= 128 && p.scale > 0.f;
}

// Tensor-core route: key tiles of 128 per CTA segment, one CTA per SM at a time.  All CTAs are equal,
// so the run takes ceil(CTAs / SMs) rounds of (fixed cost + tiles per segment); the fixed cost of a CTA
// (pipeline fill, epilogue) was measured at about 3.5 tile times.  Take the segment count that
// minimises rounds x (3.5 + tiles).
static void decode_tc_splits(const DecodeProblem &p, int *splits, int *tiles_per_split)
{
    const int nkt = (p.n + 127) / 128;
    const long long base = (long long)p.B * p.Hkv, sms = device_info().sms;
    long long hi = (32LL * sms + base - 1) / base;
    if (hi > nkt) hi = nkt;
    if (hi < 1) hi = 1;
    long long best = 1;
    double best_cost = 1e300;
    for (long long s = 1; s <= hi; ++s) {
        const int tps = (int)((nkt + s - 1) / s);
        const long long real = (nkt + tps - 1) / tps;      // segments that get at least one tile
        const long long rounds = (base * real + sms - 1) / sms;
        const double cost = (double)rounds * (3.5 + tps);
        if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
    }
    const int tps = (int)((nkt + best - 1) / best);
    *tiles_per_split = tps;
    *splits = (nkt + tps - 1) / tps;          // every segment has at least one tile
}

// Segments of the cache per K/V head: enough CTAs to fill the GPU a few times over, each with at
// least 256 keys.
int decode_splits(const DecodeProblem &p)
{
    const int group = p.H / p.Hkv;
    const int gc = group >= 8 ? 8 : group >= 4 ? 4 : group >= 2 ? 2 : 1;
    const long long ctas_per_split = (long long)p.B * p.Hkv * ((group + gc - 1) / gc);
    long long s = (4LL * device_info().sms + ctas_per_split - 1) / ctas_per_split;
    const long long cap = (p.n + 255) / 256;
    if (s > cap) s = cap;
    if (s < 1) s = 1;
    if (s > 1024) s = 1024;
    return (int)s;
}

size_t decode_workspace_bytes(const DecodeProblem &p, int dtype)
{
    if (decode_uses_tc(p, dtype)) {
        int splits, tps;
        decode_tc_splits(p, &splits, &tps);
        const size_t heads = (size_t)splits * p.B * p.H;
        return ((heads * p.d * 2 + 255) / 256) * 256 + heads * sizeof(float);
    }
    // partial results of the segments, then one counter per (K/V head, chunk of query heads)
    return (size_t)decode_splits(p) * p.B * p.H * (p.d + 2) * sizeof(float) + (size_t)p.B * p.H * sizeof(unsigned int);
}

cudaError_t decode_attn(const DecodeProblem &p, int dtype, const void *q, const void *K, const void *V, void *out,
                        float *lse, void *ws, cudaStream_t st)
{
    if (decode_uses_tc(p, dtype)) {
        int splits, tps;
        decode_tc_splits(p, &splits, &tps);
        const int G = p.H / p.Hkv;
        const size_t heads = (size_t)splits * p.B * p.H;
        void *O_part = ws;
        float *L_part = reinterpret_cast<float *>((char *)ws + ((heads * p.d * 2 + 255) / 256) * 256);
        cudaError_t e = tc_fwd_decode(p.B, p.Hkv, G, p.n, p.d, p.scale, q, K, V, O_part, L_part, splits, tps, st);
        if (e != cudaSuccess) return e;
        LaunchScope scope(MOA_KERNEL_OTHER, st);
        if (p.d == 64)
            decode_merge_tc_kernel<64><<<(unsigned)(p.B * p.H), 256, 0, st>>>((const __nv_bfloat16 *)O_part, L_part,
                                                                              (__nv_bfloat16 *)out, lse, splits, p.B, p.Hkv, G);
        else
            decode_merge_tc_kernel<128><<<(unsigned)(p.B * p.H), 256, 0, st>>>((const __nv_bfloat16 *)O_part, L_part,
                                                                               (__nv_bfloat16 *)out, lse, splits, p.B, p.Hkv, G);
        return cudaGetLastError();
    }
    float *wsf = (float *)ws;
    if (dtype == MOA_F32) {
        if (p.d == 64) return launch_decode<float, 64>(p, q, K, V, out, lse, wsf, st);
        if (p.d == 128) return launch_decode<float, 128>(p, q, K, V, out, lse, wsf, st);
    } else {
        if (p.d == 64) return launch_decode<__nv_bfloat16, 64>(p, q, K, V, out, lse, wsf, st);
        if (p.d == 128) return launch_decode<__nv_bfloat16, 128>(p, q, K, V, out, lse, wsf, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace moa
