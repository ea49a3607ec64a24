// Speculative sampling (Section 2.3 / Algorithm 1, accept-adjust-draw part),
// plain standardised sampling (Section 2.2) and the method's uniforms.
//
// spec_verify_sample is two kernels on one stream:
//   1. verify_stats_kernel streams every logit of p_1..p_{gamma+1} and
//      q_1..q_gamma exactly once from HBM.  A CTA reduces one chunk of one row
//      to (max, sum exp) with an online rescale, and also picks up the row's
//      logit at the drafted token.  No CTA talks to another: the kernel is a
//      pure map-reduce and runs at streaming bandwidth.
//   2. verify_finish_kernel, one CTA per sequence, merges the chunk statistics,
//      runs the gamma accept tests, and re-reads only row n+1 of p and q (still
//      in L2) to normalise the residual max(0, p - q) and draw from it by
//      inverse CDF.  It is chained with programmatic dependent launch, so its
//      launch latency and prologue overlap the tail of the first kernel.
#include <algorithm>
#include <cfloat>
#include <mutex>

#include <cooperative_groups.h>

#include "model.cuh"

namespace cg = cooperative_groups;

namespace spec {
namespace {

constexpr int kStatThreads = 512;
constexpr int kStatWarps = kStatThreads / 32;
constexpr int kUnroll = 4;              // 128-bit loads in flight per thread while streaming
constexpr int kMinChunkGroups = 1024;   // a CTA streams at least 4096 logits (unless the row is shorter)
constexpr int kTargetCtas = 148 * 24;   // about six waves of resident CTAs, so that the last wave costs little
constexpr int kFinishThreads = 512;
constexpr int kCdfBatch = 8;            // groups fetched per thread before any is consumed (inverse CDF, one CTA)
constexpr int kClusterCdfBatch = 4;     // the same when a cluster shares the row
constexpr int kWalkBatch = 4;           // 128-element steps fetched at once by the final walk
constexpr int kMaxCluster = 4;          // CTAs per sequence in the finishing kernel
constexpr int kSampleThreads = 512;
constexpr int kMaxGamma = 64;
constexpr int kMaxRows = 2 * kMaxGamma + 1;
constexpr float kLog2e = 1.4426950408889634f;

// 2^x with one MUFU instruction (2 ulp; results below 2^-126 flush to zero,
// which is far below anything a sum over the vocabulary can see).
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// A row of fp32 logits addressed in groups of four elements.  VEC: the vocabulary
// is a multiple of four and every row starts on a 16-byte boundary, so a group
// is one unconditional 128-bit load.  Otherwise four guarded scalar loads, with
// elements past the end of the row reading as `pad`.
template <bool VEC>
struct Row {
    const float* base;
    int vocab;

    __device__ __forceinline__ float4 load(int g, float pad) const {
        if (VEC) return __ldg(reinterpret_cast<const float4*>(base) + g);
        const int j = 4 * g;
        float4 v;
        v.x = j + 0 < vocab ? __ldg(base + j + 0) : pad;
        v.y = j + 1 < vocab ? __ldg(base + j + 1) : pad;
        v.z = j + 2 < vocab ? __ldg(base + j + 2) : pad;
        v.w = j + 3 < vocab ? __ldg(base + j + 3) : pad;
        return v;
    }
};

template <bool VEC>
__device__ __forceinline__ Row<VEC> make_row(const float* base, int vocab) {
    Row<VEC> r;
    r.base = base;
    r.vocab = vocab;
    return r;
}

// Weight functors for the inverse-CDF draw.  fetch() only loads, weigh() only
// computes, so that a caller can put several fetches in flight before it
// consumes any of them.

// Unnormalised softmax weights exp((l - max) / T) of one row; c2 = log2(e) / T.
template <bool VEC>
struct PlainWeights {
    struct Raw { float4 a; };
    Row<VEC> p;
    float max_p, c2;
    __device__ __forceinline__ Raw fetch(int g) const { return Raw{p.load(g, -INFINITY)}; }
    __device__ __forceinline__ Raw nothing() const {
        return Raw{make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY)};
    }
    __device__ __forceinline__ float one(float lp) const { return fast_exp2((lp - max_p) * c2); }
    __device__ __forceinline__ float4 weigh(const Raw& r) const {
        return make_float4(one(r.a.x), one(r.a.y), one(r.a.z), one(r.a.w));
    }
    __device__ __forceinline__ float4 operator()(int g) const { return weigh(fetch(g)); }
};

// max(0, p - q) with p, q the normalised softmaxes of two rows (Algorithm 1's
// adjusted distribution before normalisation).
template <bool VEC>
struct ResidualWeights {
    struct Raw { float4 a, b; };
    Row<VEC> p, q;
    float max_p, max_q, inv_sum_p, inv_sum_q, c2;
    __device__ __forceinline__ Raw fetch(int g) const { return Raw{p.load(g, -INFINITY), q.load(g, -INFINITY)}; }
    __device__ __forceinline__ Raw nothing() const {
        const float4 z = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        return Raw{z, z};
    }
    __device__ __forceinline__ float one(float lp, float lq) const {
        const float pv = fast_exp2((lp - max_p) * c2) * inv_sum_p;
        const float qv = fast_exp2((lq - max_q) * c2) * inv_sum_q;
        return fmaxf(0.0f, pv - qv);
    }
    __device__ __forceinline__ float4 weigh(const Raw& r) const {
        return make_float4(one(r.a.x, r.b.x), one(r.a.y, r.b.y), one(r.a.z, r.b.z), one(r.a.w, r.b.w));
    }
    __device__ __forceinline__ float4 operator()(int g) const { return weigh(fetch(g)); }
};

template <int WARPS>
struct CdfScratch {
    float part[WARPS];              // per-warp totals of the level being scanned
    float all[kMaxCluster * WARPS];  // the same for every CTA of a cluster
    float pick_before, pick_total;   // outcome of the cluster-wide scan
    int pick_part_index, pick_hit;
    int result;
    int last_positive;
};

// Sum of the weights of groups [g0, g1) by one warp, lane-strided so that every
// load instruction covers 512 contiguous bytes; BATCH fetches are in flight
// per lane before any is consumed.
template <int BATCH, class Weights>
__device__ __forceinline__ float warp_range_sum(const Weights& w, int g0, int g1, int lane) {
    float acc = 0.0f;
    for (int base = g0 + lane; base < g1; base += 32 * BATCH) {
        typename Weights::Raw raw[BATCH];
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
            const int g = base + 32 * i;
            raw[i] = g < g1 ? w.fetch(g) : w.nothing();
        }
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
            const float4 v = w.weigh(raw[i]);
            acc += (v.x + v.y) + (v.z + v.w);
        }
    }
    return warp_sum(acc);
}

// Which of `count` consecutive parts holds `target`: the first part whose
// running sum exceeds it (the same arithmetic in every thread, so every thread
// agrees).  Returns -1 if none does; *before gets the running sum in front of
// the chosen part; *fallback is the last part with positive weight (0 if none),
// for the case where rounding leaves no part above the target.
template <class PartAt>
__device__ __forceinline__ int pick_part(PartAt part_at, int count, float target, float* before, int* fallback) {
    float run = 0.0f;
    int hit = -1, last = 0;
    for (int i = 0; i < count; ++i) {
        const float v = part_at(i);
        const float next = run + v;
        if (hit < 0 && next > target) {
            hit = i;
            *before = run;
        }
        if (v > 0.0f) last = i;
        run = next;
    }
    *fallback = last;
    return hit;
}

// The draw inside one contiguous range of groups [r0, r1) by a whole CTA: `rem`
// is the target minus the weight in front of the range.  Long ranges are first
// cut into one sub-range per warp; warp 0 then walks the chosen (sub-)range 128
// elements at a time with a warp scan.  With want_hit false the answer is the
// last index of the range with positive weight.  Returns the index (or -1) to
// all threads.
template <int WARPS, class Weights>
__device__ int locate_in_range(const Weights& w, int r0, int r1, float rem, bool want_hit, CdfScratch<WARPS>& s) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        s.result = -1;
        s.last_positive = -1;
    }
    if (r1 - r0 > 4 * 32) {  // uniform across the CTA
        const int sub = (r1 - r0 + WARPS - 1) / WARPS;
        const int g0 = min(r1, r0 + warp * sub), g1 = min(r1, g0 + sub);
        const float acc = warp_range_sum<2>(w, g0, g1, lane);
        __syncthreads();  // previous users of s.part are done
        if (lane == 0) s.part[warp] = acc;
        __syncthreads();
        float before = 0.0f;
        int fallback = 0;
        int hit = pick_part([&](int i) { return s.part[i]; }, WARPS, rem, &before, &fallback);
        if (!want_hit || hit < 0) {
            want_hit = false;
            hit = fallback;
        }
        rem -= before;
        r0 = min(r1, r0 + hit * sub);
        r1 = min(r1, r0 + sub);
    }
    __syncthreads();
    if (warp == 0) {
        float run = 0.0f;
        int found = -1, last_pos = -1;
        for (int gb = r0; gb < r1 && found < 0; gb += 32 * kWalkBatch) {
            typename Weights::Raw raw[kWalkBatch];  // the whole batch is fetched before the serial scan
#pragma unroll
            for (int i = 0; i < kWalkBatch; ++i) {
                const int g = gb + 32 * i + lane;
                raw[i] = g < r1 ? w.fetch(g) : w.nothing();
            }
#pragma unroll
            for (int i = 0; i < kWalkBatch; ++i) {
                const int gs = gb + 32 * i;
                if (gs >= r1 || found >= 0) break;
                const float4 v = w.weigh(raw[i]);
                const float mine = (v.x + v.y) + (v.z + v.w);
                const float incl = warp_inclusive_scan(mine, lane);
                const unsigned over = want_hit ? __ballot_sync(kFullMask, run + incl > rem) : 0u;
                const unsigned pos = __ballot_sync(kFullMask, mine > 0.0f);
                if (pos) {
                    const int pl = 31 - __clz(pos);  // last lane with positive weight in this step
                    const float py = __shfl_sync(kFullMask, v.y, pl), pz = __shfl_sync(kFullMask, v.z, pl),
                                pw = __shfl_sync(kFullMask, v.w, pl);
                    const int pg = 4 * (gs + pl);
                    last_pos = pw > 0.f ? pg + 3 : pz > 0.f ? pg + 2 : py > 0.f ? pg + 1 : pg;
                }
                if (over) {
                    const int hl = __ffs(over) - 1;
                    const float excl = __shfl_sync(kFullMask, incl - mine, hl) + run;
                    const float hx = __shfl_sync(kFullMask, v.x, hl), hy = __shfl_sync(kFullMask, v.y, hl),
                                hz = __shfl_sync(kFullMask, v.z, hl);
                    const int hg = 4 * (gs + hl);
                    float c = excl + hx;
                    if (c > rem) found = hg;
                    else if ((c += hy) > rem) found = hg + 1;
                    else if ((c += hz) > rem) found = hg + 2;
                    else found = hg + 3;
                }
                run += __shfl_sync(kFullMask, incl, 31);
            }
        }
        if (lane == 0) {
            s.result = found;
            s.last_positive = last_pos;
        }
    }
    __syncthreads();
    const int k = s.result >= 0 ? s.result : s.last_positive;
    __syncthreads();  // scratch may be reused by the caller
    return k;
}

// Inverse-CDF draw by one CTA of 32 * WARPS threads: the smallest index k whose
// running weight sum exceeds u * (sum of all weights); the last index with
// positive weight if rounding leaves none.  The vocabulary is cut into WARPS
// contiguous segments (one per warp); the segment holding the target is then
// resolved by locate_in_range.  Returns the index to all threads, the total
// through *total_out.
template <int WARPS, class Weights>
__device__ int block_inverse_cdf(const Weights& w, int vocab, float u, CdfScratch<WARPS>& s, float* total_out) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int groups = (vocab + 3) >> 2;
    const int seg = (groups + WARPS - 1) / WARPS;
    const int g0 = min(groups, warp * seg), g1 = min(groups, g0 + seg);
    const float acc = warp_range_sum<kCdfBatch>(w, g0, g1, lane);
    if (lane == 0) s.part[warp] = acc;
    __syncthreads();
    float total = 0.0f;
#pragma unroll
    for (int i = 0; i < WARPS; ++i) total += s.part[i];
    const float target = u * total;
    float before = 0.0f;
    int fallback = 0;
    int hit = pick_part([&](int i) { return s.part[i]; }, WARPS, target, &before, &fallback);
    const bool want_hit = hit >= 0;
    if (!want_hit) hit = fallback;
    const int r0 = min(groups, hit * seg), r1 = min(groups, r0 + seg);
    const int k = locate_in_range<WARPS>(w, r0, r1, target - before, want_hit, s);
    *total_out = total;
    return max(0, min(k, vocab - 1));
}

// The same draw by a thread-block cluster: CTA `rank` of `nctas` owns a
// contiguous slice of the vocabulary, the per-warp totals of all CTAs are read
// through distributed shared memory, and only the CTA whose slice holds the
// target goes on to resolve it.  Returns the index in that CTA and -1 in the
// others; the total is returned to all.
template <int WARPS, class Weights>
__device__ int cluster_inverse_cdf(const Weights& w, int vocab, float u, CdfScratch<WARPS>& s, float* total_out) {
    cg::cluster_group cluster = cg::this_cluster();
    const int nctas = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int groups = (vocab + 3) >> 2;
    const int slice = (groups + nctas - 1) / nctas;
    const int seg = (slice + WARPS - 1) / WARPS;
    auto seg_begin = [&](int part) {  // part = cta * WARPS + warp
        const int c0 = min(groups, (part / WARPS) * slice), c1 = min(groups, c0 + slice);
        return min(c1, c0 + (part % WARPS) * seg);
    };
    auto seg_end = [&](int part) {
        const int c0 = min(groups, (part / WARPS) * slice), c1 = min(groups, c0 + slice);
        return min(c1, seg_begin(part) + seg);
    };
    const int mine = rank * WARPS + warp;
    const float acc = warp_range_sum<kClusterCdfBatch>(w, seg_begin(mine), seg_end(mine), lane);
    if (lane == 0) s.part[warp] = acc;
    cluster.sync();
    // warp 0 copies every CTA's totals into this CTA's shared memory ...
    const int parts = nctas * WARPS;
    if (warp == 0)
        for (int i = lane; i < parts; i += 32) s.all[i] = cluster.map_shared_rank(s.part, i / WARPS)[i % WARPS];
    __syncthreads();
    // ... and scans them: lane l takes the consecutive parts [l*per, (l+1)*per)
    if (warp == 0) {
        const int per = (parts + 31) / 32;
        float mine_sum = 0.0f;
        for (int i = lane * per; i < min(parts, (lane + 1) * per); ++i) mine_sum += s.all[i];
        const float incl = warp_inclusive_scan(mine_sum, lane);
        const float tot = __shfl_sync(kFullMask, incl, 31);
        const float tgt = u * tot;
        const unsigned over = __ballot_sync(kFullMask, incl > tgt);
        const unsigned pos = __ballot_sync(kFullMask, mine_sum > 0.0f);
        const int hl = over ? __ffs(over) - 1 : (pos ? 31 - __clz(pos) : 0);
        if (lane == hl) {
            float run = incl - mine_sum;
            int hit = -1, last = lane * per;
            for (int i = lane * per; i < min(parts, (lane + 1) * per); ++i) {
                if (s.all[i] > 0.0f) last = i;
                if (over && hit < 0 && run + s.all[i] > tgt) { hit = i; break; }
                run += s.all[i];
            }
            if (hit < 0) { hit = last; s.pick_hit = 0; run = 0.0f; } else { s.pick_hit = 1; }
            s.pick_part_index = hit;
            s.pick_before = run;
            s.pick_total = tot;
        }
    }
    __syncthreads();
    const float total = s.pick_total;
    const float target = u * total;
    const float before = s.pick_before;
    int hit = s.pick_part_index;
    const bool want_hit_flag = s.pick_hit != 0;
    cluster.sync();  // nobody reads another CTA's totals after this point
    const bool want_hit = want_hit_flag;
    *total_out = total;
    if (hit / WARPS != rank) return -1;
    const int k = locate_in_range<WARPS>(w, seg_begin(hit), seg_end(hit), target - before, want_hit, s);
    return max(0, min(k, vocab - 1));
}

// (max, lowest index attaining it) across a CTA of 32 * WARPS threads; the
// result is valid in thread 0.
template <int WARPS>
__device__ __forceinline__ void block_argmax(float& m, int& arg, float* red, int* red_i) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(kFullMask, m, o);
        const int oa = __shfl_xor_sync(kFullMask, arg, o);
        if (om > m || (om == m && oa < arg)) { m = om; arg = oa; }
    }
    if (lane == 0) { red[warp] = m; red_i[warp] = arg; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < WARPS; ++i)
            if (red[i] > m || (red[i] == m && red_i[i] < arg)) { m = red[i]; arg = red_i[i]; }
    }
}

// One chunk of one row, as written by verify_stats_kernel.
struct __align__(16) ChunkStat {
    float max;     // chunk maximum
    float aux;     // T > 0: sum exp((l - max) / T) over the chunk; T = 0: argmax index as int bits
    float xlogit;  // the row's logit at the drafted token, if that token falls in this chunk
    float pad;
};

// grid = (chunks, rows, batch); rows = 2*gamma+1 (T > 0: p_1..p_{gamma+1}, q_1..q_gamma)
// or gamma+1 (T = 0: only p is read).
template <bool GREEDY, bool VEC>
__global__ void __launch_bounds__(kStatThreads)
verify_stats_kernel(const float* __restrict__ target_logits, const float* __restrict__ draft_logits,
                    const int32_t* __restrict__ draft_tokens, int gamma, int vocab, float c2,
                    ChunkStat* __restrict__ stats) {
    __shared__ float red[kStatWarps];
    __shared__ float red_s[kStatWarps];
    __shared__ int red_i[kStatWarps];
    pdl_trigger();  // the finishing kernel's CTAs may take their places as this grid drains
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunk = blockIdx.x, chunks = gridDim.x;
    const int row = blockIdx.y, rows = gridDim.y;
    const int b = blockIdx.z;

    const float* src = row <= gamma
        ? target_logits + (static_cast<size_t>(b) * (gamma + 1) + row) * vocab
        : draft_logits + (static_cast<size_t>(b) * gamma + (row - gamma - 1)) * vocab;
    const Row<VEC> r = make_row<VEC>(src, vocab);
    const int groups = (vocab + 3) >> 2;
    const int per_chunk = (groups + chunks - 1) / chunks;
    const int g0 = chunk * per_chunk;
    const int g1 = min(groups, g0 + per_chunk);

    // The drafted token this row is tested at (none for p_{gamma+1}): thread 0
    // fetches the row's logit there if it lies in this chunk, so the accept test
    // needs no further trip to memory.
    float xlogit = 0.0f;
    if (tid == 0 && !GREEDY && row != gamma) {
        const int x = draft_tokens[static_cast<size_t>(b) * gamma + (row < gamma ? row : row - gamma - 1)];
        if (x >= 4 * g0 && x < min(vocab, 4 * g1)) xlogit = __ldg(src + x);
    }

    // Every thread streams groups g0+tid, g0+tid+T, ... with kUnroll 128-bit
    // loads in flight and keeps a running (max, sum exp) pair that is rescaled
    // when the maximum moves; one block-wide merge at the end.
    constexpr float kPad = -INFINITY;
    float m = -FLT_MAX;  // finite, so that (m - new_max) never becomes inf - inf
    float s = 0.0f;
    int arg = 0x7fffffff;
    for (int base = g0 + tid; base < g1; base += kUnroll * kStatThreads) {
        float4 v[kUnroll];
#pragma unroll
        for (int i = 0; i < kUnroll; ++i) {
            const int g = base + i * kStatThreads;
            v[i] = g < g1 ? r.load(g, kPad) : make_float4(kPad, kPad, kPad, kPad);
        }
        if (GREEDY) {
#pragma unroll
            for (int i = 0; i < kUnroll; ++i) {
                const int j = 4 * (base + i * kStatThreads);  // indices grow with i: '>' keeps the lowest on ties
                if (v[i].x > m) { m = v[i].x; arg = j; }
                if (v[i].y > m) { m = v[i].y; arg = j + 1; }
                if (v[i].z > m) { m = v[i].z; arg = j + 2; }
                if (v[i].w > m) { m = v[i].w; arg = j + 3; }
            }
        } else {
            float bm = m;
#pragma unroll
            for (int i = 0; i < kUnroll; ++i)
                bm = fmaxf(bm, fmaxf(fmaxf(v[i].x, v[i].y), fmaxf(v[i].z, v[i].w)));
            s *= fast_exp2((m - bm) * c2);
            m = bm;
#pragma unroll
            for (int i = 0; i < kUnroll; ++i)
                s += (fast_exp2((v[i].x - m) * c2) + fast_exp2((v[i].y - m) * c2)) +
                     (fast_exp2((v[i].z - m) * c2) + fast_exp2((v[i].w - m) * c2));
        }
    }
    ChunkStat* out = stats + (static_cast<size_t>(b) * rows + row) * chunks + chunk;
    if (GREEDY) {
        block_argmax<kStatWarps>(m, arg, red, red_i);
        if (tid == 0) *reinterpret_cast<float4*>(out) = make_float4(m, __int_as_float(arg), 0.0f, 0.0f);
    } else {
        const float wm = warp_max(m);
        s = warp_sum(s * fast_exp2((m - wm) * c2));
        if (lane == 0) { red[warp] = wm; red_s[warp] = s; }
        __syncthreads();
        if (tid == 0) {
            float bm = red[0];
#pragma unroll
            for (int i = 1; i < kStatWarps; ++i) bm = fmaxf(bm, red[i]);
            float t = 0.0f;
#pragma unroll
            for (int i = 0; i < kStatWarps; ++i) t += red_s[i] * fast_exp2((red[i] - bm) * c2);
            *reinterpret_cast<float4*>(out) = make_float4(bm, t, xlogit, 0.0f);
        }
    }
}

struct FinishShared {
    float row_max[kMaxRows];
    float row_aux[kMaxRows];
    float row_x[kMaxRows];
    CdfScratch<kFinishThreads / 32> cdf;
    float u_final;
    int n;
};

// grid = batch * cluster size, one thread-block cluster per sequence.  Everything
// after the statistics: merge, accept tests, adjusted distribution, draw.  The
// cheap decision part is repeated in every CTA of the cluster; the pass over
// row n+1 is split between them.
template <bool GREEDY, bool VEC>
__global__ void __launch_bounds__(kFinishThreads, 2)
verify_finish_kernel(const float* __restrict__ target_logits, const float* __restrict__ draft_logits,
                     const int32_t* __restrict__ draft_tokens, const float* __restrict__ uniforms, int gamma,
                     int vocab, float inv_t, int chunks, int cluster_size, const ChunkStat* __restrict__ stats,
                     const float* __restrict__ final_uniforms, float lenience, int32_t* __restrict__ n_accepted,
                     int32_t* __restrict__ next_token) {
    __shared__ FinishShared sh;
    const int tid = threadIdx.x;
    const int b = blockIdx.x / cluster_size;
    const int rank = blockIdx.x % cluster_size;
    const int rows = GREEDY ? gamma + 1 : 2 * gamma + 1;
    const float c2 = inv_t * kLog2e;
    const float* tl = target_logits + static_cast<size_t>(b) * (gamma + 1) * vocab;
    const float* ql = GREEDY ? nullptr : draft_logits + static_cast<size_t>(b) * gamma * vocab;
    const int groups = (vocab + 3) >> 2;
    const int per_chunk = (groups + chunks - 1) / chunks;

    // Inputs that the statistics kernel does not produce can be fetched before
    // waiting for it.
    float my_uniform = 0.5f;
    if (!GREEDY && tid <= gamma) my_uniform = __ldg(uniforms + static_cast<size_t>(b) * (gamma + 1) + tid);
    int my_x = -1;
    if (tid < rows && tid != gamma)
        my_x = draft_tokens[static_cast<size_t>(b) * gamma + (tid < gamma ? tid : tid - gamma - 1)];
    // lenient argmax decoding compares the target's logit at the drafted token with the row maximum
    float my_xlogit = 0.0f;
    if (GREEDY && lenience < 1.0f && tid < gamma && my_x >= 0 && my_x < vocab) my_xlogit = __ldg(tl + static_cast<size_t>(tid) * vocab + my_x);
    pdl_trigger();
    pdl_wait();

    // merge the chunk statistics of row `tid` (four loads in flight at a time)
    if (tid < rows) {
        const ChunkStat* st_r = stats + (static_cast<size_t>(b) * rows + tid) * chunks;
        float M = -FLT_MAX, A = 0.0f, X = 0.0f;
        int best = 0x7fffffff;
        const int xchunk = (my_x >= 0 && my_x < vocab) ? (my_x >> 2) / per_chunk : -1;
        for (int c0 = 0; c0 < chunks; c0 += 4) {
            float4 st[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                st[i] = c0 + i < chunks ? __ldcg(reinterpret_cast<const float4*>(st_r + c0 + i))
                                        : make_float4(-FLT_MAX, __int_as_float(0x7fffffff), 0.0f, 0.0f);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (c0 + i >= chunks) break;
                if (GREEDY) {
                    const int ci = __float_as_int(st[i].y);
                    if (st[i].x > M || (st[i].x == M && ci < best)) { M = st[i].x; best = ci; }
                } else {
                    const float nm = fmaxf(M, st[i].x);
                    A = A * fast_exp2((M - nm) * c2) + st[i].y * fast_exp2((st[i].x - nm) * c2);
                    M = nm;
                    if (c0 + i == xchunk) X = st[i].z;
                }
            }
        }
        sh.row_max[tid] = M;
        sh.row_aux[tid] = GREEDY ? __int_as_float(best) : A;
        sh.row_x[tid] = X;
    }
    if (tid == 0) sh.n = gamma;
    __syncthreads();

    // the gamma accept tests (Algorithm 1: n = index of the first rejection)
    if (tid < gamma) {
        bool reject = true;
        if (my_x >= 0 && my_x < vocab) {
            if (GREEDY) {
                // strict: x must be the lowest-index maximum; lenient (Appendix A.5 at T = 0):
                // p(x) >= l max p before standardising, i.e. logit(x) >= max logit + ln l
                reject = lenience < 1.0f ? !(my_xlogit - sh.row_max[tid] - logf(lenience) >= 0.0f)
                                         : my_x != __float_as_int(sh.row_aux[tid]);
            } else {
                const float ep = expf((sh.row_x[tid] - sh.row_max[tid]) * inv_t);
                const float eq = expf((sh.row_x[gamma + 1 + tid] - sh.row_max[gamma + 1 + tid]) * inv_t);
                // r * l * q(x) > p(x) with p = ep / Sp, q = eq / Sq, cross-multiplied (l = 1: Algorithm 1)
                reject = my_uniform * lenience * eq * sh.row_aux[tid] > ep * sh.row_aux[gamma + 1 + tid];
            }
        }
        if (reject) atomicMin(&sh.n, tid);
    }
    if (tid == gamma) sh.u_final = my_uniform;
    __syncthreads();
    const int n = sh.n;

    int token = -1;
    if (GREEDY) {
        if (rank == 0) token = __float_as_int(sh.row_aux[n]);
    } else {
        constexpr int W = kFinishThreads / 32;
        // The generation loop keys the final draw by the position it decides, which
        // depends on n: it passes one candidate uniform per possible n.
        const float u = final_uniforms ? __ldg(final_uniforms + static_cast<size_t>(b) * (gamma + 1) + n) : sh.u_final;
        PlainWeights<VEC> pw;
        pw.p = make_row<VEC>(tl + static_cast<size_t>(n) * vocab, vocab);
        pw.max_p = sh.row_max[n];
        pw.c2 = c2;
        float total = 0.0f;
        bool plain = n == gamma;
        if (!plain) {
            ResidualWeights<VEC> rw;
            rw.p = pw.p;
            rw.q = make_row<VEC>(ql + static_cast<size_t>(n) * vocab, vocab);
            rw.max_p = sh.row_max[n];
            rw.max_q = sh.row_max[gamma + 1 + n];
            rw.inv_sum_p = 1.0f / sh.row_aux[n];
            rw.inv_sum_q = 1.0f / sh.row_aux[gamma + 1 + n];
            rw.c2 = c2;
            token = cluster_inverse_cdf<W>(rw, vocab, u, sh.cdf, &total);
            plain = !(total > 0.0f) || !isfinite(total);  // vanished residual: draw from p_{n+1}
        }
        if (plain) token = cluster_inverse_cdf<W>(pw, vocab, u, sh.cdf, &total);
    }
    if (tid == 0) {
        if (rank == 0) n_accepted[b] = n;
        if (token >= 0) next_token[b] = token;  // exactly one CTA of the cluster holds the draw
    }
}

// One CTA per row: tokens[r] ~ softmax(logits[r] / T), or argmax at T = 0.
template <bool VEC>
__global__ void __launch_bounds__(kSampleThreads)
sample_kernel(const float* __restrict__ logits, size_t logit_stride, const float* __restrict__ uniforms,
              int uniform_stride, int vocab, float inv_t, bool greedy, int32_t* __restrict__ tokens,
              int token_stride) {
    constexpr int W = kSampleThreads / 32;
    __shared__ float red[W];
    __shared__ int red_i[W];
    __shared__ CdfScratch<W> cdf;
    __shared__ float s_max;
    __shared__ int s_arg;
    pdl_trigger();
    pdl_wait();
    const int tid = threadIdx.x;
    const Row<VEC> r = make_row<VEC>(logits + static_cast<size_t>(blockIdx.x) * logit_stride, vocab);
    const int groups = (vocab + 3) >> 2;
    float m = -FLT_MAX;
    int arg = 0x7fffffff;
#pragma unroll 4
    for (int g = tid; g < groups; g += kSampleThreads) {
        const float4 v = r.load(g, -INFINITY);
        const int j = 4 * g;
        if (v.x > m) { m = v.x; arg = j; }
        if (v.y > m) { m = v.y; arg = j + 1; }
        if (v.z > m) { m = v.z; arg = j + 2; }
        if (v.w > m) { m = v.w; arg = j + 3; }
    }
    block_argmax<W>(m, arg, red, red_i);
    if (tid == 0) { s_max = m; s_arg = arg; }
    __syncthreads();
    int token = s_arg;
    if (!greedy) {
        PlainWeights<VEC> pw;
        pw.p = r;
        pw.max_p = s_max;
        pw.c2 = inv_t * kLog2e;
        float total;
        token = block_inverse_cdf<W>(pw, vocab, uniforms[blockIdx.x * uniform_stride], cdf, &total);
    }
    if (tid == 0) tokens[blockIdx.x * token_stride] = max(0, min(token, vocab - 1));
}

__global__ void uniforms_kernel(uint64_t seed, const int32_t* __restrict__ positions,
                                const int32_t* __restrict__ sequences, uint32_t purpose, int count,
                                float* __restrict__ out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count)
        out[i] = method_uniform(seed, static_cast<uint32_t>(positions[i]), static_cast<uint32_t>(sequences[i]), purpose);
}

// Chunks per row: one unless the batch is too small to fill the GPU with
// whole-row CTAs; never more than the workspace was sized for.
int max_chunks(int vocab) {
    const int groups = (vocab + 3) / 4;
    return std::max(1, groups / kMinChunkGroups);
}

// CTAs per cluster in the finishing kernel: each CTA should still have a few
// thousand elements of row n+1 to sum.
int finish_cluster_size(int vocab) {
    int c = 1;
    while (c < kMaxCluster && vocab / (2 * c) >= 2048) c *= 2;
    return c;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int chunks_for(int vocab, int rows_total) {
    const int want = (kTargetCtas + rows_total - 1) / std::max(1, rows_total);
    return std::max(1, std::min(want, max_chunks(vocab)));
}

}  // namespace

// Shared with the generation loop: same launches, no argument checks.
size_t verify_sample_workspace_bytes(int batch, int gamma, int vocab) {
    const size_t rows = 2 * static_cast<size_t>(gamma) + 1;
    return static_cast<size_t>(batch) * rows * max_chunks(vocab) * sizeof(ChunkStat) + 256;
}

int launch_verify_sample(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                         const float* uniforms, const float* final_uniforms, int batch, int gamma, int vocab,
                         float temperature, float lenience, int32_t* n_accepted, int32_t* next_token, void* workspace,
                         cudaStream_t stream) {
    const bool greedy = temperature == 0.0f;
    const int rows = greedy ? gamma + 1 : 2 * gamma + 1;
    const int chunks = chunks_for(vocab, rows * batch);
    const float inv_t = greedy ? 0.0f : 1.0f / temperature;
    ChunkStat* stats = static_cast<ChunkStat*>(workspace);
    const dim3 grid(chunks, rows, batch);
    const bool vec = vocab % 4 == 0 && aligned16(target_logits) && (greedy || gamma == 0 || aligned16(draft_logits));
    const float c2 = inv_t * kLog2e;
    int status;
#define SPEC_LAUNCH_STATS(G, V)                                                                                  \
    status = launch_pdl(verify_stats_kernel<G, V>, grid, dim3(kStatThreads), 0, stream, target_logits, draft_logits, \
                        draft_tokens, gamma, vocab, c2, stats)
    if (greedy && vec) SPEC_LAUNCH_STATS(true, true);
    else if (greedy) SPEC_LAUNCH_STATS(true, false);
    else if (vec) SPEC_LAUNCH_STATS(false, true);
    else SPEC_LAUNCH_STATS(false, false);
#undef SPEC_LAUNCH_STATS
    if (status != SPEC_OK) return status;

    // One cluster per sequence; more CTAs per cluster for longer rows.
    const int cluster_size = greedy ? 1 : finish_cluster_size(vocab);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(batch * cluster_size);
    cfg.blockDim = dim3(kFinishThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_size;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const ChunkStat* stats_in = stats;
#define SPEC_LAUNCH_FINISH(G, V)                                                                                  \
    SPEC_CUDA_TRY(cudaLaunchKernelEx(&cfg, verify_finish_kernel<G, V>, target_logits, draft_logits, draft_tokens, \
                                     uniforms, gamma, vocab, inv_t, chunks, cluster_size, stats_in,              \
                                     final_uniforms, lenience, n_accepted, next_token))
    if (greedy && vec) SPEC_LAUNCH_FINISH(true, true);
    else if (greedy) SPEC_LAUNCH_FINISH(true, false);
    else if (vec) SPEC_LAUNCH_FINISH(false, true);
    else SPEC_LAUNCH_FINISH(false, false);
#undef SPEC_LAUNCH_FINISH
    return SPEC_OK;
}

// Row r reads logits + r * logit_stride and uniforms[r * uniform_stride] and
// writes tokens[r * token_stride].
int launch_sample_strided(const float* logits, size_t logit_stride, const float* uniforms, int uniform_stride,
                          int rows, int vocab, float temperature, int32_t* tokens, int token_stride,
                          cudaStream_t stream) {
    const bool greedy = temperature == 0.0f;
    const float inv_t = greedy ? 0.0f : 1.0f / temperature;
    if (vocab % 4 == 0 && logit_stride % 4 == 0 && aligned16(logits))
        return launch_pdl(sample_kernel<true>, dim3(rows), dim3(kSampleThreads), 0, stream, logits, logit_stride,
                          uniforms, uniform_stride, vocab, inv_t, greedy, tokens, token_stride);
    return launch_pdl(sample_kernel<false>, dim3(rows), dim3(kSampleThreads), 0, stream, logits, logit_stride, uniforms,
                      uniform_stride, vocab, inv_t, greedy, tokens, token_stride);
}

int launch_sample(const float* logits, const float* uniforms, int rows, int vocab, float temperature,
                  int32_t* tokens, cudaStream_t stream) {
    return launch_sample_strided(logits, static_cast<size_t>(vocab), uniforms, 1, rows, vocab, temperature, tokens, 1,
                                 stream);
}

}  // namespace spec

extern "C" size_t spec_verify_sample_workspace_bytes(int batch, int gamma, int vocab) {
    if (batch < 0 || gamma < 0 || vocab < 1) return 0;
    return spec::verify_sample_workspace_bytes(batch, gamma, vocab);
}

extern "C" int spec_verify_sample_lenient(const float* target_logits, const float* draft_logits,
                                          const int32_t* draft_tokens, const float* uniforms, int batch, int gamma,
                                          int vocab, float temperature, float lenience, int32_t* n_accepted,
                                          int32_t* next_token, void* workspace, size_t workspace_bytes, void* stream) {
    using namespace spec;
    if (!(lenience > 0.0f) || !(lenience <= 1.0f)) return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample: lenience must be in (0, 1]");
    if (batch < 0 || gamma < 0 || gamma > kMaxGamma || vocab < 1)
        return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample: batch=%d gamma=%d (max %d) vocab=%d", batch, gamma, kMaxGamma, vocab);
    if (!(temperature >= 0.0f) || !isfinite(temperature))
        return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample: temperature must be finite and >= 0");
    if (batch == 0) return SPEC_OK;
    if (batch > 65535) return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample: batch %d exceeds 65535", batch);
    const bool greedy = temperature == 0.0f;
    if (!target_logits || !n_accepted || !next_token || !workspace || (gamma > 0 && !draft_tokens) ||
        (!greedy && (!uniforms || (gamma > 0 && !draft_logits))))
        return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample: null pointer");
    if (workspace_bytes < spec_verify_sample_workspace_bytes(batch, gamma, vocab) ||
        (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample: workspace too small (%zu bytes) or not 256-byte aligned", workspace_bytes);
    return launch_verify_sample(target_logits, draft_logits, draft_tokens, uniforms, nullptr, batch, gamma, vocab,
                                temperature, lenience, n_accepted, next_token, workspace, static_cast<cudaStream_t>(stream));
}

extern "C" int spec_verify_sample(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                                  const float* uniforms, int batch, int gamma, int vocab, float temperature,
                                  int32_t* n_accepted, int32_t* next_token, void* workspace, size_t workspace_bytes,
                                  void* stream) {
    return spec_verify_sample_lenient(target_logits, draft_logits, draft_tokens, uniforms, batch, gamma, vocab, temperature,
                                      1.0f, n_accepted, next_token, workspace, workspace_bytes, stream);
}

// ---- spec_verify_sample without any allocation ---------------------------------
// The chunk statistics that the two kernels hand to each other normally live in a
// caller-provided workspace.  This variant keeps them in a fixed array inside the
// library image instead, so the call needs no device memory beyond its inputs and
// outputs.  Every GPU that loads the library holds the array until the process
// exits.
namespace {

constexpr size_t kStaticStatsBytes = 1u << 20;  // 65536 chunk statistics
static __device__ __align__(256) unsigned char g_static_stats[kStaticStatsBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};  // device address of g_static_stats, per device

// The array's name is only a host-side handle; kernels need its device address,
// which differs per device and is looked up once per device.
int static_stats_address(void** out) {
    int device = -1;
    SPEC_CUDA_TRY(cudaGetDevice(&device));
    if (device < 0 || device >= kMaxDevices) return spec::fail(SPEC_ERR_BAD_CONFIG, "device ordinal %d not supported", device);
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void* p = nullptr;
        SPEC_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_stats));
        g_static_ptr[device] = p;
    }
    *out = g_static_ptr[device];
    return SPEC_OK;
}

}  // namespace

extern "C" size_t spec_verify_sample_static_capacity(void) { return kStaticStatsBytes; }

extern "C" int spec_verify_sample_static(const float* target_logits, const float* draft_logits,
                                         const int32_t* draft_tokens, const float* uniforms, int batch, int gamma,
                                         int vocab, float temperature, int32_t* n_accepted, int32_t* next_token,
                                         void* stream) {
    using namespace spec;
    if (batch < 0 || gamma < 0 || gamma > kMaxGamma || vocab < 1)
        return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample_static: batch=%d gamma=%d (max %d) vocab=%d", batch, gamma, kMaxGamma, vocab);
    if (!(temperature >= 0.0f) || !isfinite(temperature))
        return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample_static: temperature must be finite and >= 0");
    if (batch == 0) return SPEC_OK;
    if (batch > 65535) return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample_static: batch %d exceeds 65535", batch);
    const bool greedy = temperature == 0.0f;
    if (!target_logits || !n_accepted || !next_token || (gamma > 0 && !draft_tokens) ||
        (!greedy && (!uniforms || (gamma > 0 && !draft_logits))))
        return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample_static: null pointer");
    const size_t need = verify_sample_workspace_bytes(batch, gamma, vocab);
    if (need > kStaticStatsBytes)
        return fail(SPEC_ERR_CAPACITY,
                    "spec_verify_sample_static: batch %d x gamma %d x vocab %d needs %zu bytes of statistics, the built-in "
                    "array holds %zu; use spec_verify_sample with a workspace", batch, gamma, vocab, need, kStaticStatsBytes);
    void* scratch = nullptr;
    const int status = static_stats_address(&scratch);
    if (status != SPEC_OK) return status;
    return launch_verify_sample(target_logits, draft_logits, draft_tokens, uniforms, nullptr, batch, gamma, vocab,
                                temperature, 1.0f, n_accepted, next_token, scratch, static_cast<cudaStream_t>(stream));
}

extern "C" int spec_sample(const float* logits, const float* uniforms, int rows, int vocab, float temperature,
                           int32_t* tokens, void* stream) {
    using namespace spec;
    if (rows < 0 || vocab < 1) return fail(SPEC_ERR_BAD_ARG, "spec_sample: rows=%d vocab=%d", rows, vocab);
    if (!(temperature >= 0.0f) || !isfinite(temperature))
        return fail(SPEC_ERR_BAD_ARG, "spec_sample: temperature must be finite and >= 0");
    if (rows == 0) return SPEC_OK;
    if (!logits || !tokens || (temperature > 0.0f && !uniforms)) return fail(SPEC_ERR_BAD_ARG, "spec_sample: null pointer");
    return launch_sample(logits, uniforms, rows, vocab, temperature, tokens, static_cast<cudaStream_t>(stream));
}

extern "C" int spec_uniforms(uint64_t seed, const int32_t* positions, const int32_t* sequences, int purpose, int count,
                             float* out, void* stream) {
    using namespace spec;
    if (count < 0 || purpose < 0 || purpose > 2) return fail(SPEC_ERR_BAD_ARG, "spec_uniforms: count=%d purpose=%d", count, purpose);
    if (count == 0) return SPEC_OK;
    if (!positions || !sequences || !out) return fail(SPEC_ERR_BAD_ARG, "spec_uniforms: null pointer");
    uniforms_kernel<<<(count + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        seed, positions, sequences, static_cast<uint32_t>(purpose), count, out);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}
