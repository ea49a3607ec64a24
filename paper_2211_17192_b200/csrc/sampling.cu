// Speculative sampling (Section 2.3 / Algorithm 1, accept-adjust-draw part),
// plain standardised sampling (Section 2.2) and the method's uniforms.
//
// spec_verify_sample is two kernels on one stream:
//   1. verify_stats_kernel streams every logit of p_1..p_{gamma+1} and
//      q_1..q_gamma exactly once from HBM.  A CTA reduces one chunk of one row
//      to (max, sum exp) with an online rescale, and also picks up the row's
//      logit at the drafted token.  No CTA talks to another: the kernel is a
//      pure map-reduce and runs at streaming bandwidth.
//   2. verify_finish_kernel, one cluster of CTAs per sequence, merges the chunk
//      statistics, runs the gamma accept tests, and re-reads only row n+1 of p
//      and q (still in L2) to normalise the residual max(0, p - q) and draw from
//      it by inverse CDF: every warp keeps the weights of its segment in
//      registers, the segment totals are scanned once across the cluster, and
//      the warp whose segment holds the target walks it without another trip to
//      memory.  It is chained with programmatic dependent launch, so its launch
//      latency and prologue overlap the tail of the first kernel.
#include <algorithm>
#include <cfloat>
#include <mutex>

#include <cooperative_groups.h>

#include "model.cuh"

namespace cg = cooperative_groups;

namespace spec {
namespace {

constexpr int kStatThreads = 256;
constexpr int kStatWarps = kStatThreads / 32;
constexpr int kUnroll = 4;              // 128-bit loads in flight per thread while streaming
constexpr int kMinChunkGroups = 1000;   // a CTA streams at least 4000 logits (unless the row is shorter)
constexpr int kTargetCtas = 148 * 48;   // about six waves of resident CTAs (eight of 256 threads per SM), so that the last wave
                                        // costs little; smaller CTAs stagger their reduce-and-restart pauses (512 threads: +0.8 us)
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
// elements past the end of the row reading as `pad`.  Logits below `floor` read
// as -inf: that is top-k standardisation (Section 2.2) with `floor` the row's
// k-th largest logit, and no change with floor = -inf.
template <bool VEC, bool CUT = false>
struct Row {
    const float* base;
    int vocab;
    float floor;  // used only with CUT, so that the usual path pays nothing for it

    __device__ __forceinline__ float kept(float v) const { return (!CUT || v >= floor) ? v : -INFINITY; }
    __device__ __forceinline__ float4 raw(int g, float pad) const {
        if (VEC) return __ldg(reinterpret_cast<const float4*>(base) + g);
        const int j = 4 * g;
        float4 v;
        v.x = j + 0 < vocab ? __ldg(base + j + 0) : pad;
        v.y = j + 1 < vocab ? __ldg(base + j + 1) : pad;
        v.z = j + 2 < vocab ? __ldg(base + j + 2) : pad;
        v.w = j + 3 < vocab ? __ldg(base + j + 3) : pad;
        return v;
    }
    __device__ __forceinline__ float4 load(int g, float pad) const {
        const float4 v = raw(g, pad);
        if (!CUT) return v;
        return make_float4(kept(v.x), kept(v.y), kept(v.z), kept(v.w));
    }
};

template <bool VEC, bool CUT = false>
__device__ __forceinline__ Row<VEC, CUT> make_row(const float* base, int vocab, float floor = -INFINITY) {
    Row<VEC, CUT> r;
    r.base = base;
    r.vocab = vocab;
    r.floor = floor;
    return r;
}

// Weight functors for the inverse-CDF draw.  fetch() only loads, weigh() only
// computes, so that a caller can put several fetches in flight before it
// consumes any of them.

// Unnormalised softmax weights exp((l - max) / T) of one row; c2 = log2(e) / T.
template <bool VEC, bool CUT = false>
struct PlainWeights {
    struct Raw { float4 a; };
    Row<VEC, CUT> p;
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
template <bool VEC, bool CUT = false>
struct ResidualWeights {
    struct Raw { float4 a, b; };
    Row<VEC, CUT> p, q;
    float max_p, max_q, inv_sum_p, inv_sum_q, c2;
    __device__ __forceinline__ Raw fetch(int g) const { return Raw{p.load(g, -INFINITY), q.load(g, -INFINITY)}; }
    __device__ __forceinline__ Raw nothing() const {
        const float4 z = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        return Raw{z, z};
    }
    __device__ __forceinline__ float one(float lp, float lq) const {
        // (both products are rounded before the subtraction: contracted into a multiply-add, one of them would not
        // be, and p = q would leave rounding residue instead of the exact zero that the fallback to p tests for)
        const float pv = __fmul_rn(fast_exp2((lp - max_p) * c2), inv_sum_p);
        const float qv = __fmul_rn(fast_exp2((lq - max_q) * c2), inv_sum_q);
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

// One step of the walk: the 128 elements of groups gs .. gs + 31 (lane l holds the four weights of group
// gs + l), in index order after the weight `run` already passed.  Sets `found` to the first index whose running
// sum exceeds `rem` (if want_hit), keeps `last_pos` = the last index with positive weight so far.
__device__ __forceinline__ void walk_step(const float4& v, int gs, int lane, bool want_hit, float rem, float& run, int& found,
                                          int& last_pos) {
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
                walk_step(w.weigh(raw[i]), gs, lane, want_hit, rem, run, found, last_pos);
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
    const int b0 = seg_begin(mine), b1 = seg_end(mine);
    // When a warp's segment fits one batch of fetches, the weights stay in registers: the warp whose segment
    // holds the target then walks it without going back to memory.
    const bool keep = seg <= 32 * kClusterCdfBatch;  // (uniform across the cluster)
    float4 kept[kClusterCdfBatch];
    float acc;
    if (keep) {
        typename Weights::Raw raw[kClusterCdfBatch];
#pragma unroll
        for (int i = 0; i < kClusterCdfBatch; ++i) {
            const int g = b0 + lane + 32 * i;
            raw[i] = g < b1 ? w.fetch(g) : w.nothing();
        }
        acc = 0.0f;
#pragma unroll
        for (int i = 0; i < kClusterCdfBatch; ++i) {
            kept[i] = w.weigh(raw[i]);
            acc += (kept[i].x + kept[i].y) + (kept[i].z + kept[i].w);
        }
        acc = warp_sum(acc);
    } else {
        acc = warp_range_sum<kClusterCdfBatch>(w, b0, b1, lane);
    }
    if (lane == 0) s.part[warp] = acc;
    cluster.sync();
    // warp 0 copies every CTA's totals into this CTA's shared memory ...
    const int parts = nctas * WARPS;
    if (warp == 0)
        for (int i = lane; i < parts; i += 32) s.all[i] = cluster.map_shared_rank(s.part, i / WARPS)[i % WARPS];
    __syncthreads();
    // (this CTA has read its peers' totals: it arrives at the cluster barrier now and waits for the others only
    // when it is about to leave, so the CTA that resolves the draw does not stand still meanwhile)
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
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
    const int hit = s.pick_part_index;
    const bool want_hit = s.pick_hit != 0;
    *total_out = total;
    int k = -1;
    if (hit / WARPS == rank) {  // (uniform across the CTA)
        if (keep) {
            if (warp == hit % WARPS) {
                float run = 0.0f;
                int found = -1, last_pos = -1;
#pragma unroll
                for (int i = 0; i < kClusterCdfBatch; ++i) {
                    const int gs = b0 + 32 * i;
                    if (gs >= b1 || found >= 0) break;
                    walk_step(kept[i], gs, lane, want_hit, target - before, run, found, last_pos);
                }
                if (lane == 0) {
                    s.result = found;
                    s.last_positive = last_pos;
                }
            }
            __syncthreads();
            k = s.result >= 0 ? s.result : s.last_positive;
        } else {
            k = locate_in_range<WARPS>(w, seg_begin(hit), seg_end(hit), target - before, want_hit, s);
        }
        k = max(0, min(k, vocab - 1));
    }
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");  // nobody reads this CTA's totals any more
    return k;
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
    float bad;     // T = 0: non-zero if the chunk holds a NaN or +inf logit (T > 0: the sums show it)
};

// grid = (chunks, rows, batch); rows = 2*gamma+1 (T > 0: p_1..p_{gamma+1}, q_1..q_gamma)
// or gamma+1 (T = 0: only p is read).
template <bool GREEDY, bool VEC, bool CUT>
__global__ void __launch_bounds__(kStatThreads)
verify_stats_kernel(const float* __restrict__ target_logits, const float* __restrict__ draft_logits,
                    const int32_t* __restrict__ draft_tokens, int gamma, int vocab, float c2,
                    const float* __restrict__ floors, ChunkStat* __restrict__ stats) {
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
    const float floor = CUT ? __ldcg(floors + static_cast<size_t>(b) * rows + row) : -INFINITY;
    const Row<VEC, CUT> r = make_row<VEC, CUT>(src, vocab, floor);
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
        if (x >= 4 * g0 && x < min(vocab, 4 * g1)) xlogit = r.kept(__ldg(src + x));
    }

    // Every thread streams groups g0+tid, g0+tid+T, ... with kUnroll 128-bit
    // loads in flight and keeps a running (max, sum exp) pair that is rescaled
    // when the maximum moves; one block-wide merge at the end.
    constexpr float kPad = -INFINITY;
    float m = -FLT_MAX;  // finite, so that (m - new_max) never becomes inf - inf
    float s = 0.0f;
    int arg = 0x7fffffff;
    bool bad = false;  // T = 0 only: a NaN or +inf logit (the comparisons below would pass over a NaN in silence)
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
                bad |= !(v[i].x < INFINITY) | !(v[i].y < INFINITY) | !(v[i].z < INFINITY) | !(v[i].w < INFINITY);
            }
        } else {
            float bm = m;
#pragma unroll
            for (int i = 0; i < kUnroll; ++i)
                bm = fmaxf(bm, fmaxf(fmaxf(v[i].x, v[i].y), fmaxf(v[i].z, v[i].w)));
            s *= fast_exp2((m - bm) * c2);
            m = bm;
            // exp2(v * c2 - m * c2): one multiply-add per logit (the kernel is close to issue-bound).  A thread that has
            // seen only padding keeps m = -FLT_MAX: the product is clamped so that -inf * c2 + it stays -inf.
            const float mc = fminf(-m * c2, FLT_MAX);
#pragma unroll
            for (int i = 0; i < kUnroll; ++i)
                s += (fast_exp2(fmaf(v[i].x, c2, mc)) + fast_exp2(fmaf(v[i].y, c2, mc))) +
                     (fast_exp2(fmaf(v[i].z, c2, mc)) + fast_exp2(fmaf(v[i].w, c2, mc)));
        }
    }
    ChunkStat* out = stats + (static_cast<size_t>(b) * rows + row) * chunks + chunk;
    if (GREEDY) {
        const int any_bad = __syncthreads_or(bad ? 1 : 0);
        block_argmax<kStatWarps>(m, arg, red, red_i);
        if (tid == 0) *reinterpret_cast<float4*>(out) = make_float4(m, __int_as_float(arg), 0.0f, any_bad ? 1.0f : 0.0f);
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
    float u_cand[kMaxGamma + 1];
    float u_final;
    int n;
};

// grid = batch * cluster size, one thread-block cluster per sequence.  Everything
// after the statistics: merge, accept tests, adjusted distribution, draw.  The
// cheap decision part is repeated in every CTA of the cluster; the pass over
// row n+1 is split between them.
template <bool GREEDY, bool VEC, bool CUT>
__global__ void __launch_bounds__(kFinishThreads, 2)
verify_finish_kernel(const float* __restrict__ target_logits, const float* __restrict__ draft_logits,
                     const int32_t* __restrict__ draft_tokens, const float* __restrict__ uniforms, int gamma,
                     int vocab, float inv_t, int chunks, int cluster_size, const ChunkStat* __restrict__ stats,
                     const float* __restrict__ final_uniforms, float lenience, const float* __restrict__ floors,
                     int32_t* __restrict__ n_accepted, int32_t* __restrict__ next_token, int* __restrict__ nonfinite) {
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
    // The generation loop keys the final draw by the position it decides, which depends on n: it passes one
    // candidate uniform per possible n; all of them are fetched now.
    if (!GREEDY && final_uniforms && tid <= gamma) sh.u_cand[tid] = __ldg(final_uniforms + static_cast<size_t>(b) * (gamma + 1) + tid);
    pdl_trigger();
    pdl_wait();

    // merge the chunk statistics of row `tid` (eight loads in flight at a time)
    if (tid < rows) {
        const ChunkStat* st_r = stats + (static_cast<size_t>(b) * rows + tid) * chunks;
        float M = -FLT_MAX, A = 0.0f, X = 0.0f;
        int best = 0x7fffffff;
        bool bad = false;
        const int xchunk = (my_x >= 0 && my_x < vocab) ? (my_x >> 2) / per_chunk : -1;
        constexpr int kMergeBatch = 8;  // chunk statistics fetched together
        for (int c0 = 0; c0 < chunks; c0 += kMergeBatch) {
            float4 st[kMergeBatch];
#pragma unroll
            for (int i = 0; i < kMergeBatch; ++i)
                st[i] = c0 + i < chunks ? __ldcg(reinterpret_cast<const float4*>(st_r + c0 + i))
                                        : make_float4(-FLT_MAX, __int_as_float(0x7fffffff), 0.0f, 0.0f);
#pragma unroll
            for (int i = 0; i < kMergeBatch; ++i) {
                if (c0 + i >= chunks) break;
                if (GREEDY) {
                    const int ci = __float_as_int(st[i].y);
                    if (st[i].x > M || (st[i].x == M && ci < best)) { M = st[i].x; best = ci; }
                    bad |= st[i].w != 0.0f;
                } else {
                    const float nm = fmaxf(M, st[i].x);
                    A = A * fast_exp2((M - nm) * c2) + st[i].y * fast_exp2((st[i].x - nm) * c2);
                    M = nm;
                    if (c0 + i == xchunk) X = st[i].z;
                }
            }
        }
        // a NaN or +inf logit (or a row without a finite logit) leaves a sum that is not a positive number
        if (!GREEDY) bad = !(A > 0.0f) || !isfinite(A) || !isfinite(M);
        if (bad && nonfinite && rank == 0) atomicExch(nonfinite, 1);
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
        const float u = final_uniforms ? sh.u_cand[n] : sh.u_final;
        PlainWeights<VEC, CUT> pw;
        const float* fl = CUT ? floors + static_cast<size_t>(b) * rows : nullptr;
        pw.p = make_row<VEC, CUT>(tl + static_cast<size_t>(n) * vocab, vocab, CUT ? __ldcg(fl + n) : -INFINITY);
        pw.max_p = sh.row_max[n];
        pw.c2 = c2;
        float total = 0.0f;
        bool plain = n == gamma;
        if (!plain) {
            ResidualWeights<VEC, CUT> rw;
            rw.p = pw.p;
            rw.q = make_row<VEC, CUT>(ql + static_cast<size_t>(n) * vocab, vocab, CUT ? __ldcg(fl + gamma + 1 + n) : -INFINITY);
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
template <bool VEC, bool CUT>
__global__ void __launch_bounds__(kSampleThreads)
sample_kernel(const float* __restrict__ logits, size_t logit_stride, const float* __restrict__ uniforms,
              int uniform_stride, int vocab, float inv_t, bool greedy, const float* __restrict__ floors,
              int32_t* __restrict__ tokens, int token_stride, int* __restrict__ nonfinite) {
    constexpr int W = kSampleThreads / 32;
    __shared__ float red[W];
    __shared__ int red_i[W];
    __shared__ CdfScratch<W> cdf;
    __shared__ float s_max;
    __shared__ int s_arg;
    pdl_trigger();
    pdl_wait();
    const int tid = threadIdx.x;
    const Row<VEC, CUT> r = make_row<VEC, CUT>(logits + static_cast<size_t>(blockIdx.x) * logit_stride, vocab,
                                               CUT ? __ldcg(floors + blockIdx.x) : -INFINITY);
    const int groups = (vocab + 3) >> 2;
    float m = -FLT_MAX;
    int arg = 0x7fffffff;
    bool bad = false;  // a NaN or +inf logit
#pragma unroll 4
    for (int g = tid; g < groups; g += kSampleThreads) {
        const float4 v = r.load(g, -INFINITY);
        const int j = 4 * g;
        if (v.x > m) { m = v.x; arg = j; }
        if (v.y > m) { m = v.y; arg = j + 1; }
        if (v.z > m) { m = v.z; arg = j + 2; }
        if (v.w > m) { m = v.w; arg = j + 3; }
        bad |= !(v.x < INFINITY) | !(v.y < INFINITY) | !(v.z < INFINITY) | !(v.w < INFINITY);
    }
    if (nonfinite && bad) atomicExch(nonfinite, 1);
    block_argmax<W>(m, arg, red, red_i);
    if (tid == 0) { s_max = m; s_arg = arg; }
    __syncthreads();
    int token = s_arg;
    if (!greedy) {
        PlainWeights<VEC, CUT> pw;
        pw.p = r;
        pw.max_p = s_max;
        pw.c2 = inv_t * kLog2e;
        float total;
        token = block_inverse_cdf<W>(pw, vocab, uniforms[blockIdx.x * uniform_stride], cdf, &total);
    }
    if (tid == 0) tokens[blockIdx.x * token_stride] = max(0, min(token, vocab - 1));
}

// ---- top-k and nucleus: the lowest logit that each row keeps ---------------------
// One CTA per row, several CTAs per SM.  Both cuts are a selection: the largest
// value t such that the logits at or above t number at least k (top-k), or carry
// at least top_p of the mass (nucleus).  The row is never sorted or held:
//   1. one pass finds the range [lo, hi] of the logits still in play;
//   2. one pass drops them into kSelBins equal-width bins counted from the top
//      (a count per bin, for the nucleus also the mass), a scan finds the bin in
//      which the target is crossed;
//   3. if that bin holds few logits they are copied out and ranked against each
//      other exactly; otherwise the bin's own range becomes [lo, hi] and step 2
//      repeats (heavy ties end when lo == hi).
// The bin of a logit is a monotone function of it, so the bins partition the row
// by value and the result is exact (comparisons of the logits themselves decide;
// -inf, +inf and NaN logits are never in play).  Mass is summed in fixed point
// (units of 2^-32 of the largest weight) with integer atomics, so every order of
// summation gives the same totals: a row always gives the same floor, however the
// threads interleave.  The kernel is bound by instruction issue, not by memory
// (the passes after the first hit L2), so the per-logit work is kept short: no
// float-to-int conversion for the bin, one 32-bit atomic plus a rare carry for
// the mass (a 64-bit shared-memory atomic cost 48 us of 180 on 960 rows of 32000),
// a two-instruction test before a logit is asked whether it is in the chosen bin.
constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelBins = 2048;
constexpr int kSelPerThread = kSelBins / kSelThreads;
constexpr int kSelCap = 1024;   // logits ranked against each other at the end
constexpr int kSelLevels = 40;  // every level shrinks the range; fp32 allows far fewer than this

struct SelShared {
    unsigned cnt[kSelBins];
    unsigned mass_lo[kSelBins], mass_hi[kSelBins];  // a bin's mass, low and high word (apart: the low words then spread over all banks)
    float cand[kSelCap];
    unsigned long long cand_mass[kSelCap];
    unsigned long long warp_mass[kSelWarps];
    unsigned warp_cnt[kSelWarps];
    float warp_lo[kSelWarps], warp_hi[kSelWarps];
    unsigned n_cand;
    // where the scan found the target crossed
    int bin;
    unsigned before_cnt;
    unsigned long long before_mass;
};

// f(v) for every logit of the row, kSelLoads 128-bit loads in flight per thread.
constexpr int kSelLoads = 8;

template <bool VEC, class F>
__device__ __forceinline__ void for_each_logit(const Row<VEC>& r, int groups, F f) {
    for (int g0 = threadIdx.x; g0 < groups; g0 += kSelLoads * kSelThreads) {
        float4 v[kSelLoads];
#pragma unroll
        for (int i = 0; i < kSelLoads; ++i) {
            const int g = g0 + i * kSelThreads;
            v[i] = g < groups ? r.raw(g, -INFINITY) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        }
#pragma unroll
        for (int i = 0; i < kSelLoads; ++i) {
            f(v[i].x);
            f(v[i].y);
            f(v[i].z);
            f(v[i].w);
        }
    }
}

__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// The floor among the finite logits >= kf: MASS = false, the k-th largest of
// them; MASS = true, the nucleus of mass top_p with weights exp2((l - max) * c2).
// Every thread returns the same value; -inf means "keep everything".
template <bool VEC, bool MASS>
__device__ float select_floor(const Row<VEC>& r, int groups, float kf, unsigned k, float top_p, float c2, SelShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // 1. range and number of the logits in play
    float lo = INFINITY, hi = -INFINITY;
    unsigned n = 0;
    for_each_logit(r, groups, [&](float v) {
        const bool in_play = fabsf(v) < INFINITY && v >= kf;
        const float u = in_play ? v : __int_as_float(0x7fc00000);  // (fminf and fmaxf pass over a NaN operand)
        lo = fminf(lo, u);
        hi = fmaxf(hi, u);
        n += in_play;
    });
    lo = warp_min(lo);
    hi = warp_max(hi);
    n = __reduce_add_sync(0xffffffffu, n);
    __syncthreads();  // (the shared arrays may still be read by a previous call)
    if (lane == 0) { sh.warp_lo[warp] = lo; sh.warp_hi[warp] = hi; sh.warp_cnt[warp] = n; }
    __syncthreads();
    lo = INFINITY; hi = -INFINITY; n = 0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) { lo = fminf(lo, sh.warp_lo[w]); hi = fmaxf(hi, sh.warp_hi[w]); n += sh.warp_cnt[w]; }
    if (n == 0 || (!MASS && k > n)) return kf;  // nothing to cut
    // weight exp2((l - max) * c2) of a logit in units of 2^-32 (the largest float below 2^32, so that the row's
    // maximum still fits 32 bits): a bin's mass is then one 32-bit shared-memory atomic and, rarely, a carry
    const float mc = fminf(-hi * c2, FLT_MAX);
    auto fixed_mass = [&](float v) { return __float2uint_rz(fast_exp2(fmaf(v, c2, mc)) * 4294967040.0f); };

    unsigned before_cnt = 0;
    unsigned long long before_mass = 0, goal = 0;
    for (int level = 0; level < kSelLevels; ++level) {
        if (lo == hi) return hi;  // everything left is one value: it stays whole
        const float top = hi, bottom = lo;
        // (top - v) * scale stays below kSelBins for every v >= bottom: the quarter bin absorbs the roundings
        const float scale = fminf((static_cast<float>(kSelBins) - 0.25f) / (top - bottom), FLT_MAX);
        // bin of a logit in [bottom, top], counted from the top; anything else gets no bin.  The floor is taken by
        // adding 2^23 with rounding toward zero (the sum's last bit is then worth one) instead of a conversion.
        auto bin_of = [&](float v) {
            const int b = __float_as_int(__fmaf_rz(top - v, scale, 8388608.0f)) & 0x7fffff;
            return (v >= bottom && v <= top) ? b : -1;
        };
        // 2. counts (and masses) per bin
        for (int i = tid; i < kSelBins; i += kSelThreads) {
            if (MASS) { sh.mass_lo[i] = 0; sh.mass_hi[i] = 0; } else { sh.cnt[i] = 0; }
        }
        if (tid == 0) { sh.n_cand = 0; sh.bin = kSelBins - 1; sh.before_cnt = before_cnt; sh.before_mass = before_mass; }
        __syncthreads();
        for_each_logit(r, groups, [&](float v) {
            const int b = bin_of(v);
            if (b >= 0) {
                if (MASS) {
                    const unsigned m = fixed_mass(v);
                    const unsigned was = atomicAdd(&sh.mass_lo[b], m);
                    if (was + m < was) atomicAdd(&sh.mass_hi[b], 1u);
                } else {
                    atomicAdd(&sh.cnt[b], 1u);
                }
            }
        });
        __syncthreads();
        // scan over the bins from the top: thread t owns bins t*P .. t*P+P-1
        unsigned my_cnt = 0;
        unsigned long long my_mass = 0;
#pragma unroll
        for (int i = 0; i < kSelPerThread; ++i) {
            const int b = tid * kSelPerThread + i;
            if (MASS) my_mass += (static_cast<unsigned long long>(sh.mass_hi[b]) << 32) | sh.mass_lo[b];
            else my_cnt += sh.cnt[b];
        }
        unsigned inc_cnt = my_cnt;
        unsigned long long inc_mass = my_mass;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned c = __shfl_up_sync(0xffffffffu, inc_cnt, d);
            const unsigned long long m = __shfl_up_sync(0xffffffffu, inc_mass, d);
            if (lane >= d) { inc_cnt += c; inc_mass += m; }
        }
        if (lane == 31) { sh.warp_cnt[warp] = inc_cnt; sh.warp_mass[warp] = inc_mass; }
        __syncthreads();
        unsigned ex_cnt = before_cnt + inc_cnt - my_cnt;
        unsigned long long ex_mass = before_mass + inc_mass - my_mass, all_mass = 0;
#pragma unroll
        for (int w = 0; w < kSelWarps; ++w) {
            if (w < warp) { ex_cnt += sh.warp_cnt[w]; ex_mass += sh.warp_mass[w]; }
            all_mass += sh.warp_mass[w];
        }
        if (MASS && level == 0)  // the first level sees every logit in play: top_p of their mass is the target
            goal = static_cast<unsigned long long>(ceil(static_cast<double>(top_p) * static_cast<double>(all_mass)));
        // the one thread whose bins contain the crossing records it
        if (MASS ? ex_mass < goal : ex_cnt < k) {
            unsigned run_cnt = ex_cnt;
            unsigned long long run_mass = ex_mass;
#pragma unroll
            for (int i = 0; i < kSelPerThread; ++i) {
                const int b = tid * kSelPerThread + i;
                const unsigned c = MASS ? 0u : sh.cnt[b];
                const unsigned long long m = MASS ? (static_cast<unsigned long long>(sh.mass_hi[b]) << 32) | sh.mass_lo[b] : 0ull;
                const bool was_below = MASS ? run_mass < goal : run_cnt < k;
                const bool reaches = MASS ? run_mass + m >= goal : run_cnt + c >= k;
                if (was_below && reaches) { sh.bin = b; sh.before_cnt = run_cnt; sh.before_mass = run_mass; }
                run_cnt += c;
                run_mass += m;
            }
        }
        __syncthreads();
        const int bin = sh.bin;
        before_cnt = sh.before_cnt;
        before_mass = sh.before_mass;
        // top-k knows how many logits the bin holds; the nucleus keeps no counts and finds out by copying them
        const bool few = MASS || sh.cnt[bin] <= kSelCap;
        // a cheap test that no logit of the bin fails (its centre, half its width and the roundings of bin_of, with
        // room to spare); the few that pass are then asked for their bin
        const float centre = top - (static_cast<float>(bin) + 0.5f) / scale;
        const float reach = 0.51f / scale + 2e-6f * fmaxf(fabsf(top), fabsf(bottom));
        auto in_the_bin = [&](float v) { return fabsf(v - centre) <= reach && bin_of(v) == bin; };
        if (few) {
            // 3. copy the bin's logits out and rank them against each other
            for_each_logit(r, groups, [&](float v) {
                if (in_the_bin(v)) {
                    const unsigned at = atomicAdd(&sh.n_cand, 1u);
                    if (at < kSelCap) { sh.cand[at] = v; if (MASS) sh.cand_mass[at] = fixed_mass(v); }
                }
            });
            __syncthreads();
            if (sh.n_cand <= kSelCap) {  // (always so for top-k)
                const int count = static_cast<int>(min(sh.n_cand, static_cast<unsigned>(kSelCap)));
                float best = -INFINITY;
                for (int i = tid; i < count; i += kSelThreads) {
                    const float mine = sh.cand[i];
                    unsigned c = 0;
                    unsigned long long m = 0;
                    for (int j = 0; j < count; ++j)
                        if (sh.cand[j] >= mine) { ++c; if (MASS) m += sh.cand_mass[j]; }
                    const bool enough = MASS ? before_mass + m >= goal : before_cnt + c >= k;
                    if (enough) best = fmaxf(best, mine);
                }
                best = warp_max(best);
                if (lane == 0) sh.warp_hi[warp] = best;
                __syncthreads();
                best = -INFINITY;
#pragma unroll
                for (int w = 0; w < kSelWarps; ++w) best = fmaxf(best, sh.warp_hi[w]);
                return best > -INFINITY ? best : bottom;
            }
        }
        // the bin is crowded: its own range is searched next
        float new_lo = INFINITY, new_hi = -INFINITY;
        for_each_logit(r, groups, [&](float v) {
            const bool here = in_the_bin(v);
            new_lo = fminf(new_lo, here ? v : INFINITY);
            new_hi = fmaxf(new_hi, here ? v : -INFINITY);
        });
        new_lo = warp_min(new_lo);
        new_hi = warp_max(new_hi);
        if (lane == 0) { sh.warp_lo[warp] = new_lo; sh.warp_hi[warp] = new_hi; }
        __syncthreads();
        lo = INFINITY; hi = -INFINITY;
#pragma unroll
        for (int w = 0; w < kSelWarps; ++w) { lo = fminf(lo, sh.warp_lo[w]); hi = fmaxf(hi, sh.warp_hi[w]); }
        __syncthreads();
    }
    return lo;
}

// Top-k for k up to half the number of threads, without bins: the k-th largest of the threads' own maxima is a
// value that at least k logits reach, so the k-th largest logit of the row is among those that reach it - a few
// more than k as a rule.  One pass for the maxima, one that copies out what reaches the pivot, then the exact
// ranking of step 3 above.  Returns false, having decided nothing, when fewer than k threads hold a finite logit
// or more than kSelCap logits reach the pivot (heavy ties): the binned selection then does the row.
template <bool VEC>
__device__ bool top_k_by_pivot(const Row<VEC>& r, int groups, unsigned k, SelShared& sh, float* floor) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // (measured on 960 rows of 32000: k = 40 66 us per call against 82 binned, k = 128 71, k = 200 92: the pivot sinks
    // with k and lets ever more logits through)
    if (k > static_cast<unsigned>(kSelThreads) / 2) return false;
    float mine = -INFINITY;
    unsigned n = 0;
    for_each_logit(r, groups, [&](float v) {
        const bool finite = fabsf(v) < INFINITY;
        mine = fmaxf(mine, finite ? v : -INFINITY);
        n += finite;
    });
    n = __reduce_add_sync(0xffffffffu, n);
    __syncthreads();  // (the shared arrays may still be read by a previous call)
    if (lane == 0) sh.warp_cnt[warp] = n;
    sh.cand[tid] = mine;
    if (tid == 0) sh.n_cand = 0;
    __syncthreads();
    n = 0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) n += sh.warp_cnt[w];
    if (k > n) {  // nothing to cut
        *floor = -INFINITY;
        return true;
    }
    // the k-th largest of the maxima: the largest one that at least k of them reach
    unsigned reach = 0;
    for (int j = 0; j < kSelThreads; ++j) reach += sh.cand[j] >= mine;
    float pivot = warp_max(reach >= k ? mine : -INFINITY);
    if (lane == 0) sh.warp_hi[warp] = pivot;
    __syncthreads();  // (every thread has read the maxima: the list can be reused)
    pivot = -INFINITY;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) pivot = fmaxf(pivot, sh.warp_hi[w]);
    if (!(pivot > -INFINITY)) return false;
    for_each_logit(r, groups, [&](float v) {
        if (v >= pivot && v < INFINITY) {
            const unsigned at = atomicAdd(&sh.n_cand, 1u);
            if (at < kSelCap) sh.cand[at] = v;
        }
    });
    __syncthreads();
    const unsigned total = sh.n_cand;
    if (total > kSelCap) return false;
    const int count = static_cast<int>(total);
    float best = -INFINITY;
    for (int i = tid; i < count; i += kSelThreads) {
        const float c = sh.cand[i];
        unsigned at_least = 0;
        for (int j = 0; j < count; ++j) at_least += sh.cand[j] >= c;
        if (at_least >= k) best = fmaxf(best, c);
    }
    best = warp_max(best);
    __syncthreads();  // (warp_hi has been read by everyone)
    if (lane == 0) sh.warp_hi[warp] = best;
    __syncthreads();
    best = -INFINITY;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) best = fmaxf(best, sh.warp_hi[w]);
    *floor = best;
    return true;
}

// The nucleus when top-k has already cut the row down to a few logits (those >= kf):
// one pass copies them out, then they are ranked against each other as in step 3
// above.  Returns false, having decided nothing, if more than kSelCap logits are
// in play (a large tie at the top-k floor).
template <bool VEC>
__device__ bool nucleus_of_few(const Row<VEC>& r, int groups, float kf, float top_p, float c2, SelShared& sh, float* floor) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __syncthreads();  // (the shared arrays may still be read by a previous call)
    if (tid == 0) sh.n_cand = 0;
    __syncthreads();
    for_each_logit(r, groups, [&](float v) {
        if (fabsf(v) < INFINITY && v >= kf) {
            const unsigned at = atomicAdd(&sh.n_cand, 1u);
            if (at < kSelCap) sh.cand[at] = v;
        }
    });
    __syncthreads();
    const unsigned total = sh.n_cand;
    if (total == 0 || total > kSelCap) return false;
    const int count = static_cast<int>(total);
    float row_max = -INFINITY;
    for (int i = tid; i < count; i += kSelThreads) row_max = fmaxf(row_max, sh.cand[i]);
    row_max = warp_max(row_max);
    if (lane == 0) sh.warp_hi[warp] = row_max;
    __syncthreads();
    row_max = -INFINITY;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) row_max = fmaxf(row_max, sh.warp_hi[w]);
    unsigned long long mine_sum = 0;
    for (int i = tid; i < count; i += kSelThreads) {
        const unsigned long long m = __float2ull_rz(fast_exp2((sh.cand[i] - row_max) * c2) * 1099511627776.0f);  // 2^40
        sh.cand_mass[i] = m;
        mine_sum += m;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine_sum += __shfl_xor_sync(0xffffffffu, mine_sum, o);
    __syncthreads();  // (warp_hi has been read by everyone; cand_mass is complete)
    if (lane == 0) sh.warp_mass[warp] = mine_sum;
    __syncthreads();
    unsigned long long all_mass = 0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) all_mass += sh.warp_mass[w];
    const unsigned long long goal = static_cast<unsigned long long>(ceil(static_cast<double>(top_p) * static_cast<double>(all_mass)));
    float best = -INFINITY;
    for (int i = tid; i < count; i += kSelThreads) {
        const float mine = sh.cand[i];
        unsigned long long m = 0;
        for (int j = 0; j < count; ++j)
            if (sh.cand[j] >= mine) m += sh.cand_mass[j];
        if (m >= goal) best = fmaxf(best, mine);
    }
    best = warp_max(best);
    if (lane == 0) sh.warp_lo[warp] = best;
    __syncthreads();
    best = -INFINITY;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) best = fmaxf(best, sh.warp_lo[w]);
    *floor = best > -INFINITY ? best : kf;
    return true;
}

// floors[s * (a_rows + b_rows) + r] for sequence s's a_rows rows of `a`, then its
// b_rows rows of `b`: top-k first (0 < top_k < vocab), then the nucleus (0 < top_p < 1)
// of what top-k left.
template <bool VEC>
__global__ void __launch_bounds__(kSelThreads)
cut_floor_kernel(const float* __restrict__ a, size_t a_stride, int a_rows, const float* __restrict__ b,
                 size_t b_stride, int b_rows, int vocab, int top_k, float top_p, float c2, float* __restrict__ floors) {
    __shared__ SelShared sh;
    pdl_trigger();
    pdl_wait();
    const int per_seq = a_rows + b_rows;
    const int seq = blockIdx.x / per_seq, row = blockIdx.x % per_seq;
    const float* src = row < a_rows ? a + (static_cast<size_t>(seq) * a_rows + row) * a_stride
                                    : b + (static_cast<size_t>(seq) * b_rows + (row - a_rows)) * b_stride;
    const Row<VEC> r = make_row<VEC>(src, vocab);
    const int groups = (vocab + 3) >> 2;
    float floor = -INFINITY;
    if (top_k > 0 && top_k < vocab && !top_k_by_pivot<VEC>(r, groups, static_cast<unsigned>(top_k), sh, &floor))
        floor = select_floor<VEC, false>(r, groups, -INFINITY, static_cast<unsigned>(top_k), 0.0f, 0.0f, sh);
    if (top_p > 0.0f && top_p < 1.0f) {
        // after a top-k that leaves few logits the nucleus needs no binning
        const bool few = floor > -INFINITY && top_k <= kSelCap;
        if (!few || !nucleus_of_few<VEC>(r, groups, floor, top_p, c2, sh, &floor))
            floor = select_floor<VEC, true>(r, groups, floor, 0u, top_p, c2, sh);
    }
    if (threadIdx.x == 0) floors[blockIdx.x] = floor;
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

size_t stats_bytes(int batch, int gamma, int vocab) {
    const size_t rows = 2 * static_cast<size_t>(gamma) + 1;
    return (static_cast<size_t>(batch) * rows * max_chunks(vocab) * sizeof(ChunkStat) + 255) & ~static_cast<size_t>(255);
}

}  // namespace

// Shared with the generation loop: same launches, no argument checks.
// Layout: chunk statistics, then one top-k floor per row.
size_t verify_sample_workspace_bytes(int batch, int gamma, int vocab) {
    const size_t rows = 2 * static_cast<size_t>(gamma) + 1;
    return stats_bytes(batch, gamma, vocab) + static_cast<size_t>(batch) * rows * sizeof(float) + 256;
}

bool cut_is_on(int vocab, float temperature, int top_k, float top_p) {
    return temperature > 0.0f && ((top_k > 0 && top_k < vocab) || (top_p > 0.0f && top_p < 1.0f));
}

// Top-k, then the nucleus of what is left (Section 2.2): one floor per row, one kernel.
// floors[s * (a_rows + b_rows) + r] belongs to sequence s's row r (its a_rows rows of `a`,
// then its b_rows rows of `b`).
int launch_cut_floors(const float* a, size_t a_stride, int a_rows, const float* b, size_t b_stride, int b_rows,
                      int seqs, int vocab, int top_k, float top_p, float inv_t, float* floors, cudaStream_t stream) {
    const int total = seqs * (a_rows + b_rows);
    if (total == 0) return SPEC_OK;
    const bool vec = vocab % 4 == 0 && a_stride % 4 == 0 && aligned16(a) && (b_rows == 0 || (b_stride % 4 == 0 && aligned16(b)));
    const float c2 = inv_t * kLog2e;
    if (vec)
        return launch_pdl(cut_floor_kernel<true>, dim3(total), dim3(kSelThreads), 0, stream, a, a_stride, a_rows, b, b_stride,
                          b_rows, vocab, top_k, top_p, c2, floors);
    return launch_pdl(cut_floor_kernel<false>, dim3(total), dim3(kSelThreads), 0, stream, a, a_stride, a_rows, b, b_stride,
                      b_rows, vocab, top_k, top_p, c2, floors);
}

int launch_verify_sample(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                         const float* uniforms, const float* final_uniforms, int batch, int gamma, int vocab,
                         float temperature, float lenience, int top_k, float top_p, int32_t* n_accepted,
                         int32_t* next_token, void* workspace, cudaStream_t stream, int* nonfinite) {
    const bool greedy = temperature == 0.0f;
    const int rows = greedy ? gamma + 1 : 2 * gamma + 1;
    const int chunks = chunks_for(vocab, rows * batch);
    const float inv_t = greedy ? 0.0f : 1.0f / temperature;
    ChunkStat* stats = static_cast<ChunkStat*>(workspace);
    // top-k and nucleus (Section 2.2): both models' rows are cut at their own floors
    const float* floors = nullptr;
    if (cut_is_on(vocab, temperature, top_k, top_p)) {
        float* f = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + stats_bytes(batch, gamma, vocab));
        const int st = launch_cut_floors(target_logits, static_cast<size_t>(vocab), gamma + 1, draft_logits,
                                         static_cast<size_t>(vocab), gamma, batch, vocab, top_k, top_p, inv_t, f, stream);
        if (st != SPEC_OK) return st;
        floors = f;
    }
    const dim3 grid(chunks, rows, batch);
    const bool vec = vocab % 4 == 0 && aligned16(target_logits) && (greedy || gamma == 0 || aligned16(draft_logits));
    const float c2 = inv_t * kLog2e;
    int status;
    const bool cut = floors != nullptr;  // never with greedy
#define SPEC_LAUNCH_STATS(G, V, C)                                                                               \
    status = launch_pdl(verify_stats_kernel<G, V, C>, grid, dim3(kStatThreads), 0, stream, target_logits, draft_logits, \
                        draft_tokens, gamma, vocab, c2, floors, stats)
    if (greedy && vec) SPEC_LAUNCH_STATS(true, true, false);
    else if (greedy) SPEC_LAUNCH_STATS(true, false, false);
    else if (vec && cut) SPEC_LAUNCH_STATS(false, true, true);
    else if (vec) SPEC_LAUNCH_STATS(false, true, false);
    else if (cut) SPEC_LAUNCH_STATS(false, false, true);
    else SPEC_LAUNCH_STATS(false, false, false);
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
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster_size;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    const ChunkStat* stats_in = stats;
#define SPEC_LAUNCH_FINISH(G, V, C)                                                                                  \
    SPEC_CUDA_TRY(cudaLaunchKernelEx(&cfg, verify_finish_kernel<G, V, C>, target_logits, draft_logits, draft_tokens, \
                                     uniforms, gamma, vocab, inv_t, chunks, cluster_size, stats_in,                 \
                                     final_uniforms, lenience, floors, n_accepted, next_token, nonfinite))
    if (greedy && vec) SPEC_LAUNCH_FINISH(true, true, false);
    else if (greedy) SPEC_LAUNCH_FINISH(true, false, false);
    else if (vec && cut) SPEC_LAUNCH_FINISH(false, true, true);
    else if (vec) SPEC_LAUNCH_FINISH(false, true, false);
    else if (cut) SPEC_LAUNCH_FINISH(false, false, true);
    else SPEC_LAUNCH_FINISH(false, false, false);
#undef SPEC_LAUNCH_FINISH
    return SPEC_OK;
}

// Row r reads logits + r * logit_stride and uniforms[r * uniform_stride] and
// writes tokens[r * token_stride].
// With a cut (0 < top_k < vocab or 0 < top_p < 1, and T > 0) `floor_scratch` must hold `rows` floats.
int launch_sample_strided(const float* logits, size_t logit_stride, const float* uniforms, int uniform_stride,
                          int rows, int vocab, float temperature, int top_k, float top_p, float* floor_scratch,
                          int32_t* tokens, int token_stride, cudaStream_t stream, int* nonfinite) {
    const bool greedy = temperature == 0.0f;
    const float inv_t = greedy ? 0.0f : 1.0f / temperature;
    const float* floors = nullptr;
    if (cut_is_on(vocab, temperature, top_k, top_p)) {
        const int st = launch_cut_floors(logits, logit_stride, 1, nullptr, 0, 0, rows, vocab, top_k, top_p, inv_t,
                                         floor_scratch, stream);
        if (st != SPEC_OK) return st;
        floors = floor_scratch;
    }
    const bool vec = vocab % 4 == 0 && logit_stride % 4 == 0 && aligned16(logits);
#define SPEC_LAUNCH_SAMPLE(V, C)                                                                                   \
    return launch_pdl(sample_kernel<V, C>, dim3(rows), dim3(kSampleThreads), 0, stream, logits, logit_stride, uniforms, \
                      uniform_stride, vocab, inv_t, greedy, floors, tokens, token_stride, nonfinite)
    if (vec && floors) SPEC_LAUNCH_SAMPLE(true, true);
    if (vec) SPEC_LAUNCH_SAMPLE(true, false);
    if (floors) SPEC_LAUNCH_SAMPLE(false, true);
    SPEC_LAUNCH_SAMPLE(false, false);
#undef SPEC_LAUNCH_SAMPLE
}

int launch_sample(const float* logits, const float* uniforms, int rows, int vocab, float temperature, int top_k,
                  float top_p, float* floor_scratch, int32_t* tokens, cudaStream_t stream) {
    return launch_sample_strided(logits, static_cast<size_t>(vocab), uniforms, 1, rows, vocab, temperature, top_k, top_p,
                                 floor_scratch, tokens, 1, stream, nullptr);
}

}  // namespace spec

extern "C" size_t spec_verify_sample_workspace_bytes(int batch, int gamma, int vocab) {
    if (batch < 0 || gamma < 0 || vocab < 1) return 0;
    return spec::verify_sample_workspace_bytes(batch, gamma, vocab);
}

extern "C" int spec_verify_sample_truncated(const float* target_logits, const float* draft_logits,
                                            const int32_t* draft_tokens, const float* uniforms, int batch, int gamma,
                                            int vocab, float temperature, float lenience, int top_k, float top_p,
                                            int32_t* n_accepted, int32_t* next_token, void* workspace,
                                            size_t workspace_bytes, void* stream) {
    using namespace spec;
    if (top_k < 0 || !(top_p == top_p)) return fail(SPEC_ERR_BAD_ARG, "spec_verify_sample: top_k must be >= 0 and top_p a number");
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
                                temperature, lenience, top_k, top_p, n_accepted, next_token, workspace,
                                static_cast<cudaStream_t>(stream));
}

extern "C" int spec_verify_sample_lenient(const float* target_logits, const float* draft_logits,
                                          const int32_t* draft_tokens, const float* uniforms, int batch, int gamma,
                                          int vocab, float temperature, float lenience, int32_t* n_accepted,
                                          int32_t* next_token, void* workspace, size_t workspace_bytes, void* stream) {
    return spec_verify_sample_truncated(target_logits, draft_logits, draft_tokens, uniforms, batch, gamma, vocab,
                                        temperature, lenience, 0, 1.0f, n_accepted, next_token, workspace,
                                        workspace_bytes, stream);
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
                                temperature, 1.0f, 0, 1.0f, n_accepted, next_token, scratch, static_cast<cudaStream_t>(stream));
}

extern "C" int spec_sample(const float* logits, const float* uniforms, int rows, int vocab, float temperature,
                           int32_t* tokens, void* stream) {
    using namespace spec;
    if (rows < 0 || vocab < 1) return fail(SPEC_ERR_BAD_ARG, "spec_sample: rows=%d vocab=%d", rows, vocab);
    if (!(temperature >= 0.0f) || !isfinite(temperature))
        return fail(SPEC_ERR_BAD_ARG, "spec_sample: temperature must be finite and >= 0");
    if (rows == 0) return SPEC_OK;
    if (!logits || !tokens || (temperature > 0.0f && !uniforms)) return fail(SPEC_ERR_BAD_ARG, "spec_sample: null pointer");
    return launch_sample(logits, uniforms, rows, vocab, temperature, 0, 1.0f, nullptr, tokens, static_cast<cudaStream_t>(stream));
}

extern "C" int spec_sample_truncated(const float* logits, const float* uniforms, int rows, int vocab, float temperature,
                                     int top_k, float top_p, int32_t* tokens, float* floors, void* stream) {
    using namespace spec;
    if (rows < 0 || vocab < 1 || top_k < 0 || !(top_p == top_p))
        return fail(SPEC_ERR_BAD_ARG, "spec_sample_truncated: rows=%d vocab=%d top_k=%d top_p=%g", rows, vocab, top_k, top_p);
    if (!(temperature >= 0.0f) || !isfinite(temperature))
        return fail(SPEC_ERR_BAD_ARG, "spec_sample_truncated: temperature must be finite and >= 0");
    if (rows == 0) return SPEC_OK;
    if (!logits || !tokens || (temperature > 0.0f && !uniforms) || (cut_is_on(vocab, temperature, top_k, top_p) && !floors))
        return fail(SPEC_ERR_BAD_ARG, "spec_sample_truncated: null pointer");
    return launch_sample(logits, uniforms, rows, vocab, temperature, top_k, top_p, floors, tokens,
                         static_cast<cudaStream_t>(stream));
}

extern "C" int spec_truncation_floors(const float* logits, int rows, int vocab, float temperature, int top_k, float top_p,
                                      float* floors, void* stream) {
    using namespace spec;
    if (rows < 0 || vocab < 1 || top_k < 0 || !(top_p == top_p))
        return fail(SPEC_ERR_BAD_ARG, "spec_truncation_floors: rows=%d vocab=%d top_k=%d top_p=%g", rows, vocab, top_k, top_p);
    if (!(temperature > 0.0f) || !isfinite(temperature))
        return fail(SPEC_ERR_BAD_ARG, "spec_truncation_floors: temperature must be finite and > 0");
    if (!cut_is_on(vocab, temperature, top_k, top_p))
        return fail(SPEC_ERR_BAD_ARG, "spec_truncation_floors: neither 0 < top_k < vocab nor 0 < top_p < 1");
    if (rows == 0) return SPEC_OK;
    if (!logits || !floors) return fail(SPEC_ERR_BAD_ARG, "spec_truncation_floors: null pointer");
    return launch_cut_floors(logits, static_cast<size_t>(vocab), 1, nullptr, 0, 0, rows, vocab, top_k, top_p,
                             1.0f / temperature, floors, static_cast<cudaStream_t>(stream));
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
