// Fused speculative sampling (Section 2.3 / Algorithm 1, accept-adjust-draw
// part), plain standardised sampling (Section 2.2) and the method's uniforms.
//
// One launch handles a whole batch.  Every logit is read once from HBM by the
// statistics phase: each CTA reduces one chunk of one row of p_i or q_i to a
// (max, sum exp) pair.  The CTA that finishes a sequence last (a ticket taken
// with atomicAdd; nobody waits for anybody) merges the chunk statistics, runs
// the gamma accept tests, and re-reads only row n+1 of p and q (still in L2)
// to normalise the residual max(0, p - q) and draw from it by inverse CDF.
#include "common.cuh"

namespace spec {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kGroupsPerThread = 8;                       // float4 groups held in registers
constexpr int kChunkGroups = kThreads * kGroupsPerThread;  // 2048 groups = 8192 logits per CTA
constexpr int kMaxGamma = 64;
constexpr int kMaxRows = 2 * kMaxGamma + 1;

// A row of fp32 logits addressed in groups of four elements.  Rows whose base
// is 16-byte aligned use one 128-bit load per group; others fall back to four
// scalar loads.  Elements past the end of the row read as `pad`.
struct Row {
    const float* base;
    int vocab;
    bool vec;

    __device__ __forceinline__ float4 load(int g, float pad) const {
        const int j = 4 * g;
        if (vec && j + 3 < vocab) return __ldg(reinterpret_cast<const float4*>(base) + g);
        float4 v;
        v.x = j + 0 < vocab ? __ldg(base + j + 0) : pad;
        v.y = j + 1 < vocab ? __ldg(base + j + 1) : pad;
        v.z = j + 2 < vocab ? __ldg(base + j + 2) : pad;
        v.w = j + 3 < vocab ? __ldg(base + j + 3) : pad;
        return v;
    }
};

__device__ __forceinline__ Row make_row(const float* base, int vocab) {
    Row r;
    r.base = base;
    r.vocab = vocab;
    r.vec = (reinterpret_cast<uintptr_t>(base) & 15u) == 0;
    return r;
}

// Unnormalised softmax weights exp((l - max) / T) of one row.
struct PlainWeights {
    Row p;
    float max_p, inv_t;
    __device__ __forceinline__ float4 operator()(int g) const {
        const float4 a = p.load(g, -INFINITY);
        return make_float4(expf((a.x - max_p) * inv_t), expf((a.y - max_p) * inv_t),
                           expf((a.z - max_p) * inv_t), expf((a.w - max_p) * inv_t));
    }
};

// max(0, p - q) with p, q the normalised softmaxes of two rows (Algorithm 1's
// adjusted distribution before normalisation).
struct ResidualWeights {
    Row p, q;
    float max_p, max_q, inv_sum_p, inv_sum_q, inv_t;
    __device__ __forceinline__ float one(float lp, float lq) const {
        const float pv = expf((lp - max_p) * inv_t) * inv_sum_p;
        const float qv = expf((lq - max_q) * inv_t) * inv_sum_q;
        return fmaxf(0.0f, pv - qv);
    }
    __device__ __forceinline__ float4 operator()(int g) const {
        const float4 a = p.load(g, -INFINITY);
        const float4 b = q.load(g, -INFINITY);
        return make_float4(one(a.x, b.x), one(a.y, b.y), one(a.z, b.z), one(a.w, b.w));
    }
};

struct CdfScratch {
    float warp_total[kWarps];
    float total;
    int result;
    int last_positive;
};

// Inverse-CDF draw by one CTA: the smallest index k whose running weight sum
// exceeds u * (sum of all weights); the last index with positive weight if
// rounding leaves none.  Each warp owns a contiguous segment of the vocabulary
// so that running sums follow index order.  Returns the index to all threads
// and the total through *total_out.
template <class Weights>
__device__ int block_inverse_cdf(const Weights& w, int vocab, float u, CdfScratch& s, float* total_out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int groups = (vocab + 3) >> 2;
    const int seg = (groups + kWarps - 1) / kWarps;
    const int g0 = warp * seg;
    const int g1 = min(groups, g0 + seg);

    float acc = 0.0f;
    for (int g = g0 + lane; g < g1; g += 32) {
        const float4 v = w(g);
        acc += (v.x + v.y) + (v.z + v.w);
    }
    acc = warp_sum(acc);
    if (lane == 0) s.warp_total[warp] = acc;
    if (tid == 0) {
        s.result = -1;
        s.last_positive = -1;
    }
    __syncthreads();

    float total = 0.0f;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) total += s.warp_total[i];
    const float target = u * total;
    // The segment that contains the target: first warp whose running total exceeds it.
    int hit_warp = -1;
    float before = 0.0f, run = 0.0f;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) {
        const float next = run + s.warp_total[i];
        if (hit_warp < 0 && next > target) {
            hit_warp = i;
            before = run;
        }
        run = next;
    }
    if (hit_warp < 0) {  // rounding: fall back to the last segment with positive weight
        before = 0.0f;
        run = 0.0f;
        for (int i = 0; i < kWarps; ++i) {
            if (s.warp_total[i] > 0.0f) {
                hit_warp = i;
                before = run;
            }
            run += s.warp_total[i];
        }
    }

    if (warp == hit_warp) {
        const float rem = target - before;
        float base = 0.0f;  // running sum of this segment before the current step
        int found = -1, last_pos = -1;
        for (int gs = g0; gs < g1 && found < 0; gs += 32) {
            const int g = gs + lane;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (g < g1) v = w(g);
            const float mine = (v.x + v.y) + (v.z + v.w);
            const float incl = warp_inclusive_scan(mine, lane);
            const unsigned over = __ballot_sync(kFullMask, base + incl > rem);
            const unsigned pos = __ballot_sync(kFullMask, mine > 0.0f);
            if (pos) {
                const int pl = 31 - __clz(pos);  // last lane with positive weight in this step
                const float4 pv = make_float4(__shfl_sync(kFullMask, v.x, pl), __shfl_sync(kFullMask, v.y, pl),
                                              __shfl_sync(kFullMask, v.z, pl), __shfl_sync(kFullMask, v.w, pl));
                const int pg = 4 * (gs + pl);
                last_pos = pv.w > 0.f ? pg + 3 : pv.z > 0.f ? pg + 2 : pv.y > 0.f ? pg + 1 : pg;
            }
            if (over) {
                const int hl = __ffs(over) - 1;
                const float excl = __shfl_sync(kFullMask, incl - mine, hl) + base;
                const float4 hv = make_float4(__shfl_sync(kFullMask, v.x, hl), __shfl_sync(kFullMask, v.y, hl),
                                              __shfl_sync(kFullMask, v.z, hl), __shfl_sync(kFullMask, v.w, hl));
                const int hg = 4 * (gs + hl);
                float c = excl + hv.x;
                if (c > rem) found = hg;
                else if ((c += hv.y) > rem) found = hg + 1;
                else if ((c += hv.z) > rem) found = hg + 2;
                else found = hg + 3;
            }
            base += __shfl_sync(kFullMask, incl, 31);
        }
        if (lane == 0) {
            s.result = found;
            s.last_positive = last_pos;
        }
    }
    if (tid == 0) s.total = total;
    __syncthreads();
    int k = s.result >= 0 ? s.result : s.last_positive;
    k = max(0, min(k, vocab - 1));
    *total_out = s.total;
    __syncthreads();  // scratch may be reused by the caller
    return k;
}

struct ChunkStat {
    float max;   // chunk maximum
    float aux;   // T > 0: sum exp((l - max) / T) over the chunk; T = 0: argmax index as int bits
};

struct SharedState {
    float red[kWarps];
    int red_i[kWarps];
    float row_max[kMaxRows];
    float row_aux[kMaxRows];
    CdfScratch cdf;
    int flag;
    int n;
};

// grid = (chunks, rows, batch); rows = 2*gamma+1 (T > 0: p_1..p_{gamma+1}, q_1..q_gamma)
// or gamma+1 (T = 0: only p is read).
template <bool GREEDY>
__global__ void __launch_bounds__(kThreads)
verify_sample_kernel(const float* __restrict__ target_logits, const float* __restrict__ draft_logits,
                     const int32_t* __restrict__ draft_tokens, const float* __restrict__ uniforms, int gamma,
                     int vocab, float inv_t, ChunkStat* __restrict__ stats, unsigned* __restrict__ tickets,
                     int32_t* __restrict__ n_accepted, int32_t* __restrict__ next_token) {
    __shared__ SharedState sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunk = blockIdx.x, chunks = gridDim.x;
    const int row = blockIdx.y, rows = gridDim.y;
    const int b = blockIdx.z;

    const float* tl = target_logits + static_cast<size_t>(b) * (gamma + 1) * vocab;
    const float* ql = GREEDY ? nullptr : draft_logits + static_cast<size_t>(b) * gamma * vocab;
    const float* src = row <= gamma ? tl + static_cast<size_t>(row) * vocab
                                    : ql + static_cast<size_t>(row - gamma - 1) * vocab;
    const Row r = make_row(src, vocab);
    const int groups = (vocab + 3) >> 2;
    const int per_chunk = (groups + chunks - 1) / chunks;  // <= kChunkGroups by construction of the grid
    const int g0 = chunk * per_chunk;
    const int g1 = min(groups, g0 + per_chunk);

    // ---- statistics phase: this chunk's logits, each read exactly once ----
    float4 v[kGroupsPerThread];
#pragma unroll
    for (int i = 0; i < kGroupsPerThread; ++i) {
        const int g = g0 + tid + i * kThreads;
        v[i] = g < g1 ? r.load(g, -INFINITY) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
    float m = -INFINITY;
    int arg = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < kGroupsPerThread; ++i) {
        if (GREEDY) {
            const int j = 4 * (g0 + tid + i * kThreads);
            if (v[i].x > m) { m = v[i].x; arg = j; }
            if (v[i].y > m) { m = v[i].y; arg = j + 1; }
            if (v[i].z > m) { m = v[i].z; arg = j + 2; }
            if (v[i].w > m) { m = v[i].w; arg = j + 3; }
        } else {
            m = fmaxf(m, fmaxf(fmaxf(v[i].x, v[i].y), fmaxf(v[i].z, v[i].w)));
        }
    }
    if (GREEDY) {
        // (max, lowest index) across the block
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float om = __shfl_xor_sync(kFullMask, m, o);
            const int oa = __shfl_xor_sync(kFullMask, arg, o);
            if (om > m || (om == m && oa < arg)) { m = om; arg = oa; }
        }
        if (lane == 0) { sh.red[warp] = m; sh.red_i[warp] = arg; }
        __syncthreads();
        if (tid == 0) {
            for (int i = 1; i < kWarps; ++i)
                if (sh.red[i] > m || (sh.red[i] == m && sh.red_i[i] < arg)) { m = sh.red[i]; arg = sh.red_i[i]; }
            ChunkStat st;
            st.max = m;
            st.aux = __int_as_float(arg);
            stats[(static_cast<size_t>(b) * rows + row) * chunks + chunk] = st;
        }
    } else {
        m = warp_max(m);
        if (lane == 0) sh.red[warp] = m;
        __syncthreads();
        m = sh.red[0];
#pragma unroll
        for (int i = 1; i < kWarps; ++i) m = fmaxf(m, sh.red[i]);
        __syncthreads();
        float s = 0.0f;
        if (m > -INFINITY) {
#pragma unroll
            for (int i = 0; i < kGroupsPerThread; ++i)
                s += (expf((v[i].x - m) * inv_t) + expf((v[i].y - m) * inv_t)) +
                     (expf((v[i].z - m) * inv_t) + expf((v[i].w - m) * inv_t));
        }
        s = warp_sum(s);
        if (lane == 0) sh.red[warp] = s;
        __syncthreads();
        if (tid == 0) {
            float t = 0.0f;
#pragma unroll
            for (int i = 0; i < kWarps; ++i) t += sh.red[i];
            ChunkStat st;
            st.max = m;
            st.aux = t;
            stats[(static_cast<size_t>(b) * rows + row) * chunks + chunk] = st;
        }
    }

    // ---- ticket: the last CTA of this sequence does the rest ----
    if (tid == 0) {
        __threadfence();
        const unsigned prev = atomicAdd(&tickets[b], 1u);
        sh.flag = prev == static_cast<unsigned>(rows * chunks - 1);
    }
    __syncthreads();
    if (!sh.flag) return;
    __threadfence();

    // merge chunk statistics per row
    const ChunkStat* st_b = stats + static_cast<size_t>(b) * rows * chunks;
    for (int rr = tid; rr < rows; rr += kThreads) {
        float M = -INFINITY, A = 0.0f;
        int best = 0x7fffffff;
        for (int c = 0; c < chunks; ++c) {
            const float cm = __ldcg(&st_b[rr * chunks + c].max);
            const float ca = __ldcg(&st_b[rr * chunks + c].aux);
            if (GREEDY) {
                const int ci = __float_as_int(ca);
                if (cm > M || (cm == M && ci < best)) { M = cm; best = ci; }
            } else {
                M = fmaxf(M, cm);
            }
        }
        if (GREEDY) {
            A = __int_as_float(best);
        } else {
            for (int c = 0; c < chunks; ++c) {
                const float cm = __ldcg(&st_b[rr * chunks + c].max);
                const float ca = __ldcg(&st_b[rr * chunks + c].aux);
                if (cm > -INFINITY) A += ca * expf((cm - M) * inv_t);
            }
        }
        sh.row_max[rr] = M;
        sh.row_aux[rr] = A;
    }
    __syncthreads();

    // the gamma accept tests, in order (Algorithm 1: n = first rejection)
    if (tid == 0) {
        int n = gamma;
        for (int i = 0; i < gamma; ++i) {
            const int x = draft_tokens[static_cast<size_t>(b) * gamma + i];
            bool reject = true;
            if (x >= 0 && x < vocab) {
                if (GREEDY) {
                    reject = x != __float_as_int(sh.row_aux[i]);
                } else {
                    const float ep = expf((tl[static_cast<size_t>(i) * vocab + x] - sh.row_max[i]) * inv_t);
                    const float eq = expf((ql[static_cast<size_t>(i) * vocab + x] - sh.row_max[gamma + 1 + i]) * inv_t);
                    const float rr = uniforms[static_cast<size_t>(b) * (gamma + 1) + i];
                    // r * q(x) > p(x) with p = ep / Sp, q = eq / Sq, cross-multiplied
                    reject = rr * eq * sh.row_aux[i] > ep * sh.row_aux[gamma + 1 + i];
                }
            }
            if (reject) { n = i; break; }
        }
        sh.n = n;
    }
    __syncthreads();
    const int n = sh.n;

    int token;
    if (GREEDY) {
        token = __float_as_int(sh.row_aux[n]);
    } else {
        const float u = uniforms[static_cast<size_t>(b) * (gamma + 1) + gamma];
        PlainWeights pw;
        pw.p = make_row(tl + static_cast<size_t>(n) * vocab, vocab);
        pw.max_p = sh.row_max[n];
        pw.inv_t = inv_t;
        float total = 0.0f;
        bool plain = n == gamma;
        if (!plain) {
            ResidualWeights rw;
            rw.p = pw.p;
            rw.q = make_row(ql + static_cast<size_t>(n) * vocab, vocab);
            rw.max_p = sh.row_max[n];
            rw.max_q = sh.row_max[gamma + 1 + n];
            rw.inv_sum_p = 1.0f / sh.row_aux[n];
            rw.inv_sum_q = 1.0f / sh.row_aux[gamma + 1 + n];
            rw.inv_t = inv_t;
            token = block_inverse_cdf(rw, vocab, u, sh.cdf, &total);
            plain = !(total > 0.0f) || !isfinite(total);  // vanished residual: draw from p_{n+1}
        }
        if (plain) token = block_inverse_cdf(pw, vocab, u, sh.cdf, &total);
    }
    if (tid == 0) {
        n_accepted[b] = n;
        next_token[b] = token;
        tickets[b] = 0;  // leave the workspace ready for the next launch
    }
}

// One CTA per row: tokens[r] ~ softmax(logits[r] / T), or argmax at T = 0.
__global__ void __launch_bounds__(kThreads)
sample_kernel(const float* __restrict__ logits, const float* __restrict__ uniforms, int vocab, float inv_t,
              bool greedy, int32_t* __restrict__ tokens) {
    __shared__ SharedState sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const Row r = make_row(logits + static_cast<size_t>(blockIdx.x) * vocab, vocab);
    const int groups = (vocab + 3) >> 2;
    float m = -INFINITY;
    int arg = 0x7fffffff;
    for (int g = tid; g < groups; g += kThreads) {
        const float4 v = r.load(g, -INFINITY);
        const int j = 4 * g;
        if (v.x > m) { m = v.x; arg = j; }
        if (v.y > m) { m = v.y; arg = j + 1; }
        if (v.z > m) { m = v.z; arg = j + 2; }
        if (v.w > m) { m = v.w; arg = j + 3; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(kFullMask, m, o);
        const int oa = __shfl_xor_sync(kFullMask, arg, o);
        if (om > m || (om == m && oa < arg)) { m = om; arg = oa; }
    }
    if (lane == 0) { sh.red[warp] = m; sh.red_i[warp] = arg; }
    __syncthreads();
    m = sh.red[0];
    arg = sh.red_i[0];
#pragma unroll
    for (int i = 1; i < kWarps; ++i)
        if (sh.red[i] > m || (sh.red[i] == m && sh.red_i[i] < arg)) { m = sh.red[i]; arg = sh.red_i[i]; }
    __syncthreads();
    int token = arg;
    if (!greedy) {
        PlainWeights pw;
        pw.p = r;
        pw.max_p = m;
        pw.inv_t = inv_t;
        float total;
        token = block_inverse_cdf(pw, vocab, uniforms[blockIdx.x], sh.cdf, &total);
    }
    if (tid == 0) tokens[blockIdx.x] = max(0, min(token, vocab - 1));
}

__global__ void uniforms_kernel(uint64_t seed, const int32_t* __restrict__ positions,
                                const int32_t* __restrict__ sequences, uint32_t purpose, int count,
                                float* __restrict__ out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count)
        out[i] = method_uniform(seed, static_cast<uint32_t>(positions[i]), static_cast<uint32_t>(sequences[i]), purpose);
}

int chunks_for(int vocab) {
    const int groups = (vocab + 3) / 4;
    return (groups + kChunkGroups - 1) / kChunkGroups;
}

size_t tickets_bytes(int batch) { return (static_cast<size_t>(batch) * sizeof(unsigned) + 255) / 256 * 256; }

}  // namespace

// Shared with the generation loop (generate.cu): same launch, no argument checks.
int launch_verify_sample(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                         const float* uniforms, int batch, int gamma, int vocab, float temperature,
                         int32_t* n_accepted, int32_t* next_token, void* workspace, cudaStream_t stream) {
    const bool greedy = temperature == 0.0f;
    const int chunks = chunks_for(vocab);
    const int rows = greedy ? gamma + 1 : 2 * gamma + 1;
    unsigned* tickets = static_cast<unsigned*>(workspace);
    ChunkStat* stats = reinterpret_cast<ChunkStat*>(static_cast<char*>(workspace) + tickets_bytes(batch));
    SPEC_CUDA_TRY(cudaMemsetAsync(tickets, 0, static_cast<size_t>(batch) * sizeof(unsigned), stream));
    const dim3 grid(chunks, rows, batch);
    if (greedy)
        verify_sample_kernel<true><<<grid, kThreads, 0, stream>>>(target_logits, draft_logits, draft_tokens, uniforms,
                                                                  gamma, vocab, 0.0f, stats, tickets, n_accepted,
                                                                  next_token);
    else
        verify_sample_kernel<false><<<grid, kThreads, 0, stream>>>(target_logits, draft_logits, draft_tokens, uniforms,
                                                                   gamma, vocab, 1.0f / temperature, stats, tickets,
                                                                   n_accepted, next_token);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_sample(const float* logits, const float* uniforms, int rows, int vocab, float temperature,
                  int32_t* tokens, cudaStream_t stream) {
    const bool greedy = temperature == 0.0f;
    sample_kernel<<<rows, kThreads, 0, stream>>>(logits, uniforms, vocab, greedy ? 0.0f : 1.0f / temperature, greedy,
                                                 tokens);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

}  // namespace spec

extern "C" size_t spec_verify_sample_workspace_bytes(int batch, int gamma, int vocab) {
    if (batch < 0 || gamma < 0 || vocab < 1) return 0;
    const size_t rows = 2 * static_cast<size_t>(gamma) + 1;
    return spec::tickets_bytes(batch) + static_cast<size_t>(batch) * rows * spec::chunks_for(vocab) * sizeof(spec::ChunkStat) + 256;
}

extern "C" int spec_verify_sample(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                                  const float* uniforms, int batch, int gamma, int vocab, float temperature,
                                  int32_t* n_accepted, int32_t* next_token, void* workspace, size_t workspace_bytes,
                                  void* stream) {
    using namespace spec;
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
    return launch_verify_sample(target_logits, draft_logits, draft_tokens, uniforms, batch, gamma, vocab, temperature,
                                n_accepted, next_token, workspace, static_cast<cudaStream_t>(stream));
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
