// Attention of the rows of a pass against paged K,V rows: causal over the
// decoder cache (row at position p sees keys 0..p), or over a fixed set of keys
// per sequence (the encoder's own rows; the cross-attention rows of an
// encoder-decoder), optionally with an additive relative-position bias.
//
// Work is cut by (sequence, KV head, slice of the keys).  A CTA owns one such
// piece and runs one warp per query that reads this KV head: the G query heads
// of the group times the m new rows of the sequence.  All warps of the CTA walk
// the same 32-key tiles, so the K and V rows come from HBM/L2 once per CTA and
// from L1 for the other queries.  Lane l owns d_head/32 consecutive elements of
// the head dimension throughout, so every load of a K or V row is one coalesced
// span (a page stores the rows of one head back to back).  For Q.K^T each lane
// forms its share of the 32 dot products of a tile and a 31-shuffle butterfly
// (reduce-scatter) leaves the score of key l in lane l; the warp keeps an online
// softmax (running max and sum, fp32).  For P.V every key's probability is
// broadcast with a shuffle.  A tile never straddles a page (pages hold a
// multiple of 32 tokens).
//
// Each CTA writes an unnormalised partial state (max, sum, accumulator) per
// query; attention_combine_kernel merges the key slices and emits the
// out-projection's input (fp32 and/or split into two bf16 terms).
#include <cfloat>

#include "model.cuh"

namespace spec {
namespace {

constexpr int kMaxAttnWarps = 16;
constexpr int kVBatch = 16;

template <typename KV>
struct KvLoad;

template <>
struct KvLoad<float> {
    static constexpr int kVec = 4;  // elements per 16-byte load
    __device__ static __forceinline__ void load(const float* p, float* out) {
        const float4 t = *reinterpret_cast<const float4*>(p);
        out[0] = t.x; out[1] = t.y; out[2] = t.z; out[3] = t.w;
    }
    template <int N>
    __device__ static __forceinline__ void load_n(const float* p, float* out) {
        if (N == 4) {
            load(p, out);
        } else {
            const float2 t = *reinterpret_cast<const float2*>(p);
            out[0] = t.x; out[1] = t.y;
        }
    }
};

template <>
struct KvLoad<__nv_bfloat16> {
    static constexpr int kVec = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16* p, float* out) {
        const uint4 t = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    template <int N>
    __device__ static __forceinline__ void load_n(const __nv_bfloat16* p, float* out) {
        if (N == 4) {
            const uint2 t = *reinterpret_cast<const uint2*>(p);
            out[0] = __uint_as_float(t.x << 16); out[1] = __uint_as_float(t.x & 0xffff0000u);
            out[2] = __uint_as_float(t.y << 16); out[3] = __uint_as_float(t.y & 0xffff0000u);
        } else {
            const uint32_t t = *reinterpret_cast<const uint32_t*>(p);
            out[0] = __uint_as_float(t << 16); out[1] = __uint_as_float(t & 0xffff0000u);
        }
    }
};

// grid = (slices, n_kv_heads, batch), block = 32 * warps (warps <= kMaxAttnWarps).
// Rows of sequence b are rows b*m .. b*m+m-1 of the pass.
template <typename KV, int DH>
__global__ void __launch_bounds__(32 * kMaxAttnWarps)
attention_kernel(const float* __restrict__ qkv, int q_stride, const int32_t* __restrict__ pos,
                 const int32_t* __restrict__ seq, int m_rows, int n_heads, int n_kv_heads, int ks,
                 const KV* __restrict__ kv_layer, const int32_t* __restrict__ page_table, int pages_per_seq,
                 int page_size, const int32_t* __restrict__ kv_len, const float* __restrict__ bias, int bias_span,
                 int bias_zero, float scale, float* __restrict__ part) {
    constexpr int PER_LANE = DH / 32;
    __shared__ float share[kMaxAttnWarps][DH + 2];  // states of the warps that share a query (ks > 1)
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    const int slice = blockIdx.x, slices = gridDim.x, kv_head = blockIdx.y, b = blockIdx.z;
    const int group = n_heads / n_kv_heads;
    const int queries = group * m_rows;

    // the key range of this slice: whole tiles, same for every query of the sequence
    int seq_keys = 0;
    if (kv_len) {
        seq_keys = kv_len[seq[b * m_rows]];
    } else {
        for (int j = 0; j < m_rows; ++j) seq_keys = max(seq_keys, pos[b * m_rows + j] + 1);
    }
    const int tiles = (seq_keys + 31) / 32;
    const int t0 = static_cast<int>(static_cast<long long>(tiles) * slice / slices);
    const int t1 = static_cast<int>(static_cast<long long>(tiles) * (slice + 1) / slices);

    const size_t head_stride = static_cast<size_t>(page_size) * DH;               // one head inside a page
    const size_t page_stride = 2 * static_cast<size_t>(n_kv_heads) * head_stride;  // K block + V block
    const size_t v_offset = static_cast<size_t>(n_kv_heads) * head_stride;

    // Work unit u = (query q, sub-slice sub): with ks > 1 the ks warps q, q + queries,
    // ... share query q and take every ks-th tile of the slice (then the block has
    // exactly queries * ks warps and this loop runs once).
    for (int u = warp; u < queries * ks; u += warps) {
        const int q = u % queries, sub = u / queries;
        const int j = q / group, head = kv_head * group + q % group;
        const int r = b * m_rows + j;
        const int p = pos[r];
        const int32_t* pages = page_table + seq[r] * pages_per_seq;
        float qv[PER_LANE];  // this lane's share of the (scaled) query
        KvLoad<float>::template load_n<PER_LANE>(qkv + static_cast<size_t>(r) * q_stride + head * DH + lane * PER_LANE, qv);
#pragma unroll
        for (int i = 0; i < PER_LANE; ++i) qv[i] *= scale;

        float mx = -FLT_MAX, l = 0.0f;
        float acc[PER_LANE];
#pragma unroll
        for (int i = 0; i < PER_LANE; ++i) acc[i] = 0.0f;
        // causal: positions 0..p; otherwise the sequence's key set (p < 0: inactive row, no keys)
        const int n_keys = kv_len ? (p >= 0 ? seq_keys : 0) : p + 1;
        const float* bias_row = bias ? bias + static_cast<size_t>(head) * bias_span + (bias_zero - p) : nullptr;
        for (int t = t0 + sub; t < t1; t += ks) {
            const int k0 = 32 * t;
            if (k0 >= n_keys) break;
            // the whole tile lives in one page
            const KV* tile = kv_layer + pages[k0 / page_size] * page_stride + kv_head * head_stride +
                             static_cast<size_t>(k0 % page_size) * DH;
            const int in_tile = min(32, n_keys - k0);
            // partial dot products of all 32 keys over this lane's elements ...
            float pd[32];
            const KV* kt = tile + lane * PER_LANE;
#pragma unroll
            for (int k = 0; k < 32; ++k) {
                float kv[PER_LANE];
                if (k < in_tile) {
                    KvLoad<KV>::template load_n<PER_LANE>(kt + static_cast<size_t>(k) * DH, kv);
                } else {
#pragma unroll
                    for (int i = 0; i < PER_LANE; ++i) kv[i] = 0.0f;
                }
                float d = 0.0f;
#pragma unroll
                for (int i = 0; i < PER_LANE; ++i) d = fmaf(qv[i], kv[i], d);
                pd[k] = d;
            }
            // ... summed over the lanes by a butterfly that halves the live values
            // at every step: lane l ends with the full score of key l
#pragma unroll
            for (int step = 16; step > 0; step >>= 1) {
                const bool upper = (lane & step) != 0;
#pragma unroll
                for (int i = 0; i < step; ++i) {
                    const float keep = upper ? pd[i + step] : pd[i];
                    const float send = upper ? pd[i] : pd[i + step];
                    pd[i] = keep + __shfl_xor_sync(kFullMask, send, step);
                }
            }
            float s = -FLT_MAX;
            if (lane < in_tile) s = bias_row ? pd[0] + bias_row[k0 + lane] : pd[0];
            const float m_new = fmaxf(mx, warp_max(s));
            const float pr = lane < in_tile ? expf(s - m_new) : 0.0f;
            const float rescale = expf(mx - m_new);
            l = l * rescale + warp_sum(pr);
            mx = m_new;
#pragma unroll
            for (int i = 0; i < PER_LANE; ++i) acc[i] *= rescale;
            const KV* vt = tile + v_offset + lane * PER_LANE;
#pragma unroll
            for (int j0 = 0; j0 < 32; j0 += kVBatch) {
                if (j0 < in_tile) {
                    float vv[kVBatch][PER_LANE];
#pragma unroll
                    for (int jj = 0; jj < kVBatch; ++jj) {
                        if (j0 + jj < in_tile) {
                            KvLoad<KV>::template load_n<PER_LANE>(vt + static_cast<size_t>(j0 + jj) * DH, vv[jj]);
                        } else {
#pragma unroll
                            for (int i = 0; i < PER_LANE; ++i) vv[jj][i] = 0.0f;
                        }
                    }
#pragma unroll
                    for (int jj = 0; jj < kVBatch; ++jj) {
                        const float pj = __shfl_sync(kFullMask, pr, j0 + jj);
#pragma unroll
                        for (int i = 0; i < PER_LANE; ++i) acc[i] = fmaf(pj, vv[jj][i], acc[i]);
                    }
                }
            }
        }
        if (ks > 1) {  // park the state; warp `q` merges the ks of them below
            if (lane == 0) {
                share[warp][0] = mx;
                share[warp][1] = l;
            }
#pragma unroll
            for (int i = 0; i < PER_LANE; ++i) share[warp][2 + lane * PER_LANE + i] = acc[i];
        } else {
            // partial state of (row r, head, slice): [max, sum, acc[DH]]
            float* out = part + ((static_cast<size_t>(r) * n_heads + head) * slices + slice) * (DH + 2);
            if (lane == 0) {
                out[0] = mx;
                out[1] = l;
            }
#pragma unroll
            for (int i = 0; i < PER_LANE; ++i) out[2 + lane * PER_LANE + i] = acc[i];
        }
    }
    if (ks > 1) {
        __syncthreads();
        if (warp < queries) {
            const int q = warp;
            const int j = q / group, head = kv_head * group + q % group;
            const int r = b * m_rows + j;
            float mm = -FLT_MAX;
            for (int s = 0; s < ks; ++s) mm = fmaxf(mm, share[q + s * queries][0]);
            float l = 0.0f, acc[PER_LANE];
#pragma unroll
            for (int i = 0; i < PER_LANE; ++i) acc[i] = 0.0f;
            for (int s = 0; s < ks; ++s) {  // sub-slices in index order
                const float* st = share[q + s * queries];
                const float w = expf(st[0] - mm);
                l += st[1] * w;
#pragma unroll
                for (int i = 0; i < PER_LANE; ++i) acc[i] += st[2 + lane * PER_LANE + i] * w;
            }
            float* out = part + ((static_cast<size_t>(r) * n_heads + head) * slices + slice) * (DH + 2);
            if (lane == 0) {
                out[0] = mm;
                out[1] = l;
            }
#pragma unroll
            for (int i = 0; i < PER_LANE; ++i) out[2 + lane * PER_LANE + i] = acc[i];
        }
    }
}

// grid = rows * n_heads, block = DH: merge the key slices of one (row, head).
template <int DH>
__global__ void attention_combine_kernel(const float* __restrict__ part, int slices, float* __restrict__ att,
                                         __nv_bfloat16* __restrict__ att_hi, __nv_bfloat16* __restrict__ att_lo) {
    __shared__ float w_sh[64];  // weight of every slice, then their normaliser at [slices]
    pdl_trigger();
    pdl_wait();
    const float* in = part + static_cast<size_t>(blockIdx.x) * slices * (DH + 2);
    if (threadIdx.x < 32) {  // slices <= 32: one lane per slice
        const int s = threadIdx.x;
        const float ms = s < slices ? in[s * (DH + 2)] : -FLT_MAX;
        const float ls = s < slices ? in[s * (DH + 2) + 1] : 0.0f;
        const float mm = warp_max(ms);
        const float w = s < slices ? expf(ms - mm) : 0.0f;
        const float l = warp_sum(ls * w);
        if (s < slices) w_sh[s] = w;
        if (s == 0) w_sh[32] = l;
    }
    __syncthreads();
    float o = 0.0f;
#pragma unroll 8
    for (int s = 0; s < slices; ++s) o += in[s * (DH + 2) + 2 + threadIdx.x] * w_sh[s];
    const float l = w_sh[32];
    const float y = l > 0.0f ? o / l : 0.0f;  // an inactive row has no keys
    const size_t i = static_cast<size_t>(blockIdx.x) * DH + threadIdx.x;
    if (att) att[i] = y;
    if (att_hi) {
        const __nv_bfloat16 h = __float2bfloat16_rn(y);
        att_hi[i] = h;
        att_lo[i] = __float2bfloat16_rn(y - __bfloat162float(h));
    }
}

}  // namespace

// Warps that share one query inside a CTA (only when all queries then fit the
// block in one round), and key slices (CTAs) per (sequence, KV head): about one
// 32-key tile per warp when the batch is small, one wave of CTAs at most.
int attention_sub_slices(int queries) {
    return queries * 2 <= kMaxAttnWarps ? kMaxAttnWarps / queries : 1;
}

int attention_slices(int batch, int n_kv_heads, int queries, int max_len) {
    const int ks = attention_sub_slices(queries);
    // CTAs that fit the GPU at once: the kernel holds 128 registers per thread, so an
    // SM takes 16 warps of it; one wave of CTAs beats more, thinner slices
    const int warps = std::min(kMaxAttnWarps, std::max(1, queries * ks));
    const int resident = 148 * std::max(1, 16 / warps);
    const int want = std::max(1, resident / (batch * n_kv_heads));
    const int tiles = (max_len + 31) / 32;
    const int most = std::max(1, (tiles + ks - 1) / ks);
    return std::max(1, std::min(std::min(want, most), 32));
}

size_t attention_partial_elems(int rows, int n_heads, int d_head, int slices) {
    return static_cast<size_t>(rows) * n_heads * slices * (d_head + 2);
}

int launch_attention(const Model& m, const AttnSource& src, const RowMeta& rows, int batch, int m_rows, int slices,
                     float* part, float* att, __nv_bfloat16* att_hi, __nv_bfloat16* att_lo, cudaStream_t stream) {
    const int group = m.cfg.n_heads / m.cfg.n_kv_heads;
    const int ks = attention_sub_slices(group * m_rows);
    const int warps = std::min(kMaxAttnWarps, std::max(1, group * m_rows * ks));
    const dim3 grid(slices, m.cfg.n_kv_heads, batch);
    const float scale = 1.0f / sqrtf(static_cast<float>(m.cfg.d_head));
    const int n_rows = batch * m_rows;
#define SPEC_ATTN(KV, DH)                                                                                         \
    do {                                                                                                          \
        int status = launch_pdl(attention_kernel<KV, DH>, grid, dim3(32 * warps), 0, stream, src.q, src.q_stride, \
                                rows.pos, rows.seq, m_rows, m.cfg.n_heads, m.cfg.n_kv_heads, ks,                  \
                                static_cast<const KV*>(src.pool.kv), src.pool.page_table, src.pool.pages_per_seq,     \
                                src.pool.page_size,                                                               \
                                src.kv_len, src.bias, src.bias_span, src.bias_zero, scale, part);                 \
        if (status != SPEC_OK) return status;                                                                     \
        return launch_pdl(attention_combine_kernel<DH>, dim3(n_rows * m.cfg.n_heads), dim3(DH), 0, stream,         \
                          static_cast<const float*>(part), slices, att, att_hi, att_lo);                          \
    } while (0)
    if (src.pool.elem_bytes == 2) {
        if (m.cfg.d_head == 64) SPEC_ATTN(__nv_bfloat16, 64);
        else SPEC_ATTN(__nv_bfloat16, 128);
    } else {
        if (m.cfg.d_head == 64) SPEC_ATTN(float, 64);
        else SPEC_ATTN(float, 128);
    }
#undef SPEC_ATTN
    return SPEC_OK;
}

}  // namespace spec
