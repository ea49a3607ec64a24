// Causal attention of the new rows against the paged KV cache.
//
// One warp per (row, query head).  Keys are taken 32 at a time, one per lane:
// a lane reads its key's d_head values with 16-byte loads (a page stores the
// keys of one head back to back, so a warp's loads cover one contiguous span),
// takes the dot product with the query held in shared memory, and the warp
// keeps an online softmax (running max and sum, fp32).  For P.V the lanes turn
// to the head dimension: lane l owns d_head/32 output elements and every key's
// probability is broadcast with a shuffle.
#include <cfloat>

#include "model.cuh"

namespace spec {
namespace {

constexpr int kAttnWarps = 4;

template <typename KV>
struct KvLoad;

template <>
struct KvLoad<float> {
    static constexpr int kVec = 4;  // elements per 16-byte load
    __device__ static __forceinline__ void load(const float* p, float* out) {
        const float4 t = *reinterpret_cast<const float4*>(p);
        out[0] = t.x; out[1] = t.y; out[2] = t.z; out[3] = t.w;
    }
    __device__ static __forceinline__ float one(const float* p) { return *p; }
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
    __device__ static __forceinline__ float one(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};

// grid = ceil(rows * n_heads / kAttnWarps), block = 32 * kAttnWarps
template <typename KV, int DH>
__global__ void __launch_bounds__(32 * kAttnWarps)
attention_kernel(const float* __restrict__ qkv, const int32_t* __restrict__ pos, const int32_t* __restrict__ seq,
                 int n_rows, int n_heads, int n_kv_heads, const KV* __restrict__ kv_layer,
                 const int32_t* __restrict__ page_table, int pages_per_seq, int page_size, float scale,
                 float* __restrict__ att) {
    __shared__ float q_sh[kAttnWarps][DH];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int task = blockIdx.x * kAttnWarps + warp;
    if (task >= n_rows * n_heads) return;
    const int r = task / n_heads, head = task % n_heads;
    const int p = pos[r];
    constexpr int PER_LANE = DH / 32;
    float* out = att + (static_cast<size_t>(r) * n_heads + head) * DH;
    if (p < 0) {
#pragma unroll
        for (int i = 0; i < PER_LANE; ++i) out[lane * PER_LANE + i] = 0.0f;
        return;
    }
    const int kv_head = head / (n_heads / n_kv_heads);
    const int qkv_dim = (n_heads + 2 * n_kv_heads) * DH;
    const float* q = qkv + static_cast<size_t>(r) * qkv_dim + head * DH;
    for (int i = lane; i < DH; i += 32) q_sh[warp][i] = q[i] * scale;
    __syncwarp();

    const int32_t* pages = page_table + seq[r] * pages_per_seq;
    const size_t head_stride = static_cast<size_t>(page_size) * DH;             // one head inside a page
    const size_t page_stride = 2 * static_cast<size_t>(n_kv_heads) * head_stride;  // K block + V block
    const size_t v_offset = static_cast<size_t>(n_kv_heads) * head_stride;

    float m = -FLT_MAX, l = 0.0f;
    float acc[PER_LANE];
#pragma unroll
    for (int i = 0; i < PER_LANE; ++i) acc[i] = 0.0f;

    const int n_keys = p + 1;  // causal: positions 0..p
    for (int k0 = 0; k0 < n_keys; k0 += 32) {
        const int key = k0 + lane;
        float s = -FLT_MAX;
        if (key < n_keys) {
            const KV* kp = kv_layer + pages[key / page_size] * page_stride + kv_head * head_stride +
                           static_cast<size_t>(key % page_size) * DH;
            float dot = 0.0f;
#pragma unroll
            for (int d0 = 0; d0 < DH; d0 += KvLoad<KV>::kVec) {
                float kvv[KvLoad<KV>::kVec];
                KvLoad<KV>::load(kp + d0, kvv);
#pragma unroll
                for (int e = 0; e < KvLoad<KV>::kVec; ++e) dot = fmaf(q_sh[warp][d0 + e], kvv[e], dot);
            }
            s = dot;
        }
        const float m_new = fmaxf(m, warp_max(s));
        const float pr = key < n_keys ? expf(s - m_new) : 0.0f;
        const float rescale = expf(m - m_new);
        l = l * rescale + warp_sum(pr);
        m = m_new;
#pragma unroll
        for (int i = 0; i < PER_LANE; ++i) acc[i] *= rescale;
        const int in_tile = min(32, n_keys - k0);
        for (int j = 0; j < in_tile; ++j) {
            const float pj = __shfl_sync(kFullMask, pr, j);
            const int kj = k0 + j;
            const KV* vp = kv_layer + pages[kj / page_size] * page_stride + v_offset + kv_head * head_stride +
                           static_cast<size_t>(kj % page_size) * DH + lane * PER_LANE;
#pragma unroll
            for (int i = 0; i < PER_LANE; ++i) acc[i] = fmaf(pj, KvLoad<KV>::one(vp + i), acc[i]);
        }
    }
    const float inv = 1.0f / l;
#pragma unroll
    for (int i = 0; i < PER_LANE; ++i) out[lane * PER_LANE + i] = acc[i] * inv;
}

}  // namespace

int launch_attention(const Model& m, int layer, const RowMeta& rows, int n_rows, const float* qkv, float* att,
                     const int32_t* page_table, int pages_per_seq, int page_size, cudaStream_t stream) {
    const char* kv_layer = static_cast<const char*>(m.kv) + static_cast<size_t>(layer) * m.layer_stride;
    const int tasks = n_rows * m.cfg.n_heads;
    const int grid = (tasks + kAttnWarps - 1) / kAttnWarps;
    const float scale = 1.0f / sqrtf(static_cast<float>(m.cfg.d_head));
#define SPEC_ATTN(KV, DH)                                                                                       \
    attention_kernel<KV, DH><<<grid, 32 * kAttnWarps, 0, stream>>>(                                             \
        qkv, rows.pos, rows.seq, n_rows, m.cfg.n_heads, m.cfg.n_kv_heads, reinterpret_cast<const KV*>(kv_layer), \
        page_table, pages_per_seq, page_size, scale, att)
    if (m.kv_elem_bytes == 2) {
        if (m.cfg.d_head == 64) SPEC_ATTN(__nv_bfloat16, 64);
        else SPEC_ATTN(__nv_bfloat16, 128);
    } else {
        if (m.cfg.d_head == 64) SPEC_ATTN(float, 64);
        else SPEC_ATTN(float, 128);
    }
#undef SPEC_ATTN
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

}  // namespace spec
