// Causal attention of the new rows against the paged KV cache.
//
// One CTA per (row, query head); its warps split the keys between them in tiles
// of 32 (tile t goes to warp t mod kAttnWarps) and merge their partial softmax
// states at the end.  Inside a tile each lane owns one key: it reads that key's
// d_head values with 16-byte loads (a page stores the keys of one head back to
// back, so a warp's loads cover one contiguous span), takes the dot product
// with the query held in shared memory, and the warp keeps an online softmax
// (running max and sum, fp32).  For P.V the lanes turn to the head dimension:
// lane l owns d_head/32 output elements, the tile's V rows are fetched eight at
// a time, and every key's probability is broadcast with a shuffle.  A tile
// never straddles a page (pages hold a multiple of 32 tokens).
#include <cfloat>

#include "model.cuh"

namespace spec {
namespace {

constexpr int kAttnWarps = 8;

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

// grid = rows * n_heads, block = 32 * kAttnWarps
template <typename KV, int DH>
__global__ void __launch_bounds__(32 * kAttnWarps)
attention_kernel(const float* __restrict__ qkv, const int32_t* __restrict__ pos, const int32_t* __restrict__ seq,
                 int n_heads, int n_kv_heads, const KV* __restrict__ kv_layer,
                 const int32_t* __restrict__ page_table, int pages_per_seq, int page_size, float scale,
                 float* __restrict__ att) {
    constexpr int PER_LANE = DH / 32;
    __shared__ float q_sh[DH];
    __shared__ float part_m[kAttnWarps], part_l[kAttnWarps];
    __shared__ float part_acc[kAttnWarps][DH];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = blockIdx.x / n_heads, head = blockIdx.x % n_heads;
    const int p = pos[r];
    float* out = att + (static_cast<size_t>(r) * n_heads + head) * DH;
    if (p < 0) {  // inactive row
        for (int i = threadIdx.x; i < DH; i += blockDim.x) out[i] = 0.0f;
        return;
    }
    const int kv_head = head / (n_heads / n_kv_heads);
    const int qkv_dim = (n_heads + 2 * n_kv_heads) * DH;
    const float* q = qkv + static_cast<size_t>(r) * qkv_dim + head * DH;
    for (int i = threadIdx.x; i < DH; i += blockDim.x) q_sh[i] = q[i] * scale;
    __syncthreads();

    const int32_t* pages = page_table + seq[r] * pages_per_seq;
    const size_t head_stride = static_cast<size_t>(page_size) * DH;               // one head inside a page
    const size_t page_stride = 2 * static_cast<size_t>(n_kv_heads) * head_stride;  // K block + V block
    const size_t v_offset = static_cast<size_t>(n_kv_heads) * head_stride;

    float m = -FLT_MAX, l = 0.0f;
    float acc[PER_LANE];
#pragma unroll
    for (int i = 0; i < PER_LANE; ++i) acc[i] = 0.0f;

    const int n_keys = p + 1;  // causal: positions 0..p
    for (int k0 = 32 * warp; k0 < n_keys; k0 += 32 * kAttnWarps) {
        // the whole tile lives in one page
        const KV* tile = kv_layer + pages[k0 / page_size] * page_stride + kv_head * head_stride +
                         static_cast<size_t>(k0 % page_size) * DH;
        const int in_tile = min(32, n_keys - k0);
        float s = -FLT_MAX;
        if (lane < in_tile) {
            const KV* kp = tile + static_cast<size_t>(lane) * DH;
            float dot = 0.0f;
#pragma unroll
            for (int d0 = 0; d0 < DH; d0 += KvLoad<KV>::kVec) {
                float kvv[KvLoad<KV>::kVec];
                KvLoad<KV>::load(kp + d0, kvv);
#pragma unroll
                for (int e = 0; e < KvLoad<KV>::kVec; ++e) dot = fmaf(q_sh[d0 + e], kvv[e], dot);
            }
            s = dot;
        }
        const float m_new = fmaxf(m, warp_max(s));
        const float pr = lane < in_tile ? expf(s - m_new) : 0.0f;
        const float rescale = expf(m - m_new);
        l = l * rescale + warp_sum(pr);
        m = m_new;
#pragma unroll
        for (int i = 0; i < PER_LANE; ++i) acc[i] *= rescale;
        const KV* vt = tile + v_offset + lane * PER_LANE;
        for (int j0 = 0; j0 < in_tile; j0 += 8) {
            float vv[8][PER_LANE];
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int i = 0; i < PER_LANE; ++i)
                    vv[j][i] = j0 + j < in_tile ? KvLoad<KV>::one(vt + static_cast<size_t>(j0 + j) * DH + i) : 0.0f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float pj = __shfl_sync(kFullMask, pr, (j0 + j) & 31);
#pragma unroll
                for (int i = 0; i < PER_LANE; ++i) acc[i] = fmaf(pj, vv[j][i], acc[i]);
            }
        }
    }
    // merge the warps' partial states
    if (lane == 0) { part_m[warp] = m; part_l[warp] = l; }
#pragma unroll
    for (int i = 0; i < PER_LANE; ++i) part_acc[warp][lane * PER_LANE + i] = acc[i];
    __syncthreads();
    float mm = part_m[0];
#pragma unroll
    for (int w = 1; w < kAttnWarps; ++w) mm = fmaxf(mm, part_m[w]);
    float ll = 0.0f;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) ll += part_l[w] * expf(part_m[w] - mm);
    for (int i = threadIdx.x; i < DH; i += blockDim.x) {
        float o = 0.0f;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) o += part_acc[w][i] * expf(part_m[w] - mm);
        out[i] = o / ll;
    }
}

}  // namespace

int launch_attention(const Model& m, int layer, const RowMeta& rows, int n_rows, const float* qkv, float* att,
                     const int32_t* page_table, int pages_per_seq, int page_size, cudaStream_t stream) {
    const char* kv_layer = static_cast<const char*>(m.kv) + static_cast<size_t>(layer) * m.layer_stride;
    const int grid = n_rows * m.cfg.n_heads;
    const float scale = 1.0f / sqrtf(static_cast<float>(m.cfg.d_head));
#define SPEC_ATTN(KV, DH)                                                                                       \
    attention_kernel<KV, DH><<<grid, 32 * kAttnWarps, 0, stream>>>(                                             \
        qkv, rows.pos, rows.seq, m.cfg.n_heads, m.cfg.n_kv_heads, reinterpret_cast<const KV*>(kv_layer),         \
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
