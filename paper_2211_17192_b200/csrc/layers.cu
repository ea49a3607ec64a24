// The small kernels of a decoder block: embedding gather, RMSNorm, rotary
// positions + K/V append into the paged cache, FFN activations.  All of them
// move O(rows * d) bytes and exist to keep the residual stream in fp32 around
// the weight-streaming GEMMs.
#include "model.cuh"

namespace spec {
namespace {

__device__ __forceinline__ float load_elem(const void* base, size_t i, bool bf16) {
    return bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(base)[i]) : static_cast<const float*>(base)[i];
}

// grid = rows, block = 128
__global__ void embed_kernel(const void* __restrict__ tok_emb, const void* __restrict__ pos_emb, bool bf16,
                             bool add_pos, const int32_t* __restrict__ token, const int32_t* __restrict__ pos, int d,
                             int vocab, int max_positions, float* __restrict__ h) {
    const int r = blockIdx.x;
    const int t = min(max(token[r], 0), vocab - 1);
    const int p = min(max(pos[r], 0), max_positions - 1);
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = load_elem(tok_emb, static_cast<size_t>(t) * d + i, bf16);
        if (add_pos) v += load_elem(pos_emb, static_cast<size_t>(p) * d + i, bf16);
        h[static_cast<size_t>(r) * d + i] = v;
    }
}

// grid = rows, block = 256; d is a multiple of 4
__global__ void rmsnorm_kernel(const float* __restrict__ in, const float* __restrict__ gain,
                               const int32_t* __restrict__ src_rows, int d, float eps, float* __restrict__ out) {
    __shared__ float red[8];
    const int r = blockIdx.x;
    const float4* x = reinterpret_cast<const float4*>(in + static_cast<size_t>(src_rows ? src_rows[r] : r) * d);
    const float4* g = reinterpret_cast<const float4*>(gain);
    float4* y = reinterpret_cast<float4*>(out + static_cast<size_t>(r) * d);
    float ss = 0.0f;
    for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {
        const float4 v = x[i];
        ss += (v.x * v.x + v.y * v.y) + (v.z * v.z + v.w * v.w);
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float total = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) total += red[i];
    const float scale = rsqrtf(total / static_cast<float>(d) + eps);
    for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {
        const float4 v = x[i];
        const float4 gg = g[i];
        y[i] = make_float4(v.x * scale * gg.x, v.y * scale * gg.y, v.z * scale * gg.z, v.w * scale * gg.w);
    }
}

// grid = rows, block = 128.  qkv row layout: [q heads | k heads | v heads], d_head each.
template <typename KV>
__global__ void rope_append_kernel(float* __restrict__ qkv, const int32_t* __restrict__ pos,
                                   const int32_t* __restrict__ seq, int n_heads, int n_kv_heads, int d_head,
                                   bool rotary, float rope_base, KV* __restrict__ kv_layer,
                                   const int32_t* __restrict__ page_table, int pages_per_seq, int page_size) {
    const int r = blockIdx.x;
    const int p = pos[r];
    if (p < 0) return;
    const int half = d_head / 2;
    float* row = qkv + static_cast<size_t>(r) * (n_heads + 2 * n_kv_heads) * d_head;
    if (rotary) {
        // q heads and k heads are contiguous: (n_heads + n_kv_heads) * half rotations
        const int pairs = (n_heads + n_kv_heads) * half;
        for (int i = threadIdx.x; i < pairs; i += blockDim.x) {
            const int head = i / half, j = i % half;
            // angle = position * base^(-2j / d_head), evaluated in double so that
            // large positions do not lose the fractional turn
            const double inv_freq = pow(static_cast<double>(rope_base), -2.0 * j / static_cast<double>(d_head));
            double s, c;
            sincos(static_cast<double>(p) * inv_freq, &s, &c);
            float* hp = row + head * d_head;
            const float x1 = hp[j], x2 = hp[j + half];
            hp[j] = x1 * static_cast<float>(c) - x2 * static_cast<float>(s);
            hp[j + half] = x2 * static_cast<float>(c) + x1 * static_cast<float>(s);
        }
        __syncthreads();
    }
    const int page = page_table[seq[r] * pages_per_seq + p / page_size];
    const int slot = p % page_size;
    const int kv_dim = n_kv_heads * d_head;
    const float* k = row + n_heads * d_head;
    const float* v = k + kv_dim;
    for (int i = threadIdx.x; i < kv_dim; i += blockDim.x) {
        const int head = i / d_head, e = i % d_head;
        const size_t base = ((static_cast<size_t>(page) * 2) * n_kv_heads + head) * page_size + slot;
        const size_t v_off = static_cast<size_t>(n_kv_heads) * page_size;
        kv_layer[base * d_head + e] = static_cast<KV>(k[i]);
        kv_layer[(base + v_off) * d_head + e] = static_cast<KV>(v[i]);
    }
}

__device__ __forceinline__ float gelu_tanh(float x) {
    const float k = 0.7978845608028654f;  // sqrt(2 / pi)
    return 0.5f * x * (1.0f + tanhf(k * (x + 0.044715f * x * x * x)));
}

__device__ __forceinline__ float silu(float x) { return x / (1.0f + expf(-x)); }

__global__ void ffn_act_kernel(const float* __restrict__ u, int n_rows, int d_ff, int ffn, float* __restrict__ f) {
    const size_t total = static_cast<size_t>(n_rows) * d_ff;
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const size_t r = i / d_ff, c = i % d_ff;
        if (ffn == SPEC_FFN_GELU) {
            f[i] = gelu_tanh(u[i]);
        } else {
            const float gate = u[r * 2 * d_ff + c], up = u[r * 2 * d_ff + d_ff + c];
            f[i] = (ffn == SPEC_FFN_SWIGLU ? silu(gate) : gelu_tanh(gate)) * up;
        }
    }
}

}  // namespace

int launch_embed(const Model& m, const RowMeta& rows, int n_rows, float* h, cudaStream_t stream) {
    embed_kernel<<<n_rows, 128, 0, stream>>>(m.tok_emb, m.pos_emb, m.bf16(), m.cfg.arch == SPEC_ARCH_GPT, rows.token,
                                             rows.pos, m.cfg.d_model, m.cfg.vocab, m.cfg.max_positions, h);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_rmsnorm(const float* in, const float* gain, const int32_t* src_rows, int n_rows, int d, float eps,
                   float* out, cudaStream_t stream) {
    rmsnorm_kernel<<<n_rows, 256, 0, stream>>>(in, gain, src_rows, d, eps, out);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_rope_append(const Model& m, int layer, const RowMeta& rows, int n_rows, float* qkv,
                       const int32_t* page_table, int pages_per_seq, int page_size, cudaStream_t stream) {
    char* kv_layer = static_cast<char*>(m.kv) + static_cast<size_t>(layer) * m.layer_stride;
    const bool rotary = m.cfg.arch == SPEC_ARCH_LLAMA;
    if (m.kv_elem_bytes == 2)
        rope_append_kernel<__nv_bfloat16><<<n_rows, 128, 0, stream>>>(
            qkv, rows.pos, rows.seq, m.cfg.n_heads, m.cfg.n_kv_heads, m.cfg.d_head, rotary, m.cfg.rope_base,
            reinterpret_cast<__nv_bfloat16*>(kv_layer), page_table, pages_per_seq, page_size);
    else
        rope_append_kernel<float><<<n_rows, 128, 0, stream>>>(
            qkv, rows.pos, rows.seq, m.cfg.n_heads, m.cfg.n_kv_heads, m.cfg.d_head, rotary, m.cfg.rope_base,
            reinterpret_cast<float*>(kv_layer), page_table, pages_per_seq, page_size);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_ffn_act(const float* u, int n_rows, int d_ff, int ffn, float* f, cudaStream_t stream) {
    const size_t total = static_cast<size_t>(n_rows) * d_ff;
    const int blocks = static_cast<int>(std::min<size_t>((total + 255) / 256, 148 * 8));
    ffn_act_kernel<<<blocks, 256, 0, stream>>>(u, n_rows, d_ff, ffn, f);
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

}  // namespace spec
