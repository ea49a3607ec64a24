// The small kernels between the weight-streaming GEMMs of a decoder block.
// Each one also finishes the GEMM before it (adds up the split-K partial sums
// in a fixed order, adds the residual) and prepares the input of the GEMM after
// it (fp32, and/or split into two bf16 terms for the tensor-core path), so that
// a block is nine launches: norm, qkv GEMM, rope + KV append, attention,
// out-projection GEMM, norm, FFN-in GEMM, activation, FFN-out GEMM.
#include <cmath>

#include "attn_unit.cuh"

namespace spec {
namespace {

__device__ __forceinline__ float load_elem(const void* base, size_t i, bool bf16) {
    return bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(base)[i]) : static_cast<const float*>(base)[i];
}

// x = hi + lo with hi = bf16(x), lo = bf16(x - hi): 16 mantissa bits survive.
__device__ __forceinline__ void store_split(__nv_bfloat16* hi, __nv_bfloat16* lo, size_t i, float x) {
    const __nv_bfloat16 h = __float2bfloat16_rn(x);
    hi[i] = h;
    lo[i] = __float2bfloat16_rn(x - __bfloat162float(h));
}

// sum of the split-K partial results of element i, in split order
__device__ __forceinline__ float sum_partials(const float* __restrict__ partial, int splits, size_t stride, size_t i) {
    // eight loads in flight at a time (the adds stay in split order, so the sum is the reduction kernels')
    float acc = 0.0f;
    for (int s0 = 0; s0 < splits; s0 += 8) {
        float p[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) p[k] = s0 + k < splits ? partial[static_cast<size_t>(s0 + k) * stride + i] : 0.0f;
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (s0 + k < splits) acc = (s0 + k == 0) ? p[k] : acc + p[k];
    }
    return acc;
}

// The same for two elements at once (their loads share the flight).
__device__ __forceinline__ void sum_partials2(const float* __restrict__ partial, int splits, size_t stride, size_t i1,
                                              size_t i2, float* out1, float* out2) {
    float a = 0.0f, b = 0.0f;
    for (int s0 = 0; s0 < splits; s0 += 8) {
        float p[8], q[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const bool live = s0 + k < splits;
            p[k] = live ? partial[static_cast<size_t>(s0 + k) * stride + i1] : 0.0f;
            q[k] = live ? partial[static_cast<size_t>(s0 + k) * stride + i2] : 0.0f;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (s0 + k < splits) {
                a = (s0 + k == 0) ? p[k] : a + p[k];
                b = (s0 + k == 0) ? q[k] : b + q[k];
            }
    }
    *out1 = a;
    *out2 = b;
}

// grid = rows, block = 128
__global__ void embed_kernel(const void* __restrict__ tok_emb, const void* __restrict__ pos_emb, bool bf16,
                             bool add_pos, const int32_t* __restrict__ token, const int32_t* __restrict__ pos, int d,
                             int vocab, int max_positions, float* __restrict__ h) {
    pdl_trigger();
    pdl_wait();
    const int r = blockIdx.x;
    const int t = min(max(token[r], 0), vocab - 1);
    const int p = min(max(pos[r], 0), max_positions - 1);
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = load_elem(tok_emb, static_cast<size_t>(t) * d + i, bf16);
        if (add_pos) v += load_elem(pos_emb, static_cast<size_t>(p) * d + i, bf16);
        h[static_cast<size_t>(r) * d + i] = v;
    }
}

// grid = rows, block = kNormThreads; d is a multiple of 4.  Row r of the output is
// RMSNorm(h[src(r)]) * gain.  If `partial` is given, h[r] += sum of the partial
// results first (the residual add of the GEMM that produced them) and the new h
// is stored.  A thread holds up to kNormPerThread float4 of the row in registers,
// so every load of the row and of its partial sums is in flight at once.
constexpr int kNormThreads = 1024;
constexpr int kNormPerThread = 4;  // rows up to 16384 wide

template <int THREADS>
__global__ void __launch_bounds__(THREADS)
norm_kernel(float* h, const float* __restrict__ partial, int splits, int n_rows, const float* __restrict__ gain,
            const int32_t* __restrict__ src_rows, int d, float eps, float* __restrict__ out,
            __nv_bfloat16* __restrict__ out_hi, __nv_bfloat16* __restrict__ out_lo) {
    __shared__ float red[THREADS / 32];
    const int r = blockIdx.x;
    const int groups = d / 4;
    // the gains are constants: fetched while the kernel before this one is still finishing
    float4 gg[kNormPerThread];
#pragma unroll
    for (int j = 0; j < kNormPerThread; ++j) {
        const int g = threadIdx.x + j * THREADS;
        gg[j] = g < groups ? *reinterpret_cast<const float4*>(gain + 4 * g) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    pdl_wait();
    // The GEMM that follows is released only now, when the GEMM before this kernel is complete: released earlier, its CTAs
    // take the places of that GEMM's leaving CTAs and their first weight tiles compete with the tail of its stream
    // (measured per 7B block: 94.5 -> 93.1 us; releasing at the end of this kernel instead: 95.1).
    pdl_trigger();
    const size_t src = static_cast<size_t>(src_rows ? src_rows[r] : r) * d;
    const size_t stride = static_cast<size_t>(n_rows) * d;
    float4 v[kNormPerThread];
    float ss = 0.0f;
#pragma unroll
    for (int j = 0; j < kNormPerThread; ++j) {
        const int g = threadIdx.x + j * THREADS;
        v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (g < groups) {
            v[j] = *reinterpret_cast<const float4*>(h + src + 4 * g);
            if (partial) {
                for (int s0 = 0; s0 < splits; s0 += 8) {  // eight loads in flight at a time, added in split order
                    float4 p[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        p[k] = s0 + k < splits ? *reinterpret_cast<const float4*>(partial + (s0 + k) * stride + src + 4 * g)
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (s0 + k < splits) { v[j].x += p[k].x; v[j].y += p[k].y; v[j].z += p[k].z; v[j].w += p[k].w; }
                }
                *reinterpret_cast<float4*>(h + src + 4 * g) = v[j];
            }
            ss += (v[j].x * v[j].x + v[j].y * v[j].y) + (v[j].z * v[j].z + v[j].w * v[j].w);
        }
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float total = 0.0f;
#pragma unroll
    for (int i = 0; i < THREADS / 32; ++i) total += red[i];
    const float scale = rsqrtf(total / static_cast<float>(d) + eps);
    const size_t dst = static_cast<size_t>(r) * d;
#pragma unroll
    for (int j = 0; j < kNormPerThread; ++j) {
        const int g = threadIdx.x + j * THREADS;
        if (g < groups) {
            const float y[4] = {v[j].x * scale * gg[j].x, v[j].y * scale * gg[j].y, v[j].z * scale * gg[j].z,
                                v[j].w * scale * gg[j].w};
            if (out) *reinterpret_cast<float4*>(out + dst + 4 * g) = make_float4(y[0], y[1], y[2], y[3]);
            if (out_hi) {
#pragma unroll
                for (int e = 0; e < 4; ++e) store_split(out_hi, out_lo, dst + 4 * g + e, y[e]);
            }
        }
    }
}

// grid = (n_heads + 2 n_kv_heads, rows), block = d_head / 2.  qkv row layout:
// [q heads | k heads | v heads], d_head each.  A CTA finishes one head of one row
// of the qkv GEMM (optional partial sums), applies rotary positions (q and k
// heads; thread j owns the pair j, j + d_head/2), leaves q in `qkv` for the
// attention kernel, and appends K or V to the paged cache.
template <typename KV>
__global__ void qkv_kernel(float* __restrict__ qkv, const float* __restrict__ partial, int splits, int n_rows,
                           const int32_t* __restrict__ pos, const int32_t* __restrict__ seq, int n_heads,
                           int n_kv_heads, int d_head, const float2* __restrict__ rope_table,
                           KV* __restrict__ kv_layer, const int32_t* __restrict__ page_table, int pages_per_seq,
                           int page_size) {
    pdl_trigger();
    pdl_wait();
    const int head = blockIdx.x, r = blockIdx.y, j = threadIdx.x;
    const int p = pos[r];
    const int half = d_head / 2;
    const int width = (n_heads + 2 * n_kv_heads) * d_head;
    const size_t at = static_cast<size_t>(r) * width + head * d_head;
    float x1, x2;
    if (partial) {
        const size_t stride = static_cast<size_t>(n_rows) * width;
        sum_partials2(partial, splits, stride, at + j, at + j + half, &x1, &x2);
    } else {
        x1 = qkv[at + j];
        x2 = qkv[at + j + half];
    }
    const bool is_q = head < n_heads, is_k = !is_q && head < n_heads + n_kv_heads;
    if (rope_table && p >= 0 && (is_q || is_k)) {
        const float2 t = rope_table[static_cast<size_t>(p) * half + j];  // (cos, sin) of position p
        const float y1 = x1 * t.x - x2 * t.y, y2 = x2 * t.x + x1 * t.y;
        x1 = y1;
        x2 = y2;
    }
    if (is_q) {
        qkv[at + j] = x1;
        qkv[at + j + half] = x2;
        return;
    }
    if (p < 0) return;  // inactive row: nothing is cached
    const int kv_head = is_k ? head - n_heads : head - n_heads - n_kv_heads;
    const int page = page_table[seq[r] * pages_per_seq + p / page_size];
    const size_t block = (static_cast<size_t>(page) * 2 + (is_k ? 0 : 1)) * n_kv_heads + kv_head;
    KV* dst = kv_layer + (block * page_size + p % page_size) * d_head;
    dst[j] = to_cached<KV>(x1);
    dst[j + half] = to_cached<KV>(x2);
}

// logits[dst(i)] = table[token[src(i)]] for a table model: grid = (chunks, rows), block = 256.
__global__ void table_logits_kernel(const void* __restrict__ table, bool bf16, int vocab, const int32_t* __restrict__ token,
                                    const int32_t* __restrict__ src_rows, const int32_t* __restrict__ dst_rows,
                                    float* __restrict__ logits) {
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.y;
    const int t = min(max(token[src_rows ? src_rows[i] : i], 0), vocab - 1);
    float* out = logits + static_cast<size_t>(dst_rows ? dst_rows[i] : i) * vocab;
    for (int v = blockIdx.x * blockDim.x + threadIdx.x; v < vocab; v += gridDim.x * blockDim.x)
        out[v] = load_elem(table, static_cast<size_t>(t) * vocab + v, bf16);
}

// Copy-from-context draft: logits row i is one-hot (0 at the guess, -inf elsewhere), the
// guess being what followed the most recent earlier occurrence of the last `ngram`
// tokens of the sequence up to the row's position, or the last token again if there is
// none.  Positions below length[seq] read the committed tokens, later ones this
// iteration's guesses.  grid = (chunks, rows): every CTA repeats the search (a few
// thousand token compares) and writes its share of the row.
__global__ void copy_logits_kernel(const int32_t* __restrict__ tokens, int max_len, const int32_t* __restrict__ length,
                                   const int32_t* __restrict__ draft_tokens, int gamma, const int32_t* __restrict__ row_pos,
                                   const int32_t* __restrict__ row_seq, const int32_t* __restrict__ src_rows,
                                   const int32_t* __restrict__ dst_rows, int ngram, int vocab, float* __restrict__ logits) {
    __shared__ int best[32];
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.y;
    const int r = src_rows ? src_rows[i] : i;
    const int b = row_seq[r], last = row_pos[r];
    const int committed = length[b];
    const int32_t* seq = tokens + static_cast<size_t>(b) * max_len;
    const int32_t* guesses = draft_tokens + static_cast<size_t>(b) * gamma;
    auto at = [&](int p) { return p < committed ? seq[p] : guesses[min(p - committed, gamma - 1)]; };
    // j = end of an earlier occurrence of the suffix: ngram-1 <= j <= last-1
    int found = -1;
    for (int j = last - 1 - static_cast<int>(threadIdx.x); j >= ngram - 1; j -= blockDim.x) {
        bool same = true;
        for (int k = 0; k < ngram && same; ++k) same = at(j - k) == at(last - k);
        if (same) { found = j; break; }  // this thread's later candidates are all older
    }
    found = __reduce_max_sync(0xffffffffu, found);
    if ((threadIdx.x & 31) == 0) best[threadIdx.x >> 5] = found;
    __syncthreads();
    for (int w = 0; w < static_cast<int>(blockDim.x) / 32; ++w) found = max(found, best[w]);
    const int guess = min(max(at(found >= 0 ? found + 1 : last), 0), vocab - 1);
    float* out = logits + static_cast<size_t>(dst_rows ? dst_rows[i] : i) * vocab;
    for (int v = blockIdx.x * blockDim.x + threadIdx.x; v < vocab; v += gridDim.x * blockDim.x)
        out[v] = v == guess ? 0.0f : -INFINITY;
}

__device__ __forceinline__ float gelu_tanh(float x) {
    const float k = 0.7978845608028654f;  // sqrt(2 / pi)
    return 0.5f * x * (1.0f + tanhf(k * (x + 0.044715f * x * x * x)));
}

__device__ __forceinline__ float silu(float x) { return x / (1.0f + expf(-x)); }

// f = gelu(u)  |  gelu(gate) * up  |  silu(gate) * up, with u either given in
// full or as the partial sums of the FFN-in GEMM.
__global__ void ffn_act_kernel(const float* __restrict__ u, const float* __restrict__ partial, int splits, int n_rows,
                               int d_ff, int ffn, float* __restrict__ f, __nv_bfloat16* __restrict__ f_hi,
                               __nv_bfloat16* __restrict__ f_lo) {
    pdl_trigger();
    pdl_wait();
    const size_t total = static_cast<size_t>(n_rows) * d_ff;
    const int width = ffn == SPEC_FFN_GELU ? d_ff : 2 * d_ff;
    const size_t stride = static_cast<size_t>(n_rows) * width;
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const size_t r = i / d_ff, c = i % d_ff;
        const size_t a = r * width + c;
        float y;
        if (ffn == SPEC_FFN_GELU) {
            y = gelu_tanh(partial ? sum_partials(partial, splits, stride, a) : u[a]);
        } else {
            float gate, up;
            if (partial) {
                sum_partials2(partial, splits, stride, a, a + d_ff, &gate, &up);
            } else {
                gate = u[a];
                up = u[a + d_ff];
            }
            y = (ffn == SPEC_FFN_SWIGLU ? silu(gate) : gelu_tanh(gate)) * up;
        }
        if (f) f[i] = y;
        if (f_hi) store_split(f_hi, f_lo, i, y);
    }
}

}  // namespace

int launch_embed(const Model& m, const RowMeta& rows, int n_rows, float* h, cudaStream_t stream) {
    return launch_pdl(embed_kernel, dim3(n_rows), dim3(128), 0, stream, m.tok_emb, m.pos_emb, m.bf16(),
                      m.cfg.arch == SPEC_ARCH_GPT, rows.token, rows.pos, m.cfg.d_model, m.cfg.vocab,
                      m.cfg.max_positions, h);
}

int launch_table_logits(const void* table, bool bf16, int vocab, const int32_t* token, const int32_t* src_rows,
                        const int32_t* dst_rows, int n_rows, float* logits, cudaStream_t stream) {
    const int chunks = std::max(1, std::min((vocab + 255) / 256, 32));
    return launch_pdl(table_logits_kernel, dim3(chunks, n_rows), dim3(256), 0, stream, table, bf16, vocab, token, src_rows,
                      dst_rows, logits);
}

int launch_copy_logits(const int32_t* tokens, int max_len, const int32_t* length, const int32_t* draft_tokens, int gamma,
                       const RowMeta& rows, const int32_t* src_rows, const int32_t* dst_rows, int n_rows, int ngram,
                       int vocab, float* logits, cudaStream_t stream) {
    const int chunks = std::max(1, std::min((vocab + 255) / 256, 16));
    return launch_pdl(copy_logits_kernel, dim3(chunks, n_rows), dim3(256), 0, stream, tokens, max_len, length, draft_tokens,
                      gamma, rows.pos, rows.seq, src_rows, dst_rows, ngram, vocab, logits);
}

int launch_norm(float* h, const float* partial, int splits, int rows_total, const float* gain, const int32_t* src_rows,
                int n_rows, int d, float eps, float* out, __nv_bfloat16* out_hi, __nv_bfloat16* out_lo,
                cudaStream_t stream) {
    if (d % 4 || d > 4 * kNormThreads * kNormPerThread)
        return fail(SPEC_ERR_BAD_CONFIG, "norm: width %d is not a multiple of 4 or exceeds %d", d, 4 * kNormThreads * kNormPerThread);
    // a thread per 128-bit group of the row where the row is narrow (fewer warps to reduce over)
    const int groups = d / 4;
    if (groups <= 128)
        return launch_pdl(norm_kernel<128>, dim3(n_rows), dim3(128), 0, stream, h, partial, splits, rows_total, gain, src_rows, d,
                          eps, out, out_hi, out_lo);
    if (groups <= 256)
        return launch_pdl(norm_kernel<256>, dim3(n_rows), dim3(256), 0, stream, h, partial, splits, rows_total, gain, src_rows, d,
                          eps, out, out_hi, out_lo);
    return launch_pdl(norm_kernel<kNormThreads>, dim3(n_rows), dim3(kNormThreads), 0, stream, h, partial, splits, rows_total,
                      gain, src_rows, d, eps, out, out_hi, out_lo);
}

int launch_qkv(int n_heads, int n_kv_heads, int d_head, const float2* rope, const KvPool& pool, const RowMeta& rows,
               int n_rows, float* qkv, const float* partial, int splits, cudaStream_t stream) {
    const dim3 grid(n_heads + 2 * n_kv_heads, n_rows);
    const dim3 block(d_head / 2);
    if (pool.dtype == SPEC_DTYPE_FP16)
        return launch_pdl(qkv_kernel<__half>, grid, block, 0, stream, qkv, partial, splits, n_rows, rows.pos, rows.seq, n_heads,
                          n_kv_heads, d_head, rope, static_cast<__half*>(pool.kv), pool.page_table, pool.pages_per_seq,
                          pool.page_size);
    if (pool.dtype == SPEC_DTYPE_BF16)
        return launch_pdl(qkv_kernel<__nv_bfloat16>, grid, block, 0, stream, qkv, partial, splits, n_rows, rows.pos,
                          rows.seq, n_heads, n_kv_heads, d_head, rope, static_cast<__nv_bfloat16*>(pool.kv),
                          pool.page_table, pool.pages_per_seq, pool.page_size);
    return launch_pdl(qkv_kernel<float>, grid, block, 0, stream, qkv, partial, splits, n_rows, rows.pos, rows.seq,
                      n_heads, n_kv_heads, d_head, rope, static_cast<float*>(pool.kv), pool.page_table,
                      pool.pages_per_seq, pool.page_size);
}

int launch_ffn_act(const float* u, const float* partial, int splits, int n_rows, int d_ff, int ffn, float* f,
                   __nv_bfloat16* f_hi, __nv_bfloat16* f_lo, cudaStream_t stream) {
    const size_t total = static_cast<size_t>(n_rows) * d_ff;
    const int blocks = static_cast<int>(std::min<size_t>((total + 255) / 256, 148 * 8));
    return launch_pdl(ffn_act_kernel, dim3(blocks), dim3(256), 0, stream, u, partial, splits, n_rows, d_ff, ffn, f,
                      f_hi, f_lo);
}

// (cos, sin) of position * base^(-2j / d_head), evaluated in double precision on
// the host and rounded once to fp32: [positions][d_head / 2].
void fill_rope_table(std::vector<float2>& table, int positions, int d_head, double base) {
    const int half = d_head / 2;
    table.resize(static_cast<size_t>(positions) * half);
    for (int j = 0; j < half; ++j) {
        const double inv_freq = std::pow(base, -2.0 * j / static_cast<double>(d_head));
        for (int p = 0; p < positions; ++p) {
            const double a = static_cast<double>(p) * inv_freq;
            table[static_cast<size_t>(p) * half + j] = make_float2(static_cast<float>(std::cos(a)), static_cast<float>(std::sin(a)));
        }
    }
}

}  // namespace spec
