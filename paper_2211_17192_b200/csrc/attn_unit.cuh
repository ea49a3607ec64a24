// One (sequence, KV head, key slice) piece of attention with one warp per query: the
// body shared by the stand-alone attention kernel and by the persistent pass kernel.
//
// The caller's warps (index `warp` of `warps`, any subset of a CTA) run one warp per query
// that reads this KV head: the G query heads of the group times the m new rows of the
// sequence.  All warps walk the same 32-key tiles, so the K and V rows come from HBM/L2
// once per CTA and from L1 for the other queries.  Lane l owns d_head/32 consecutive
// elements of the head dimension throughout, so every load of a K or V row is one
// coalesced span (a page stores the rows of one head back to back).  For Q.K^T each
// lane forms its share of the 32 dot products of a tile and a 31-shuffle butterfly
// (reduce-scatter) leaves the score of key l in lane l; the warp keeps an online
// softmax (running max and sum, fp32).  For P.V every key's probability is broadcast
// with a shuffle.  A tile never straddles a page (pages hold a multiple of 32 tokens).
#pragma once

#include <cfloat>
#include <cuda_fp16.h>

#include "model.cuh"

namespace spec {

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
    __device__ static __forceinline__ void convert_n(const uint32_t* w, float* out) {  // N / 2 packed words
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
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

// fp16 -> fp32 with integer operations and one multiplication by a power of two (exact for zeros,
// subnormals and normals; cached rows are finite, see to_cached): plain arithmetic that the compiler
// schedules freely around the loads, unlike an opaque conversion instruction.
__device__ __forceinline__ float2 half2_bits_to_float2(uint32_t w) {
    const float lo = __uint_as_float((w & 0x7fffu) << 13) * 0x1p112f;
    const float hi = __uint_as_float((w >> 3) & 0x0fffe000u) * 0x1p112f;
    return make_float2(__uint_as_float(__float_as_uint(lo) | ((w & 0x8000u) << 16)),
                       __uint_as_float(__float_as_uint(hi) | (w & 0x80000000u)));
}

template <>
struct KvLoad<__half> {
    static constexpr int kVec = 8;
    __device__ static __forceinline__ void load(const __half* p, float* out) {
        const uint4 t = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = half2_bits_to_float2(w[i]);
            out[2 * i] = f.x;
            out[2 * i + 1] = f.y;
        }
    }
    template <int N>
    __device__ static __forceinline__ void convert_n(const uint32_t* w, float* out) {  // N / 2 packed words
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            const float2 f = half2_bits_to_float2(w[i]);
            out[2 * i] = f.x;
            out[2 * i + 1] = f.y;
        }
    }
    template <int N>
    __device__ static __forceinline__ void load_n(const __half* p, float* out) {
        if (N == 4) {
            const uint2 t = *reinterpret_cast<const uint2*>(p);
            const float2 a = half2_bits_to_float2(t.x), b = half2_bits_to_float2(t.y);
            out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
        } else {
            const float2 a = half2_bits_to_float2(*reinterpret_cast<const uint32_t*>(p));
            out[0] = a.x; out[1] = a.y;
        }
    }
};

// A value as it is stored in a cached K,V row (fp16: clamped to the finite range first).
template <typename KV>
__device__ __forceinline__ KV to_cached(float x) { return static_cast<KV>(x); }
template <>
__device__ __forceinline__ __half to_cached<__half>(float x) { return __float2half_rn(fminf(fmaxf(x, -65504.0f), 65504.0f)); }

// Synchronisation of the warps that take part: the whole CTA, or a named barrier.
struct CtaSync {
    __device__ static __forceinline__ void sync() { __syncthreads(); }
};
template <int ID, int THREADS>
struct NamedSync {
    __device__ static __forceinline__ void sync() { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(THREADS) : "memory"); }
};

// Work unit u = (query q, sub-slice sub): with ks > 1 the ks warps q, q + queries, ...
// share query q and take every ks-th tile of the slice (the caller then has at least
// queries * ks warps, so every unit has a warp of its own).  The unnormalised state
// (max, sum, accumulator[DH]) of query (row r, head) for this slice goes to `part`
// [(r * n_heads + head) * slices + slice][DH + 2], or, with `park`, to share[q] for a
// merge by the caller.  `share` holds one state per warp.  known_keys >= 0: the number of
// keys of sequence b (otherwise it is read from kv_len or from the rows' positions).
template <typename KV, int DH, typename Sync>
__device__ __forceinline__ void attend_slice(const float* __restrict__ qkv, int q_stride, const int32_t* __restrict__ pos,
                                             const int32_t* __restrict__ seq, int m_rows, int n_heads, int n_kv_heads, int ks,
                                             const KV* __restrict__ kv_layer, const int32_t* __restrict__ page_table,
                                             int pages_per_seq, int page_size, const int32_t* __restrict__ kv_len,
                                             const float* __restrict__ bias, int bias_span, int bias_zero, float scale,
                                             float* __restrict__ part, int slice, int slices, int kv_head, int b, int warp,
                                             int warps, int lane, float (*share)[DH + 2], bool park, int known_keys = -1) {
    constexpr int PER_LANE = DH / 32;
    const int group = n_heads / n_kv_heads;
    const int queries = group * m_rows;

    // the key range of this slice: whole tiles, same for every query of the sequence
    int seq_keys = 0;
    if (known_keys >= 0) {  // (the caller has the sequence's key count at hand)
        seq_keys = known_keys;
    } else if (kv_len) {
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
            // With short heads there are registers to spare: the first batch of V rows is requested
            // together with K, so that the tile waits for memory once instead of twice.
            constexpr bool kEarlyV = PER_LANE <= 2;
            const KV* vt = tile + v_offset + lane * PER_LANE;
            float v_first[kEarlyV ? kVBatch : 1][PER_LANE];
            if (kEarlyV) {
#pragma unroll
                for (int jj = 0; jj < kVBatch; ++jj) {
                    if (jj < in_tile) {
                        KvLoad<KV>::template load_n<PER_LANE>(vt + static_cast<size_t>(jj) * DH, v_first[kEarlyV ? jj : 0]);
                    } else {
#pragma unroll
                        for (int i = 0; i < PER_LANE; ++i) v_first[kEarlyV ? jj : 0][i] = 0.0f;
                    }
                }
            }
            // partial dot products of all 32 keys over this lane's elements ...
            float pd[32];
            const KV* kt = tile + lane * PER_LANE;
            if constexpr (sizeof(KV) == 2) {
                // 16-bit rows: every key's raw words are requested before the first one is converted (the
                // conversion arithmetic between a load and the next would otherwise keep few loads in flight)
                uint32_t raw[32][PER_LANE / 2];
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                    const uint32_t* src = reinterpret_cast<const uint32_t*>(kt + static_cast<size_t>(k < in_tile ? k : 0) * DH);
                    if (PER_LANE == 4) {
                        const uint2 t = *reinterpret_cast<const uint2*>(src);
                        raw[k][0] = t.x;
                        raw[k][PER_LANE / 2 - 1] = t.y;
                    } else {
                        raw[k][0] = *src;
                    }
                }
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                    float kv[PER_LANE];
                    KvLoad<KV>::template convert_n<PER_LANE>(raw[k], kv);
                    float d = 0.0f;
#pragma unroll
                    for (int i = 0; i < PER_LANE; ++i) d = fmaf(qv[i], kv[i], d);
                    pd[k] = k < in_tile ? d : 0.0f;
                }
            } else {
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
#pragma unroll
            for (int j0 = 0; j0 < 32; j0 += kVBatch) {
                if (j0 < in_tile) {
                    float vv[kVBatch][PER_LANE];
#pragma unroll
                    for (int jj = 0; jj < kVBatch; ++jj) {
                        if (kEarlyV && j0 == 0) {
#pragma unroll
                            for (int i = 0; i < PER_LANE; ++i) vv[jj][i] = v_first[kEarlyV ? jj : 0][i];
                        } else if constexpr (sizeof(KV) != 2) {
                            if (j0 + jj < in_tile) {
                                KvLoad<KV>::template load_n<PER_LANE>(vt + static_cast<size_t>(j0 + jj) * DH, vv[jj]);
                            } else {
#pragma unroll
                                for (int i = 0; i < PER_LANE; ++i) vv[jj][i] = 0.0f;
                            }
                        }
                    }
                    if constexpr (sizeof(KV) == 2) {  // raw words of the whole batch first, then the conversions
                        if (!(kEarlyV && j0 == 0)) {
                            uint32_t raw[kVBatch][PER_LANE / 2];
#pragma unroll
                            for (int jj = 0; jj < kVBatch; ++jj) {
                                const uint32_t* src = reinterpret_cast<const uint32_t*>(vt + static_cast<size_t>(j0 + jj < in_tile ? j0 + jj : 0) * DH);
                                if (PER_LANE == 4) {
                                    const uint2 t = *reinterpret_cast<const uint2*>(src);
                                    raw[jj][0] = t.x;
                                    raw[jj][PER_LANE / 2 - 1] = t.y;
                                } else {
                                    raw[jj][0] = *src;
                                }
                            }
#pragma unroll
                            for (int jj = 0; jj < kVBatch; ++jj) {
                                KvLoad<KV>::template convert_n<PER_LANE>(raw[jj], vv[jj]);
                                if (j0 + jj >= in_tile) {
#pragma unroll
                                    for (int i = 0; i < PER_LANE; ++i) vv[jj][i] = 0.0f;
                                }
                            }
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
        if (ks > 1 || park) {  // park the state (ks > 1: warp `q` merges the ks of them below)
            if (lane == 0) {
                share[warp][0] = mx;
                share[warp][1] = l;
            }
#pragma unroll
            for (int i = 0; i < PER_LANE; ++i) share[warp][2 + lane * PER_LANE + i] = acc[i];
        } else {
            // partial state of (row r, head, slice): [max, sum, acc[DH]]
            float* dst = part + ((static_cast<size_t>(r) * n_heads + head) * slices + slice) * (DH + 2);
            if (lane == 0) {
                dst[0] = mx;
                dst[1] = l;
            }
#pragma unroll
            for (int i = 0; i < PER_LANE; ++i) dst[2 + lane * PER_LANE + i] = acc[i];
        }
    }
    if (ks > 1) {
        Sync::sync();
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
            // (warp q is the only reader of the rows it merged, so it may reuse row q)
            float* dst = park ? share[q] : part + ((static_cast<size_t>(r) * n_heads + head) * slices + slice) * (DH + 2);
            __syncwarp();
            if (lane == 0) {
                dst[0] = mm;
                dst[1] = l;
            }
#pragma unroll
            for (int i = 0; i < PER_LANE; ++i) dst[2 + lane * PER_LANE + i] = acc[i];
        }
    }
}

}  // namespace spec
