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
#include <climits>
#include <type_traits>

#include "attn_unit.cuh"

namespace spec {
namespace {

// ---- merging the key slices inside a thread-block cluster ---------------------
// The CTAs of one (sequence, KV head) - one per key slice - are launched as a
// cluster.  Each leaves the states of its queries, [query][max, sum, O[DH]], in
// its own shared memory; after a cluster barrier the CTAs share out the queries,
// read the slices' states through distributed shared memory, merge them in
// slice order and write the attention output.  No partial state goes through
// global memory and no second kernel is needed.
struct AttnOut {
    float* att;             // fp32 [rows][n_heads * DH] or nullptr
    __nv_bfloat16 *hi, *lo;  // the same as two bf16 terms, or nullptr
};

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ float ld_peer_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote));
    return v;
}

constexpr int kMaxClusterSlices = 8;  // portable cluster size; larger clusters of these fat CTAs schedule too slowly

// `fin`: this CTA's states of queries q_base .. q_base + n_q - 1 of the (sequence b,
// KV head) group; query q is row b * m_rows + q / group, head kv_head * group + q % group.
template <int DH>
__device__ __forceinline__ void cluster_merge_write(const float* fin, int n_q, int q_base, int queries, int b, int m_rows,
                                                    int group, int kv_head, int n_heads, int slices, const AttnOut& out) {
    cluster_arrive();
    cluster_wait();  // every slice's states are in place
    const uint32_t base = static_cast<uint32_t>(__cvta_generic_to_shared(fin));
    const int rank = blockIdx.x;  // the cluster spans the slice dimension of the grid
    for (int qi = rank; qi < n_q && q_base + qi < queries; qi += slices) {
        const int q = q_base + qi;
        const size_t at = (static_cast<size_t>(b * m_rows + q / group) * n_heads + kv_head * group + q % group) * DH;
        const uint32_t state = base + static_cast<uint32_t>(qi * (DH + 2) * 4);
        for (int e = threadIdx.x; e < DH; e += blockDim.x) {
            float ms[kMaxClusterSlices], ls[kMaxClusterSlices], os[kMaxClusterSlices];
#pragma unroll
            for (int s = 0; s < kMaxClusterSlices; ++s) {
                ms[s] = s < slices ? ld_peer_f32(state, s) : -FLT_MAX;
                ls[s] = s < slices ? ld_peer_f32(state + 4, s) : 0.0f;
                os[s] = s < slices ? ld_peer_f32(state + 8 + 4 * e, s) : 0.0f;
            }
            float mm = -FLT_MAX;
#pragma unroll
            for (int s = 0; s < kMaxClusterSlices; ++s) mm = fmaxf(mm, ms[s]);
            float l = 0.0f, o = 0.0f;
#pragma unroll
            for (int s = 0; s < kMaxClusterSlices; ++s) {  // slices in index order
                if (s < slices) {                              // (uniform: absent slices cost no exponential)
                    const float w = expf(ms[s] - mm);
                    l += ls[s] * w;
                    o += os[s] * w;
                }
            }
            const float y = l > 0.0f ? o / l : 0.0f;  // an inactive row has no keys
            if (out.att) out.att[at + e] = y;
            if (out.hi) {
                const __nv_bfloat16 h = __float2bfloat16_rn(y);
                out.hi[at + e] = h;
                out.lo[at + e] = __float2bfloat16_rn(y - __bfloat162float(h));
            }
        }
    }
    cluster_arrive();
    cluster_wait();  // nobody leaves while a peer may still read its shared memory
}

// grid = (slices, n_kv_heads, batch), block = 32 * warps (warps <= kMaxAttnWarps).
// Rows of sequence b are rows b*m .. b*m+m-1 of the pass.
// FUSED (needs queries * ks <= kMaxAttnWarps, i.e. one round of work units): the
// grid is launched as clusters over the slice dimension and writes `out` itself.
template <typename KV, int DH, bool FUSED>
__global__ void __launch_bounds__(32 * kMaxAttnWarps)
attention_kernel(const float* __restrict__ qkv, int q_stride, const int32_t* __restrict__ pos,
                 const int32_t* __restrict__ seq, int m_rows, int n_heads, int n_kv_heads, int ks,
                 const KV* __restrict__ kv_layer, const int32_t* __restrict__ page_table, int pages_per_seq,
                 int page_size, const int32_t* __restrict__ kv_len, const float* __restrict__ bias, int bias_span,
                 int bias_zero, float scale, float* __restrict__ part, const AttnOut out) {
    __shared__ float share[kMaxAttnWarps][DH + 2];  // states of the warps that share a query (ks > 1)
    pdl_trigger();
    pdl_wait();
    attend_slice<KV, DH, CtaSync>(qkv, q_stride, pos, seq, m_rows, n_heads, n_kv_heads, ks, kv_layer, page_table, pages_per_seq,
                                  page_size, kv_len, bias, bias_span, bias_zero, scale, part, blockIdx.x, gridDim.x, blockIdx.y,
                                  blockIdx.z, threadIdx.x >> 5, blockDim.x >> 5, threadIdx.x & 31, share, FUSED);
    const int slices = gridDim.x, kv_head = blockIdx.y, b = blockIdx.z;
    const int group = n_heads / n_kv_heads;
    const int queries = group * m_rows;
    if (FUSED) {
        __syncthreads();
        cluster_merge_write<DH>(&share[0][0], queries, 0, queries, b, m_rows, group, kv_head, n_heads, slices, out);
    }
}

// ---- the same attention on the tensor cores, for many queries per KV head ----
//
// With grouped query heads, several new rows per sequence and a batch of
// sequences, the kernel above re-reads every K,V tile from L1 once per query.
// Here the (up to 16) queries that share a KV head form the M side of
// mma.sync.m16n8k8 (tf32, fp32 accumulate): a warp stages a 16-key tile of K and
// of V in shared memory once (cp.async for fp32 rows; 16-bit rows are converted
// on the way in), computes S = Q K^T for all queries, keeps the online softmax in
// the accumulator layout (a row's maximum and sum live in a quad of lanes), and
// accumulates O += P V.  The warps of a CTA take the 16-key tiles of its key slice
// in turn (a slice is short enough that a warp seldom sees a second tile, so one
// staged tile per warp is kept: a second stage halves the CTAs per SM) and merge
// their states at the end; the partial state per (row, head, slice) has the same
// format as above, so attention_combine_kernel serves both.
constexpr int kMmaWarps = 8;
constexpr int kMmaStages = 1;  // staged tiles per warp (2: the next tile loads while this one is multiplied)

__device__ __forceinline__ uint32_t to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}

__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(dst));
    const int bytes = valid ? 16 : 0;  // 0: the 16 bytes are zero-filled
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

constexpr int kTileKeys = 16;  // keys per staged tile of the tensor-core kernel

// A 16-key tile of one KV head ([key][DH] in the pool) into shared memory rows of
// DH + 4 floats; keys at or beyond n_valid become zeros.
template <int DH>
__device__ __forceinline__ void stage_tile(const float* tile, int n_valid, float* dst, int lane) {
    constexpr int kChunks = DH / 4;
    for (int i = lane; i < kTileKeys * kChunks; i += 32) {
        const int row = i / kChunks, c = i % kChunks;
        const bool valid = row < n_valid;
        cp_async16(dst + row * (DH + 4) + 4 * c, tile + static_cast<size_t>(valid ? row : 0) * DH + 4 * c, valid);
    }
}
// (16-bit rows: converted on the way into shared memory; a lane requests all its 16-byte chunks of
// the tile before it converts the first, so that they are in flight together)
template <int DH, typename KV16>
__device__ __forceinline__ void stage_tile(const KV16* tile, int n_valid, float* dst, int lane) {
    constexpr int kChunks = DH / 8;
    constexpr int kPerLane = kTileKeys * kChunks / 32;
    uint4 raw[kPerLane];
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) {
        const int i = lane + 32 * j, row = i / kChunks, c = i % kChunks;
        raw[j] = *reinterpret_cast<const uint4*>(tile + static_cast<size_t>(row < n_valid ? row : 0) * DH + 8 * c);
    }
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) {
        const int i = lane + 32 * j, row = i / kChunks, c = i % kChunks;
        float v[8];
        const uint32_t w[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
        KvLoad<KV16>::template convert_n<8>(w, v);
        if (row >= n_valid) {
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = 0.0f;
        }
        float* d = dst + row * (DH + 4) + 8 * c;
        *reinterpret_cast<float4*>(d) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4*>(d + 4) = make_float4(v[4], v[5], v[6], v[7]);
    }
}

// IN_TURN: K and V of a tile share one buffer - V is loaded once the scores are done with K.
// Half the shared memory per warp, so two CTAs share an SM (d_head 128), at the price of
// a second exposed load per tile: it pays when the launch has CTAs for more than one wave.
template <int DH, bool IN_TURN>
struct MmaSmem {
    static constexpr int kRow = DH + 4;              // floats per staged row (bank-conflict-free fragments)
    static constexpr int kQ = 16 * kRow;             // the queries, scaled and rounded to tf32
    static constexpr int kTile = kTileKeys * kRow;   // one staged K or V tile
    static constexpr int kStage = (IN_TURN ? 1 : 2) * kTile;  // K and V of one tile
    static constexpr int kPStride = 20;              // floats per row of the probabilities (bank-conflict-free)
    static constexpr int kP = 16 * kPStride;         // probabilities of one tile
    static constexpr int kPerWarp = kMmaStages * kStage + kP;
    static constexpr size_t kBytes = static_cast<size_t>(kQ + kMmaWarps * kPerWarp) * sizeof(float);
};

// grid = (slices, n_kv_heads * m_blocks, batch), block = 32 * kMmaWarps.
template <typename KV, int DH, bool FUSED, bool IN_TURN>
__global__ void __launch_bounds__(32 * kMmaWarps)
attention_mma_kernel(const float* __restrict__ qkv, int q_stride, const int32_t* __restrict__ pos,
                     const int32_t* __restrict__ seq, int m_rows, int n_heads, int n_kv_heads, int m_blocks,
                     const KV* __restrict__ kv_layer, const int32_t* __restrict__ page_table, int pages_per_seq,
                     int page_size, const int32_t* __restrict__ kv_len, const float* __restrict__ bias, int bias_span,
                     int bias_zero, float scale, float* __restrict__ part, const AttnOut out) {
    using S = MmaSmem<DH, IN_TURN>;
    extern __shared__ __align__(16) float smem_f[];
    __shared__ int q_pos[16], q_row[16], q_head[16];
    __shared__ float merge_w[16][kMmaWarps], merge_m[16];
    pdl_trigger();
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int slice = blockIdx.x, slices = gridDim.x, b = blockIdx.z;
    const int kv_head = blockIdx.y / m_blocks, mb = blockIdx.y % m_blocks;
    const int group = n_heads / n_kv_heads;
    const int queries = group * m_rows;
    float* Qs = smem_f;
    float* stage0 = smem_f + S::kQ + warp * S::kPerWarp;  // stage s: K tile, then V tile
    float* Ps = stage0 + kMmaStages * S::kStage;

    if (tid < 16) {
        const int q = mb * 16 + tid;
        const bool live = q < queries;
        const int j = live ? q / group : 0;
        q_row[tid] = b * m_rows + j;
        q_head[tid] = kv_head * group + (live ? q % group : 0);
        q_pos[tid] = live ? pos[b * m_rows + j] : -1;
    }
    int seq_keys = 0;
    if (kv_len) {
        seq_keys = kv_len[seq[b * m_rows]];
    } else {
        for (int j = 0; j < m_rows; ++j) seq_keys = max(seq_keys, pos[b * m_rows + j] + 1);
    }
    const int tiles = (seq_keys + 31) / 32;
    const int t0 = static_cast<int>(static_cast<long long>(tiles) * slice / slices);
    const int t1 = static_cast<int>(static_cast<long long>(tiles) * (slice + 1) / slices);
    const size_t head_stride = static_cast<size_t>(page_size) * DH;
    const size_t page_stride = 2 * static_cast<size_t>(n_kv_heads) * head_stride;
    const size_t v_offset = static_cast<size_t>(n_kv_heads) * head_stride;
    const int32_t* pages = page_table + seq[b * m_rows] * pages_per_seq;
    __syncthreads();  // (the queries' positions)

    // the two query rows of this lane: g and g + 8
    const int p_lo = q_pos[g], p_hi = q_pos[g + 8];
    const int keys_lo = p_lo < 0 ? 0 : kv_len ? seq_keys : p_lo + 1;
    const int keys_hi = p_hi < 0 ? 0 : kv_len ? seq_keys : p_hi + 1;
    const float* bias_lo = bias ? bias + static_cast<size_t>(q_head[g]) * bias_span + (bias_zero - p_lo) : nullptr;
    const float* bias_hi = bias ? bias + static_cast<size_t>(q_head[g + 8]) * bias_span + (bias_zero - p_hi) : nullptr;
    float m_lo = -FLT_MAX, m_hi = -FLT_MAX, l_lo = 0.0f, l_hi = 0.0f;
    float o[DH / 8][4];
#pragma unroll
    for (int n = 0; n < DH / 8; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) o[n][i] = 0.0f;

    // This warp's tiles: the slice's 16-key tiles warp, warp + kMmaWarps, ... (a short slice
    // then still gives every warp a tile, and the chain a warp runs through stays short)
    const int tile0 = 2 * t0, tile1 = min(2 * t1, (seq_keys + kTileKeys - 1) / kTileKeys);
    const int my_tiles = tile0 + warp < tile1 ? (tile1 - tile0 - warp + kMmaWarps - 1) / kMmaWarps : 0;
    auto first_key = [&](int i) { return kTileKeys * (tile0 + warp + i * kMmaWarps); };
    auto issue = [&](int i) {  // tile i into stage i & 1 (an empty group if there is no such tile)
        if (i < my_tiles) {
            const int k0 = first_key(i);
            const int n_valid = min(kTileKeys, seq_keys - k0);
            if (n_valid > 0) {
                const KV* tile = kv_layer + pages[k0 / page_size] * page_stride + kv_head * head_stride +
                                 static_cast<size_t>(k0 % page_size) * DH;
                float* st = stage0 + (i % kMmaStages) * S::kStage;
                stage_tile<DH>(tile, n_valid, st, lane);
                if (!IN_TURN) stage_tile<DH>(tile + v_offset, n_valid, st + S::kTile, lane);
            }
        }
        cp_async_commit();
    };
    // the first tiles are requested before the queries are staged
#pragma unroll
    for (int i = 0; i < kMmaStages; ++i) issue(i);
    for (int i = tid; i < 16 * DH; i += 32 * kMmaWarps) {
        const int qi = i / DH, e = i % DH;
        const float v = q_pos[qi] >= 0 ? qkv[static_cast<size_t>(q_row[qi]) * q_stride + q_head[qi] * DH + e] * scale : 0.0f;
        Qs[qi * S::kRow + e] = __uint_as_float(to_tf32(v));
    }
    __syncthreads();
    for (int i = 0; i < my_tiles; ++i) {
        const int k0 = first_key(i);
        cp_async_wait<kMmaStages - 1>();  // tile i has landed (later tiles may still be in flight)
        __syncwarp();
        if (k0 < seq_keys) {
            const float* Kt = stage0 + (i % kMmaStages) * S::kStage;
            const float* Vt = IN_TURN ? Kt : Kt + S::kTile;
            // S = Q K^T: two blocks of 8 keys; even and odd k-steps go to separate accumulators
            // (four independent MMA chains instead of two), added at the end
            float s[2][4], s_odd[2][4];
#pragma unroll
            for (int nb = 0; nb < 2; ++nb)
#pragma unroll
                for (int j = 0; j < 4; ++j) s[nb][j] = s_odd[nb][j] = 0.0f;
#pragma unroll 4
            for (int ks = 0; ks < DH / 8; ks += 2) {
                uint32_t a[2][4];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    a[h][0] = __float_as_uint(Qs[g * S::kRow + (ks + h) * 8 + t]);
                    a[h][1] = __float_as_uint(Qs[(g + 8) * S::kRow + (ks + h) * 8 + t]);
                    a[h][2] = __float_as_uint(Qs[g * S::kRow + (ks + h) * 8 + t + 4]);
                    a[h][3] = __float_as_uint(Qs[(g + 8) * S::kRow + (ks + h) * 8 + t + 4]);
                }
#pragma unroll
                for (int nb = 0; nb < 2; ++nb) {
                    const float* kr = Kt + (nb * 8 + g) * S::kRow + ks * 8 + t;
                    mma_tf32(s[nb], a[0], __float_as_uint(kr[0]), __float_as_uint(kr[4]));
                    mma_tf32(s_odd[nb], a[1], __float_as_uint(kr[8]), __float_as_uint(kr[12]));
                }
            }
#pragma unroll
            for (int nb = 0; nb < 2; ++nb)
#pragma unroll
                for (int j = 0; j < 4; ++j) s[nb][j] += s_odd[nb][j];
            // mask, bias, online softmax (rows g and g + 8; a row's 16 scores sit in its quad of lanes)
            float tmax_lo = -FLT_MAX, tmax_hi = -FLT_MAX;
#pragma unroll
            for (int nb = 0; nb < 2; ++nb)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int key = k0 + nb * 8 + 2 * t + (j & 1);
                    const bool hi_row = j >= 2;
                    const bool valid = key < (hi_row ? keys_hi : keys_lo);
                    float v = s[nb][j];
                    if (valid && bias) v += hi_row ? bias_hi[key] : bias_lo[key];
                    s[nb][j] = valid ? v : -FLT_MAX;
                    if (hi_row) tmax_hi = fmaxf(tmax_hi, s[nb][j]);
                    else tmax_lo = fmaxf(tmax_lo, s[nb][j]);
                }
            tmax_lo = fmaxf(tmax_lo, __shfl_xor_sync(kFullMask, tmax_lo, 1));
            tmax_lo = fmaxf(tmax_lo, __shfl_xor_sync(kFullMask, tmax_lo, 2));
            tmax_hi = fmaxf(tmax_hi, __shfl_xor_sync(kFullMask, tmax_hi, 1));
            tmax_hi = fmaxf(tmax_hi, __shfl_xor_sync(kFullMask, tmax_hi, 2));
            const float new_lo = fmaxf(m_lo, tmax_lo), new_hi = fmaxf(m_hi, tmax_hi);
            const float r_lo = expf(m_lo - new_lo), r_hi = expf(m_hi - new_hi);
            float sum_lo = 0.0f, sum_hi = 0.0f;
#pragma unroll
            for (int nb = 0; nb < 2; ++nb)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool hi_row = j >= 2;
                    const float pv = s[nb][j] > -FLT_MAX ? expf(s[nb][j] - (hi_row ? new_hi : new_lo)) : 0.0f;
                    if (hi_row) sum_hi += pv;
                    else sum_lo += pv;
                    Ps[(hi_row ? g + 8 : g) * S::kPStride + nb * 8 + 2 * t + (j & 1)] = __uint_as_float(to_tf32(pv));
                }
            sum_lo += __shfl_xor_sync(kFullMask, sum_lo, 1);
            sum_lo += __shfl_xor_sync(kFullMask, sum_lo, 2);
            sum_hi += __shfl_xor_sync(kFullMask, sum_hi, 1);
            sum_hi += __shfl_xor_sync(kFullMask, sum_hi, 2);
            l_lo = l_lo * r_lo + sum_lo;
            l_hi = l_hi * r_hi + sum_hi;
            m_lo = new_lo;
            m_hi = new_hi;
            __syncwarp();  // every lane's probabilities are in shared memory
            if (IN_TURN) {  // the scores are done with K: V takes its place
                const int n_valid = min(kTileKeys, seq_keys - k0);
                const KV* tile = kv_layer + pages[k0 / page_size] * page_stride + kv_head * head_stride +
                                 static_cast<size_t>(k0 % page_size) * DH;
                stage_tile<DH>(tile + v_offset, n_valid, stage0 + (i % kMmaStages) * S::kStage, lane);
                cp_async_commit();
                cp_async_wait<0>();
                __syncwarp();
            }

            // O = O * rescale + P V
            uint32_t pa[2][4];
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                pa[ks][0] = __float_as_uint(Ps[g * S::kPStride + ks * 8 + t]);
                pa[ks][1] = __float_as_uint(Ps[(g + 8) * S::kPStride + ks * 8 + t]);
                pa[ks][2] = __float_as_uint(Ps[g * S::kPStride + ks * 8 + t + 4]);
                pa[ks][3] = __float_as_uint(Ps[(g + 8) * S::kPStride + ks * 8 + t + 4]);
            }
#pragma unroll
            for (int n = 0; n < DH / 8; ++n) {
                o[n][0] *= r_lo; o[n][1] *= r_lo; o[n][2] *= r_hi; o[n][3] *= r_hi;
#pragma unroll
                for (int ks = 0; ks < 2; ++ks) {
                    const float* vr = Vt + (ks * 8 + t) * S::kRow + n * 8 + g;
                    mma_tf32(o[n], pa[ks], __float_as_uint(vr[0]), __float_as_uint(vr[4 * S::kRow]));
                }
            }
        }
        __syncwarp();  // this stage (and the probabilities) are free again
        issue(i + kMmaStages);
    }
    cp_async_wait<0>();

    // park this warp's state in its own tile buffer: [query][max, sum, O[DH]]
    __syncthreads();
    float* st = stage0;  // 16 * (DH + 2) floats fit a stage
#pragma unroll
    for (int n = 0; n < DH / 8; ++n) {
        st[g * (DH + 2) + 2 + n * 8 + 2 * t] = o[n][0];
        st[g * (DH + 2) + 2 + n * 8 + 2 * t + 1] = o[n][1];
        st[(g + 8) * (DH + 2) + 2 + n * 8 + 2 * t] = o[n][2];
        st[(g + 8) * (DH + 2) + 2 + n * 8 + 2 * t + 1] = o[n][3];
    }
    if (t == 0) {
        st[g * (DH + 2)] = m_lo;
        st[g * (DH + 2) + 1] = l_lo;
        st[(g + 8) * (DH + 2)] = m_hi;
        st[(g + 8) * (DH + 2) + 1] = l_hi;
    }
    __syncthreads();
    // The weight exp(m_w - max) of every (query, warp) is formed once - thread 8 q + w takes warp w's state of
    // query q, the maximum goes round its group of eight lanes - instead of once per element of the state.
    if (tid < 16 * kMmaWarps) {
        static_assert(kMmaWarps == 8, "the groups of eight lanes below are the warps of one query");
        const int qi = tid / kMmaWarps, w = tid % kMmaWarps;
        const float m_w = smem_f[S::kQ + w * S::kPerWarp + qi * (DH + 2)];
        float mm = m_w;
        mm = fmaxf(mm, __shfl_xor_sync(kFullMask, mm, 1));
        mm = fmaxf(mm, __shfl_xor_sync(kFullMask, mm, 2));
        mm = fmaxf(mm, __shfl_xor_sync(kFullMask, mm, 4));
        merge_w[qi][w] = expf(m_w - mm);
        if (w == 0) merge_m[qi] = mm;
    }
    __syncthreads();
    // merge the warps (in warp order) and write the slice's partial state of every live query
    // (fused: into the queries' buffer, which nobody needs any more, for the cluster merge)
    for (int i = tid; i < 16 * (DH + 2); i += 32 * kMmaWarps) {
        const int qi = i / (DH + 2), e = i % (DH + 2);
        if (mb * 16 + qi >= queries) continue;
        float merged;
        if (e == 0) {
            merged = merge_m[qi];
        } else {
            merged = 0.0f;
#pragma unroll
            for (int w = 0; w < kMmaWarps; ++w) merged += smem_f[S::kQ + w * S::kPerWarp + qi * (DH + 2) + e] * merge_w[qi][w];
        }
        if (FUSED) Qs[i] = merged;
        else part[((static_cast<size_t>(q_row[qi]) * n_heads + q_head[qi]) * slices + slice) * (DH + 2) + e] = merged;
    }
    if (FUSED) {
        __syncthreads();
        cluster_merge_write<DH>(Qs, 16, mb * 16, queries, b, m_rows, group, kv_head, n_heads, slices, out);
    }
}

// ---- fp16 K,V rows on the f16 tensor-core path --------------------------------
//
// With 16-bit rows the cache needs no conversion: 64-key tiles of K and of V go
// from the pool to shared memory as they are (tiled TMA copies that one thread asks
// for, completion counted on an mbarrier per stage; a ring of two or three stages: the
// next tiles load while tile i is multiplied) and feed mma.sync.m16n8k16 (f16 operands,
// fp32 accumulate) through ldmatrix.  A CTA owns (key slice, KV head, sequence)
// and ALL the queries of that KV head - up to 64, as MB blocks of 16 - so K and
// V of the slice are fetched once, whatever the number of rows.  Its four warps
// are (query block, part of the tile's keys): warp w takes query block w % MB
// and keys [16 MB (w / MB), 16 MB (w / MB + 1)) of every tile; the key parts of a
// query block merge at the end.  Scores, the online softmax and the output
// accumulate in fp32; q (scaled) and the probabilities are rounded to fp16 (11
// significant bits, one more than the tf32 path above keeps).
constexpr int kF16Warps = 4;
constexpr int kF16TileKeys = 64;
constexpr int kF16MaxQueries = 64;  // per CTA (MB = 4)

// A staged K or V tile is DH / 64 column blocks of [64 keys][64 halves], as the copies' 128-byte swizzle leaves them:
// rows of 128 bytes without padding, the 16-byte chunks of a row permuted, chunk c of row r at position
// c ^ (r & 7), so that the eight rows an ldmatrix reads hit eight different bank groups.  Three stages (tiles
// i + 1 and i + 2 on their way while tile i is multiplied) for up to 32 queries, two for 64: two CTAs per SM
// either way, and 128 KB of K,V in flight per SM instead of 64 - the kernel is bound by the latency of the tiles.
template <int DH, int MB>
struct F16Smem {
    static constexpr int kStages = MB <= 2 ? 3 : 2;
    static constexpr int kRow = DH;                      // halves per staged query row (K and V rows: 64 per column block)
    static constexpr int kQ = 16 * MB * kRow;            // the queries (halves)
    static constexpr int kTile = kF16TileKeys * kRow;    // one K or V tile (halves)
    static constexpr int kStage = 2 * kTile;             // K, then V
    static constexpr size_t kBytes = static_cast<size_t>(kQ + kStages * kStage) * sizeof(__half);
    // the epilogue reuses the stages: four warps' states first, the merged states behind them (in place when a
    // query block has a single key part, MB = 4: there is nothing to merge then)
    static_assert((kF16Warps * 16 + (MB == kF16Warps ? 0 : 16 * MB)) * (DH + 2) * sizeof(float) <= kStages * kStage * sizeof(__half),
                  "states and merged states must fit the stages");
};
// Offset (in halves) of element `col` (a multiple of 8) of row `row` in a staged tile or in the staged queries.
template <int DH>
__device__ __forceinline__ int f16_at(int row, int col) { return row * DH + ((((col >> 3) ^ row) & 7) << 3) + (col & ~63); }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const __half* p) {
    const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(p));
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], const __half* p) {
    const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(p));
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&h);
}

__device__ __forceinline__ float exp2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ int g_attn_error;  // set when the bounded wait for a tile of the f16 kernel ran out (0 = none)

// Waits, with a limit, for the phase of the given parity; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = static_cast<uint32_t>(__cvta_generic_to_shared(bar));
    for (uint32_t spin = 0; spin < (1u << 22); ++spin) {
        uint32_t done;
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t"
            "}"
            : "=r"(done)
            : "r"(addr), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}

// grid = (slices, n_kv_heads * q_blocks, batch), block = 128; q_blocks = ceil(queries / 64).  kv_map: the layer's pool
// as a matrix of rows of DH halves (cached_f16_rows_map).
// Scores are kept in base-2 units (q is scaled by log2(e) / sqrt(d_head), the bias by log2(e)), so every
// exponential is one ex2.approx; the running maximum goes back to natural units when the state is stored.
template <int DH, int MB, bool FUSED>
__global__ void __launch_bounds__(32 * kF16Warps)
attention_f16_kernel(const float* __restrict__ qkv, int q_stride, const int32_t* __restrict__ pos,
                     const int32_t* __restrict__ seq, int m_rows, int n_heads, int n_kv_heads, int q_blocks,
                     const __grid_constant__ CUtensorMap kv_map, const int32_t* __restrict__ page_table, int pages_per_seq,
                     int page_size, const int32_t* __restrict__ kv_len, const float* __restrict__ bias, int bias_span,
                     int bias_zero, float scale, float* __restrict__ part, const AttnOut out) {
    using S = F16Smem<DH, MB>;
    constexpr int KP = kF16Warps / MB;        // key parts of a tile
    constexpr int KW = kF16TileKeys / KP;     // keys of a tile that one warp multiplies (16 MB)
    constexpr int NB = KW / 8;                // 8-key blocks of those
    constexpr int CH = DH / 8;                // 16-byte chunks of a row
    constexpr int QN = 16 * MB;               // queries of this CTA
    constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
    extern __shared__ __align__(1024) unsigned char smem_raw[];  // (the swizzled boxes want 1024-byte alignment)
    __shared__ int q_pos[QN], q_row[QN], q_head[QN];
    __shared__ __align__(8) uint64_t landed[S::kStages];  // a stage's tile has arrived (counted in bytes)
    __half* Qs = reinterpret_cast<__half*>(smem_raw);
    __half* stages = Qs + S::kQ;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
#pragma unroll
        for (int st = 0; st < S::kStages; ++st)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(&landed[st]))));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_trigger();
    pdl_wait();
    const int g = lane >> 2, t = lane & 3;
    const int mb = warp % MB, kw0 = (warp / MB) * KW;
    const int slice = blockIdx.x, slices = gridDim.x, b = blockIdx.z;
    const int kv_head = blockIdx.y / q_blocks, qb = blockIdx.y % q_blocks;
    const int group = n_heads / n_kv_heads;
    const int queries = group * m_rows;

    if (tid < QN) {
        const int q = qb * kF16MaxQueries + tid;
        const bool live = q < queries;
        const int j = live ? q / group : 0;
        q_row[tid] = b * m_rows + j;
        q_head[tid] = kv_head * group + (live ? q % group : 0);
        q_pos[tid] = live ? pos[b * m_rows + j] : -1;
    }
    int seq_keys = 0;
    if (kv_len) {
        seq_keys = kv_len[seq[b * m_rows]];
    } else {
        for (int j = 0; j < m_rows; ++j) seq_keys = max(seq_keys, pos[b * m_rows + j] + 1);
    }
    const int tiles = (seq_keys + kF16TileKeys - 1) / kF16TileKeys;
    const int t0 = static_cast<int>(static_cast<long long>(tiles) * slice / slices);
    const int t1 = static_cast<int>(static_cast<long long>(tiles) * (slice + 1) / slices);
    const int my_tiles = t1 - t0;
    const int32_t* pages = page_table + seq[b * m_rows] * pages_per_seq;
    const int page_shift = __ffs(page_size) - 1;  // (pages hold a power of two of tokens)

    // Tile i of the slice into stage i % kStages: thread 0 asks for it as tiled copies of 32 rows x 64 halves (a
    // 32-key half of the tile lies inside one page; the pool is one matrix of rows of DH halves, the rows of page p
    // being ((2 p + [V]) n_kv_heads + head) page_size + token), which arrive with the 16-byte chunks of every
    // 128-byte row permuted - chunk c of row r at c ^ (r & 7) - so that ldmatrix sees no bank conflict.  A stage
    // holds K then V, each as DH / 64 column blocks of [64 keys][64 halves].  Keys at or beyond seq_keys are
    // whatever the pool holds there (zeros or an earlier sequence's rows): they are masked, and finite.
    // (the page entries of a tile are fetched one tile ahead of the copies that need them)
    auto fetch_pages = [&](int i, int (&pg)[2]) {
        if (tid == 0 && i < my_tiles) {
            const int k0 = kF16TileKeys * (t0 + i);
#pragma unroll
            for (int h = 0; h < 2; ++h) pg[h] = pages[min(k0 + 32 * h, seq_keys - 1) >> page_shift];
        }
    };
    auto issue = [&](int i, const int (&pg)[2]) {
        if (tid == 0 && i < my_tiles) {
            const int k0 = kF16TileKeys * (t0 + i);
            const int st = i % S::kStages;
            const uint32_t bar = static_cast<uint32_t>(__cvta_generic_to_shared(&landed[st]));
            const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(stages + st * S::kStage));
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the stage was read with ldmatrix before
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(static_cast<uint32_t>(S::kStage * sizeof(__half)))
                         : "memory");
#pragma unroll
            for (int v = 0; v < 2; ++v)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int row = ((2 * pg[h] + v) * n_kv_heads + kv_head) * page_size + ((k0 + 32 * h) & (page_size - 1));
#pragma unroll
                    for (int c = 0; c < DH / 64; ++c) {
                        const uint32_t d = dst + static_cast<uint32_t>((v * S::kTile + c * kF16TileKeys * 64 + h * 32 * 64) * sizeof(__half));
                        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                                     ::"r"(d), "l"(&kv_map), "r"(c * 64), "r"(row), "r"(bar)
                                     : "memory");
                    }
                }
        }
    };
    int pg_next[2] = {0, 0};
#pragma unroll
    for (int t = 0; t < S::kStages - 1; ++t) {  // the first tiles are requested before the queries are staged
        fetch_pages(t, pg_next);
        issue(t, pg_next);
    }
    fetch_pages(S::kStages - 1, pg_next);
    __syncthreads();  // (the queries' positions)
    const float q_scale = scale * kLog2e;
    for (int i = tid; i < QN * DH; i += 32 * kF16Warps) {
        const int qi = i / DH, e = i % DH;
        const float v = q_pos[qi] >= 0 ? qkv[static_cast<size_t>(q_row[qi]) * q_stride + q_head[qi] * DH + e] * q_scale : 0.0f;
        Qs[f16_at<DH>(qi, e & ~7) + (e & 7)] = __float2half_rn(v);
    }

    // the two query rows of this lane: g and g + 8 of query block mb.  A row beyond the live queries sees
    // every key (its output is never written): it then never forces the masked path on its warp.
    const int p_lo = q_pos[mb * 16 + g], p_hi = q_pos[mb * 16 + g + 8];
    const int keys_lo = p_lo < 0 ? INT_MAX : kv_len ? seq_keys : p_lo + 1;
    const int keys_hi = p_hi < 0 ? INT_MAX : kv_len ? seq_keys : p_hi + 1;
    const float* bias_lo = bias && p_lo >= 0 ? bias + static_cast<size_t>(q_head[mb * 16 + g]) * bias_span + (bias_zero - p_lo) : nullptr;
    const float* bias_hi = bias && p_hi >= 0 ? bias + static_cast<size_t>(q_head[mb * 16 + g + 8]) * bias_span + (bias_zero - p_hi) : nullptr;
    float m_lo = -FLT_MAX, m_hi = -FLT_MAX, l_lo = 0.0f, l_hi = 0.0f;
    float o[DH / 8][4];
#pragma unroll
    for (int n = 0; n < DH / 8; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) o[n][i] = 0.0f;
    uint32_t qf[DH / 16][4];
    // lane-dependent parts of the ldmatrix addresses, formed once (the chunk permutation XORs with lane & 7):
    // K: row (nb*8 + l7), chunk kp*4 + (lane >> 3); V: row (kk*16 + l7 + 8*((lane >> 3) & 1)), chunk n2*2 + (lane >> 4)
    const int l7 = lane & 7;
    const int k_lane = l7 * 64 + ((((lane >> 3) ^ l7) & 7) << 3);            // even kp; odd kp flips chunk bit 2
    const int v_row = (l7 + 8 * ((lane >> 3) & 1)) * 64;
    int v_chunk[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v_chunk[j] = ((((j << 1) | (lane >> 4)) ^ l7) & 7) << 3;
    // keys that every row of this warp sees (no mask needed below it), and that any live row sees
    const int all_see = min(__reduce_min_sync(kFullMask, min(keys_lo, keys_hi)), seq_keys);
    const int any_sees = min(__reduce_max_sync(kFullMask, max(p_lo < 0 ? 0 : keys_lo, p_hi < 0 ? 0 : keys_hi)), seq_keys);

    for (int i = 0; i < my_tiles; ++i) {
        // tile i has landed (a wait that runs out is recorded and the pass goes on with what the stage holds: no
        // thread leaves the loop alone, and the host sees the error)
        if (!mbar_wait_bounded(&landed[i % S::kStages], (i / S::kStages) & 1)) atomicCAS(&g_attn_error, 0, 1);
        __syncthreads();                     // everybody is done with tile i - 1, whose stage
        issue(i + S::kStages - 1, pg_next);  // takes the tile that is kStages - 1 ahead
        fetch_pages(i + S::kStages, pg_next);
        if (i == 0) {  // (the first barrier also covered the staged queries)
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks)
                ldsm_x4(qf[ks], Qs + f16_at<DH>(mb * 16 + (lane & 7) + 8 * ((lane >> 3) & 1), ks * 16 + 8 * (lane >> 4)));
        }
        const int k0 = kF16TileKeys * (t0 + i) + kw0;  // this warp's first key of the tile
        if (k0 >= any_sees) continue;  // nothing here that a live row of this warp may see
        const __half* Kt = stages + (i % S::kStages) * S::kStage + kw0 * 64;  // (kw0 is a multiple of 16: the permutation is unchanged)
        const __half* Vt = Kt + S::kTile;
        // S = Q K^T
        float s[NB][4];
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
            for (int j = 0; j < 4; ++j) s[nb][j] = 0.0f;
#pragma unroll
        for (int kp = 0; kp < DH / 32; ++kp) {
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
                uint32_t kf[4];
                ldsm_x4(kf, Kt + nb * 8 * 64 + (kp >> 1) * (kF16TileKeys * 64) + ((kp & 1) ? (k_lane ^ 32) : k_lane));
                mma_f16(s[nb], qf[2 * kp], kf[0], kf[1]);
                mma_f16(s[nb], qf[2 * kp + 1], kf[2], kf[3]);
            }
        }
        // bias and mask (rows g and g + 8; a row's KW scores sit in its quad of lanes)
        if (bias) {
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int key = k0 + nb * 8 + 2 * t + (j & 1);
                    const float* bp = j >= 2 ? bias_hi : bias_lo;
                    if (bp && key < (j >= 2 ? keys_hi : keys_lo)) s[nb][j] = fmaf(bp[key], kLog2e, s[nb][j]);
                }
        }
        if (k0 + KW > all_see) {  // (warp-uniform) some row of this warp does not see some key of the block
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int key = k0 + nb * 8 + 2 * t + (j & 1);
                    if (key >= (j >= 2 ? keys_hi : keys_lo) || key >= seq_keys) s[nb][j] = -FLT_MAX;
                }
        }
        float tmax_lo = -FLT_MAX, tmax_hi = -FLT_MAX;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
            tmax_lo = fmaxf(tmax_lo, fmaxf(s[nb][0], s[nb][1]));
            tmax_hi = fmaxf(tmax_hi, fmaxf(s[nb][2], s[nb][3]));
        }
        tmax_lo = fmaxf(tmax_lo, __shfl_xor_sync(kFullMask, tmax_lo, 1));
        tmax_lo = fmaxf(tmax_lo, __shfl_xor_sync(kFullMask, tmax_lo, 2));
        tmax_hi = fmaxf(tmax_hi, __shfl_xor_sync(kFullMask, tmax_hi, 1));
        tmax_hi = fmaxf(tmax_hi, __shfl_xor_sync(kFullMask, tmax_hi, 2));
        const float new_lo = fmaxf(m_lo, tmax_lo), new_hi = fmaxf(m_hi, tmax_hi);
        // (a masked score is -FLT_MAX: minus the maximum it stays far below ex2's underflow, unless the whole
        // row is masked so far - then the maximum is -FLT_MAX too and the terms are dropped explicitly)
        const bool none_lo = new_lo == -FLT_MAX, none_hi = new_hi == -FLT_MAX;
        float sum_lo = 0.0f, sum_hi = 0.0f;
        uint32_t pa[NB / 2][4];  // the probabilities as A fragments: 16 keys per k-step
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
            const float p0 = none_lo ? 0.0f : exp2_approx(s[nb][0] - new_lo), p1 = none_lo ? 0.0f : exp2_approx(s[nb][1] - new_lo);
            const float p2 = none_hi ? 0.0f : exp2_approx(s[nb][2] - new_hi), p3 = none_hi ? 0.0f : exp2_approx(s[nb][3] - new_hi);
            sum_lo += p0 + p1;
            sum_hi += p2 + p3;
            pa[nb / 2][(nb & 1) * 2] = pack_half2(p0, p1);
            pa[nb / 2][(nb & 1) * 2 + 1] = pack_half2(p2, p3);
        }
        sum_lo += __shfl_xor_sync(kFullMask, sum_lo, 1);
        sum_lo += __shfl_xor_sync(kFullMask, sum_lo, 2);
        sum_hi += __shfl_xor_sync(kFullMask, sum_hi, 1);
        sum_hi += __shfl_xor_sync(kFullMask, sum_hi, 2);
        // O = O * rescale + P V (the rescale is skipped while no row of the warp has a new maximum)
        if (__any_sync(kFullMask, new_lo != m_lo || new_hi != m_hi)) {
            const float r_lo = exp2_approx(m_lo - new_lo), r_hi = exp2_approx(m_hi - new_hi);
            l_lo *= r_lo;
            l_hi *= r_hi;
#pragma unroll
            for (int n = 0; n < DH / 8; ++n) {
                o[n][0] *= r_lo; o[n][1] *= r_lo; o[n][2] *= r_hi; o[n][3] *= r_hi;
            }
            m_lo = new_lo;
            m_hi = new_hi;
        }
        l_lo += sum_lo;
        l_hi += sum_hi;
#pragma unroll
        for (int n2 = 0; n2 < DH / 16; ++n2) {
#pragma unroll
            for (int kk = 0; kk < NB / 2; ++kk) {
                uint32_t vf[4];
                ldsm_x4_trans(vf, Vt + kk * 16 * 64 + v_row + (n2 >> 2) * (kF16TileKeys * 64) + v_chunk[n2 & 3]);
                mma_f16(o[2 * n2], pa[kk], vf[0], vf[1]);
                mma_f16(o[2 * n2 + 1], pa[kk], vf[2], vf[3]);
            }
        }
    }
    // (every tile that was asked for has been waited for: nothing is in flight)

    // park this warp's state in stage 0: [warp][query of the block][max (base-2 units), sum, O[DH]]
    __syncthreads();
    float* states = reinterpret_cast<float*>(stages);
    // (one key part per query block: every weight below is 1 and the merged state is the state, in place)
    float* merged_buf = KP == 1 ? states : states + kF16Warps * 16 * (DH + 2);
    {
        float* st = states + warp * 16 * (DH + 2);
#pragma unroll
        for (int n = 0; n < DH / 8; ++n) {
            *reinterpret_cast<float2*>(st + g * (DH + 2) + 2 + n * 8 + 2 * t) = make_float2(o[n][0], o[n][1]);
            *reinterpret_cast<float2*>(st + (g + 8) * (DH + 2) + 2 + n * 8 + 2 * t) = make_float2(o[n][2], o[n][3]);
        }
        if (t == 0) {
            st[g * (DH + 2)] = m_lo;
            st[g * (DH + 2) + 1] = l_lo;
            st[(g + 8) * (DH + 2)] = m_hi;
            st[(g + 8) * (DH + 2) + 1] = l_hi;
        }
    }
    __syncthreads();
    // Merge the key parts of every query block (in part order).  One slice in all: the merged state is the
    // whole answer and is normalised and written here.  Otherwise the slice's state of every live query goes
    // to the cluster merge (FUSED) or to global memory for the combine kernel, its maximum in natural units.
    const bool whole = FUSED && slices == 1;
    for (int i = tid; i < QN * (DH + 2); i += 32 * kF16Warps) {
        const int qi = i / (DH + 2), e = i % (DH + 2);
        const int q = qb * kF16MaxQueries + qi;
        if (q >= queries && !(FUSED && !whole)) continue;
        const float* sw0 = states + ((qi / 16) * 16 * (DH + 2)) + (qi % 16) * (DH + 2);  // warp (qi / 16) + MB * part
        float mm = -FLT_MAX;
#pragma unroll
        for (int kp = 0; kp < KP; ++kp) mm = fmaxf(mm, sw0[kp * MB * 16 * (DH + 2)]);
        float merged = 0.0f, l = 0.0f;
#pragma unroll
        for (int kp = 0; kp < KP; ++kp) {
            const float* sw = sw0 + kp * MB * 16 * (DH + 2);
            const float w = exp2_approx(sw[0] - mm);  // (both -FLT_MAX: weight 1 on an empty state)
            merged += sw[e] * w;
            l += sw[1] * w;
        }
        if (e == 0) merged = mm == -FLT_MAX ? -FLT_MAX : mm * kLn2;
        if (whole) {
            if (e < 2) continue;
            const float y = l > 0.0f ? merged / l : 0.0f;  // an inactive row has no keys
            const size_t at = (static_cast<size_t>(q_row[qi]) * n_heads + q_head[qi]) * DH + (e - 2);
            if (out.att) out.att[at] = y;
            if (out.hi) {
                const __nv_bfloat16 h = __float2bfloat16_rn(y);
                out.hi[at] = h;
                out.lo[at] = __float2bfloat16_rn(y - __bfloat162float(h));
            }
        } else if (FUSED) {
            merged_buf[i] = merged;
        } else {
            part[((static_cast<size_t>(q_row[qi]) * n_heads + q_head[qi]) * slices + slice) * (DH + 2) + e] = merged;
        }
    }
    if (FUSED && !whole) {
        __syncthreads();
        cluster_merge_write<DH>(merged_buf, QN, qb * kF16MaxQueries, queries, b, m_rows, group, kv_head, n_heads, slices, out);
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
    // every load of this kernel is requested at once: the accumulators do not depend on the weights
    float acc[32];
#pragma unroll
    for (int s = 0; s < 32; ++s) acc[s] = s < slices ? in[s * (DH + 2) + 2 + threadIdx.x] : 0.0f;
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
#pragma unroll
    for (int s = 0; s < 32; ++s) o += s < slices ? acc[s] * w_sh[s] : 0.0f;  // slices in index order
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

// The tensor-core kernel serves bf16 models (its tf32 products stay far inside
// their 2e-2 logit bar, not inside the 1e-4 bar of fp32 models) once a KV head
// has enough queries to fill a good part of a 16-row block.
constexpr int kF16MinPairs = 16;  // (sequence, KV head) pairs from which fp16 K,V rows take the f16 kernel
constexpr int kF16LoneQueryPairs = 64;  // ... and from which it takes passes of fewer than four queries per KV head

bool attention_uses_mma(const Model& m, int batch, int m_rows, int max_keys) {
    const int queries = (m.cfg.n_heads / m.cfg.n_kv_heads) * m_rows;
    // With fewer than 5 queries per KV head, or little work in all (query-key pairs over the
    // whole launch), the warp-per-query kernel wins: its CTAs are lighter to launch.
    const long long pairs = static_cast<long long>(batch) * m.cfg.n_kv_heads * queries * max_keys;
    // (four queries - a one-row pass of a model with four query heads per KV head - pay where the CTAs share the SMs:
    // with fp16 K,V rows, i.e. the f16 kernel, from 16 (sequence, KV head) pairs on - measured on the 7B shape, one row,
    // per block, against the warp-per-query kernel: 4 sequences 95 vs 104 us, 8 sequences 101 vs 120, at 1788 cached
    // tokens 105 vs 138; with fp32 rows from 128 pairs on: batch 16 4.16 -> 4.05 ms per pass, batch 8 3.46 -> 3.48)
    const int groups = batch * m.cfg.n_kv_heads;
    int min_queries = groups >= (m.kv_dtype == SPEC_DTYPE_FP16 ? kF16MinPairs : 128) ? 4 : 5;
    // from 64 pairs on the f16 kernel also takes a lone query (a draft model's step in a batch): its tiles come through
    // a ring of asynchronous copies, where the warp-per-query kernel's CTAs, by then several tiles per warp, wait on each in turn
    // (160M-shaped draft, one row, per block: 6 sequences 36.7 vs 41.5 us, 16 sequences 42.8 vs 58.5, 32 sequences 54.3 vs
    // 80.2; 4 sequences 34.7 vs 35.3: no difference below)
    if (m.kv_dtype == SPEC_DTYPE_FP16 && groups >= kF16LoneQueryPairs) min_queries = 1;
    return m.bf16() && queries >= min_queries && pairs >= 65536;
}

// fp16 K,V rows take the f16 tensor-core kernel where the tf32 one would run, from 16 (sequence, KV head)
// pairs on: measured on the 7B shape with 1024 cached tokens, per block, against the tf32 kernel converting
// the same rows: batch 2 x 3 rows 97.0 vs 97.8 us, 2 x 7 105 vs 108, 3 x 3 99 vs 117, 3 x 7 113 vs 136,
// 4 x 3 104 vs 110, 8 x 3 113 vs 135, 16 x 5 165 vs 227, 32 x 7 317 vs 452, 32 x 1 141 vs 185; at batch 1
// (8 pairs) its 64-key tiles leave too few CTAs and it loses up to 3 us per block (7 rows: 100 vs 97).
bool attention_uses_f16(const Model& m, int batch, int m_rows, int max_keys) {
    return m.kv_dtype == SPEC_DTYPE_FP16 && batch * m.cfg.n_kv_heads >= kF16MinPairs && attention_uses_mma(m, batch, m_rows, max_keys);
}

// The key slices can be merged inside a cluster (no second kernel) whenever a CTA
// holds all its queries' states at once: always on the tensor-core path, and on
// the warp-per-query path when the queries fit one round of warps.  It is done
// when the slice count that balances the keys is at most 8: long contexts want
// more slices than a cluster schedules well, and keep the separate combine kernel.
bool attention_merges_in_cluster(const Model& m, int batch, int m_rows, int max_keys) {
    return attention_uses_mma(m, batch, m_rows, max_keys) || (m.cfg.n_heads / m.cfg.n_kv_heads) * m_rows <= kMaxAttnWarps;
}

int attention_slices(const Model& m, int batch, int m_rows, int max_len) {
    const int cap = 32;
    const int n_kv_heads = m.cfg.n_kv_heads;
    const int queries = (m.cfg.n_heads / n_kv_heads) * m_rows;
    const int tiles = (max_len + 31) / 32;
    if (attention_uses_f16(m, batch, m_rows, max_len)) {
        // one wave of CTAs (two per SM at d_head 128, four at 64), a 64-key tile per slice at least
        const int groups = batch * n_kv_heads * ((queries + kF16MaxQueries - 1) / kF16MaxQueries);
        const int resident = 148 * (m.cfg.d_head == 64 ? 4 : 2);
        const int want = std::max(1, resident / groups);
        const int most = std::max(1, (max_len + kF16TileKeys - 1) / kF16TileKeys);
        int slices = std::max(1, std::min(std::min(want, most), cap));
        // clusters are placed a cluster at a time: past 128 SMs' worth of CTAs a launch waits for room (7B shape, one
        // row, per block: 12 sequences 3 slices x 96 heads 119 us, 2 x 96 106; 6 sequences 6 x 48 109, 5 x 48 99)
        const int room = 128 * (m.cfg.d_head == 64 ? 4 : 2);
        if (slices <= kMaxClusterSlices && groups * slices > room) slices = std::max(1, room / groups);
        return slices;
    }
    if (attention_uses_mma(m, batch, m_rows, max_len)) {
        // one wave of CTAs (shared memory allows one per SM at d_head 128, two at 64; twice that from 64
        // (sequence, KV head, query block) groups on, where K and V share a buffer - measured: 16 sequences
        // x 3 rows 5.11 -> 4.41 ms per 7B pass, 32 groups unchanged); a 16-key tile per warp at least
        const int m_blocks = (queries + 15) / 16;
        const int groups = batch * n_kv_heads * m_blocks;
        const int resident = 148 * (m.cfg.d_head == 64 ? 2 : 1) * (groups >= 64 ? 2 : 1);
        const int want = std::max(1, resident / groups);
        const int most = std::max(1, (2 * tiles + kMmaWarps - 1) / kMmaWarps);  // (tiles: 32 keys; a warp's unit is 16)
        return std::max(1, std::min(std::min(want, most), cap));
    }
    const int ks = attention_sub_slices(queries);
    // CTAs that fit the GPU at once: the kernel holds 128 registers per thread, so an
    // SM takes 16 warps of it; one wave of CTAs beats more, thinner slices
    const int warps = std::min(kMaxAttnWarps, std::max(1, queries * ks));
    const int resident = 148 * std::max(1, 16 / warps);
    const int groups = batch * n_kv_heads;
    const int want = std::max(1, resident / groups);
    int most = std::max(1, (tiles + ks - 1) / ks);
    // A lone query per KV head (a draft model's serial step): a tile per warp would leave the K,V rows of a
    // head to a few SMs, whose ingest then bounds the kernel; a full cluster of thinner slices spreads them
    // (measured per block of the 160M-shaped draft, 1024 cached tokens: 3 slices 30.3 us, 8 slices 29.4;
    // 1788 tokens: 31.5 -> 31.0; more than a cluster merges, with the combine kernel: 29.6 - 29.8).
    if (queries == 1) most = std::max(1, std::min(kMaxClusterSlices, (tiles + 3) / 4));
    int slices = std::max(1, std::min(std::min(want, most), cap));
    // Clusters of these SM-filling CTAs are placed a cluster at a time, beside the neighbouring kernels that overlap
    // them: beyond 128 CTAs a launch waits for room (draft, 4 sequences: 3 slices x 48 heads 42.4 us per block,
    // 2 x 48 35.6; 2 sequences: 6 x 24 39.7, 5 x 24 32.3).  Launches without clusters do not mind.
    if (warps == kMaxAttnWarps && slices <= kMaxClusterSlices && attention_merges_in_cluster(m, batch, m_rows, max_len) &&
        groups * slices > 128)
        slices = std::max(1, 128 / groups);
    return slices;
}

size_t attention_partial_elems(int rows, int n_heads, int d_head, int slices) {
    return static_cast<size_t>(rows) * n_heads * slices * (d_head + 2);
}

// What launch_attention does for this shape: which kernel, how many key slices, whether the
// slices merge inside a cluster (no combine kernel), whether K and V share one staging buffer.
AttentionPlan attention_plan(const Model& m, int batch, int m_rows, int max_keys) {
    AttentionPlan plan{};
    plan.tensor_cores = attention_uses_f16(m, batch, m_rows, max_keys) ? 2 : attention_uses_mma(m, batch, m_rows, max_keys) ? 1 : 0;
    plan.slices = attention_slices(m, batch, m_rows, max_keys);
    plan.cluster_merge = attention_merges_in_cluster(m, batch, m_rows, max_keys) && plan.slices <= kMaxClusterSlices ? 1 : 0;
    const int queries = (m.cfg.n_heads / m.cfg.n_kv_heads) * m_rows;
    plan.in_turn = plan.tensor_cores == 1 && batch * m.cfg.n_kv_heads * ((queries + 15) / 16) >= 32 ? 1 : 0;
    return plan;
}

int attention_take_error() {
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_attn_error, sizeof(int)) != cudaSuccess) return -1;
    if (v) cudaMemcpyToSymbol(g_attn_error, &zero, sizeof(int));
    return v;
}

namespace {

// A launch with programmatic stream serialization and, if cluster_x > 0, clusters of
// cluster_x CTAs along x.
template <typename... KArgs, typename... Args>
int launch_attn(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, int cluster_x, cudaStream_t stream,
                Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (cluster_x > 0) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = static_cast<unsigned>(cluster_x);
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (pdl_enabled()) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
    if (err != cudaSuccess) return fail(SPEC_ERR_CUDA, "attention launch failed: %s", cudaGetErrorString(err));
    return SPEC_OK;
}

template <typename KV, int DH>
int launch_attention_variant(const Model& m, const AttnSource& src, const RowMeta& rows, int batch, int m_rows, int slices,
                             int max_keys, float* part, const AttnOut& out, cudaStream_t stream) {
    const int group = m.cfg.n_heads / m.cfg.n_kv_heads;
    const int queries = group * m_rows;
    const float scale = 1.0f / sqrtf(static_cast<float>(m.cfg.d_head));
    const int n_rows = batch * m_rows;
    const bool fused = attention_merges_in_cluster(m, batch, m_rows, max_keys) && slices <= kMaxClusterSlices;
    const KV* pool = static_cast<const KV*>(src.pool.kv);
    int status;
    if constexpr (std::is_same<KV, __half>::value) {
        if (attention_uses_f16(m, batch, m_rows, max_keys)) {
            const int q_blocks = (queries + kF16MaxQueries - 1) / kF16MaxQueries;
            const int per_cta = std::min(queries, kF16MaxQueries);
            const dim3 grid(slices, m.cfg.n_kv_heads * q_blocks, batch);
            CUtensorMap kv_map;  // the layer's pool as rows of d_head halves
            status = cached_f16_rows_map(src.pool.kv, static_cast<unsigned long long>(src.pool.n_pages) * 2 * m.cfg.n_kv_heads *
                                                          src.pool.page_size, DH, &kv_map);
            if (status != SPEC_OK) return status;
#define SPEC_LAUNCH_F16(MB, F, CLUSTER)                                                                                 \
    do {                                                                                                                \
        static std::atomic<unsigned long long> configured{0};                                                           \
        if (first_use_on_this_device(configured))                                                                       \
            SPEC_CUDA_TRY(cudaFuncSetAttribute(attention_f16_kernel<DH, MB, F>,                                         \
                                               cudaFuncAttributeMaxDynamicSharedMemorySize,                             \
                                               static_cast<int>(F16Smem<DH, MB>::kBytes)));                             \
        status = launch_attn(attention_f16_kernel<DH, MB, F>, grid, dim3(32 * kF16Warps), F16Smem<DH, MB>::kBytes,      \
                             CLUSTER, stream, src.q, src.q_stride, rows.pos, rows.seq, m_rows, m.cfg.n_heads,           \
                             m.cfg.n_kv_heads, q_blocks, kv_map, src.pool.page_table, src.pool.pages_per_seq,           \
                             src.pool.page_size, src.kv_len, src.bias, src.bias_span, src.bias_zero, scale, part, out); \
    } while (0)
            if (per_cta <= 16) { if (fused) SPEC_LAUNCH_F16(1, true, slices); else SPEC_LAUNCH_F16(1, false, 0); }
            else if (per_cta <= 32) { if (fused) SPEC_LAUNCH_F16(2, true, slices); else SPEC_LAUNCH_F16(2, false, 0); }
            else { if (fused) SPEC_LAUNCH_F16(4, true, slices); else SPEC_LAUNCH_F16(4, false, 0); }
#undef SPEC_LAUNCH_F16
            if (status != SPEC_OK || fused) return status;
            return launch_pdl(attention_combine_kernel<DH>, dim3(n_rows * m.cfg.n_heads), dim3(DH), 0, stream,
                              static_cast<const float*>(part), slices, out.att, out.hi, out.lo);
        }
    }
    if (attention_uses_mma(m, batch, m_rows, max_keys)) {
        const int m_blocks = (queries + 15) / 16;
        const dim3 grid(slices, m.cfg.n_kv_heads * m_blocks, batch);
        // K and V of a tile in turn (two CTAs per SM) once there are (sequence, KV head, query block)
        // groups for more than a thin wave: measured on the 7B shape, better from 32 groups on
        const bool in_turn = batch * m.cfg.n_kv_heads * m_blocks >= 32;
#define SPEC_LAUNCH_MMA(F, T, CLUSTER)                                                                                  \
    do {                                                                                                                \
        static std::atomic<unsigned long long> configured{0};                                                           \
        if (first_use_on_this_device(configured))                                                                       \
            SPEC_CUDA_TRY(cudaFuncSetAttribute(attention_mma_kernel<KV, DH, F, T>,                                      \
                                               cudaFuncAttributeMaxDynamicSharedMemorySize,                             \
                                               static_cast<int>(MmaSmem<DH, T>::kBytes)));                              \
        status = launch_attn(attention_mma_kernel<KV, DH, F, T>, grid, dim3(32 * kMmaWarps), MmaSmem<DH, T>::kBytes,    \
                             CLUSTER, stream, src.q, src.q_stride, rows.pos, rows.seq, m_rows, m.cfg.n_heads,           \
                             m.cfg.n_kv_heads, m_blocks, pool, src.pool.page_table, src.pool.pages_per_seq,            \
                             src.pool.page_size, src.kv_len, src.bias, src.bias_span, src.bias_zero, scale, part, out); \
    } while (0)
        if (fused && in_turn) SPEC_LAUNCH_MMA(true, true, slices);
        else if (fused) SPEC_LAUNCH_MMA(true, false, slices);
        else if (in_turn) SPEC_LAUNCH_MMA(false, true, 0);
        else SPEC_LAUNCH_MMA(false, false, 0);
#undef SPEC_LAUNCH_MMA
    } else {
        const int ks = attention_sub_slices(queries);
        const int warps = std::min(kMaxAttnWarps, std::max(1, queries * ks));
        const dim3 grid(slices, m.cfg.n_kv_heads, batch);
        status = fused ? launch_attn(attention_kernel<KV, DH, true>, grid, dim3(32 * warps), 0, slices, stream, src.q, src.q_stride,
                                     rows.pos, rows.seq, m_rows, m.cfg.n_heads, m.cfg.n_kv_heads, ks, pool, src.pool.page_table,
                                     src.pool.pages_per_seq, src.pool.page_size, src.kv_len, src.bias, src.bias_span,
                                     src.bias_zero, scale, part, out)
                       : launch_attn(attention_kernel<KV, DH, false>, grid, dim3(32 * warps), 0, 0, stream, src.q, src.q_stride,
                                     rows.pos, rows.seq, m_rows, m.cfg.n_heads, m.cfg.n_kv_heads, ks, pool, src.pool.page_table,
                                     src.pool.pages_per_seq, src.pool.page_size, src.kv_len, src.bias, src.bias_span,
                                     src.bias_zero, scale, part, out);
    }
    if (status != SPEC_OK || fused) return status;
    return launch_pdl(attention_combine_kernel<DH>, dim3(n_rows * m.cfg.n_heads), dim3(DH), 0, stream,
                      static_cast<const float*>(part), slices, out.att, out.hi, out.lo);
}

}  // namespace

int launch_attention(const Model& m, const AttnSource& src, const RowMeta& rows, int batch, int m_rows, int slices,
                     int max_keys, float* part, float* att, __nv_bfloat16* att_hi, __nv_bfloat16* att_lo, cudaStream_t stream) {
    const AttnOut out{att, att_hi, att_lo};
    if (src.pool.dtype == SPEC_DTYPE_BF16) {
        if (m.cfg.d_head == 64) return launch_attention_variant<__nv_bfloat16, 64>(m, src, rows, batch, m_rows, slices, max_keys, part, out, stream);
        return launch_attention_variant<__nv_bfloat16, 128>(m, src, rows, batch, m_rows, slices, max_keys, part, out, stream);
    }
    if (src.pool.dtype == SPEC_DTYPE_FP16) {
        if (m.cfg.d_head == 64) return launch_attention_variant<__half, 64>(m, src, rows, batch, m_rows, slices, max_keys, part, out, stream);
        return launch_attention_variant<__half, 128>(m, src, rows, batch, m_rows, slices, max_keys, part, out, stream);
    }
    if (m.cfg.d_head == 64) return launch_attention_variant<float, 64>(m, src, rows, batch, m_rows, slices, max_keys, part, out, stream);
    return launch_attention_variant<float, 128>(m, src, rows, batch, m_rows, slices, max_keys, part, out, stream);
}

}  // namespace spec
