// One forward pass over a few rows as ONE persistent kernel.
//
// A decoding pass over gamma + 1 rows is a stream of weights (Section 3.4: the rows share
// one read of every matrix) interrupted by short dependent steps: normalisation, rotary
// positions, attention, the activation.  Launched as a chain of kernels, every one of those
// steps leaves HBM idle while it runs and while the next GEMM fills its pipeline.  Here the
// whole pass is one cooperative kernel with one CTA per SM:
//
//   * warp 0 streams weight tiles with bulk copies into a ring of shared-memory stages.  It
//     depends on nothing but free stages, so it runs ahead through every dependent step
//     and across GEMM boundaries: while the other warps sit in a grid-wide barrier or in
//     the attention, the ring keeps filling with the next matrix.
//   * every GEMM is cut "stream-K" fashion: the (128-feature tile, 64-column block) units
//     of a matrix, in the tile-major order in which they are stored, are dealt out in
//     equal contiguous runs, one per CTA, so that every SM streams the same number of
//     bytes of every matrix whatever its shape.  A run covers parts of one to three
//     tiles; each part is accumulated in tensor memory (tcgen05.mma, M 128 x N 16) and
//     written as a partial sum; the consumer adds the parts of a tile in CTA order.
//   * the activation operand of a GEMM is built by its consumer: a few warps of every CTA
//     form the 16 x 64 block that goes with a weight tile straight from the producer's
//     results (residual stream + partial sums, times the norm gain; attention output;
//     gated activation of the FFN-in partial sums), split it into two bf16 terms and
//     store it in the MMA's swizzled layout.  RMSNorm's row scale is applied by whoever
//     consumes the GEMM (W (s x) = s (W x)), so no step waits for a row reduction.
//   * between dependent steps there is one grid-wide barrier (a counter in global
//     memory); steps: qkv GEMM | rotary + K,V append | attention | slice merge | out
//     projection | FFN-in | FFN-out, and at the end LM head | logits.
//
// Every wait (mbarrier, grid barrier) is bounded; on expiry the kernel records an error,
// tells the other CTAs, waits for its own copies in flight, frees its tensor memory and
// returns.
#include <algorithm>
#include <cstdlib>
#include <mutex>
#include <vector>

#include "attn_unit.cuh"

#define SPEC_TRY_STATUS(...)                      \
    do {                                          \
        const int status__ = (__VA_ARGS__);       \
        if (status__ != SPEC_OK) return status__; \
    } while (0)

namespace spec {
namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kStages = 10;                       // even: see the roles of gemm_step
constexpr int kABytes = 128 * 64 * 2;             // one weight tile
constexpr int kBBytes = 16 * 64 * 2;              // one term of the activation block (16 rows)
constexpr int kStageBytes = kABytes + 2 * kBBytes;
constexpr int kMaxRows = 16;                      // N of the MMA
constexpr int kBuilders = 8;                      // warps 8 .. 15 (a power of two)
constexpr int kWorkers = 14;                      // warps 2 .. 15 in the steps between GEMMs
constexpr int kBarThreads = kThreads - 32;        // everybody but the weight producer
constexpr int kMaxSlices = 32;
constexpr uint32_t kSpinLimit = 1u << 24;

__device__ int g_mega_error;  // first bounded wait that expired (0 = none)

constexpr int kMaxTileCounts = 4096;  // tiles of all GEMM shapes of a model together

struct Smem {
    static constexpr int kRing = kStages * kStageBytes;
    static constexpr int kBars = kRing;                                // wfull, bfull, empty [kStages]; acc_full, acc_empty [2]
    static constexpr int kTmemSlot = kBars + (3 * kStages + 4) * 8;
    static constexpr int kAbort = kTmemSlot + 4;                      // abort flag, then the barrier's verdict
    static constexpr int kScale = kAbort + 8;                         // row scales [16]
    static constexpr int kRowPos = kScale + 16 * 4;                   // the rows' positions, sequence slots; key count per sequence
    static constexpr int kShare = (kRowPos + 3 * 16 * 4 + 15) / 16 * 16;  // attention states, one per worker warp
    static constexpr int kCounts = kShare + kWorkers * (128 + 2) * 4;     // parts per tile of every GEMM shape
    static constexpr int kTotal = kCounts + kMaxTileCounts + 1024 /* alignment slack */;
};

// ---- PTX wrappers -------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}
// Bounded wait for the phase with the given parity; false on time-out or once the CTA is giving up.
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {  // non-blocking form
    uint32_t done;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}
// `nap` > 0: the caller can afford to react late; it sleeps that many nanoseconds between polls, so
// that its polling does not take issue slots from the warps that share its scheduler.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, unsigned nap = 0) {
    if (mbar_test(bar, parity)) return true;
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if (nap) __nanosleep(nap);
        if ((spin & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// 16 KB of global memory to shared memory, completion counted on an mbarrier.  The weights are read
// once per pass: they are marked evict-first so that they do not push the activations, the partial
// sums and the prefetched K,V rows out of L2.
__device__ __forceinline__ uint64_t evict_first_policy() {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(smem_u32(dst)),
        "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
// asks for a range of global memory (16-byte aligned, a multiple of 16 bytes) to be brought into L2
__device__ __forceinline__ void prefetch_l2(const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr & 0x3FFFF) >> 4);
    d |= static_cast<uint64_t>(1) << 16;
    d |= static_cast<uint64_t>(1024 >> 4) << 32;  // 8-row groups are 1024 bytes apart
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;          // 128-byte swizzle
    return d;
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 16
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kMaxRows >> 3) << 17) |
                                (static_cast<uint32_t>(128 >> 4) << 24);
__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(kInstrDesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
template <int ID, int THREADS>
__device__ __forceinline__ void named_sync() { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(THREADS) : "memory"); }
// Loads that are requested in program order and whose results may stay outstanding: the compiler
// keeps `asm volatile` statements in order, so a run of these is a run of loads in flight together.
__device__ __forceinline__ float2 ld_f2(const float* p) {
    float2 v;
    asm volatile("ld.global.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ float ld_f1(const float* p) {
    float v;
    asm volatile("ld.global.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

// ---- what the kernel is given --------------------------------------------------
struct MegaLayer {
    const float *ln1, *ln2, *lnx;
    const __nv_bfloat16 *wqkv, *wo, *w_in, *w_out, *wq_x, *wo_x;  // tile-major copies
    void* kv;        // this block's K,V pool
    void* cross_kv;  // encoder-decoder: its cross-attention K,V pool
};

struct MegaArgs {
    // model
    int arch, n_layers, d, n_heads, n_kv_heads, dh, d_ff, ffn, vocab, max_positions, emb_bf16;
    float eps;
    const void *tok_emb, *pos_emb;
    const float* ln_f;
    const __nv_bfloat16* head;
    const float2* rope;
    const MegaLayer* layers;
    // caches
    const int32_t* page_table;
    int pages_per_seq, page_size;
    const int32_t* src_page_table;
    int src_pages_per_seq;
    const int32_t* src_len;
    const float* dec_bias;
    int bias_span, bias_zero;
    // the pass
    int n_rows, m_rows, batch;
    const int32_t *row_token, *row_pos, *row_seq;
    int n_logit_rows;
    const int32_t *logit_src, *logit_dst;
    float* logits;
    // scratch
    float* h[2];      // residual stream [16][d], two copies used in turn
    float* ssq[2];    // per 64-column block of a row: sum of squares [k_blocks][16]
    float* part[2];   // partial sums of the GEMMs, used in turn
    float* q;         // q rows (and nothing else) [16][n_heads * dh]
    float* att;       // attention output [16][n_heads * dh]
    float* attn_part; // per key slice: (max, sum, accumulator) of every (row, head)
    unsigned* sync;   // [0..1] the grid barrier's 64-bit arrival count, [2] the give-up flag
    // parts per tile of every GEMM shape of the model (bytes, made on the host): offsets by kind
    // 0 qkv, 1 out-projection, 2 cross q, 3 cross out-projection, 4 FFN-in, 5 FFN-out, 6 LM head
    const uint8_t* tile_counts;
    int count_offset[7];
    int count_total;
    unsigned long long* trace;  // optional: every CTA's clock when it arrives at every grid barrier (diagnostic)
    int trace_capacity;
};

struct GemmDesc {
    const __nv_bfloat16* w;
    int n_out, k, tiles, kbn;
    unsigned units;  // tiles * kbn; units * CTAs stays below 2^32 (checked on the host)
};

__device__ __forceinline__ int gemms_per_layer(const MegaArgs& a) { return a.arch == SPEC_ARCH_T5 ? 6 : 4; }

__device__ __forceinline__ GemmDesc make_desc(const __nv_bfloat16* w, int n_out, int k) {
    GemmDesc g;
    g.w = w;
    g.n_out = n_out;
    g.k = k;
    g.tiles = (n_out + 127) / 128;
    g.kbn = (k + 63) / 64;
    g.units = static_cast<unsigned>(g.tiles) * static_cast<unsigned>(g.kbn);
    return g;
}

// Kind of GEMM number g (see MegaArgs::count_offset).
__device__ __forceinline__ int gemm_kind(const MegaArgs& a, int g) {
    const int per = gemms_per_layer(a);
    if (g >= per * a.n_layers) return 6;
    const int which = g % per;
    return a.arch != SPEC_ARCH_T5 && which >= 2 ? which + 2 : which;
}

// GEMM number g of the pass, in program order.
__device__ __forceinline__ GemmDesc gemm_desc(const MegaArgs& a, int g) {
    const int per = gemms_per_layer(a);
    const int q_dim = a.n_heads * a.dh, kv_dim = a.n_kv_heads * a.dh;
    if (g >= per * a.n_layers) return make_desc(a.head, a.vocab, a.d);
    const MegaLayer& L = a.layers[g / per];
    int which = g % per;
    if (a.arch != SPEC_ARCH_T5 && which >= 2) which += 2;
    switch (which) {
        case 0: return make_desc(L.wqkv, q_dim + 2 * kv_dim, a.d);
        case 1: return make_desc(L.wo, a.d, q_dim);
        case 2: return make_desc(L.wq_x, q_dim, a.d);
        case 3: return make_desc(L.wo_x, a.d, q_dim);
        case 4: return make_desc(L.w_in, a.ffn == SPEC_FFN_GELU ? a.d_ff : 2 * a.d_ff, a.d);
        default: return make_desc(L.w_out, a.d, a.d_ff);
    }
}

// The contiguous run of units of CTA c (of P): [unit_begin(c), unit_begin(c + 1)).
__host__ __device__ __forceinline__ unsigned unit_begin(unsigned units, int c, int P) {
    return units * static_cast<unsigned>(c) / static_cast<unsigned>(P);
}
__host__ __device__ __forceinline__ int cta_of_unit(unsigned units, unsigned u, int P) {
    int c = static_cast<int>(u * static_cast<unsigned>(P) / units);
    while (c + 1 < P && unit_begin(units, c + 1, P) <= u) ++c;
    return c;
}

// Partial sums of a GEMM: for tile t the part of CTA c is slot j = c - first(t), first(t) the CTA
// that owns the tile's first unit; [(t * jmax + j) * 16 + row][128 features].  (A matrix with
// fewer units than CTAs gives a CTA one unit or none: then slot j is the tile's j-th unit.)
struct TileParts {
    const float* base;  // part 0, row 0, feature 0 of the tile; parts are 16 * 128 floats apart
    int count;
};
struct PartialView {
    const float* base;
    const uint8_t* counts;  // parts per tile (shared memory)
    int jmax;
    __device__ __forceinline__ TileParts tile(int t) const {
        return TileParts{base + static_cast<size_t>(t) * jmax * (kMaxRows * 128), counts[t]};
    }
};

// The most CTAs that contribute to one tile: a tile's kbn units meet runs of per = units / P
// (or one more) units.
__host__ __device__ inline int max_contributors(unsigned units, int kbn, int P) {
    const int per = static_cast<int>(units / static_cast<unsigned>(P));
    if (per == 0) return kbn;  // fewer units than CTAs: every unit may be another CTA's
    return static_cast<int>((kbn + per - 2) / per + 1);
}

__device__ __forceinline__ PartialView partial_view(const MegaArgs& a, int g, int P, const uint8_t* counts_sh) {
    const GemmDesc gd = gemm_desc(a, g);
    PartialView v;
    v.base = a.part[g & 1];
    v.counts = counts_sh + a.count_offset[gemm_kind(a, g)];
    v.jmax = max_contributors(gd.units, gd.kbn, P);
    return v;
}

// sum of a column pair (features off, off + 1 of the tile) over the tile's parts, in CTA order
__device__ __forceinline__ float2 sum_parts2(const TileParts& tp, int off, int row) {
    const float* p0 = tp.base + row * 128 + off;
    float2 acc = *reinterpret_cast<const float2*>(p0);
    for (int j = 1; j < tp.count; ++j) {
        const float2 p = *reinterpret_cast<const float2*>(p0 + static_cast<size_t>(j) * (kMaxRows * 128));
        acc.x += p.x;
        acc.y += p.y;
    }
    return acc;
}

__device__ __forceinline__ float gelu_tanh(float x) {
    const float k = 0.7978845608028654f;
    return 0.5f * x * (1.0f + tanhf(k * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float silu(float x) { return x / (1.0f + expf(-x)); }

// RMSNorm's scale of a row from the per-block sums of squares (every warp that needs it
// evaluates the same expression on the same values).
// This lane's share of a row's sum of squares: blocks lane, lane + 32, ..., four loads in flight.
__device__ __forceinline__ float row_ssq_share(const float* ssq, int kbn, int row, int lane) {
    float s = 0.0f;
    for (int kb0 = lane; kb0 < kbn; kb0 += 128) {
        float v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = ld_f1(ssq + min(kb0 + 32 * i, kbn - 1) * kMaxRows + row);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (kb0 + 32 * i < kbn) s += v[i];
    }
    return s;
}
__device__ __forceinline__ float row_scale(const float* ssq, int kbn, int row, int d, float eps, int lane) {
    return rsqrtf(warp_sum(row_ssq_share(ssq, kbn, row, lane)) / static_cast<float>(d) + eps);
}

// Per-thread view of the kernel's shared state.
struct Cta {
    uint8_t* ring;
    uint64_t *wfull, *bfull, *empty, *acc_full, *acc_empty;
    volatile int* abort_flag;
    volatile int* verdict;  // written by one thread inside the grid barrier: 1 = carry on, 0 = unwind
    float* scale;
    const int *row_pos, *row_seq, *seq_keys;  // shared-memory copies: per row, per row, per sequence of the pass
    const uint8_t* counts;                    // shared-memory copy of MegaArgs::tile_counts
    uint32_t tmem;
    int c, P;         // this CTA, CTAs
    unsigned n;       // units this CTA has been through (all GEMMs so far)
    int items;        // accumulator parts this CTA has been through
    int barriers;     // grid barriers this CTA has been through
};

enum Source { kSrcEmbed, kSrcResid, kSrcPlain, kSrcAct };

// Grid-wide barrier of everybody but the weight producers.
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Grid-wide barrier of everybody but the weight producers.  One 64-bit word counts arrivals for
// ever: P CTAs arrive at every barrier, so the arrivals of the k-th barrier since the word was
// zero take the values k P .. k P + P - 1 and the barrier is complete once the word reaches
// (k + 1) P.  Nothing is ever reset, so the state a launch leaves behind (a multiple of P) is the
// next launch's starting point whatever the two launches were.  A second word tells every CTA to
// unwind after a wait has run out.
__device__ __forceinline__ bool grid_sync(const MegaArgs& a, Cta& cta) {
    named_sync<1, kBarThreads>();
    ++cta.barriers;
    const int stamp = 2 + (cta.barriers - 1) * cta.P + cta.c;  // every CTA's arrival at every barrier
    if (a.trace && threadIdx.x == 32 && stamp < a.trace_capacity) a.trace[stamp] = global_ns();
    if (threadIdx.x == 32) {
        unsigned long long* word = reinterpret_cast<unsigned long long*>(a.sync);
        volatile unsigned* give_up = a.sync + 2;
        if (*cta.abort_flag) {
            *give_up = 1u;
        } else {
            unsigned long long old;
            asm volatile("atom.add.release.gpu.global.u64 %0, [%1], %2;" : "=l"(old) : "l"(word), "l"(1ull) : "memory");
            const unsigned long long target = (old / static_cast<unsigned>(cta.P) + 1ull) * static_cast<unsigned>(cta.P);
            bool done = false;
            for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
                unsigned long long v;
                asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
                if (v >= target) { done = true; break; }
                if ((spin & 63u) == 63u && *give_up) break;
                if (spin > 4096) __nanosleep(64);
            }
            if (!done) {
                *cta.abort_flag = 1;
                *give_up = 1u;
                atomicCAS(&g_mega_error, 0, 100);
            }
        }
        *cta.verdict = *cta.abort_flag == 0 ? 1 : 0;  // one reader of the flag, so that every thread takes the same way
    }
    named_sync<1, kBarThreads>();
    return *cta.verdict != 0;
}

// A warp waits on an mbarrier: lane 0 polls (bounded), every lane learns the outcome.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int lane, unsigned nap = 0) {
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, abort_flag, nap) ? 1 : 0;
    ok = __shfl_sync(kFullMask, ok, 0);
    if (ok) mbar_try(bar, parity);  // (the phase is complete: every lane observes it before it touches the data)
    return ok != 0;
}

// ---- the weight stream -----------------------------------------------------------
__device__ void produce_weights(const MegaArgs& a, Cta& cta) {
    const int total = gemms_per_layer(a) * a.n_layers + 1;
    unsigned n = 0;
    bool ok = true;
    const uint64_t policy = evict_first_policy();
    for (int g = 0; g < total && ok; ++g) {
        const GemmDesc gd = gemm_desc(a, g);
        const unsigned u0 = unit_begin(gd.units, cta.c, cta.P), u1 = unit_begin(gd.units, cta.c + 1, cta.P);
        for (unsigned u = u0; u < u1; ++u, ++n) {
            const int s = static_cast<int>(n % kStages);
            const uint32_t round = n / kStages;
            if (!mbar_wait(&cta.empty[s], (round & 1u) ^ 1u, cta.abort_flag)) { ok = false; break; }
            mbar_expect_tx(&cta.wfull[s], kABytes);
            bulk_load(cta.ring + s * kStageBytes, gd.w + static_cast<size_t>(u) * (kABytes / 2), kABytes, &cta.wfull[s], policy);
        }
    }
    if (!ok) {
        atomicCAS(&g_mega_error, 0, 1);
        // copies already issued still land: wait for them (each has its own barrier phase) before the CTA may leave
        for (unsigned m = n > kStages ? n - kStages : 0; m < n; ++m) {
            const int s = static_cast<int>(m % kStages);
            for (uint32_t spin = 0; spin < kSpinLimit; ++spin)
                if (mbar_try(&cta.wfull[s], (m / kStages) & 1u)) break;
        }
    }
}

// ---- the activation block of one unit ----------------------------------------------
// Two columns per lane: columns kb * 64 + 2 * lane, + 1 of every row, as two bf16 terms in the
// swizzled K-major layout of the MMA's N side.
struct BuildCtx {
    Source src;
    int k_total;                 // inner dimension of this GEMM
    const float* gain;           // norm gain (embed / resid)
    const float* h_in;           // resid: residual stream before the update
    float* h_out;                // embed / resid: updated residual stream (written by the tile-0 units)
    float* ssq_out;
    const float* ssq_in;         // act: the sums of squares that go with the FFN-in GEMM's operand
    PartialView prev;            // resid / act: the producer GEMM's partial sums
    const float* plain;          // plain: fp32 rows [16][k_total]
};

__device__ __forceinline__ void store_pair(uint8_t* stage, int row, int lane, float x0, float x1) {
    const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
    const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0)), l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
    const int col = 2 * lane;
    const uint32_t off = (row >> 3) * 1024 + (row & 7) * 128 + (((col >> 3) ^ (row & 7)) << 4) + (col & 7) * 2;
    __nv_bfloat162 hv, lv;
    hv.x = h0; hv.y = h1;
    lv.x = l0; lv.y = l1;
    *reinterpret_cast<__nv_bfloat162*>(stage + kABytes + off) = hv;
    *reinterpret_cast<__nv_bfloat162*>(stage + kABytes + kBBytes + off) = lv;
}

constexpr int kRowBatch = 4;  // rows of a block whose loads are requested together

// Parts j0 .. j0 + N - 1 of a column pair of one row, requested together.  Every load is
// unconditional (an index past the last part re-reads the last part; the sum skips it): a load
// whose result feeds a select would make the thread wait for it before it requests the next one.
template <int N>
__device__ __forceinline__ void load_parts(const TileParts& tp, int off, int row, int j0, float2 (&p)[N]) {
    const float* p0 = tp.base + row * 128 + off;
#pragma unroll
    for (int j = 0; j < N; ++j)
        p[j] = ld_f2(p0 + static_cast<size_t>(min(j0 + j, tp.count - 1)) * (kMaxRows * 128));
}
// their sum in part order, continued over the parts beyond the first N (rare: many CTAs on one tile)
template <int N>
__device__ __forceinline__ float2 sum_loaded(const TileParts& tp, int off, int row, const float2 (&p)[N]) {
    float2 acc = p[0];
#pragma unroll
    for (int j = 1; j < N; ++j)
        if (j < tp.count) {
            acc.x += p[j].x;
            acc.y += p[j].y;
        }
    for (int j0 = N; j0 < tp.count; j0 += N) {
        float2 more[N];
        load_parts<N>(tp, off, row, j0, more);
#pragma unroll
        for (int j = 0; j < N; ++j)
            if (j0 + j < tp.count) {
                acc.x += more[j].x;
                acc.y += more[j].y;
            }
    }
    return acc;
}

template <int SRC>
__device__ __forceinline__ void build_block(const MegaArgs& a, const Cta& cta, const BuildCtx& b, uint8_t* stage, int tile, int kb,
                                            int lane) {
    constexpr int PB = SRC == kSrcAct ? 4 : 8;      // parts in flight per row and tile
    constexpr int UP = SRC == kSrcAct ? PB : 1;
    const int col = kb * 64 + 2 * lane;
    const bool live = col < b.k_total;
    const bool writer = tile == 0 && (SRC == kSrcEmbed || SRC == kSrcResid);
    const bool gated = SRC == kSrcAct && a.ffn != SPEC_FFN_GELU;
    float2 gain = make_float2(0.f, 0.f);
    if (live && b.gain) gain = *reinterpret_cast<const float2*>(b.gain + col);
    // the parts of the producer's tile(s) this lane's columns come from
    TileParts tp{nullptr, 0}, tp_up{nullptr, 0};
    if (live && (SRC == kSrcResid || SRC == kSrcAct)) tp = b.prev.tile(col >> 7);
    if (live && gated) tp_up = b.prev.tile((a.d_ff + col) >> 7);
    const int off = col & 127, off_up = (a.d_ff + col) & 127;
    for (int r0 = 0; r0 < a.n_rows; r0 += kRowBatch) {
        float2 v[kRowBatch], pa[kRowBatch][PB], pb[kRowBatch][UP];
        // ---- every load of these rows is requested before anything is used ----
#pragma unroll
        for (int i = 0; i < kRowBatch; ++i) {
            const int r = r0 + i;
            v[i] = make_float2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < PB; ++j) pa[i][j] = make_float2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < UP; ++j) pb[i][j] = make_float2(0.f, 0.f);
            if (!live || r >= a.n_rows) continue;
            if (SRC == kSrcEmbed) {
                const int t = min(max(a.row_token[r], 0), a.vocab - 1);
                const size_t at = static_cast<size_t>(t) * a.d + col;
                if (a.emb_bf16) {
                    const __nv_bfloat162 e = *reinterpret_cast<const __nv_bfloat162*>(static_cast<const __nv_bfloat16*>(a.tok_emb) + at);
                    v[i] = make_float2(__bfloat162float(e.x), __bfloat162float(e.y));
                } else {
                    v[i] = *reinterpret_cast<const float2*>(static_cast<const float*>(a.tok_emb) + at);
                }
                if (a.arch == SPEC_ARCH_GPT) {
                    const int p = min(max(a.row_pos[r], 0), a.max_positions - 1);
                    const size_t pat = static_cast<size_t>(p) * a.d + col;
                    if (a.emb_bf16) {
                        const __nv_bfloat162 e = *reinterpret_cast<const __nv_bfloat162*>(static_cast<const __nv_bfloat16*>(a.pos_emb) + pat);
                        v[i].x += __bfloat162float(e.x);
                        v[i].y += __bfloat162float(e.y);
                    } else {
                        const float2 e = *reinterpret_cast<const float2*>(static_cast<const float*>(a.pos_emb) + pat);
                        v[i].x += e.x;
                        v[i].y += e.y;
                    }
                }
            } else if (SRC == kSrcResid) {
                v[i] = ld_f2(b.h_in + static_cast<size_t>(r) * a.d + col);
                load_parts<PB>(tp, off, r, 0, pa[i]);
            } else if (SRC == kSrcPlain) {
                v[i] = ld_f2(b.plain + static_cast<size_t>(r) * b.k_total + col);
            } else {
                load_parts<PB>(tp, off, r, 0, pa[i]);
                if (gated) load_parts<UP>(tp_up, off_up, r, 0, pb[i]);
            }
        }
        // ---- combine, keep the updated stream (tile-0 units), split, store ----
#pragma unroll
        for (int i = 0; i < kRowBatch; ++i) {
            const int r = r0 + i;
            if (r >= a.n_rows) break;
            float2 x = v[i];
            if (live && SRC == kSrcResid) {
                const float2 p = sum_loaded<PB>(tp, off, r, pa[i]);
                x.x += p.x;
                x.y += p.y;
            } else if (live && SRC == kSrcAct) {  // the FFN's activation of the FFN-in sums, RMSNorm's scale applied here
                const float s = cta.scale[r];
                const float2 gate = sum_loaded<PB>(tp, off, r, pa[i]);
                if (!gated) {
                    x = make_float2(gelu_tanh(s * gate.x), gelu_tanh(s * gate.y));
                } else {
                    const float2 up = sum_loaded<UP>(tp_up, off_up, r, pb[i]);
                    if (a.ffn == SPEC_FFN_SWIGLU) x = make_float2(silu(s * gate.x) * (s * up.x), silu(s * gate.y) * (s * up.y));
                    else x = make_float2(gelu_tanh(s * gate.x) * (s * up.x), gelu_tanh(s * gate.y) * (s * up.y));
                }
            }
            if (writer) {  // one unit per column block keeps the new residual stream and its sum of squares
                if (live) *reinterpret_cast<float2*>(b.h_out + static_cast<size_t>(r) * a.d + col) = x;
                const float ss = warp_sum(x.x * x.x + x.y * x.y);
                if (lane == 0) b.ssq_out[kb * kMaxRows + r] = ss;
            }
            if (b.gain) {
                x.x *= gain.x;
                x.y *= gain.y;
            }
            store_pair(stage, r, lane, x.x, x.y);
        }
    }
}

// ---- one GEMM: every role of the CTA but the weight producer ---------------------------
// Leaves the partial sums of this CTA's parts in a.part[g & 1].
// Roles.  The ring is two interleaved half-rings: the units this CTA goes through are numbered
// n = 0, 1, 2, ... over the whole pass; unit n uses stage n % kStages (kStages is even), so even
// units use even stages and odd units odd stages.  Issuer X (warp 1 + X) takes the units of
// parity X, in order, into accumulator X of the part; builder warp 8 + b takes the units with
// n % 8 == b, in order.  Every mbarrier of a stage is therefore waited on by threads that go
// through that stage's phases in order (a wait by parity cannot tell a phase from the one two
// before it, so nobody may get two phases ahead of a barrier).
template <typename Prefetch>
__device__ void gemm_step(const MegaArgs& a, Cta& cta, int g, const BuildCtx& b, Prefetch prefetch) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const GemmDesc gd = gemm_desc(a, g);
    const unsigned u0 = unit_begin(gd.units, cta.c, cta.P), u1 = unit_begin(gd.units, cta.c + 1, cta.P);
    const int count = static_cast<int>(u1 - u0);
    // parts: the run cut at tile boundaries
    const int t_first = count > 0 ? static_cast<int>(u0 / gd.kbn) : 0;
    const int t_last = count > 0 ? static_cast<int>((u1 - 1) / gd.kbn) : -1;
    const int n_parts = t_last - t_first + 1;

    if (warp == 1 || warp == 2) {
        // ---- MMA issuers (one thread's wait / issue / commit chain per unit is longer than a unit's
        // share of the HBM stream, hence two of them; the epilogue adds their accumulators) ----
        if (lane == 0) {
            const unsigned which = warp - 1;
            bool ok = true;
            for (int part = 0; part < n_parts && ok; ++part) {
                const int t = t_first + part;
                const unsigned a0 = max(u0, static_cast<unsigned>(t) * gd.kbn), a1 = min(u1, static_cast<unsigned>(t + 1) * gd.kbn);
                const unsigned n0 = cta.n + (a0 - u0), n1 = cta.n + (a1 - u0);  // the part's units, pass-wide numbering
                const int it = cta.items + part, buf = it & 1;
                if (!mbar_wait(&cta.acc_empty[buf], ((static_cast<uint32_t>(it) >> 1) & 1u) ^ 1u, cta.abort_flag)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = cta.tmem + static_cast<uint32_t>((2 * buf + which) * kMaxRows);
                bool first = true;
                for (unsigned n = n0 + ((n0 ^ which) & 1u); n < n1; n += 2) {
                    const int s = static_cast<int>(n % kStages);
                    if (!mbar_wait(&cta.bfull[s], (n / kStages) & 1u, cta.abort_flag)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t base = smem_u32(cta.ring + s * kStageBytes);
                    const uint64_t a_desc = smem_desc_sw128(base), hi_desc = smem_desc_sw128(base + kABytes),
                                   lo_desc = smem_desc_sw128(base + kABytes + kBBytes);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t step = static_cast<uint64_t>((k * 32) >> 4);
                        mma_f16(acc, a_desc + step, hi_desc + step, (!first || k > 0) ? 1u : 0u);
                        mma_f16(acc, a_desc + step, lo_desc + step, 1u);
                    }
                    first = false;
                    mma_commit(&cta.empty[s]);
                }
                if (ok) mma_commit(&cta.acc_full[buf]);
            }
            if (!ok) atomicCAS(&g_mega_error, 0, 2);
        }
    } else if (warp >= 4 && warp < 8) {
        // ---- epilogue: warp w reads accumulator lanes 32 (w & 3) .. + 31 ----
        float* out = a.part[g & 1];
        const int jmax = max_contributors(gd.units, gd.kbn, cta.P);
        for (int part = 0; part < n_parts; ++part) {
            const int t = t_first + part;
            const unsigned a0 = max(u0, static_cast<unsigned>(t) * gd.kbn), a1 = min(u1, static_cast<unsigned>(t + 1) * gd.kbn);
            const unsigned n0 = cta.n + (a0 - u0), n1 = cta.n + (a1 - u0);
            const int it = cta.items + part, buf = it & 1;
            if (!warp_wait(&cta.acc_full[buf], (static_cast<uint32_t>(it) >> 1) & 1u, cta.abort_flag, lane)) {
                atomicCAS(&g_mega_error, 0, 3);
                break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // accumulator X holds the part's units of parity X: at least one of the two was used
            const bool both = n1 - n0 > 1;
            const uint32_t lanes = static_cast<uint32_t>((warp & 3) * 32) << 16;
            float v[16];
            tmem_ld16(cta.tmem + lanes + static_cast<uint32_t>((2 * buf + (both ? 0 : (n0 & 1u))) * kMaxRows), v);
            if (both) {
                float w[16];
                tmem_ld16(cta.tmem + lanes + static_cast<uint32_t>((2 * buf + 1) * kMaxRows), w);
#pragma unroll
                for (int r = 0; r < 16; ++r) v[r] += w[r];
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&cta.acc_empty[buf]);
            const int j = gd.units < static_cast<unsigned>(cta.P)
                              ? static_cast<int>(u0 % gd.kbn)
                              : cta.c - cta_of_unit(gd.units, static_cast<unsigned>(t) * gd.kbn, cta.P);
            float* dst = out + ((static_cast<size_t>(t) * jmax + j) * kMaxRows) * 128 + (warp & 3) * 32 + lane;
#pragma unroll
            for (int r = 0; r < kMaxRows; ++r)
                if (r < a.n_rows) dst[r * 128] = v[r];
        }
    } else if (warp == 3) {
        prefetch(lane);  // (the one warp without a role in a GEMM)
    } else {
        // ---- builders: a unit's block is announced once its weight tile has landed too, so that the
        // issuers wait on one barrier per unit ----
        const unsigned bi = warp - 8;
        if (b.src == kSrcAct) {  // RMSNorm's scale of every row, from the FFN-in GEMM's operand
            for (int r = bi; r < a.n_rows; r += kBuilders) {
                const float s = row_scale(b.ssq_in, (a.d + 63) / 64, r, a.d, a.eps, lane);
                if (lane == 0) cta.scale[r] = s;
            }
            named_sync<2, kBuilders * 32>();
        }
        for (unsigned i = (bi - cta.n) & (kBuilders - 1); i < static_cast<unsigned>(count); i += kBuilders) {
            const unsigned n = cta.n + i, u = u0 + i;
            const int s = static_cast<int>(n % kStages);
            if (!warp_wait(&cta.empty[s], ((n / kStages) & 1u) ^ 1u, cta.abort_flag, lane)) {
                atomicCAS(&g_mega_error, 0, 4);
                break;
            }
            uint8_t* stage = cta.ring + s * kStageBytes;
            const int tile = static_cast<int>(u / gd.kbn), kb = static_cast<int>(u % gd.kbn);
            switch (b.src) {
                case kSrcEmbed: build_block<kSrcEmbed>(a, cta, b, stage, tile, kb, lane); break;
                case kSrcResid: build_block<kSrcResid>(a, cta, b, stage, tile, kb, lane); break;
                case kSrcPlain: build_block<kSrcPlain>(a, cta, b, stage, tile, kb, lane); break;
                default: build_block<kSrcAct>(a, cta, b, stage, tile, kb, lane); break;
            }
            fence_async_smem();
            if (!warp_wait(&cta.wfull[s], (n / kStages) & 1u, cta.abort_flag, lane)) {
                atomicCAS(&g_mega_error, 0, 6);
                break;
            }
            __syncwarp();  // every lane's stores (and their proxy fences) come before the arrival
            if (lane == 0) mbar_arrive(&cta.bfull[s]);
        }
    }
    cta.n += count;
    cta.items += n_parts;
    __syncwarp();  // (the issuers' warps re-converge before the barrier that follows)
}

// ---- rotary positions, K,V append, q rows: finishes the projection GEMM g ----------------
// n_kv_heads = 0: queries only (cross-attention).
template <typename KV>
__device__ void qkv_step(const MegaArgs& a, const Cta& cta, int g, const float* ssq, int n_heads, int n_kv_heads, bool rope,
                         KV* kv_layer) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp < 2) return;
    const PartialView pv = partial_view(a, g, cta.P, cta.counts);
    const int heads = n_heads + 2 * n_kv_heads, half = a.dh / 2;
    const int kbn_d = (a.d + 63) / 64;
    const int units = a.n_rows * heads;
    // unit i -> CTA i % P, worker (i / P) % kWorkers
    for (int i = cta.c + cta.P * (warp - 2); i < units; i += cta.P * kWorkers) {
        const int r = i / heads, head = i % heads;
        const int p = cta.row_pos[r];
        const bool is_q = head < n_heads, is_k = !is_q && head < n_heads + n_kv_heads;
        // lane owns the pairs (j, j + 1) of the first half and the same of the second half; every
        // load of the unit (sums of squares, parts, rotation, page) is requested before any is used
        const int j = 2 * lane;
        const bool live = j < half;
        const int col = head * a.dh + j;
        const float sq = row_ssq_share(ssq, kbn_d, r, lane);
        TileParts t1{nullptr, 0}, t2{nullptr, 0};
        float2 p1[8], p2[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) p1[k] = p2[k] = make_float2(0.f, 0.f);
        float4 cs = make_float4(1.f, 0.f, 1.f, 0.f);
        int page = 0;
        if (live) {
            t1 = pv.tile(col >> 7);
            t2 = pv.tile((col + half) >> 7);
            load_parts<8>(t1, col & 127, r, 0, p1);
            load_parts<8>(t2, (col + half) & 127, r, 0, p2);
            if (rope && p >= 0 && (is_q || is_k)) cs = *reinterpret_cast<const float4*>(a.rope + static_cast<size_t>(p) * half + j);  // (cos, sin) x 2
            if (!is_q && p >= 0) page = a.page_table[cta.row_seq[r] * a.pages_per_seq + p / a.page_size];
        }
        const float s = rsqrtf(warp_sum(sq) / static_cast<float>(a.d) + a.eps);
        if (!live) continue;
        float2 x1 = sum_loaded<8>(t1, col & 127, r, p1), x2 = sum_loaded<8>(t2, (col + half) & 127, r, p2);
        x1.x *= s; x1.y *= s; x2.x *= s; x2.y *= s;
        const float2 y1 = make_float2(x1.x * cs.x - x2.x * cs.y, x1.y * cs.z - x2.y * cs.w);
        const float2 y2 = make_float2(x2.x * cs.x + x1.x * cs.y, x2.y * cs.z + x1.y * cs.w);
        if (is_q) {
            float* dst = a.q + static_cast<size_t>(r) * (n_heads * a.dh) + col;
            *reinterpret_cast<float2*>(dst) = y1;
            *reinterpret_cast<float2*>(dst + half) = y2;
        } else if (p >= 0) {
            const int kv_head = is_k ? head - n_heads : head - n_heads - n_kv_heads;
            const size_t block = (static_cast<size_t>(page) * 2 + (is_k ? 0 : 1)) * n_kv_heads + kv_head;
            KV* dst = kv_layer + (block * a.page_size + p % a.page_size) * a.dh + j;
            dst[0] = static_cast<KV>(y1.x);
            dst[1] = static_cast<KV>(y1.y);
            dst[half] = static_cast<KV>(y2.x);
            dst[half + 1] = static_cast<KV>(y2.y);
        }
    }
}

// ---- attention: (sequence, KV head, key slice) pieces dealt out to the CTAs ----------------
template <typename KV, int DH>
__device__ void attention_step(const MegaArgs& a, const Cta& cta, const KV* kv_layer, const int32_t* page_table,
                               int pages_per_seq, const int32_t* kv_len, const float* bias, int slices, float (*share)[DH + 2]) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp < 2) return;
    const int queries = (a.n_heads / a.n_kv_heads) * a.m_rows;
    const int ks = queries * 2 <= kWorkers ? kWorkers / queries : 1;
    const float scale = rsqrtf(static_cast<float>(DH));
    const int pieces = a.batch * a.n_kv_heads * slices;
    for (int u = cta.c; u < pieces; u += cta.P) {
        const int slice = u % slices, kv_head = (u / slices) % a.n_kv_heads, b = u / (slices * a.n_kv_heads);
        attend_slice<KV, DH, NamedSync<3, kWorkers * 32>>(a.q, a.n_heads * DH, a.row_pos, a.row_seq, a.m_rows, a.n_heads, a.n_kv_heads,
                                                         ks, kv_layer, page_table, pages_per_seq, a.page_size, kv_len, bias,
                                                         a.bias_span, a.bias_zero, scale, a.attn_part, slice, slices, kv_head, b,
                                                         warp - 2, kWorkers, lane, share, false, kv_len ? -1 : cta.seq_keys[b]);
        if (ks > 1) named_sync<3, kWorkers * 32>();  // the shared states are free again
    }
}

// merge of the key slices of every (row, head): one warp each
template <int DH>
__device__ void combine_step(const MegaArgs& a, const Cta& cta, int slices) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp < 2) return;
    constexpr int PAIRS = DH / 64;  // float2 per lane: the lane's DH / 32 consecutive elements
    const int units = a.n_rows * a.n_heads;
    for (int i = cta.c + cta.P * (warp - 2); i < units; i += cta.P * kWorkers) {
        const float* in = a.attn_part + static_cast<size_t>(i) * slices * (DH + 2);
        // the states' (max, sum) and the first eight accumulators are requested together
        const float ms_raw = ld_f1(in + min(lane, slices - 1) * (DH + 2)), ls_raw = ld_f1(in + min(lane, slices - 1) * (DH + 2) + 1);
        float2 o[PAIRS];
#pragma unroll
        for (int e = 0; e < PAIRS; ++e) o[e] = make_float2(0.f, 0.f);
        float w = 0.0f, l = 0.0f;
        for (int s0 = 0; s0 < slices; s0 += 8) {
            float2 v[8][PAIRS];
#pragma unroll
            for (int k = 0; k < 8; ++k)
#pragma unroll
                for (int e = 0; e < PAIRS; ++e)
                    v[k][e] = ld_f2(in + min(s0 + k, slices - 1) * (DH + 2) + 2 + lane * (2 * PAIRS) + 2 * e);  // (weight 0 past the last slice)
            if (s0 == 0) {
                const float ms = lane < slices ? ms_raw : -FLT_MAX, ls = lane < slices ? ls_raw : 0.0f;
                const float mm = warp_max(ms);
                w = lane < slices ? expf(ms - mm) : 0.0f;
                l = warp_sum(ls * w);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {  // slices in index order
                const float ws = __shfl_sync(kFullMask, w, (s0 + k) & 31);
#pragma unroll
                for (int e = 0; e < PAIRS; ++e) {
                    o[e].x += v[k][e].x * ws;
                    o[e].y += v[k][e].y * ws;
                }
            }
        }
#pragma unroll
        for (int e = 0; e < PAIRS; ++e)  // (an inactive row has no keys)
            *reinterpret_cast<float2*>(a.att + static_cast<size_t>(i) * DH + lane * (2 * PAIRS) + 2 * e) =
                make_float2(l > 0.0f ? o[e].x / l : 0.0f, l > 0.0f ? o[e].y / l : 0.0f);
    }
}

// Asks for the cached K,V rows that this CTA's attention pieces of one block will read to be
// brought into L2 (one warp; lane = 32-key tile of the piece).  Issued while the block's first
// GEMM streams, so that the attention finds its keys in L2.
template <typename KV, int DH>
__device__ void prefetch_keys(const MegaArgs& a, const Cta& cta, const KV* kv_layer, int slices, int lane) {
    const int pieces = a.batch * a.n_kv_heads * slices;
    const size_t head_stride = static_cast<size_t>(a.page_size) * DH;
    const size_t page_stride = 2 * static_cast<size_t>(a.n_kv_heads) * head_stride;
    const size_t v_offset = static_cast<size_t>(a.n_kv_heads) * head_stride;
    for (int u = cta.c; u < pieces; u += cta.P) {
        const int slice = u % slices, kv_head = (u / slices) % a.n_kv_heads, b = u / (slices * a.n_kv_heads);
        const int seq_keys = cta.seq_keys[b];
        const int tiles = (seq_keys + 31) / 32;
        const int t0 = static_cast<int>(static_cast<long long>(tiles) * slice / slices);
        const int t1 = static_cast<int>(static_cast<long long>(tiles) * (slice + 1) / slices);
        for (int t = t0 + lane; t < t1; t += 32) {
            const int k0 = 32 * t;
            const int page = a.page_table[cta.row_seq[b * a.m_rows] * a.pages_per_seq + k0 / a.page_size];
            const KV* tile = kv_layer + page * page_stride + kv_head * head_stride + static_cast<size_t>(k0 % a.page_size) * DH;
            prefetch_l2(tile, 32 * DH * sizeof(KV));
            prefetch_l2(tile + v_offset, 32 * DH * sizeof(KV));
        }
    }
}

// key slices per (sequence, KV head): about one piece per CTA, at least one 32-key tile per
// sub-slice, from the rows' own positions (the same on every CTA)
__device__ __forceinline__ int choose_slices(const MegaArgs& a, int P, int longest_keys) {
    const int queries = (a.n_heads / a.n_kv_heads) * a.m_rows;
    const int ks = queries * 2 <= kWorkers ? kWorkers / queries : 1;
    const int tiles = (longest_keys + 31) / 32;
    const int want = max(1, P / (a.batch * a.n_kv_heads));
    const int most = max(1, (tiles + ks - 1) / ks);
    return max(1, min(min(want, most), kMaxSlices));
}

// ---- the kernel ------------------------------------------------------------------------------
template <typename KV, int DH>
__global__ void __launch_bounds__(kThreads, 1) pass_kernel(const __grid_constant__ MegaArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    Cta cta;
    cta.ring = smem;
    cta.wfull = reinterpret_cast<uint64_t*>(smem + Smem::kBars);
    cta.bfull = cta.wfull + kStages;
    cta.empty = cta.bfull + kStages;
    cta.acc_full = cta.empty + kStages;
    cta.acc_empty = cta.acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + Smem::kTmemSlot);
    cta.abort_flag = reinterpret_cast<volatile int*>(smem + Smem::kAbort);
    cta.verdict = cta.abort_flag + 1;
    cta.scale = reinterpret_cast<float*>(smem + Smem::kScale);
    float(*share)[DH + 2] = reinterpret_cast<float(*)[DH + 2]>(smem + Smem::kShare);
    cta.c = blockIdx.x;
    cta.P = gridDim.x;
    cta.n = 0;
    cta.items = 0;
    cta.barriers = 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&cta.wfull[s], 1);
            mbar_init(&cta.bfull[s], 1);
            mbar_init(&cta.empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&cta.acc_full[i], 2);
            mbar_init(&cta.acc_empty[i], 4);
        }
        *cta.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // rows of the activation blocks that no pass row fills must still hold finite numbers
    for (int i = threadIdx.x; i < kStages * 2 * kBBytes / 16; i += kThreads) {
        const int s = i / (2 * kBBytes / 16), o = i % (2 * kBBytes / 16);
        *reinterpret_cast<uint4*>(smem + s * kStageBytes + kABytes + o * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_async_smem();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(64));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    cta.tmem = *tmem_slot;
    {
        int* rows_sh = reinterpret_cast<int*>(smem + Smem::kRowPos);
        cta.row_pos = rows_sh;
        cta.row_seq = rows_sh + 16;
        cta.seq_keys = rows_sh + 32;
        if (threadIdx.x < 16) {
            const int r = threadIdx.x;
            rows_sh[r] = r < a.n_rows ? a.row_pos[r] : -1;
            rows_sh[16 + r] = r < a.n_rows ? a.row_seq[r] : 0;
            int keys = 0;  // of sequence r of the pass: its rows' largest position + 1
            if (r < a.batch)
                for (int j = 0; j < a.m_rows; ++j) keys = max(keys, a.row_pos[r * a.m_rows + j] + 1);
            rows_sh[32 + r] = keys;
        }
        uint8_t* counts_sh = smem + Smem::kCounts;
        for (int i = threadIdx.x; i < a.count_total; i += kThreads) counts_sh[i] = a.tile_counts[i];
        cta.counts = counts_sh;
        __syncthreads();
    }
    if (a.trace && cta.c == 0 && threadIdx.x == 32 && a.trace_capacity > 1) {  // (CTAs; start of the pass)
        a.trace[0] = gridDim.x;
        a.trace[1] = global_ns();
    }

    if (warp == 0) {
        if (lane == 0) produce_weights(a, cta);
        __syncwarp();
    } else {
        const int per = gemms_per_layer(a);
        const int q_dim = a.n_heads * DH;
        int hb = 0;  // which copy of the residual stream (and of the sums of squares) is current
        bool ok = true;
        // the longest key set of any sequence of the pass
        int longest = 0;
        for (int b = 0; b < a.batch; ++b) longest = max(longest, cta.seq_keys[b]);
        const int slices = choose_slices(a, cta.P, longest);
        for (int l = 0; l < a.n_layers && ok; ++l) {
            const MegaLayer& L = a.layers[l];
            int g = l * per;
            BuildCtx b{};
            // ---- projection of the normalised stream; the stream itself is brought up to date on the way ----
            b.src = l == 0 ? kSrcEmbed : kSrcResid;
            b.k_total = a.d;
            b.gain = L.ln1;
            b.h_in = a.h[hb];
            b.h_out = a.h[hb ^ 1];
            b.ssq_out = a.ssq[hb ^ 1];
            if (l > 0) b.prev = partial_view(a, g - 1, cta.P, cta.counts);
            gemm_step(a, cta, g, b, [&](int ln) { prefetch_keys<KV, DH>(a, cta, static_cast<const KV*>(L.kv), slices, ln); });
            hb ^= 1;
            if (!(ok = grid_sync(a, cta))) break;
            qkv_step<KV>(a, cta, g, a.ssq[hb], a.n_heads, a.n_kv_heads, a.arch == SPEC_ARCH_LLAMA, static_cast<KV*>(L.kv));
            if (!(ok = grid_sync(a, cta))) break;
            attention_step<KV, DH>(a, cta, static_cast<const KV*>(L.kv), a.page_table, a.pages_per_seq, nullptr,
                                   a.arch == SPEC_ARCH_T5 ? a.dec_bias : nullptr, slices, share);
            if (!(ok = grid_sync(a, cta))) break;
            combine_step<DH>(a, cta, slices);
            if (!(ok = grid_sync(a, cta))) break;
            // ---- out-projection ----
            ++g;
            b = BuildCtx{};
            b.src = kSrcPlain;
            b.k_total = q_dim;
            b.plain = a.att;
            gemm_step(a, cta, g, b, [](int) {});
            if (!(ok = grid_sync(a, cta))) break;
            // ---- FFN-in on the normalised, updated stream ----
            ++g;
            b = BuildCtx{};
            b.src = kSrcResid;
            b.k_total = a.d;
            b.gain = L.ln2;
            b.h_in = a.h[hb];
            b.h_out = a.h[hb ^ 1];
            b.ssq_out = a.ssq[hb ^ 1];
            b.prev = partial_view(a, g - 1, cta.P, cta.counts);
            gemm_step(a, cta, g, b, [](int) {});
            hb ^= 1;
            if (!(ok = grid_sync(a, cta))) break;
            // ---- FFN-out on the activation of the FFN-in sums ----
            ++g;
            b = BuildCtx{};
            b.src = kSrcAct;
            b.k_total = a.d_ff;
            b.ssq_in = a.ssq[hb];
            b.prev = partial_view(a, g - 1, cta.P, cta.counts);
            gemm_step(a, cta, g, b, [](int) {});
            if (!(ok = grid_sync(a, cta))) break;
        }
        if (ok && a.n_logit_rows > 0) {
            // ---- final norm and LM head ----
            const int g = per * a.n_layers;
            BuildCtx b{};
            b.src = kSrcResid;
            b.k_total = a.d;
            b.gain = a.ln_f;
            b.h_in = a.h[hb];
            b.h_out = a.h[hb ^ 1];
            b.ssq_out = a.ssq[hb ^ 1];
            b.prev = partial_view(a, g - 1, cta.P, cta.counts);
            gemm_step(a, cta, g, b, [](int) {});
            hb ^= 1;
            ok = grid_sync(a, cta);
            if (ok) {
                // logits[dst(i)][n] = scale(src(i)) * sum of the parts
                const int kbn_d = (a.d + 63) / 64;
                if (warp >= 2)
                    for (int r = warp - 2; r < a.n_rows; r += kWorkers) {
                        const float s = row_scale(a.ssq[hb], kbn_d, r, a.d, a.eps, lane);
                        if (lane == 0) cta.scale[r] = s;
                    }
                named_sync<1, kBarThreads>();
                const PartialView pv = partial_view(a, g, cta.P, cta.counts);
                const int pairs = a.vocab / 2;  // (the vocabulary is even whenever this kernel is used)
                const long long total = static_cast<long long>(a.n_logit_rows) * pairs;
                for (long long i = static_cast<long long>(cta.c) * kBarThreads + (threadIdx.x - 32); i < total;
                     i += static_cast<long long>(cta.P) * kBarThreads) {
                    const int li = static_cast<int>(i / pairs), col = 2 * static_cast<int>(i % pairs);
                    const int src = a.logit_src ? a.logit_src[li] : li, dst = a.logit_dst ? a.logit_dst[li] : li;
                    const float2 v = sum_parts2(pv.tile(col >> 7), col & 127, src);
                    const float s = cta.scale[src];
                    *reinterpret_cast<float2*>(a.logits + static_cast<size_t>(dst) * a.vocab + col) = make_float2(v.x * s, v.y * s);
                }
            }
        }
        if (!ok) atomicCAS(&g_mega_error, 0, 5);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(cta.tmem), "r"(64));
}

}  // namespace

// ---- host side ---------------------------------------------------------------------------------
namespace {

template <typename KV, int DH>
int launch_variant(const MegaArgs& args, int ctas, cudaStream_t stream) {
    static std::atomic<unsigned long long> configured{0};
    if (first_use_on_this_device(configured))
        SPEC_CUDA_TRY(cudaFuncSetAttribute(pass_kernel<KV, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::kTotal));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Smem::kTotal;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;  // every CTA resident at once: the grid barrier needs it
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, pass_kernel<KV, DH>, args);
    if (err != cudaSuccess) return fail(SPEC_ERR_CUDA, "pass kernel launch failed: %s", cudaGetErrorString(err));
    return SPEC_OK;
}

template <typename KV, int DH>
int resident_ctas(int* out) {
    SPEC_CUDA_TRY(cudaFuncSetAttribute(pass_kernel<KV, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::kTotal));
    int per_sm = 0, device = 0, sms = 0;
    SPEC_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pass_kernel<KV, DH>, kThreads, Smem::kTotal));
    SPEC_CUDA_TRY(cudaGetDevice(&device));
    SPEC_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    *out = per_sm >= 1 ? sms : 0;  // one CTA per SM
    return SPEC_OK;
}

struct Shape {
    int n_out, k;
};

std::mutex g_sync_mutex;
std::vector<unsigned*> g_sync_words;  // the barrier words of every live context

std::vector<Shape> gemm_shapes(const Model& m) {
    const spec_model_cfg& c = m.cfg;
    std::vector<Shape> v = {{m.qkv_dim(), c.d_model}, {c.d_model, m.q_dim()}, {m.ffn_in_dim(), c.d_model}, {c.d_model, c.d_ff},
                            {c.vocab, c.d_model}};
    if (m.t5()) {
        v.push_back({m.q_dim(), c.d_model});
        v.push_back({c.d_model, m.q_dim()});
    }
    return v;
}

// the GEMM shapes by kind (MegaArgs::count_offset); n_out 0: the model has no such GEMM
std::vector<Shape> kind_shapes(const Model& m) {
    const spec_model_cfg& c = m.cfg;
    std::vector<Shape> v = {{m.qkv_dim(), c.d_model}, {c.d_model, m.q_dim()}, {0, 0}, {0, 0}, {m.ffn_in_dim(), c.d_model},
                            {c.d_model, c.d_ff}, {c.vocab, c.d_model}};
    if (m.t5()) {
        v[2] = {m.q_dim(), c.d_model};
        v[3] = {c.d_model, m.q_dim()};
    }
    return v;
}

bool model_fits(const Model& m, int ctas) {
    const spec_model_cfg& c = m.cfg;
    if (!m.bf16() || (c.arch != SPEC_ARCH_GPT && c.arch != SPEC_ARCH_LLAMA)) return false;
    if (c.vocab % 2 || c.d_model % 8 || c.d_ff % 8 || m.packed.empty() || !m.packed_head) return false;
    int tiles = 0;
    for (const Shape& sh : gemm_shapes(m)) {
        const unsigned long long units = static_cast<unsigned long long>((sh.n_out + 127) / 128) * ((sh.k + 63) / 64);
        if (units * static_cast<unsigned long long>(ctas + 1) >= (1ull << 32)) return false;
        if (max_contributors(static_cast<unsigned>(units), (sh.k + 63) / 64, ctas) > 255) return false;
        tiles += (sh.n_out + 127) / 128;
    }
    return tiles <= kMaxTileCounts;
}

}  // namespace

// Scratch of the persistent pass kernel for the models of a context (those it can serve).
int pass_scratch_init(PassScratch& s, const Model* models, int n_models, std::vector<void*>& allocations) {
    s.ctas = 0;
    int ctas = 0;
    SPEC_TRY_STATUS(resident_ctas<float, 64>(&ctas));
    int other = 0;
    SPEC_TRY_STATUS(resident_ctas<float, 128>(&other));
    ctas = std::min(ctas, other);
    SPEC_TRY_STATUS(resident_ctas<__nv_bfloat16, 64>(&other));
    ctas = std::min(ctas, other);
    SPEC_TRY_STATUS(resident_ctas<__nv_bfloat16, 128>(&other));
    ctas = std::min(ctas, other);
    if (ctas < 1) return SPEC_OK;
    size_t d = 0, q = 0, part = 0, attn = 0;
    bool any = false;
    for (int i = 0; i < n_models; ++i) {
        const Model& m = models[i];
        if (!model_fits(m, ctas)) continue;
        any = true;
        d = std::max<size_t>(d, m.cfg.d_model);
        q = std::max<size_t>(q, m.q_dim());
        attn = std::max<size_t>(attn, static_cast<size_t>(kMaxRows) * m.cfg.n_heads * kMaxSlices * (m.cfg.d_head + 2));
        for (const Shape& sh : gemm_shapes(m)) {
            const int tiles = (sh.n_out + 127) / 128, kbn = (sh.k + 63) / 64;
            part = std::max(part, static_cast<size_t>(tiles) * max_contributors(static_cast<unsigned>(tiles) * kbn, kbn, ctas) * kMaxRows * 128);
        }
    }
    if (!any) return SPEC_OK;
    auto alloc = [&](void** out, size_t bytes) -> int {
        void* p = nullptr;
        const cudaError_t err = cudaMalloc(&p, std::max<size_t>(bytes, 256));
        if (err != cudaSuccess) {
            cudaGetLastError();
            return fail(SPEC_ERR_OOM, "cudaMalloc of %zu bytes failed: %s", bytes, cudaGetErrorString(err));
        }
        allocations.push_back(p);
        *out = p;
        return SPEC_OK;
    };
    for (int i = 0; i < 2; ++i) {
        SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.h[i]), kMaxRows * d * sizeof(float)));
        SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.ssq[i]), ((d + 63) / 64) * kMaxRows * sizeof(float)));
        SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.part[i]), part * sizeof(float)));
    }
    SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.q), kMaxRows * q * sizeof(float)));
    SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.att), kMaxRows * q * sizeof(float)));
    SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.attn_part), attn * sizeof(float)));
    SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.sync), 256));
    SPEC_CUDA_TRY(cudaMemset(s.sync, 0, 256));
    for (int i = 0; i < n_models; ++i) {
        const Model& m = models[i];
        s.layers[i] = nullptr;
        s.tile_counts[i] = nullptr;
        if (!model_fits(m, ctas)) continue;
        {   // parts per tile of every GEMM kind
            std::vector<uint8_t> counts;
            const std::vector<Shape> kinds = kind_shapes(m);
            for (int k = 0; k < 7; ++k) {
                s.count_offset[i][k] = static_cast<int>(counts.size());
                if (kinds[k].n_out == 0) continue;
                const int tiles = (kinds[k].n_out + 127) / 128, kbn = (kinds[k].k + 63) / 64;
                const unsigned units = static_cast<unsigned>(tiles) * kbn;
                for (int t = 0; t < tiles; ++t) {
                    int count = kbn;  // fewer units than CTAs: every unit is a part of its own
                    if (units >= static_cast<unsigned>(ctas))
                        count = cta_of_unit(units, static_cast<unsigned>(t + 1) * kbn - 1u, ctas) -
                                cta_of_unit(units, static_cast<unsigned>(t) * kbn, ctas) + 1;
                    counts.push_back(static_cast<uint8_t>(count));
                }
            }
            s.count_total[i] = static_cast<int>(counts.size());
            SPEC_TRY_STATUS(alloc(&s.tile_counts[i], counts.size()));
            SPEC_CUDA_TRY(cudaMemcpy(s.tile_counts[i], counts.data(), counts.size(), cudaMemcpyHostToDevice));
        }
        std::vector<MegaLayer> host(m.cfg.n_layers);
        for (int l = 0; l < m.cfg.n_layers; ++l) {
            const spec_layer_weights &w = m.layers[l], &pw = m.packed[l];
            MegaLayer& L = host[l];
            L.ln1 = w.ln1;
            L.ln2 = w.ln2;
            L.lnx = w.lnx;
            L.wqkv = static_cast<const __nv_bfloat16*>(pw.wqkv);
            L.wo = static_cast<const __nv_bfloat16*>(pw.wo);
            L.w_in = static_cast<const __nv_bfloat16*>(pw.w_in);
            L.w_out = static_cast<const __nv_bfloat16*>(pw.w_out);
            L.wq_x = static_cast<const __nv_bfloat16*>(pw.wq_x);
            L.wo_x = static_cast<const __nv_bfloat16*>(pw.wo_x);
            L.kv = static_cast<char*>(m.kv) + static_cast<size_t>(l) * m.layer_stride;
            L.cross_kv = m.cross_kv ? static_cast<char*>(m.cross_kv) + static_cast<size_t>(l) * m.cross_stride : nullptr;
        }
        SPEC_TRY_STATUS(alloc(&s.layers[i], host.size() * sizeof(MegaLayer)));
        SPEC_CUDA_TRY(cudaMemcpy(s.layers[i], host.data(), host.size() * sizeof(MegaLayer), cudaMemcpyHostToDevice));
    }
    s.ctas = ctas;
    std::lock_guard<std::mutex> lock(g_sync_mutex);
    g_sync_words.push_back(s.sync);
    return SPEC_OK;
}

bool pass_kernel_serves(const PassScratch& s, const Model& m, int which, int n_rows, int n_logit_rows) {
    return s.ctas > 0 && s.layers[which] != nullptr && n_rows >= 1 && n_rows <= kMaxRows && n_logit_rows <= kMaxRows;
}

int launch_pass(const PassScratch& s, const Model& m, int which, const RowMeta& rows, const PassTables& t, int batch, int m_rows,
                int n_logit_rows, const int32_t* logit_src, const int32_t* logit_dst, float* logits, cudaStream_t stream,
                unsigned long long* trace, int trace_capacity) {
    const spec_model_cfg& c = m.cfg;
    MegaArgs a{};
    a.arch = c.arch;
    a.n_layers = c.n_layers;
    a.d = c.d_model;
    a.n_heads = c.n_heads;
    a.n_kv_heads = c.n_kv_heads;
    a.dh = c.d_head;
    a.d_ff = c.d_ff;
    a.ffn = c.ffn;
    a.vocab = c.vocab;
    a.max_positions = c.max_positions;
    a.emb_bf16 = m.bf16() ? 1 : 0;
    a.eps = c.rms_eps;
    a.tok_emb = m.tok_emb;
    a.pos_emb = m.pos_emb;
    a.ln_f = m.ln_f;
    a.head = static_cast<const __nv_bfloat16*>(m.packed_head);
    a.rope = m.rope_table;
    a.layers = static_cast<const MegaLayer*>(s.layers[which]);
    a.page_table = t.page_table;
    a.pages_per_seq = t.pages_per_seq;
    a.page_size = t.page_size;
    a.src_page_table = t.src_page_table;
    a.src_pages_per_seq = t.src_pages_per_seq;
    a.src_len = t.src_len;
    a.dec_bias = m.dec_bias;
    a.bias_span = t.bias_span;
    a.bias_zero = t.bias_zero;
    a.n_rows = batch * m_rows;
    a.m_rows = m_rows;
    a.batch = batch;
    a.row_token = rows.token;
    a.row_pos = rows.pos;
    a.row_seq = rows.seq;
    a.n_logit_rows = n_logit_rows;
    a.logit_src = logit_src;
    a.logit_dst = logit_dst;
    a.logits = logits;
    for (int i = 0; i < 2; ++i) {
        a.h[i] = s.h[i];
        a.ssq[i] = s.ssq[i];
        a.part[i] = s.part[i];
    }
    a.q = s.q;
    a.att = s.att;
    a.attn_part = s.attn_part;
    a.sync = s.sync;
    a.tile_counts = static_cast<const uint8_t*>(s.tile_counts[which]);
    for (int k = 0; k < 7; ++k) a.count_offset[k] = s.count_offset[which][k];
    a.count_total = s.count_total[which];
    a.trace = trace;
    a.trace_capacity = trace_capacity;
    const bool kv16 = m.kv_elem_bytes == 2;
    if (c.d_head == 64) return kv16 ? launch_variant<__nv_bfloat16, 64>(a, s.ctas, stream) : launch_variant<float, 64>(a, s.ctas, stream);
    return kv16 ? launch_variant<__nv_bfloat16, 128>(a, s.ctas, stream) : launch_variant<float, 128>(a, s.ctas, stream);
}

void pass_scratch_release(PassScratch& s) {
    std::lock_guard<std::mutex> lock(g_sync_mutex);
    g_sync_words.erase(std::remove(g_sync_words.begin(), g_sync_words.end(), s.sync), g_sync_words.end());
    s.ctas = 0;
}

// Non-zero if the pass kernel gave up on a bounded wait since the last call (then the barrier
// words of every context are reset, so that the next launch starts clean).  Synchronises.
int pass_take_error() {
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_mega_error, sizeof(int)) != cudaSuccess) return -1;
    if (v) {
        cudaMemcpyToSymbol(g_mega_error, &zero, sizeof(int));
        std::lock_guard<std::mutex> lock(g_sync_mutex);
        for (unsigned* w : g_sync_words) cudaMemset(w, 0, 256);
    }
    return v;
}

}  // namespace spec
