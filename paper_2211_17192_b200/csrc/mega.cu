// One forward pass over a few rows as ONE persistent kernel (an option of the context:
// spec_runtime_cfg::pass_kernel; the chain of kernels in engine.cu is the default, see below).
//
// A decoding pass over gamma + 1 rows is a stream of weights (Section 3.4: the rows share
// one read of every matrix) interrupted by short dependent steps: normalisation, rotary
// positions, attention, the activation.  Here the whole pass is one cooperative kernel with
// one CTA per SM:
//
//   * warp 0 streams weight tiles with bulk copies into a ring of shared-memory stages.  It
//     depends on nothing but free stages, so it runs ahead through every dependent step
//     and across GEMM boundaries: while the other warps sit in a grid-wide barrier or in
//     the attention, the ring keeps filling with the next matrix.
//   * every GEMM is cut "stream-K" fashion: the (128-feature tile, 64-column block) units
//     of a matrix, in the tile-major order in which they are stored, are dealt out in
//     equal contiguous runs, one per CTA, so that every SM streams the same number of
//     bytes of every matrix whatever its shape.  A run covers parts of one to three
//     tiles; each part is accumulated in tensor memory (tcgen05.mma, M 128 x N 16).  A
//     tile with one part is finished by its CTA; otherwise the parts go to global memory
//     and the CTA that writes the last one (a counter per tile) adds them up in CTA order.
//   * the activation operand of a GEMM is built by its consumer: eight warps of every CTA
//     form the 16 x 64 block that goes with a weight tile from the step before (residual
//     stream times the norm gain; attention output; gated activation of the FFN-in
//     rows), split it into two bf16 terms and store it in the MMA's swizzled layout.
//     RMSNorm's row scale is applied by whoever consumes the GEMM (W (s x) = s (W x)); the
//     sums of squares come from the CTAs that finish the tiles of the residual stream.
//   * between dependent steps there is one grid-wide barrier (a counter in global memory
//     that is never reset); steps per block: qkv GEMM | rotary + K,V append | attention |
//     slice merge | out-projection | FFN-in | FFN-out; at the end the LM head, whose
//     finished tiles are the logits.
//
// Every wait (mbarrier, grid barrier) is bounded; on expiry the kernel records an error,
// tells the other CTAs, waits for its own copies in flight, frees its tensor memory and
// returns.
//
// Measured on a B200 (7B-shaped blocks, 3 rows, 1024 cached tokens): the weight stream alone
// runs at the HBM copy rate, but every step pays about two microseconds of barrier and two
// to four of start-up and finish (operand load, part count, part re-read: each a round
// trip to L2), seven times per block: 109 us per block against 88 us for the kernel chain,
// and more on small models whose steps move almost no bytes.  Hence an option, not the
// default.
#include <algorithm>
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
    static constexpr int kAbort = kTmemSlot + 4;                      // abort flag, the barrier's verdict, the epilogue's "last part" flag
    static constexpr int kScale = kAbort + 12;                        // row scales [16]
    static constexpr int kRowPos = kScale + 16 * 4;                   // per row: position, sequence slot, (per sequence) key count, token, logits row
    static constexpr int kShare = (kRowPos + 5 * 16 * 4 + 15) / 16 * 16;  // attention states, one per worker warp
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

// (past L1: for values that another SM wrote during this phase)
__device__ __forceinline__ float ld_cg_f1(const float* p) {
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
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
    const int32_t *logit_src, *logit_dst;  // (distinct source rows)
    float* logits;
    // scratch
    float* h;         // residual stream [16][d]
    float* ssq[2];    // sums of squares of the stream's rows per 32-column group [d / 32][16], used in turn
    float* part[2];   // partial sums of the GEMMs' tiles, used in turn
    float* out;       // output of the GEMM before (projection rows, FFN-in rows) [16][n_out]
    float* att;       // attention output [16][n_heads * dh]
    float* attn_part; // per key slice: (max, sum, accumulator) of every (row, head)
    unsigned* ticket[2];  // per tile: parts written so far (back to zero once the tile is finished)
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
    switch (gemm_kind(a, g)) {
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

// The most CTAs that contribute to one tile: a tile's kbn units meet runs of per = units / P
// (or one more) units.
__host__ __device__ inline int max_contributors(unsigned units, int kbn, int P) {
    const int per = static_cast<int>(units / static_cast<unsigned>(P));
    if (per == 0) return kbn;  // fewer units than CTAs: every unit may be another CTA's
    return static_cast<int>((kbn + per - 2) / per + 1);
}

__device__ __forceinline__ float gelu_tanh(float x) {
    const float k = 0.7978845608028654f;
    return 0.5f * x * (1.0f + tanhf(k * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float silu(float x) { return x / (1.0f + expf(-x)); }

// RMSNorm's scale of a row from the sums of squares of its 32-column groups (every warp that needs
// it evaluates the same expression on the same values): this lane's share, four loads in flight.
__device__ __forceinline__ float row_ssq_share(const float* ssq, int groups, int row, int lane) {
    float s = 0.0f;
    for (int g0 = lane; g0 < groups; g0 += 128) {
        float v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = ld_f1(ssq + min(g0 + 32 * i, groups - 1) * kMaxRows + row);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (g0 + 32 * i < groups) s += v[i];
    }
    return s;
}
__device__ __forceinline__ float row_scale(const float* ssq, int groups, int row, int d, float eps, int lane) {
    return rsqrtf(warp_sum(row_ssq_share(ssq, groups, row, lane)) / static_cast<float>(d) + eps);
}

// Per-thread view of the kernel's shared state.
struct Cta {
    uint8_t* ring;
    uint64_t *wfull, *bfull, *empty, *acc_full, *acc_empty;
    volatile int* abort_flag;
    volatile int* verdict;  // written by one thread inside the grid barrier: 1 = carry on, 0 = unwind
    volatile int* last;     // written by one epilogue thread: 1 = this CTA wrote a tile's last part
    float* scale;
    const int *row_pos, *row_seq, *seq_keys, *row_tok, *row_logit;  // shared-memory copies: per row / per sequence of the pass
    const uint8_t* counts;  // shared-memory copy of MegaArgs::tile_counts
    uint32_t tmem;
    int c, P;         // this CTA, CTAs
    unsigned n;       // units this CTA has been through (all GEMMs so far)
    int items;        // accumulator parts this CTA has been through
    int barriers;     // grid barriers this CTA has been through
};

enum Source { kSrcNorm, kSrcPlain, kSrcAct };
enum Sink { kSinkRows, kSinkStream, kSinkLogits };

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
    int k_total;        // inner dimension of this GEMM
    const float* gain;  // norm: the gain; the row scale is left to whoever consumes the GEMM
    const float* rows;  // norm: the residual stream [16][k_total]; plain: fp32 rows [16][k_total];
                        // act: the FFN-in rows [16][d_ff or 2 d_ff]
    const float* ssq;   // act: the sums of squares that go with the FFN-in GEMM's operand
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

template <int SRC>
__device__ __forceinline__ void build_block(const MegaArgs& a, const Cta& cta, const BuildCtx& b, uint8_t* stage, int kb, int lane) {
    const int col = kb * 64 + 2 * lane;
    const bool live = col < b.k_total;  // (columns past the matrix meet zero weights: they must be finite, so zero)
    const bool gated = SRC == kSrcAct && a.ffn != SPEC_FFN_GELU;
    const int width = SRC == kSrcAct ? (gated ? 2 * a.d_ff : a.d_ff) : b.k_total;
    float2 gain = make_float2(1.f, 1.f);
    if (SRC == kSrcNorm && live) gain = ld_f2(b.gain + col);
    for (int r0 = 0; r0 < a.n_rows; r0 += kRowBatch) {
        float2 v[kRowBatch], up[kRowBatch];
        // ---- every load of these rows is requested before anything is used ----
#pragma unroll
        for (int i = 0; i < kRowBatch; ++i) {
            const int r = min(r0 + i, a.n_rows - 1);
            v[i] = up[i] = make_float2(0.f, 0.f);
            if (live) {
                v[i] = ld_f2(b.rows + static_cast<size_t>(r) * width + col);
                if (gated) up[i] = ld_f2(b.rows + static_cast<size_t>(r) * width + a.d_ff + col);
            }
        }
#pragma unroll
        for (int i = 0; i < kRowBatch; ++i) {
            const int r = r0 + i;
            if (r >= a.n_rows) break;
            float2 x = v[i];
            if (SRC == kSrcNorm) {
                x.x *= gain.x;
                x.y *= gain.y;
            } else if (SRC == kSrcAct && live) {  // the FFN's activation, RMSNorm's scale of the FFN-in operand applied here
                const float s = cta.scale[r];
                if (!gated) x = make_float2(gelu_tanh(s * x.x), gelu_tanh(s * x.y));
                else if (a.ffn == SPEC_FFN_SWIGLU) x = make_float2(silu(s * x.x) * (s * up[i].x), silu(s * x.y) * (s * up[i].y));
                else x = make_float2(gelu_tanh(s * x.x) * (s * up[i].x), gelu_tanh(s * x.y) * (s * up[i].y));
            }
            store_pair(stage, r, lane, x.x, x.y);
        }
    }
}

// ---- what becomes of a GEMM's output tiles ------------------------------------------------
struct SinkCtx {
    Sink sink;
    float* rows;          // rows: [16][n_out]
    float* ssq_out;       // stream: sums of squares of the updated stream, per 32-column group
    const float* ssq_in;  // logits: the sums of squares that go with the LM head's operand
};

// ---- one GEMM: every role of the CTA but the weight producer ---------------------------
// Roles.  The ring is two interleaved half-rings: the units this CTA goes through are numbered
// n = 0, 1, 2, ... over the whole pass; unit n uses stage n % kStages (kStages is even), so even
// units use even stages and odd units odd stages.  Issuer X (warp 1 + X) takes the units of
// parity X, in order, into accumulator X of the part; builder warp 8 + b takes the units with
// n % 8 == b, in order.  Every mbarrier of a stage is therefore waited on by threads that go
// through that stage's phases in order (a wait by parity cannot tell a phase from the one two
// before it, so nobody may get two phases ahead of a barrier).
//
// A tile's parts (one per CTA whose run meets the tile) go to global memory; the CTA that
// writes the last one (a counter per tile tells) adds them up in CTA order, so the sum does
// not depend on who does it, and passes the tile on: rows for the next step, the residual
// stream with its sums of squares, or logits.
template <typename Prefetch>
__device__ void gemm_step(const MegaArgs& a, Cta& cta, int g, const BuildCtx& b, const SinkCtx& o, Prefetch prefetch) {
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
        // ---- epilogue: warp w holds features 32 (w & 3) .. + 31 of the tile, one per lane ----
        const int quarter = warp & 3;
        float* parts = a.part[g & 1];
        unsigned* ticket = a.ticket[g & 1];
        const uint8_t* counts = cta.counts + a.count_offset[gemm_kind(a, g)];
        const int jmax = max_contributors(gd.units, gd.kbn, cta.P);
        const int groups_d = (a.d + 31) / 32;
        if (o.sink == kSinkLogits) {  // RMSNorm's scale of every row, from the LM head's operand
            for (int r = quarter; r < a.n_rows; r += 4) {
                const float s = row_scale(o.ssq_in, groups_d, r, a.d, a.eps, lane);
                if (lane == 0) cta.scale[r] = s;
            }
            named_sync<4, 128>();
        }
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
            const uint32_t lanes = static_cast<uint32_t>(quarter * 32) << 16;
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
            const int feature = quarter * 32 + lane, col = t * 128 + feature;
            const int n_parts_of_tile = counts[t];
            if (n_parts_of_tile > 1) {
                // this CTA's part to memory; whoever writes a tile's last part adds them all up
                const int j = gd.units < static_cast<unsigned>(cta.P)
                                  ? static_cast<int>(u0 % gd.kbn)
                                  : cta.c - cta_of_unit(gd.units, static_cast<unsigned>(t) * gd.kbn, cta.P);
                float* tile_parts = parts + static_cast<size_t>(t) * jmax * (kMaxRows * 128);
                float* dst = tile_parts + static_cast<size_t>(j) * (kMaxRows * 128) + feature;
#pragma unroll
                for (int r = 0; r < kMaxRows; ++r)
                    if (r < a.n_rows) dst[r * 128] = v[r];
                named_sync<4, 128>();  // (the four warps' stores come before the count below: it releases them)
                if (warp == 4 && lane == 0) {
                    unsigned before;
                    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], %2;" : "=r"(before) : "l"(ticket + t), "r"(1u) : "memory");
                    const int last = before == static_cast<unsigned>(n_parts_of_tile - 1) ? 1 : 0;
                    if (last) ticket[t] = 0u;  // (nobody touches it again before the next GEMM that uses this array)
                    *cta.last = last;
                }
                named_sync<4, 128>();
                if (!*cta.last) continue;
                // the parts in CTA order, four rows' loads in flight at a time (read past L1: other SMs wrote them)
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    if (q4 * 4 >= a.n_rows) break;
                    for (int j0 = 0; j0 < n_parts_of_tile; j0 += 8) {
                        float p[4][8];
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int jj = 0; jj < 8; ++jj)
                                p[i][jj] = ld_cg_f1(tile_parts + static_cast<size_t>(min(j0 + jj, n_parts_of_tile - 1)) * (kMaxRows * 128) +
                                                    min(q4 * 4 + i, a.n_rows - 1) * 128 + feature);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float acc = j0 == 0 ? p[i][0] : v[q4 * 4 + i] + p[i][0];
#pragma unroll
                            for (int jj = 1; jj < 8; ++jj)
                                if (j0 + jj < n_parts_of_tile) acc += p[i][jj];
                            v[q4 * 4 + i] = acc;
                        }
                    }
                }
            }
            // ---- the finished tile ----
            if (o.sink == kSinkRows) {
                if (col < gd.n_out) {
#pragma unroll
                    for (int r = 0; r < kMaxRows; ++r)
                        if (r < a.n_rows) o.rows[static_cast<size_t>(r) * gd.n_out + col] = v[r];
                }
            } else if (o.sink == kSinkStream) {  // h += tile; the new rows' sums of squares per 32-column group
                float hv[16];
#pragma unroll
                for (int r = 0; r < kMaxRows; ++r)
                    hv[r] = (r < a.n_rows && col < a.d) ? ld_cg_f1(a.h + static_cast<size_t>(r) * a.d + col) : 0.0f;
#pragma unroll
                for (int r = 0; r < kMaxRows; ++r) {
                    if (r < a.n_rows) {
                        const float x = col < a.d ? hv[r] + v[r] : 0.0f;
                        if (col < a.d) a.h[static_cast<size_t>(r) * a.d + col] = x;
                        const float ss = warp_sum(x * x);
                        if (lane == 0 && t * 4 + quarter < groups_d) o.ssq_out[(t * 4 + quarter) * kMaxRows + r] = ss;
                    }
                }
            } else {  // logits of the rows that have a destination
                if (col < gd.n_out) {
#pragma unroll
                    for (int r = 0; r < kMaxRows; ++r) {
                        if (r < a.n_rows) {
                            const int dst = cta.row_logit[r];
                            if (dst >= 0) a.logits[static_cast<size_t>(dst) * a.vocab + col] = v[r] * cta.scale[r];
                        }
                    }
                }
            }
        }
    } else if (warp == 3) {
        prefetch(lane);  // (the one warp without a role in a GEMM)
    } else {
        // ---- builders: a unit's block is announced once its weight tile has landed too, so that the
        // issuers wait on one barrier per unit ----
        const unsigned bi = warp - 8;
        if (b.src == kSrcAct) {  // RMSNorm's scale of every row, from the FFN-in GEMM's operand
            for (int r = bi; r < a.n_rows; r += kBuilders) {
                const float s = row_scale(b.ssq, (a.d + 31) / 32, r, a.d, a.eps, lane);
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
            const int kb = static_cast<int>(u % gd.kbn);
            switch (b.src) {
                case kSrcNorm: build_block<kSrcNorm>(a, cta, b, stage, kb, lane); break;
                case kSrcPlain: build_block<kSrcPlain>(a, cta, b, stage, kb, lane); break;
                default: build_block<kSrcAct>(a, cta, b, stage, kb, lane); break;
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

// ---- the residual stream's first value: token (+ position) embeddings, and its sums of squares ----
__device__ void embed_step(const MegaArgs& a, const Cta& cta, float* ssq_out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp < 2) return;
    const int groups = (a.d + 31) / 32;  // a warp per 32 columns
    for (int i = cta.c + cta.P * (warp - 2); i < groups; i += cta.P * kWorkers) {
        const int col = i * 32 + lane;
        for (int r = 0; r < a.n_rows; ++r) {
            float x = 0.0f;
            if (col < a.d) {
                const int t = min(max(cta.row_tok[r], 0), a.vocab - 1);
                const size_t at = static_cast<size_t>(t) * a.d + col;
                x = a.emb_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(a.tok_emb)[at]) : static_cast<const float*>(a.tok_emb)[at];
                if (a.arch == SPEC_ARCH_GPT) {
                    const int p = min(max(cta.row_pos[r], 0), a.max_positions - 1);
                    const size_t pat = static_cast<size_t>(p) * a.d + col;
                    x += a.emb_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(a.pos_emb)[pat]) : static_cast<const float*>(a.pos_emb)[pat];
                }
                a.h[static_cast<size_t>(r) * a.d + col] = x;
            }
            const float ss = warp_sum(x * x);
            if (lane == 0) ssq_out[i * kMaxRows + r] = ss;
        }
    }
}

// ---- rotary positions, K,V append, q rows: finishes the projection whose rows are in a.out -----
// n_kv_heads = 0: queries only (cross-attention).
template <typename KV>
__device__ void qkv_step(const MegaArgs& a, const Cta& cta, const float* ssq, int n_heads, int n_kv_heads, bool rope, KV* kv_layer) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp < 2) return;
    const int heads = n_heads + 2 * n_kv_heads, half = a.dh / 2;
    const int width = heads * a.dh;
    const int groups_d = (a.d + 31) / 32;
    const int units = a.n_rows * heads;
    // unit i -> CTA i % P, worker (i / P) % kWorkers
    for (int i = cta.c + cta.P * (warp - 2); i < units; i += cta.P * kWorkers) {
        const int r = i / heads, head = i % heads;
        const int p = cta.row_pos[r];
        const bool is_q = head < n_heads, is_k = !is_q && head < n_heads + n_kv_heads;
        // lane owns the pairs (j, j + 1) of the first half and the same of the second half; every
        // load of the unit (sums of squares, values, rotation, page) is requested before any is used
        const int j = 2 * lane;
        const bool live = j < half;
        const int col = head * a.dh + j;
        const float sq = row_ssq_share(ssq, groups_d, r, lane);
        float2 x1 = make_float2(0.f, 0.f), x2 = x1;
        float4 cs = make_float4(1.f, 0.f, 1.f, 0.f);
        int page = 0;
        if (live) {
            x1 = ld_f2(a.out + static_cast<size_t>(r) * width + col);
            x2 = ld_f2(a.out + static_cast<size_t>(r) * width + col + half);
            if (rope && p >= 0 && (is_q || is_k)) cs = *reinterpret_cast<const float4*>(a.rope + static_cast<size_t>(p) * half + j);  // (cos, sin) x 2
            if (!is_q && p >= 0) page = a.page_table[cta.row_seq[r] * a.pages_per_seq + p / a.page_size];
        }
        const float s = rsqrtf(warp_sum(sq) / static_cast<float>(a.d) + a.eps);
        if (!live) continue;
        x1.x *= s; x1.y *= s; x2.x *= s; x2.y *= s;
        const float2 y1 = make_float2(x1.x * cs.x - x2.x * cs.y, x1.y * cs.z - x2.y * cs.w);
        const float2 y2 = make_float2(x2.x * cs.x + x1.x * cs.y, x2.y * cs.z + x1.y * cs.w);
        if (is_q) {  // q stays in place (rotated, scaled) for the attention
            float* dst = a.out + static_cast<size_t>(r) * width + col;
            *reinterpret_cast<float2*>(dst) = y1;
            *reinterpret_cast<float2*>(dst + half) = y2;
        } else if (p >= 0) {
            const int kv_head = is_k ? head - n_heads : head - n_heads - n_kv_heads;
            const size_t block = (static_cast<size_t>(page) * 2 + (is_k ? 0 : 1)) * n_kv_heads + kv_head;
            KV* dst = kv_layer + (block * a.page_size + p % a.page_size) * a.dh + j;
            dst[0] = to_cached<KV>(y1.x);
            dst[1] = to_cached<KV>(y1.y);
            dst[half] = to_cached<KV>(y2.x);
            dst[half + 1] = to_cached<KV>(y2.y);
        }
    }
}

// ---- attention: (sequence, KV head, key slice) pieces dealt out to the CTAs ----------------
template <typename KV, int DH>
__device__ void attention_step(const MegaArgs& a, const Cta& cta, const float* q, int q_stride, const KV* kv_layer,
                               const int32_t* page_table, int pages_per_seq, const int32_t* kv_len, const float* bias, int slices,
                               float (*share)[DH + 2]) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp < 2) return;
    const int queries = (a.n_heads / a.n_kv_heads) * a.m_rows;
    const int ks = queries * 2 <= kWorkers ? kWorkers / queries : 1;
    const float scale = rsqrtf(static_cast<float>(DH));
    const int pieces = a.batch * a.n_kv_heads * slices;
    for (int u = cta.c; u < pieces; u += cta.P) {
        const int slice = u % slices, kv_head = (u / slices) % a.n_kv_heads, b = u / (slices * a.n_kv_heads);
        attend_slice<KV, DH, NamedSync<3, kWorkers * 32>>(q, q_stride, a.row_pos, a.row_seq, a.m_rows, a.n_heads, a.n_kv_heads,
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
    cta.last = cta.abort_flag + 2;
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
    {   // what every step needs of the rows, in shared memory
        int* rows_sh = reinterpret_cast<int*>(smem + Smem::kRowPos);
        cta.row_pos = rows_sh;
        cta.row_seq = rows_sh + 16;
        cta.seq_keys = rows_sh + 32;
        cta.row_tok = rows_sh + 48;
        cta.row_logit = rows_sh + 64;
        if (threadIdx.x < 16) {
            const int r = threadIdx.x;
            rows_sh[r] = r < a.n_rows ? a.row_pos[r] : -1;
            rows_sh[16 + r] = r < a.n_rows ? a.row_seq[r] : 0;
            int keys = 0;  // of sequence r of the pass: its rows' largest position + 1
            if (r < a.batch)
                for (int j = 0; j < a.m_rows; ++j) keys = max(keys, a.row_pos[r * a.m_rows + j] + 1);
            rows_sh[32 + r] = keys;
            rows_sh[48 + r] = r < a.n_rows ? a.row_token[r] : 0;
            // the logits row that pass row r feeds (none: -1)
            rows_sh[64 + r] = !a.logit_src && r < a.n_logit_rows ? (a.logit_dst ? a.logit_dst[r] : r) : -1;
        }
        uint8_t* counts_sh = smem + Smem::kCounts;
        for (int i = threadIdx.x; i < a.count_total; i += kThreads) counts_sh[i] = a.tile_counts[i];
        cta.counts = counts_sh;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    cta.tmem = *tmem_slot;
    if (a.logit_src && threadIdx.x < a.n_logit_rows) {
        const int src = a.logit_src[threadIdx.x];
        if (src >= 0 && src < 16) reinterpret_cast<int*>(smem + Smem::kRowPos)[64 + src] = a.logit_dst ? a.logit_dst[threadIdx.x] : threadIdx.x;
    }
    __syncthreads();
    if (a.trace && cta.c == 0 && threadIdx.x == 32 && a.trace_capacity > 1) {  // (CTAs; start of the pass)
        a.trace[0] = gridDim.x;
        a.trace[1] = global_ns();
    }

    if (warp == 0) {
        if (lane == 0) produce_weights(a, cta);
        __syncwarp();
    } else {
        const int per = gemms_per_layer(a);
        const int q_dim = a.n_heads * DH, qkv_dim = (a.n_heads + 2 * a.n_kv_heads) * DH;
        int hb = 0;  // which copy of the stream's sums of squares is current
        // the longest key set of any sequence of the pass
        int longest = 0;
        for (int b = 0; b < a.batch; ++b) longest = max(longest, cta.seq_keys[b]);
        const int slices = choose_slices(a, cta.P, longest);
        embed_step(a, cta, a.ssq[0]);
        bool ok = grid_sync(a, cta);
        for (int l = 0; l < a.n_layers && ok; ++l) {
            const MegaLayer& L = a.layers[l];
            int g = l * per;
            // ---- projection of the normalised stream ----
            gemm_step(a, cta, g, BuildCtx{kSrcNorm, a.d, L.ln1, a.h, nullptr}, SinkCtx{kSinkRows, a.out, nullptr, nullptr},
                      [&](int ln) { prefetch_keys<KV, DH>(a, cta, static_cast<const KV*>(L.kv), slices, ln); });
            if (!(ok = grid_sync(a, cta))) break;
            qkv_step<KV>(a, cta, a.ssq[hb], a.n_heads, a.n_kv_heads, a.arch == SPEC_ARCH_LLAMA, static_cast<KV*>(L.kv));
            if (!(ok = grid_sync(a, cta))) break;
            attention_step<KV, DH>(a, cta, a.out, qkv_dim, static_cast<const KV*>(L.kv), a.page_table, a.pages_per_seq, nullptr,
                                   a.arch == SPEC_ARCH_T5 ? a.dec_bias : nullptr, slices, share);
            if (!(ok = grid_sync(a, cta))) break;
            combine_step<DH>(a, cta, slices);
            if (!(ok = grid_sync(a, cta))) break;
            // ---- out-projection into the stream ----
            ++g;
            gemm_step(a, cta, g, BuildCtx{kSrcPlain, q_dim, nullptr, a.att, nullptr}, SinkCtx{kSinkStream, nullptr, a.ssq[hb ^ 1], nullptr},
                      [](int) {});
            hb ^= 1;
            if (!(ok = grid_sync(a, cta))) break;
            // ---- FFN-in on the normalised stream ----
            ++g;
            gemm_step(a, cta, g, BuildCtx{kSrcNorm, a.d, L.ln2, a.h, nullptr}, SinkCtx{kSinkRows, a.out, nullptr, nullptr}, [](int) {});
            if (!(ok = grid_sync(a, cta))) break;
            // ---- FFN-out on the activation of the FFN-in rows, into the stream ----
            ++g;
            gemm_step(a, cta, g, BuildCtx{kSrcAct, a.d_ff, nullptr, a.out, a.ssq[hb]}, SinkCtx{kSinkStream, nullptr, a.ssq[hb ^ 1], nullptr},
                      [](int) {});
            hb ^= 1;
            if (!(ok = grid_sync(a, cta))) break;
        }
        if (ok && a.n_logit_rows > 0)  // ---- final norm and LM head: the finished tiles are the logits ----
            gemm_step(a, cta, per * a.n_layers, BuildCtx{kSrcNorm, a.d, a.ln_f, a.h, nullptr},
                      SinkCtx{kSinkLogits, nullptr, nullptr, a.ssq[hb]}, [](int) {});
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

struct LiveScratch {
    unsigned *sync, *ticket[2];
    int ticket_count;
};
std::mutex g_sync_mutex;
std::vector<LiveScratch> g_live;  // the barrier words and part counters of every live context

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
    SPEC_TRY_STATUS(resident_ctas<__half, 64>(&other));
    ctas = std::min(ctas, other);
    SPEC_TRY_STATUS(resident_ctas<__half, 128>(&other));
    ctas = std::min(ctas, other);
    if (ctas < 1) return SPEC_OK;
    size_t d = 0, q = 0, part = 0, attn = 0, out = 0, tiles_most = 0;
    bool any = false;
    for (int i = 0; i < n_models; ++i) {
        const Model& m = models[i];
        if (!model_fits(m, ctas)) continue;
        any = true;
        d = std::max<size_t>(d, m.cfg.d_model);
        q = std::max<size_t>(q, m.q_dim());
        out = std::max<size_t>({out, static_cast<size_t>(m.qkv_dim()), static_cast<size_t>(m.ffn_in_dim()), static_cast<size_t>(m.q_dim())});
        attn = std::max<size_t>(attn, static_cast<size_t>(kMaxRows) * m.cfg.n_heads * kMaxSlices * (m.cfg.d_head + 2));
        for (const Shape& sh : gemm_shapes(m)) {
            const int tiles = (sh.n_out + 127) / 128, kbn = (sh.k + 63) / 64;
            tiles_most = std::max<size_t>(tiles_most, tiles);
            part = std::max(part, static_cast<size_t>(tiles) * max_contributors(static_cast<unsigned>(tiles) * kbn, kbn, ctas) * kMaxRows * 128);
        }
    }
    if (!any) return SPEC_OK;
    auto alloc = [&](void** out_ptr, size_t bytes) -> int {
        void* p = nullptr;
        const cudaError_t err = cudaMalloc(&p, std::max<size_t>(bytes, 256));
        if (err != cudaSuccess) {
            cudaGetLastError();
            return fail(SPEC_ERR_OOM, "cudaMalloc of %zu bytes failed: %s", bytes, cudaGetErrorString(err));
        }
        allocations.push_back(p);
        *out_ptr = p;
        return SPEC_OK;
    };
    SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.h), kMaxRows * d * sizeof(float)));
    for (int i = 0; i < 2; ++i) {
        SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.ssq[i]), ((d + 31) / 32) * kMaxRows * sizeof(float)));
        SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.part[i]), part * sizeof(float)));
        SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.ticket[i]), tiles_most * sizeof(unsigned)));
        SPEC_CUDA_TRY(cudaMemset(s.ticket[i], 0, tiles_most * sizeof(unsigned)));
    }
    s.ticket_count = static_cast<int>(tiles_most);
    SPEC_TRY_STATUS(alloc(reinterpret_cast<void**>(&s.out), kMaxRows * out * sizeof(float)));
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
    g_live.push_back(LiveScratch{s.sync, {s.ticket[0], s.ticket[1]}, s.ticket_count});
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
    a.h = s.h;
    for (int i = 0; i < 2; ++i) {
        a.ssq[i] = s.ssq[i];
        a.part[i] = s.part[i];
        a.ticket[i] = s.ticket[i];
    }
    a.out = s.out;
    a.att = s.att;
    a.attn_part = s.attn_part;
    a.sync = s.sync;
    a.tile_counts = static_cast<const uint8_t*>(s.tile_counts[which]);
    for (int k = 0; k < 7; ++k) a.count_offset[k] = s.count_offset[which][k];
    a.count_total = s.count_total[which];
    a.trace = trace;
    a.trace_capacity = trace_capacity;
    if (m.kv_dtype == SPEC_DTYPE_FP16)
        return c.d_head == 64 ? launch_variant<__half, 64>(a, s.ctas, stream) : launch_variant<__half, 128>(a, s.ctas, stream);
    if (m.kv_dtype == SPEC_DTYPE_BF16)
        return c.d_head == 64 ? launch_variant<__nv_bfloat16, 64>(a, s.ctas, stream) : launch_variant<__nv_bfloat16, 128>(a, s.ctas, stream);
    return c.d_head == 64 ? launch_variant<float, 64>(a, s.ctas, stream) : launch_variant<float, 128>(a, s.ctas, stream);
}

void pass_scratch_release(PassScratch& s) {
    std::lock_guard<std::mutex> lock(g_sync_mutex);
    g_live.erase(std::remove_if(g_live.begin(), g_live.end(), [&](const LiveScratch& l) { return l.sync == s.sync; }), g_live.end());
    s.ctas = 0;
}

// Non-zero if the pass kernel gave up on a bounded wait since the last call (then the barrier
// words and part counters of every context are reset, so that the next launch starts clean).
// Synchronises.
int pass_take_error() {
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_mega_error, sizeof(int)) != cudaSuccess) return -1;
    if (v) {
        cudaMemcpyToSymbol(g_mega_error, &zero, sizeof(int));
        std::lock_guard<std::mutex> lock(g_sync_mutex);
        for (const LiveScratch& l : g_live) {
            cudaMemset(l.sync, 0, 256);
            for (int i = 0; i < 2; ++i) cudaMemset(l.ticket[i], 0, l.ticket_count * sizeof(unsigned));
        }
    }
    return v;
}

}  // namespace spec
