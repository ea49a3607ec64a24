// Skinny weight-streaming GEMM on the 5th-generation tensor cores:
//   partial[s][r][n] = sum over the k-range of split s of x[r][k] * W[n][k]
// for a few activation rows against a bf16 weight matrix W [n_out, k] that is
// streamed from HBM exactly once.
//
// The weights take the M side of the MMA ("swap A/B"): a CTA owns 128 output
// features, TMA brings [128 x 64] bf16 weight tiles (128-byte swizzle) into a
// ring of shared-memory stages, and one thread issues tcgen05.mma (kind::f16,
// M = 128, N = padded token count, K = 16) into an fp32 accumulator in tensor
// memory.  The token side carries the activations split into two bf16 terms,
// x = hi + lo, issued as two MMAs into the same accumulator, so that the
// result keeps ~16 mantissa bits of the fp32 activations while the weight
// tile is still read once.  Split-K over the grid keeps every SM streaming for
// matrices with few 128-row tiles; partial sums go to a workspace and are added
// up in a fixed order by reduce_partials_kernel (no atomics, bit-reproducible).
//
// Every wait on an mbarrier is bounded; on expiry the kernel records an error
// code and unwinds (tensor memory is freed on every path).
#include <cuda.h>

#include <map>
#include <mutex>
#include <tuple>

#include "model.cuh"

namespace spec {
namespace {

constexpr int kTileM = 128;     // output features per CTA (MMA M)
constexpr int kTileK = 64;      // bf16 elements per k-block: one 128-byte swizzle row
constexpr int kMmaK = 16;       // K of one tcgen05.mma.kind::f16
constexpr int kThreads = 128;
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ int g_gemm_error;  // first device-side time-out (0 = none)

// ---- PTX wrappers ----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

// Bounded wait for the phase with the given parity; false on time-out.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t limit = kSpinLimit) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t spin = 0; spin < limit; ++spin) {
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

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

// The same with an L2 eviction-priority hint.  The weights are read once per pass: marked
// evict-first they do not push the activations, partial sums and prefetched K,V rows out of L2.
__device__ __forceinline__ void tma_load_2d_hint(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes
// long and 128-byte swizzled: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr & 0x3FFFF) >> 4);   // start address, 16-byte units
    d |= static_cast<uint64_t>(1) << 16;                 // leading byte offset (unused with swizzle)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;         // stride byte offset between 8-row groups
    d |= static_cast<uint64_t>(1) << 46;                 // descriptor version of this architecture
    d |= static_cast<uint64_t>(2) << 61;                 // 128-byte swizzle
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
           (static_cast<uint32_t>(kTileM >> 4) << 24);
}

__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The mbarrier gets one arrival once every MMA issued so far has finished.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
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

template <int N_TOK>
struct Smem {
    // two CTAs per SM up to 128 rows; wider tiles fill the SM alone
    static constexpr int kStages = N_TOK <= 16 ? 5 : N_TOK <= 32 ? 4 : N_TOK <= 80 ? 3 : N_TOK <= 128 ? 2 : 3;
    static constexpr int kABytes = kTileM * kTileK * 2;   // 16 KB
    static constexpr int kBBytes = N_TOK * kTileK * 2;     // one of hi / lo
    static constexpr int kStageBytes = kABytes + 2 * kBBytes;
    static constexpr int kTotal = kStages * kStageBytes + 1024 /* alignment slack */ + 256 /* barriers */;
};

// grid = (tiles of 128 features x token tiles, splits), block = 128.
template <int N_TOK>
__global__ void __launch_bounds__(kThreads)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_hi,
               const __grid_constant__ CUtensorMap map_lo, float* __restrict__ partial, int n_out, int n_rows,
               int k_blocks, int packed, int drill) {
    // drill > 0 (spec_timeout_drill): the producer requests nothing and arms no barrier, and every wait gives
    // up after `drill` polls: the path a lost copy would take, with no copy in flight when the CTA leaves
    using S = Smem<N_TOK>;
    const uint32_t limit = drill > 0 ? static_cast<uint32_t>(drill) : kSpinLimit;
    constexpr int kTmemCols = N_TOK <= 32 ? 32 : N_TOK <= 64 ? 64 : N_TOK <= 128 ? 128 : 256;  // a power of two that holds N_TOK columns
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + S::kStages * S::kStageBytes);
    uint64_t* empty_bar = full_bar + S::kStages;
    uint64_t* acc_bar = empty_bar + S::kStages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_bar + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // (the token tiles of one weight tile are neighbours in launch order: they run side by side and the second
    // finds the weights in L2 - with the token tile as the slowest grid dimension a 224-row launch read every
    // weight from HBM twice)
    const int token_tiles = (n_rows + N_TOK - 1) / N_TOK;
    const int tile = blockIdx.x / token_tiles, split = blockIdx.y, splits = gridDim.y, tok0 = (blockIdx.x % token_tiles) * N_TOK;
    const int kb0 = static_cast<int>(static_cast<long long>(k_blocks) * split / splits);
    const int kb1 = static_cast<int>(static_cast<long long>(k_blocks) * (split + 1) / splits);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::kStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(acc_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // one warp owns the tensor-memory allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTmemCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_acc = *tmem_slot;
    bool ok = true;

    if (warp == 0 && lane == 0 && drill <= 0) {
        // ---- producer: weights and both activation terms of one k-block per stage ----
        // The weights do not depend on the kernel before this one: the first
        // ring of weight tiles is already streaming while that kernel finishes.
        // Weight tile of k-block kb: in the row-major matrix the box at (kb*64, tile*128);
        // in the tile-major copy the 128 consecutive 128-byte rows of tile (tile, kb).
        uint64_t stream_once;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(stream_once));
        auto load_w = [&](void* dst, int kb, uint64_t* bar) {
            if (packed) tma_load_2d_hint(dst, &map_w, 0, (tile * k_blocks + kb) * kTileM, bar, stream_once);
            else tma_load_2d_hint(dst, &map_w, kb * kTileK, tile * kTileM, bar, stream_once);
        };
        const int total = kb1 - kb0;
        const int ahead = min(total, S::kStages);
        for (int it = 0; it < ahead; ++it) {
            mbar_expect_tx(&full_bar[it], S::kStageBytes);
            load_w(smem + it * S::kStageBytes, kb0 + it, &full_bar[it]);
        }
        pdl_wait();  // the activations are written by the previous kernel
        for (int it = 0; it < ahead; ++it) {
            uint8_t* stage = smem + it * S::kStageBytes;
            tma_load_2d(stage + S::kABytes, &map_hi, (kb0 + it) * kTileK, tok0, &full_bar[it]);
            tma_load_2d(stage + S::kABytes + S::kBBytes, &map_lo, (kb0 + it) * kTileK, tok0, &full_bar[it]);
        }
        for (int it = ahead; it < total; ++it) {
            const int kb = kb0 + it, s = it % S::kStages;
            if (!mbar_wait(&empty_bar[s], ((it / S::kStages) - 1) & 1, limit)) { ok = false; break; }
            uint8_t* stage = smem + s * S::kStageBytes;
            mbar_expect_tx(&full_bar[s], S::kStageBytes);
            load_w(stage, kb, &full_bar[s]);
            tma_load_2d(stage + S::kABytes, &map_hi, kb * kTileK, tok0, &full_bar[s]);
            tma_load_2d(stage + S::kABytes + S::kBBytes, &map_lo, kb * kTileK, tok0, &full_bar[s]);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer ----
        constexpr uint32_t idesc = instr_desc(N_TOK);
        for (int kb = kb0; kb < kb1; ++kb) {
            const int it = kb - kb0, s = it % S::kStages;
            if (!mbar_wait(&full_bar[s], (it / S::kStages) & 1, limit)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_addr = smem_u32(smem + s * S::kStageBytes);
            const uint64_t a_desc = smem_desc_sw128(a_addr);
            const uint64_t hi_desc = smem_desc_sw128(a_addr + S::kABytes);
            const uint64_t lo_desc = smem_desc_sw128(a_addr + S::kABytes + S::kBBytes);
#pragma unroll
            for (int k = 0; k < kTileK / kMmaK; ++k) {
                const uint64_t step = static_cast<uint64_t>((k * kMmaK * 2) >> 4);  // 32 bytes along K, in 16-byte units
                mma_f16(tmem_acc, a_desc + step, hi_desc + step, idesc, (it > 0 || k > 0) ? 1u : 0u);
                mma_f16(tmem_acc, a_desc + step, lo_desc + step, idesc, 1u);
            }
            mma_commit(&empty_bar[s]);  // the stage may be refilled once these MMAs have read it
        }
        if (ok) mma_commit(acc_bar);  // accumulator complete
    }
    __syncwarp();
    pdl_wait();  // (already satisfied for the producer) nothing below may overtake the previous kernel
    // The next kernel is released here, when this CTA's copies and MMAs have been issued, not at the top: the small
    // kernel that follows a GEMM has no prologue worth starting early, and its CTAs arriving while the stream is at
    // full rate cost more than they gain (measured per block: 97M shape 28.8 -> 27.0 us, 7B 94.8 -> 94.5).
    pdl_trigger();

    // ---- epilogue: all four warps, warp w reads accumulator lanes 32w .. 32w+31 ----
    if (kb1 > kb0) {  // one lane polls, the warp takes one decision (the tensor-memory loads below are warp-wide)
        int done = 1;
        if (lane == 0) done = mbar_wait(acc_bar, 0, limit) ? 1 : 0;
        done = __shfl_sync(0xffffffffu, done, 0);
        if (done) mbar_wait(acc_bar, 0, 1);  // (complete: every lane observes the phase)
        else ok = false;
    }
    ok = __all_sync(0xffffffffu, ok);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int feature = tile * kTileM + warp * 32 + lane;
    float* out = partial + (static_cast<size_t>(split) * n_rows) * n_out + feature;
    if (ok) {
#pragma unroll
        for (int c0 = 0; c0 < N_TOK; c0 += 16) {
            if (tok0 + c0 < n_rows) {  // uniform across the warp
                float v[16];
                if (kb1 > kb0) {
                    tmem_ld16(tmem_acc + (static_cast<uint32_t>(warp * 32) << 16) + c0, v);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = 0.0f;
                }
                if (feature < n_out) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int r = tok0 + c0 + i;
                        if (r < n_rows) out[static_cast<size_t>(r) * n_out] = v[i];
                    }
                }
            }
        }
    } else {
        atomicCAS(&g_gemm_error, 0, 1 + warp);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(kTmemCols));
    }
}

// Tile-major copy of a row-major bf16 matrix W [n_out, k]: tile (t, kb) holds rows
// t*128 .. t*128+127, columns kb*64 .. kb*64+63 as 128 consecutive 128-byte rows,
// tiles ordered (t, kb); rows and columns past the matrix are zero.  Inside a row
// the eight 16-byte chunks are stored in the order of the 128-byte shared-memory
// swizzle (chunk c of row r sits at position c ^ (r & 7)), so that a plain copy of
// the 16 KB tile to a 1024-byte aligned address is the layout the MMA's operand
// descriptor expects.  One 16-byte vector (8 elements) per thread.
__global__ void pack_weight_kernel(const __nv_bfloat16* __restrict__ w, int n_out, int k, int k_blocks, size_t vectors,
                                   __nv_bfloat16* __restrict__ out) {
    for (size_t v = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; v < vectors;
         v += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const size_t tile_index = v / (kTileM * kTileK / 8);
        const int within = static_cast<int>(v % (kTileM * kTileK / 8));
        const int r = within / (kTileK / 8), c8 = within % (kTileK / 8);
        const int row = static_cast<int>(tile_index / k_blocks) * kTileM + r;
        const int col = static_cast<int>(tile_index % k_blocks) * kTileK + (c8 ^ (r & 7)) * 8;
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (row < n_out && col < k) val = *reinterpret_cast<const uint4*>(w + static_cast<size_t>(row) * k + col);
        *reinterpret_cast<uint4*>(out + v * 8) = val;
    }
}

// x (fp32) -> hi = bf16(x), lo = bf16(x - hi); grid-stride, 4 elements per thread
__global__ void split_bf16_kernel(const float* __restrict__ x, size_t n, __nv_bfloat16* __restrict__ hi,
                                  __nv_bfloat16* __restrict__ lo) {
    pdl_trigger();
    pdl_wait();
    for (size_t i = (blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x) * 4; i < n;
         i += static_cast<size_t>(gridDim.x) * blockDim.x * 4) {
        const float4 v = *reinterpret_cast<const float4*>(x + i);
        const float f[4] = {v.x, v.y, v.z, v.w};
        __nv_bfloat16 h[4], l[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            h[j] = __float2bfloat16_rn(f[j]);
            l[j] = __float2bfloat16_rn(f[j] - __bfloat162float(h[j]));
        }
        *reinterpret_cast<uint2*>(hi + i) = *reinterpret_cast<const uint2*>(h);
        *reinterpret_cast<uint2*>(lo + i) = *reinterpret_cast<const uint2*>(l);
    }
}

// y[dst(r)][n] = sum_s partial[s][r][n] (+ residual[r][n]), splits added in index order
__global__ void reduce_partials_kernel(const float* __restrict__ partial, int splits, int n_rows, int n_out,
                                       const float* residual, const int32_t* __restrict__ dst_rows, float* y) {
    pdl_trigger();
    pdl_wait();
    const size_t total = static_cast<size_t>(n_rows) * n_out;
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        float acc = 0.0f;
        for (int s0 = 0; s0 < splits; s0 += 8) {  // eight loads in flight at a time, added in split order
            float p[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) p[k] = s0 + k < splits ? partial[static_cast<size_t>(s0 + k) * total + i] : 0.0f;
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (s0 + k < splits) acc = (s0 + k == 0) ? p[k] : acc + p[k];
        }
        if (residual) acc += residual[i];
        const size_t r = i / n_out, n = i % n_out;
        y[(dst_rows ? static_cast<size_t>(dst_rows[r]) : r) * n_out + n] = acc;
    }
}

// ---- host side ----------------------------------------------------------------
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
    static EncodeFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeFn>(p);
    }();
    return fn;
}

// A bf16 matrix [rows, cols] row-major, fetched in boxes of [box_rows, 64], with the 128-byte
// swizzle applied on the way in unless the data is stored swizzled already.
int make_map(const void* base, int rows, int cols, int box_rows, bool swizzle, CUtensorMap* out) {
    EncodeFn fn = encode_fn();
    if (!fn) return fail(SPEC_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
    const cuuint32_t box[2] = {kTileK, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t elem[2] = {1, 1};
    const CUresult res = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (res != CUDA_SUCCESS) return fail(SPEC_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", static_cast<int>(res));
    return SPEC_OK;
}

struct MapKey {
    const void* base;
    int rows, cols, box_rows, swizzle;
    bool operator<(const MapKey& o) const {
        return std::tie(base, rows, cols, box_rows, swizzle) < std::tie(o.base, o.rows, o.cols, o.box_rows, o.swizzle);
    }
};

// Tensor maps are pure functions of (address, shape, box): cached process-wide.
int cached_map(const void* base, int rows, int cols, int box_rows, bool swizzle, CUtensorMap* out) {
    static std::mutex mu;
    static std::map<MapKey, CUtensorMap> cache;
    std::lock_guard<std::mutex> lock(mu);
    const MapKey key{base, rows, cols, box_rows, swizzle ? 1 : 0};
    auto it = cache.find(key);
    if (it == cache.end()) {
        CUtensorMap m;
        const int status = make_map(base, rows, cols, box_rows, swizzle, &m);
        if (status != SPEC_OK) return status;
        it = cache.emplace(key, m).first;
    }
    *out = it->second;
    return SPEC_OK;
}

template <int N_TOK>
int launch_tc(const CUtensorMap& mw, const CUtensorMap& mhi, const CUtensorMap& mlo, float* partial, int n_out,
              int n_rows, int k_blocks, int splits, int packed, cudaStream_t stream, int drill = 0) {
    static std::atomic<unsigned long long> configured{0};
    if (first_use_on_this_device(configured))
        SPEC_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<N_TOK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           Smem<N_TOK>::kTotal));
    const dim3 grid(((n_out + kTileM - 1) / kTileM) * ((n_rows + N_TOK - 1) / N_TOK), splits, 1);
    return launch_pdl(gemm_tc_kernel<N_TOK>, grid, dim3(kThreads), Smem<N_TOK>::kTotal, stream, mw, mhi, mlo, partial,
                      n_out, n_rows, k_blocks, packed, drill);
}

}  // namespace

// Rows per CTA (the MMA's N): the smallest multiple of 16 that holds the rows, so that up to 192 rows
// the weights are streamed once and no MMA column is padding (the tensor-core work and the activation
// tiles that every CTA re-reads grow with the padded row count: an 80-row tile for 80 rows instead of
// a 96-row one took 8 % off the pass at batch 16 x 5 rows); more rows take several tiles, neighbours in
// launch order (measured: a 256-row tile leaves room for two pipeline stages only and is slower than
// two passes of 128).
int gemm_tc_token_tile(int n_rows) {
    if (n_rows <= 16) return 16;
    if (n_rows <= 32) return 32;
    if (n_rows <= 48) return 48;
    if (n_rows <= 64) return 64;
    if (n_rows <= 80) return 80;
    if (n_rows <= 96) return 96;
    if (n_rows <= 112) return 112;
    if (n_rows <= 128) return 128;
    if (n_rows <= 160) return 160;
    if (n_rows <= 192) return 192;
    if (n_rows <= 240) return 80;  // three tiles of 80 (three stages each) beat two of 112 or 128: 274 / 302 / 313 us
                                   // per 7B block at 224 rows
    return 128;
}

int cached_f16_rows_map(const void* base, unsigned long long rows, int cols, CUtensorMap* out) {
    static std::mutex mu;
    static std::map<std::tuple<const void*, unsigned long long, int>, CUtensorMap> cache;
    std::lock_guard<std::mutex> lock(mu);
    const auto key = std::make_tuple(base, rows, cols);
    auto it = cache.find(key);
    if (it == cache.end()) {
        EncodeFn fn = encode_fn();
        if (!fn) return fail(SPEC_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
        const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
        const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
        const cuuint32_t box[2] = {64, 32};
        const cuuint32_t elem[2] = {1, 1};
        CUtensorMap m;
        const CUresult res = fn(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (res != CUDA_SUCCESS) return fail(SPEC_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", static_cast<int>(res));
        it = cache.emplace(key, m).first;
    }
    *out = it->second;
    return SPEC_OK;
}

// Split-K factor: the smallest one that fills the last wave of CTAs to 85 %, with
// at least two k-blocks per split.
int gemm_tc_splits(int n_out, int k, int n_rows) {
    const int n_tok = gemm_tc_token_tile(n_rows);
    const int tiles = ((n_out + kTileM - 1) / kTileM) * ((n_rows + n_tok - 1) / n_tok);
    const int k_blocks = (k + kTileK - 1) / kTileK;
    const int resident = 148 * (n_tok <= 128 ? 2 : 1);
    const int max_splits = std::max(1, std::min(k_blocks / 2, 16));
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= max_splits; ++s) {
        const int ctas = tiles * s;
        const int waves = (ctas + resident - 1) / resident;
        const double eff = static_cast<double>(ctas) / (static_cast<double>(waves) * resident);
        if (eff > best_eff + 1e-9) {
            best_eff = eff;
            best = s;
        }
        if (eff >= 0.85) return s;
    }
    return best;
}

size_t gemm_tc_partial_elems(int n_out, int k, int n_rows) {
    return static_cast<size_t>(gemm_tc_splits(n_out, k, n_rows)) * n_rows * n_out;
}

size_t packed_weight_elems(int n_out, int k) {
    return static_cast<size_t>((n_out + kTileM - 1) / kTileM) * ((k + kTileK - 1) / kTileK) * kTileM * kTileK;
}

int launch_pack_weight(const void* w, int n_out, int k, void* out, cudaStream_t stream) {
    if (k % 8 != 0) return fail(SPEC_ERR_BAD_CONFIG, "pack: inner dimension %d is not a multiple of 8", k);
    const size_t vectors = packed_weight_elems(n_out, k) / 8;
    const int blocks = static_cast<int>(std::min<size_t>((vectors + 255) / 256, 148 * 16));
    pack_weight_kernel<<<blocks, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(w), n_out, k, (k + kTileK - 1) / kTileK,
                                                   vectors, static_cast<__nv_bfloat16*>(out));
    SPEC_CUDA_TRY(cudaGetLastError());
    return SPEC_OK;
}

int launch_split_bf16(const float* x, size_t n, __nv_bfloat16* hi, __nv_bfloat16* lo, cudaStream_t stream) {
    const int blocks = static_cast<int>(std::min<size_t>((n / 4 + 255) / 256, 148 * 8));
    return launch_pdl(split_bf16_kernel, dim3(std::max(blocks, 1)), dim3(256), 0, stream, x, n, hi, lo);
}

// partial[s][r][n] for x already split into hi + lo (both [hi_rows, k] bf16, the
// first n_rows rows valid); s < gemm_tc_splits(n_out, k, n_rows).
int launch_gemm_tc_partials(const __nv_bfloat16* hi, const __nv_bfloat16* lo, int hi_rows, const void* w, bool packed,
                            int n_rows, int n_out, int k, float* partial, cudaStream_t stream) {
    if (n_rows <= 0) return SPEC_OK;
    if (k % 8 != 0) return fail(SPEC_ERR_BAD_CONFIG, "gemm: inner dimension %d is not a multiple of 8", k);
    const int n_tok = gemm_tc_token_tile(n_rows);
    const int splits = gemm_tc_splits(n_out, k, n_rows);
    const int k_blocks = (k + kTileK - 1) / kTileK;
    CUtensorMap mw, mhi, mlo;
    const int tiles = (n_out + kTileM - 1) / kTileM;
    // tile-major weights are one long [tiles * k_blocks * 128, 64] matrix of 128-byte rows
    // (stored swizzled already: copied as they are)
    int status = packed ? cached_map(w, tiles * k_blocks * kTileM, kTileK, kTileM, false, &mw)
                        : cached_map(w, n_out, k, kTileM, true, &mw);
    if (status == SPEC_OK) status = cached_map(hi, hi_rows, k, n_tok, true, &mhi);
    if (status == SPEC_OK) status = cached_map(lo, hi_rows, k, n_tok, true, &mlo);
    if (status != SPEC_OK) return status;
    const int pk = packed ? 1 : 0;
    switch (n_tok) {
        case 16: return launch_tc<16>(mw, mhi, mlo, partial, n_out, n_rows, k_blocks, splits, pk, stream);
        case 32: return launch_tc<32>(mw, mhi, mlo, partial, n_out, n_rows, k_blocks, splits, pk, stream);
        case 48: return launch_tc<48>(mw, mhi, mlo, partial, n_out, n_rows, k_blocks, splits, pk, stream);
        case 64: return launch_tc<64>(mw, mhi, mlo, partial, n_out, n_rows, k_blocks, splits, pk, stream);
        case 80: return launch_tc<80>(mw, mhi, mlo, partial, n_out, n_rows, k_blocks, splits, pk, stream);
        case 96: return launch_tc<96>(mw, mhi, mlo, partial, n_out, n_rows, k_blocks, splits, pk, stream);
        case 112: return launch_tc<112>(mw, mhi, mlo, partial, n_out, n_rows, k_blocks, splits, pk, stream);
        case 128: return launch_tc<128>(mw, mhi, mlo, partial, n_out, n_rows, k_blocks, splits, pk, stream);
        case 160: return launch_tc<160>(mw, mhi, mlo, partial, n_out, n_rows, k_blocks, splits, pk, stream);
        default: return launch_tc<192>(mw, mhi, mlo, partial, n_out, n_rows, k_blocks, splits, pk, stream);
    }
}

// y[dst(r)] = x[r] . W^T (+ residual[r]): the partial sums, then their reduction.
int launch_gemm_tc(const __nv_bfloat16* hi, const __nv_bfloat16* lo, int hi_rows, const void* w, bool packed,
                   const float* residual, const int32_t* dst_rows, int n_rows, int n_out, int k, float* partial,
                   float* y, cudaStream_t stream) {
    if (n_rows <= 0) return SPEC_OK;
    const int status = launch_gemm_tc_partials(hi, lo, hi_rows, w, packed, n_rows, n_out, k, partial, stream);
    if (status != SPEC_OK) return status;
    const int splits = gemm_tc_splits(n_out, k, n_rows);
    const size_t total = static_cast<size_t>(n_rows) * n_out;
    const int blocks = static_cast<int>(std::min<size_t>((total + 255) / 256, 148 * 8));
    return launch_pdl(reduce_partials_kernel, dim3(blocks), dim3(256), 0, stream, static_cast<const float*>(partial),
                      splits, n_rows, n_out, residual, dst_rows, y);
}

// Non-zero if a tensor-core GEMM gave up on a bounded wait since the last call.
int gemm_tc_take_error() {
    int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_gemm_error, sizeof(int)) != cudaSuccess) return -1;
    if (v) cudaMemcpyToSymbol(g_gemm_error, &zero, sizeof(int));
    return v;
}

}  // namespace spec

// ---- C ABI: one linear layer, for tests and benchmarks of the GEMM kernels ----
namespace {
size_t align256(size_t v) { return (v + 255) / 256 * 256; }
int padded_rows(int rows) { return (rows + 255) / 256 * 256; }
}  // namespace

extern "C" size_t spec_linear_workspace_bytes(int rows, int n_out, int k) {
    if (rows < 1 || n_out < 1 || k < 1) return 0;
    const size_t split_bytes = align256(static_cast<size_t>(padded_rows(rows)) * k * 2);
    return 2 * split_bytes + align256(spec::gemm_tc_partial_elems(n_out, k, rows) * sizeof(float)) + 256;
}

extern "C" int spec_linear(const float* x, const void* w, int w_dtype, int rows, int n_out, int k, int path, float* y,
                           void* workspace, size_t workspace_bytes, void* stream) {
    using namespace spec;
    if (!x || !w || !y) return fail(SPEC_ERR_BAD_ARG, "spec_linear: null pointer");
    if (rows < 1 || n_out < 1 || k < 8 || k % 8) return fail(SPEC_ERR_BAD_ARG, "spec_linear: rows=%d n_out=%d k=%d (k must be a multiple of 8)", rows, n_out, k);
    if (w_dtype != SPEC_DTYPE_FP32 && w_dtype != SPEC_DTYPE_BF16) return fail(SPEC_ERR_BAD_ARG, "spec_linear: dtype %d", w_dtype);
    if (path < 0 || path > 3) return fail(SPEC_ERR_BAD_ARG, "spec_linear: path %d", path);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool tensor = w_dtype == SPEC_DTYPE_BF16 && path != 1;
    if (path >= 2 && w_dtype != SPEC_DTYPE_BF16) return fail(SPEC_ERR_BAD_CONFIG, "spec_linear: the tensor-core path needs bf16 weights");
    if (!tensor) return launch_gemm_rows(x, w, w_dtype == SPEC_DTYPE_BF16, nullptr, nullptr, rows, n_out, k, y, st);
    if (!workspace || workspace_bytes < spec_linear_workspace_bytes(rows, n_out, k) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return fail(SPEC_ERR_BAD_ARG, "spec_linear: workspace missing, too small or not 256-byte aligned");
    const size_t split_bytes = align256(static_cast<size_t>(padded_rows(rows)) * k * 2);
    char* base = static_cast<char*>(workspace);
    __nv_bfloat16* hi = reinterpret_cast<__nv_bfloat16*>(base);
    __nv_bfloat16* lo = reinterpret_cast<__nv_bfloat16*>(base + split_bytes);
    float* partial = reinterpret_cast<float*>(base + 2 * split_bytes);
    // rows past `rows` of the padded tile are read by the MMA (their results are discarded): keep them finite
    SPEC_CUDA_TRY(cudaMemsetAsync(base, 0, 2 * split_bytes, st));
    int status = launch_split_bf16(x, static_cast<size_t>(rows) * k, hi, lo, st);
    if (status != SPEC_OK) return status;
    return launch_gemm_tc(hi, lo, padded_rows(rows), w, path == 3, nullptr, nullptr, rows, n_out, k, partial, y, st);
}

extern "C" int spec_linear_partials(const float* x, const void* w_packed, int rows, int n_out, int k, int split_input,
                                    void* workspace, size_t workspace_bytes, float** partial, int* splits, void* stream) {
    using namespace spec;
    if (!w_packed || (split_input && !x)) return fail(SPEC_ERR_BAD_ARG, "spec_linear_partials: null pointer");
    if (rows < 1 || n_out < 1 || k < 8 || k % 8) return fail(SPEC_ERR_BAD_ARG, "spec_linear_partials: rows=%d n_out=%d k=%d (k must be a multiple of 8)", rows, n_out, k);
    if (!workspace || workspace_bytes < spec_linear_workspace_bytes(rows, n_out, k) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return fail(SPEC_ERR_BAD_ARG, "spec_linear_partials: workspace missing, too small or not 256-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t split_bytes = align256(static_cast<size_t>(padded_rows(rows)) * k * 2);
    char* base = static_cast<char*>(workspace);
    __nv_bfloat16* hi = reinterpret_cast<__nv_bfloat16*>(base);
    __nv_bfloat16* lo = reinterpret_cast<__nv_bfloat16*>(base + split_bytes);
    float* sums = reinterpret_cast<float*>(base + 2 * split_bytes);
    if (split_input) {
        SPEC_CUDA_TRY(cudaMemsetAsync(base, 0, 2 * split_bytes, st));
        const int status = launch_split_bf16(x, static_cast<size_t>(rows) * k, hi, lo, st);
        if (status != SPEC_OK) return status;
    }
    if (partial) *partial = sums;
    if (splits) *splits = gemm_tc_splits(n_out, k, rows);
    return launch_gemm_tc_partials(hi, lo, padded_rows(rows), w_packed, true, rows, n_out, k, sums, st);
}

extern "C" size_t spec_packed_weight_bytes(int n_out, int k) {
    if (n_out < 1 || k < 1) return 0;
    return spec::packed_weight_elems(n_out, k) * 2;
}

extern "C" int spec_pack_weight(const void* w, int n_out, int k, void* packed, void* stream) {
    using namespace spec;
    if (!w || !packed || n_out < 1 || k < 8 || k % 8) return fail(SPEC_ERR_BAD_ARG, "spec_pack_weight: bad argument");
    return launch_pack_weight(w, n_out, k, packed, static_cast<cudaStream_t>(stream));
}

// ---- C ABI: a bounded wait that runs out, on purpose ----
namespace {
__device__ __align__(1024) unsigned char g_drill_tile[128 * 64 * 2];  // what the drill's tensor maps point at (never read)
}

extern "C" int spec_timeout_drill(void* stream) {
    using namespace spec;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    void* base = nullptr;
    SPEC_CUDA_TRY(cudaGetSymbolAddress(&base, g_drill_tile));
    CUtensorMap mw, mx;
    int status = cached_map(base, 128, 64, 128, true, &mw);
    if (status == SPEC_OK) status = cached_map(base, 16, 64, 16, true, &mx);
    if (status != SPEC_OK) return status;
    SPEC_CUDA_TRY(cudaStreamSynchronize(st));
    gemm_tc_take_error();  // (whatever was pending is not this drill's)
    // one CTA, one k-block, nothing requested: the MMA issuer's wait and the epilogue's wait run out after 4096 polls
    status = launch_tc<16>(mw, mx, mx, reinterpret_cast<float*>(base), 128, 1, 1, 1, 0, st, 4096);
    if (status != SPEC_OK) return status;
    SPEC_CUDA_TRY(cudaStreamSynchronize(st));
    const int code = gemm_tc_take_error();
    if (code > 0) return fail(SPEC_ERR_DEVICE_TIMEOUT, "drill: the kernel gave up on a bounded wait (code %d), freed its tensor memory and returned", code);
    return fail(SPEC_ERR_CUDA, "drill: the kernel did not report the wait that should have run out");
}

extern "C" int spec_device_error(void) {
    const int gemm = spec::gemm_tc_take_error(), pass = spec::pass_take_error(), attn = spec::attention_take_error();
    return gemm ? gemm : pass ? pass : attn;
}
