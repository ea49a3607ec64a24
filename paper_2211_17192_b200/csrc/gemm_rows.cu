// Skinny weight-streaming GEMM on the FMA pipes: y[r] = x[r] . W^T for a few
// activation rows against an [n_out, k] weight matrix that is read exactly once
// per row tile.  This is the plain-ALU path: the only path for fp32 models
// (whose 1e-4 relative logit tolerance rules out tf32) and the reference the
// tensor-core path is checked against for bf16 weights.  Activations stay fp32.
//
// A warp owns NPW output features.  Each lane walks k in 16-byte steps of the
// weight rows (8 bf16 or 4 fp32 elements), so a warp-level load covers 512
// contiguous bytes of one weight row; the matching activation values come from
// L1 (every warp of the CTA reads the same few rows).  Partial sums are reduced
// across the lanes at the end.
#include "model.cuh"

namespace spec {
namespace {

constexpr int kGemmWarps = 8;

template <typename WT>
struct WVec;  // 16 bytes of weights, widened to fp32

template <>
struct WVec<float> {
    static constexpr int kElems = 4;
    float v[4];
    __device__ __forceinline__ void load(const float* p) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
};

template <>
struct WVec<__nv_bfloat16> {
    static constexpr int kElems = 8;
    float v[8];
    __device__ __forceinline__ void load(const __nv_bfloat16* p) {
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {  // bf16 -> fp32 is a 16-bit shift
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

// grid = (ceil(n_out / (kGemmWarps * NPW)), ceil(n_rows / MT)), block = 32 * kGemmWarps
template <typename WT, int MT, int NPW>
__global__ void __launch_bounds__(32 * kGemmWarps)
gemm_rows_kernel(const float* __restrict__ x, const WT* __restrict__ w, const float* residual,
                 const int32_t* __restrict__ dst_rows, int n_rows, int n_out, int k, float* y) {
    constexpr int E = WVec<WT>::kElems;
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n0 = (blockIdx.x * kGemmWarps + warp) * NPW;
    const int r0 = blockIdx.y * MT;
    if (n0 >= n_out) return;

    float acc[NPW][MT];
#pragma unroll
    for (int j = 0; j < NPW; ++j)
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[j][m] = 0.0f;

    for (int kk = lane * E; kk < k; kk += 32 * E) {
        WVec<WT> wv[NPW];
#pragma unroll
        for (int j = 0; j < NPW; ++j) {
            const int n = min(n0 + j, n_out - 1);
            wv[j].load(w + static_cast<size_t>(n) * k + kk);
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const int r = min(r0 + m, n_rows - 1);
            float xv[E];
#pragma unroll
            for (int e = 0; e < E; e += 4) {
                const float4 t = __ldg(reinterpret_cast<const float4*>(x + static_cast<size_t>(r) * k + kk + e));
                xv[e] = t.x; xv[e + 1] = t.y; xv[e + 2] = t.z; xv[e + 3] = t.w;
            }
#pragma unroll
            for (int j = 0; j < NPW; ++j)
#pragma unroll
                for (int e = 0; e < E; ++e) acc[j][m] = fmaf(wv[j].v[e], xv[e], acc[j][m]);
        }
    }
#pragma unroll
    for (int j = 0; j < NPW; ++j)
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const float s = warp_sum(acc[j][m]);
            const int n = n0 + j, r = r0 + m;
            if (lane == 0 && n < n_out && r < n_rows) {
                const size_t dst = static_cast<size_t>(dst_rows ? dst_rows[r] : r) * n_out + n;
                y[dst] = residual ? s + residual[static_cast<size_t>(r) * n_out + n] : s;
            }
        }
}

template <typename WT, int MT, int NPW>
int launch(const float* x, const void* w, const float* residual, const int32_t* dst_rows, int n_rows, int n_out,
            int k, float* y, cudaStream_t stream) {
    const dim3 grid((n_out + kGemmWarps * NPW - 1) / (kGemmWarps * NPW), (n_rows + MT - 1) / MT);
    return launch_pdl(gemm_rows_kernel<WT, MT, NPW>, grid, dim3(32 * kGemmWarps), 0, stream, x,
                      static_cast<const WT*>(w), residual, dst_rows, n_rows, n_out, k, y);
}

template <typename WT>
int dispatch(const float* x, const void* w, const float* residual, const int32_t* dst_rows, int n_rows, int n_out,
              int k, float* y, cudaStream_t stream) {
    if (n_rows <= 2) return launch<WT, 2, 4>(x, w, residual, dst_rows, n_rows, n_out, k, y, stream);
    if (n_rows <= 4) return launch<WT, 4, 4>(x, w, residual, dst_rows, n_rows, n_out, k, y, stream);
    if (n_rows <= 8) return launch<WT, 8, 4>(x, w, residual, dst_rows, n_rows, n_out, k, y, stream);
    return launch<WT, 16, 2>(x, w, residual, dst_rows, n_rows, n_out, k, y, stream);
}

}  // namespace

int launch_gemm_rows(const float* x, const void* w, bool w_bf16, const float* residual, const int32_t* dst_rows,
                     int n_rows, int n_out, int k, float* y, cudaStream_t stream) {
    if (n_rows <= 0) return SPEC_OK;
    if (k % 8 != 0) return fail(SPEC_ERR_BAD_CONFIG, "gemm: inner dimension %d is not a multiple of 8", k);
    if (w_bf16) return dispatch<__nv_bfloat16>(x, w, residual, dst_rows, n_rows, n_out, k, y, stream);
    return dispatch<float>(x, w, residual, dst_rows, n_rows, n_out, k, y, stream);
}

}  // namespace spec
