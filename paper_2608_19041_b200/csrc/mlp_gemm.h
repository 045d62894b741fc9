// GEMM argument block and the fused epilogues shared by the CUDA-core and tensor-core
// GEMM kernels of the MLP.
#pragma once

#include <cuda_runtime.h>

namespace umd {

// C[M,N] = A[M,K] (row-major, lda) x B[K,N] (row-major, ldb), then
//   mode 0 (forward):  y = C + bias[n];  pre[m,n] = y (if pre);  out[m,n] = SiLU(y) + res[m,n]
//   mode 1 (backward): dh = C + res[m,n] + rvec[n];  out[m,n] = dh (if out);
//                      pre[m,n] = dh * SiLU'(pre[m,n]) (if pre)
// res / rvec apply only to columns below res_n / rvec_n when those are non-zero.
struct GemmArgs {
    const float* A; int lda;
    const float* B; int ldb;
    int M, N, K;
    int mode;
    const float* bias;
    const float* res; int ldres; int res_n;
    const float* rvec; int rvec_n;
    float* pre; int ldpre;
    float* out; int ldout;
    // tensor-core path only: pre-split copies of B (hi / lo TF32 parts), K-major [N][K]
    const float* Bt_hi; const float* Bt_lo; int ldbt;
    float* A_hi; float* A_lo;     // scratch [M][K] for the split of A
    int* err;                     // device error word (bounded-wait expiry)
};

__device__ __forceinline__ float sigmoidf_(float x) { return 1.0f / (1.0f + expf(-x)); }
__device__ __forceinline__ float silu(float x) { return x * sigmoidf_(x); }
__device__ __forceinline__ float silu_grad(float x) {
    const float s = sigmoidf_(x);
    return s * (1.0f + x * (1.0f - s));
}

// epilogue for four consecutive columns n..n+3 of row m (n multiple of 4, n < N)
__device__ __forceinline__ void gemm_epilogue4(const GemmArgs& g, int m, int n, float* v) {
    if (g.mode == 0) {
        const float4 b = __ldg(reinterpret_cast<const float4*>(g.bias + n));
        v[0] += b.x; v[1] += b.y; v[2] += b.z; v[3] += b.w;
        if (g.pre) *reinterpret_cast<float4*>(g.pre + (size_t)m * g.ldpre + n) = make_float4(v[0], v[1], v[2], v[3]);
        float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
        if (g.res) r = *reinterpret_cast<const float4*>(g.res + (size_t)m * g.ldres + n);
        *reinterpret_cast<float4*>(g.out + (size_t)m * g.ldout + n) =
            make_float4(silu(v[0]) + r.x, silu(v[1]) + r.y, silu(v[2]) + r.z, silu(v[3]) + r.w);
    } else {
        if (g.res && (g.res_n == 0 || n < g.res_n)) {
            const float4 r = *reinterpret_cast<const float4*>(g.res + (size_t)m * g.ldres + n);
            v[0] += r.x; v[1] += r.y; v[2] += r.z; v[3] += r.w;
        }
        if (g.rvec && (g.rvec_n == 0 || n < g.rvec_n)) {
            const float4 r = __ldg(reinterpret_cast<const float4*>(g.rvec + n));
            v[0] += r.x; v[1] += r.y; v[2] += r.z; v[3] += r.w;
        }
        if (g.out) *reinterpret_cast<float4*>(g.out + (size_t)m * g.ldout + n) = make_float4(v[0], v[1], v[2], v[3]);
        if (g.pre) {
            float4* p = reinterpret_cast<float4*>(g.pre + (size_t)m * g.ldpre + n);
            const float4 y = *p;
            *p = make_float4(v[0] * silu_grad(y.x), v[1] * silu_grad(y.y), v[2] * silu_grad(y.z),
                             v[3] * silu_grad(y.w));
        }
    }
}

cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t st);
bool gemm_tc_supported(const GemmArgs& g);
cudaError_t launch_gemm_tc(const GemmArgs& g, cudaStream_t st);

}  // namespace umd
