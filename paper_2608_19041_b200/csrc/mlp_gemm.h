// GEMM argument block and the fused epilogues shared by the CUDA-core and tensor-core
// GEMM kernels of the MLP.
#pragma once

#include <cuda_runtime.h>

#include <cstdint>

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
    float* A_hi; float* A_lo;     // [M][K] TF32 split of A: filled by the caller if a_presplit, else by a split kernel
    int a_presplit;
    // TF32 split of the value the next GEMM of the chain consumes (mode 0: out, mode 1: the new
    // pre), written by the epilogue with row pitch ldnxt when non-null
    float* nxt_hi; float* nxt_lo; int ldnxt;
    // tensor-core path, mode 0, last layer: instead of storing out (and pre), the epilogue dots
    // each output row with head_w over the CTA's columns, head_part[m * head_parts + column
    // tile], and, when nxt_hi is set, leaves the split of head_w[n] * SiLU'(y[m,n]) there (the
    // seed of the backward pass)
    const float* head_w; float* head_part; int head_parts;
    // tensor-core path, mode 0 / head: per-row bias bias_rows[row_type[m] * N + n] instead of bias[n]
    const float* bias_rows; const int* row_type;
    int lda_split;                // row pitch of A_hi / A_lo (0 = K)
    int variant;                  // tensor-core kernel: 3 = one tile per CTA, otherwise the persistent one
    int* err;                     // device error word (bounded-wait expiry)
};

__device__ __forceinline__ float sigmoidf_(float x) { return 1.0f / (1.0f + expf(-x)); }
__device__ __forceinline__ float silu(float x) { return x * sigmoidf_(x); }
__device__ __forceinline__ float silu_grad(float x) {
    const float s = sigmoidf_(x);
    return s * (1.0f + x * (1.0f - s));
}

// x = hi + lo with hi = round-to-nearest TF32 of x and lo = round-to-nearest TF32 of (x - hi)
__device__ __forceinline__ void split_tf32(float x, float& hi, float& lo) {
    uint32_t hb, lb;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hb) : "f"(x));
    hi = __uint_as_float(hb);
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(lb) : "f"(x - hi));
    lo = __uint_as_float(lb);
}
__device__ __forceinline__ void store_split4(float* hi, float* lo, size_t off, float4 v) {
    float4 h, l;
    split_tf32(v.x, h.x, l.x); split_tf32(v.y, h.y, l.y); split_tf32(v.z, h.z, l.z); split_tf32(v.w, h.w, l.w);
    *reinterpret_cast<float4*>(hi + off) = h;
    *reinterpret_cast<float4*>(lo + off) = l;
}

// epilogue for four consecutive columns n..n+3 of row m (n multiple of 4, n < N)
__device__ __forceinline__ void gemm_epilogue4(const GemmArgs& g, int m, int n, float* v) {
    if (g.mode == 0) {
        const float4 b = __ldg(reinterpret_cast<const float4*>(g.bias + n));
        v[0] += b.x; v[1] += b.y; v[2] += b.z; v[3] += b.w;
        if (g.pre) *reinterpret_cast<float4*>(g.pre + (size_t)m * g.ldpre + n) = make_float4(v[0], v[1], v[2], v[3]);
        float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
        if (g.res) r = *reinterpret_cast<const float4*>(g.res + (size_t)m * g.ldres + n);
        const float4 o = make_float4(silu(v[0]) + r.x, silu(v[1]) + r.y, silu(v[2]) + r.z, silu(v[3]) + r.w);
        *reinterpret_cast<float4*>(g.out + (size_t)m * g.ldout + n) = o;
        if (g.nxt_hi) store_split4(g.nxt_hi, g.nxt_lo, (size_t)m * g.ldnxt + n, o);
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
            const float4 o = make_float4(v[0] * silu_grad(y.x), v[1] * silu_grad(y.y), v[2] * silu_grad(y.z),
                                         v[3] * silu_grad(y.w));
            *p = o;
            if (g.nxt_hi) store_split4(g.nxt_hi, g.nxt_lo, (size_t)m * g.ldnxt + n, o);
        }
    }
}

cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t st);
bool gemm_tc_supported(const GemmArgs& g);
bool gemm_tc_available();      // the driver's tensor-map encoder could be resolved
int gemm_tc_pick_variant(int M, int N, int requested);   // 2 (persistent) or 3 (one tile per CTA) for path 2
constexpr int kGemmTcBN = 128;  // column tile of the tensor-core GEMM
// partial head sums per row that the fused last-layer epilogue of a variant leaves
inline int gemm_tc_head_parts(int N, int variant) { return (variant == 3 ? 1 : 2) * ((N + kGemmTcBN - 1) / kGemmTcBN); }
cudaError_t launch_gemm_tc(const GemmArgs& g, cudaStream_t st);

}  // namespace umd
