// GEMM argument block and the fused epilogues shared by the CUDA-core and tensor-core
// GEMM kernels of the MLP.
#pragma once

#include <cuda_fp16.h>
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
    // tensor-core path, mode 0: the residual given as a half-precision split (row pitch ldres)
    // instead of res: the split the previous layer left for this layer's A operand
    const __half* res_hi; const __half* res_lo;
    const float* rvec; int rvec_n;
    float* pre; int ldpre;
    float* out; int ldout;
    // tensor-core path only: pre-split copies of B (hi / lo half-precision parts, scaled by a power
    // of two, see acc_scale), K-major [N][K]
    const __half* Bt_hi; const __half* Bt_lo; int ldbt;
    __half* A_hi; __half* A_lo;   // [M][K] half-precision split of A: filled by the caller if a_presplit, else by a split kernel
    int a_presplit;
    // half-precision split of the value the next GEMM of the chain consumes (mode 0: out, mode 1:
    // the new pre), written by the epilogue with row pitch ldnxt when non-null
    __half* nxt_hi; __half* nxt_lo; int ldnxt;
    // tensor-core path: powers of two that keep the low parts of the splits out of the subnormal
    // range of half precision.  The accumulator is multiplied by acc_scale (the inverse of the
    // weights' scale) before anything else; the backward chain carries gradients multiplied by a
    // common factor, so rvec is multiplied by rvec_scale (that factor) on its way in, `out` by
    // out_scale on its way out (its inverse at the end of the chain), and the seed the last
    // forward layer leaves for the backward pass by seed_scale.  The CUDA-core path sets all to 1.
    float acc_scale, rvec_scale, out_scale, seed_scale;
    // tensor-core path, mode 0, last layer: instead of storing out (and pre), the epilogue dots
    // each output row with head_w over the CTA's columns, head_part[m * head_parts + column
    // tile], and, when nxt_hi is set, leaves the split of head_w[n] * SiLU'(y[m,n]) there (the
    // seed of the backward pass)
    const float* head_w; float* head_part; int head_parts;
    // tensor-core path, mode 0 / head: per-row bias bias_rows[row_type[m] * N + n] instead of bias[n]
    const float* bias_rows; const int* row_type;
    int lda_split;                // row pitch of A_hi / A_lo (0 = K)
    int variant;                  // tensor-core kernel: 3 = one tile per CTA, 4 = two-CTA persistent, otherwise the one-CTA persistent one
    int* err;                     // device error word (bounded-wait expiry)
    // tensor-core path: polls before a wait on the operand pipeline gives up (0 = the default, a
    // fraction of a second), and a diagnostic that makes every CTA leave its k-th operand stage
    // unloaded (0 = off), so that the give-up path can be exercised: the wait for that stage then
    // runs out, the kernel returns with kErrPipelineTimeout set, and nothing hangs
    int spin_limit, test_skip_kblock;
};

// Logistic function from the hardware base-2 exponential and reciprocal (two transcendental
// instructions instead of some twenty for expf and a correctly rounded division, in every element
// of every GEMM epilogue).  The exponent -x log2(e) is rounded once, which leaves a relative error
// of about 4e-8 |x| in exp(-x); the logistic function damps it by s (1 - s) <= min(1/4, exp(-|x|)),
// so the result stays within two single-precision roundings for every x.
__device__ __forceinline__ float sigmoidf_(float x) { return __fdividef(1.0f, 1.0f + __expf(-x)); }
__device__ __forceinline__ float silu(float x) { return x * sigmoidf_(x); }
__device__ __forceinline__ float silu_grad(float x) {
    const float s = sigmoidf_(x);
    return s * (1.0f + x * (1.0f - s));
}

// x = hi + lo with hi = x rounded to half precision and lo = (x - hi) rounded to half precision:
// 22 significant bits, as long as lo stays a normal number (|x| above 2^-3 or so; below that the
// absolute error is the subnormal spacing, 2^-25, which is why gradients and weights are carried
// multiplied by a power of two)
__device__ __forceinline__ void split_f16(float x, __half& hi, __half& lo) {
    hi = __float2half_rn(x);
    lo = __float2half_rn(x - __half2float(hi));
}
// four consecutive columns (off a multiple of 4): one 8-byte store per part.  The conversions are
// the packed ones (two floats to a half2, a half2 to two floats): those run on the FMA pipes,
// whereas the scalar float-to-half conversion shares the transcendental unit with the
// exponential and the reciprocal of SiLU, which is what the fused epilogue is bound by.
__device__ __forceinline__ void store_split4(__half* hi, __half* lo, size_t off, float4 v) {
    const __half2 h01 = __floats2half2_rn(v.x, v.y), h23 = __floats2half2_rn(v.z, v.w);
    const float2 f01 = __half22float2(h01), f23 = __half22float2(h23);
    const __half2 l01 = __floats2half2_rn(v.x - f01.x, v.y - f01.y), l23 = __floats2half2_rn(v.z - f23.x, v.w - f23.y);
    uint2 hw, lw;
    hw.x = *reinterpret_cast<const uint32_t*>(&h01); hw.y = *reinterpret_cast<const uint32_t*>(&h23);
    lw.x = *reinterpret_cast<const uint32_t*>(&l01); lw.y = *reinterpret_cast<const uint32_t*>(&l23);
    *reinterpret_cast<uint2*>(hi + off) = hw;
    *reinterpret_cast<uint2*>(lo + off) = lw;
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

// hi + lo of four consecutive columns, through the read-only path
__device__ __forceinline__ float4 load_split4(const __half* hi, const __half* lo, size_t off) {
    const uint2 hw = __ldg(reinterpret_cast<const uint2*>(hi + off)), lw = __ldg(reinterpret_cast<const uint2*>(lo + off));
    const float2 h0 = __half22float2(*reinterpret_cast<const __half2*>(&hw.x)), h1 = __half22float2(*reinterpret_cast<const __half2*>(&hw.y));
    const float2 l0 = __half22float2(*reinterpret_cast<const __half2*>(&lw.x)), l1 = __half22float2(*reinterpret_cast<const __half2*>(&lw.y));
    return make_float4(h0.x + l0.x, h0.y + l0.y, h1.x + l1.x, h1.y + l1.y);
}

cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t st);
bool gemm_tc_supported(const GemmArgs& g);
bool gemm_tc_available();      // the driver's tensor-map encoder could be resolved
// whether a model of hidden width F runs its MLP on the tensor-core GEMM under `path` (the
// half-precision operand rows must be multiples of 16 bytes)
inline bool mlp_uses_tc(int F, int path) { return path >= 2 && (F & 7) == 0 && gemm_tc_available(); }
int gemm_tc_pick_variant(int M, int N, int requested);   // 2 (persistent) or 3 (one tile per CTA) for path 2
constexpr int kGemmTcBN = 128;  // column tile of the tensor-core GEMM
// partial head sums per row that the fused last-layer epilogue of a variant leaves
inline int gemm_tc_head_parts(int N, int variant) {
    if (variant == 4) return (N + 31) / 32;        // one per 32-column chunk
    return (variant == 3 ? 1 : 4) * ((N + kGemmTcBN - 1) / kGemmTcBN);
}
cudaError_t launch_gemm_tc(const GemmArgs& g, cudaStream_t st);

}  // namespace umd
