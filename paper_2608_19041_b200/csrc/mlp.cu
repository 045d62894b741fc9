// Atomic-energy MLP: residual SiLU layers, scalar head, and the input vector-Jacobian
// product (no weight gradients).  Each dense layer is one GEMM whose epilogue applies
// bias / SiLU / identity residual (forward) or the residual add and the SiLU derivative
// (backward), so activations make one trip through memory per layer.
//
// This file holds the CUDA-core fp32 GEMM (any width that is a multiple of 4) and the
// layer schedule; the tensor-core GEMM lives in mlp_tc.cu and plugs into the same
// schedule and epilogues.
#include "kernels.h"
#include "mlp_gemm.h"

namespace umd {

namespace {

constexpr int BM = 64, BN = 64, BK = 16;

__global__ void __launch_bounds__(256) k_gemm_simt(const GemmArgs g) {
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    // loader coordinates: A tile 64 rows x 16 k (float4 along k), B tile 16 k x 64 cols
    const int ar = tid >> 2, ak = (tid & 3) * 4;
    const int bk = tid >> 4, bc = (tid & 15) * 4;
    for (int k0 = 0; k0 < g.K; k0 += BK) {
        float4 av = make_float4(0.f, 0.f, 0.f, 0.f), bv = make_float4(0.f, 0.f, 0.f, 0.f);
        if (m0 + ar < g.M && k0 + ak < g.K)
            av = *reinterpret_cast<const float4*>(g.A + (size_t)(m0 + ar) * g.lda + k0 + ak);
        if (k0 + bk < g.K && n0 + bc < g.N)
            bv = __ldg(reinterpret_cast<const float4*>(g.B + (size_t)(k0 + bk) * g.ldb + n0 + bc));
        As[ak][ar] = av.x; As[ak + 1][ar] = av.y; As[ak + 2][ar] = av.z; As[ak + 3][ar] = av.w;
        *reinterpret_cast<float4*>(&Bs[bk][bc]) = bv;
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            const float4 a4 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] += a[i] * b[j];
        }
        __syncthreads();
    }
    const int n = n0 + tx * 4;
    if (n >= g.N) return;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= g.M) continue;
        float v[4] = {acc[i][0], acc[i][1], acc[i][2], acc[i][3]};
        gemm_epilogue4(g, m, n, v);
    }
}

// scalar head: E_i = h . w_head + b_head + E_ref[type]; seeds the backward pass with
// dE/dY_last = w_head * SiLU'(Y_last)
__global__ void k_head(int n, int F, const float* __restrict__ h, const float* __restrict__ w, float b_head,
                       const float* __restrict__ e_ref, const int* __restrict__ type_s, int a0,
                       float* __restrict__ pre_last, double* __restrict__ e_atom, bool want_grad) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= n) return;
    const float* hr = h + (size_t)warp * F;
    float s = 0.f;
    for (int f = lane; f < F; f += 32) s += hr[f] * __ldg(w + f);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0)
        e_atom[a0 + warp] = (double)s + (double)b_head + (double)__ldg(e_ref + type_s[a0 + warp]);
    if (want_grad) {
        float* pr = pre_last + (size_t)warp * F;
        for (int f = lane; f < F; f += 32) {
            const float v = __ldg(w + f) * silu_grad(pr[f]);
            pr[f] = v;
        }
    }
}

// tensor-core path: the last layer's epilogue left one partial dot product per column tile
__global__ void k_head_finish(int n, int parts, const float* __restrict__ part, float b_head,
                              const float* __restrict__ e_ref, const int* __restrict__ type_s, int a0,
                              double* __restrict__ e_atom) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    double s = 0.0;
    for (int p = 0; p < parts; ++p) s += (double)part[(size_t)i * parts + p];
    e_atom[a0 + i] = s + (double)b_head + (double)__ldg(e_ref + type_s[a0 + i]);
}

}  // namespace

cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t st) {
    if (g.M <= 0 || g.N <= 0) return cudaSuccess;
    dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM);
    k_gemm_simt<<<grid, 256, 0, st>>>(g);
    return cudaGetLastError();
}

// a model runs all of its layers on one kind of GEMM (the two keep gradients on different scales)
static cudaError_t run_gemm(const GemmArgs& g, bool tc, cudaStream_t st) {
    if (!tc) return launch_gemm_simt(g, st);
    if (!gemm_tc_supported(g)) return cudaErrorInvalidValue;
    return launch_gemm_tc(g, st);
}

cudaError_t launch_mlp_forward(const MlpArgs& a, cudaStream_t st) {
    const Dims& d = a.d;
    const int n = a.n, F = d.F, NH = d.n_hidden;
    if (n <= 0) return cudaSuccess;
    const size_t layer = (size_t)n * F;
    float* hb[2] = {a.hbuf, a.hbuf + layer};
    const bool res0 = (d.D_out == F);
    const bool tc = a.tc_hi && a.tc_lo && mlp_uses_tc(F, a.path);
    const int variant = tc ? gemm_tc_pick_variant(n, F, a.path) : a.path;
    // the backward seed goes to the slot the last layer does not read its input from
    const int seed_slot = NH & 1;
    cudaError_t e;
    // ---- forward --------------------------------------------------------------------
    for (int t = 0; t < NH; ++t) {
        GemmArgs g = {};
        g.mode = 0;
        g.acc_scale = tc ? a.m.w_scale_inv[t] : 1.0f; g.rvec_scale = 1.0f; g.out_scale = 1.0f;
        g.seed_scale = tc ? a.m.grad_scale : 1.0f;
        g.M = n; g.N = F;
        if (t == 0) { g.A = a.desc; g.lda = d.DP; g.K = d.DP; g.res = res0 ? a.desc : nullptr; g.ldres = d.DP; }
        else { g.A = hb[(t - 1) & 1]; g.lda = F; g.K = F; g.res = hb[(t - 1) & 1]; g.ldres = F; }
        g.B = a.m.theta[t]; g.ldb = F;
        g.Bt_hi = a.m.thetaT_hi[t]; g.Bt_lo = a.m.thetaT_lo[t]; g.ldbt = t == 0 ? d.DP : F;
        // tensor-core path: the split of layer t's input sits in slot t & 1 (layer 0's is made by
        // the split kernel), and the epilogue leaves the split of its output in the other slot
        g.A_hi = a.tc_hi + (size_t)(t & 1) * a.tc_slot; g.A_lo = a.tc_lo + (size_t)(t & 1) * a.tc_slot;
        g.a_presplit = t > 0 || (tc && a.desc_presplit); g.err = a.err; g.variant = variant;
        g.spin_limit = a.spin_limit; g.test_skip_kblock = t == 0 ? a.test_skip_kblock : 0;
        if (tc && t + 1 < NH) {
            g.nxt_hi = a.tc_hi + (size_t)((t + 1) & 1) * a.tc_slot; g.nxt_lo = a.tc_lo + (size_t)((t + 1) & 1) * a.tc_slot;
            g.ldnxt = F;
        }
        g.bias = a.m.bias[t];
        if (tc && t == 0 && a.fold_x0) {
            // the first C0 feature columns are constants per species: their share of the product
            // sits in the per-species bias, and the GEMM starts at column C0 of A and of Theta_1^T
            g.A_hi += d.C0; g.A_lo += d.C0; g.lda_split = d.DP; g.K = d.DP - d.C0;
            g.Bt_hi += d.C0; g.Bt_lo += d.C0;
            g.bias_rows = a.m.type_bias; g.row_type = a.type_s + a.a0;
        }
        g.pre = a.want_grad ? a.pre + (size_t)t * layer : nullptr; g.ldpre = F;
        g.out = hb[t & 1]; g.ldout = F;
        if (tc) {
            // the activations travel as their split only: the residual of layer t is the split this
            // layer reads as its A operand, and no fp32 copy of the output is stored
            g.out = nullptr;
            if (t > 0) { g.res = nullptr; g.res_hi = g.A_hi; g.res_lo = g.A_lo; g.ldres = F; }
        }
        if (tc && t == NH - 1) {
            // last layer: the epilogue takes the head's dot product and the backward seed, so
            // neither the activations nor the pre-activations of this layer are stored
            g.head_w = a.m.w_head; g.head_part = hb[t & 1]; g.head_parts = gemm_tc_head_parts(F, variant);
            g.out = nullptr; g.pre = nullptr;
            if (a.want_grad) {
                g.nxt_hi = a.tc_hi + (size_t)seed_slot * a.tc_slot; g.nxt_lo = a.tc_lo + (size_t)seed_slot * a.tc_slot;
                g.ldnxt = F;
            }
        }
        if ((e = run_gemm(g, tc, st)) != cudaSuccess) return e;
    }
    if (tc) {
        const int parts = gemm_tc_head_parts(F, variant);
        k_head_finish<<<(n + 255) / 256, 256, 0, st>>>(n, parts, hb[(NH - 1) & 1], a.m.b_head, a.m.e_ref, a.type_s, a.a0,
                                                        a.e_atom);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    } else {
        const int warps = 8, blocks = (n + warps - 1) / warps;
        k_head<<<blocks, warps * 32, 0, st>>>(n, F, hb[(NH - 1) & 1], a.m.w_head, a.m.b_head, a.m.e_ref, a.type_s,
                                             a.a0, a.want_grad ? a.pre + (size_t)(NH - 1) * layer : nullptr,
                                             a.e_atom, a.want_grad);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// backward: dE/dY_t sits in pre[t]; dE/dh_t alternates between the two hbuf slots
cudaError_t launch_mlp_backward(const MlpArgs& a, cudaStream_t st) {
    const Dims& d = a.d;
    const int n = a.n, F = d.F, NH = d.n_hidden;
    if (n <= 0) return cudaSuccess;
    const size_t layer = (size_t)n * F;
    float* hb[2] = {a.hbuf, a.hbuf + layer};
    const bool res0 = (d.D_out == F);
    cudaError_t e;
    const bool tc = a.tc_hi && a.tc_lo && mlp_uses_tc(F, a.path);
    const int variant = tc ? gemm_tc_pick_variant(n, F, a.path) : a.path;
    // tensor-core path: every gradient of the chain is carried multiplied by grad_scale (the seed
    // came that way); the head weights join it with the same factor and the last GEMM removes it
    const float gs = tc ? a.m.grad_scale : 1.0f;
    int sp = NH & 1;           // tensor-core path: slot with the half-precision split of pre[t] (the forward pass left the seed here)
    int slot = 0;              // slot holding dE/dh_t (unused while the gradient is w_head itself)
    bool vec_grad = true;      // dE/dh_t == w_head for every atom (top layer)
    for (int t = NH - 1; t >= 1; --t) {
        GemmArgs g = {};
        g.mode = 1;
        g.acc_scale = tc ? a.m.w_scale_inv[t] : 1.0f; g.rvec_scale = gs; g.out_scale = 1.0f; g.seed_scale = 1.0f;
        g.M = n; g.N = F; g.K = F;
        g.A = a.pre + (size_t)t * layer; g.lda = F;
        g.B = a.m.thetaT[t]; g.ldb = F;
        g.Bt_hi = a.m.theta_hi[t]; g.Bt_lo = a.m.theta_lo[t]; g.ldbt = F;
        g.A_hi = a.tc_hi + (size_t)sp * a.tc_slot; g.A_lo = a.tc_lo + (size_t)sp * a.tc_slot;
        g.a_presplit = tc; g.err = a.err; g.variant = variant; g.spin_limit = a.spin_limit;
        if (tc) { g.nxt_hi = a.tc_hi + (size_t)(1 - sp) * a.tc_slot; g.nxt_lo = a.tc_lo + (size_t)(1 - sp) * a.tc_slot; g.ldnxt = F; }
        sp = 1 - sp;
        if (vec_grad) g.rvec = a.m.w_head; else { g.res = hb[slot]; g.ldres = F; }
        const int out_slot = vec_grad ? 0 : 1 - slot;
        const bool need_dh = (t - 1 >= 1) || res0;
        g.out = need_dh ? hb[out_slot] : nullptr; g.ldout = F;
        g.pre = a.pre + (size_t)(t - 1) * layer; g.ldpre = F;
        if ((e = run_gemm(g, tc, st)) != cudaSuccess) return e;
        slot = out_slot; vec_grad = false;
    }
    {
        GemmArgs g = {};
        g.mode = 1;
        g.acc_scale = tc ? a.m.w_scale_inv[0] : 1.0f; g.rvec_scale = gs; g.out_scale = 1.0f / gs; g.seed_scale = 1.0f;
        g.M = n; g.N = d.DP; g.K = F;
        g.A = a.pre; g.lda = F;
        g.B = a.m.thetaT[0]; g.ldb = d.DP;
        g.Bt_hi = a.m.theta_hi[0]; g.Bt_lo = a.m.theta_lo[0]; g.ldbt = F;
        g.A_hi = a.tc_hi + (size_t)sp * a.tc_slot; g.A_lo = a.tc_lo + (size_t)sp * a.tc_slot;
        g.a_presplit = tc; g.err = a.err; g.variant = variant; g.spin_limit = a.spin_limit;
        // this GEMM's epilogue is a plain store, so its main loop sets the pace, and the two-CTA
        // kernel's is the faster one (measured: 122 against 147 us on 131072 rows, N = 416, K = 384)
        if (tc && a.path == 2 && variant == 2) g.variant = gemm_tc_pick_variant(n, d.DP, 4);
        if (res0) {
            if (vec_grad) { g.rvec = a.m.w_head; g.rvec_n = F; }
            else { g.res = hb[slot]; g.ldres = F; g.res_n = F; }
        }
        g.out = a.desc; g.ldout = d.DP;
        if (tc && a.fold_x0) {        // no gradient is needed for the per-species constant columns
            g.N = d.DP - d.C0;
            g.Bt_hi += (size_t)d.C0 * F; g.Bt_lo += (size_t)d.C0 * F;
            g.out = a.desc + d.C0;
        }
        if ((e = run_gemm(g, tc, st)) != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace umd
