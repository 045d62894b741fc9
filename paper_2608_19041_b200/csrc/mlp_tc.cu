// Tensor-core GEMM for the MLP layers on sm_100a: TMA loads into 64-byte-swizzled shared
// memory, tcgen05.mma (kind::f16) issued by one thread, fp32 accumulator in tensor memory,
// tcgen05.ld epilogue with the fused bias / SiLU / residual (or SiLU-derivative) step.
//
// Precision: a single half-precision (or TF32) product carries 11 significant bits, far short
// of the 1e-5 parity target, so every operand is split into two half-precision numbers,
// x = hi + lo with hi = half(x) and lo = half(x - hi), and each K step issues three MMAs,
// A_lo B_hi + A_hi B_lo + A_hi B_hi (the lo*lo term, ~2^-22, is dropped): the same 22
// significant bits as a split into two TF32 numbers, at twice the tensor-core rate (K = 16 per
// instruction instead of 8) and half the operand bytes (hi and lo together are as large as the
// fp32 value).  Half precision has the narrower exponent: a low part below 2^-14 is subnormal
// and keeps an absolute error of 2^-25.  Activations are O(1), where that is at the level of
// single-precision rounding; weights and back-propagated gradients are small numbers, so the
// weights are stored multiplied by a power of two chosen per layer at create time and the
// backward chain carries its gradients multiplied by one chosen from the head weights
// (GemmArgs::acc_scale, rvec_scale, out_scale, seed_scale); powers of two change no mantissa.
// Weights are split once on the host; activations are split by the kernel that produces them
// (the invariants kernel, a GEMM epilogue; a small split kernel remains for callers that hand in
// an unsplit operand).
//
// Tiling of the first kernel below: one CTA computes a 128 x 128 output tile; K advances in blocks of 32 halves (one
// 64-byte swizzle span) through a 3-stage ring of {A_hi, A_lo, B_hi, B_lo} tiles (32 KB per
// stage), so two CTAs fit on an SM and one CTA's epilogue overlaps the other's main loop.
// This kernel keeps the hi*hi sum and the cross terms in two accumulators (256 columns of
// tensor memory per CTA); the persistent kernel further down, which needs all 512 columns
// for its double buffering, sums all three products into one.
// Warp 0 is the TMA producer, warp 1 issues the MMAs and owns the tensor-memory
// allocation, warps 2-5 run the epilogue (one 32-lane quarter of tensor memory each).
// Every mbarrier wait is bounded: on expiry the kernel flags an error word and carries on,
// so a wedged pipeline ends with a wrong result and an error code instead of a hang, and
// tensor memory is always released.
#include <cuda.h>

#include <cstdint>

#include "common.cuh"
#include "mlp_gemm.h"

namespace umd {

namespace {

constexpr int BM = 128, BN = kGemmTcBN, BK = 32, STAGES = 3;   // BK in half-precision elements
constexpr int MMA_K = 16;                              // K of one kind::f16 instruction (32 bytes of a row)
constexpr uint32_t TILE_BYTES = BM * BK * 2;          // 8 KB, also BN * BK * 2
constexpr uint32_t STAGE_BYTES = 4 * TILE_BYTES;      // A_hi, A_lo, B_hi, B_lo
constexpr uint32_t BAR_BYTES = 128;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + BAR_BYTES;
constexpr uint32_t TMEM_COLS = 256;                   // two accumulators: hi*hi, and the two cross terms
constexpr int EPITCH = BN + 4;                        // epilogue staging pitch: 16-byte rows, odd in 16-byte units
constexpr int kSpinLimit = 4000000;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  After `limit` polls it gives up: the CTA's abort flag is raised, the error word
// gets kErrPipelineTimeout, and from then on every wait of the CTA returns at once, the producer
// stops issuing copies and the MMA warp stops issuing instructions, so that a wedged pipeline
// ends with a wrong result and an error code instead of a hang.  Returns false on that path.
__device__ __forceinline__ bool mbar_wait_a(uint32_t bar, uint32_t parity, int* err, volatile int* abort_flag, int limit) {
    if (*abort_flag) return false;
    for (int i = 0; i < limit; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (i > 64) __nanosleep(32);
    }
    *abort_flag = 1;
    if (err) atomicOr(err, kErrPipelineTimeout);
    return false;
}
// plain bounded wait of the shutdown path (no flag, no error: the caller is already giving up)
__device__ __forceinline__ void mbar_wait_quiet(uint32_t bar, uint32_t parity, int limit) {
    for (int i = 0; i < limit; ++i) {
        if (mbar_try(bar, parity)) return;
        if (i > 64) __nanosleep(32);
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
// shared-memory matrix descriptor: K-major tile, 64-byte swizzle, rows 64 B apart, 8-row
// groups 512 B apart
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)1 << 16) | ((uint64_t)(512 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)4 << 61);
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// instruction descriptor: D = F32, A = B = F16 (format code 0), both K-major, N = 128, M = 128
constexpr uint32_t kIdesc = (1u << 4) | (0u << 7) | (0u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

// MODE 0: forward layer, 1: backward layer, 2: last forward layer with the fused head
template <int MODE>
__global__ void __launch_bounds__(192, 2)
k_gemm_tc(const __grid_constant__ CUtensorMap mAh, const __grid_constant__ CUtensorMap mAl,
          const __grid_constant__ CUtensorMap mBh, const __grid_constant__ CUtensorMap mBl, const GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t bars = tiles + STAGES * STAGE_BYTES;       // full[s], empty[s], accum, then the tmem slot
    const uint32_t accum_bar = bars + 8 * (2 * STAGES), drain_bar = accum_bar + 24;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + (bars - raw) + 8 * (2 * STAGES + 1));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + (bars - raw) + 8 * (2 * STAGES + 2));
    const int limit = g.spin_limit > 0 ? g.spin_limit : kSpinLimit;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int KB = (g.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(bars + 8 * s, 1); mbar_init(bars + 8 * (STAGES + s), 1); }
        mbar_init(accum_bar, 1);
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {                                   // TMA producer
            int issued[STAGES];                           // k-block last loaded into each stage (-1: none)
            for (int s = 0; s < STAGES; ++s) issued[s] = -1;
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % STAGES, u = kb / STAGES;
                if (u > 0 && !mbar_wait_a(bars + 8 * (STAGES + s), (u - 1) & 1, g.err, abort_flag, limit)) break;
                if (*abort_flag) break;
                if (g.test_skip_kblock && kb == g.test_skip_kblock - 1) continue;   // diagnostic: this stage never arrives
                const uint32_t full = bars + 8 * s, sa = tiles + s * STAGE_BYTES;
                mbar_expect_tx(full, STAGE_BYTES);
                tma_load_2d(sa, &mAh, kb * BK, m0, full);
                tma_load_2d(sa + TILE_BYTES, &mAl, kb * BK, m0, full);
                tma_load_2d(sa + 2 * TILE_BYTES, &mBh, kb * BK, n0, full);
                tma_load_2d(sa + 3 * TILE_BYTES, &mBl, kb * BK, n0, full);
                issued[s] = kb;
            }
            if (*abort_flag)                              // giving up: let the copies still in flight land first
                for (int s = 0; s < STAGES; ++s)
                    if (issued[s] >= 0) mbar_wait_quiet(bars + 8 * s, (issued[s] / STAGES) & 1, limit);
        }
    } else if (warp == 1) {
        if (lane == 0) {                                   // MMA issuer
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % STAGES, u = kb / STAGES;
                if (!mbar_wait_a(bars + 8 * s, u & 1, g.err, abort_flag, limit)) break;
                tc_fence_after();
                const uint32_t sa = tiles + s * STAGE_BYTES;
#pragma unroll
                for (int k = 0; k < BK / MMA_K; ++k) {
                    const uint64_t ah = umma_desc(sa + k * 32), al = umma_desc(sa + TILE_BYTES + k * 32);
                    const uint64_t bh = umma_desc(sa + 2 * TILE_BYTES + k * 32), bl = umma_desc(sa + 3 * TILE_BYTES + k * 32);
                    // The accumulator truncates once per instruction.  The cross terms, 2^-11 of
                    // the result, get an accumulator of their own, where that loss is 2^-11 as
                    // small, and the main sum sees a third of the instructions.
                    const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                    umma_f16(tmem + BN, al, bh, kIdesc, acc);
                    umma_f16(tmem + BN, ah, bl, kIdesc, 1u);
                    umma_f16(tmem, ah, bh, kIdesc, acc);
                }
                umma_commit(bars + 8 * (STAGES + s));      // frees the stage when these MMAs retire
            }
            umma_commit(accum_bar);
            if (*abort_flag) {                             // every instruction issued so far has to retire before the
                umma_commit(drain_bar);                    // tensor memory goes back
                mbar_wait_quiet(drain_bar, 0, limit);
            }
        }
    } else {                                               // epilogue: warps 2..5 -> lane quarters 2,3,0,1
        // Tensor memory hands each thread one accumulator row; global memory wants a warp
        // on one row.  The tile is therefore turned through shared memory (the operand
        // ring is free once the accumulator barrier has fired): each warp parks its 32
        // rows with a padded pitch, then walks them row by row, lanes across columns, so
        // every global access of the fused epilogue is one contiguous 512-byte segment.
        const int q = warp & 3;
        mbar_wait_a(accum_bar, 0, g.err, abort_flag, limit);
        tc_fence_after();
        float* stage = reinterpret_cast<float*>(smem_raw + (tiles - raw)) + (size_t)q * 32 * EPITCH;
        const float sc = g.acc_scale;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
            float v[32], w[32];
            tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
            tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(BN + c0), w);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                *reinterpret_cast<float4*>(stage + lane * EPITCH + c0 + 4 * j) =
                    make_float4(sc * (v[4 * j] + w[4 * j]), sc * (v[4 * j + 1] + w[4 * j + 1]), sc * (v[4 * j + 2] + w[4 * j + 2]),
                                sc * (v[4 * j + 3] + w[4 * j + 3]));
        }
        __syncwarp();
        const int n = n0 + 4 * lane;
        const bool valid = n < g.N;
        {
            float4 bias = make_float4(0.f, 0.f, 0.f, 0.f), rvec = bias, hw = bias;
            if (valid && MODE != 1 && !g.bias_rows) bias = __ldg(reinterpret_cast<const float4*>(g.bias + n));
            if (valid && MODE == 2) hw = __ldg(reinterpret_cast<const float4*>(g.head_w + n));
            const bool use_res = valid && (g.res || g.res_hi) && (MODE != 1 || g.res_n == 0 || n < g.res_n);
            if (valid && MODE == 1 && g.rvec && (g.rvec_n == 0 || n < g.rvec_n)) {
                rvec = __ldg(reinterpret_cast<const float4*>(g.rvec + n));
                rvec.x *= g.rvec_scale; rvec.y *= g.rvec_scale; rvec.z *= g.rvec_scale; rvec.w *= g.rvec_scale;
            }
            const int rows = min(32, g.M - (m0 + q * 32));
            // The stores below may alias the loads as far as the compiler knows, so the rows
            // are taken in batches: all global loads of a batch are issued before its first
            // store, which keeps RB rows (not one) in flight per warp.
            constexpr int RB = 8;
            const bool rd_pre = valid && MODE == 1 && g.pre;
#pragma unroll 1
            for (int r0 = 0; r0 < rows; r0 += RB) {
                float4 res[RB], y[RB];
#pragma unroll
                for (int j = 0; j < RB; ++j) {
                    const size_t m = (size_t)(m0 + q * 32 + r0 + j);
                    res[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                    y[j] = res[j];
                    if (r0 + j < rows) {
                        if (use_res) {
                            if (MODE != 1 && g.res_hi) res[j] = load_split4(g.res_hi, g.res_lo, m * g.ldres + n);
                            else res[j] = __ldg(reinterpret_cast<const float4*>(g.res + m * g.ldres + n));
                        }
                        if (MODE == 1 && rd_pre) y[j] = __ldg(reinterpret_cast<const float4*>(g.pre + m * g.ldpre + n));
                        if (MODE != 1 && valid && g.bias_rows)      // per-species bias: carried in the y slot
                            y[j] = __ldg(reinterpret_cast<const float4*>(g.bias_rows + (size_t)g.row_type[m] * g.N + n));
                    }
                }
#pragma unroll
                for (int j = 0; j < RB; ++j) {
                    if (r0 + j >= rows) break;
                    const size_t m = (size_t)(m0 + q * 32 + r0 + j);
                    float4 a = *reinterpret_cast<const float4*>(stage + (r0 + j) * EPITCH + 4 * lane);
                    if (MODE != 1) {
                        const float4 bb = g.bias_rows ? y[j] : bias;
                        a.x += bb.x; a.y += bb.y; a.z += bb.z; a.w += bb.w;
                        const float4 o = make_float4(silu(a.x) + res[j].x, silu(a.y) + res[j].y, silu(a.z) + res[j].z,
                                                     silu(a.w) + res[j].w);
                        if (MODE == 2) {           // last layer: row . w_head, and the backward seed
                            float part = valid ? o.x * hw.x + o.y * hw.y + o.z * hw.z + o.w * hw.w : 0.f;
#pragma unroll
                            for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
                            if (lane == 0) g.head_part[m * g.head_parts + blockIdx.x] = part;
                            if (valid && g.nxt_hi)
                                store_split4(g.nxt_hi, g.nxt_lo, m * g.ldnxt + n,
                                             make_float4(g.seed_scale * hw.x * silu_grad(a.x), g.seed_scale * hw.y * silu_grad(a.y),
                                                         g.seed_scale * hw.z * silu_grad(a.z), g.seed_scale * hw.w * silu_grad(a.w)));
                        } else if (valid) {
                            if (g.pre) *reinterpret_cast<float4*>(g.pre + m * g.ldpre + n) = a;
                            if (g.out) *reinterpret_cast<float4*>(g.out + m * g.ldout + n) = o;
                            if (g.nxt_hi) store_split4(g.nxt_hi, g.nxt_lo, m * g.ldnxt + n, o);
                        }
                    } else if (valid) {
                        a.x += res[j].x + rvec.x; a.y += res[j].y + rvec.y; a.z += res[j].z + rvec.z; a.w += res[j].w + rvec.w;
                        if (g.out) *reinterpret_cast<float4*>(g.out + m * g.ldout + n) = make_float4(g.out_scale * a.x, g.out_scale * a.y, g.out_scale * a.z, g.out_scale * a.w);
                        if (g.pre) {
                            const float4 o = make_float4(a.x * silu_grad(y[j].x), a.y * silu_grad(y[j].y),
                                                         a.z * silu_grad(y[j].z), a.w * silu_grad(y[j].w));
                            // the next GEMM of the chain reads the split (gemm_tc_supported insists on it)
                            store_split4(g.nxt_hi, g.nxt_lo, m * g.ldnxt + n, o);
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------------------------------
// Persistent variant: one CTA per SM walks work items of 256 rows x 128 columns.  An item
// uses two accumulators (rows 0..127 and 128..255) that share every B tile, so the weights
// cross L2 -> shared memory half as often as with one 128 x 128 tile per CTA; tensor memory
// holds two such pairs (512 columns), so the epilogue of item i overlaps the main loop of
// item i + 1.  Warp 0: TMA producer, warp 1: MMA issuer, warps 2..17: epilogue (warp % 4 =
// lane quarter of tensor memory; of the four warps of a quarter, one per accumulator of the
// pair and per 64-column half).  The fused epilogue is a few dozen dependent instructions per
// element (exponential, reciprocal, conversions) and is bound by instruction latency, not by
// memory: with eight warps (two per scheduler) it took twice as long as an item's MMAs; sixteen
// hide that latency.  The epilogue turns the tile through a staging area of its own, 32 columns
// at a time.
constexpr int P_STAGES = 3;
constexpr uint32_t P_STAGE_BYTES = 6 * TILE_BYTES;    // A0_hi, A0_lo, A1_hi, A1_lo, B_hi, B_lo
constexpr int P_EPW = 16;                              // epilogue warps
constexpr int P_SPITCH = 32 + 4;                       // staging row pitch (floats)
constexpr uint32_t P_STAGING_BYTES = P_EPW * 32 * P_SPITCH * 4;
constexpr int P_SMEM_BYTES = P_STAGES * P_STAGE_BYTES + P_STAGING_BYTES + 1024 + BAR_BYTES;
constexpr int P_THREADS = (2 + P_EPW) * 32;

template <int MODE>
__global__ void __launch_bounds__(P_THREADS, 1)
k_gemm_tcp(const __grid_constant__ CUtensorMap mAh, const __grid_constant__ CUtensorMap mAl,
           const __grid_constant__ CUtensorMap mBh, const __grid_constant__ CUtensorMap mBl, const GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t staging = tiles + P_STAGES * P_STAGE_BYTES;
    const uint32_t bars = staging + P_STAGING_BYTES;   // full[3], empty[3], acc_full[2], acc_empty[2], tmem slot, abort flag
    const uint32_t acc_full = bars + 8 * (2 * P_STAGES), acc_empty = acc_full + 16;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + (acc_empty + 16 - raw));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + (acc_empty + 24 - raw));
    const uint32_t drain_bar = acc_empty + 32;
    const int limit = g.spin_limit > 0 ? g.spin_limit : kSpinLimit;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = (g.K + BK - 1) / BK;
    const int ntn = (g.N + BN - 1) / BN, ntm = (g.M + 2 * BM - 1) / (2 * BM);
    const int items = ntn * ntm;

    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) { mbar_init(bars + 8 * s, 1); mbar_init(bars + 8 * (P_STAGES + s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full + 8 * b, 1); mbar_init(acc_empty + 8 * b, P_EPW); }
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void*)tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {                                   // TMA producer
            int gk = 0;
            int issued[P_STAGES];                         // k-block count of the last load into each stage (-1: none)
            for (int s = 0; s < P_STAGES; ++s) issued[s] = -1;
            for (int it = blockIdx.x; it < items && !*abort_flag; it += gridDim.x) {
                const int m0 = (it / ntn) * 2 * BM, n0 = (it % ntn) * BN;
                for (int kb = 0; kb < KB; ++kb, ++gk) {
                    const int s = gk % P_STAGES, u = gk / P_STAGES;
                    if (u > 0 && !mbar_wait_a(bars + 8 * (P_STAGES + s), (u - 1) & 1, g.err, abort_flag, limit)) break;
                    if (*abort_flag) break;
                    if (g.test_skip_kblock && gk == g.test_skip_kblock - 1) continue;   // diagnostic: this stage never arrives
                    issued[s] = gk;
                    const uint32_t full = bars + 8 * s, sa = tiles + s * P_STAGE_BYTES;
                    mbar_expect_tx(full, P_STAGE_BYTES);
                    tma_load_2d(sa, &mAh, kb * BK, m0, full);
                    tma_load_2d(sa + TILE_BYTES, &mAl, kb * BK, m0, full);
                    tma_load_2d(sa + 2 * TILE_BYTES, &mAh, kb * BK, m0 + BM, full);
                    tma_load_2d(sa + 3 * TILE_BYTES, &mAl, kb * BK, m0 + BM, full);
                    tma_load_2d(sa + 4 * TILE_BYTES, &mBh, kb * BK, n0, full);
                    tma_load_2d(sa + 5 * TILE_BYTES, &mBl, kb * BK, n0, full);
                }
            }
            if (*abort_flag)                              // giving up: let the copies still in flight land first
                for (int s = 0; s < P_STAGES; ++s)
                    if (issued[s] >= 0) mbar_wait_quiet(bars + 8 * s, (issued[s] / P_STAGES) & 1, limit);
        }
    } else if (warp == 1) {
        if (lane == 0) {                                   // MMA issuer
            int gk = 0, li = 0;
            for (int it = blockIdx.x; it < items && !*abort_flag; it += gridDim.x, ++li) {
                const int b = li & 1, v = li >> 1;
                if (v > 0 && !mbar_wait_a(acc_empty + 8 * b, (v - 1) & 1, g.err, abort_flag, limit)) break;
                tc_fence_after();
                const uint32_t d0 = tmem + (uint32_t)(b * 256), d1 = d0 + 128u;
                for (int kb = 0; kb < KB; ++kb, ++gk) {
                    const int s = gk % P_STAGES, u = gk / P_STAGES;
                    if (!mbar_wait_a(bars + 8 * s, u & 1, g.err, abort_flag, limit)) break;
                    tc_fence_after();
                    const uint32_t sa = tiles + s * P_STAGE_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / MMA_K; ++k) {
                        const uint64_t bh = umma_desc(sa + 4 * TILE_BYTES + k * 32), bl = umma_desc(sa + 5 * TILE_BYTES + k * 32);
                        const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                        {
                            const uint64_t ah = umma_desc(sa + k * 32), al = umma_desc(sa + TILE_BYTES + k * 32);
                            umma_f16(d0, al, bh, kIdesc, acc);
                            umma_f16(d0, ah, bl, kIdesc, 1u);
                            umma_f16(d0, ah, bh, kIdesc, 1u);
                        }
                        {
                            const uint64_t ah = umma_desc(sa + 2 * TILE_BYTES + k * 32), al = umma_desc(sa + 3 * TILE_BYTES + k * 32);
                            umma_f16(d1, al, bh, kIdesc, acc);
                            umma_f16(d1, ah, bl, kIdesc, 1u);
                            umma_f16(d1, ah, bh, kIdesc, 1u);
                        }
                    }
                    umma_commit(bars + 8 * (P_STAGES + s));    // frees the stage when these MMAs retire
                }
                umma_commit(acc_full + 8 * b);
            }
            if (*abort_flag) {                             // every instruction issued so far has to retire before the
                umma_commit(drain_bar);                    // tensor memory goes back
                mbar_wait_quiet(drain_bar, 0, limit);
            }
        }
    } else {                                               // epilogue
        const int e = warp - 2, q = warp & 3, h = (e >> 2) & 1, p = e >> 3;
        float* stage = reinterpret_cast<float*>(smem_raw + (staging - raw)) + (size_t)e * 32 * P_SPITCH;
        const int rr = lane >> 3, c4 = (lane & 7) * 4;       // eight lanes per row, four columns per lane
        const float sc = g.acc_scale;
        int li = 0;
        for (int it = blockIdx.x; it < items; it += gridDim.x, ++li) {
            const int b = li & 1, v = li >> 1;
            const int ct = it % ntn;
            const int mrow0 = (it / ntn) * 2 * BM + h * BM + q * 32, n0 = ct * BN + p * 64;
            mbar_wait_a(acc_full + 8 * b, v & 1, g.err, abort_flag, limit);
            tc_fence_after();
            const uint32_t tacc = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * 256 + h * 128 + p * 64);
#pragma unroll 1
            for (int ch = 0; ch < 2; ++ch) {               // two chunks of 32 columns
                {
                    float vv[32];
                    tmem_ld32(tacc + (uint32_t)(ch * 32), vv);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<float4*>(stage + lane * P_SPITCH + 4 * j) =
                            make_float4(sc * vv[4 * j], sc * vv[4 * j + 1], sc * vv[4 * j + 2], sc * vv[4 * j + 3]);
                }
                if (ch == 1) {                             // the accumulator has been read out: hand it back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acc_empty + 8 * b) : "memory");
                }
                __syncwarp();
                const int n = n0 + ch * 32 + c4;
                const bool valid = n < g.N;
                float4 bias = make_float4(0.f, 0.f, 0.f, 0.f), rvec = bias, hw = bias;
                if (valid && MODE != 1 && !g.bias_rows) bias = __ldg(reinterpret_cast<const float4*>(g.bias + n));
                if (valid && MODE == 2) hw = __ldg(reinterpret_cast<const float4*>(g.head_w + n));
                const bool use_res = valid && (g.res || g.res_hi) && (MODE != 1 || g.res_n == 0 || n < g.res_n);
                if (valid && MODE == 1 && g.rvec && (g.rvec_n == 0 || n < g.rvec_n)) {
                    rvec = __ldg(reinterpret_cast<const float4*>(g.rvec + n));
                    rvec.x *= g.rvec_scale; rvec.y *= g.rvec_scale; rvec.z *= g.rvec_scale; rvec.w *= g.rvec_scale;
                }
                const bool rd_pre = valid && MODE == 1 && g.pre;
                constexpr int RB = 4;                      // iterations (four rows each) whose loads are issued together
#pragma unroll 1
                for (int i0 = 0; i0 < 8; i0 += RB) {
                    float4 res[RB], y[RB];
#pragma unroll
                    for (int j = 0; j < RB; ++j) {
                        const int m = mrow0 + 4 * (i0 + j) + rr;
                        res[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                        y[j] = res[j];
                        if (m < g.M) {
                            if (use_res) {
                                if (MODE != 1 && g.res_hi) res[j] = load_split4(g.res_hi, g.res_lo, (size_t)m * g.ldres + n);
                                else res[j] = __ldg(reinterpret_cast<const float4*>(g.res + (size_t)m * g.ldres + n));
                            }
                            if (MODE == 1 && rd_pre) y[j] = __ldg(reinterpret_cast<const float4*>(g.pre + (size_t)m * g.ldpre + n));
                            if (MODE != 1 && valid && g.bias_rows)  // per-species bias: carried in the y slot
                                y[j] = __ldg(reinterpret_cast<const float4*>(g.bias_rows + (size_t)__ldg(g.row_type + m) * g.N + n));
                        }
                    }
#pragma unroll
                    for (int j = 0; j < RB; ++j) {
                        const int r = 4 * (i0 + j) + rr;
                        const size_t m = (size_t)(mrow0 + r);
                        const bool okm = mrow0 + r < g.M;
                        const float4 rj = res[j], yj = y[j];
                        float4 a = *reinterpret_cast<const float4*>(stage + r * P_SPITCH + c4);
                        if (MODE != 1) {
                            const float4 bb = g.bias_rows ? yj : bias;
                            a.x += bb.x; a.y += bb.y; a.z += bb.z; a.w += bb.w;
                            const float4 o = make_float4(silu(a.x) + rj.x, silu(a.y) + rj.y, silu(a.z) + rj.z, silu(a.w) + rj.w);
                            if (MODE == 2) {               // last layer: row . w_head over these 32 columns, and the seed
                                float part = valid ? o.x * hw.x + o.y * hw.y + o.z * hw.z + o.w * hw.w : 0.f;
#pragma unroll
                                for (int off = 4; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
                                if ((lane & 7) == 0 && okm) g.head_part[m * g.head_parts + 4 * ct + 2 * p + ch] = part;
                                if (valid && okm && g.nxt_hi)
                                    store_split4(g.nxt_hi, g.nxt_lo, m * g.ldnxt + n,
                                                 make_float4(g.seed_scale * hw.x * silu_grad(a.x), g.seed_scale * hw.y * silu_grad(a.y),
                                                             g.seed_scale * hw.z * silu_grad(a.z), g.seed_scale * hw.w * silu_grad(a.w)));
                            } else if (valid && okm) {
                                if (g.pre) *reinterpret_cast<float4*>(g.pre + m * g.ldpre + n) = a;
                                if (g.out) *reinterpret_cast<float4*>(g.out + m * g.ldout + n) = o;
                                if (g.nxt_hi) store_split4(g.nxt_hi, g.nxt_lo, m * g.ldnxt + n, o);
                            }
                        } else if (valid && okm) {
                            a.x += rj.x + rvec.x; a.y += rj.y + rvec.y; a.z += rj.z + rvec.z; a.w += rj.w + rvec.w;
                            if (g.out)
                                *reinterpret_cast<float4*>(g.out + m * g.ldout + n) =
                                    make_float4(g.out_scale * a.x, g.out_scale * a.y, g.out_scale * a.z, g.out_scale * a.w);
                            if (g.pre)                     // the next GEMM of the chain reads the split (gemm_tc_supported insists on it)
                                store_split4(g.nxt_hi, g.nxt_lo, m * g.ldnxt + n,
                                             make_float4(a.x * silu_grad(yj.x), a.y * silu_grad(yj.y), a.z * silu_grad(yj.z),
                                                         a.w * silu_grad(yj.w)));
                        }
                    }
                }
                __syncwarp();                              // staging rows are rewritten by the next chunk
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// ---------------------------------------------------------------------------------------
// Two-CTA variant (tcgen05 cta_group::2): the CTAs of a cluster of two, on the two SMs of a
// pair, work on one item of 256 rows x NT columns (NT <= 256).  Each CTA loads its own 128 rows
// of A and its own half of the weight tile; one thread of the first CTA issues MMAs of shape
// 256 x NT x 16 that read A from both CTAs' shared memory and each half of B once for both, and
// each CTA's tensor memory receives the accumulator of its own 128 rows.  Per SM an MMA step then
// reads 8 KB of shared memory in 128 cycles where the one-CTA kernel reads 8 KB in 64, the whole
// bandwidth of an SM's shared memory, which held its main loop at half the tensor rate; and a
// stage is 32 KB instead of 48, so four stages fit.
//   barriers (same offsets in both CTAs): full[s] is used in the first CTA only and counts the
//   bytes of both CTAs' copies (each CTA's TMA names that barrier); empty[s] and acc_full[b] are
//   signalled in both CTAs at once by a multicast tcgen05.commit; acc_empty[b] of the first CTA
//   collects the epilogue warps of both (the second CTA's warps arrive remotely).
// Warp roles as in the one-CTA persistent kernel (the second CTA's warp 1 only takes part in the
// tensor-memory allocation); sixteen epilogue warps per CTA: four lane quarters x four groups of
// 64 columns.  Every wait is bounded as there; the cluster barrier at the end keeps either CTA
// from leaving while the other may still signal it or read its shared memory.
constexpr int C2_STAGES = 4;
constexpr uint32_t C2_STAGE_BYTES = 4 * TILE_BYTES;    // A_hi, A_lo, B_hi, B_lo (B: at most 128 rows of the half tile)
constexpr int C2_SMEM_BYTES = C2_STAGES * C2_STAGE_BYTES + P_STAGING_BYTES + 1024 + BAR_BYTES;

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// the address, in the cluster's shared window, of the same offset in the first CTA's shared memory
__device__ __forceinline__ uint32_t in_first_cta(uint32_t addr) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(0u));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void umma_f16_pair(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
// arrive on the barrier at this offset in both CTAs once the MMAs issued so far have retired
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}

template <int MODE>
__global__ void __launch_bounds__(P_THREADS, 1)
k_gemm_tc2(const __grid_constant__ CUtensorMap mAh, const __grid_constant__ CUtensorMap mAl,
           const __grid_constant__ CUtensorMap mBh, const __grid_constant__ CUtensorMap mBl, const GemmArgs g, const int NT) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t staging = tiles + C2_STAGES * C2_STAGE_BYTES;
    const uint32_t bars = staging + P_STAGING_BYTES;   // full[4], empty[4], acc_full[2], acc_empty[2], drain, tmem slot, abort flag
    const uint32_t acc_full = bars + 8 * (2 * C2_STAGES), acc_empty = acc_full + 16, drain_bar = acc_empty + 16;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + (drain_bar + 8 - raw));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + (drain_bar + 12 - raw));
    const int limit = g.spin_limit > 0 ? g.spin_limit : kSpinLimit;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const int KB = (g.K + BK - 1) / BK;
    const int ntn = (g.N + NT - 1) / NT, ntm = (g.M + 2 * BM - 1) / (2 * BM);
    const int items = ntn * ntm;
    const int cid = blockIdx.x >> 1, ncl = gridDim.x >> 1;
    const uint32_t b_tile_bytes = (uint32_t)(NT / 2) * BK * 2;          // one half of the column tile, hi or lo

    if (threadIdx.x == 0) {
        for (int s = 0; s < C2_STAGES; ++s) { mbar_init(bars + 8 * s, 1); mbar_init(bars + 8 * (C2_STAGES + s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full + 8 * b, 1); mbar_init(acc_empty + 8 * b, 2 * P_EPW); }
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void*)tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                    // both CTAs' barriers are initialised before either signals the other
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {                                   // TMA producer (both CTAs)
            int gk = 0;
            int issued[C2_STAGES];
            for (int s = 0; s < C2_STAGES; ++s) issued[s] = -1;
            for (int it = cid; it < items && !*abort_flag; it += ncl) {
                const int m0 = (it / ntn) * 2 * BM + (int)rank * BM, n0 = (it % ntn) * NT + (int)rank * (NT / 2);
                for (int kb = 0; kb < KB; ++kb, ++gk) {
                    const int s = gk % C2_STAGES, u = gk / C2_STAGES;
                    if (u > 0 && !mbar_wait_a(bars + 8 * (C2_STAGES + s), (u - 1) & 1, g.err, abort_flag, limit)) break;
                    if (*abort_flag) break;
                    if (g.test_skip_kblock && gk == g.test_skip_kblock - 1) continue;   // diagnostic: this stage never arrives
                    issued[s] = gk;
                    const uint32_t full = bars + 8 * s, full0 = in_first_cta(full), sa = tiles + s * C2_STAGE_BYTES;
                    if (rank == 0) mbar_expect_tx(full, 2 * (2 * TILE_BYTES + 2 * b_tile_bytes));   // the bytes of both CTAs
                    tma_load_2d_pair(sa, &mAh, kb * BK, m0, full0);
                    tma_load_2d_pair(sa + TILE_BYTES, &mAl, kb * BK, m0, full0);
                    tma_load_2d_pair(sa + 2 * TILE_BYTES, &mBh, kb * BK, n0, full0);
                    tma_load_2d_pair(sa + 3 * TILE_BYTES, &mBl, kb * BK, n0, full0);
                }
            }
            // giving up: let the copies still in flight land first (the first CTA sees their barrier; the
            // second waits out the same number of polls)
            if (*abort_flag)
                for (int s = 0; s < C2_STAGES; ++s)
                    if (issued[s] >= 0) mbar_wait_quiet(bars + 8 * s, (issued[s] / C2_STAGES) & 1, rank == 0 ? limit : limit / 4 + 1);
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {                      // MMA issuer (first CTA only)
            // instruction descriptor: D = F32, A = B = F16, both K-major, N = NT, M = 256
            const uint32_t idesc = (1u << 4) | ((uint32_t)(NT >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
            int gk = 0, li = 0;
            for (int it = cid; it < items && !*abort_flag; it += ncl, ++li) {
                const int b = li & 1, v = li >> 1;
                if (v > 0 && !mbar_wait_a(acc_empty + 8 * b, (v - 1) & 1, g.err, abort_flag, limit)) break;
                tc_fence_after();
                const uint32_t d0 = tmem + (uint32_t)(b * 256);
                for (int kb = 0; kb < KB; ++kb, ++gk) {
                    const int s = gk % C2_STAGES, u = gk / C2_STAGES;
                    if (!mbar_wait_a(bars + 8 * s, u & 1, g.err, abort_flag, limit)) break;
                    tc_fence_after();
                    const uint32_t sa = tiles + s * C2_STAGE_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / MMA_K; ++k) {
                        const uint64_t ah = umma_desc(sa + k * 32), al = umma_desc(sa + TILE_BYTES + k * 32);
                        const uint64_t bh = umma_desc(sa + 2 * TILE_BYTES + k * 32), bl = umma_desc(sa + 3 * TILE_BYTES + k * 32);
                        const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                        umma_f16_pair(d0, al, bh, idesc, acc);
                        umma_f16_pair(d0, ah, bl, idesc, 1u);
                        umma_f16_pair(d0, ah, bh, idesc, 1u);
                    }
                    umma_commit_pair(bars + 8 * (C2_STAGES + s));      // frees the stage in both CTAs when these MMAs retire
                }
                umma_commit_pair(acc_full + 8 * b);
            }
            if (*abort_flag) {                             // every instruction issued so far has to retire before the
                umma_commit_pair(drain_bar);               // tensor memory goes back
                mbar_wait_quiet(drain_bar, 0, limit);
            }
        }
    } else {                                               // epilogue (both CTAs)
        const int e = warp - 2, q = warp & 3, cg = e >> 2;
        float* stage = reinterpret_cast<float*>(smem_raw + (staging - raw)) + (size_t)e * 32 * P_SPITCH;
        const int rr = lane >> 3, c4 = (lane & 7) * 4;       // eight lanes per row, four columns per lane
        const float sc = g.acc_scale;
        int li = 0;
        for (int it = cid; it < items; it += ncl, ++li) {
            const int b = li & 1, v = li >> 1;
            const int mrow0 = (it / ntn) * 2 * BM + (int)rank * BM + q * 32, nt0 = (it % ntn) * NT;
            const int n_end = min(g.N, nt0 + NT);          // columns of this item: [nt0, n_end)
            mbar_wait_a(acc_full + 8 * b, v & 1, g.err, abort_flag, limit);
            tc_fence_after();
            const uint32_t tacc = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * 256 + cg * 64);
#pragma unroll 1
            for (int ch = 0; ch < 2; ++ch) {               // two chunks of 32 columns
                const int nc0 = nt0 + cg * 64 + ch * 32;   // first column of the chunk
                const bool chunk_on = nc0 < n_end;         // (uniform over the warp)
                if (chunk_on) {
                    float vv[32];
                    tmem_ld32(tacc + (uint32_t)(ch * 32), vv);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<float4*>(stage + lane * P_SPITCH + 4 * j) =
                            make_float4(sc * vv[4 * j], sc * vv[4 * j + 1], sc * vv[4 * j + 2], sc * vv[4 * j + 3]);
                }
                if (ch == 1) {                             // the accumulator has been read out: hand it back to the first CTA
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(in_first_cta(acc_empty + 8 * b));
                }
                __syncwarp();
                if (!chunk_on) continue;
                const int n = nc0 + c4;
                const bool valid = n < n_end;
                float4 bias = make_float4(0.f, 0.f, 0.f, 0.f), rvec = bias, hw = bias;
                if (valid && MODE != 1 && !g.bias_rows) bias = __ldg(reinterpret_cast<const float4*>(g.bias + n));
                if (valid && MODE == 2) hw = __ldg(reinterpret_cast<const float4*>(g.head_w + n));
                const bool use_res = valid && (g.res || g.res_hi) && (MODE != 1 || g.res_n == 0 || n < g.res_n);
                if (valid && MODE == 1 && g.rvec && (g.rvec_n == 0 || n < g.rvec_n)) {
                    rvec = __ldg(reinterpret_cast<const float4*>(g.rvec + n));
                    rvec.x *= g.rvec_scale; rvec.y *= g.rvec_scale; rvec.z *= g.rvec_scale; rvec.w *= g.rvec_scale;
                }
                const bool rd_pre = valid && MODE == 1 && g.pre;
                constexpr int RB = 4;                      // iterations (four rows each) whose loads are issued together
#pragma unroll 1
                for (int i0 = 0; i0 < 8; i0 += RB) {
                    float4 res[RB], y[RB];
#pragma unroll
                    for (int j = 0; j < RB; ++j) {
                        const int m = mrow0 + 4 * (i0 + j) + rr;
                        res[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                        y[j] = res[j];
                        if (m < g.M) {
                            if (use_res) {
                                if (MODE != 1 && g.res_hi) res[j] = load_split4(g.res_hi, g.res_lo, (size_t)m * g.ldres + n);
                                else res[j] = __ldg(reinterpret_cast<const float4*>(g.res + (size_t)m * g.ldres + n));
                            }
                            if (MODE == 1 && rd_pre) y[j] = __ldg(reinterpret_cast<const float4*>(g.pre + (size_t)m * g.ldpre + n));
                            if (MODE != 1 && valid && g.bias_rows)  // per-species bias: carried in the y slot
                                y[j] = __ldg(reinterpret_cast<const float4*>(g.bias_rows + (size_t)__ldg(g.row_type + m) * g.N + n));
                        }
                    }
#pragma unroll
                    for (int j = 0; j < RB; ++j) {
                        const int r = 4 * (i0 + j) + rr;
                        const size_t m = (size_t)(mrow0 + r);
                        const bool okm = mrow0 + r < g.M;
                        const float4 rj = res[j], yj = y[j];
                        float4 a = *reinterpret_cast<const float4*>(stage + r * P_SPITCH + c4);
                        if (MODE != 1) {
                            const float4 bb = g.bias_rows ? yj : bias;
                            a.x += bb.x; a.y += bb.y; a.z += bb.z; a.w += bb.w;
                            const float4 o = make_float4(silu(a.x) + rj.x, silu(a.y) + rj.y, silu(a.z) + rj.z, silu(a.w) + rj.w);
                            if (MODE == 2) {               // last layer: row . w_head over these 32 columns, and the seed
                                float part = valid ? o.x * hw.x + o.y * hw.y + o.z * hw.z + o.w * hw.w : 0.f;
#pragma unroll
                                for (int off = 4; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
                                if ((lane & 7) == 0 && okm) g.head_part[m * g.head_parts + (nc0 >> 5)] = part;
                                if (valid && okm && g.nxt_hi)
                                    store_split4(g.nxt_hi, g.nxt_lo, m * g.ldnxt + n,
                                                 make_float4(g.seed_scale * hw.x * silu_grad(a.x), g.seed_scale * hw.y * silu_grad(a.y),
                                                             g.seed_scale * hw.z * silu_grad(a.z), g.seed_scale * hw.w * silu_grad(a.w)));
                            } else if (valid && okm) {
                                if (g.pre) *reinterpret_cast<float4*>(g.pre + m * g.ldpre + n) = a;
                                if (g.out) *reinterpret_cast<float4*>(g.out + m * g.ldout + n) = o;
                                if (g.nxt_hi) store_split4(g.nxt_hi, g.nxt_lo, m * g.ldnxt + n, o);
                            }
                        } else if (valid && okm) {
                            a.x += rj.x + rvec.x; a.y += rj.y + rvec.y; a.z += rj.z + rvec.z; a.w += rj.w + rvec.w;
                            if (g.out)
                                *reinterpret_cast<float4*>(g.out + m * g.ldout + n) =
                                    make_float4(g.out_scale * a.x, g.out_scale * a.y, g.out_scale * a.z, g.out_scale * a.w);
                            if (g.pre)                     // the next GEMM of the chain reads the split (gemm_tc_supported insists on it)
                                store_split4(g.nxt_hi, g.nxt_lo, m * g.ldnxt + n,
                                             make_float4(a.x * silu_grad(yj.x), a.y * silu_grad(yj.y), a.z * silu_grad(yj.z),
                                                         a.w * silu_grad(yj.w)));
                        }
                    }
                }
                __syncwarp();                              // staging rows are rewritten by the next chunk
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                    // neither CTA leaves (or frees tensor memory) while the other may still touch it
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// half-precision split of an fp32 matrix, rows [M][K] (K a multiple of 4)
__global__ void k_split_f16(const float* __restrict__ A, int lda, int M, int K, __half* __restrict__ hi,
                            __half* __restrict__ lo) {
    const int k4 = K >> 2;
    const size_t total = (size_t)M * k4;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int m = (int)(i / k4), k = (int)(i - (size_t)m * k4) * 4;
        const float4 x = *reinterpret_cast<const float4*>(A + (size_t)m * lda + k);
        store_split4(hi, lo, (size_t)m * K + k, x);
    }
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
    static EncodeFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(p);
    }
    return fn;
}

// 2-D map over a row-major [rows][cols] half-precision matrix with row pitch ld (elements); box =
// 32 cols x 128 rows
bool make_map(CUtensorMap* map, const __half* ptr, int rows, int cols, int ld, int box_rows = BM) {
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<__half*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool gemm_tc_available() { return encode_fn() != nullptr; }

// The persistent kernel needs about one 256 x 128 item per SM to fill the machine; below half of
// that the one-tile-per-CTA kernel, with twice as many and half as long CTAs, finishes sooner.
int gemm_tc_pick_variant(int M, int N, int requested) {
    if (requested == 4) {      // two-CTA kernel where there is enough work for the pairs, else one tile per CTA
        static int n_sm4 = 0;
        if (n_sm4 == 0) {
            int dev = 0;
            if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm4, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
                n_sm4 = 148;
        }
        const int items1 = ((N + BN - 1) / BN) * ((M + BM - 1) / BM);
        return items1 <= n_sm4 ? 3 : 4;
    }
    if (requested != 2) return requested;
    static int n_sm = 0;
    if (n_sm == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            n_sm = 148;
    }
    const int items = ((N + BN - 1) / BN) * ((M + 2 * BM - 1) / (2 * BM));
    return 2 * items <= n_sm ? 3 : 2;
}

bool gemm_tc_supported(const GemmArgs& g) {
    // rows of the half-precision operands start on 16-byte boundaries (tensor-map strides, and the
    // column offset of a folded first layer); the epilogue works on four fp32 columns at a time
    const int lda_s = g.lda_split ? g.lda_split : g.K;
    if (g.mode == 1 && g.pre && !g.nxt_hi) return false;     // pre is read through the read-only path, never rewritten
    return g.A_hi && g.A_lo && g.Bt_hi && g.Bt_lo && g.M > 0 && g.N >= 4 && g.K >= 8 && (g.K & 3) == 0 &&
           (g.N & 3) == 0 && (lda_s & 7) == 0 && (g.ldbt & 7) == 0 &&
           (reinterpret_cast<uintptr_t>(g.A_hi) & 15) == 0 && (reinterpret_cast<uintptr_t>(g.A_lo) & 15) == 0 &&
           (reinterpret_cast<uintptr_t>(g.Bt_hi) & 15) == 0 && (reinterpret_cast<uintptr_t>(g.Bt_lo) & 15) == 0 &&
           encode_fn() != nullptr;
}

// column tile of the two-CTA kernel: N cut into the fewest tiles of at most 256 columns, equal widths, a
// multiple of 16 (of 32 for the fused head, whose partial sums are indexed by 32-column chunk)
int gemm_tc2_tile(int N, bool head) {
    const int tiles = (N + 255) / 256, q = head ? 32 : 16;
    int nt = ((N + tiles - 1) / tiles + q - 1) / q * q;
    return nt > 256 ? 256 : nt;
}

template <int MODE>
cudaError_t launch_tc2(const CUtensorMap& mAh, const CUtensorMap& mAl, const CUtensorMap& mBh, const CUtensorMap& mBl,
                       const GemmArgs& g, int NT, cudaStream_t st) {
    static int max_clusters = 0;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(P_THREADS); cfg.dynamicSmemBytes = C2_SMEM_BYTES; cfg.stream = st; cfg.attrs = at; cfg.numAttrs = 1;
    if (max_clusters == 0) {
        cudaError_t e = cudaFuncSetAttribute(k_gemm_tc2<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, C2_SMEM_BYTES);
        if (e != cudaSuccess) return e;
        cfg.gridDim = dim3(2 * 74);
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, k_gemm_tc2<MODE>, &cfg);      // pairs of SMs that can hold a cluster at once
        if (e != cudaSuccess) return e;
        if (n < 1) return cudaErrorInvalidConfiguration;
        max_clusters = n;
    }
    const int items = ((g.N + NT - 1) / NT) * ((g.M + 2 * BM - 1) / (2 * BM));
    const int ncl = items < max_clusters ? items : max_clusters;
    cfg.gridDim = dim3(2 * ncl);
    return cudaLaunchKernelEx(&cfg, k_gemm_tc2<MODE>, mAh, mAl, mBh, mBl, g, NT);
}

cudaError_t launch_gemm_tc(const GemmArgs& g, cudaStream_t st) {
    static bool attr_set = false;
    static int n_sm = 0;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_gemm_tc<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tc<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tcp<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tcp<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tcp<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES);
        int dev = 0;
        if (e == cudaSuccess) e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    if (!g.a_presplit) {
        const size_t total = (size_t)g.M * (g.K >> 2);
        int blocks = (int)((total + 255) / 256);
        if (blocks > 148 * 16) blocks = 148 * 16;
        k_split_f16<<<blocks, 256, 0, st>>>(g.A, g.lda, g.M, g.K, g.A_hi, g.A_lo);
    }
    CUtensorMap mAh, mAl, mBh, mBl;
    const int lda_s = g.lda_split ? g.lda_split : g.K;
    if (!make_map(&mAh, g.A_hi, g.M, g.K, lda_s) || !make_map(&mAl, g.A_lo, g.M, g.K, lda_s) ||
        !make_map(&mBh, g.Bt_hi, g.N, g.K, g.ldbt) || !make_map(&mBl, g.Bt_lo, g.N, g.K, g.ldbt))
        return cudaErrorInvalidValue;
    const int mode = g.mode == 1 ? 1 : (g.head_w ? 2 : 0);
    if (g.variant == 4) {                                  // two-CTA persistent kernel: each CTA loads half of the column tile
        const int NT = gemm_tc2_tile(g.N, mode == 2);
        if (!make_map(&mBh, g.Bt_hi, g.N, g.K, g.ldbt, NT / 2) || !make_map(&mBl, g.Bt_lo, g.N, g.K, g.ldbt, NT / 2))
            return cudaErrorInvalidValue;
        if (mode == 1) return launch_tc2<1>(mAh, mAl, mBh, mBl, g, NT, st);
        if (mode == 2) return launch_tc2<2>(mAh, mAl, mBh, mBl, g, NT, st);
        return launch_tc2<0>(mAh, mAl, mBh, mBl, g, NT, st);
    }
    if (g.variant == 3) {                                  // one 128 x 128 tile per CTA, two CTAs per SM
        dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM);
        if (mode == 1) k_gemm_tc<1><<<grid, 192, SMEM_BYTES, st>>>(mAh, mAl, mBh, mBl, g);
        else if (mode == 2) k_gemm_tc<2><<<grid, 192, SMEM_BYTES, st>>>(mAh, mAl, mBh, mBl, g);
        else k_gemm_tc<0><<<grid, 192, SMEM_BYTES, st>>>(mAh, mAl, mBh, mBl, g);
    } else {                                               // persistent, 256 x 128 items
        const int items = ((g.N + BN - 1) / BN) * ((g.M + 2 * BM - 1) / (2 * BM));
        const int grid = items < n_sm ? items : n_sm;
        if (mode == 1) k_gemm_tcp<1><<<grid, P_THREADS, P_SMEM_BYTES, st>>>(mAh, mAl, mBh, mBl, g);
        else if (mode == 2) k_gemm_tcp<2><<<grid, P_THREADS, P_SMEM_BYTES, st>>>(mAh, mAl, mBh, mBl, g);
        else k_gemm_tcp<0><<<grid, P_THREADS, P_SMEM_BYTES, st>>>(mAh, mAl, mBh, mBl, g);
    }
    return cudaGetLastError();
}

}  // namespace umd
