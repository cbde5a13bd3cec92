// Device helpers shared by the local-solver kernels: mbarrier / cp.async wrappers, the per-step header that the
// staging warps prepare, and the scalar coordinate steps of the three losses.
#pragma once

#include <math_constants.h>

#include "chicle_internal.cuh"

namespace chicle {

constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int kRootIters = 2; // Halley steps of the logistic root (see logistic_root)

// Per-step header prepared by the staging warps. 48 bytes, 16-byte aligned, so that the chain reads it with two
// 128-bit shared-memory loads: {row_start, coord, nnz} and {p0, p1, p2, p3}.
struct alignas(16) SlotHdr {
    int64_t row_start;
    int32_t coord;
    int32_t nnz;
    float p0, p1, p2, p3;
    int32_t pad[4];
};
static_assert(sizeof(SlotHdr) == 48, "header size");

// Explicit shared-memory accesses with 32-bit addresses. The chain's loops are latency-bound; generic-address
// loads through pointers the compiler cannot prove to be shared cost several times more per access.
__device__ __forceinline__ float lds_f32(uint32_t a)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t a)
{
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ float4 lds_f32x4(uint32_t a)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ int4 lds_s32x4(uint32_t a)
{
    int4 v;
    asm volatile("ld.shared.v4.s32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void sts_f32(uint32_t a, float v)
{
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(v) : "memory");
}

__device__ __forceinline__ int32_t lds_s32(uint32_t a)
{
    int32_t v;
    asm volatile("ld.shared.s32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void sts_s32(uint32_t a, int32_t v)
{
    asm volatile("st.shared.s32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void sts_u16(uint32_t a, uint32_t v)
{
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"((uint16_t)v) : "memory");
}
__device__ __forceinline__ int32_t atoms_cas(uint32_t a, int32_t expect, int32_t v)
{
    int32_t old;
    asm volatile("atom.shared.cas.b32 %0, [%1], %2, %3;" : "=r"(old) : "r"(a), "r"(expect), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ int32_t atoms_add(uint32_t a, int32_t v)
{
    int32_t old;
    asm volatile("atom.shared.add.s32 %0, [%1], %2;" : "=r"(old) : "r"(a), "r"(v) : "memory");
    return old;
}

// Sum over the warp through a 32-float shared-memory buffer: every lane stores its partial, then reads all 32 with
// eight 128-bit loads and adds them in a fixed tree. About 100 cycles against about 150 for five shuffle rounds.
// `buf` must be 16-byte aligned; the caller separates successive uses with __syncwarp().
__device__ __forceinline__ float warp_sum_smem(float x, uint32_t buf, int lane)
{
    sts_f32(buf + 4u * lane, x);
    __syncwarp();
    const float4 a0 = lds_f32x4(buf), a1 = lds_f32x4(buf + 16), a2 = lds_f32x4(buf + 32), a3 = lds_f32x4(buf + 48);
    const float4 a4 = lds_f32x4(buf + 64), a5 = lds_f32x4(buf + 80), a6 = lds_f32x4(buf + 96), a7 = lds_f32x4(buf + 112);
    const float s0 = (a0.x + a0.y) + (a0.z + a0.w), s1 = (a1.x + a1.y) + (a1.z + a1.w);
    const float s2 = (a2.x + a2.y) + (a2.z + a2.w), s3 = (a3.x + a3.y) + (a3.z + a3.w);
    const float s4 = (a4.x + a4.y) + (a4.z + a4.w), s5 = (a5.x + a5.y) + (a5.z + a5.w);
    const float s6 = (a6.x + a6.y) + (a6.z + a6.w), s7 = (a7.x + a7.y) + (a7.z + a7.w);
    return ((s0 + s1) + (s2 + s3)) + ((s4 + s5) + (s6 + s7));
}

struct SolverParams {
    const int64_t *indptr;
    const int32_t *indices;
    const float *values;
    const float *labels;
    const float *sqnorm;
    float *alpha;
    const float *vbase; // v (dual losses) or v - y (ridge)
    float *U;           // K x dim
    const int64_t *part_off;
    const int32_t *perm; // epochs x n_coord
    uint32_t *status;
    int64_t n_coord, dim, H;
    const int64_t *steps_k; // K step budgets of this round, one per partition (each at most its size), or nullptr: H rules
    const int64_t *first_k; // look-ahead solver only: where in its visiting order each partition starts in this launch
                            // (a round cut into slices), or nullptr: at the start
    float lam_n, inv_n, lambda, sigma;
    int cap, nslot, multi_epoch;
};

// Coordinate steps partition k (of nk coordinates) takes this round.
__device__ __forceinline__ int64_t partition_steps(const SolverParams &P, int64_t k, int64_t nk)
{
    if (nk <= 0) return 0;
    if (P.steps_k) return P.steps_k[k];
    return P.H == 0 ? nk : P.H;
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t a, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t a)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(a) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t a, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(a), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_arrive_noinc(uint32_t bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
// Bulk copy global -> shared by the copy engine (no load/store-unit traffic on the SM); both addresses and the size
// must be multiples of 16 bytes. Completion is counted in bytes on an mbarrier.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Bounded wait for a whole warp (every lane must call it). Lane 0 polls, backing off with nanosleep so that waiting
// warps do not crowd the shared-memory pipeline that the latency-bound chain warp depends on; the others are parked
// at the warp barrier. Returns false when the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status)
{
    int ok = 1;
    if ((threadIdx.x & 31) == 0) {
        ok = 0;
        for (uint32_t it = 0; it < kSpinLimit; ++it) {
            if (mbar_try_wait(bar, parity)) { ok = 1; break; }
            if (it >= 2) __nanosleep(it < 64 ? 32 : 256);
            if ((it & 31u) == 31u && *abort_flag) break;
        }
        if (!ok && !*abort_flag) {
            *abort_flag = 1;
            atomicOr(status, ST_WAIT_TIMEOUT);
        }
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    __syncwarp();
    return ok != 0;
}

__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// a' = sigmoid(z) at the root of F(z) = z + q sigmoid(z) - c: the root is taken on the convex branch z <= 0 (a positive
// root is reflected first), from a Lambert-W-like start, by two Halley steps (cubic convergence): they leave 5.9e-7 in
// a' against the exact root over q in [1e-3, 1e6], |m| <= 60 in an fp32 emulation (three Newton steps: 2.1e-7, four:
// 1.8e-7, the fp32 floor). Measured on the logistic configuration (the recurrence is one dependent chain of these
// solves): two Halley steps 296 ns per coordinate step, three Newton steps 338 ns, four Newton steps 297 ns.
// `log_q` is log(q) (-inf for q = 0): a constant of the coordinate, so callers that prepare their constants ahead pass it.
__device__ __forceinline__ float logistic_root(float c, float q, float log_q)
{
    const bool flip = c > 0.5f * q;
    if (flip) c = q - c;
    const float kappa = log_q + c;
    float z = kappa <= 0.0f ? fminf(c, 0.0f) : fminf(c - (kappa - __logf(1.0f + kappa)), 0.0f);
#pragma unroll
    for (int it = 0; it < kRootIters; ++it) {
        // with e = exp z, s = 1 + e: F = A / s, F' = B / s^2, F'' = C / s^3 for A = (z - c) s + q e, B = s^2 + q e,
        // C = q e (1 - e); the Halley step 2 F F' / (2 F'^2 - F F'') = 2 A B s / (2 B^2 - A C)
        const float e = __expf(z);
        const float s = 1.0f + e, qe = q * e;
        const float A = fmaf(z - c, s, qe), B = fmaf(s, s, qe), C = qe * (1.0f - e);
        z = fminf(z - __fdividef(2.0f * A * B * s, fmaf(2.0f * B, B, -A * C)), 0.0f);
    }
    const float e = __expf(z);
    const float r = __frcp_rn(1.0f + e);
    return flip ? r : e * r;
}

__device__ __forceinline__ float logistic_root(float c, float q)
{
    return logistic_root(c, q, q > 0.0f ? __logf(q) : -CUDART_INF_F);
}

// Scalar steps. `dot` is x_c . v_local (dual) or c_j . (v_local - y) (ridge). Returns delta and the new state.
template <int LOSS, class Hdr>
__device__ __forceinline__ void coordinate_step(float dot, const Hdr &h, float &delta, float &new_state)
{
    if (LOSS == CHICLE_LOSS_RIDGE_PRIMAL) {
        // p0 = 1/n, p1 = w_j, p2 = 1 / (sigma' |c_j|^2 / n + lambda), p3 = lambda
        const float g = fmaf(dot, h.p0, h.p3 * h.p1);
        delta = -g * h.p2;
        new_state = h.p1 + delta;
    } else if (LOSS == CHICLE_LOSS_HINGE_DUAL) {
        // p0 = y / (lambda n), p1 = a, p2 = lambda n / (sigma' |x|^2) (inf for a zero row), p3 = y
        const float m = dot * h.p0;
        const float t = fmaf(1.0f - m, h.p2, h.p1);
        const float a_new = fminf(fmaxf(t, 0.0f), 1.0f);
        delta = h.p3 * (a_new - h.p1);
        new_state = h.p3 * a_new;
    } else {
        // logistic: p0 = y / (lambda n), p1 = a, p2 = q = sigma' |x|^2 / (lambda n), p3 = y.
        const float q = h.p2, a = h.p1;
        const float a_new = logistic_root(fmaf(q, a, -(dot * h.p0)), q);
        delta = h.p3 * (a_new - a);
        new_state = h.p3 * a_new;
    }
}


} // namespace chicle
