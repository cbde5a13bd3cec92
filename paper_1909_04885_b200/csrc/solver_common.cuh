// Device helpers shared by the local-solver kernels: mbarrier / cp.async wrappers, the per-step header that the
// staging warps prepare, and the scalar coordinate steps of the three losses.
#pragma once

#include <math_constants.h>

#include "chicle_internal.cuh"

namespace chicle {

constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int kNewtonIters = 5;

struct SlotHdr {
    int64_t row_start;
    int32_t coord;
    int32_t nnz;
    float p0, p1, p2, p3;
    int32_t pad[2];
};
static_assert(sizeof(SlotHdr) == 40 || sizeof(SlotHdr) == 48, "header size");

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
    float lam_n, inv_n, lambda, sigma;
    int cap, nslot, multi_epoch;
};

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
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Bounded wait. Returns false when the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 31u) == 31u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicOr(status, ST_WAIT_TIMEOUT);
    return false;
}

__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Scalar steps. `dot` is x_c . v_local (dual) or c_j . (v_local - y) (ridge). Returns delta and the new state.
template <int LOSS>
__device__ __forceinline__ void coordinate_step(float dot, const SlotHdr &h, float &delta, float &new_state)
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
        // Root of z + q sigmoid(z) = c on its convex branch (after reflecting a positive root), Newton from a
        // Lambert-W-like start, fixed iteration count.
        const float q = h.p2, a = h.p1;
        const float m = dot * h.p0;
        float c = fmaf(q, a, -m);
        const bool flip = c > 0.5f * q;
        if (flip) c = q - c;
        const float kappa = q > 0.0f ? __logf(q) + c : -CUDART_INF_F;
        float z = kappa <= 0.0f ? fminf(c, 0.0f) : fminf(c - (kappa - __logf(1.0f + kappa)), 0.0f);
#pragma unroll
        for (int it = 0; it < kNewtonIters; ++it) {
            const float e = __expf(z);
            const float r = __frcp_rn(1.0f + e);
            const float p = e * r;
            const float F = fmaf(q, p, z) - c;
            const float Fp = fmaf(q * p, r, 1.0f); // 1 + q p (1 - p), 1 - p = 1 / (1 + e)
            z = fminf(z - __fdividef(F, Fp), 0.0f);
        }
        const float e = __expf(z);
        const float r = __frcp_rn(1.0f + e);
        const float a_new = flip ? r : e * r;
        delta = h.p3 * (a_new - a);
        new_state = h.p3 * a_new;
    }
}


} // namespace chicle
