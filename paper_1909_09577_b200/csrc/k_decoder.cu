// Decoder tail and evaluation-mode helpers: log-softmax over the class (channel) axis with its adjoint,
// and the per-channel 1/sqrt(var + eps) that turns running variances into the factor the apply kernel takes.
// One thread owns one (sample, frame) position and walks the channels (stride T'): loads of a warp are
// contiguous in time, and the handful of classes of a CTC head makes the channel loop short.
#include "common.cuh"
#include "kernels.h"

namespace sc {
namespace {

// The class scores z arrive in float32 (the contraction's accumulators, not yet rounded to the activation type):
// rounding them first would put an error of half a unit of the activation type into every log-probability twice.
template <typename T>
__global__ void __launch_bounds__(256)
log_softmax_fwd_kernel(const float* __restrict__ z, T* __restrict__ y, const int* __restrict__ len_out, int B, int C, int Tp) {
    pdl_sync();
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    if (idx >= (long long)B * Tp) return;
    const int b = (int)(idx / Tp), t = (int)(idx - (long long)b * Tp);
    const size_t off = (size_t)b * C * Tp + t;
    if (t >= min(len_out[b], Tp)) {
        for (int c = 0; c < C; ++c) stf(y + off + (size_t)c * Tp, 0.f);
        return;
    }
    const float* p = z + off;
    float m = -INFINITY;
    for (int c = 0; c < C; ++c) m = fmaxf(m, p[(size_t)c * Tp]);
    float s = 0.f;
    for (int c = 0; c < C; ++c) s += expf(p[(size_t)c * Tp] - m);
    const float lse = m + logf(s);
    for (int c = 0; c < C; ++c) stf(y + off + (size_t)c * Tp, p[(size_t)c * Tp] - lse);
}

// dz[c] = [t < len] * (g[c] - exp(logp[c]) * sum_c' g[c'])
template <typename T>
__global__ void __launch_bounds__(256)
log_softmax_bwd_kernel(T* __restrict__ dz, const T* __restrict__ g, const T* __restrict__ logp,
                       const int* __restrict__ len_out, int B, int C, int Tp) {
    pdl_sync();
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    if (idx >= (long long)B * Tp) return;
    const int b = (int)(idx / Tp), t = (int)(idx - (long long)b * Tp);
    const size_t off = (size_t)b * C * Tp + t;
    if (t >= min(len_out[b], Tp)) {
        for (int c = 0; c < C; ++c) stf(dz + off + (size_t)c * Tp, 0.f);
        return;
    }
    float sg = 0.f;
    for (int c = 0; c < C; ++c) sg += ldf(g + off + (size_t)c * Tp);
    for (int c = 0; c < C; ++c) {
        const size_t o = off + (size_t)c * Tp;
        stf(dz + o, ldf(g + o) - expf(ldf(logp + o)) * sg);
    }
}

__global__ void invstd_from_var_kernel(const float* __restrict__ var, float eps, float* __restrict__ invstd, int C) {
    pdl_sync();
    const int o = blockIdx.x * blockDim.x + threadIdx.x;
    if (o < C) invstd[o] = 1.f / sqrtf(var[o] + eps);
}

}  // namespace

#define SC_DISPATCH(dtype, ...)                                             \
    switch (dtype) {                                                        \
        case F32: { using T = float; __VA_ARGS__; break; }                  \
        case F16: { using T = __half; __VA_ARGS__; break; }                 \
        default:  { using T = __nv_bfloat16; __VA_ARGS__; break; }          \
    }

void log_softmax_fwd(const Launch& L, int dtype, const float* z, void* y, const int* len_out, int B, int C, int Tp) {
    KScope ks_(L, KC_EW, (4.0 + dtype_size(dtype)) * B * C * Tp, 0.0);
    const unsigned grid = (unsigned)(((long long)B * Tp + 255) / 256);
    SC_DISPATCH(dtype, (launch_k(L, log_softmax_fwd_kernel<T>, grid, 256, 0, z, (T*)y, len_out, B, C, Tp)));
    L.count();
}

void log_softmax_bwd(const Launch& L, int dtype, void* dz, const void* g, const void* logp, const int* len_out, int B,
                     int C, int Tp) {
    KScope ks_(L, KC_EW, 3.0 * dtype_size(dtype) * B * C * Tp, 0.0);
    const unsigned grid = (unsigned)(((long long)B * Tp + 255) / 256);
    SC_DISPATCH(dtype, (launch_k(L, log_softmax_bwd_kernel<T>, grid, 256, 0, (T*)dz, (const T*)g, (const T*)logp, len_out, B, C, Tp)));
    L.count();
}

void invstd_from_var(const Launch& L, const float* var, float eps, float* invstd, int C) {
    KScope ks_(L, KC_EW, 8.0 * C, 0.0);
    launch_k(L, invstd_from_var_kernel, (C + 255) / 256, 256, 0, var, eps, invstd, C);
    L.count();
}

}  // namespace sc
