// Non-separable K-tap convolution over time (the convolution of the original Jasper block, which the separable block
// factorises) as plain SIMT tiled contractions with fp32 accumulation: a block variant, not the hot path.
//   forward          v[b,o,t']  = sum_{c,k} w[o,c,k] * xm[b,c,t'*s + k*dil - P]          (xm: x, zero outside [0, len_in[b]))
//   input gradient   dx[b,c,t]  = sum_{o,k} w[o,c,k] * gv[b,o,(t + P - k*dil) / s]       (terms with a whole quotient in [0, len_out[b]))
//   weight gradient  dw[o,c,k]  = sum_{b,t'} gv[b,o,t'] * xm[b,c,t'*s + k*dil - P]
// Each is the pointwise contraction of k_gemm_simt.cu repeated over the taps with a shifted, bounds-checked operand:
// 64 x 64 output tile, 16-deep steps, 4 x 4 outputs per thread.
#include <algorithm>

#include "common.cuh"
#include "kernels.h"

namespace sc {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, NT = 256;

struct ConvGeom { int B, Cin, Cout, T, Tp, K, s, dil, P; };

template <typename X> struct IsHalfT { static constexpr bool value = false; };
template <> struct IsHalfT<__half> { static constexpr bool value = true; };

__device__ __forceinline__ void fma_tile(const float (&As)[BK][BM + 4], const float (&Bs)[BK][BN + 4], int tx, int ty, float (&acc)[4][4]) {
#pragma unroll
    for (int k = 0; k < BK; ++k) {
        const float4 av = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
        const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
        const float aa[4] = {av.x, av.y, av.z, av.w}, bb[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(aa[i], bb[j], acc[i][j]);
    }
}

template <typename T, typename OT>
__global__ void __launch_bounds__(NT)
conv_fwd_kernel(ConvGeom g, const T* __restrict__ w, const T* __restrict__ x, OT* __restrict__ out, const float* __restrict__ bias,
                const int* __restrict__ len_in, const int* __restrict__ len_out, int* status) {
    pdl_sync();
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int b = blockIdx.z, m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const int lo = min(len_out[b], g.Tp), li = min(len_in[b], g.T);
    OT* o = out + (long long)b * g.Cout * g.Tp;
    if (n0 >= lo) {                           // tile wholly in padding
        for (int i = tid; i < BM * BN; i += NT) {
            const int m = m0 + i / BN, n = n0 + i % BN;
            if (m < g.Cout && n < g.Tp) stf(o + (long long)m * g.Tp + n, 0.f);
        }
        return;
    }
    float acc[4][4] = {};
    const T* xb = x + (long long)b * g.Cin * g.T;
    for (int k = 0; k < g.K; ++k) {
        const int shift = k * g.dil - g.P;
        for (int c0 = 0; c0 < g.Cin; c0 += BK) {
            for (int i = tid; i < BM * BK; i += NT) {
                const int kk = i % BK, m = i / BK;
                const int gm = m0 + m, gc = c0 + kk;
                As[kk][m] = (gm < g.Cout && gc < g.Cin) ? ldf(w + ((long long)gm * g.Cin + gc) * g.K + k) : 0.f;
            }
            for (int i = tid; i < BN * BK; i += NT) {
                const int n = i % BN, kk = i / BN;
                const int gc = c0 + kk, tin = (n0 + n) * g.s + shift;
                Bs[kk][n] = (gc < g.Cin && tin >= 0 && tin < li) ? ldf(xb + (long long)gc * g.T + tin) : 0.f;
            }
            __syncthreads();
            fma_tile(As, Bs, tx, ty, acc);
            __syncthreads();
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= g.Cout) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= g.Tp) continue;
            float v = acc[i][j] + (bias ? bias[m] : 0.f);
            if (n >= lo) v = 0.f;
            if (IsHalfT<OT>::value && fabsf(v) > 65504.f) { v = copysignf(65504.f, v); raise_status(status, kErrRange); }
            stf(o + (long long)m * g.Tp + n, v);
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(NT)
conv_dgrad_kernel(ConvGeom g, const T* __restrict__ w, const T* __restrict__ gv, T* __restrict__ dx,
                  const int* __restrict__ len_in, const int* __restrict__ len_out) {
    pdl_sync();
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int b = blockIdx.z, m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;      // m: input channel, n: input frame
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const int lo = min(len_out[b], g.Tp), li = min(len_in[b], g.T);
    T* o = dx + (long long)b * g.Cin * g.T;
    if (n0 >= li) {
        for (int i = tid; i < BM * BN; i += NT) {
            const int m = m0 + i / BN, n = n0 + i % BN;
            if (m < g.Cin && n < g.T) stf(o + (long long)m * g.T + n, 0.f);
        }
        return;
    }
    float acc[4][4] = {};
    const T* gb = gv + (long long)b * g.Cout * g.Tp;
    for (int k = 0; k < g.K; ++k) {
        const int shift = g.P - k * g.dil;
        for (int o0 = 0; o0 < g.Cout; o0 += BK) {
            for (int i = tid; i < BM * BK; i += NT) {
                const int m = i % BM, kk = i / BM;
                const int gm = m0 + m, go = o0 + kk;
                As[kk][m] = (gm < g.Cin && go < g.Cout) ? ldf(w + ((long long)go * g.Cin + gm) * g.K + k) : 0.f;
            }
            for (int i = tid; i < BN * BK; i += NT) {
                const int n = i % BN, kk = i / BN;
                const int go = o0 + kk, q = n0 + n + shift;
                float v = 0.f;
                if (go < g.Cout && q >= 0) {
                    const int tp = q / g.s;
                    if (tp * g.s == q && tp < lo) v = ldf(gb + (long long)go * g.Tp + tp);
                }
                Bs[kk][n] = v;
            }
            __syncthreads();
            fma_tile(As, Bs, tx, ty, acc);
            __syncthreads();
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= g.Cin) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= g.T) continue;
            stf(o + (long long)m * g.T + n, n < li ? acc[i][j] : 0.f);      // the input was masked: no gradient beyond len_in
        }
    }
}

// z = tap * nslices + slice; slice sl sums the samples sl, sl + nslices, ...
template <typename T>
__global__ void __launch_bounds__(NT)
conv_wgrad_kernel(ConvGeom g, int nslices, const T* __restrict__ gv, const T* __restrict__ x, float* __restrict__ partials,
                  const int* __restrict__ len_in, const int* __restrict__ len_out) {
    pdl_sync();
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int k = blockIdx.z / nslices, sl = blockIdx.z % nslices;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;                        // m: output channel, n: input channel
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const int shift = k * g.dil - g.P;
    float acc[4][4] = {};
    for (int b = sl; b < g.B; b += nslices) {
        const int lo = min(len_out[b], g.Tp), li = min(len_in[b], g.T);
        const T* gb = gv + (long long)b * g.Cout * g.Tp;
        const T* xb = x + (long long)b * g.Cin * g.T;
        for (int t0 = 0; t0 < lo; t0 += BK) {
            for (int i = tid; i < BM * BK; i += NT) {
                const int kk = i % BK, m = i / BK;
                const int gm = m0 + m, t = t0 + kk;
                As[kk][m] = (gm < g.Cout && t < lo) ? ldf(gb + (long long)gm * g.Tp + t) : 0.f;
            }
            for (int i = tid; i < BN * BK; i += NT) {
                const int kk = i % BK, n = i / BK;
                const int gc = n0 + n, tin = (t0 + kk) * g.s + shift;
                Bs[kk][n] = (gc < g.Cin && t0 + kk < lo && tin >= 0 && tin < li) ? ldf(xb + (long long)gc * g.T + tin) : 0.f;
            }
            __syncthreads();
            fma_tile(As, Bs, tx, ty, acc);
            __syncthreads();
        }
    }
    float* p = partials + (long long)sl * g.Cout * g.Cin * g.K;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= g.Cout) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n < g.Cin) p[((long long)m * g.Cin + n) * g.K + k] = acc[i][j];
        }
    }
}

ConvGeom geom(int B, int Cin, int Cout, int T, int Tp, int K, int s, int dil) {
    return ConvGeom{B, Cin, Cout, T, Tp, K, s, dil, (dil * (K - 1)) / 2};
}
int wgrad_slices(int B) { return std::min(B, 4); }

}  // namespace

#define SC_DISPATCH(dtype, ...)                                             \
    switch (dtype) {                                                        \
        case F32: { using T = float; __VA_ARGS__; break; }                  \
        case F16: { using T = __half; __VA_ARGS__; break; }                 \
        default:  { using T = __nv_bfloat16; __VA_ARGS__; break; }          \
    }

void conv_fwd_simt(const Launch& L, int dtype, const void* w, const void* x, const float* bias, void* v, int out_dtype,
                   const int* len_in, const int* len_out, int B, int Cin, int Cout, int T, int Tp, int K, int stride, int dil) {
    KScope ks_(L, KC_PW_FWD, (double)B * (dtype_size(dtype) * (double)Cin * T + dtype_size(out_dtype) * (double)Cout * Tp),
               2.0 * B * Tp * Cin * Cout * K);
    const ConvGeom g = geom(B, Cin, Cout, T, Tp, K, stride, dil);
    dim3 grid((Tp + BN - 1) / BN, (Cout + BM - 1) / BM, B);
    if (out_dtype == dtype) {
        SC_DISPATCH(dtype, (launch_k(L, conv_fwd_kernel<T, T>, grid, NT, 0, g, (const T*)w, (const T*)x, (T*)v, bias, len_in, len_out, L.status)));
    } else {      // bfloat16 operands, float16 result (the type v is kept in)
        launch_k(L, conv_fwd_kernel<__nv_bfloat16, __half>, grid, NT, 0, g, (const __nv_bfloat16*)w, (const __nv_bfloat16*)x, (__half*)v,
                 bias, len_in, len_out, L.status);
    }
    L.count();
}

void conv_dgrad_simt(const Launch& L, int dtype, const void* w, const void* gv, void* dx, const int* len_in, const int* len_out,
                     int B, int Cin, int Cout, int T, int Tp, int K, int stride, int dil) {
    KScope ks_(L, KC_PW_DGRAD, (double)dtype_size(dtype) * B * ((double)Cin * T + (double)Cout * Tp), 2.0 * B * Tp * Cin * Cout * K);
    const ConvGeom g = geom(B, Cin, Cout, T, Tp, K, stride, dil);
    dim3 grid((T + BN - 1) / BN, (Cin + BM - 1) / BM, B);
    SC_DISPATCH(dtype, (launch_k(L, conv_dgrad_kernel<T>, grid, NT, 0, g, (const T*)w, (const T*)gv, (T*)dx, len_in, len_out)));
    L.count();
}

size_t conv_wgrad_scratch_bytes(int B, int Cin, int Cout, int K) {
    return (size_t)wgrad_slices(B) * Cin * Cout * K * sizeof(float);
}

void conv_wgrad_simt(const Launch& L, int dtype, const void* gv, const void* x, float* dw, float* partials, int accumulate,
                     const int* len_in, const int* len_out, int B, int Cin, int Cout, int T, int Tp, int K, int stride, int dil) {
    const int ns = wgrad_slices(B);
    {
        KScope ks_(L, KC_PW_WGRAD, (double)dtype_size(dtype) * B * ((double)Cin * T + (double)Cout * Tp), 2.0 * B * Tp * Cin * Cout * K);
        const ConvGeom g = geom(B, Cin, Cout, T, Tp, K, stride, dil);
        dim3 grid((Cin + BN - 1) / BN, (Cout + BM - 1) / BM, K * ns);
        SC_DISPATCH(dtype, (launch_k(L, conv_wgrad_kernel<T>, grid, NT, 0, g, ns, (const T*)gv, (const T*)x, partials, len_in, len_out)));
        L.count();
    }
    reduce_partials(L, partials, ns, (int64_t)Cin * Cout * K, dw, accumulate, nullptr);
}

}  // namespace sc
