// Depthwise (per-channel) correlation over time: forward, input gradient, tap gradient.
//
// Stride-1 layers (all but the first layer of the encoder) use register-blocked kernels: a thread
// owns R consecutive outputs, keeps a 2R-wide sliding window of the shared-memory tile and R taps
// in registers and performs R*R FMAs per 2R shared loads.  The input gradient of a stride-1
// correlation is the same correlation with flipped taps, so one kernel serves both.  Any other
// stride goes through plain tiled kernels.
#include "common.cuh"
#include "kernels.h"
#include <type_traits>
#include <algorithm>

namespace sc {
namespace {

constexpr int R = 8;          // outputs (or taps) per thread
constexpr int CH = 8;         // channels per CTA in the stride-1 kernel (one warp each)
constexpr int TT = 32 * R;    // outputs per channel per CTA

// Conflict-free placement for 16-byte shared loads at an 8-float lane pitch.
__device__ __forceinline__ int phys(int i) { return i + ((i >> 5) << 2); }

// Saturating store for half outputs: a value outside the half range is clamped and reported.
template <typename TO>
__device__ __forceinline__ void guard_range(float (&acc)[8], int* status) {
    if (sizeof(TO) == 2 && !std::is_same<TO, __nv_bfloat16>::value) {
        bool over = false;
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            if (fabsf(acc[r]) > 65504.f) { over = true; acc[r] = copysignf(65504.f, acc[r]); }
        }
        if (over) raise_status(status, kErrRange);
    }
}

template <typename TI, typename TW, typename TO>
__global__ void __launch_bounds__(32 * CH)
dw_corr_s1_kernel(const TI* __restrict__ in, const TW* __restrict__ w, TO* __restrict__ out,
                  const TO* __restrict__ add1, const TO* __restrict__ add2, const float* __restrict__ gmax,
                  const int* __restrict__ len_src, const int* __restrict__ len_dst,
                  int C, int Tt, int K, int Kpad, int flip, int* status) {
    pdl_sync();
    using T = TO;
    extern __shared__ float smem[];
    const int lane = threadIdx.x, wrp = threadIdx.y;
    const int b = blockIdx.z, c = blockIdx.y * CH + wrp, t0 = blockIdx.x * TT;
    if (c >= C) return;                       // warps are independent: no CTA-wide barrier below
    const int P = (K - 1) / 2;
    const int XW = TT + Kpad;                 // logical tile width
    float* xs = smem + (size_t)wrp * (phys(XW) + 4 + Kpad);
    float* ws = xs + phys(XW) + 4;
    const int ls = min(len_src[b], Tt), ld = min(len_dst[b], Tt);
    const size_t row = ((size_t)b * C + c) * Tt;
    T* orow = out + row;
    const bool vec = (Tt % 8 == 0);

    if (t0 >= ld) {                           // tile lies wholly in padding: zeros
        float z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        const int t = t0 + lane * R;
        if (vec) { if (t < Tt) st8<T>(orow + t, z); }
        else { for (int r = 0; r < R; ++r) if (t + r < Tt) stf(orow + t + r, 0.f); }
        return;
    }
    // taps (zero padded to Kpad)
    for (int k = lane; k < Kpad; k += 32)
        ws[k] = (k < K) ? ldf(w + (size_t)c * K + (flip ? K - 1 - k : k)) : 0.f;
    // input tile: logical index i <-> frame tau = t0 - P + i, zero outside [0, ls)
    const TI* irow = in + row;
    const int tau0 = t0 - P;
    if (vec) {
        const int a0 = (tau0 >= 0) ? (tau0 & ~7) : -(((-tau0) + 7) & ~7);   // floor to a multiple of 8
        const int nchunk = (tau0 + XW - a0 + 7) / 8;
        for (int j = lane; j < nchunk; j += 32) {
            const int ta = a0 + 8 * j;
            float f[8];
            if (ta >= 0 && ta < ls) ld8<TI>(irow + ta, f);
            else {
#pragma unroll
                for (int e = 0; e < 8; ++e) f[e] = 0.f;
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int i = ta + e - tau0;
                if (i >= 0 && i < XW) xs[phys(i)] = (ta + e < ls) ? f[e] : 0.f;
            }
        }
    } else {
        for (int i = lane; i < XW; i += 32) {
            const int tau = tau0 + i;
            xs[phys(i)] = (tau >= 0 && tau < ls) ? ldf(irow + tau) : 0.f;
        }
    }
    __syncwarp();

    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.f;
    float win[2 * R];
    const int base = lane * R;
    {
        const float4 a = *reinterpret_cast<const float4*>(xs + phys(base));
        const float4 bq = *reinterpret_cast<const float4*>(xs + phys(base + 4));
        win[0] = a.x; win[1] = a.y; win[2] = a.z; win[3] = a.w;
        win[4] = bq.x; win[5] = bq.y; win[6] = bq.z; win[7] = bq.w;
    }
    for (int kk = 0; kk < Kpad; kk += R) {
        const float4 a = *reinterpret_cast<const float4*>(xs + phys(base + kk + R));
        const float4 bq = *reinterpret_cast<const float4*>(xs + phys(base + kk + R + 4));
        win[8] = a.x; win[9] = a.y; win[10] = a.z; win[11] = a.w;
        win[12] = bq.x; win[13] = bq.y; win[14] = bq.z; win[15] = bq.w;
        const float4 w0 = *reinterpret_cast<const float4*>(ws + kk);
        const float4 w1 = *reinterpret_cast<const float4*>(ws + kk + 4);
        const float wv[R] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int q = 0; q < R; ++q)
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r] = fmaf(wv[q], win[r + q], acc[r]);
#pragma unroll
        for (int r = 0; r < R; ++r) win[r] = win[r + R];
    }

    const int t = t0 + base;
    if (t >= Tt) return;
    if (gmax) {
        const float inv = 1.f / pow2_scale(*gmax);
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r] *= inv;
    }
    guard_range<TO>(acc, status);
    if (vec) {
        if (add1) { float f[8]; ld8<T>(add1 + row + t, f);
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r] += f[r]; }
        if (add2) { float f[8]; ld8<T>(add2 + row + t, f);
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r] += f[r]; }
#pragma unroll
        for (int r = 0; r < R; ++r) if (t + r >= ld) acc[r] = 0.f;
        st8<T>(orow + t, acc);
    } else {
        for (int r = 0; r < R; ++r) {
            if (t + r >= Tt) break;
            float q = acc[r];
            if (add1) q += ldf(add1 + row + t + r);
            if (add2) q += ldf(add2 + row + t + r);
            stf(orow + t + r, (t + r < ld) ? q : 0.f);
        }
    }
}

// ---- any stride: plain tiled kernels (used by the stride-2 first layer) ---------------------
constexpr int GT = 256;   // outputs per CTA

template <typename T, typename TO>
__global__ void __launch_bounds__(GT)
dw_fwd_generic_kernel(const T* __restrict__ x, const T* __restrict__ w, TO* __restrict__ u,
                      const int* __restrict__ len_in, const int* __restrict__ len_out,
                      int C, int Tt, int Tp, int K, int s, int dil, int* status) {
    pdl_sync();
    extern __shared__ float smem[];
    const int b = blockIdx.z, c = blockIdx.y, t0 = blockIdx.x * GT;
    const int P = (dil * (K - 1)) / 2, XW = (GT - 1) * s + (K - 1) * dil + 1;
    float* xs = smem;
    float* ws = smem + XW;
    const int li = min(len_in[b], Tt), lo = min(len_out[b], Tp);
    const T* xrow = x + ((size_t)b * C + c) * Tt;
    for (int k = threadIdx.x; k < K; k += GT) ws[k] = ldf(w + (size_t)c * K + k);
    const int tau0 = t0 * s - P;
    for (int i = threadIdx.x; i < XW; i += GT) {
        const int tau = tau0 + i;
        xs[i] = (tau >= 0 && tau < li) ? ldf(xrow + tau) : 0.f;
    }
    __syncthreads();
    const int t = t0 + threadIdx.x;
    if (t >= Tp) return;
    float acc = 0.f;
    for (int k = 0; k < K; ++k) acc = fmaf(ws[k], xs[threadIdx.x * s + k * dil], acc);
    if (std::is_same<TO, __half>::value && fabsf(acc) > 65504.f) { acc = copysignf(65504.f, acc); raise_status(status, kErrRange); }
    stf(u + ((size_t)b * C + c) * Tp + t, (t < lo) ? acc : 0.f);
}

template <typename TG, typename T>
__global__ void __launch_bounds__(GT)
dw_dgrad_generic_kernel(const TG* __restrict__ gu, const T* __restrict__ w, T* __restrict__ dx,
                        const T* __restrict__ add1, const T* __restrict__ add2, const float* __restrict__ gmax,
                        const int* __restrict__ len_in, const int* __restrict__ len_out,
                        int C, int Tt, int Tp, int K, int s, int dil) {
    pdl_sync();
    extern __shared__ float smem[];
    const int b = blockIdx.z, c = blockIdx.y, tau0 = blockIdx.x * GT;
    const int P = (dil * (K - 1)) / 2;
    // outputs tau0..tau0+GT-1 read gu[t] for t in [tlo, thi]
    const int num = tau0 + P - (K - 1) * dil;
    const int tlo = (num >= 0) ? (num + s - 1) / s : -((-num) / s);
    const int thi = (tau0 + GT - 1 + P) / s;
    const int GW = thi - tlo + 1;
    float* gs = smem;
    float* ws = smem + GW;
    const int li = min(len_in[b], Tt), lo = min(len_out[b], Tp);
    const TG* grow = gu + ((size_t)b * C + c) * Tp;
    for (int k = threadIdx.x; k < K; k += GT) ws[k] = ldf(w + (size_t)c * K + k);
    for (int i = threadIdx.x; i < GW; i += GT) {
        const int t = tlo + i;
        gs[i] = (t >= 0 && t < lo) ? ldf(grow + t) : 0.f;
    }
    __syncthreads();
    const int tau = tau0 + threadIdx.x;
    if (tau >= Tt) return;
    float acc = 0.f;
    for (int k = 0; k < K; ++k) {
        const int q = tau + P - k * dil;
        if (q >= 0 && q % s == 0) { const int t = q / s; if (t >= tlo && t <= thi) acc = fmaf(ws[k], gs[t - tlo], acc); }
    }
    const size_t o = ((size_t)b * C + c) * Tt + tau;
    if (gmax) acc *= 1.f / pow2_scale(*gmax);
    if (add1) acc += ldf(add1 + o);
    if (add2) acc += ldf(add2 + o);
    stf(dx + o, (tau < li) ? acc : 0.f);
}

// One warp per (b,c) row; lane k-strided taps; plain but correct for any stride.
template <typename TG, typename T>
__global__ void __launch_bounds__(128)
dw_wgrad_generic_kernel(const TG* __restrict__ gu, const T* __restrict__ x, float* __restrict__ partials,
                        const int* __restrict__ len_in, const int* __restrict__ len_out,
                        int B, int C, int Tt, int Tp, int K, int s, int dil) {
    pdl_sync();
    const int c = blockIdx.x, lane = threadIdx.x & 31, wrp = threadIdx.x >> 5;
    const int P = (dil * (K - 1)) / 2;
    // partials[b][c][k]; warps stride over samples
    for (int b = wrp; b < B; b += 4) {
        const int li = min(len_in[b], Tt), lo = min(len_out[b], Tp);
        const TG* grow = gu + ((size_t)b * C + c) * Tp;
        const T* xrow = x + ((size_t)b * C + c) * Tt;
        for (int k = 0; k < K; ++k) {
            float acc = 0.f;
            for (int t = lane; t < lo; t += 32) {
                const int tau = t * s + k * dil - P;
                if (tau >= 0 && tau < li) acc = fmaf(ldf(grow + t), ldf(xrow + tau), acc);
            }
            acc = warp_sum(acc);
            if (lane == 0) partials[((size_t)b * C + c) * K + k] = acc;
        }
    }
}

// Any stride, K <= 128: CTA = (channel, sample); thread (k, group) accumulates tap k over the frames
// t = group (mod ngroups) of a shared-memory tile; groups are then summed in order.
constexpr int WS_TT = 512;
template <typename TG, typename T>
__global__ void __launch_bounds__(128)
dw_wgrad_strided_kernel(const TG* __restrict__ gu, const T* __restrict__ x, float* __restrict__ partials,
                        const int* __restrict__ len_in, const int* __restrict__ len_out,
                        int C, int Tt, int Tp, int K, int s) {
    pdl_sync();
    extern __shared__ float smem[];
    const int c = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const int P = (K - 1) / 2, XW = (WS_TT - 1) * s + K;
    float* gs = smem;                 // [WS_TT]
    float* xs = smem + WS_TT;         // [XW]
    float* red = xs + XW;             // [128]
    const int ngrp = 128 / K, k = tid % K, grp = tid / K;
    const bool active = grp < ngrp;
    const int li = min(len_in[b], Tt), lo = min(len_out[b], Tp);
    const TG* grow = gu + ((size_t)b * C + c) * Tp;
    const T* xrow = x + ((size_t)b * C + c) * Tt;
    float acc = 0.f;
    for (int t0 = 0; t0 < lo; t0 += WS_TT) {
        __syncthreads();
        for (int i = tid; i < WS_TT; i += 128) gs[i] = (t0 + i < lo) ? ldf(grow + t0 + i) : 0.f;
        for (int i = tid; i < XW; i += 128) {
            const int tau = t0 * s - P + i;
            xs[i] = (tau >= 0 && tau < li) ? ldf(xrow + tau) : 0.f;
        }
        __syncthreads();
        if (active) {
            const int n = min(WS_TT, lo - t0);
            for (int t = grp; t < n; t += ngrp) acc = fmaf(gs[t], xs[t * s + k], acc);
        }
    }
    __syncthreads();
    red[tid] = active ? acc : 0.f;
    __syncthreads();
    if (tid < K) {
        float sum = 0.f;
        for (int g = 0; g < ngrp; ++g) sum += red[g * K + tid];
        partials[((size_t)b * C + c) * K + tid] = sum;
    }
}

// ---- stride-1 tap gradient: register-blocked --------------------------------------------------
// CTA = one channel, a group of BG samples.  Thread (kg, seg): tap group kg (R taps) x time segment.
constexpr int WG_THREADS = 128;
constexpr int WG_TT = 1024;     // frames per shared-memory tile
constexpr int WG_BG = 8;        // samples per CTA

template <typename TG, typename T>
__global__ void __launch_bounds__(WG_THREADS)
dw_wgrad_s1_kernel(const TG* __restrict__ gu, const T* __restrict__ x, float* __restrict__ partials,
                   const int* __restrict__ len_in, const int* __restrict__ len_out,
                   int B, int C, int Tt, int K, int Kpad) {
    pdl_sync();
    extern __shared__ float smem[];
    const int c = blockIdx.x, bg = blockIdx.y;
    const int P = (K - 1) / 2;
    const int NG = Kpad / R;                       // tap groups
    const int nseg = WG_THREADS / NG;              // time segments
    const int seglen = ((WG_TT + nseg - 1) / nseg + R - 1) / R * R;
    const int GW = nseg * seglen;                  // >= WG_TT, zero filled beyond
    const int XW = GW + Kpad;
    float* gs = smem;                              // [GW]
    float* xs = smem + GW;                         // [XW]: index i <-> frame t0 - P + i
    float* red = xs + XW;                          // [nseg][Kpad]
    const int tid = threadIdx.x;
    const bool active = tid < NG * nseg;
    const int kg = tid % NG, seg = tid / NG;
    float acc[R];
#pragma unroll
    for (int q = 0; q < R; ++q) acc[q] = 0.f;

    const int b_end = min(B, (bg + 1) * WG_BG);
    for (int b = bg * WG_BG; b < b_end; ++b) {
        const int li = min(len_in[b], Tt), lo = min(len_out[b], Tt);
        const TG* grow = gu + ((size_t)b * C + c) * Tt;
        const T* xrow = x + ((size_t)b * C + c) * Tt;
        for (int t0 = 0; t0 < lo; t0 += WG_TT) {
            __syncthreads();
            for (int i = tid; i < GW; i += WG_THREADS) {
                const int t = t0 + i;
                gs[i] = (i < WG_TT && t < lo) ? ldf(grow + t) : 0.f;
            }
            for (int i = tid; i < XW; i += WG_THREADS) {
                const int tau = t0 - P + i;
                xs[i] = (tau >= 0 && tau < li) ? ldf(xrow + tau) : 0.f;
            }
            __syncthreads();
            if (active) {
                const int ts = seg * seglen;
                const float* xp = xs + ts + kg * R;
                float win[2 * R];
#pragma unroll
                for (int r = 0; r < R; ++r) win[r] = xp[r];
                for (int tt = 0; tt < seglen; tt += R) {
#pragma unroll
                    for (int r = 0; r < R; ++r) win[R + r] = xp[tt + R + r];
                    float g[R];
#pragma unroll
                    for (int r = 0; r < R; ++r) g[r] = gs[ts + tt + r];
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int q = 0; q < R; ++q) acc[q] = fmaf(g[r], win[r + q], acc[q]);
#pragma unroll
                    for (int r = 0; r < R; ++r) win[r] = win[R + r];
                }
            }
        }
    }
    __syncthreads();
    if (active) {
#pragma unroll
        for (int q = 0; q < R; ++q) red[seg * Kpad + kg * R + q] = acc[q];
    }
    __syncthreads();
    for (int k = tid; k < K; k += WG_THREADS) {
        float sum = 0.f;
        for (int sgi = 0; sgi < nseg; ++sgi) sum += red[sgi * Kpad + k];
        partials[((size_t)bg * C + c) * K + k] = sum;
    }
}

// ---- stride-1 tap gradient, register accumulators ------------------------------------------------
// dwd[c,k] = sum_{b,t} gu[b,c,t] * x[b,c,t+k-P].  A thread owns 8 consecutive frames of gu (registers)
// and ALL taps: 8*NCH accumulators in registers, a 16-wide sliding window of x from shared memory, so
// the inner loop is 64 FMAs per two 16-byte shared loads.  Threads sweep the (row, 8-frame chunk)
// pairs of NR staged rows; the per-thread accumulators are summed over the warp with shuffles and over
// the CTA's warps in a fixed order (the "warp-level time reduction"), one partial per CTA.
constexpr int WR_THREADS = 128;

template <typename TG, typename T, int NCH>
__global__ void __launch_bounds__(WR_THREADS, 3)
dw_wgrad_reg_kernel(const TG* __restrict__ gu, const T* __restrict__ x, float* __restrict__ partials,
                    const int* __restrict__ len_in, const int* __restrict__ len_out,
                    int B, int C, int Tt, int K, int Ppad, int NR, int NST, int RSP) {
    pdl_sync();
    extern __shared__ float smem[];
    const int tid = threadIdx.x, lane = tid & 31, wrp = tid >> 5;
    const int c = blockIdx.x;
    const int P = (K - 1) / 2, shift = Ppad - P;
    const int cpr = Tt / 8;                        // 8-frame chunks per row (Tt % 8 == 0)
    const int XW = Tt + 8 * NCH + 8;               // x row: Ppad zeros, Tt frames, zeros up to XW
    float* gs = smem;                              // [NR][RSP]
    float* xs = smem + (size_t)NR * RSP;           // [NR][RSP]
    float acc[8 * NCH];
#pragma unroll
    for (int i = 0; i < 8 * NCH; ++i) acc[i] = 0.f;

    for (int st = 0; st < NST; ++st) {
        const int b0 = (blockIdx.y * NST + st) * NR;
        if (b0 >= B) break;
        const int nr = min(NR, B - b0);
        __syncthreads();
        // zero the halos of x (frames before 0 and after Tt) -- everything else is overwritten
        for (int i = tid; i < nr * (XW - Tt); i += WR_THREADS) {
            const int r = i / (XW - Tt), j = i - r * (XW - Tt);
            const int col = j < Ppad ? j : Tt + j;
            xs[r * RSP + phys(col)] = 0.f;
        }
        for (int i = tid; i < nr * cpr; i += WR_THREADS) {
            const int r = i / cpr, t = (i - r * cpr) * 8;
            const int b = b0 + r;
            const int li = min(len_in[b], Tt), lo = min(len_out[b], Tt);
            const size_t off = ((size_t)b * C + c) * Tt + t;
            float fg[8], fx[8];
            if (t < lo) ld8<TG>(gu + off, fg);
            if (t < li) ld8<T>(x + off, fx);
#pragma unroll
            for (int e = 0; e < 8; ++e) { if (t + e >= lo) fg[e] = 0.f; if (t + e >= li) fx[e] = 0.f; }
            float* gd = gs + r * RSP + phys(t);
            // Ppad is a multiple of 4 only, so the two halves may straddle a 32-float padding boundary
            float* xd0 = xs + r * RSP + phys(t + Ppad);
            float* xd1 = xs + r * RSP + phys(t + Ppad + 4);
            *reinterpret_cast<float4*>(gd) = make_float4(fg[0], fg[1], fg[2], fg[3]);
            *reinterpret_cast<float4*>(gd + 4) = make_float4(fg[4], fg[5], fg[6], fg[7]);
            *reinterpret_cast<float4*>(xd0) = make_float4(fx[0], fx[1], fx[2], fx[3]);
            *reinterpret_cast<float4*>(xd1) = make_float4(fx[4], fx[5], fx[6], fx[7]);
        }
        __syncthreads();
        for (int i = tid; i < nr * cpr; i += WR_THREADS) {
            const int r = i / cpr, t = (i - r * cpr) * 8;
            const float* gp = gs + r * RSP;
            const float* xp = xs + r * RSP;
            float g[8], win[16];
            {
                const float4 a = *reinterpret_cast<const float4*>(gp + phys(t));
                const float4 bq = *reinterpret_cast<const float4*>(gp + phys(t + 4));
                g[0] = a.x; g[1] = a.y; g[2] = a.z; g[3] = a.w; g[4] = bq.x; g[5] = bq.y; g[6] = bq.z; g[7] = bq.w;
                const float4 c0 = *reinterpret_cast<const float4*>(xp + phys(t));
                const float4 c1 = *reinterpret_cast<const float4*>(xp + phys(t + 4));
                win[0] = c0.x; win[1] = c0.y; win[2] = c0.z; win[3] = c0.w;
                win[4] = c1.x; win[5] = c1.y; win[6] = c1.z; win[7] = c1.w;
            }
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                const float4 c0 = *reinterpret_cast<const float4*>(xp + phys(t + 8 * ch + 8));
                const float4 c1 = *reinterpret_cast<const float4*>(xp + phys(t + 8 * ch + 12));
                win[8] = c0.x; win[9] = c0.y; win[10] = c0.z; win[11] = c0.w;
                win[12] = c1.x; win[13] = c1.y; win[14] = c1.z; win[15] = c1.w;
#pragma unroll
                for (int q = 0; q < 8; ++q)
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr) acc[8 * ch + q] = fmaf(g[rr], win[rr + q], acc[8 * ch + q]);
#pragma unroll
                for (int q = 0; q < 8; ++q) win[q] = win[q + 8];
            }
        }
    }
    // warp tree, then the four warps in order
    __syncthreads();
    float* red = smem;                             // [4][8*NCH]
#pragma unroll
    for (int i = 0; i < 8 * NCH; ++i) {
        float v = warp_sum(acc[i]);
        if (lane == 0) red[wrp * 8 * NCH + i] = v;
    }
    __syncthreads();
    for (int k = tid; k < K; k += WR_THREADS) {
        const int kk = k + shift;
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < WR_THREADS / 32; ++w) sum += red[w * 8 * NCH + kk];
        partials[((size_t)blockIdx.y * C + c) * K + k] = sum;
    }
}

// ---- the same for 16-bit tensors: rows stay 16-bit in shared memory, filled by cp.async ----------
// Shared rows hold the raw 16-bit values (half the footprint, and 16-byte lane pitch is conflict-free
// without padding); conversion to fp32 happens in registers.  Two buffers: the next pass's rows are in
// flight (cp.async) while the current pass computes.
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async8(void* dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <typename T> __device__ __forceinline__ void cvt8(const uint4& r, float (&f)[8]);
template <> __device__ __forceinline__ void cvt8<__half>(const uint4& r, float (&f)[8]) {
    const __half2* h = reinterpret_cast<const __half2*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float2 q = __half22float2(h[i]); f[2 * i] = q.x; f[2 * i + 1] = q.y; }
}
template <> __device__ __forceinline__ void cvt8<__nv_bfloat16>(const uint4& r, float (&f)[8]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u); }
}

template <typename TG, typename T, int NCH>
__global__ void __launch_bounds__(WR_THREADS, (NCH <= 8 ? 4 : 3))
dw_wgrad_reg16_kernel(const TG* __restrict__ gu, const T* __restrict__ x, float* __restrict__ partials,
                      const int* __restrict__ len_in, const int* __restrict__ len_out,
                      int B, int C, int Tt, int K, int Ppad, int NR, int NST, int RS) {
    pdl_sync();
    static_assert(sizeof(TG) == 2 && sizeof(T) == 2, "16-bit tensors only");
    extern __shared__ __align__(16) unsigned short smem16[];
    const int tid = threadIdx.x, lane = tid & 31, wrp = tid >> 5;
    const int c = blockIdx.x;
    const int P = (K - 1) / 2, shift = Ppad - P;
    const int cpr = Tt / 8;
    const int XW = Tt + 8 * NCH + 8;
    const int halo = XW - Tt;
    const size_t bufsz = (size_t)2 * NR * RS;               // elements per buffer: g rows then x rows
    float acc[8 * NCH];
#pragma unroll
    for (int i = 0; i < 8 * NCH; ++i) acc[i] = 0.f;
    // lengths of this CTA's rows, read once (NR * NST <= 32 rows)
    __shared__ int s_li[32], s_lo[32];
    if (tid < NR * NST) {
        const int b = blockIdx.y * NST * NR + tid;
        s_li[tid] = b < B ? min(len_in[b], Tt) : 0;
        s_lo[tid] = b < B ? min(len_out[b], Tt) : 0;
    }
    __syncthreads();

    auto issue = [&](int st) {
        const int b0 = (blockIdx.y * NST + st) * NR;
        const int nr = min(NR, B - b0);
        unsigned short* gs = smem16 + (st & 1) * bufsz;
        unsigned short* xs = gs + (size_t)NR * RS;
        for (int i = tid; i < nr * halo; i += WR_THREADS) {
            const int r = i / halo, j = i - r * halo;
            xs[r * RS + (j < Ppad ? j : Tt + j)] = 0;
        }
        int r = tid / cpr, t = (tid - r * cpr) * 8;
        for (int i = tid; i < nr * cpr; i += WR_THREADS, t += WR_THREADS * 8) {
            while (t >= Tt) { t -= Tt; ++r; }
            const int b = b0 + r;
            const int li = s_li[st * NR + r], lo = s_lo[st * NR + r];
            const size_t off = ((size_t)b * C + c) * Tt + t;
            unsigned short* gd = gs + r * RS + t;
            unsigned short* xd = xs + r * RS + t + Ppad;
            if (t < lo) cp_async16(gd, gu + off); else *reinterpret_cast<uint4*>(gd) = make_uint4(0, 0, 0, 0);
            if (t < li) cp_async8(xd, x + off); else *reinterpret_cast<uint2*>(xd) = make_uint2(0, 0);
            if (t + 4 < li) cp_async8(xd + 4, x + off + 4); else *reinterpret_cast<uint2*>(xd + 4) = make_uint2(0, 0);
        }
        cp_async_commit();
    };
    // after this thread's copies have landed: zero the tail of the vector a length falls into
    auto patch = [&](int st) {
        const int b0 = (blockIdx.y * NST + st) * NR;
        const int nr = min(NR, B - b0);
        unsigned short* gs = smem16 + (st & 1) * bufsz;
        unsigned short* xs = gs + (size_t)NR * RS;
        // the copies that can straddle a length were issued by thread (row*cpr + len/8) % 128: that thread waits
        // for its own copies above, so it is the one that may overwrite the tail
        for (int r = 0; r < nr; ++r) {
            const int li = s_li[st * NR + r], lo = s_lo[st * NR + r];
            if ((lo & 7) && ((r * cpr + (lo >> 3)) % WR_THREADS) == tid)
                for (int e = lo; e < ((lo + 7) & ~7); ++e) gs[r * RS + e] = 0;
            if ((li & 7) && ((r * cpr + (li >> 3)) % WR_THREADS) == tid)
                for (int e = li; e < ((li + 7) & ~7); ++e) xs[r * RS + Ppad + e] = 0;
        }
    };

    const int nst = min(NST, (B - (int)blockIdx.y * NST * NR + NR - 1) / NR);   // passes with at least one row
    if (nst > 0) issue(0);
    for (int st = 0; st < nst; ++st) {
        if (st + 1 < nst) { issue(st + 1); cp_async_wait<1>(); } else { cp_async_wait<0>(); }
        patch(st);
        __syncthreads();
        const int b0 = (blockIdx.y * NST + st) * NR;
        const int nr = min(NR, B - b0);
        const unsigned short* gs = smem16 + (st & 1) * bufsz;
        const unsigned short* xs = gs + (size_t)NR * RS;
        int r = tid / cpr, t = (tid - r * cpr) * 8;          // chunk index -> (row, frame), then stepped without divisions
        for (int i = tid; i < nr * cpr; i += WR_THREADS, t += WR_THREADS * 8) {
            while (t >= Tt) { t -= Tt; ++r; }
            if (t >= s_lo[st * NR + r]) continue;          // gradient is zero in padding: nothing to add
            const unsigned short* xp = xs + r * RS + t;
            float g[8], win[16];
            cvt8<TG>(*reinterpret_cast<const uint4*>(gs + r * RS + t), g);
            {
                float lo8[8];
                cvt8<T>(*reinterpret_cast<const uint4*>(xp), lo8);
#pragma unroll
                for (int q = 0; q < 8; ++q) win[q] = lo8[q];
            }
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                float hi8[8];
                cvt8<T>(*reinterpret_cast<const uint4*>(xp + 8 * ch + 8), hi8);
#pragma unroll
                for (int q = 0; q < 8; ++q) win[8 + q] = hi8[q];
#pragma unroll
                for (int q = 0; q < 8; ++q)
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr) acc[8 * ch + q] = fmaf(g[rr], win[rr + q], acc[8 * ch + q]);
#pragma unroll
                for (int q = 0; q < 8; ++q) win[q] = win[q + 8];
            }
        }
        __syncthreads();
    }
    float* red = reinterpret_cast<float*>(smem16);       // [4][8*NCH]
    {
        // Warp reduction that halves the number of live values at every step: lane pairs (l, l^s) split the
        // values between them, each keeps one half and adds the partner's copy of it.  VP/32 sums per lane
        // remain after five steps (VP - VP/32 shuffles instead of 5 VP); the pairing is fixed, so is the order.
        constexpr int VP = (8 * NCH + 31) / 32 * 32;
        float v[VP];
#pragma unroll
        for (int i = 0; i < VP; ++i) v[i] = i < 8 * NCH ? acc[i] : 0.f;
        int base = 0;
#pragma unroll
        for (int sstep = 16, n = VP / 2; sstep >= 1; sstep >>= 1, n >>= 1) {
            const bool up = (lane & sstep) != 0;
#pragma unroll
            for (int i = 0; i < n; ++i) {
                const float lo = v[i], hi = v[i + n];
                const float got = __shfl_xor_sync(0xffffffffu, up ? lo : hi, sstep);
                v[i] = (up ? hi : lo) + got;
            }
            if (up) base += n;
        }
#pragma unroll
        for (int i = 0; i < VP / 32; ++i)
            if (base + i < 8 * NCH) red[wrp * 8 * NCH + base + i] = v[i];
    }
    __syncthreads();
    for (int k = tid; k < K; k += WR_THREADS) {
        const int kk = k + shift;
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < WR_THREADS / 32; ++w) sum += red[w * 8 * NCH + kk];
        partials[((size_t)blockIdx.y * C + c) * K + k] = sum;
    }
}

inline int kpad(int K) { return (K + R - 1) / R * R; }
inline int host_phys(int i) { return i + ((i >> 5) << 2); }

}  // namespace

// (activation type T, internal operand type OT): fp32 -> (float, float); fp16 -> (half, half);
// bf16 -> (bf16, half) for layers with a depthwise step.
#define SC_DISPATCH_IO(dtype, odt, ...)                                                         \
    if (dtype == F32) { using T = float; using OT = float; __VA_ARGS__; }                        \
    else if (dtype == F16) { using T = __half; using OT = __half; __VA_ARGS__; }                 \
    else if (odt == F16) { using T = __nv_bfloat16; using OT = __half; __VA_ARGS__; }            \
    else { using T = __nv_bfloat16; using OT = __nv_bfloat16; __VA_ARGS__; }

void dw_fwd(const Launch& L, int dtype, int odt, const void* x, const void* wd, void* u, const int* len_in,
            const int* len_out, int B, int C, int Tt, int Tp, int K, int s, int dil) {
    KScope ks_(L, KC_DW_FWD, (double)B * C * (dtype_size(dtype) * Tt + dtype_size(odt) * Tp), 2.0 * B * C * Tp * K);
    const bool plain = dil == 1 && (K & 1);      // odd K, adjacent taps: the forms the specialised kernels are written for
    if (!L.simt_only && plain && dw_tc_supported(dtype, Tt, K, s)) {
        dw_tc_fwd(L, dtype, odt, x, wd, u, len_in, len_out, B, C, Tt, K);
        return;
    }
    if (s == 1 && plain) {
        const int Kp = kpad(K);
        const size_t smem = (size_t)CH * (host_phys(TT + Kp) + 4 + Kp) * sizeof(float);
        dim3 grid((Tt + TT - 1) / TT, (C + CH - 1) / CH, B), block(32, CH);
        SC_DISPATCH_IO(dtype, odt, (launch_k(L, dw_corr_s1_kernel<T, T, OT>, grid, block, smem, 
                                       (const T*)x, (const T*)wd, (OT*)u, nullptr, nullptr, nullptr, len_in, len_out, C, Tt,
                                       K, Kp, 0, L.status)));
    } else {
        const size_t smem = (size_t)((GT - 1) * s + (K - 1) * dil + 1 + K) * sizeof(float);
        dim3 grid((Tp + GT - 1) / GT, C, B);
        SC_DISPATCH_IO(dtype, odt, (launch_k(L, dw_fwd_generic_kernel<T, OT>, grid, GT, smem, 
                                       (const T*)x, (const T*)wd, (OT*)u, len_in, len_out, C, Tt, Tp, K, s, dil, L.status)));
    }
    L.count();
}

void dw_dgrad(const Launch& L, int dtype, int odt, const void* gu, const void* wd, void* dx, const void* add1,
              const void* add2, const float* gmax, const int* len_in, const int* len_out, int B, int C, int Tt,
              int Tp, int K, int s, int dil) {
    const bool plain = dil == 1 && (K & 1);
    KScope ks_(L, KC_DW_DGRAD, (double)B * C * (dtype_size(dtype) * Tt * (1 + (add1 ? 1 : 0) + (add2 ? 1 : 0)) + dtype_size(odt) * Tp),
               2.0 * B * C * Tp * K);
    if (!L.simt_only && plain && dw_tc_supported(dtype, Tt, K, s)) {
        dw_tc_dgrad(L, dtype, odt, gu, wd, dx, add1, add2, gmax, len_in, len_out, B, C, Tt, K);
        return;
    }
    if (s == 1 && plain) {
        const int Kp = kpad(K);
        const size_t smem = (size_t)CH * (host_phys(TT + Kp) + 4 + Kp) * sizeof(float);
        dim3 grid((Tt + TT - 1) / TT, (C + CH - 1) / CH, B), block(32, CH);
        SC_DISPATCH_IO(dtype, odt, (launch_k(L, dw_corr_s1_kernel<OT, T, T>, grid, block, smem, 
                                       (const OT*)gu, (const T*)wd, (T*)dx, (const T*)add1, (const T*)add2, gmax, len_out,
                                       len_in, C, Tt, K, Kp, 1, L.status)));
    } else {
        const size_t smem = (size_t)((GT + (K - 1) * dil + 1) / s + 4 + K) * sizeof(float);
        dim3 grid((Tt + GT - 1) / GT, C, B);
        SC_DISPATCH_IO(dtype, odt, (launch_k(L, dw_dgrad_generic_kernel<OT, T>, grid, GT, smem, 
                                       (const OT*)gu, (const T*)wd, (T*)dx, (const T*)add1, (const T*)add2, gmax, len_in,
                                       len_out, C, Tt, Tp, K, s, dil)));
    }
    L.count();
}

size_t dw_wgrad_scratch_bytes(int B, int C, int K) { return (size_t)B * C * K * sizeof(float); }

void dw_wgrad(const Launch& L, int dtype, int odt, const void* gu, const void* x, float* dwd, float* partials,
              int accumulate, const float* gmax, const int* len_in, const int* len_out, int B, int C, int Tt,
              int Tp, int K, int s, int dil) {
    const bool plain = dil == 1 && (K & 1);
    int nsplit;
    {
    KScope ks_(L, KC_DW_WGRAD, (double)B * C * (dtype_size(dtype) * Tt + dtype_size(odt) * Tp), 2.0 * B * C * Tp * K);
    const int P = (K - 1) / 2, Ppad = (P + 3) / 4 * 4;
    const int nch = (K + (Ppad - P) + 7) / 8;
    // the register kernels stage whole rows: one row (double-buffered) must fit their shared-memory limit
    const bool reg_fits = (dtype == F32) ? (size_t)2 * ((host_phys(Tt + 8 * nch + 8) + 4 + 3) / 4 * 4) * sizeof(float) <= 64 * 1024
                                         : (size_t)2 * 2 * ((Tt + 8 * nch + 8 + 7) / 8 * 8) * 2 <= 96 * 1024;
    if (plain && s == 1 && Tt % 8 == 0 && nch >= 2 && nch <= 12 && reg_fits) {
        // rows staged per pass: the count whose (rows x chunks) best fills the 128 threads
        const int cpr = Tt / 8;
        const int NST = (dtype == F32) ? 2 : 4;
        if (dtype == F32) {
            const int rs = host_phys(Tt + 8 * nch + 8) + 4, rsp = (rs + 3) / 4 * 4;
            int NR = 1; double best = 0.0;
            for (int nr = 1; nr <= 8 && nr <= B; ++nr) {
                if ((size_t)2 * nr * rsp * sizeof(float) > 64 * 1024) break;
                const int work = nr * cpr, iters = (work + WR_THREADS - 1) / WR_THREADS;
                const double eff = (double)work / (iters * WR_THREADS);
                if (eff > best + 1e-9) { best = eff; NR = nr; }
            }
            nsplit = (B + NR * NST - 1) / (NR * NST);
            const size_t smem = std::max((size_t)2 * NR * rsp, (size_t)4 * 8 * nch) * sizeof(float);
            dim3 grid(C, nsplit);
#define SC_WR_CASE(N)                                                                                          \
            case N: {                                                                                          \
                auto kern = dw_wgrad_reg_kernel<float, float, N>;                                              \
                set_max_smem_once<dw_wgrad_reg_kernel<float, float, N>>(64 * 1024);                            \
                launch_k(L, kern, grid, WR_THREADS, smem, (const float*)gu, (const float*)x, partials, len_in, len_out, \
                                                           B, C, Tt, K, Ppad, NR, NST, rsp);                   \
            } break;
            switch (nch) {
                SC_WR_CASE(2) SC_WR_CASE(3) SC_WR_CASE(4) SC_WR_CASE(5) SC_WR_CASE(6) SC_WR_CASE(7) SC_WR_CASE(8)
                SC_WR_CASE(9) SC_WR_CASE(10) SC_WR_CASE(11) SC_WR_CASE(12)
            }
#undef SC_WR_CASE
        } else {
            const int RS = (Tt + 8 * nch + 8 + 7) / 8 * 8;
            int NR = 1; double best = 0.0;
            for (int nr = 1; nr <= 8 && nr <= B; ++nr) {
                if ((size_t)2 * 2 * nr * RS * 2 > 96 * 1024) break;
                const int work = nr * cpr, iters = (work + WR_THREADS - 1) / WR_THREADS;
                const double eff = (double)work / (iters * WR_THREADS);
                if (eff > best + 1e-9) { best = eff; NR = nr; }
            }
            nsplit = (B + NR * NST - 1) / (NR * NST);
            const size_t smem = std::max((size_t)2 * 2 * NR * RS * 2, (size_t)4 * 8 * nch * sizeof(float));
            dim3 grid(C, nsplit);
#define SC_WR_CASE(N)                                                                                          \
            case N: {                                                                                          \
                if (dtype == F16) {                                                                            \
                    auto kern = dw_wgrad_reg16_kernel<__half, __half, N>;                                      \
                    set_max_smem_once<dw_wgrad_reg16_kernel<__half, __half, N>>(96 * 1024);   \
                    launch_k(L, kern, grid, WR_THREADS, smem, (const __half*)gu, (const __half*)x, partials, len_in, len_out, \
                                                               B, C, Tt, K, Ppad, NR, NST, RS);               \
                } else if (odt == F16) {                                                                       \
                    auto kern = dw_wgrad_reg16_kernel<__half, __nv_bfloat16, N>;                               \
                    set_max_smem_once<dw_wgrad_reg16_kernel<__half, __nv_bfloat16, N>>(96 * 1024);   \
                    launch_k(L, kern, grid, WR_THREADS, smem, (const __half*)gu, (const __nv_bfloat16*)x, partials, len_in, len_out, \
                                                               B, C, Tt, K, Ppad, NR, NST, RS);               \
                } else {                                                                                       \
                    auto kern = dw_wgrad_reg16_kernel<__nv_bfloat16, __nv_bfloat16, N>;                        \
                    set_max_smem_once<dw_wgrad_reg16_kernel<__nv_bfloat16, __nv_bfloat16, N>>(96 * 1024);   \
                    launch_k(L, kern, grid, WR_THREADS, smem, (const __nv_bfloat16*)gu, (const __nv_bfloat16*)x, partials, len_in, len_out, \
                                                               B, C, Tt, K, Ppad, NR, NST, RS);               \
                }                                                                                              \
            } break;
            switch (nch) {
                SC_WR_CASE(2) SC_WR_CASE(3) SC_WR_CASE(4) SC_WR_CASE(5) SC_WR_CASE(6) SC_WR_CASE(7) SC_WR_CASE(8)
                SC_WR_CASE(9) SC_WR_CASE(10) SC_WR_CASE(11) SC_WR_CASE(12)
            }
#undef SC_WR_CASE
        }
    } else if (plain && s == 1) {
        const int Kp = kpad(K), NG = Kp / R, nseg = WG_THREADS / NG;
        const int seglen = ((WG_TT + nseg - 1) / nseg + R - 1) / R * R;
        const int GW = nseg * seglen;
        const size_t smem = (size_t)(GW + GW + Kp + nseg * Kp) * sizeof(float);
        nsplit = (B + WG_BG - 1) / WG_BG;
        dim3 grid(C, nsplit);
        SC_DISPATCH_IO(dtype, odt, (launch_k(L, dw_wgrad_s1_kernel<OT, T>, grid, WG_THREADS, smem, 
                                       (const OT*)gu, (const T*)x, partials, len_in, len_out, B, C, Tt, K, Kp)));
    } else if (plain && K <= 128) {
        nsplit = B;
        const size_t smem = (size_t)(WS_TT + (WS_TT - 1) * s + K + 128) * sizeof(float);
        dim3 grid(C, B);
        SC_DISPATCH_IO(dtype, odt, (launch_k(L, dw_wgrad_strided_kernel<OT, T>, grid, 128, smem, 
                                       (const OT*)gu, (const T*)x, partials, len_in, len_out, C, Tt, Tp, K, s)));
    } else {
        nsplit = B;
        SC_DISPATCH_IO(dtype, odt, (launch_k(L, dw_wgrad_generic_kernel<OT, T>, C, 128, 0, 
                                       (const OT*)gu, (const T*)x, partials, len_in, len_out, B, C, Tt, Tp, K, s, dil)));
    }
    L.count();
    }
    reduce_partials(L, partials, nsplit, (int64_t)C * K, dwd, accumulate, gmax);
}

}  // namespace sc
