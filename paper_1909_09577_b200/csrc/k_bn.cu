// Lengths, masked batch-norm statistics / apply / backward, and small elementwise kernels.
// All of these stream [B,C,T] tensors once; one CTA handles one (sample, channel) row so that the
// per-channel coefficients are loaded once and reductions stay inside the CTA (warp shuffles +
// one shared-memory step).  Cross-CTA reductions go through per-row partials that a finalize
// kernel sums in a fixed order, so results are bit-repeatable.
#include <algorithm>

#include "common.cuh"
#include "kernels.h"

namespace sc {
namespace {

constexpr int kRowThreads = 256;          // 8 warps per CTA, one (sample, channel) row per warp
constexpr int kRowsPerCta = kRowThreads / 32;
#define SC_ROW_SETUP(nrows)                                                  \
    const int row = blockIdx.x * kRowsPerCta + (threadIdx.x >> 5);          \
    if (row >= (nrows)) return;                                              \
    const int lane = threadIdx.x & 31;

template <typename T>
__device__ __forceinline__ void load_chunk(const T* row, int t0, int Tp, bool vec, float (&f)[8]) {
    if (vec && t0 + 8 <= Tp) { ld8<T>(row + t0, f); return; }
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = (t0 + i < Tp) ? ldf(row + t0 + i) : 0.f;
}
template <typename T>
__device__ __forceinline__ void store_chunk(T* row, int t0, int Tp, bool vec, const float (&f)[8]) {
    if (vec && t0 + 8 <= Tp) { st8<T>(row + t0, f); return; }
#pragma unroll
    for (int i = 0; i < 8; ++i) if (t0 + i < Tp) stf(row + t0 + i, f[i]);
}

// Sum of `v` over the warp that owns the row; result valid in every lane.
template <int N>
__device__ __forceinline__ void block_sum(float (&v)[N]) {
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = warp_sum(v[i]);
}

__device__ __forceinline__ float block_max(float v) { return warp_max(v); }

__global__ void lengths_kernel(const int* __restrict__ len_in, int B, int T_in, int stride,
                               int* __restrict__ len_out, int* __restrict__ nvalid, int* __restrict__ blk_off,
                               int* status) {
    pdl_sync();
    // single CTA; B is small (<= a few thousand)
    __shared__ int total;
    if (threadIdx.x == 0) total = 0;
    __syncthreads();
    int local = 0;
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        int l = len_in[b];
        if (l < 1 || l > T_in) { raise_status(status, kErrLengths); l = min(max(l, 0), T_in); }
        int lo = (l + stride - 1) / stride;
        len_out[b] = lo;
        local += lo;
    }
    atomicAdd(&total, local);   // integer: order-independent
    __syncthreads();
    if (threadIdx.x == 0) {
        *nvalid = total;
        if (blk_off) {              // B is small: a serial scan by one thread
            int acc = 0;
            for (int b = 0; b < B; ++b) { blk_off[b] = acc; acc += (len_out[b] + 63) / 64; }
            blk_off[B] = acc;
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(kRowThreads)
bn_stats_kernel(const T* __restrict__ v, const int* __restrict__ len_out, int nrows, int C, int Tp,
                float2* __restrict__ partials) {
    pdl_sync();
    SC_ROW_SETUP(nrows)
    const int b = row / C;
    const int len = min(len_out[b], Tp);
    const T* p = v + (size_t)row * Tp;
    const bool vec = (Tp % 8 == 0);
    float s[1] = {0.f};
    for (int t0 = lane * 8; t0 < len; t0 += 256) {
        float f[8];
        load_chunk(p, t0, Tp, vec, f);
#pragma unroll
        for (int i = 0; i < 8; ++i) if (t0 + i < len) s[0] += f[i];
    }
    block_sum(s);
    const float mean = len > 0 ? s[0] / (float)len : 0.f;
    float q[1] = {0.f};
    for (int t0 = lane * 8; t0 < len; t0 += 256) {
        float f[8];
        load_chunk(p, t0, Tp, vec, f);
#pragma unroll
        for (int i = 0; i < 8; ++i) if (t0 + i < len) { float d = f[i] - mean; q[0] += d * d; }
    }
    block_sum(q);
    if (lane == 0) partials[row] = make_float2(s[0], q[0]);
}

// Thirty-two channels per CTA, one per lane, so that every load of a warp is one contiguous run of the
// [part][channel] partial array.  Warp w takes parts w, w + 32, ... in increasing order; the thirty-two
// warp results are combined in warp order, so the result is bit-repeatable.  One pass: with a pivot c
// (the mean of the channel's first part, which always holds at least one valid frame)
//   sum = sum_p sum_p,   M2 = sum_p [M2_p + n_p (mean_p - c)^2]  -  N (mean - c)^2,
// and because c lies within the spread of the data the subtraction cancels nothing that matters.
// No term depends on the previous one, so a lane's few loads are all in flight together.
constexpr int kFinWarps = 32;
__global__ void __launch_bounds__(32 * kFinWarps)
bn_finalize_kernel(const float2* __restrict__ partials, int parts_per_b, int tile_w,
                   const int* __restrict__ len_out, const int* __restrict__ nvalid, int B,
                   int C, float eps, float momentum, float* __restrict__ mean_out,
                   float* __restrict__ invstd_out, float* running_mean, float* running_var) {
    pdl_sync();
    __shared__ float2 s_red[kFinWarps][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int o = blockIdx.x * 32 + lane;
    const bool act = o < C;
    const int nparts = B * parts_per_b;
    auto count_of = [&](int pi) -> int {
        const int b = pi / parts_per_b, j = pi - b * parts_per_b;
        return max(0, min(len_out[b] - j * tile_w, tile_w));
    };
    float s1 = 0.f, q = 0.f;
    if (act) {
        const float c = partials[o].x / (float)max(1, count_of(0));
        for (int p0 = w; p0 < nparts; p0 += 8 * kFinWarps) {
            float2 v[8]; int cnt[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {        // issue every load before the first use
                const int pi = p0 + i * kFinWarps;
                cnt[i] = pi < nparts ? count_of(pi) : 0;
                v[i] = cnt[i] > 0 ? partials[(size_t)pi * C + o] : make_float2(0.f, 0.f);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (cnt[i] > 0) {
                    const float n = (float)cnt[i];
                    const float d = v[i].x / n - c;
                    s1 += v[i].x;
                    q += fmaf(n * d, d, v[i].y);
                }
            }
        }
    }
    s_red[w][lane] = make_float2(s1, q);
    __syncthreads();
    if (w != 0 || !act) return;
    // the tail runs in float: a double divide and square root would cost this latency-bound kernel more than the
    // whole merge, and the pivot keeps the subtraction below free of cancellation
    const float N = (float)(*nvalid);
    const float c = partials[o].x / (float)max(1, count_of(0));
    float t = 0.f, m2 = 0.f;
#pragma unroll
    for (int i = 0; i < kFinWarps; ++i) { t += s_red[i][lane].x; m2 += s_red[i][lane].y; }
    const float mean = N > 0.f ? t / N : 0.f;
    const float dm = mean - c;
    float var = N > 0.f ? (m2 - N * dm * dm) / N : 0.f;
    var = fmaxf(var, 0.f);
    mean_out[o] = mean;
    invstd_out[o] = 1.f / sqrtf(var + eps);
    if (running_mean) running_mean[o] = (1.f - momentum) * running_mean[o] + momentum * mean;
    if (running_var) {
        const float unb = N > 1.f ? var * (N / (N - 1.f)) : var;
        running_var[o] = (1.f - momentum) * running_var[o] + momentum * unb;
    }
}

// The same merge for the per-(CTA, channel) partials (count, sum, M2) of the flattened-block contraction.
// CTA c of the contraction contributed to M tile m iff its unit range [c U / G, (c+1) U / G) meets
// [m nblk, (m+1) nblk); the pivot is the mean of the first contributing CTA's partial.
__global__ void __launch_bounds__(32 * kFinWarps)
bn_finalize_flat_kernel(const float4* __restrict__ partials, int G, int tiles_m, int rows_per_tile,
                        const int* __restrict__ blk_off, const int* __restrict__ nvalid, int B, int C, float eps,
                        float momentum, float* __restrict__ mean_out, float* __restrict__ invstd_out,
                        float* running_mean, float* running_var) {
    pdl_sync();
    __shared__ float2 s_red[kFinWarps][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int o = blockIdx.x * 32 + lane;
    const bool act = o < C;
    const long long nblk = blk_off[B];
    const long long U = (long long)tiles_m * nblk;
    const int m = min(o, C - 1) / rows_per_tile;
    const long long lo = m * nblk, hi = lo + nblk;
    const bool small = U * (G + 1) < (1ll << 31);      // the same quotients in 32-bit arithmetic (no 64-bit divisions)
    auto takes_part = [&](int c) -> bool {
        long long b0, b1;
        if (small) { b0 = (uint32_t)U * (uint32_t)c / (uint32_t)G; b1 = (uint32_t)U * (uint32_t)(c + 1) / (uint32_t)G; }
        else { b0 = U * c / G; b1 = U * (c + 1) / G; }
        return max(b0, lo) < min(b1, hi);
    };
    int c_first = U > 0 ? (small ? (int)((uint32_t)lo * (uint32_t)G / (uint32_t)U) : (int)(lo * G / U)) : 0;
    while (c_first < G - 1 && !takes_part(c_first)) ++c_first;
    float pivot = 0.f;
    if (act && U > 0) { const float4 pv = partials[(size_t)c_first * C + o]; pivot = pv.x > 0.f ? pv.y / pv.x : 0.f; }
    float s1 = 0.f, q = 0.f;
    if (act && U > 0) {
        for (int c0 = w; c0 < G; c0 += 8 * kFinWarps) {
            float4 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {        // issue every load before the first use
                const int c = c0 + i * kFinWarps;
                v[i] = (c < G && takes_part(c)) ? partials[(size_t)c * C + o] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (v[i].x > 0.f) {
                    const float d = v[i].y / v[i].x - pivot;
                    s1 += v[i].y;
                    q += fmaf(v[i].x * d, d, v[i].z);
                }
            }
        }
    }
    s_red[w][lane] = make_float2(s1, q);
    __syncthreads();
    if (w != 0 || !act) return;
    const float N = (float)(*nvalid);
    float t = 0.f, m2 = 0.f;
#pragma unroll
    for (int i = 0; i < kFinWarps; ++i) { t += s_red[i][lane].x; m2 += s_red[i][lane].y; }
    const float mean = N > 0.f ? t / N : 0.f;
    const float dm = mean - pivot;
    float var = N > 0.f ? (m2 - N * dm * dm) / N : 0.f;
    var = fmaxf(var, 0.f);
    mean_out[o] = mean;
    invstd_out[o] = 1.f / sqrtf(var + eps);
    if (running_mean) running_mean[o] = (1.f - momentum) * running_mean[o] + momentum * mean;
    if (running_var) {
        const float unb = N > 1.f ? var * (N / (N - 1.f)) : var;
        running_var[o] = (1.f - momentum) * running_var[o] + momentum * unb;
    }
}

template <typename T, typename NT>
__global__ void __launch_bounds__(kRowThreads) bn_apply_kernel(ApplyArgs a) {
    pdl_sync();
    SC_ROW_SETUP(a.B * a.C)
    const int b = row / a.C, o = row % a.C;
    const int Tp = a.Tp, len = min(a.len_out[b], Tp);
    const bool vec = (Tp % 8 == 0);
    const size_t off = (size_t)row * Tp;
    const NT* __restrict__ v = (const NT*)a.v + off;
    const T* __restrict__ xr = a.residual == 1 ? (const T*)a.xres + off : nullptr;
    const NT* __restrict__ vr = a.residual == 2 ? (const NT*)a.vr + off : nullptr;
    T* __restrict__ y = (T*)a.y + off;
    const float mu = a.mean[o], is = a.invstd[o], ga = a.gamma[o], be = a.beta[o];
    float mur = 0.f, isr = 0.f, gar = 0.f, ber = 0.f;
    if (a.residual == 2) { mur = a.mean_r[o]; isr = a.invstd_r[o]; gar = a.gamma_r[o]; ber = a.beta_r[o]; }
    for (int t0 = lane * 8; t0 < Tp; t0 += 256) {
        float out[8];
        if (t0 < len) {
            float f[8], r[8];
            load_chunk(v, t0, Tp, vec, f);
            if (a.residual == 1) load_chunk(xr, t0, Tp, vec, r);
            else if (a.residual == 2) {
                load_chunk(vr, t0, Tp, vec, r);
#pragma unroll
                for (int i = 0; i < 8; ++i) r[i] = fmaf(gar, bn_norm(r[i], mur, isr), ber);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) r[i] = 0.f;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float bn = fmaf(ga, bn_norm(f[i], mu, is), be);   // the backward pass recomputes exactly this
                float q;
                if (a.res_before_relu) { q = bn + r[i]; if (a.has_relu) q = fmaxf(q, 0.f); }
                else { q = (a.has_relu ? fmaxf(bn, 0.f) : bn) + r[i]; }
                out[i] = (t0 + i < len) ? q : 0.f;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) out[i] = 0.f;
        }
        store_chunk(y, t0, Tp, vec, out);
    }
}

// Shared by the reduce and apply steps of the backward pass: per element gate and normalised value.
template <typename T, typename NT>
struct BwdRow {
    const T* __restrict__ g; const T* __restrict__ y; const NT* __restrict__ v; const NT* __restrict__ vr;
    float gam, bet, mu, is, mur, isr;
    int len, Tp;
    bool vec;
    __device__ BwdRow(const BnBwdArgs& a, int row, int b, int o) {
        Tp = a.Tp; len = min(a.len_out[b], Tp); vec = (Tp % 8 == 0);
        g = (const T*)a.g + (size_t)row * Tp;
        y = a.y ? (const T*)a.y + (size_t)row * Tp : nullptr;
        v = a.has_bn ? (const NT*)a.v + (size_t)row * Tp : nullptr;
        vr = (a.residual == 2) ? (const NT*)a.vr + (size_t)row * Tp : nullptr;
        const bool own_gate = a.has_relu && !a.res_before_relu && a.has_bn;
        gam = own_gate ? a.gamma[o] : 1.f; bet = own_gate ? a.beta[o] : 0.f;
        mu = a.has_bn ? a.mean[o] : 0.f; is = a.has_bn ? a.invstd[o] : 0.f;
        mur = (a.residual == 2) ? a.mean_r[o] : 0.f; isr = (a.residual == 2) ? a.invstd_r[o] : 0.f;
    }
    // ga: gated upstream gradient; gr: gradient reaching the residual sum; vn/vnr: normalised values
    __device__ __forceinline__ void chunk(const BnBwdArgs& a, int t0, float (&ga)[8], float (&gr)[8],
                                          float (&vn)[8], float (&vnr)[8]) const {
        float fg[8], fy[8];
        load_chunk(g, t0, Tp, vec, fg);
        const bool need_y = a.has_relu && a.res_before_relu;
        if (need_y) load_chunk(y, t0, Tp, vec, fy);
        if (a.has_bn) {
            load_chunk(v, t0, Tp, vec, vn);
#pragma unroll
            for (int i = 0; i < 8; ++i) vn[i] = bn_norm(vn[i], mu, is);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) vn[i] = 0.f;
        }
        if (a.residual == 2) {
            load_chunk(vr, t0, Tp, vec, vnr);
#pragma unroll
            for (int i = 0; i < 8; ++i) vnr[i] = bn_norm(vnr[i], mur, isr);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) vnr[i] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const bool in = (t0 + i < len);
            const float gm = in ? fg[i] : 0.f;
            bool gate = true;
            if (a.has_relu) gate = a.res_before_relu ? (fy[i] > 0.f) : (fmaf(gam, vn[i], bet) > 0.f);
            ga[i] = gate ? gm : 0.f;
            gr[i] = a.res_before_relu ? ga[i] : gm;
            if (!in) { vn[i] = 0.f; vnr[i] = 0.f; }
        }
    }
};

// Partial sums of the backward reduction live in a [sample][slot][channel] array, so that the finalize
// kernel, which gives one channel to each lane, reads contiguous runs.
__device__ __forceinline__ size_t bwd_part_index(const BnBwdArgs& a, int b, int slot, int o) {
    return ((size_t)b * a.nslots + slot) * a.C + o;
}

template <typename T, typename NT>
__global__ void __launch_bounds__(kRowThreads) bn_bwd_reduce_kernel(BnBwdArgs a) {
    pdl_sync();
    SC_ROW_SETUP(a.B * a.C)
    const int b = row / a.C, o = row % a.C;
    BwdRow<T, NT> R(a, row, b, o);
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    float amax = 0.f;
    for (int t0 = lane * 8; t0 < R.len; t0 += 256) {
        float ga[8], gr[8], vh[8], vhr[8];
        R.chunk(a, t0, ga, gr, vh, vhr);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            s[0] += ga[i]; s[1] += ga[i] * vh[i]; s[2] += gr[i]; s[3] += gr[i] * vhr[i];
            amax = fmaxf(amax, fmaxf(fabsf(ga[i]), fabsf(gr[i])));
        }
    }
    block_sum(s);
    if (a.gmax) amax = block_max(amax);
    if (lane == 0) {
        a.partials[bwd_part_index(a, b, 0, o)] = make_float4(s[0], s[1], s[2], s[3]);
        if (a.gmax) a.amax_part[bwd_part_index(a, b, 0, o)] = amax;
    }
}

// Thirty-two channels per CTA, one per lane; warp w takes samples w, w + 32, ... with all their slots (every
// load issued before the first add) and the thirty-two warp results are combined in warp order
// (bit-repeatable).
constexpr int kBwdMaxSlotsUnrolled = 8;
__global__ void __launch_bounds__(32 * kFinWarps)
bn_bwd_finalize_kernel(BnBwdArgs a, const float* gamma, const float* gamma_r, float* dgamma, float* dbeta,
                       float* dgamma_r, float* dbeta_r, float* dbias, int accumulate) {
    pdl_sync();
    __shared__ float4 s_sum[kFinWarps][32];
    __shared__ float s_max[kFinWarps][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int o = blockIdx.x * 32 + lane;
    const bool act = o < a.C;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f, amax = 0.f;
    if (act) {
        const uint32_t vpr = (uint32_t)(a.Tp / 8);
        for (int b = w; b < a.B; b += kFinWarps) {
            int used = 1;
            if (a.nslots > 1) {      // slots in use for this row (see bn_bwd_reduce_fast_kernel); r * vpr < 2^31
                const uint32_t r = (uint32_t)b * (uint32_t)a.C + (uint32_t)o;
                used = (int)((((r + 1u) * vpr - 1u) >> a.vpw_shift) - ((r * vpr) >> a.vpw_shift)) + 1;
            }
            for (int sl0 = 0; sl0 < used; sl0 += kBwdMaxSlotsUnrolled) {
                float4 pv[kBwdMaxSlotsUnrolled]; float am[kBwdMaxSlotsUnrolled];
#pragma unroll
                for (int i = 0; i < kBwdMaxSlotsUnrolled; ++i) {
                    const bool use = sl0 + i < used;
                    pv[i] = use ? a.partials[bwd_part_index(a, b, sl0 + i, o)] : make_float4(0.f, 0.f, 0.f, 0.f);
                    am[i] = (use && a.gmax) ? a.amax_part[bwd_part_index(a, b, sl0 + i, o)] : 0.f;
                }
#pragma unroll
                for (int i = 0; i < kBwdMaxSlotsUnrolled; ++i) {
                    s0 += pv[i].x; s1 += pv[i].y; s2 += pv[i].z; s3 += pv[i].w;
                    amax = fmaxf(amax, am[i]);
                }
            }
        }
    }
    s_sum[w][lane] = make_float4(s0, s1, s2, s3);
    s_max[w][lane] = amax;
    __syncthreads();
    if (w != 0 || !act) return;
    float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
    amax = 0.f;
#pragma unroll
    for (int i = 0; i < kFinWarps; ++i) {
        const float4 q = s_sum[i][lane];
        d0 += q.x; d1 += q.y; d2 += q.z; d3 += q.w;
        amax = fmaxf(amax, s_max[i][lane]);
    }
    const float N = (float)(*a.nvalid);
    if (a.gmax) {
        // |gv| <= |k| (max|ga| + |c1| + max|vhat| |c2|) and max|vhat| <= sqrt(N); a maximum is order-free,
        // so the integer atomic on the (non-negative) float's bit pattern keeps the result repeatable
        float bound = amax;
        if (a.has_bn)
            bound = fabsf(gamma[o] * a.invstd[o]) * (amax + fabsf((float)d0) / N + sqrtf(N) * fabsf((float)d1) / N);
        if (a.residual == 2)     // the residual branch's gradient shares the scale
            bound = fmaxf(bound, fabsf(gamma_r[o] * a.invstd_r[o]) *
                                     (amax + fabsf((float)d2) / N + sqrtf(N) * fabsf((float)d3) / N));
        if (bound < 3.0e38f) atomicMax(reinterpret_cast<unsigned int*>(a.gmax), __float_as_uint(bound));
    }
    auto put = [&](float* dst, float val) {
        if (dst) dst[o] = accumulate ? dst[o] + val : val;
    };
    if (a.has_bn) {
        put(dbeta, d0); put(dgamma, d1);
        a.coef[o] = make_float4(gamma[o] * a.invstd[o], (float)d0 / N, (float)d1 / N, 0.f);
    } else {
        put(dbias, d0);
        a.coef[o] = make_float4(1.f, 0.f, 0.f, 0.f);
    }
    if (a.residual == 2) {
        put(dbeta_r, d2); put(dgamma_r, d3);
        a.coef_r[o] = make_float4(gamma_r[o] * a.invstd_r[o], (float)d2 / N, (float)d3 / N, 0.f);
    }
}

template <typename T, typename NT, typename GT>
__global__ void __launch_bounds__(kRowThreads) bn_bwd_apply_kernel(BnBwdArgs a) {
    pdl_sync();
    SC_ROW_SETUP(a.B * a.C)
    const int b = row / a.C, o = row % a.C;
    BwdRow<T, NT> R(a, row, b, o);
    const float4 cf = a.coef[o];
    const float sc = a.gmax ? pow2_scale(*a.gmax) : 1.f;      // multiplying by it is exact: a power of two
    const float4 cr = (a.residual == 2) ? a.coef_r[o] : make_float4(0.f, 0.f, 0.f, 0.f);
    __half* __restrict__ gv16 = a.gv16 ? (__half*)a.gv16 + (size_t)row * R.Tp : nullptr;
    __half* __restrict__ gvr16 = a.gvr16 ? (__half*)a.gvr16 + (size_t)row * R.Tp : nullptr;
    GT* __restrict__ gv = (GT*)a.gv + (size_t)row * R.Tp;
    T* __restrict__ gvr = (a.residual == 2) ? (T*)a.gvr + (size_t)row * R.Tp : nullptr;
    T* __restrict__ gres = (a.residual == 1) ? (T*)a.gres + (size_t)row * R.Tp : nullptr;
    for (int t0 = lane * 8; t0 < R.Tp; t0 += 256) {
        float o1[8], o2[8];
        if (t0 < R.len) {
            float ga[8], gr[8], vh[8], vhr[8];
            R.chunk(a, t0, ga, gr, vh, vhr);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const bool in = (t0 + i < R.len);
                o1[i] = in ? cf.x * (ga[i] - cf.y - vh[i] * cf.z) : 0.f;
                if (a.residual == 2) o2[i] = in ? cr.x * (gr[i] - cr.y - vhr[i] * cr.z) : 0.f;
                else o2[i] = gr[i];
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) { o1[i] = 0.f; o2[i] = 0.f; }
        }
        const int nin = R.len - t0;
        if (gv16) {              // half copy for the weight gradient; gv itself keeps plain rounding
            float h[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) h[i] = o1[i] * sc;
            diffuse8<__half>(h, nin);
            store_chunk(gv16, t0, R.Tp, R.vec, h);
        } else {
            if (a.gv_scaled) {
#pragma unroll
                for (int i = 0; i < 8; ++i) o1[i] *= sc;
            }
            diffuse8<GT>(o1, nin);
        }
        if (gvr16) {
            float h[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) h[i] = o2[i] * sc;
            diffuse8<__half>(h, nin);
            store_chunk(gvr16, t0, R.Tp, R.vec, h);
        } else if (a.residual == 2) {
            diffuse8<T>(o2, nin);
        }
        store_chunk(gv, t0, R.Tp, R.vec, o1);
        if (gvr) store_chunk(gvr, t0, R.Tp, R.vec, o2);
        if (gres) store_chunk(gres, t0, R.Tp, R.vec, o2);
    }
}

// Per-channel constants of the forward apply step and of the backward kernels, loaded (or, in the
// channel-per-CTA kernels, computed) once and passed by value.
struct FwdChan { float mu, is, ga, be, mur, isr, gar, ber; };
struct BwdChan { float mu, is, ga, be, mur, isr; float4 cf, cr; };

// One 8-frame vector of the forward apply step: y = [t < len] * relu(gamma * vhat + beta (+ r)); n = frames of the
// vector inside the sample (0: wholly padding), rv / rr = the raw 16 bytes of v and of the residual operand.
template <typename T, typename NT, int RES>
__device__ __forceinline__ void apply_core(T* yp, int n, const uint4& rv, const uint4& rr, const FwdChan& c) {
    float out[8];
    if (n > 0) {
        float f[8], r[8];
        cvt8<NT>(rv, f);
        if (RES == 1) cvt8<T>(rr, r);
        if (RES == 2) cvt8<NT>(rr, r);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float rres = 0.f;
            if (RES == 1) rres = r[i];
            if (RES == 2) rres = fmaf(c.gar, bn_norm(r[i], c.mur, c.isr), c.ber);
            const float q = fmaxf(fmaf(c.ga, bn_norm(f[i], c.mu, c.is), c.be) + rres, 0.f);
            out[i] = i < n ? q : 0.f;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = 0.f;
    }
    st8<T>(yp, out);
}
template <typename T, typename NT, int RES>
__device__ __forceinline__ void apply_vec(const ApplyArgs& a, int o, int n, size_t off, const uint4& rv, const uint4& rr) {
    FwdChan c{};
    if (n > 0) {
        c.mu = a.mean[o]; c.is = a.invstd[o]; c.ga = a.gamma[o]; c.be = a.beta[o];
        if (RES == 2) { c.mur = a.mean_r[o]; c.isr = a.invstd_r[o]; c.gar = a.gamma_r[o]; c.ber = a.beta_r[o]; }
    }
    apply_core<T, NT, RES>((T*)a.y + off, n, rv, rr, c);
}

// One 8-frame vector of the backward apply step (gv and the residual branch's gradient), computed and stored.
template <typename T, typename NT, typename GT, int RES>
__device__ __forceinline__ void bwd_apply_core(const BnBwdArgs& a, int n, size_t off, float sc, bool fold, const uint4& rg,
                                               const uint4& rv, const uint4& rr, const uint4& ry, const BwdChan& c) {
    float o1[8], o2[8];
    if (n > 0) {
        float g[8], y[8], vn[8], vnr[8];
        cvt8<T>(rg, g);
        cvt8<NT>(rv, vn);
        const uint64_t nmu2 = pk::pack(-c.mu, -c.mu), is2 = pk::pack(c.is, c.is);
        uint64_t vn2[4], vr2[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) vn2[q] = pk::bn_norm2(pk::pack(vn[2 * q], vn[2 * q + 1]), nmu2, is2);
        if (RES == 2) {
            cvt8<NT>(rr, vnr);
            const uint64_t nmur2 = pk::pack(-c.mur, -c.mur), isr2 = pk::pack(c.isr, c.isr);
#pragma unroll
            for (int q = 0; q < 4; ++q) vr2[q] = pk::bn_norm2(pk::pack(vnr[2 * q], vnr[2 * q + 1]), nmur2, isr2);
        }
        bool gate[8];
        if (RES == 0) {
            // without a residual the forward output is relu(gamma * vhat + beta), rounded to the
            // activation type: the gate is recomputed from v and the output need not be read
            const uint64_t ga2 = pk::pack(c.ga, c.ga), be2 = pk::pack(c.be, c.be);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float a0, a1;
                pk::unpack(pk::fma(ga2, vn2[q], be2), a0, a1);
                gate[2 * q] = rounds_positive<T>(a0); gate[2 * q + 1] = rounds_positive<T>(a1);
            }
        } else {
            cvt8<T>(ry, y);
#pragma unroll
            for (int i = 0; i < 8; ++i) gate[i] = y[i] > 0.f;
        }
        // gv = k (ga - c1 - c2 vhat) as two fused multiply-adds; when gv itself is the scaled half tensor the
        // power-of-two scale is folded into k (exact)
        const float4 cf = c.cf;
        const float kx = (fold ? sc : 1.f) * cf.x;
        const uint64_t kx2 = pk::pack(kx, kx), k02 = pk::pack(-kx * cf.y, -kx * cf.y), k22 = pk::pack(-kx * cf.z, -kx * cf.z);
        uint64_t kr2 = 0, r02 = 0, r22 = 0;
        if (RES == 2) {
            const float4 cr = c.cr;
            kr2 = pk::pack(cr.x, cr.x); r02 = pk::pack(-cr.x * cr.y, -cr.x * cr.y); r22 = pk::pack(-cr.x * cr.z, -cr.x * cr.z);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const bool in0 = 2 * q < n, in1 = 2 * q + 1 < n;
            const float g0 = (in0 && gate[2 * q]) ? g[2 * q] : 0.f;
            const float g1 = (in1 && gate[2 * q + 1]) ? g[2 * q + 1] : 0.f;
            const uint64_t ga2 = pk::pack(g0, g1);
            float x0, x1;
            pk::unpack(pk::fma(k22, vn2[q], pk::fma(kx2, ga2, k02)), x0, x1);
            o1[2 * q] = in0 ? x0 : 0.f; o1[2 * q + 1] = in1 ? x1 : 0.f;
            if (RES == 2) {
                pk::unpack(pk::fma(r22, vr2[q], pk::fma(kr2, ga2, r02)), x0, x1);
                o2[2 * q] = in0 ? x0 : 0.f; o2[2 * q + 1] = in1 ? x1 : 0.f;
            }
            if (RES == 1) { o2[2 * q] = g0; o2[2 * q + 1] = g1; }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) { o1[i] = 0.f; o2[i] = 0.f; }
    }
    if (a.gv16) {            // half copy for the weight gradient; gv itself keeps plain rounding
        float h[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) h[i] = o1[i] * sc;
        diffuse8<__half>(h, n);
        st8<__half>((__half*)a.gv16 + off, h);
    } else {
        diffuse8<GT>(o1, n);
    }
    if (RES == 2) {
        if (a.gvr16) {
            float h[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) h[i] = o2[i] * sc;
            diffuse8<__half>(h, n);
            st8<__half>((__half*)a.gvr16 + off, h);
        } else {
            diffuse8<T>(o2, n);
        }
    }
    st8<GT>((GT*)a.gv + off, o1);
    if (RES == 2) st8<T>((T*)a.gvr + off, o2);
    if (RES == 1) st8<T>((T*)a.gres + off, o2);
}

template <typename T, typename NT, typename GT, int RES>
__device__ __forceinline__ void bwd_apply_vec(const BnBwdArgs& a, int o, int n, size_t off, float sc, bool fold,
                                              const uint4& rg, const uint4& rv, const uint4& rr, const uint4& ry) {
    BwdChan c{};
    if (n > 0) {
        c.mu = a.mean[o]; c.is = a.invstd[o]; c.cf = a.coef[o];
        if (RES == 0) { c.ga = a.gamma[o]; c.be = a.beta[o]; }
        if (RES == 2) { c.mur = a.mean_r[o]; c.isr = a.invstd_r[o]; c.cr = a.coef_r[o]; }
    }
    bwd_apply_core<T, NT, GT, RES>(a, n, off, sc, fold, rg, rv, rr, ry, c);
}

// One 8-frame vector of the backward reduction: s0 = sum ga, s1 = sum ga * vhat, s3 = sum ga * vhat_r, m = max |ga|
// over its n (> 0) frames inside the sample.
template <typename T, typename NT, int RES>
__device__ __forceinline__ void reduce_core(int n, const uint4& rg, const uint4& rv, const uint4& rr, const uint4& ry,
                                            const BwdChan& c, float& s0, float& s1, float& s3, float& m_out) {
    float g[8], y[8], vn[8], vnr[8];
    cvt8<T>(rg, g);
    cvt8<NT>(rv, vn);
    const uint64_t nmu2 = pk::pack(-c.mu, -c.mu), is2 = pk::pack(c.is, c.is);
    uint64_t vn2[4], vr2[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) vn2[q] = pk::bn_norm2(pk::pack(vn[2 * q], vn[2 * q + 1]), nmu2, is2);
    if (RES == 2) {
        cvt8<NT>(rr, vnr);
        const uint64_t nmur2 = pk::pack(-c.mur, -c.mur), isr2 = pk::pack(c.isr, c.isr);
#pragma unroll
        for (int q = 0; q < 4; ++q) vr2[q] = pk::bn_norm2(pk::pack(vnr[2 * q], vnr[2 * q + 1]), nmur2, isr2);
    }
    bool gate[8];
    if (RES == 0) {          // gate from v (see bn_bwd_apply_fast_kernel)
        const uint64_t ga2 = pk::pack(c.ga, c.ga), be2 = pk::pack(c.be, c.be);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float a0, a1;
            pk::unpack(pk::fma(ga2, vn2[q], be2), a0, a1);
            gate[2 * q] = rounds_positive<T>(a0); gate[2 * q + 1] = rounds_positive<T>(a1);
        }
    } else {
        cvt8<T>(ry, y);
#pragma unroll
        for (int i = 0; i < 8; ++i) gate[i] = y[i] > 0.f;
    }
    uint64_t s0_2 = pk::pack(0.f, 0.f), s1_2 = pk::pack(0.f, 0.f), s3_2 = pk::pack(0.f, 0.f);
    float m = 0.f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float g0 = (2 * q < n && gate[2 * q]) ? g[2 * q] : 0.f;
        const float g1 = (2 * q + 1 < n && gate[2 * q + 1]) ? g[2 * q + 1] : 0.f;
        const uint64_t ga2 = pk::pack(g0, g1);
        s0_2 = pk::add(s0_2, ga2);
        s1_2 = pk::fma(ga2, vn2[q], s1_2);
        if (RES == 2) s3_2 = pk::fma(ga2, vr2[q], s3_2);
        m = fmaxf(m, fmaxf(fabsf(g0), fabsf(g1)));
    }
    float t0_, t1_;
    pk::unpack(s0_2, t0_, t1_); s0 = t0_ + t1_;
    pk::unpack(s1_2, t0_, t1_); s1 = t0_ + t1_;
    pk::unpack(s3_2, t0_, t1_); s3 = t0_ + t1_;
    m_out = m;
}

template <typename T, typename NT, int RES>
__device__ __forceinline__ void reduce_vec(const BnBwdArgs& a, int o, int n, const uint4& rg, const uint4& rv, const uint4& rr,
                                           const uint4& ry, float& s0, float& s1, float& s3, float& m_out) {
    BwdChan c{};
    c.mu = a.mean[o]; c.is = a.invstd[o];
    if (RES == 0) { c.ga = a.gamma[o]; c.be = a.beta[o]; }
    if (RES == 2) { c.mur = a.mean_r[o]; c.isr = a.invstd_r[o]; }
    reduce_core<T, NT, RES>(n, rg, rv, rr, ry, c, s0, s1, s3, m_out);
}

// ---- flattened fast paths (the encoder's configuration: BN + ReLU, residual joined before the ReLU,
// rows a multiple of 8 frames).  A warp takes 32 * V consecutive 8-frame vectors, lane l the vectors
// l, l + 32, ...: no row tails, and V independent 16-byte loads per tensor in flight per thread.
template <typename T, typename NT, int RES, int V>
__global__ void __launch_bounds__(256) bn_apply_fast_kernel(ApplyArgs a, int vpr, long long total) {
    pdl_sync();
    const uint32_t tid = blockIdx.x * 256u + threadIdx.x;        // the launcher guarantees total < 2^31
    const uint32_t base = (tid >> 5) * (32u * V) + (threadIdx.x & 31), tot = (uint32_t)total;
    size_t off[V]; int nin[V], ch[V];
    uint4 rv[V], rr[V];
#pragma unroll
    for (int j = 0; j < V; ++j) {
        const uint32_t idx = base + 32u * j;
        nin[j] = -1; ch[j] = 0; off[j] = 0;
        rv[j] = make_uint4(0, 0, 0, 0); rr[j] = make_uint4(0, 0, 0, 0);
        if (idx < tot) {
            const int row = (int)a.dvpr.div(idx), t0 = ((int)idx - row * vpr) * 8;
            const int b = (int)a.dC.div((uint32_t)row);
            ch[j] = row - b * a.C;
            nin[j] = max(0, min(a.len_out[b], a.Tp) - t0);
            off[j] = (size_t)row * a.Tp + t0;
            if (nin[j] > 0) {
                rv[j] = *reinterpret_cast<const uint4*>((const NT*)a.v + off[j]);
                if (RES == 1) rr[j] = *reinterpret_cast<const uint4*>((const T*)a.xres + off[j]);
                if (RES == 2) rr[j] = *reinterpret_cast<const uint4*>((const NT*)a.vr + off[j]);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < V; ++j) {
        if (nin[j] < 0) continue;
        apply_vec<T, NT, RES>(a, ch[j], nin[j], off[j], rv[j], rr[j]);
    }
}

template <typename T, typename NT, typename GT, int RES, int V>
__global__ void __launch_bounds__(256) bn_bwd_apply_fast_kernel(BnBwdArgs a, int vpr, long long total) {
    pdl_sync();
    const uint32_t tid = blockIdx.x * 256u + threadIdx.x;        // the launcher guarantees total < 2^31
    const uint32_t base = (tid >> 5) * (32u * V) + (threadIdx.x & 31), tot = (uint32_t)total;
    const float sc = a.gmax ? pow2_scale(*a.gmax) : 1.f;          // multiplying by it is exact: a power of two
    const bool fold = !a.gv16 && a.gv_scaled;
    size_t off[V]; int nin[V], ch[V];
    uint4 rg[V], rv[V], rr[V], ry[V];
#pragma unroll
    for (int j = 0; j < V; ++j) {
        const uint32_t idx = base + 32u * j;
        nin[j] = -1; ch[j] = 0; off[j] = 0;
        rg[j] = rv[j] = rr[j] = ry[j] = make_uint4(0, 0, 0, 0);
        if (idx < tot) {
            const int row = (int)a.dvpr.div(idx), t0 = ((int)idx - row * vpr) * 8;
            const int b = (int)a.dC.div((uint32_t)row);
            ch[j] = row - b * a.C;
            nin[j] = max(0, min(a.len_out[b], a.Tp) - t0);        // frames of this vector inside the sample
            off[j] = (size_t)row * a.Tp + t0;
            if (nin[j] > 0) {
                rg[j] = *reinterpret_cast<const uint4*>((const T*)a.g + off[j]);
                rv[j] = *reinterpret_cast<const uint4*>((const NT*)a.v + off[j]);
                if (RES == 2) rr[j] = *reinterpret_cast<const uint4*>((const NT*)a.vr + off[j]);
                if (RES != 0) ry[j] = *reinterpret_cast<const uint4*>((const T*)a.y + off[j]);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < V; ++j) {
        if (nin[j] < 0) continue;
        bwd_apply_vec<T, NT, GT, RES>(a, ch[j], nin[j], off[j], sc, fold, rg[j], rv[j], rr[j], ry[j]);
    }
}

// Flattened reduce: a warp's 32 * V consecutive vectors belong to at most two rows (vpr >= 32 * V), so two
// masked warp reductions give one partial per (row, warp) pair.  Row r's partials sit in slots
// [0, last_warp(r) - first_warp(r)] with first_warp(r) = (r * vpr) / (32 * V): a static assignment,
// summed later in slot order.
template <typename T, typename NT, int RES, int V>
__global__ void __launch_bounds__(256) bn_bwd_reduce_fast_kernel(BnBwdArgs a, int vpr, long long total) {
    pdl_sync();
    const uint32_t tid = blockIdx.x * 256u + threadIdx.x;        // the launcher guarantees total < 2^31
    const int lane = threadIdx.x & 31;
    const uint32_t wg = tid >> 5;                                // global warp index
    const uint32_t warp_first = wg * (32u * V), tot = (uint32_t)total;
    if (warp_first >= tot) return;
    const int row0 = (int)a.dvpr.div(warp_first);
    int nin[V], ch[V], rw[V];
    uint4 rg[V], rv[V], rr[V], ry[V];
#pragma unroll
    for (int j = 0; j < V; ++j) {
        const uint32_t idx = warp_first + 32u * j + lane;
        nin[j] = 0; ch[j] = 0; rw[j] = row0;
        rg[j] = rv[j] = rr[j] = ry[j] = make_uint4(0, 0, 0, 0);
        if (idx < tot) {
            const int row = (int)a.dvpr.div(idx), t0 = ((int)idx - row * vpr) * 8;
            const int b = (int)a.dC.div((uint32_t)row);
            rw[j] = row; ch[j] = row - b * a.C;
            nin[j] = max(0, min(a.len_out[b], a.Tp) - t0);
            if (nin[j] > 0) {
                const size_t off = (size_t)row * a.Tp + t0;
                rg[j] = *reinterpret_cast<const uint4*>((const T*)a.g + off);
                rv[j] = *reinterpret_cast<const uint4*>((const NT*)a.v + off);
                if (RES == 2) rr[j] = *reinterpret_cast<const uint4*>((const NT*)a.vr + off);
                if (RES != 0) ry[j] = *reinterpret_cast<const uint4*>((const T*)a.y + off);
            }
        }
    }
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    float amx[2] = {0.f, 0.f};
#pragma unroll
    for (int j = 0; j < V; ++j) {
        const int n = nin[j];
        if (n <= 0) continue;
        float s0, s1, s3, m;
        reduce_vec<T, NT, RES>(a, ch[j], n, rg[j], rv[j], rr[j], ry[j], s0, s1, s3, m);
        const int seg = rw[j] != row0 ? 1 : 0;
        acc[seg][0] += s0; acc[seg][1] += s1; acc[seg][2] += s0; acc[seg][3] += s3;
        amx[seg] = fmaxf(amx[seg], m);
    }
#pragma unroll
    for (int seg = 0; seg < 2; ++seg) {
        const int r = row0 + seg;
        const uint32_t rfirst = (uint32_t)r * (uint32_t)vpr;           // first vector of row r
        if (seg == 1 && rfirst >= warp_first + 32u * V) break;         // warp lies inside one row (uniform)
        float v[4] = {acc[seg][0], acc[seg][1], RES == 2 ? acc[seg][2] : 0.f, RES == 2 ? acc[seg][3] : 0.f};
#pragma unroll
        for (int i = 0; i < (RES == 2 ? 4 : 2); ++i) v[i] = warp_sum(v[i]);
        const float m = a.gmax ? warp_max(amx[seg]) : 0.f;
        if (lane == 0 && rfirst < tot) {
            const int slot = (int)(wg - rfirst / (32u * V));
            const int b = (int)a.dC.div((uint32_t)r), o = r - b * a.C;
            a.partials[bwd_part_index(a, b, slot, o)] = make_float4(v[0], v[1], v[2], v[3]);
            if (a.gmax) a.amax_part[bwd_part_index(a, b, slot, o)] = m;
        }
    }
}

// ---- channel-per-CTA backward reduction ----------------------------------------------------------------
// One CTA streams channel o of every sample: B * vpr 8-frame vectors, numbered sample-major, thread t the vectors
// t, t + blockDim, ... in batches of U independent 16-byte loads per tensor, sums in registers.  Because the CTA sees
// the whole channel it needs no per-row partials and no finalize launch: it ends with the channel's coefficients.
// (The same mapping was measured for the two apply kernels and lost to the flattened one: a CTA that hops between
// the 32 rows of a channel streams about 10 % slower than one that walks the tensor in address order, and a forward
// apply that merges the contraction's statistics partials in its prologue pays that merge once per CTA.)
constexpr int kChThreads = 512;

// Backward reduction of channel o over every sample, then the channel's coefficients, parameter gradients and its
// term of the bound on |gv| (what bn_bwd_finalize_kernel does for the row-mapped reduction).
template <typename T, typename NT, int RES>
__global__ void __launch_bounds__(kChThreads, 2)
bn_bwd_reduce_ch_kernel(BnBwdArgs a, int vpr, const float* gamma_r, float* dgamma, float* dbeta, float* dgamma_r,
                        float* dbeta_r, int accumulate) {
    pdl_sync();
    constexpr int NT_ = kChThreads;
    constexpr int U = RES == 2 ? 2 : 4;            // 16-byte loads in flight per thread: U * (2 or 4 tensors)
    __shared__ float4 s_sum[NT_ / 32];
    const int o = blockIdx.x, tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    BwdChan c{};
    c.mu = a.mean[o]; c.is = a.invstd[o];
    if (RES == 0) { c.ga = a.gamma[o]; c.be = a.beta[o]; }
    if (RES == 2) { c.mur = a.mean_r[o]; c.isr = a.invstd_r[o]; }
    const int nvec = a.B * vpr;
    float s0 = 0.f, s1 = 0.f, s3 = 0.f, amax = 0.f;
    for (int jb = tid; jb < nvec; jb += U * NT_) {
        int nin[U];
        uint4 rg[U], rv[U], rr[U], ry[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int j = jb + u * NT_;
            nin[u] = 0;
            rg[u] = rv[u] = rr[u] = ry[u] = make_uint4(0, 0, 0, 0);
            if (j < nvec) {
                const int b = (int)a.dvpr.div((uint32_t)j), t0 = (j - b * vpr) * 8;
                nin[u] = max(0, min(a.len_out[b], a.Tp) - t0);
                if (nin[u] > 0) {
                    const size_t off = ((size_t)b * a.C + o) * a.Tp + t0;
                    rg[u] = *reinterpret_cast<const uint4*>((const T*)a.g + off);
                    rv[u] = *reinterpret_cast<const uint4*>((const NT*)a.v + off);
                    if (RES == 2) rr[u] = *reinterpret_cast<const uint4*>((const NT*)a.vr + off);
                    if (RES != 0) ry[u] = *reinterpret_cast<const uint4*>((const T*)a.y + off);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (nin[u] <= 0) continue;
            float q0, q1, q3, m;
            reduce_core<T, NT, RES>(nin[u], rg[u], rv[u], rr[u], ry[u], c, q0, q1, q3, m);
            s0 += q0; s1 += q1; s3 += q3; amax = fmaxf(amax, m);
        }
    }
    s0 = warp_sum(s0); s1 = warp_sum(s1);
    if (RES == 2) s3 = warp_sum(s3);
    if (a.gmax) amax = warp_max(amax);
    if (lane == 0) s_sum[w] = make_float4(s0, s1, s3, amax);
    __syncthreads();
    if (tid != 0) return;
    float d0 = 0.f, d1 = 0.f, d3 = 0.f;
    amax = 0.f;
#pragma unroll
    for (int i = 0; i < NT_ / 32; ++i) {                // warp order: bit-repeatable
        const float4 q = s_sum[i];
        d0 += q.x; d1 += q.y; d3 += q.z; amax = fmaxf(amax, q.w);
    }
    const float N = (float)(*a.nvalid);
    const float k = a.gamma[o] * c.is;
    const float kr = RES == 2 ? gamma_r[o] * c.isr : 0.f;
    if (a.gmax) {            // see bn_bwd_finalize_kernel
        float bound = fabsf(k) * (amax + fabsf(d0) / N + sqrtf(N) * fabsf(d1) / N);
        if (RES == 2) bound = fmaxf(bound, fabsf(kr) * (amax + fabsf(d0) / N + sqrtf(N) * fabsf(d3) / N));
        if (bound < 3.0e38f) atomicMax(reinterpret_cast<unsigned int*>(a.gmax), __float_as_uint(bound));
    }
    auto put = [&](float* dst, float val) {
        if (dst) dst[o] = accumulate ? dst[o] + val : val;
    };
    put(dbeta, d0); put(dgamma, d1);
    a.coef[o] = make_float4(k, d0 / N, d1 / N, 0.f);
    if (RES == 2) {
        put(dbeta_r, d0); put(dgamma_r, d3);            // the residual sum receives the same gated gradient
        a.coef_r[o] = make_float4(kr, d0 / N, d3 / N, 0.f);
    }
}

template <typename T>
__global__ void __launch_bounds__(kRowThreads)
ew_add_masked_kernel(T* out, const T* a, const T* b, const T* c, const int* len, int nrows, int C, int Tt) {
    pdl_sync();
    SC_ROW_SETUP(nrows)
    const int bb = row / C;
    const int l = min(len[bb], Tt);
    const bool vec = (Tt % 8 == 0);
    const size_t off = (size_t)row * Tt;
    for (int t0 = lane * 8; t0 < Tt; t0 += 256) {
        float f[8];
        if (t0 < l) {
            load_chunk(a + off, t0, Tt, vec, f);
            if (b) { float q[8]; load_chunk(b + off, t0, Tt, vec, q);
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] += q[i]; }
            if (c) { float q[8]; load_chunk(c + off, t0, Tt, vec, q);
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] += q[i]; }
#pragma unroll
            for (int i = 0; i < 8; ++i) if (t0 + i >= l) f[i] = 0.f;
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = 0.f;
        }
        store_chunk(out + off, t0, Tt, vec, f);
    }
}

}  // namespace

#define SC_DISPATCH3(dtype, ...)                                                              \
    switch (dtype) {                                                                          \
        case F32: { using T = float; using NT = float; __VA_ARGS__; break; }                  \
        case F16: { using T = __half; using NT = __half; __VA_ARGS__; break; }                \
        default:  { using T = __nv_bfloat16; using NT = __half; __VA_ARGS__; break; }         \
    }
// 16-bit activation types only (the flattened kernels move 16-byte vectors of 8 elements)
#define SC_DISPATCH16(dtype, ...)                                                             \
    if (dtype == F16) { using T = __half; using NT = __half; __VA_ARGS__; }                   \
    else { using T = __nv_bfloat16; using NT = __half; __VA_ARGS__; }
#define SC_DISPATCH(dtype, ...)                                             \
    switch (dtype) {                                                        \
        case F32: { using T = float; __VA_ARGS__; break; }                  \
        case F16: { using T = __half; __VA_ARGS__; break; }                 \
        default:  { using T = __nv_bfloat16; __VA_ARGS__; break; }          \
    }

void lengths(const Launch& L, const int* len_in, int B, int T_in, int stride, int* len_out, int* nvalid, int* blk_off) {
    KScope ks_(L, KC_LENGTHS, 8.0 * B, 0.0);
    launch_k(L, lengths_kernel, 1, 256, 0, len_in, B, T_in, stride, len_out, nvalid, blk_off, L.status);
    L.count();
}

void bn_stats(const Launch& L, int vdtype, const void* v, const int* len_out, int B, int C, int Tp,
              float2* partials) {
    KScope ks_(L, KC_BN_STATS, (double)dtype_size(vdtype) * B * C * Tp, 0.0);
    if (vdtype == F32) launch_k(L, bn_stats_kernel<float>, (B * C + kRowsPerCta - 1) / kRowsPerCta, kRowThreads, 0, (const float*)v, len_out, B * C, C, Tp, partials);
    else launch_k(L, bn_stats_kernel<__half>, (B * C + kRowsPerCta - 1) / kRowsPerCta, kRowThreads, 0, (const __half*)v, len_out, B * C, C, Tp, partials);
    L.count();
}

void bn_finalize(const Launch& L, const float2* partials, int parts_per_b, int tile_w, const int* len_out,
                 const int* nvalid, int B, int C, float eps, float momentum, float* mean, float* invstd,
                 float* running_mean, float* running_var) {
    KScope ks_(L, KC_BN_FINALIZE, 8.0 * B * parts_per_b * C, 0.0);
    launch_k(L, bn_finalize_kernel, (C + 31) / 32, 32 * kFinWarps, 0, partials, parts_per_b, tile_w, len_out, nvalid, B, C,
                                                                     eps, momentum, mean, invstd, running_mean, running_var);
    L.count();
}

void bn_finalize_flat(const Launch& L, const float4* partials, int grid, int tiles_m, int rows_per_tile,
                      const int* blk_off, const int* nvalid, int B, int C, float eps, float momentum, float* mean,
                      float* invstd, float* running_mean, float* running_var) {
    KScope ks_(L, KC_BN_FINALIZE, 16.0 * grid * C / std::max(1, tiles_m), 0.0);
    launch_k(L, bn_finalize_flat_kernel, (C + 31) / 32, 32 * kFinWarps, 0, partials, grid, tiles_m, rows_per_tile, blk_off, nvalid, B,
                                                                          C, eps, momentum, mean, invstd, running_mean, running_var);
    L.count();
}

// the flattened kernels index with 32 bits
static bool fits32(int B, int C, int Tp) { return (long long)B * C * (Tp / 8) < (1ll << 31) && (long long)B * C * Tp < (1ll << 31); }
static unsigned fast_grid(long long total, int V) { return (unsigned)((total + 256ll * V - 1) / (256ll * V)); }

// Algorithmic bytes per element of the batch-norm kernels: every tensor they must read or write, once.
// The channel-per-CTA reduction pays off once a channel holds a few vectors per thread; below that (or with few
// channels) the row-mapped kernel and its separate finalize step are used.
static bool channel_mapped(int B, int C, int Tp) { return C >= 32 && (long long)B * (Tp / 8) >= 1024; }

void bn_apply(const Launch& L, int dtype, const ApplyArgs& a_in) {
    ApplyArgs a = a_in;
    const double e = (double)dtype_size(dtype), en = (double)dtype_size(ntype_of(dtype));
    KScope ks_(L, KC_BN_APPLY, (double)a.B * a.C * a.Tp * (en + e + (a.residual == 1 ? e : 0) + (a.residual == 2 ? en : 0)), 0.0);
    if (dtype != F32 && a.Tp % 8 == 0 && a.has_relu && a.res_before_relu && fits32(a.B, a.C, a.Tp)) {
        const int vpr = a.Tp / 8;
        a.dvpr = FastDiv((uint32_t)vpr); a.dC = FastDiv((uint32_t)a.C);
        const long long total = (long long)a.B * a.C * vpr;
        const unsigned grid = fast_grid(total, 2);
#define SC_APPLY_FAST(RES) SC_DISPATCH16(dtype, (launch_k(L, bn_apply_fast_kernel<T, NT, RES, 2>, grid, 256, 0, a, vpr, total)))
        if (a.residual == 0) { SC_APPLY_FAST(0); } else if (a.residual == 1) { SC_APPLY_FAST(1); } else { SC_APPLY_FAST(2); }
#undef SC_APPLY_FAST
        L.count();
        return;
    }
    SC_DISPATCH3(dtype, (launch_k(L, bn_apply_kernel<T, NT>, (a.B * a.C + kRowsPerCta - 1) / kRowsPerCta, kRowThreads, 0, a)));
    L.count();
}

void bn_bwd_reduce(const Launch& L, int dtype, BnBwdArgs& a) {
    a.nslots = 1; a.vpw = 32; a.vpw_shift = 5;
    const double e = (double)dtype_size(dtype), en = (double)dtype_size(ntype_of(dtype));
    if (dtype != F32 && a.Tp % 8 == 0 && a.Tp >= 256 && a.has_bn && a.has_relu && a.res_before_relu && fits32(a.B, a.C, a.Tp)) {
        a.dvpr = FastDiv((uint32_t)(a.Tp / 8)); a.dC = FastDiv((uint32_t)a.C);
        KScope ks2_(L, KC_BN_BWD_REDUCE, (double)a.B * a.C * a.Tp * (e * (a.residual == 0 ? 1 : 2) + en * (a.residual == 2 ? 2 : 1)), 0.0);
        const int vpr = a.Tp / 8;
        a.nslots = bn_bwd_max_slots(a.Tp);
        const long long total = (long long)a.B * a.C * vpr;
        const int V = vpr >= 64 ? 2 : 1;
        a.vpw = 32 * V; a.vpw_shift = V == 2 ? 6 : 5;
        const unsigned grid = fast_grid(total, V);
#define SC_RED_FAST(RES)                                                                                                   \
        if (V == 2) { SC_DISPATCH16(dtype, (launch_k(L, bn_bwd_reduce_fast_kernel<T, NT, RES, 2>, grid, 256, 0, a, vpr, total))); } \
        else { SC_DISPATCH16(dtype, (launch_k(L, bn_bwd_reduce_fast_kernel<T, NT, RES, 1>, grid, 256, 0, a, vpr, total))); }
        if (a.residual == 2) { SC_RED_FAST(2); } else if (a.residual == 1) { SC_RED_FAST(1); } else { SC_RED_FAST(0); }
#undef SC_RED_FAST
        L.count();
        return;
    }
    KScope ks_(L, KC_BN_BWD_REDUCE, (double)a.B * a.C * a.Tp * (e * (a.has_relu && a.res_before_relu ? 2 : 1) + (a.has_bn ? en : 0) + (a.residual == 2 ? en : 0)), 0.0);
    SC_DISPATCH3(dtype, (launch_k(L, bn_bwd_reduce_kernel<T, NT>, (a.B * a.C + kRowsPerCta - 1) / kRowsPerCta, kRowThreads, 0, a)));
    L.count();
}

void bn_bwd_finalize(const Launch& L, const BnBwdArgs& a, const float* gamma, const float* gamma_r,
                     float* dgamma, float* dbeta, float* dgamma_r, float* dbeta_r, float* dbias,
                     int accumulate) {
    KScope ks_(L, KC_BN_BWD_FINALIZE, 16.0 * a.B * a.C * a.nslots, 0.0);
    launch_k(L, bn_bwd_finalize_kernel, (a.C + 31) / 32, 32 * kFinWarps, 0, a, gamma, gamma_r, dgamma, dbeta, dgamma_r,
                                                                          dbeta_r, dbias, accumulate);
    L.count();
}

void bn_bwd_reduce_finalize(const Launch& L, int dtype, BnBwdArgs& a, const float* gamma, const float* gamma_r,
                            float* dgamma, float* dbeta, float* dgamma_r, float* dbeta_r, float* dbias, int accumulate) {
    const bool fast = dtype != F32 && a.Tp % 8 == 0 && a.has_bn && a.has_relu && a.res_before_relu && fits32(a.B, a.C, a.Tp);
    if (fast && channel_mapped(a.B, a.C, a.Tp)) {
        a.nslots = 1; a.vpw = 32; a.vpw_shift = 5;
        const double e = (double)dtype_size(dtype), en = (double)dtype_size(ntype_of(dtype));
        KScope ks_(L, KC_BN_BWD_REDUCE, (double)a.B * a.C * a.Tp * (e * (a.residual == 0 ? 1 : 2) + en * (a.residual == 2 ? 2 : 1)), 0.0);
        const int vpr = a.Tp / 8;
        a.dvpr = FastDiv((uint32_t)vpr);
#define SC_RED_CH(RES) SC_DISPATCH16(dtype, (launch_k(L, bn_bwd_reduce_ch_kernel<T, NT, RES>, (unsigned)a.C, kChThreads, 0, a, vpr, \
                                                       gamma_r, dgamma, dbeta, dgamma_r, dbeta_r, accumulate)))
        if (a.residual == 2) { SC_RED_CH(2); } else if (a.residual == 1) { SC_RED_CH(1); } else { SC_RED_CH(0); }
#undef SC_RED_CH
        L.count();
        return;
    }
    bn_bwd_reduce(L, dtype, a);
    bn_bwd_finalize(L, a, gamma, gamma_r, dgamma, dbeta, dgamma_r, dbeta_r, dbias, accumulate);
}

void bn_bwd_apply(const Launch& L, int dtype, const BnBwdArgs& a_in) {
    BnBwdArgs a = a_in;
    const bool fast_apply = dtype != F32 && a.Tp % 8 == 0 && a.has_bn && a.has_relu && a.res_before_relu && fits32(a.B, a.C, a.Tp);
    const double e = (double)dtype_size(dtype), en = (double)dtype_size(ntype_of(dtype));
    KScope ks_(L, KC_BN_BWD_APPLY, (double)a.B * a.C * a.Tp * (e * (a.has_relu && a.res_before_relu && !(fast_apply && a.residual == 0) ? 2 : 1) + (a.has_bn ? en : 0) + (a.residual == 2 ? en : 0) + (double)dtype_size(a.gv_dtype) + (a.residual != 0 ? e : 0)), 0.0);
    if (fast_apply) {
        const int vpr = a.Tp / 8;
        a.dvpr = FastDiv((uint32_t)vpr); a.dC = FastDiv((uint32_t)a.C);
        const long long total = (long long)a.B * a.C * vpr;
        const unsigned grid = fast_grid(total, 2);
#define SC_BWD_FAST(RES)                                                                                             \
        if (dtype == BF16 && a.gv_dtype == F16)                                                                      \
            launch_k(L, bn_bwd_apply_fast_kernel<__nv_bfloat16, __half, __half, RES, 2>, grid, 256, 0, a, vpr, total); \
        else { SC_DISPATCH16(dtype, (launch_k(L, bn_bwd_apply_fast_kernel<T, NT, T, RES, 2>, grid, 256, 0, a, vpr, total))); }
        if (a.residual == 0) { SC_BWD_FAST(0); } else if (a.residual == 1) { SC_BWD_FAST(1); } else { SC_BWD_FAST(2); }
#undef SC_BWD_FAST
        L.count();
        return;
    }
    if (dtype == BF16 && a.gv_dtype == F16)
        launch_k(L, bn_bwd_apply_kernel<__nv_bfloat16, __half, __half>, (a.B * a.C + kRowsPerCta - 1) / kRowsPerCta, kRowThreads, 0, a);
    else
        SC_DISPATCH3(dtype, (launch_k(L, bn_bwd_apply_kernel<T, NT, T>, (a.B * a.C + kRowsPerCta - 1) / kRowsPerCta, kRowThreads, 0, a)));
    L.count();
}

void ew_add_masked(const Launch& L, int dtype, void* out, const void* a, const void* b, const void* c,
                   const int* len, int B, int C, int Tt) {
    KScope ks_(L, KC_EW, (double)dtype_size(dtype) * B * C * Tt * (2 + (b ? 1 : 0) + (c ? 1 : 0)), 0.0);
    SC_DISPATCH(dtype, (launch_k(L, ew_add_masked_kernel<T>, (B * C + kRowsPerCta - 1) / kRowsPerCta, kRowThreads, 0, (T*)out, (const T*)a, (const T*)b,
                                                                                      (const T*)c, len, B * C, C, Tt)));
    L.count();
}

__global__ void convert_bf16_to_f16_kernel(const __nv_bfloat16* __restrict__ src, __half* __restrict__ dst, long long n) {
    pdl_sync();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = __float2half_rn(__bfloat162float(src[i]));
}
void convert_bf16_to_f16(const Launch& L, const void* src, void* dst, int64_t n) {
    KScope ks_(L, KC_EW, 4.0 * n, 0.0);
    launch_k(L, convert_bf16_to_f16_kernel, (unsigned)((n + 255) / 256), 256, 0, (const __nv_bfloat16*)src, (__half*)dst, n);
    L.count();
}

__global__ void convert_many_kernel(ConvertList list) {
    pdl_sync();
    const int item = blockIdx.y;
    const __nv_bfloat16* src = (const __nv_bfloat16*)list.src[item];
    __half* dst = (__half*)list.dst[item];
    const int n = list.n[item];
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
        dst[i] = __float2half_rn(__bfloat162float(src[i]));
}
void convert_bf16_to_f16_many(const Launch& L, const ConvertList& list) {
    if (list.count == 0) return;
    double total = 0;
    for (int i = 0; i < list.count; ++i) total += list.n[i];
    KScope ks_(L, KC_EW, 4.0 * total, 0.0);
    launch_k(L, convert_many_kernel, dim3(64, list.count), 256, 0, list);
    L.count();
}

namespace {
// one 8-frame vector per thread (rows are a multiple of 8 frames) or one element per thread
__global__ void __launch_bounds__(256)
mask_convert_f16_kernel(__half* __restrict__ out, const __nv_bfloat16* __restrict__ in, const int* __restrict__ len,
                        int C, int Tt, long long total, int vec, int* status) {
    pdl_sync();
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    if (idx >= total) return;
    const int per_row = vec ? Tt / 8 : Tt;
    const long long row = idx / per_row;
    const int t0 = (int)(idx - row * per_row) * (vec ? 8 : 1);
    const int l = min(len[row / C], Tt);
    const size_t off = (size_t)row * Tt + t0;
    bool over = false;
    if (vec) {
        float f[8];
        if (t0 < l) {
            ld8<__nv_bfloat16>(in + off, f);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (t0 + i >= l) f[i] = 0.f;
                if (fabsf(f[i]) > 65504.f) { f[i] = copysignf(65504.f, f[i]); over = true; }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = 0.f;
        }
        st8<__half>(out + off, f);
    } else {
        float f = t0 < l ? __bfloat162float(in[off]) : 0.f;
        if (fabsf(f) > 65504.f) { f = copysignf(65504.f, f); over = true; }
        out[off] = __float2half_rn(f);
    }
    if (over) raise_status(status, kErrRange);
}
}  // namespace

void mask_convert_f16(const Launch& L, void* out, const void* in, const int* len, int B, int C, int Tt) {
    KScope ks_(L, KC_EW, 4.0 * B * C * Tt, 0.0);
    const int vec = (Tt % 8 == 0) ? 1 : 0;
    const long long total = (long long)B * C * (vec ? Tt / 8 : Tt);
    launch_k(L, mask_convert_f16_kernel, (unsigned)((total + 255) / 256), 256, 0, (__half*)out, (const __nv_bfloat16*)in, len,
                                                                                C, Tt, total, vec, L.status);
    L.count();
}

void mask_copy(const Launch& L, int dtype, void* out, const void* in, const int* len, int B, int C, int Tt) {
    ew_add_masked(L, dtype, out, in, nullptr, nullptr, len, B, C, Tt);
}

}  // namespace sc
