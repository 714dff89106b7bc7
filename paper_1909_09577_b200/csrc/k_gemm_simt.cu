// Pointwise (1x1) convolution as plain SIMT tiled GEMMs with fp32 accumulation.
// These serve the fp32 path (whose tolerance rules out reduced-precision tensor-core formats) and
// any shape the tensor-core kernels do not tile.  64x64 output tile, 16-deep k-steps, 4x4 per thread.
#include "common.cuh"
#include "kernels.h"

namespace sc {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, NT = 256;

// D[m,n] = sum_k A(m,k) * B(k,n) for one z-slice; operand access is described by strides so that the
// three contractions (forward, input gradient, weight gradient) share the kernel.
struct GemmDesc {
    int M, N, Kd;
    // A(m,k) = a[z*a_z + m*a_m + k*a_k];  B(k,n) = b[z*b_z + k*b_k + n*b_n]
    long long a_z, a_m, a_k, b_z, b_k, b_n;
    // weight gradient: k runs over (sample, frame): k -> (k / kt) * kz + (k % kt) for both operands
    int kt; long long a_kz, b_kz;
    int k_begin_per_z, k_len_per_z;   // split-K: slice z covers k in [z*k_len, (z+1)*k_len)
};

template <typename X> struct IsHalf { static constexpr bool value = false; };
template <> struct IsHalf<__half> { static constexpr bool value = true; };

template <typename T, typename OT, int MODE>   // MODE 0: fwd (bias+mask, T out) 1: dgrad (T out) 2: wgrad (float partial out)
__global__ void __launch_bounds__(NT)
gemm_simt_kernel(GemmDesc d, const T* __restrict__ a, const T* __restrict__ b, void* __restrict__ out,
                 const float* __restrict__ bias, const int* __restrict__ len_out, int* status) {
    pdl_sync();
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int z = blockIdx.z;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    int kb = 0, ke = d.Kd;
    const T* ap = a; const T* bp = b;
    if (MODE == 2) { kb = z * d.k_len_per_z; ke = min(d.Kd, kb + d.k_len_per_z); }
    else { ap += (long long)z * d.a_z; bp += (long long)z * d.b_z; }

    // fwd-mode early exit: tile wholly in padding -> zeros
    if (MODE == 0 && len_out && n0 >= len_out[z]) {
        OT* o = (OT*)out + (long long)z * d.M * d.N;
        for (int i = tid; i < BM * BN; i += NT) {
            const int m = m0 + i / BN, n = n0 + i % BN;
            if (m < d.M && n < d.N) stf(o + (long long)m * d.N + n, 0.f);
        }
        return;
    }

    for (int k0 = kb; k0 < ke; k0 += BK) {
        // A tile: choose the thread->element map by which index is contiguous in memory
        for (int i = tid; i < BM * BK; i += NT) {
            int m, k;
            if (d.a_k == 1 || MODE == 2) { k = i % BK; m = i / BK; } else { m = i % BM; k = i / BM; }
            const int gm = m0 + m, gk = k0 + k;
            float v = 0.f;
            if (gm < d.M && gk < ke) {
                long long off = (MODE == 2) ? (long long)(gk / d.kt) * d.a_kz + (gk % d.kt) + (long long)gm * d.a_m
                                            : (long long)gm * d.a_m + (long long)gk * d.a_k;
                v = ldf(ap + off);
            }
            As[k][m] = v;
        }
        for (int i = tid; i < BN * BK; i += NT) {
            int n, k;
            if (MODE == 2) { k = i % BK; n = i / BK; } else { n = i % BN; k = i / BN; }
            const int gn = n0 + n, gk = k0 + k;
            float v = 0.f;
            if (gn < d.N && gk < ke) {
                long long off = (MODE == 2) ? (long long)(gk / d.kt) * d.b_kz + (gk % d.kt) + (long long)gn * d.b_n
                                            : (long long)gk * d.b_k + (long long)gn * d.b_n;
                v = ldf(bp + off);
            }
            Bs[k][n] = v;
        }
        __syncthreads();
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
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= d.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= d.N) continue;
            if (MODE == 0) {
                float v = acc[i][j] + (bias ? bias[m] : 0.f);
                if (len_out && n >= len_out[z]) v = 0.f;
                if (sizeof(OT) == 2 && fabsf(v) > 65504.f && IsHalf<OT>::value) { v = copysignf(65504.f, v); raise_status(status, kErrRange); }
                stf((OT*)out + ((long long)z * d.M + m) * d.N + n, v);
            } else if (MODE == 1) {
                stf((OT*)out + ((long long)z * d.M + m) * d.N + n, acc[i][j]);
            } else {
                ((float*)out)[((long long)z * d.M + m) * d.N + n] = acc[i][j];
            }
        }
    }
}

__global__ void reduce_partials_kernel(const float* __restrict__ p, int nsplit, long long n,
                                       float* __restrict__ out, int accumulate, const float* __restrict__ gmax) {
    pdl_sync();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = 0.f;
    for (int k = 0; k < nsplit; ++k) s += p[(long long)k * n + i];
    if (gmax) s *= 1.f / pow2_scale(*gmax);
    out[i] = accumulate ? out[i] + s : s;
}

// Four consecutive elements per thread, eight splits in flight at a time; the order of the additions
// is the same as in the scalar kernel (split 0 first), so both give the same bits.
__global__ void __launch_bounds__(256)
reduce_partials_vec4_kernel(const float4* __restrict__ p, int nsplit, long long n4, float4* __restrict__ out,
                            int accumulate, const float* __restrict__ gmax) {
    pdl_sync();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    int k = 0;
    for (; k + 8 <= nsplit; k += 8) {
        float4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = p[(long long)(k + j) * n4 + i];
#pragma unroll
        for (int j = 0; j < 8; ++j) { s.x += v[j].x; s.y += v[j].y; s.z += v[j].z; s.w += v[j].w; }
    }
    for (; k < nsplit; ++k) {
        const float4 v = p[(long long)k * n4 + i];
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    if (gmax) { const float r = 1.f / pow2_scale(*gmax); s.x *= r; s.y *= r; s.z *= r; s.w *= r; }
    if (accumulate) { const float4 o = out[i]; s.x += o.x; s.y += o.y; s.z += o.z; s.w += o.w; }
    out[i] = s;
}

}  // namespace

#define SC_DISPATCH(dtype, ...)                                             \
    switch (dtype) {                                                        \
        case F32: { using T = float; __VA_ARGS__; break; }                  \
        case F16: { using T = __half; __VA_ARGS__; break; }                 \
        default:  { using T = __nv_bfloat16; __VA_ARGS__; break; }          \
    }

void reduce_partials(const Launch& L, const float* partials, int nsplit, int64_t n, float* out, int accumulate,
                     const float* gmax) {
    KScope ks_(L, KC_REDUCE, 4.0 * (nsplit + 1) * n, 0.0);
    if (n % 4 == 0 && (reinterpret_cast<uintptr_t>(partials) & 15) == 0 && (reinterpret_cast<uintptr_t>(out) & 15) == 0)
        launch_k(L, reduce_partials_vec4_kernel, (unsigned)((n / 4 + 255) / 256), 256, 0, 
            reinterpret_cast<const float4*>(partials), nsplit, n / 4, reinterpret_cast<float4*>(out), accumulate, gmax);
    else
        launch_k(L, reduce_partials_kernel, (unsigned)((n + 255) / 256), 256, 0, partials, nsplit, n, out, accumulate, gmax);
    L.count();
}

void gemm_fwd_simt(const Launch& L, int dtype, const void* w, const void* u, const float* bias, void* v,
                   int out_dtype, const int* len_out, int B, int Cin, int Cout, int Tp) {
    KScope ks_(L, KC_PW_FWD, (double)B * Tp * (dtype_size(dtype) * Cin + dtype_size(out_dtype) * Cout), 2.0 * B * Tp * Cin * Cout);
    GemmDesc d{};
    d.M = Cout; d.N = Tp; d.Kd = Cin;
    d.a_z = 0; d.a_m = Cin; d.a_k = 1;
    d.b_z = (long long)Cin * Tp; d.b_k = Tp; d.b_n = 1;
    dim3 grid((Tp + BN - 1) / BN, (Cout + BM - 1) / BM, B);
    if (out_dtype == dtype) {
        SC_DISPATCH(dtype, (launch_k(L, gemm_simt_kernel<T, T, 0>, grid, NT, 0, d, (const T*)w, (const T*)u, v, bias, len_out, L.status)));
    } else if (dtype == BF16 && out_dtype == F16) {   // bfloat16 operands, float16 result
        launch_k(L, gemm_simt_kernel<__nv_bfloat16, __half, 0>, grid, NT, 0, d, (const __nv_bfloat16*)w, (const __nv_bfloat16*)u, v, bias, len_out, L.status);
    } else if (dtype == BF16) {   // 16-bit operands, float result
        launch_k(L, gemm_simt_kernel<__nv_bfloat16, float, 0>, grid, NT, 0, d, (const __nv_bfloat16*)w, (const __nv_bfloat16*)u, v, bias, len_out, L.status);
    } else {
        launch_k(L, gemm_simt_kernel<__half, float, 0>, grid, NT, 0, d, (const __half*)w, (const __half*)u, v, bias, len_out, L.status);
    }
    L.count();
}

void gemm_dgrad_simt(const Launch& L, int dtype, const void* w, const void* gv, void* gu, int B, int Cin,
                     int Cout, int Tp) {
    KScope ks_(L, KC_PW_DGRAD, (double)dtype_size(dtype) * B * Tp * (Cin + Cout), 2.0 * B * Tp * Cin * Cout);
    GemmDesc d{};
    d.M = Cin; d.N = Tp; d.Kd = Cout;
    d.a_z = 0; d.a_m = 1; d.a_k = Cin;            // A(m=c, k=o) = w[o*Cin + c]
    d.b_z = (long long)Cout * Tp; d.b_k = Tp; d.b_n = 1;
    dim3 grid((Tp + BN - 1) / BN, (Cin + BM - 1) / BM, B);
    SC_DISPATCH(dtype, (launch_k(L, gemm_simt_kernel<T, T, 1>, grid, NT, 0, d, (const T*)w, (const T*)gv, gu, nullptr, nullptr, nullptr)));
    L.count();
}

static int wgrad_splits(int B) { return B; }   // one k-slice per sample

size_t gemm_wgrad_simt_scratch_bytes(int B, int Cin, int Cout) {
    return (size_t)wgrad_splits(B) * Cin * Cout * sizeof(float);
}

void gemm_wgrad_simt(const Launch& L, int dtype, const void* gv, const void* u, float* dw, float* partials,
                     int accumulate, int B, int Cin, int Cout, int Tp, const float* gmax) {
    const int ns = wgrad_splits(B);
    {
    KScope ks_(L, KC_PW_WGRAD, (double)dtype_size(dtype) * B * Tp * (Cin + Cout), 2.0 * B * Tp * Cin * Cout);
    GemmDesc d{};
    d.M = Cout; d.N = Cin; d.Kd = B * Tp;
    d.kt = Tp;
    d.a_m = Tp; d.a_kz = (long long)Cout * Tp;    // A(m=o, k=(b,t)) = gv[b,o,t]
    d.b_n = Tp; d.b_kz = (long long)Cin * Tp;     // B(k=(b,t), n=c) = u[b,c,t]
    d.k_len_per_z = Tp;
    dim3 grid((Cin + BN - 1) / BN, (Cout + BM - 1) / BM, ns);
    SC_DISPATCH(dtype, (launch_k(L, gemm_simt_kernel<T, T, 2>, grid, NT, 0, d, (const T*)gv, (const T*)u, partials, nullptr, nullptr, nullptr)));
    L.count();
    }
    reduce_partials(L, partials, ns, (int64_t)Cin * Cout, dw, accumulate, gmax);
}

}  // namespace sc
