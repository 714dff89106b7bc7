// Shared device helpers: storage-type conversion, warp reductions, status word.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace sc {

enum DType : int { F32 = 0, F16 = 1, BF16 = 2 };

// Device status codes (mirrors sc_status in the public header).
constexpr int kErrLengths = -8;
constexpr int kErrTimeout = -9;
constexpr int kErrRange = -12;

// Power-of-two scale that brings a tensor with the given absolute maximum into [0.5, 1).
// Multiplying by it (and later by its reciprocal) is exact.
__device__ __forceinline__ float pow2_scale(float amax) {
    if (!(amax > 0.f) || !(amax < 3.0e38f)) return 1.f;
    int e;
    frexpf(amax, &e);
    e = max(-100, min(100, e));
    return ldexpf(1.f, -e);
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

template <typename T> struct IO;
template <> struct IO<float> {
    static __device__ __forceinline__ float ld(const float* p) { return *p; }
    static __device__ __forceinline__ void st(float* p, float v) { *p = v; }
};
template <> struct IO<__half> {
    static __device__ __forceinline__ float ld(const __half* p) { return __half2float(*p); }
    static __device__ __forceinline__ void st(__half* p, float v) { *p = __float2half_rn(v); }
};
template <> struct IO<__nv_bfloat16> {
    static __device__ __forceinline__ float ld(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void st(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

template <typename T> __device__ __forceinline__ float ldf(const T* p) { return IO<T>::ld(p); }
template <typename T> __device__ __forceinline__ void stf(T* p, float v) { IO<T>::st(p, v); }

// Round a float through the storage type (what a store followed by a load would give).
template <typename T> __device__ __forceinline__ float round_io(float v);
template <> __device__ __forceinline__ float round_io<float>(float v) { return v; }
template <> __device__ __forceinline__ float round_io<__half>(float v) { return __half2float(__float2half_rn(v)); }
template <> __device__ __forceinline__ float round_io<__nv_bfloat16>(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

// vhat = (v - mean) * invstd in exactly these two float operations wherever it is needed (forward apply,
// backward reduce and apply): the normalised value is never stored, and the ReLU decision derived from it
// must be the same bit on every path.
__device__ __forceinline__ float bn_norm(float v, float mu, float is) { return __fmul_rn(__fsub_rn(v, mu), is); }

// Two-wide fp32 arithmetic (one instruction for a pair of floats; each lane rounds like the scalar
// instruction, so a value computed here equals the one computed by the scalar helper above).
namespace pk {
__device__ __forceinline__ uint64_t pack(float a, float b) { uint64_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ void unpack(uint64_t r, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r)); }
__device__ __forceinline__ uint64_t add(uint64_t a, uint64_t b) { uint64_t r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ uint64_t mul(uint64_t a, uint64_t b) { uint64_t r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ uint64_t fma(uint64_t a, uint64_t b, uint64_t c) { uint64_t r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r; }
// (v - mu) * is for a pair: nmu = pack(-mu, -mu), is2 = pack(is, is); same bits as bn_norm on each lane
__device__ __forceinline__ uint64_t bn_norm2(uint64_t v, uint64_t nmu, uint64_t is2) { return mul(add(v, nmu), is2); }
}  // namespace pk

// Is the value, once rounded to the storage type T, greater than zero?  Rounding to nearest even sends
// everything up to half the smallest subnormal to zero, so the test is a comparison with that constant:
// the same decision as round_io<T>(a) > 0 without the two conversions.
template <typename T> __device__ __forceinline__ bool rounds_positive(float a);
template <> __device__ __forceinline__ bool rounds_positive<float>(float a) { return a > 0.f; }
template <> __device__ __forceinline__ bool rounds_positive<__half>(float a) { return a > 0x1p-25f; }
template <> __device__ __forceinline__ bool rounds_positive<__nv_bfloat16>(float a) { return a > 0x1p-134f; }

// Rounds the first n of 8 consecutive values to the storage type with error diffusion: the rounding
// residual of one element is added to the next before it is rounded, so the residuals of a vector do
// not add up.  Plain rounding is biased whenever the values sit on a lattice that the storage grid
// resolves only up to a constant offset (a 16-bit gradient times a short binary fraction, minus a
// per-channel constant); a bias of a fraction of a unit in the last place per element, summed over
// every frame of a channel by the weight-gradient contraction, would dominate that gradient's error.
template <typename ST> __device__ __forceinline__ void diffuse8(float (&v)[8], int n) {
    if (sizeof(ST) == 4) return;
    float r = 0.f;
    if (n >= 8) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float t = v[i] + r;
            const float q = round_io<ST>(t);
            r = t - q;
            v[i] = q;
        }
        return;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i < n) {
            const float t = v[i] + r;
            const float q = round_io<ST>(t);
            r = t - q;
            v[i] = q;
        }
    }
}

// 8 consecutive elements <-> 8 floats.  Pointers must be aligned to 8 elements.
template <typename T> __device__ __forceinline__ void ld8(const T* p, float (&f)[8]);
template <> __device__ __forceinline__ void ld8<float>(const float* p, float (&f)[8]) {
    float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}
template <> __device__ __forceinline__ void ld8<__half>(const __half* p, float (&f)[8]) {
    uint4 r = *reinterpret_cast<const uint4*>(p);
    const __half2* h = reinterpret_cast<const __half2*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 q = __half22float2(h[i]); f[2 * i] = q.x; f[2 * i + 1] = q.y; }
}
template <> __device__ __forceinline__ void ld8<__nv_bfloat16>(const __nv_bfloat16* p, float (&f)[8]) {
    uint4 r = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 q = __bfloat1622float2(h[i]); f[2 * i] = q.x; f[2 * i + 1] = q.y; }
}
// the same conversion from a 16-byte vector that is already in registers (16-bit types)
template <typename T> __device__ __forceinline__ void cvt8(const uint4& r, float (&f)[8]);
template <> __device__ __forceinline__ void cvt8<__half>(const uint4& r, float (&f)[8]) {
    const __half2* h = reinterpret_cast<const __half2*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 q = __half22float2(h[i]); f[2 * i] = q.x; f[2 * i + 1] = q.y; }
}
template <> __device__ __forceinline__ void cvt8<__nv_bfloat16>(const uint4& r, float (&f)[8]) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 q = __bfloat1622float2(h[i]); f[2 * i] = q.x; f[2 * i + 1] = q.y; }
}
template <typename T> __device__ __forceinline__ void st8(T* p, const float (&f)[8]);
template <> __device__ __forceinline__ void st8<float>(float* p, const float (&f)[8]) {
    *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
    *reinterpret_cast<float4*>(p + 4) = make_float4(f[4], f[5], f[6], f[7]);
}
template <> __device__ __forceinline__ void st8<__half>(__half* p, const float (&f)[8]) {
    uint4 r;
    __half2* h = reinterpret_cast<__half2*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2half2_rn(f[2 * i], f[2 * i + 1]);
    *reinterpret_cast<uint4*>(p) = r;
}
template <> __device__ __forceinline__ void st8<__nv_bfloat16>(__nv_bfloat16* p, const float (&f)[8]) {
    uint4 r;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    *reinterpret_cast<uint4*>(p) = r;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Chan/Welford merge of (n_a, mean_a, M2_a) with (n_b, mean_b, M2_b).
__device__ __forceinline__ void chan_merge(float& n, float& mean, float& m2, float nb, float meanb, float m2b) {
    if (nb == 0.f) return;
    float nt = n + nb;
    float d = meanb - mean;
    mean += d * (nb / nt);
    m2 += m2b + d * d * (n * nb / nt);
    n = nt;
}

// Programmatic dependent launch.  Every kernel of the library is launched so that it may start while the
// kernel before it on the stream is still draining; it therefore (1) tells the runtime right away that its own
// dependents may be launched -- the trigger fires once every CTA has said so, i.e. when the last wave is on
// the SMs -- and (2) waits for the kernels before it to complete, with their writes visible, before it reads
// or writes global memory.  Work placed before pdl_wait() (barrier set-up, tensor-memory allocation,
// descriptor prefetch) overlaps the previous kernel's tail.  Both are no-ops in a kernel launched without
// the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_sync() { pdl_launch_dependents(); pdl_wait(); }

__device__ __forceinline__ void raise_status(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}

}  // namespace sc
