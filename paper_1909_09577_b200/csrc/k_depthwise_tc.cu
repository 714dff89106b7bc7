// Stride-1 depthwise correlation on the tensor cores (forward and input gradient).
//
// For one channel the K-tap correlation over time is a banded Toeplitz product.  Time is cut into
// blocks of 64 frames; output block i only needs input blocks i-1, i, i+1 (K <= 129):
//     U_i[j] = sum_{d in {-1,0,1}} sum_{j'} X_{i+d}[j'] * T_d[j', j],   T_d[j', j] = w[j' + 64 d - j + P].
// The MMA runs with the 64-frame blocks of many samples as its M rows, the 64 positions inside a
// block as N, and the position inside the input block as the contraction:  D = sum_d A_d * T_d with
// fp32 accumulation in tensor memory.  A is staged by the CTA's threads (coalesced 16-byte loads)
// into a no-swizzle layout whose rows sit 16 bytes apart inside each 8-element column chunk, so the
// shifted operand A_d is the same buffer with its start address moved by d rows -- the input is read
// from HBM once and staged once.  Every sample's row run carries one zero block in front and behind
// (the "same" padding and the separation between samples); their output rows are discarded.
// Frames at or beyond a sample's length are zeroed while staging (the padding mask).  After
// tcgen05.ld a thread owns one whole 64-frame output block: 128 contiguous bytes per lane, lanes
// contiguous, so stores coalesce.  The input gradient is the same product with the taps flipped.
#include <type_traits>

#include "common.cuh"
#include "kernels.h"
#include "sm100.cuh"

namespace sc {
namespace {

constexpr int NB = 64;              // frames per block
constexpr int MAXROWS = 256;        // block rows (incl. separators) per CTA: two MMA M-tiles
constexpr int ROWS_ALLOC = 265;     // + one slack row in front, a few behind; 8m+1 so that the eight
                                    // chunk columns start in different 16-byte bank groups
constexpr int kThreads = 256;       // warps 0-3 read back M-tile 0, warps 4-7 M-tile 1

__device__ __forceinline__ uint64_t desc_noswz(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46);
}

template <typename T> struct Fmt16;
template <> struct Fmt16<__half> { static constexpr uint32_t v = 0; };
template <> struct Fmt16<__nv_bfloat16> { static constexpr uint32_t v = 1; };

template <typename T> __device__ __forceinline__ unsigned short bits16(float v);
template <> __device__ __forceinline__ unsigned short bits16<__half>(float v) { return __half_as_ushort(__float2half_rn(v)); }
template <> __device__ __forceinline__ unsigned short bits16<__nv_bfloat16>(float v) { return __bfloat16_as_ushort(__float2bfloat16_rn(v)); }

// TI: type of the input tensor and of both MMA operands; TW: tap type; TO: output (and add1/add2) type.
template <typename TI, typename TW, typename TO, bool FLIP>
__global__ void __launch_bounds__(kThreads)
dw_tc_kernel(const TI* __restrict__ in, const TW* __restrict__ w, TO* __restrict__ out,
             const TO* __restrict__ add1, const TO* __restrict__ add2, const float* __restrict__ gmax,
             const int* __restrict__ len_src, const int* __restrict__ len_dst,
             int B, int C, int Tt, int K, int nb, int* status) {
    pdl_sync();
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
    uint4* A16 = reinterpret_cast<uint4*>(smem);                        // [8 chunks][ROWS_ALLOC] 16-byte units
    uint4* B16 = A16 + 8 * ROWS_ALLOC;                                  // [3 shifts][8 chunks][64 rows]
    // coef[128 + delta] = coefficient that input position (output position + delta) contributes, as
    // 16-bit operand bits; zero outside the taps.  |delta| <= 127, plus slack for the 5-word reads.
    uint32_t* coefw = reinterpret_cast<uint32_t*>(B16 + 3 * 8 * 64);    // 132 words = 264 halfwords
    uint64_t* bar = reinterpret_cast<uint64_t*>(coefw + 132);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar + 1);
    int* lens = reinterpret_cast<int*>(tmem_slot + 2);                  // [nb <= 128] source lengths

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c = blockIdx.x, b0 = blockIdx.y * nb;
    const int nbh = min(nb, B - b0);                 // samples in this CTA
    const int nblk = (Tt + NB - 1) / NB, S = nblk + 2;
    const int rows = nbh * S;
    const int nmt = (rows + 127) / 128;
    const int P = (K - 1) / 2;
    const int vpr = Tt / 8;                          // 16-byte vectors per row (Tt is a multiple of 8)

    if (tid == 0) { ptx::mbar_init(bar, 1); ptx::fence_barrier_init(); }
    if (warp == 0) { ptx::tmem_alloc(tmem_slot, 128); ptx::tmem_relinquish(); }
    for (int i = tid; i < 8 * ROWS_ALLOC; i += kThreads) A16[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < nbh; i += kThreads) lens[i] = len_src[b0 + i];
    for (int i = tid; i < 264; i += kThreads) {
        const int delta = i - 128;
        const int kk = FLIP ? P - delta : delta + P;
        reinterpret_cast<unsigned short*>(coefw)[i] =
            (delta >= -127 && delta <= 127 && kk >= 0 && kk < K) ? bits16<TI>(ldf(w + (size_t)c * K + kk)) : (unsigned short)0;
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // ---- stage the input rows: frame t = 64 i + 8 q + e  ->  A16[q][1 + seg*S + 1 + i] ----
    // All of a thread's loads are issued before the first store so that they overlap (a CTA stages at
    // most nb * nblk * 8 <= 2048 vectors, i.e. 8 per thread).
    {
        const int nvec = nbh * vpr;
        uint4 v[8];
        int dst[8];
        int seg = tid / vpr, vq = tid - seg * vpr;          // vector index -> (sample, vector in row), stepped without divisions
#pragma unroll
        for (int it = 0; it < 8; ++it, vq += kThreads) {
            const int idx = tid + it * kThreads;
            while (vq >= vpr) { vq -= vpr; ++seg; }
            dst[it] = -1;
            if (idx < nvec) {
                const int t = vq * 8;
                const int ls = min(lens[seg], Tt);
                if (t < ls) {
                    v[it] = *reinterpret_cast<const uint4*>(in + ((size_t)(b0 + seg) * C + c) * Tt + t);
                    dst[it] = (vq & 7) * ROWS_ALLOC + 1 + seg * S + 1 + (vq >> 3);
                    if (t + 8 > ls) dst[it] |= (ls - t) << 20;      // the length falls inside this vector
                }
            }
        }
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            if (dst[it] < 0) continue;
            const int keep = dst[it] >> 20;
            if (keep) {
                unsigned short* h = reinterpret_cast<unsigned short*>(&v[it]);
#pragma unroll
                for (int e = 0; e < 8; ++e) if (e >= keep) h[e] = 0;
            }
            A16[dst[it] & 0xFFFFF] = v[it];
        }
    }
    // ---- Toeplitz blocks: B16[d][q][n] holds T_d[j' = 8q..8q+7, j = n] ----
    for (int idx = tid; idx < 3 * 8 * 64; idx += kThreads) {
        const int d = idx / 512, q = (idx >> 6) & 7, n = idx & 63;
        // eight consecutive deltas starting at 8q + 64(d-1) - n: an unaligned 16-byte window of coef
        const int s0 = 8 * q + NB * (d - 1) - n + 128;           // in [1, 247]
        const uint32_t* cw = coefw + (s0 >> 1);
        const uint32_t sh = (s0 & 1) * 16;
        const uint32_t w0 = cw[0], w1 = cw[1], w2 = cw[2], w3 = cw[3], w4 = cw[4];
        B16[idx] = make_uint4(__funnelshift_r(w0, w1, sh), __funnelshift_r(w1, w2, sh), __funnelshift_r(w2, w3, sh),
                              __funnelshift_r(w3, w4, sh));
    }
    ptx::fence_proxy_async();                        // generic-proxy writes -> visible to the tensor core
    __syncthreads();

    if (tid == 0) {
        constexpr uint32_t IDESC = ptx::instr_desc(Fmt16<TI>::v, 0, 0, 128, NB);
        const uint32_t aA = ptx::smem_u32(A16), aB = ptx::smem_u32(B16);
        for (int mt = 0; mt < nmt; ++mt) {
#pragma unroll
            for (int d = 0; d < 3; ++d) {
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint64_t adesc = desc_noswz(aA + ((2 * ks) * ROWS_ALLOC + 1 + mt * 128 + (d - 1)) * 16,
                                                      ROWS_ALLOC * 16, 128);
                    const uint64_t bdesc = desc_noswz(aB + (d * 8 + 2 * ks) * 1024, 1024, 128);
                    ptx::mma_f16(tmem + mt * NB, adesc, bdesc, IDESC, (d > 0 || ks > 0) ? 1u : 0u);
                }
            }
        }
        ptx::mma_commit(bar);
    }
    __syncwarp();

    bool ok = ptx::mbar_wait(bar, 0);
    ok = __all_sync(0xffffffffu, ok);
    ptx::tc_fence_after();
    if (ok) {
        const float inv = gmax ? 1.f / pow2_scale(*gmax) : 1.f;
        const int mt = warp >> 2, wq = warp & 3;          // this warp's M-tile and TMEM lane quarter
        if (mt < nmt) {
            const int Rw = mt * 128 + wq * 32 + lane;
            const int seg = Rw / S, sr = Rw - seg * S;
            const bool live = (Rw < rows) && sr >= 1 && sr <= nblk;
            const int b = b0 + seg;
            const int ld = live ? min(len_dst[b], Tt) : 0;
            const size_t rbase = ((size_t)b * C + c) * Tt;
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                uint32_t r[32];
                ptx::tmem_ld32(tmem + ((uint32_t)(wq * 32) << 16) + mt * NB + 32 * h, r);
                ptx::tmem_ld_wait();
                if (!live) continue;
#pragma unroll
                for (int g8 = 0; g8 < 4; ++g8) {
                    const int t = (sr - 1) * NB + 32 * h + 8 * g8;
                    if (t >= Tt) break;
                    float f[8];
                    if (t >= ld) {                                   // whole vector in padding
#pragma unroll
                        for (int e = 0; e < 8; ++e) f[e] = 0.f;
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(r[8 * g8 + e]);
                        if (gmax) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) f[e] *= inv;
                        }
                        if (add1) { float a[8]; ld8<TO>(add1 + rbase + t, a);
#pragma unroll
                            for (int e = 0; e < 8; ++e) f[e] += a[e]; }
                        if (add2) { float a[8]; ld8<TO>(add2 + rbase + t, a);
#pragma unroll
                            for (int e = 0; e < 8; ++e) f[e] += a[e]; }
                        if (t + 8 > ld) {                            // the length falls inside this vector
#pragma unroll
                            for (int e = 0; e < 8; ++e) if (t + e >= ld) f[e] = 0.f;
                        }
                        if (std::is_same<TO, __half>::value) {       // range guard: one max over the vector, clamp only if hit
                            float m = 0.f;
#pragma unroll
                            for (int e = 0; e < 8; ++e) m = fmaxf(m, fabsf(f[e]));
                            if (m > 65504.f) {
#pragma unroll
                                for (int e = 0; e < 8; ++e) f[e] = fminf(fmaxf(f[e], -65504.f), 65504.f);
                                raise_status(status, kErrRange);
                            }
                        }
                    }
                    st8<TO>(out + rbase + t, f);
                }
            }
        }
    } else if (tid == 0) {
        raise_status(status, kErrTimeout);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem, 128);
}

constexpr size_t kSmemBytes = (size_t)(8 * ROWS_ALLOC + 3 * 8 * 64) * 16 + 132 * 4 + 64 + 128 * 4 + 128;   // A, B, coef, barrier, alignment

template <typename TI, typename TW, typename TO, bool FLIP>
void launch_tc(const Launch& L, const void* in, const void* w, void* out, const void* add1, const void* add2,
               const float* gmax, const int* len_src, const int* len_dst, int B, int C, int Tt, int K) {
    auto kern = dw_tc_kernel<TI, TW, TO, FLIP>;
    set_max_smem_once<dw_tc_kernel<TI, TW, TO, FLIP>>((int)kSmemBytes);
    const int S = (Tt + NB - 1) / NB + 2;
    const int nb = std::max(1, std::min(B, MAXROWS / S));
    dim3 grid(C, (B + nb - 1) / nb);
    launch_k(L, kern, grid, kThreads, kSmemBytes, (const TI*)in, (const TW*)w, (TO*)out, (const TO*)add1, (const TO*)add2,
                                                   gmax, len_src, len_dst, B, C, Tt, K, nb, L.status);
    L.count();
}

}  // namespace

bool dw_tc_supported(int dtype, int Tt, int K, int s) {
    return dtype != F32 && s == 1 && Tt % 8 == 0 && K <= 129 && (Tt + NB - 1) / NB + 2 <= MAXROWS;
}

void dw_tc_fwd(const Launch& L, int dtype, int odt, const void* x, const void* wd, void* u, const int* len_in,
               const int* len_out, int B, int C, int Tt, int K) {
    if (dtype == F16) launch_tc<__half, __half, __half, false>(L, x, wd, u, nullptr, nullptr, nullptr, len_in, len_out, B, C, Tt, K);
    else if (odt == F16) launch_tc<__nv_bfloat16, __nv_bfloat16, __half, false>(L, x, wd, u, nullptr, nullptr, nullptr, len_in, len_out, B, C, Tt, K);
    else launch_tc<__nv_bfloat16, __nv_bfloat16, __nv_bfloat16, false>(L, x, wd, u, nullptr, nullptr, nullptr, len_in, len_out, B, C, Tt, K);
}

void dw_tc_dgrad(const Launch& L, int dtype, int odt, const void* gu, const void* wd, void* dx, const void* add1,
                 const void* add2, const float* gmax, const int* len_in, const int* len_out, int B, int C, int Tt,
                 int K) {
    if (dtype == F16) launch_tc<__half, __half, __half, true>(L, gu, wd, dx, add1, add2, gmax, len_out, len_in, B, C, Tt, K);
    else if (odt == F16) launch_tc<__half, __nv_bfloat16, __nv_bfloat16, true>(L, gu, wd, dx, add1, add2, gmax, len_out, len_in, B, C, Tt, K);
    else launch_tc<__nv_bfloat16, __nv_bfloat16, __nv_bfloat16, true>(L, gu, wd, dx, add1, add2, gmax, len_out, len_in, B, C, Tt, K);
}

}  // namespace sc
