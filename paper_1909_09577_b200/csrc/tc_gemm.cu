// Pointwise (1x1) convolution contractions on the 5th-generation tensor cores.
//
// One kernel template serves the three contractions of the block:
//   forward          v[b]  = wp  * u[b]          D[o,t]  A = wp  (K-major)    B = u[b]  (N-major: time contiguous)
//   input gradient   gu[b] = wp^T * gv[b]        D[c,t]  A = wp^T (M-major)   B = gv[b] (N-major)
//   weight gradient  dwp   = sum_b gv[b] u[b]^T  D[o,c]  A = gv[b] (K-major)  B = u[b]  (K-major), K = (sample, frame)
// Operands are staged by TMA (128-byte swizzle) into a ring of shared-memory stages, one elected
// thread issues tcgen05.mma with the fp32 accumulator in tensor memory (output channels on TMEM lanes,
// time -- or input channels -- on TMEM columns), and four warps read the accumulator back with
// tcgen05.ld.  Because a thread then owns one output channel and a run of consecutive frames, the
// forward epilogue computes the masked batch-norm partial statistics in registers, from the fp32
// accumulators, before the store.  Tiles that lie wholly in a sample's padding are never computed.
// Every mbarrier wait is bounded; on expiry the CTA raises the device status word and leaves.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>

#include "common.cuh"
#include "sm100.cuh"
#include "tc_gemm.h"

namespace sc {
namespace {

enum { MODE_FWD = 0, MODE_DGRAD = 1, MODE_WGRAD = 2 };
constexpr int BK = 64;            // contraction elements per stage (one 128-byte swizzle row)
constexpr int kThreads = 128;

struct TcParams {
    void* out; const float* bias; const int* len_out; float2* stats; int* status;
    int M;          // rows of D in total (C_out for forward / weight gradient, C_in for input gradient)
    int Ncols;      // columns of D in total (T' for forward / input gradient, C_in for weight gradient)
    int Kdim;       // forward: C_in, input gradient: C_out
    int B, Tp;
    int zero_fill;  // skipped (all-padding) tiles must still be written as zeros
    int out_kind;   // forward: type of the result tensor: 0 = the operand type, 1 = float32, 2 = float16
    int nkb_t;      // weight gradient: 64-frame blocks per sample
    int kb_per_split, nkb_total;
};

template <typename T> struct Fmt;
template <> struct Fmt<__half> { static constexpr uint32_t v = 0; };
template <> struct Fmt<__nv_bfloat16> { static constexpr uint32_t v = 1; };

// Coalesced store of a warp's 32 x 32 accumulator block.  After tcgen05.ld lane l holds 32 consecutive
// columns of row l; storing that directly makes every store instruction touch 32 different rows with
// 16 bytes each (half-filled sectors).  The block is transposed through a per-warp shared-memory
// buffer (row pitch 36 floats) so that each instruction writes whole 128-byte (fp32) or 64-byte
// (16-bit) row segments.  `rows_left` / `cols_left` bound the valid part; cols are a multiple of 8.
// A float16 result beyond the half range is clamped to the largest finite value and flagged.
__device__ __forceinline__ void clamp_half32(float (&f)[32], int* status) {
    float m4[4] = {0.f, 0.f, 0.f, 0.f};          // four independent chains: the maximum is latency-bound otherwise
#pragma unroll
    for (int i = 0; i < 32; ++i) m4[i & 3] = fmaxf(m4[i & 3], fabsf(f[i]));
    const float m = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
    if (m > 65504.f) {
#pragma unroll
        for (int i = 0; i < 32; ++i) f[i] = fminf(fmaxf(f[i], -65504.f), 65504.f);
        raise_status(status, kErrRange);
    }
}
constexpr int kStgPitch = 36;
constexpr int kStgFloatsPerWarp = 32 * kStgPitch;
template <typename OT>
__device__ __forceinline__ void store_block_staged(float* stg, const float (&f)[32], OT* out, size_t ld,
                                                   int rows_left, int cols_left, int lane) {
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 8; ++i)
        *reinterpret_cast<float4*>(stg + lane * kStgPitch + 4 * i) = make_float4(f[4 * i], f[4 * i + 1], f[4 * i + 2], f[4 * i + 3]);
    __syncwarp();
    if (sizeof(OT) == 4) {
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int r = it * 4 + (lane >> 3), c = (lane & 7) * 4;
            if (r < rows_left && c < cols_left) {
                const float4 v = *reinterpret_cast<const float4*>(stg + r * kStgPitch + c);
                *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + (size_t)r * ld + c) = v;
            }
        }
    } else {
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int r = it * 8 + (lane >> 2), c = (lane & 3) * 8;
            if (r < rows_left && c < cols_left) {
                const float4 a = *reinterpret_cast<const float4*>(stg + r * kStgPitch + c);
                const float4 b = *reinterpret_cast<const float4*>(stg + r * kStgPitch + c + 4);
                const float g[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
                st8<OT>(out + (size_t)r * ld + c, g);
            }
        }
    }
}

template <typename T, int MODE, int MT, int BN, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, TcParams p) {
    pdl_sync();
    constexpr int A_BYTES = MT * 128 * 128;        // MT sub-tiles of 128 rows x 128 bytes
    constexpr int B_BYTES = BN * 128;
    constexpr int STAGE = A_BYTES + B_BYTES;
    constexpr uint32_t TMEM_COLS = MT * BN;
    static_assert(TMEM_COLS == 64 || TMEM_COLS == 128 || TMEM_COLS == 256 || TMEM_COLS == 512, "tmem columns");
    constexpr uint32_t IDESC = ptx::instr_desc(Fmt<T>::v, MODE == MODE_DGRAD ? 1u : 0u, MODE == MODE_WGRAD ? 0u : 1u, 128, BN);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE);
    uint64_t* empty = full + STAGES;
    uint64_t* accum = empty + STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);
    float* stg_all = reinterpret_cast<float*>(smem + STAGES * STAGE + 256);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * BN;
    const int m0 = blockIdx.y * (128 * MT);
    const int z = blockIdx.z;                      // sample (forward / input gradient) or k-split (weight gradient)

    int len = p.Tp;
    if (MODE != MODE_WGRAD) {
        if (p.len_out) len = min(p.len_out[z], p.Tp);
        if (n0 >= len) {                           // whole tile in padding
            if (p.zero_fill) {
                const int esz = (MODE == MODE_FWD && p.out_kind == 1) ? 4 : (int)sizeof(T);
                const int vec_per_row = BN * esz / 16;
                for (int i = tid; i < 128 * MT * vec_per_row; i += kThreads) {
                    const int r = m0 + i / vec_per_row, cb = (i % vec_per_row) * (16 / esz);
                    if (r < p.M && n0 + cb < p.Ncols) {
                        uint8_t* dst = reinterpret_cast<uint8_t*>(p.out) + (((size_t)z * p.M + r) * p.Ncols + n0 + cb) * esz;
                        *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);   // Ncols is a multiple of 8
                    }
                }
            }
            return;
        }
    }

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
        ptx::mbar_init(accum, 1);
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&mapA);
        ptx::prefetch_tensormap(&mapB);
    }
    if (warp == 0) { ptx::tmem_alloc(tmem_slot, TMEM_COLS); ptx::tmem_relinquish(); }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // k-block range of this CTA
    int kb_begin = 0, kb_end = (p.Kdim + BK - 1) / BK;
    if (MODE == MODE_WGRAD) { kb_begin = z * p.kb_per_split; kb_end = min(p.nkb_total, kb_begin + p.kb_per_split); }
    // weight gradient: blocks that start in a sample's padding are skipped (by every role alike)
    auto kb_valid = [&](int kb, int& b, int& t0) -> bool {
        if (MODE != MODE_WGRAD) return true;
        b = kb / p.nkb_t; t0 = (kb % p.nkb_t) * BK;
        const int l = p.len_out ? min(p.len_out[b], p.Tp) : p.Tp;
        return t0 < l;
    };

    if (warp == 0) {
        if (lane == 0) {                           // ---- TMA producer ----
            int it = 0;
            for (int kb = kb_begin; kb < kb_end; ++kb) {
                int b = 0, t0 = 0;
                if (!kb_valid(kb, b, t0)) continue;
                const int s = it % STAGES, ph = (it / STAGES) & 1;
                if (!ptx::mbar_wait(&empty[s], ph ^ 1)) { raise_status(p.status, kErrTimeout); break; }
                ptx::mbar_arrive_expect_tx(&full[s], STAGE);
                uint8_t* sA = smem + s * STAGE;
                uint8_t* sB = sA + A_BYTES;
                const int k0 = kb * BK;
                if (MODE == MODE_FWD) {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) ptx::tma_load_2d(sA + mt * 16384, &mapA, &full[s], k0, m0 + mt * 128);
#pragma unroll
                    for (int j = 0; j < BN / 64; ++j) ptx::tma_load_3d(sB + j * 8192, &mapB, &full[s], n0 + 64 * j, k0, z);
                } else if (MODE == MODE_DGRAD) {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                        for (int j = 0; j < 2; ++j)
                            ptx::tma_load_2d(sA + mt * 16384 + j * 8192, &mapA, &full[s], m0 + mt * 128 + 64 * j, k0);
#pragma unroll
                    for (int j = 0; j < BN / 64; ++j) ptx::tma_load_3d(sB + j * 8192, &mapB, &full[s], n0 + 64 * j, k0, z);
                } else {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) ptx::tma_load_3d(sA + mt * 16384, &mapA, &full[s], t0, m0 + mt * 128, b);
                    ptx::tma_load_3d(sB, &mapB, &full[s], t0, n0, b);
                }
                ++it;
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {                           // ---- MMA issuer ----
            int it = 0;
            for (int kb = kb_begin; kb < kb_end; ++kb) {
                int b = 0, t0 = 0;
                if (!kb_valid(kb, b, t0)) continue;
                const int s = it % STAGES, ph = (it / STAGES) & 1;
                if (!ptx::mbar_wait(&full[s], ph)) { raise_status(p.status, kErrTimeout); break; }
                ptx::tc_fence_after();
                const uint32_t aA = ptx::smem_u32(smem + s * STAGE), aB = aA + A_BYTES;
#pragma unroll
                for (int ks = 0; ks < BK / 16; ++ks) {
                    const uint64_t bdesc = (MODE == MODE_WGRAD) ? ptx::smem_desc(aB + ks * 32, 16, 1024)
                                                                : ptx::smem_desc(aB + ks * 2048, 8192, 1024);
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        const uint64_t adesc = (MODE == MODE_DGRAD) ? ptx::smem_desc(aA + mt * 16384 + ks * 2048, 8192, 1024)
                                                                    : ptx::smem_desc(aA + mt * 16384 + ks * 32, 16, 1024);
                        ptx::mma_f16(tmem + mt * BN, adesc, bdesc, IDESC, (it > 0 || ks > 0) ? 1u : 0u);
                    }
                }
                ptx::mma_commit(&empty[s]);        // frees the stage once these MMAs have read it
                ++it;
            }
            ptx::mma_commit(accum);                // accumulator complete
        }
        __syncwarp();
    }

    // did this CTA accumulate anything? (weight gradient with every block in padding: no)
    bool any = true;
    if (MODE == MODE_WGRAD) {
        any = false;
        for (int kb = kb_begin; kb < kb_end && !any; ++kb) { int b, t0; any = kb_valid(kb, b, t0); }
    }

    // ---- epilogue: all four warps; warp w owns TMEM lanes 32w..32w+31 ----
    bool ok = ptx::mbar_wait(accum, 0);
    ok = __all_sync(0xffffffffu, ok);
    ptx::tc_fence_after();
    if (ok) {
#pragma unroll 1
        for (int mt = 0; mt < MT; ++mt) {
            const int row = m0 + mt * 128 + warp * 32 + lane;
            float sn = 0.f, smean = 0.f, sm2 = 0.f;
            const float bias = (MODE == MODE_FWD && p.bias && row < p.M) ? p.bias[row] : 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                if (n0 + c0 >= p.Ncols) break;
                float f[32];
                if (any) {
                    uint32_t r[32];
                    ptx::tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + mt * BN + c0, r);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) f[i] = __uint_as_float(r[i]) + bias;
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) f[i] = 0.f;
                }
                if (MODE == MODE_FWD) {
                    const int nv = max(0, min(32, len - (n0 + c0)));
                    if (p.stats && nv > 0) {
                        float s = 0.f;
#pragma unroll
                        for (int i = 0; i < 32; ++i) if (i < nv) s += f[i];
                        const float cm = s / (float)nv;
                        float q = 0.f;
#pragma unroll
                        for (int i = 0; i < 32; ++i) if (i < nv) { const float d = f[i] - cm; q = fmaf(d, d, q); }
                        chan_merge(sn, smean, sm2, (float)nv, cm, q);
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i) if (i >= nv) f[i] = 0.f;
                    if (p.out_kind == 2 || (p.out_kind == 0 && sizeof(T) == 2 && Fmt<T>::v == 0)) clamp_half32(f, p.status);
                }
                {
                    const int row_w = m0 + mt * 128 + warp * 32;             // first row of this warp's block
                    const size_t base = ((size_t)z * p.M + row_w) * p.Ncols + n0 + c0;
                    float* stg = stg_all + warp * kStgFloatsPerWarp;
                    const int rl = p.M - row_w, cl = p.Ncols - (n0 + c0);
                    if ((MODE == MODE_FWD && p.out_kind == 1) || MODE == MODE_WGRAD)
                        store_block_staged<float>(stg, f, reinterpret_cast<float*>(p.out) + base, p.Ncols, rl, cl, lane);
                    else if (MODE == MODE_FWD && p.out_kind == 2)
                        store_block_staged<__half>(stg, f, reinterpret_cast<__half*>(p.out) + base, p.Ncols, rl, cl, lane);
                    else
                        store_block_staged<T>(stg, f, reinterpret_cast<T*>(p.out) + base, p.Ncols, rl, cl, lane);
                }
            }
            if (MODE == MODE_FWD && p.stats && row < p.M)
                p.stats[((size_t)z * gridDim.x + blockIdx.x) * p.M + row] = make_float2(smean * sn, sm2);
        }
    } else if (tid == 0) {
        raise_status(p.status, kErrTimeout);
        // give copies that may still be in flight time to land before the CTA's shared memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem, TMEM_COLS);
}

// ---- persistent, warp-specialised form for the forward and input-gradient contractions -----------
// One CTA per SM loops over output tiles (tile = blockIdx.x + i * gridDim.x).  The first 4*MT warps are
// the epilogue (warp e reads M-sub-tile e/4, TMEM lanes 32(e%4)..+31), the next warp is the TMA
// producer, the last one issues the MMAs.
// The accumulator is double-buffered in tensor memory, so the epilogue of tile i (TMEM -> registers ->
// statistics -> global stores) overlaps the loads and MMAs of tile i+1; the shared-memory ring keeps
// running across tile boundaries.  Barrier set-up and the TMEM allocation are paid once per CTA.

template <typename T, int MODE, int MT, int BN, int STAGES>
__global__ void __launch_bounds__(32 * (4 * MT + 2), 1)
tc_gemm_persistent_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                          TcParams p, int tiles_n, int tiles_m, int tiles_total) {
    pdl_sync();
    static_assert(MODE == MODE_FWD || MODE == MODE_DGRAD, "forward / input gradient only");
    constexpr int A_BYTES = MT * 128 * 128;
    constexpr int B_BYTES = BN * 128;
    constexpr int STAGE = A_BYTES + B_BYTES;
    constexpr uint32_t ACC_COLS = MT * BN;
    constexpr uint32_t TMEM_COLS = 2 * ACC_COLS;
    static_assert(TMEM_COLS == 128 || TMEM_COLS == 256 || TMEM_COLS == 512, "tmem columns");
    constexpr uint32_t IDESC = ptx::instr_desc(Fmt<T>::v, MODE == MODE_DGRAD ? 1u : 0u, 1u, 128, BN);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE);
    uint64_t* empty = full + STAGES;
    uint64_t* acc_full = empty + STAGES;       // [2]
    uint64_t* acc_empty = acc_full + 2;        // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    float* stg_all = reinterpret_cast<float*>(smem + STAGES * STAGE + 256);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
        for (int i = 0; i < 2; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], 128 * MT); }
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&mapA);
        ptx::prefetch_tensormap(&mapB);
    }
    if (warp == 0) { ptx::tmem_alloc(tmem_slot, TMEM_COLS); ptx::tmem_relinquish(); }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int nkb = (p.Kdim + BK - 1) / BK;

    // tile -> (n0, m0, sample); returns false for a tile wholly in the sample's padding
    auto tile_info = [&](int tile, int& n0, int& m0, int& z, int& len) -> bool {
        const int tn = tile % tiles_n, r = tile / tiles_n;
        n0 = tn * BN; m0 = (r % tiles_m) * (128 * MT); z = r / tiles_m;
        len = p.len_out ? min(p.len_out[z], p.Tp) : p.Tp;
        return n0 < len;
    };

    if (warp == 4 * MT) {
        if (lane == 0) {                              // ---- TMA producer ----
            int it = 0;
            bool dead = false;
            for (int tile = blockIdx.x; tile < tiles_total && !dead; tile += gridDim.x) {
                int n0, m0, z, len;
                if (!tile_info(tile, n0, m0, z, len)) continue;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!ptx::mbar_wait(&empty[s], ph ^ 1)) { raise_status(p.status, kErrTimeout); dead = true; break; }
                    ptx::mbar_arrive_expect_tx(&full[s], STAGE);
                    uint8_t* sA = smem + s * STAGE;
                    uint8_t* sB = sA + A_BYTES;
                    const int k0 = kb * BK;
                    if (MODE == MODE_FWD) {
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) ptx::tma_load_2d(sA + mt * 16384, &mapA, &full[s], k0, m0 + mt * 128);
                    } else {
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                            for (int j = 0; j < 2; ++j)
                                ptx::tma_load_2d(sA + mt * 16384 + j * 8192, &mapA, &full[s], m0 + mt * 128 + 64 * j, k0);
                    }
#pragma unroll
                    for (int j = 0; j < BN / 64; ++j) ptx::tma_load_3d(sB + j * 8192, &mapB, &full[s], n0 + 64 * j, k0, z);
                }
            }
        }
        __syncwarp();
    } else if (warp == 4 * MT + 1) {
        if (lane == 0) {                              // ---- MMA issuer ----
            int it = 0, j = 0;
            bool dead = false;
            for (int tile = blockIdx.x; tile < tiles_total && !dead; tile += gridDim.x) {
                int n0, m0, z, len;
                if (!tile_info(tile, n0, m0, z, len)) continue;
                const int buf = j & 1;
                if (!ptx::mbar_wait(&acc_empty[buf], ((j >> 1) & 1) ^ 1)) { raise_status(p.status, kErrTimeout); break; }
                ptx::tc_fence_after();
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!ptx::mbar_wait(&full[s], ph)) { raise_status(p.status, kErrTimeout); dead = true; break; }
                    ptx::tc_fence_after();
                    const uint32_t aA = ptx::smem_u32(smem + s * STAGE), aB = aA + A_BYTES;
#pragma unroll
                    for (int ks = 0; ks < BK / 16; ++ks) {
                        const uint64_t bdesc = ptx::smem_desc(aB + ks * 2048, 8192, 1024);
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
                            const uint64_t adesc = (MODE == MODE_DGRAD) ? ptx::smem_desc(aA + mt * 16384 + ks * 2048, 8192, 1024)
                                                                        : ptx::smem_desc(aA + mt * 16384 + ks * 32, 16, 1024);
                            ptx::mma_f16(tmem + buf * ACC_COLS + mt * BN, adesc, bdesc, IDESC, (kb > 0 || ks > 0) ? 1u : 0u);
                        }
                    }
                    ptx::mma_commit(&empty[s]);
                }
                if (!dead) ptx::mma_commit(&acc_full[buf]);
                ++j;
            }
        }
        __syncwarp();
    } else {                                          // ---- epilogue warps ----
        const int mt = warp >> 2, wq = warp & 3;
        int j = 0;
        for (int tile = blockIdx.x; tile < tiles_total; tile += gridDim.x) {
            int n0, m0, z, len;
            if (!tile_info(tile, n0, m0, z, len)) {
                if (p.zero_fill) {
                    const int esz = (MODE == MODE_FWD && p.out_kind == 1) ? 4 : (int)sizeof(T);
                    const int vec_per_row = BN * esz / 16;
                    for (int i = tid; i < 128 * MT * vec_per_row; i += 128 * MT) {
                        const int r = m0 + i / vec_per_row, cb = (i % vec_per_row) * (16 / esz);
                        if (r < p.M && n0 + cb < p.Ncols) {
                            uint8_t* dst = reinterpret_cast<uint8_t*>(p.out) + (((size_t)z * p.M + r) * p.Ncols + n0 + cb) * esz;
                            *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
                        }
                    }
                }
                continue;
            }
            const int buf = j & 1;
            bool ok = ptx::mbar_wait(&acc_full[buf], (j >> 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { if (lane == 0) raise_status(p.status, kErrTimeout); break; }
            ptx::tc_fence_after();
            {
                const int row = m0 + mt * 128 + wq * 32 + lane;
                float sn = 0.f, smean = 0.f, sm2 = 0.f;
                const float bias = (MODE == MODE_FWD && p.bias && row < p.M) ? p.bias[row] : 0.f;
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    if (n0 + c0 >= p.Ncols) break;
                    float f[32];
                    {
                        uint32_t r[32];
                        ptx::tmem_ld32(tmem + ((uint32_t)(wq * 32) << 16) + buf * ACC_COLS + mt * BN + c0, r);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) f[i] = __uint_as_float(r[i]) + bias;
                    }
                    if (MODE == MODE_FWD) {
                        const int nv = max(0, min(32, len - (n0 + c0)));
                        if (p.stats && nv > 0) {
                            // sums about a pivot taken from the row itself (its first frame in this tile):
                            // one pass, and no cancellation beyond the spread of the data
                            if (c0 == 0) smean = f[0];
                            if (nv == 32) {
#pragma unroll
                                for (int i = 0; i < 32; ++i) { const float d = f[i] - smean; sn += d; sm2 = fmaf(d, d, sm2); }
                            } else {
#pragma unroll
                                for (int i = 0; i < 32; ++i) if (i < nv) { const float d = f[i] - smean; sn += d; sm2 = fmaf(d, d, sm2); }
                            }
                        }
#pragma unroll
                        for (int i = 0; i < 32; ++i) if (i >= nv) f[i] = 0.f;
                        if (p.out_kind == 2 || (p.out_kind == 0 && sizeof(T) == 2 && Fmt<T>::v == 0)) clamp_half32(f, p.status);
                    }
                    {
                        const int row_w = m0 + mt * 128 + wq * 32;
                        const size_t base = ((size_t)z * p.M + row_w) * p.Ncols + n0 + c0;
                        float* stg = stg_all + warp * kStgFloatsPerWarp;
                        const int rl = p.M - row_w, cl = p.Ncols - (n0 + c0);
                        if (MODE == MODE_FWD && p.out_kind == 1)
                            store_block_staged<float>(stg, f, reinterpret_cast<float*>(p.out) + base, p.Ncols, rl, cl, lane);
                        else if (MODE == MODE_FWD && p.out_kind == 2)
                            store_block_staged<__half>(stg, f, reinterpret_cast<__half*>(p.out) + base, p.Ncols, rl, cl, lane);
                        else
                            store_block_staged<T>(stg, f, reinterpret_cast<T*>(p.out) + base, p.Ncols, rl, cl, lane);
                    }
                }
                if (MODE == MODE_FWD && p.stats && row < p.M) {
                    // (sum, M2 about the tile mean) from the pivot-shifted sums; cnt = valid frames of this tile
                    const float cnt = (float)max(1, min(BN, len - n0));
                    p.stats[((size_t)z * tiles_n + (n0 / BN)) * p.M + row] =
                        make_float2(fmaf(smean, cnt, sn), sm2 - sn * sn / cnt);
                }
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(&acc_empty[buf]);        // this thread is done reading the accumulator
            ++j;
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem, TMEM_COLS);
}

// ---- persistent forward / input-gradient contraction over a flattened list of 64-frame blocks -----------
// The N dimension of these contractions is (sample, frame).  Cutting it per sample into fixed tiles wastes
// the tail of every sample (800 frames = 6.25 tiles of 128) and leaves the last wave of tiles mostly idle.
// Here the valid 64-frame blocks of all samples form one list (a sample of len' frames contributes
// ceil(len'/64) blocks; blocks wholly in padding are not in the list), a work unit is (128*MT-row M tile,
// block), and CTA c of G takes the contiguous unit range [c U / G, (c+1) U / G): every CTA gets the same
// number of blocks to within one.  Inside its range a CTA forms tiles of up to four consecutive blocks of one
// M tile; an N-major B operand is a row of independent 64-column sub-tiles in shared memory, so the blocks of
// a tile need not be adjacent in memory nor belong to one sample, and one MMA covers N = 64 * blocks columns.
// Roles as above (epilogue warps, one TMA thread, one MMA thread); the accumulator (MT x 256 columns) fills
// tensor memory, so the epilogue of a tile is not overlapped with the next tile's MMAs, only with its loads.
// Statistics: a thread owns one output channel for the CTA's whole range of an M tile, sums about a pivot taken
// from the row's first valid frame, and writes one (count, sum, M2) partial per (CTA, channel).
constexpr int kFlatMaxNB = 4;          // blocks per tile (N up to 256)
constexpr int kFlatMaxB = 2048;        // samples whose block offsets fit the shared-memory copy
constexpr int kFlatMaxGrid = 320;
constexpr int kOutPitch = 80;          // bytes per row of a warp's 32 x 32 staging block of 16-bit values
constexpr int kOutStageBytes = 32 * kOutPitch;

struct FlatParams {
    void* out; const float* bias; const int* len_out; const int* blk_off; float4* stats; int* status;
    int M;          // rows of D in total (C_out forward, C_in input gradient)
    int Kdim;       // forward: C_in, input gradient: C_out
    int B, Tp, nbT; // nbT = ceil(Tp / 64)
    int tiles_m;
    int zero_fill;  // blocks wholly in padding must be written as zeros
    int out_half;   // the result is float16 although the operands are bfloat16
    int out_f32;    // the result is float32 (one M sub-tile per CTA only: narrow heads such as the class scores)
    int tma_out;    // 16-bit result leaves through TMA stores (third tensor map: 32 frames x 32 rows, 64-byte swizzle)
    int stg_stride; // bytes of staging per epilogue warp (a multiple of 512)
    int stg_nbuf;   // 2: a warp alternates between two 2 KiB staging buffers, so that it need not wait for the store
                    // before last to have read its source
};

// Coalesced store of a warp's 32 x 32 block as 16-bit values: lane l holds 32 consecutive columns of row l;
// the block goes through a per-warp shared-memory buffer (row pitch 80 bytes: conflict-free both ways) so that
// each store instruction writes whole 64-byte row segments.  cols_left is a multiple of 8.
template <typename OT>
__device__ __forceinline__ void store_block16(uint8_t* stg, const float (&f)[32], OT* out, size_t ld, int rows_left,
                                              int cols_left, int lane) {
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float g[8] = {f[8 * i], f[8 * i + 1], f[8 * i + 2], f[8 * i + 3], f[8 * i + 4], f[8 * i + 5], f[8 * i + 6], f[8 * i + 7]};
        st8<OT>(reinterpret_cast<OT*>(stg + lane * kOutPitch + i * 16), g);
    }
    __syncwarp();
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int r = it * 8 + (lane >> 2), c = (lane & 3) * 8;
        if (r < rows_left && c < cols_left) {
            const uint4 v = *reinterpret_cast<const uint4*>(stg + r * kOutPitch + (lane & 3) * 16);
            *reinterpret_cast<uint4*>(out + (size_t)r * ld + c) = v;
        }
    }
}

// Staging for a TMA store of the same block: dense 64-byte rows, the 16-byte chunk c of row r in slot
// c ^ ((r >> 1) & 3) -- the 64-byte swizzle of the tensor map, which also keeps the row-wise writes free of bank
// conflicts.  The warp's registers then cross the load/store path once (to shared memory); the copy engine does the
// rest, clipping rows and frames beyond the tensor.
template <typename OT>
__device__ __forceinline__ void stage_block16_swz(uint8_t* stg, const float (&f)[32], int lane) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float g[8] = {f[8 * i], f[8 * i + 1], f[8 * i + 2], f[8 * i + 3], f[8 * i + 4], f[8 * i + 5], f[8 * i + 6], f[8 * i + 7]};
        st8<OT>(reinterpret_cast<OT*>(stg + lane * 64 + ((i ^ ((lane >> 1) & 3)) << 4)), g);
    }
}

// largest b in [0, B) with off[b] <= j  (off is non-decreasing, off[0] = 0, j < off[B])
__device__ __forceinline__ int flat_find_sample(const int* off, int B, int j) {
    int lo = 0, hi = B - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (off[mid] <= j) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// next tile of a CTA's unit range: M tile m, first block j, nb blocks
template <int NB>
__device__ __forceinline__ bool flat_next_tile(uint32_t& pos, uint32_t end, uint32_t nblk, int& m, int& j, int& nb) {
    if (pos >= end) return false;
    const uint32_t mm = pos / nblk, jj = pos - mm * nblk;
    m = (int)mm; j = (int)jj;
    nb = (int)min((uint32_t)NB, min(end - pos, nblk - jj));
    pos += nb;
    return true;
}

// Shapes: MT M sub-tiles of 128 rows, NB blocks per tile, NBUF accumulator buffers (MT * NB * 64 * NBUF <= 512
// tensor-memory columns).  With NBUF = 2 the epilogue of a tile overlaps the MMAs of the next one.
// OCC = CTAs per SM: with 2, each CTA has a two-stage ring and half of tensor memory, and the two CTAs of an SM
// cover each other's set-up, pipeline fill and epilogue.
// EPI = epilogue warps per 32 accumulator rows: with 2, the two warps that may read the same quarter of tensor
// memory's lanes take one 32-column half of every block each.  A warp's work on a 32 x 32 block is a chain of short
// latencies (tensor-memory load, statistics, staging, fence, store issue); twice the warps overlap twice as many of
// these chains, and the accumulator -- the only one, so the next tile's MMAs wait for it -- is free in half the time.
template <int MT, int NB, int OCC, int EPI = 1> struct FlatCfg {
    static constexpr int A_BYTES = MT * 128 * 128;
    static constexpr int STAGE = A_BYTES + NB * 8192;
    static constexpr int STAGES = OCC == 2 ? 2 : (STAGE <= 49152 ? 4 : 3);
    // per-warp staging: 32 x 32 16-bit values, or (one M sub-tile, one CTA per SM only) 32 x 32 floats for a float32 result
    static constexpr int STG = EPI >= 2 ? 2048 : ((MT == 1 && OCC == 1) ? kStgFloatsPerWarp * 4 : kOutStageBytes);
    static constexpr int MAXB = (OCC == 2 || EPI >= 2) ? 256 : kFlatMaxB;
    static constexpr int smem_bytes(int B) { return STAGES * STAGE + 256 + 4 * MT * EPI * STG + (B + 1) * 4 + 1024; }
};

template <typename T, int MODE, int MT, int NB, int NBUF, int OCC, int EPI>
__global__ void __launch_bounds__(32 * (4 * MT * EPI + 2), OCC)
tc_gemm_flat_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                    const __grid_constant__ CUtensorMap mapO, FlatParams p) {
    pdl_launch_dependents();
    static_assert(MODE == MODE_FWD || MODE == MODE_DGRAD, "forward / input gradient only");
    constexpr int A_BYTES = FlatCfg<MT, NB, OCC, EPI>::A_BYTES;
    constexpr int STAGE = FlatCfg<MT, NB, OCC, EPI>::STAGE;
    constexpr int STAGES = FlatCfg<MT, NB, OCC, EPI>::STAGES;
    constexpr uint32_t ACC_COLS = MT * NB * 64;
    constexpr uint32_t TMEM_COLS = ACC_COLS * NBUF;
    static_assert(TMEM_COLS == 128 || TMEM_COLS == 256 || TMEM_COLS == 512, "tensor-memory columns");
    static_assert(EPI == 1 || ((EPI == 2 || EPI == 4) && OCC == 1), "epilogue warps per lane quarter");
    constexpr int EW = 4 * MT * EPI;               // epilogue warps; then the producer warp and the MMA warp

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* stg_all = smem + STAGES * STAGE;      // per-warp staging: 512-byte aligned (the swizzle of the output map)
    uint64_t* full = reinterpret_cast<uint64_t*>(stg_all + EW * p.stg_stride);
    uint64_t* empty = full + STAGES;
    uint64_t* acc_full = empty + STAGES;       // [NBUF]
    uint64_t* acc_empty = acc_full + NBUF;     // [NBUF]
    // One accumulator: a tile's epilogue first reports the columns of its blocks 0 and 1 drained, then the whole
    // accumulator.  A following tile of at most two blocks (the ragged end of a CTA's range) lives in those columns
    // alone, so its MMAs are issued under the second half of the epilogue.
    uint64_t* acc_half = acc_empty + NBUF;     // [NBUF], used when NBUF == 1
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_half + NBUF);
    int* s_off = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(full) + 256);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
        for (int i = 0; i < NBUF; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], 32 * EW); ptx::mbar_init(&acc_half[i], 32 * EW); }
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&mapA);
        ptx::prefetch_tensormap(&mapB);
        if (p.tma_out) ptx::prefetch_tensormap(&mapO);
    }
    if (warp == 0) { ptx::tmem_alloc(tmem_slot, TMEM_COLS); ptx::tmem_relinquish(); }
    pdl_wait();                                   // everything above overlaps the previous kernel's tail
    for (int i = tid; i <= p.B; i += blockDim.x) s_off[i] = p.blk_off[i];
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int nkb = (p.Kdim + BK - 1) / BK;
    const int nblk = s_off[p.B];
    // 32-bit arithmetic throughout (the launcher bounds the unit count): 64-bit divisions in front of the first copy
    // cost every CTA about a microsecond.  floor(U * c / G) = (U / G) * c + ((U % G) * c) / G, every product below 2^32
    const uint32_t U = (uint32_t)p.tiles_m * (uint32_t)nblk;
    const uint32_t Uq = U / gridDim.x, Ur = U - Uq * gridDim.x;
    const uint32_t u_begin = Uq * blockIdx.x + (Ur * blockIdx.x) / gridDim.x;
    const uint32_t u_end = Uq * (blockIdx.x + 1) + (Ur * (blockIdx.x + 1)) / gridDim.x;

    if (warp == EW) {
        if (lane == 0) {                              // ---- TMA producer ----
            int it = 0, m, j, nb;
            bool dead = false;
            uint32_t pos = u_begin;
            while (!dead && flat_next_tile<NB>(pos, u_end, nblk, m, j, nb)) {
                int bb[NB], tt[NB];
                int b = flat_find_sample(s_off, p.B, j);
#pragma unroll
                for (int i = 0; i < NB; ++i) {
                    if (i < nb) {
                        while (j + i >= s_off[b + 1]) ++b;
                        bb[i] = b; tt[i] = (j + i - s_off[b]) * 64;
                    } else { bb[i] = 0; tt[i] = 0; }
                }
                const int m0 = m * (128 * MT);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!ptx::mbar_wait(&empty[s], ph ^ 1)) { raise_status(p.status, kErrTimeout); dead = true; break; }
                    ptx::mbar_arrive_expect_tx(&full[s], A_BYTES + nb * 8192);
                    uint8_t* sA = smem + s * STAGE;
                    uint8_t* sB = sA + A_BYTES;
                    const int k0 = kb * BK;
                    if (MODE == MODE_FWD) {
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) ptx::tma_load_2d(sA + mt * 16384, &mapA, &full[s], k0, m0 + mt * 128);
                    } else {
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                            for (int h = 0; h < 2; ++h)
                                ptx::tma_load_2d(sA + mt * 16384 + h * 8192, &mapA, &full[s], m0 + mt * 128 + 64 * h, k0);
                    }
#pragma unroll
                    for (int i = 0; i < NB; ++i)
                        if (i < nb) ptx::tma_load_3d(sB + i * 8192, &mapB, &full[s], tt[i], k0, bb[i]);
                }
            }
        }
        __syncwarp();
    } else if (warp == EW + 1) {
        if (lane == 0) {                              // ---- MMA issuer ----
            int it = 0, jt = 0, m, j, nb;
            bool dead = false;
            uint32_t pos = u_begin;
            while (!dead && flat_next_tile<NB>(pos, u_end, nblk, m, j, nb)) {
                const int buf = jt % NBUF;
                const uint32_t par_prev = ((jt / NBUF) & 1) ^ 1;      // completion of the phase the previous user of `buf` arrives on
                bool whole_later = false;
                if (NBUF == 1) {
                    // every phase of both barriers is waited for, in order (a parity wait cannot tell phases two apart):
                    // the half always here, the whole accumulator here or, for a tile of at most two blocks, after its MMAs
                    if (!ptx::mbar_wait(&acc_half[0], par_prev)) { raise_status(p.status, kErrTimeout); break; }
                    whole_later = nb <= 2;
                }
                if (!whole_later && !ptx::mbar_wait(&acc_empty[buf], par_prev)) { raise_status(p.status, kErrTimeout); break; }
                ptx::tc_fence_after();
                const uint32_t idesc = ptx::instr_desc(Fmt<T>::v, MODE == MODE_DGRAD ? 1u : 0u, 1u, 128, 64u * nb);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!ptx::mbar_wait(&full[s], ph)) { raise_status(p.status, kErrTimeout); dead = true; break; }
                    ptx::tc_fence_after();
                    const uint32_t aA = ptx::smem_u32(smem + s * STAGE), aB = aA + A_BYTES;
#pragma unroll
                    for (int ks = 0; ks < BK / 16; ++ks) {
                        const uint64_t bdesc = ptx::smem_desc(aB + ks * 2048, 8192, 1024);
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
                            const uint64_t adesc = (MODE == MODE_DGRAD) ? ptx::smem_desc(aA + mt * 16384 + ks * 2048, 8192, 1024)
                                                                        : ptx::smem_desc(aA + mt * 16384 + ks * 32, 16, 1024);
                            ptx::mma_f16(tmem + buf * ACC_COLS + mt * (NB * 64), adesc, bdesc, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
                        }
                    }
                    ptx::mma_commit(&empty[s]);
                }
                if (!dead) ptx::mma_commit(&acc_full[buf]);
                if (!dead && whole_later && !ptx::mbar_wait(&acc_empty[buf], par_prev)) { raise_status(p.status, kErrTimeout); break; }
                ++jt;
            }
        }
        __syncwarp();
    } else {                                          // ---- epilogue warps ----
        const int mt = (warp >> 2) % MT, wq = warp & 3;
        const int hsel = (warp >> 2) / MT;            // EPI > 1: which of a tile's 32-column chunks this warp takes: chunk
                                                      // 2 * block + half belongs to the warp with hsel == chunk % EPI
        uint8_t* stg = stg_all + warp * p.stg_stride;
        uint32_t nstore = 0;                          // TMA stores issued by this warp
        if (p.zero_fill) {
            // blocks wholly in padding: sample b's blocks [off[b+1]-off[b], nbT); CTAs share them round-robin
            const int inv_per_m = p.B * p.nbT - nblk;
            const uint32_t total_inv = (uint32_t)p.tiles_m * (uint32_t)inv_per_m;
            for (uint32_t q = blockIdx.x; q < total_inv; q += gridDim.x) {
                const int m = (int)(q / (uint32_t)inv_per_m), jj = (int)(q - (uint32_t)m * (uint32_t)inv_per_m);
                int lo = 0, hi = p.B - 1;              // largest b with b * nbT - off[b] <= jj
                while (lo < hi) {
                    const int mid = (lo + hi + 1) >> 1;
                    if (mid * p.nbT - s_off[mid] <= jj) lo = mid; else hi = mid - 1;
                }
                const int b = lo;
                const int t0 = ((s_off[b + 1] - s_off[b]) + (jj - (b * p.nbT - s_off[b]))) * 64;
                for (int i = tid; i < 128 * MT * 8; i += 32 * EW) {
                    const int r = m * (128 * MT) + (i >> 3), cb = (i & 7) * 8;
                    if (r < p.M && t0 + cb < p.Tp) {
                        const size_t e = ((size_t)b * p.M + r) * p.Tp + t0 + cb;
                        if (MT == 1 && OCC == 1 && p.out_f32) {
                            *reinterpret_cast<uint4*>(reinterpret_cast<float*>(p.out) + e) = make_uint4(0, 0, 0, 0);
                            *reinterpret_cast<uint4*>(reinterpret_cast<float*>(p.out) + e + 4) = make_uint4(0, 0, 0, 0);
                        } else {
                            *reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(p.out) + e) = make_uint4(0, 0, 0, 0);
                        }
                    }
                }
            }
        }
        int jt = 0, m, j, nb, cur_m = -1;
        uint32_t pos = u_begin;
        float sn = 0.f, sd = 0.f, sq = 0.f, pivot = 0.f;     // statistics of this thread's channel over the CTA's range of one M tile
        bool dead = false;            // a wait ran out: no further accumulator is touched, but every pair barrier below is still met
        auto flush_stats = [&]() {
            if (MODE != MODE_FWD || !p.stats || cur_m < 0) return;
            float n = sn, sum = fmaf(pivot, sn, sd), m2 = sn > 0.f ? sq - sd * sd / sn : 0.f;
            if (EPI > 1) {
                // the EPI warps of a row hold the statistics of its column chunks: the others hand their triples
                // over through their staging buffers (their stores have read them by then), the first merges them
                // in warp order (Chan) and writes
                const uint32_t bar_id = 1 + mt * 4 + wq;
                if (hsel > 0) {
                    if (p.tma_out && lane == 0) ptx::bulk_wait_read();
                    __syncwarp();
                    reinterpret_cast<float4*>(stg)[lane] = make_float4(n, sum, m2, 0.f);
                }
                asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(32 * EPI) : "memory");
                if (hsel == 0) {
#pragma unroll
                    for (int e = 1; e < EPI; ++e) {
                        const float4 o = reinterpret_cast<const float4*>(stg + e * 4 * MT * p.stg_stride)[lane];
                        if (o.x > 0.f) {
                            if (n > 0.f) {
                                const float nt = n + o.x, dlt = o.y / o.x - sum / n;
                                m2 += o.z + dlt * dlt * (n * o.x / nt);
                                sum += o.y; n = nt;
                            } else { n = o.x; sum = o.y; m2 = o.z; }
                        }
                    }
                }
                asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(32 * EPI) : "memory");
                if (hsel > 0) return;
            }
            const int row = cur_m * (128 * MT) + mt * 128 + wq * 32 + lane;
            if (row < p.M) p.stats[(size_t)blockIdx.x * p.M + row] = make_float4(n, sum, m2, 0.f);
        };
        while (flat_next_tile<NB>(pos, u_end, nblk, m, j, nb)) {
            if (m != cur_m) { flush_stats(); cur_m = m; sn = sd = sq = 0.f; }
            const int buf = jt % NBUF;
            if (dead) { ++jt; continue; }
            if (!ptx::mbar_wait_warp(&acc_full[buf], (jt / NBUF) & 1)) { if (lane == 0) raise_status(p.status, kErrTimeout); dead = true; ++jt; continue; }
            ptx::tc_fence_after();
            const int row_w = m * (128 * MT) + mt * 128 + wq * 32;
            const int row = row_w + lane;
            const float bias = (MODE == MODE_FWD && p.bias && row < p.M) ? p.bias[row] : 0.f;
            int b = flat_find_sample(s_off, p.B, j);
            for (int i = 0; i < nb; ++i) {
                while (j + i >= s_off[b + 1]) ++b;
                const int t0 = (j + i - s_off[b]) * 64;
                const int len = min(p.len_out[b], p.Tp);
#pragma unroll 1
                for (int h = 0; h < 2; ++h) {
                    if (EPI > 1 && ((2 * i + h) % EPI) != hsel) continue;
                    const int c0 = t0 + 32 * h;
                    if (c0 >= p.Tp) break;
                    float f[32];
                    {
                        uint32_t r[32];
                        ptx::tmem_ld32(tmem + ((uint32_t)(wq * 32) << 16) + buf * ACC_COLS + mt * (NB * 64) + i * 64 + h * 32, r);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int q = 0; q < 32; ++q) f[q] = __uint_as_float(r[q]);
                    }
                    if (MODE == MODE_FWD) {
                        if (p.bias) {
#pragma unroll
                            for (int q = 0; q < 32; ++q) f[q] += bias;
                        }
                        const int nv = max(0, min(32, len - c0));
                        if (p.stats && nv > 0) {
                            if (sn == 0.f) pivot = f[0];
                            if (nv == 32) {
                                // d = f - pivot, sum d, sum d^2 in four independent chains (a warp has one other warp to
                                // share its scheduler with, so dependent adds would leave the issue slots empty; the
                                // two-wide fp32 instructions were measured slower per element than the scalar ones)
                                float d4[4] = {0.f, 0.f, 0.f, 0.f}, q4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                                for (int q = 0; q < 32; ++q) {
                                    const float d = f[q] - pivot;
                                    d4[q & 3] += d;
                                    q4[q & 3] = fmaf(d, d, q4[q & 3]);
                                }
                                sd += (d4[0] + d4[1]) + (d4[2] + d4[3]);
                                sq += (q4[0] + q4[1]) + (q4[2] + q4[3]);
                            } else {
#pragma unroll
                                for (int q = 0; q < 32; ++q) if (q < nv) { const float d = f[q] - pivot; sd += d; sq = fmaf(d, d, sq); }
                            }
                            sn += (float)nv;
                        }
                        if (nv < 32) {
#pragma unroll
                            for (int q = 0; q < 32; ++q) if (q >= nv) f[q] = 0.f;
                        }
                        if (!p.out_f32 && (p.out_half || Fmt<T>::v == 0)) clamp_half32(f, p.status);
                    }
                    const size_t base = ((size_t)b * p.M + row_w) * p.Tp + c0;
                    const int rl = p.M - row_w, cl = p.Tp - c0;
                    if (p.tma_out) {
                        // the previous store from this buffer has read its source; write, publish to the copy engine, store
                        uint8_t* sb = stg + ((p.stg_nbuf == 2 && (nstore & 1)) ? 2048 : 0);
                        if (lane == 0) { if (p.stg_nbuf == 2) ptx::bulk_wait_read1(); else ptx::bulk_wait_read(); }
                        __syncwarp();
                        if (MODE == MODE_FWD && p.out_half) stage_block16_swz<__half>(sb, f, lane);
                        else stage_block16_swz<T>(sb, f, lane);
                        ptx::fence_proxy_async();
                        __syncwarp();
                        if (row_w < p.M) {                                  // no box starts outside the tensor
                            if (lane == 0) { ptx::tma_store_3d(&mapO, sb, c0, row_w, b); ptx::bulk_commit(); }
                            ++nstore;
                        }
                    } else if (MT == 1 && OCC == 1 && MODE == MODE_FWD && p.out_f32)
                        store_block_staged<float>(reinterpret_cast<float*>(stg), f, reinterpret_cast<float*>(p.out) + base, p.Tp, rl, cl, lane);
                    else if (MODE == MODE_FWD && p.out_half)
                        store_block16<__half>(stg, f, reinterpret_cast<__half*>(p.out) + base, p.Tp, rl, cl, lane);
                    else
                        store_block16<T>(stg, f, reinterpret_cast<T*>(p.out) + base, p.Tp, rl, cl, lane);
                }
                if (NBUF == 1 && i == 1 && nb > 2) {  // this thread is done with the columns of blocks 0 and 1
                    ptx::tc_fence_before();
                    ptx::mbar_arrive(&acc_half[0]);
                }
            }
            ptx::tc_fence_before();
            if (NBUF == 1 && nb <= 2) ptx::mbar_arrive(&acc_half[0]);
            ptx::mbar_arrive(&acc_empty[buf]);        // this thread is done reading the accumulator
            ++jt;
        }
        flush_stats();
        if (p.tma_out && lane == 0) ptx::bulk_wait_all();     // this thread's stores have completed
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem, TMEM_COLS);
}

// Self-test of the bounded-wait exit: one thread waits on an mbarrier on which nothing ever arrives, with a
// short poll limit; the wait gives up, raises the timeout status and the kernel returns normally.  No copy is
// in flight and no tensor memory is held, so there is nothing to drain.
__global__ void bounded_wait_selftest_kernel(int* status) {
    pdl_sync();
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        ptx::fence_barrier_init();
        bool ok = false;
        for (uint32_t i = 0; i < (1u << 12) && !ok; ++i) ok = ptx::mbar_try_wait(&bar, 0);
        if (!ok) raise_status(status, kErrTimeout);
    }
}

// ---- host side -------------------------------------------------------------------------------
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

// Encoded tensor maps, kept per context: a training loop presents the same tensors every step, and encoding a map
// costs the host a few microseconds, of which a step with several hundred launches has few to spare.  Direct-mapped
// by a hash of everything the encoding depends on; a collision just re-encodes.
struct TcMapCache {
    static constexpr int kSlots = 1024;
    struct Key {
        const void* base; uint64_t dims[3]; uint32_t box[3]; int32_t dtype, rank, swizzle;
        bool operator==(const Key& o) const {
            return base == o.base && dtype == o.dtype && rank == o.rank && swizzle == o.swizzle && dims[0] == o.dims[0] &&
                   dims[1] == o.dims[1] && dims[2] == o.dims[2] && box[0] == o.box[0] && box[1] == o.box[1] && box[2] == o.box[2];
        }
    };
    struct alignas(64) Slot { CUtensorMap map; Key key; bool used; };
    Slot slots[kSlots];
};

void tc_destroy(TcState* st) {
    delete st->map_cache;
    st->map_cache = nullptr;
}

bool tc_make_map(const TcState* st, void* map_out, int dtype, const void* base, int rank, const uint64_t* dims,
                 const uint32_t* box, int swizzle_bytes) {
    CUtensorMap* m = static_cast<CUtensorMap*>(map_out);
    TcMapCache::Slot* slot = nullptr;
    TcMapCache::Key key{};
    if (st->map_cache) {
        key.base = base; key.dtype = dtype; key.rank = rank; key.swizzle = swizzle_bytes;
        for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
        uint64_t h = reinterpret_cast<uintptr_t>(base) * 0x9E3779B97F4A7C15ull;
        for (int i = 0; i < 3; ++i) h = (h ^ key.dims[i] ^ ((uint64_t)key.box[i] << 40)) * 0xC2B2AE3D27D4EB4Full;
        h ^= (uint64_t)(dtype * 131 + rank * 17 + swizzle_bytes);
        slot = &st->map_cache->slots[(h >> 32) % TcMapCache::kSlots];
        if (slot->used && slot->key == key) { *m = slot->map; return true; }
    }
    cuuint64_t gdim[3]; cuuint64_t gstride[2]; cuuint32_t bdim[3]; cuuint32_t estr[3] = {1, 1, 1};
    uint64_t stride = 2;
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i]; bdim[i] = box[i];
        stride *= dims[i];
        if (i + 1 < rank) gstride[i] = stride;
    }
    CUresult r = reinterpret_cast<EncodeFn>(st->encode_fn)(
        m, dtype == F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
        const_cast<void*>(base), gdim, gstride, bdim, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
        swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { fprintf(stderr, "sepconv: cuTensorMapEncodeTiled failed (%d)\n", (int)r); return false; }
    if (slot) { slot->map = *m; slot->key = key; slot->used = true; }
    return true;
}

namespace {
bool make_map(const TcState* st, CUtensorMap* m, int dtype, const void* base, int rank, const uint64_t* dims,
              const uint32_t* box, int swizzle_bytes = 128) {
    return tc_make_map(st, m, dtype, base, rank, dims, box, swizzle_bytes);
}
// map of a [B, M, Tp] 16-bit result for the epilogue's stores: boxes of 32 frames x 32 rows, 64-byte swizzle
bool make_out_map(const TcState* st, CUtensorMap* m, const void* out, int B, int M, int Tp) {
    const uint64_t d[3] = {(uint64_t)Tp, (uint64_t)M, (uint64_t)B};
    const uint32_t b[3] = {32, 32, 1};
    return make_map(st, m, F16, out, 3, d, b, 64);
}

template <typename T, int MODE, int MT, int BN, int STAGES>
void launch(const Launch& L, dim3 grid, const CUtensorMap& a, const CUtensorMap& b, const TcParams& p) {
    constexpr int smem = STAGES * (MT * 16384 + BN * 128) + 1024 + 256 + 4 * kStgFloatsPerWarp * 4;
    auto kern = tc_gemm_kernel<T, MODE, MT, BN, STAGES>;
    set_max_smem_once<tc_gemm_kernel<T, MODE, MT, BN, STAGES>>(smem);
    launch_k(L, kern, grid, kThreads, smem, a, b, p);
    L.count();
}

template <int MODE, int MT, int BN, int STAGES>
void launch_dt(int dtype, const Launch& L, dim3 grid, const CUtensorMap& a, const CUtensorMap& b, const TcParams& p) {
    if (dtype == F16) launch<__half, MODE, MT, BN, STAGES>(L, grid, a, b, p);
    else launch<__nv_bfloat16, MODE, MT, BN, STAGES>(L, grid, a, b, p);
}

template <typename T, int MODE, int MT, int BN, int STAGES>
void launch_persistent(const Launch& L, int sm_count, const CUtensorMap& a, const CUtensorMap& b, const TcParams& p,
                       int tiles_n, int tiles_m, int batch) {
    constexpr int smem = STAGES * (MT * 16384 + BN * 128) + 1024 + 256 + 4 * MT * kStgFloatsPerWarp * 4;
    auto kern = tc_gemm_persistent_kernel<T, MODE, MT, BN, STAGES>;
    set_max_smem_once<tc_gemm_persistent_kernel<T, MODE, MT, BN, STAGES>>(smem);
    const int total = tiles_n * tiles_m * batch;
    launch_k(L, kern, std::min(sm_count, total), 32 * (4 * MT + 2), smem, a, b, p, tiles_n, tiles_m, total);
    L.count();
}
template <int MODE, int MT, int BN, int STAGES>
void launch_persistent_dt(int dtype, const Launch& L, int sm_count, const CUtensorMap& a, const CUtensorMap& b,
                          const TcParams& p, int tiles_n, int tiles_m, int batch) {
    if (dtype == F16) launch_persistent<__half, MODE, MT, BN, STAGES>(L, sm_count, a, b, p, tiles_n, tiles_m, batch);
    else launch_persistent<__nv_bfloat16, MODE, MT, BN, STAGES>(L, sm_count, a, b, p, tiles_n, tiles_m, batch);
}

bool shape_ok(const TcState* st, int dtype, int Cin, int Cout, int Tp) {
    return st && st->ready && (dtype == F16 || dtype == BF16) && Tp % 8 == 0 && Cin % 8 == 0 && Cin >= 8 && Cout >= 1 && Tp >= 8;
}

constexpr int FWD_BN = 128;

struct WgradPlan { int mt, bn, tiles, nsplit, kb_per_split, nkb_total, nkb_t; };
WgradPlan plan_wgrad(int B, int Cin, int Cout, int Tp) {
    WgradPlan w;
    // one 128-row M sub-tile per CTA: twice the output tiles of the two-sub-tile form, so half the k-slices are
    // needed to fill the SMs and the fp32 partials (written once, read once by the reduction) halve
    w.mt = 1;
    w.bn = Cin >= 512 ? 256 : (Cin > 64 ? 128 : 64);
    w.tiles = ((Cout + 128 * w.mt - 1) / (128 * w.mt)) * ((Cin + w.bn - 1) / w.bn);
    w.nkb_t = (Tp + BK - 1) / BK;
    w.nkb_total = B * w.nkb_t;
    int ns = std::max(1, 148 / w.tiles);        // one CTA per SM, one wave
    ns = std::min(ns, w.nkb_total);
    w.kb_per_split = (w.nkb_total + ns - 1) / ns;
    w.nsplit = (w.nkb_total + w.kb_per_split - 1) / w.kb_per_split;
    return w;
}

}  // namespace

void selftest_bounded_wait(const Launch& L) {
    launch_k(L, bounded_wait_selftest_kernel, 1, 32, 0, L.status);
    L.count();
}

int tc_init(TcState* st, int device, int sm_count) {
    (void)device;
    st->sm_count = sm_count;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    st->encode_fn = (e == cudaSuccess && q == cudaDriverEntryPointSuccess) ? fn : nullptr;
    st->ready = st->encode_fn != nullptr;
    st->persistent = true;
    if (st->ready && !st->map_cache) st->map_cache = new TcMapCache();      // value-initialised: every slot unused
    if (!st->ready) { fprintf(stderr, "sepconv: cuTensorMapEncodeTiled not available\n"); return -11; }
    return 0;
}

int tc_max_parts_per_sample(int Tp) { return (Tp + FWD_BN - 1) / FWD_BN; }

bool tc_fwd_supported(const TcState* st, int dtype, int Cin, int Cout, int Tp) { return shape_ok(st, dtype, Cin, Cout, Tp); }
bool tc_dgrad_supported(const TcState* st, int dtype, int Cin, int Cout, int Tp) { return shape_ok(st, dtype, Cin, Cout, Tp); }
bool tc_wgrad_supported(const TcState* st, int dtype, int Cin, int Cout, int Tp) { return shape_ok(st, dtype, Cin, Cout, Tp); }

size_t tc_wgrad_scratch_bytes(const TcState*, int Cin, int Cout) {
    // upper bound over every batch size: at most 148 / tiles splits
    WgradPlan w = plan_wgrad(1 << 20, Cin, Cout, 64);
    return (size_t)w.nsplit * Cin * Cout * sizeof(float);
}

namespace {
template <typename T, int MODE, int MT, int NB, int NBUF, int OCC = 1, int EPI = 1>
void launch_flat(const Launch& L, int sm_count, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& o, const FlatParams& p_in,
                 int* grid_out) {
    using Cfg = FlatCfg<MT, NB, OCC, EPI>;
    FlatParams p = p_in;
    // per-warp staging: the shape's own size, or (TMA stores, one CTA per SM, room left) two 2 KiB buffers
    constexpr int kSmemMax = 232448;
    p.stg_stride = Cfg::STG; p.stg_nbuf = Cfg::STG >= 4096 ? 2 : 1;
    if (p.tma_out && OCC == 1 && Cfg::STG < 4096 && Cfg::smem_bytes(p.B) + 4 * MT * EPI * (4096 - Cfg::STG) <= kSmemMax) {
        p.stg_stride = 4096; p.stg_nbuf = 2;
    }
    const int smem = Cfg::smem_bytes(p.B) + 4 * MT * EPI * (p.stg_stride - Cfg::STG);
    auto kern = tc_gemm_flat_kernel<T, MODE, MT, NB, NBUF, OCC, EPI>;
    set_max_smem_once<tc_gemm_flat_kernel<T, MODE, MT, NB, NBUF, OCC, EPI>>(OCC == 1 ? kSmemMax : Cfg::smem_bytes(Cfg::MAXB));
    const long long units = (long long)p.tiles_m * p.B * p.nbT;
    const int grid = (int)std::max(1ll, std::min<long long>(std::min(sm_count * OCC, kFlatMaxGrid), units));
    launch_k(L, kern, grid, 32 * (4 * MT * EPI + 2), smem, a, b, o, p);
    L.count();
    if (grid_out) *grid_out = grid;
}
// shape 0: 256 x 256 tiles, one accumulator; 1: 256 x 128 tiles, two accumulators; 2: 128 x 256 tiles, two accumulators;
// 3: 128 x 256 tiles, one accumulator, two CTAs per SM; 0 takes sixteen epilogue warps (two per 32 accumulator rows) when
// the batch's block offsets fit beside their staging buffers, 4 is 0 with eight epilogue warps always
template <typename T, int MODE>
void launch_flat_shape(int shape, int mt, const Launch& L, int sm_count, const CUtensorMap& a, const CUtensorMap& b,
                       const CUtensorMap& o, const FlatParams& p, int* grid_out) {
    if (shape == 3 && !p.out_f32 && p.B <= FlatCfg<1, 4, 2>::MAXB) { launch_flat<T, MODE, 1, 4, 1, 2>(L, sm_count, a, b, o, p, grid_out); return; }
    // 5: 128 x 256 tiles, two accumulators, sixteen epilogue warps (four per 32 accumulator rows)
    if (shape == 5 && mt == 1 && p.tma_out && p.B <= FlatCfg<1, 4, 1, 4>::MAXB) { launch_flat<T, MODE, 1, 4, 2, 1, 4>(L, sm_count, a, b, o, p, grid_out); return; }
    if (mt == 1) { launch_flat<T, MODE, 1, 4, 2>(L, sm_count, a, b, o, p, grid_out); return; }
    // sixteen epilogue warps need TMA stores (their 2 KiB staging buffers have the store's layout) and a batch
    // whose block offsets fit beside those buffers
    if (shape == 0 && p.tma_out && p.B <= FlatCfg<2, 4, 1, 2>::MAXB) launch_flat<T, MODE, 2, 4, 1, 1, 2>(L, sm_count, a, b, o, p, grid_out);
    else if (shape == 0 || shape == 4) launch_flat<T, MODE, 2, 4, 1>(L, sm_count, a, b, o, p, grid_out);
    else launch_flat<T, MODE, 2, 2, 2>(L, sm_count, a, b, o, p, grid_out);
}
template <int MODE>
void launch_flat_dt(int dtype, int shape, int mt, const Launch& L, int sm_count, const CUtensorMap& a, const CUtensorMap& b,
                    const CUtensorMap& o, const FlatParams& p, int* grid_out) {
    if (dtype == F16) launch_flat_shape<__half, MODE>(shape, mt, L, sm_count, a, b, o, p, grid_out);
    else launch_flat_shape<__nv_bfloat16, MODE>(shape, mt, L, sm_count, a, b, o, p, grid_out);
}
// the flattened-block kernel counts its work units (M tiles x 64-frame blocks) in 32 bits
inline bool flat_units_fit(int B, int Tp, int rows) { return (long long)((rows + 127) / 128) * B * ((Tp + 63) / 64) < (1ll << 31); }
// M sub-tiles per CTA for a given tile shape and row count
inline int flat_mt(int shape, int rows) { return (shape == 2 || shape == 3 || shape == 5 || rows <= 128) ? 1 : 2; }
}  // namespace

size_t tc_stats_bytes(int B, int Cout, int Tp) {
    return std::max((size_t)B * tc_max_parts_per_sample(Tp) * Cout * sizeof(float2), (size_t)kFlatMaxGrid * Cout * sizeof(float4));
}

void tc_gemm_fwd(const TcState* st, const Launch& L, int dtype, const void* w, const void* u, const float* bias,
                 void* v, int out_dtype, const int* len_out, const int* blk_off, int B, int Cin, int Cout, int Tp,
                 void* partials, StatsLayout* layout) {
    // algorithmic bytes: operand and result once each (16-bit), weights once
    KScope ks_(L, KC_PW_FWD, (double)B * Tp * (2.0 * Cin + dtype_size(out_dtype) * Cout) + 2.0 * Cin * Cout, 2.0 * B * Tp * Cin * Cout);
    CUtensorMap ma, mb;
    const uint64_t da[2] = {(uint64_t)Cin, (uint64_t)Cout};
    const uint32_t ba[2] = {64, 128};
    const uint64_t db[3] = {(uint64_t)Tp, (uint64_t)Cin, (uint64_t)B};
    const uint32_t bb[3] = {64, 64, 1};
    if (layout) *layout = StatsLayout{};
    if (!make_map(st, &ma, dtype, w, 2, da, ba) || !make_map(st, &mb, dtype, u, 3, db, bb)) return;
    int mt = Cout > 128 ? 2 : 1;
    if (st->flat && blk_off && B <= kFlatMaxB && flat_units_fit(B, Tp, Cout) && (out_dtype != F32 || Cout <= 128)) {
        mt = flat_mt(st->flat_shape, Cout);
        FlatParams p{};
        p.out = v; p.bias = bias; p.len_out = len_out; p.blk_off = blk_off; p.stats = (float4*)partials; p.status = L.status;
        p.M = Cout; p.Kdim = Cin; p.B = B; p.Tp = Tp; p.nbT = (Tp + 63) / 64;
        p.tiles_m = (Cout + 128 * mt - 1) / (128 * mt);
        p.zero_fill = partials ? 0 : 1;     // a linear layer's result is the block output: padding must read as zero
        p.out_half = (out_dtype == F16 && dtype != F16) ? 1 : 0;
        p.out_f32 = out_dtype == F32 ? 1 : 0;
        CUtensorMap mo = ma;
        p.tma_out = (!p.out_f32 && make_out_map(st, &mo, v, B, Cout, Tp)) ? 1 : 0;
        int grid = 0;
        launch_flat_dt<MODE_FWD>(dtype, st->flat_shape, mt, L, st->sm_count, ma, mb, mo, p, &grid);
        if (layout && partials) { layout->kind = 2; layout->grid = grid; layout->tiles_m = p.tiles_m; layout->rows_per_tile = 128 * mt; }
        return;
    }
    TcParams p{};
    p.out = v; p.bias = bias; p.len_out = len_out; p.stats = (float2*)partials; p.status = L.status;
    p.M = Cout; p.Ncols = Tp; p.Kdim = Cin; p.B = B; p.Tp = Tp;
    p.zero_fill = partials ? 0 : 1;
    p.out_kind = out_dtype == F32 ? 1 : (out_dtype == dtype ? 0 : 2);
    dim3 grid((Tp + FWD_BN - 1) / FWD_BN, (Cout + 128 * mt - 1) / (128 * mt), B);
    if (mt == 2) launch_persistent_dt<MODE_FWD, 2, FWD_BN, 3>(dtype, L, st->sm_count, ma, mb, p, grid.x, grid.y, B);
    else launch_persistent_dt<MODE_FWD, 1, FWD_BN, 6>(dtype, L, st->sm_count, ma, mb, p, grid.x, grid.y, B);
    if (layout && partials) { layout->kind = 1; layout->parts_per_b = grid.x; layout->tile_w = FWD_BN; }
}

void tc_gemm_dgrad(const TcState* st, const Launch& L, int dtype, const void* w, const void* gv, void* gu, int B,
                   int Cin, int Cout, int Tp, const int* len_out, const int* blk_off) {
    KScope ks_(L, KC_PW_DGRAD, 2.0 * B * Tp * (Cin + Cout) + 2.0 * Cin * Cout, 2.0 * B * Tp * Cin * Cout);
    CUtensorMap ma, mb;
    const uint64_t da[2] = {(uint64_t)Cin, (uint64_t)Cout};
    const uint32_t ba[2] = {64, 64};
    const uint64_t db[3] = {(uint64_t)Tp, (uint64_t)Cout, (uint64_t)B};
    const uint32_t bb[3] = {64, 64, 1};
    if (!make_map(st, &ma, dtype, w, 2, da, ba) || !make_map(st, &mb, dtype, gv, 3, db, bb)) return;
    int mt = Cin > 128 ? 2 : 1;
    if (st->flat && blk_off && B <= kFlatMaxB && flat_units_fit(B, Tp, Cin)) {
        mt = flat_mt(st->flat_shape, Cin);
        FlatParams p{};
        p.out = gu; p.len_out = len_out; p.blk_off = blk_off; p.status = L.status;
        p.M = Cin; p.Kdim = Cout; p.B = B; p.Tp = Tp; p.nbT = (Tp + 63) / 64;
        p.tiles_m = (Cin + 128 * mt - 1) / (128 * mt);
        p.zero_fill = 1;
        CUtensorMap mo = ma;
        p.tma_out = make_out_map(st, &mo, gu, B, Cin, Tp) ? 1 : 0;
        launch_flat_dt<MODE_DGRAD>(dtype, st->flat_shape, mt, L, st->sm_count, ma, mb, mo, p, nullptr);
        return;
    }
    TcParams p{};
    p.out = gu; p.len_out = len_out; p.status = L.status;
    p.M = Cin; p.Ncols = Tp; p.Kdim = Cout; p.B = B; p.Tp = Tp; p.zero_fill = 1;
    dim3 grid((Tp + FWD_BN - 1) / FWD_BN, (Cin + 128 * mt - 1) / (128 * mt), B);
    if (mt == 2) launch_persistent_dt<MODE_DGRAD, 2, FWD_BN, 3>(dtype, L, st->sm_count, ma, mb, p, grid.x, grid.y, B);
    else launch_persistent_dt<MODE_DGRAD, 1, FWD_BN, 6>(dtype, L, st->sm_count, ma, mb, p, grid.x, grid.y, B);
}

void tc_gemm_wgrad(const TcState* st, const Launch& L, int dtype, const void* gv, const void* u, float* dw,
                   float* partials, int accumulate, int B, int Cin, int Cout, int Tp, const int* len_out,
                   const float* gmax) {
    const WgradPlan w = plan_wgrad(B, Cin, Cout, Tp);
    {
        KScope ks_(L, KC_PW_WGRAD, 2.0 * B * Tp * (Cin + Cout), 2.0 * B * Tp * Cin * Cout);
        CUtensorMap ma, mb;
        const uint64_t da[3] = {(uint64_t)Tp, (uint64_t)Cout, (uint64_t)B};
        const uint32_t ba[3] = {64, 128, 1};
        const uint64_t db[3] = {(uint64_t)Tp, (uint64_t)Cin, (uint64_t)B};
        const uint32_t bb[3] = {64, (uint32_t)w.bn, 1};
        if (!make_map(st, &ma, dtype, gv, 3, da, ba) || !make_map(st, &mb, dtype, u, 3, db, bb)) return;
        TcParams p{};
        p.out = partials; p.len_out = len_out; p.status = L.status;
        p.M = Cout; p.Ncols = Cin; p.B = B; p.Tp = Tp;
        p.nkb_t = w.nkb_t; p.kb_per_split = w.kb_per_split; p.nkb_total = w.nkb_total;
        dim3 grid((Cin + w.bn - 1) / w.bn, (Cout + 128 * w.mt - 1) / (128 * w.mt), w.nsplit);
        if (w.mt == 2) {
            if (w.bn == 256) launch_dt<MODE_WGRAD, 2, 256, 3>(dtype, L, grid, ma, mb, p);
            else if (w.bn == 128) launch_dt<MODE_WGRAD, 2, 128, 3>(dtype, L, grid, ma, mb, p);
            else launch_dt<MODE_WGRAD, 2, 64, 4>(dtype, L, grid, ma, mb, p);
        } else {
            if (w.bn == 256) launch_dt<MODE_WGRAD, 1, 256, 3>(dtype, L, grid, ma, mb, p);
            else if (w.bn == 128) launch_dt<MODE_WGRAD, 1, 128, 4>(dtype, L, grid, ma, mb, p);
            else launch_dt<MODE_WGRAD, 1, 64, 4>(dtype, L, grid, ma, mb, p);
        }
    }
    reduce_partials(L, partials, w.nsplit, (int64_t)Cin * Cout, dw, accumulate, gmax);
}

}  // namespace sc
