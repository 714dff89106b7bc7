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
    int out_f32;    // forward: the result tensor is float32
    int nkb_t;      // weight gradient: 64-frame blocks per sample
    int kb_per_split, nkb_total;
};

template <typename T> struct Fmt;
template <> struct Fmt<__half> { static constexpr uint32_t v = 0; };
template <> struct Fmt<__nv_bfloat16> { static constexpr uint32_t v = 1; };

__device__ __forceinline__ void store32(float* dst, const float (&f)[32]) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
        reinterpret_cast<float4*>(dst)[i] = make_float4(f[4 * i], f[4 * i + 1], f[4 * i + 2], f[4 * i + 3]);
}
template <typename T>
__device__ __forceinline__ void store32(T* dst, const float (&f)[32]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float g[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) g[j] = f[8 * i + j];
        st8<T>(dst + 8 * i, g);
    }
}

template <typename OT>
__device__ __forceinline__ void store_row_chunk(OT* row, int col0, int ncols_total, const float (&f)[32]) {
    if (col0 + 32 <= ncols_total) { store32(row + col0, f); return; }
    for (int i = 0; i < 32; ++i) if (col0 + i < ncols_total) stf(row + col0 + i, f[i]);
}

template <typename T, int MODE, int MT, int BN, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, TcParams p) {
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

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * BN;
    const int m0 = blockIdx.y * (128 * MT);
    const int z = blockIdx.z;                      // sample (forward / input gradient) or k-split (weight gradient)

    int len = p.Tp;
    if (MODE != MODE_WGRAD) {
        if (p.len_out) len = min(p.len_out[z], p.Tp);
        if (n0 >= len) {                           // whole tile in padding
            if (p.zero_fill) {
                const int esz = (MODE == MODE_FWD && p.out_f32) ? 4 : (int)sizeof(T);
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
                }
                if (row < p.M) {
                    const size_t rbase = ((size_t)z * p.M + row) * p.Ncols;
                    if (MODE == MODE_FWD && p.out_f32) store_row_chunk(reinterpret_cast<float*>(p.out) + rbase, n0 + c0, p.Ncols, f);
                    else if (MODE == MODE_WGRAD) store_row_chunk(reinterpret_cast<float*>(p.out) + rbase, n0 + c0, p.Ncols, f);
                    else store_row_chunk(reinterpret_cast<T*>(p.out) + rbase, n0 + c0, p.Ncols, f);
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

// ---- host side -------------------------------------------------------------------------------
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool make_map(const TcState* st, CUtensorMap* m, int dtype, const void* base, int rank, const uint64_t* dims,
              const uint32_t* box) {
    cuuint64_t gdim[3]; cuuint64_t gstride[2]; cuuint32_t bdim[3]; cuuint32_t estr[3] = {1, 1, 1};
    uint64_t stride = 2;
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i]; bdim[i] = box[i];
        stride *= dims[i];
        if (i + 1 < rank) gstride[i] = stride;
    }
    CUresult r = reinterpret_cast<EncodeFn>(st->encode_fn)(
        m, dtype == F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
        const_cast<void*>(base), gdim, gstride, bdim, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { fprintf(stderr, "sepconv: cuTensorMapEncodeTiled failed (%d)\n", (int)r); return false; }
    return true;
}

template <typename T, int MODE, int MT, int BN, int STAGES>
void launch(const Launch& L, dim3 grid, const CUtensorMap& a, const CUtensorMap& b, const TcParams& p) {
    constexpr int smem = STAGES * (MT * 16384 + BN * 128) + 1024 + 256;
    static bool configured = false;
    auto kern = tc_gemm_kernel<T, MODE, MT, BN, STAGES>;
    if (!configured) {
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        configured = true;
    }
    kern<<<grid, kThreads, smem, L.stream>>>(a, b, p);
    L.count();
}

template <int MODE, int MT, int BN, int STAGES>
void launch_dt(int dtype, const Launch& L, dim3 grid, const CUtensorMap& a, const CUtensorMap& b, const TcParams& p) {
    if (dtype == F16) launch<__half, MODE, MT, BN, STAGES>(L, grid, a, b, p);
    else launch<__nv_bfloat16, MODE, MT, BN, STAGES>(L, grid, a, b, p);
}

bool shape_ok(const TcState* st, int dtype, int Cin, int Cout, int Tp) {
    return st && st->ready && (dtype == F16 || dtype == BF16) && Tp % 8 == 0 && Cin % 8 == 0 && Cin >= 8 && Cout >= 1 && Tp >= 8;
}

constexpr int FWD_BN = 128;

struct WgradPlan { int mt, bn, tiles, nsplit, kb_per_split, nkb_total, nkb_t; };
WgradPlan plan_wgrad(int B, int Cin, int Cout, int Tp) {
    WgradPlan w;
    w.mt = Cout >= 512 ? 2 : 1;
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

int tc_init(TcState* st, int device, int sm_count) {
    (void)device;
    st->sm_count = sm_count;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    st->encode_fn = (e == cudaSuccess && q == cudaDriverEntryPointSuccess) ? fn : nullptr;
    st->ready = st->encode_fn != nullptr;
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

bool tc_gemm_fwd(const TcState* st, const Launch& L, int dtype, const void* w, const void* u, const float* bias,
                 void* v, int out_dtype, const int* len_out, int B, int Cin, int Cout, int Tp, float2* partials,
                 int* parts_per_b, int* tile_w) {
    KScope ks_(L, KC_PW_FWD, (double)B * Tp * (2.0 * Cin + dtype_size(out_dtype) * Cout), 2.0 * B * Tp * Cin * Cout);
    CUtensorMap ma, mb;
    const uint64_t da[2] = {(uint64_t)Cin, (uint64_t)Cout};
    const uint32_t ba[2] = {64, 128};
    const uint64_t db[3] = {(uint64_t)Tp, (uint64_t)Cin, (uint64_t)B};
    const uint32_t bb[3] = {64, 64, 1};
    if (!make_map(st, &ma, dtype, w, 2, da, ba) || !make_map(st, &mb, dtype, u, 3, db, bb)) return false;
    TcParams p{};
    p.out = v; p.bias = bias; p.len_out = len_out; p.stats = partials; p.status = L.status;
    p.M = Cout; p.Ncols = Tp; p.Kdim = Cin; p.B = B; p.Tp = Tp;
    p.zero_fill = partials ? 0 : 1;     // a linear layer's result is the block output: padding must read as zero
    p.out_f32 = (out_dtype == F32);
    const int mt = Cout > 128 ? 2 : 1;
    dim3 grid((Tp + FWD_BN - 1) / FWD_BN, (Cout + 128 * mt - 1) / (128 * mt), B);
    if (mt == 2) launch_dt<MODE_FWD, 2, FWD_BN, 2>(dtype, L, grid, ma, mb, p);
    else launch_dt<MODE_FWD, 1, FWD_BN, 3>(dtype, L, grid, ma, mb, p);
    *parts_per_b = grid.x; *tile_w = FWD_BN;
    return partials != nullptr;
}

void tc_gemm_dgrad(const TcState* st, const Launch& L, int dtype, const void* w, const void* gv, void* gu, int B,
                   int Cin, int Cout, int Tp, const int* len_out) {
    KScope ks_(L, KC_PW_DGRAD, 2.0 * B * Tp * (Cin + Cout), 2.0 * B * Tp * Cin * Cout);
    CUtensorMap ma, mb;
    const uint64_t da[2] = {(uint64_t)Cin, (uint64_t)Cout};
    const uint32_t ba[2] = {64, 64};
    const uint64_t db[3] = {(uint64_t)Tp, (uint64_t)Cout, (uint64_t)B};
    const uint32_t bb[3] = {64, 64, 1};
    if (!make_map(st, &ma, dtype, w, 2, da, ba) || !make_map(st, &mb, dtype, gv, 3, db, bb)) return;
    TcParams p{};
    p.out = gu; p.len_out = len_out; p.status = L.status;
    p.M = Cin; p.Ncols = Tp; p.Kdim = Cout; p.B = B; p.Tp = Tp; p.zero_fill = 1;
    const int mt = Cin > 128 ? 2 : 1;
    dim3 grid((Tp + FWD_BN - 1) / FWD_BN, (Cin + 128 * mt - 1) / (128 * mt), B);
    if (mt == 2) launch_dt<MODE_DGRAD, 2, FWD_BN, 2>(dtype, L, grid, ma, mb, p);
    else launch_dt<MODE_DGRAD, 1, FWD_BN, 3>(dtype, L, grid, ma, mb, p);
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
