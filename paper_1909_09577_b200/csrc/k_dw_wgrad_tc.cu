// Depthwise tap gradient (stride 1) on the tensor cores.
//
//   dwd[c,k] = sum_{b,t} gu[b,c,t] * x[b,c,t+k-P]
//
// is, for one channel, the correlation of two long signals at K lags.  Time is cut into blocks of 128
// frames.  With  G[(b,tb), j] = gu[b,c,128 tb + j]  and the window  X[(b,tb), j'] = x[b,c,128 tb - Pa + j']
// (Pa = P rounded up to a multiple of 8, so that the window starts on a 16-byte boundary) the product
//   D[j, j'] = sum_{(b,tb)} G[(b,tb), j] * X[(b,tb), j']                (128 x N, N = 127 + K + Pa - P)
// holds every lag on a diagonal:  dwd[c,k] = sum_j D[j, j + k + Pa - P].
// The contraction index is (sample, time block), so both operands are "MN-major" (time contiguous) and
// come straight from HBM through TMA boxes of (64 frames x 1 channel x BB samples), 128-byte swizzle;
// frames outside [0,T) are zero-filled by the TMA unit (the "same" padding).  One elected thread issues
// tcgen05.mma into a 128 x N fp32 accumulator in tensor memory; the accumulator is double-buffered so
// that the diagonal sums of one (channel, split) unit overlap the loads and MMAs of the next.
// Roles: warps 0-3 epilogue (TMEM -> shared memory -> diagonal sums), warps 4-7 operand preparation
// (x is converted to the type of gu and masked by the sample length, in place), warp 8 TMA producer,
// warp 9 MMA issuer.  Every wait is bounded; on expiry the CTA raises the status word and leaves.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>

#include "common.cuh"
#include "kernels.h"
#include "sm100.cuh"
#include "tc_gemm.h"

namespace sc {
namespace {

constexpr int WT_STAGES = 6;
constexpr int WT_STAGE_BYTES = 24576;      // 128 frames of gu + up to 256 frames of x, 32 samples, 16-bit
constexpr int WT_THREADS = 320;
constexpr int WT_ACC_COLS = 256;
constexpr int WT_MAX_CHUNKS = 64;
constexpr int WT_STG_PITCH = 33;

struct WtParams {
    float* partials; const int* len_in; const int* len_out; int* status;
    int B, C, T, K, Pa, delta;
    int BB;              // samples per contraction step (16 or 32)
    int nxb;             // 64-frame boxes in the x window
    int N;               // accumulator columns in use
    int nchunks, ntb;    // contraction steps per channel = nchunks * ntb
    int S, ks_per_split; // splits per channel
    int units;           // C * S
    int prep;            // 1: the x window needs converting and/or masking
    int mask;            // 1: x may be non-zero at or beyond the sample length
};

template <typename T> struct FmtW;
template <> struct FmtW<__half> { static constexpr uint32_t v = 0; };
template <> struct FmtW<__nv_bfloat16> { static constexpr uint32_t v = 1; };

// One 16-byte vector (8 frames) of x: convert TX -> TG, zero frames at or beyond `nvalid`.
template <typename TG, typename TX>
__device__ __forceinline__ uint4 prep8(uint4 raw, int nvalid, bool& over) {
    float f[8];
    if (std::is_same<TX, __half>::value) {
        const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) { float2 q = __half22float2(h[i]); f[2 * i] = q.x; f[2 * i + 1] = q.y; }
    } else {
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) { float2 q = __bfloat1622float2(h[i]); f[2 * i] = q.x; f[2 * i + 1] = q.y; }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) if (i >= nvalid) f[i] = 0.f;
    uint4 r;
    if (std::is_same<TG, __half>::value) {
        if (!std::is_same<TX, __half>::value) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (fabsf(f[i]) > 65504.f) { f[i] = copysignf(65504.f, f[i]); over = true; }
        }
        __half2* h = reinterpret_cast<__half2*>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) h[i] = __floats2half2_rn(f[2 * i], f[2 * i + 1]);
    } else {
        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    }
    return r;
}

__device__ __forceinline__ void bar_sync_named(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

template <typename TG, typename TX>
__global__ void __launch_bounds__(WT_THREADS, 1)
dw_wgrad_tc_kernel(const __grid_constant__ CUtensorMap mapG, const __grid_constant__ CUtensorMap mapX, WtParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + WT_STAGES * WT_STAGE_BYTES);
    uint64_t* conv = full + WT_STAGES;
    uint64_t* empty = conv + WT_STAGES;
    uint64_t* acc_full = empty + WT_STAGES;    // [2]
    uint64_t* acc_empty = acc_full + 2;        // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    int* chunk_len = reinterpret_cast<int*>(tmem_slot + 2);                 // [WT_MAX_CHUNKS]
    float* stg_all = reinterpret_cast<float*>(chunk_len + WT_MAX_CHUNKS);   // [4][32][33]
    float* xw = stg_all + 4 * 32 * WT_STG_PITCH;                            // [4][128]
    int* epi_fail = reinterpret_cast<int*>(xw + 4 * 128);                   // set when an epilogue wait expired

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g_bytes = 2 * p.BB * 128, box_bytes = p.BB * 128;
    const int stage_tx = g_bytes + p.nxb * box_bytes;

    if (tid == 0) {
        for (int s = 0; s < WT_STAGES; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&conv[s], 4); ptx::mbar_init(&empty[s], 1); }
        for (int i = 0; i < 2; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], 128); }
        *epi_fail = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&mapG);
        ptx::prefetch_tensormap(&mapX);
    }
    // longest output length in every sample chunk: time blocks past it hold only zeros of gu
    for (int ch = tid; ch < p.nchunks && ch < WT_MAX_CHUNKS; ch += WT_THREADS) {
        int m = 0;
        for (int b = ch * p.BB; b < min(p.B, (ch + 1) * p.BB); ++b) m = max(m, min(p.len_out[b], p.T));
        chunk_len[ch] = m;
    }
    if (warp == 0) { ptx::tmem_alloc(tmem_slot, 2 * WT_ACC_COLS); ptx::tmem_relinquish(); }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int ks_total = p.nchunks * p.ntb;

    // contraction step ks of a unit that starts at ks0: skipped when its time block lies past every
    // sample of its chunk (never the unit's first step, so that an accumulator is always written)
    auto step_on = [&](int ks, int ks0, int& chunk, int& tb) -> bool {
        chunk = ks / p.ntb; tb = ks - chunk * p.ntb;
        if (ks == ks0 || chunk >= WT_MAX_CHUNKS) return true;
        return tb * 128 < chunk_len[chunk];
    };

    if (warp == 8) {
        if (lane == 0) {                               // ---- TMA producer ----
            int it = 0; bool dead = false;
            for (int unit = blockIdx.x; unit < p.units && !dead; unit += gridDim.x) {
                const int c = unit / p.S, sp = unit - c * p.S;
                const int ks0 = sp * p.ks_per_split, ks1 = min(ks0 + p.ks_per_split, ks_total);
                for (int ks = ks0; ks < ks1; ++ks) {
                    int chunk, tb;
                    if (!step_on(ks, ks0, chunk, tb)) continue;
                    const int s = it % WT_STAGES, ph = (it / WT_STAGES) & 1;
                    if (!ptx::mbar_wait(&empty[s], ph ^ 1)) { raise_status(p.status, kErrTimeout); dead = true; break; }
                    ptx::mbar_arrive_expect_tx(&full[s], stage_tx);
                    uint8_t* sG = smem + s * WT_STAGE_BYTES;
                    uint8_t* sX = sG + g_bytes;
                    const int b0 = chunk * p.BB, t0 = tb * 128;
                    ptx::tma_load_3d(sG, &mapG, &full[s], t0, c, b0);
                    ptx::tma_load_3d(sG + box_bytes, &mapG, &full[s], t0 + 64, c, b0);
                    for (int q = 0; q < p.nxb; ++q)
                        ptx::tma_load_3d(sX + q * box_bytes, &mapX, &full[s], t0 - p.Pa + 64 * q, c, b0);
                    ++it;
                }
            }
        }
        __syncwarp();
    } else if (warp == 9) {
        if (lane == 0) {                               // ---- MMA issuer ----
            const uint32_t idesc = ptx::instr_desc(FmtW<TG>::v, 1u, 1u, 128, (uint32_t)p.N);
            int it = 0, j = 0; bool dead = false;
            for (int unit = blockIdx.x; unit < p.units && !dead; unit += gridDim.x, ++j) {
                const int c = unit / p.S, sp = unit - c * p.S;
                const int ks0 = sp * p.ks_per_split, ks1 = min(ks0 + p.ks_per_split, ks_total);
                const int buf = j & 1;
                if (!ptx::mbar_wait(&acc_empty[buf], ((j >> 1) & 1) ^ 1)) { raise_status(p.status, kErrTimeout); break; }
                ptx::tc_fence_after();
                int done = 0;
                for (int ks = ks0; ks < ks1; ++ks) {
                    int chunk, tb;
                    if (!step_on(ks, ks0, chunk, tb)) continue;
                    const int s = it % WT_STAGES, ph = (it / WT_STAGES) & 1;
                    if (!ptx::mbar_wait(&full[s], ph) || !ptx::mbar_wait(&conv[s], ph)) {
                        raise_status(p.status, kErrTimeout); dead = true; break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t aG = ptx::smem_u32(smem + s * WT_STAGE_BYTES), aX = aG + g_bytes;
                    for (int kk = 0; kk < p.BB / 16; ++kk) {
                        const uint64_t adesc = ptx::smem_desc(aG + kk * 2048, box_bytes, 1024);
                        const uint64_t bdesc = ptx::smem_desc(aX + kk * 2048, box_bytes, 1024);
                        ptx::mma_f16(tmem + buf * WT_ACC_COLS, adesc, bdesc, idesc, (done > 0 || kk > 0) ? 1u : 0u);
                    }
                    ptx::mma_commit(&empty[s]);
                    ++done; ++it;
                }
                if (!dead) ptx::mma_commit(&acc_full[buf]);
            }
        }
        __syncwarp();
    } else if (warp >= 4) {                            // ---- operand preparation (warps 4-7) ----
        const int ctid = tid - 128;
        int it = 0; bool dead = false; bool over = false;
        for (int unit = blockIdx.x; unit < p.units && !dead; unit += gridDim.x) {
            const int c = unit / p.S, sp = unit - c * p.S;
            (void)c;
            const int ks0 = sp * p.ks_per_split, ks1 = min(ks0 + p.ks_per_split, ks_total);
            for (int ks = ks0; ks < ks1; ++ks) {
                int chunk, tb;
                if (!step_on(ks, ks0, chunk, tb)) continue;
                const int s = it % WT_STAGES, ph = (it / WT_STAGES) & 1;
                bool ok = ptx::mbar_wait(&full[s], ph);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { if (lane == 0) raise_status(p.status, kErrTimeout); dead = true; break; }
                if (p.prep) {
                    uint4* sX = reinterpret_cast<uint4*>(smem + s * WT_STAGE_BYTES + g_bytes);
                    const int nvec = p.nxb * p.BB * 8;
                    const int tx0 = tb * 128 - p.Pa, b0 = chunk * p.BB;
                    for (int v = ctid; v < nvec; v += 128) {
                        const int q = v / (p.BB * 8), r = (v >> 3) % p.BB, pv = v & 7;
                        const int lv = pv ^ (r & 7);                       // 128-byte swizzle: logical 16-byte slot
                        const int t = tx0 + 64 * q + 8 * lv;
                        const int b = b0 + r;
                        int nvalid = 8;
                        if (p.mask) nvalid = (b < p.B) ? (min(p.len_in[b], p.T) - t) : 0;
                        sX[v] = prep8<TG, TX>(sX[v], nvalid, over);
                    }
                    ptx::fence_proxy_async();
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&conv[s]);
                ++it;
            }
        }
        if (over) raise_status(p.status, kErrRange);
    } else {                                           // ---- epilogue (warps 0-3) ----
        float* stg = stg_all + warp * 32 * WT_STG_PITCH;
        const int nq = (31 + p.delta + p.K + 31) / 32;     // 32-column chunks this warp reads
        int j = 0;
        for (int unit = blockIdx.x; unit < p.units; unit += gridDim.x, ++j) {
            const int c = unit / p.S, sp = unit - c * p.S;
            const int buf = j & 1;
            bool ok = ptx::mbar_wait(&acc_full[buf], (j >> 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok && lane == 0) { raise_status(p.status, kErrTimeout); atomicExch(epi_fail, 1); }
            bar_sync_named(1, 128);                        // the four warps leave together or not at all
            if (*reinterpret_cast<volatile int*>(epi_fail)) break;
            ptx::tc_fence_after();
            float acc[4] = {0.f, 0.f, 0.f, 0.f};           // taps lane, lane+32, lane+64, lane+96
            for (int q = 0; q < nq; ++q) {
                uint32_t r[32];
                ptx::tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + buf * WT_ACC_COLS + warp * 32 + q * 32, r);
                ptx::tmem_ld_wait();
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 32; ++i) stg[lane * WT_STG_PITCH + i] = __uint_as_float(r[i]);
                __syncwarp();
                // row l of this warp is frame j = 32 warp + l; it holds columns 32 warp + 32 q + i, and the
                // entry of tap k sits at column j + delta + k, i.e. i = l + delta + k - 32 q
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const int k = lane + 32 * m;
                    if (k < p.K) {
                        const int off = p.delta + k - 32 * q;
                        const int lo = max(0, -off), hi = min(31, 31 - off);
                        float a = acc[m];
                        for (int l = lo; l <= hi; ++l) a += stg[l * WT_STG_PITCH + l + off];
                        acc[m] = a;
                    }
                }
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(&acc_empty[buf]);             // accumulator buffer may be overwritten
#pragma unroll
            for (int m = 0; m < 4; ++m) xw[warp * 128 + lane + 32 * m] = acc[m];
            bar_sync_named(1, 128);
            if (tid < p.K) {
                const float v = ((xw[tid] + xw[128 + tid]) + xw[256 + tid]) + xw[384 + tid];
                p.partials[((size_t)sp * p.C + c) * p.K + tid] = v;
            }
            bar_sync_named(1, 128);
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem, 2 * WT_ACC_COLS);
}

constexpr int kWtSmem = WT_STAGES * WT_STAGE_BYTES + 1024 /* alignment */ + 256 /* barriers */ +
                        WT_MAX_CHUNKS * 4 + 4 * 32 * WT_STG_PITCH * 4 + 4 * 128 * 4 + 16;

template <typename TG, typename TX>
void launch_wt(const Launch& L, int grid, const CUtensorMap& mg, const CUtensorMap& mx, const WtParams& p) {
    auto kern = dw_wgrad_tc_kernel<TG, TX>;
    static bool configured = false;
    if (!configured) {
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kWtSmem);
        configured = true;
    }
    kern<<<grid, WT_THREADS, kWtSmem, L.stream>>>(mg, mx, p);
    L.count();
}

}  // namespace

bool dw_wgrad_tc_supported(const TcState* st, int dtype, int B, int T, int K, int s) {
    if (!st || !st->ready || dtype == F32 || s != 1) return false;
    if (B < 16 || T % 8 != 0 || T < 128 || (K & 1) == 0 || K > 127) return false;
    const int P = (K - 1) / 2, Pa = (P + 7) / 8 * 8;
    return 127 + K + (Pa - P) <= 256;
}

void dw_wgrad_tc(const TcState* st, const Launch& L, int dtype, int odt, const void* gu, const void* x, float* dwd,
                 float* partials, int accumulate, const float* gmax, const int* len_in, const int* len_out, int B,
                 int C, int T, int K, int x_clean) {
    WtParams p{};
    {
        KScope ks_(L, KC_DW_WGRAD, (double)B * C * T * (dtype_size(dtype) + dtype_size(odt)), 2.0 * B * C * T * K);
        const int P = (K - 1) / 2;
        p.partials = partials; p.len_in = len_in; p.len_out = len_out; p.status = L.status;
        p.B = B; p.C = C; p.T = T; p.K = K;
        p.Pa = (P + 7) / 8 * 8; p.delta = p.Pa - P;
        p.BB = B >= 32 ? 32 : 16;
        p.N = (127 + K + p.delta + 15) / 16 * 16;
        p.nxb = (p.N + 63) / 64;
        p.nchunks = (B + p.BB - 1) / p.BB;
        p.ntb = (T + 127) / 128;
        const int steps = p.nchunks * p.ntb;
        // splits per channel: the count that minimises (rounds of units over the SMs) x (steps + epilogue)
        const int sms = std::max(1, st->sm_count);
        int bestS = 1; double best = 1e30;
        for (int S = 1; S <= std::min(steps, 8); ++S) {
            const int per = (steps + S - 1) / S;
            if ((S - 1) * per >= steps) continue;            // an empty split
            const int rounds = (C * S + sms - 1) / sms;
            const double cost = (double)rounds * (per + 1.5);
            if (cost < best - 1e-9) { best = cost; bestS = S; }
        }
        p.S = bestS; p.ks_per_split = (steps + bestS - 1) / bestS;
        p.units = C * p.S;
        p.mask = x_clean ? 0 : 1;
        p.prep = (dtype != odt || p.mask) ? 1 : 0;
        CUtensorMap mg, mx;
        const uint64_t dims[3] = {(uint64_t)T, (uint64_t)C, (uint64_t)B};
        const uint32_t box[3] = {64, 1, (uint32_t)p.BB};
        if (!tc_make_map(st, &mg, odt, gu, 3, dims, box) || !tc_make_map(st, &mx, dtype, x, 3, dims, box)) return;
        const int grid = std::min(sms, p.units);
        if (odt == F16 && dtype == F16) launch_wt<__half, __half>(L, grid, mg, mx, p);
        else if (odt == F16) launch_wt<__half, __nv_bfloat16>(L, grid, mg, mx, p);
        else launch_wt<__nv_bfloat16, __nv_bfloat16>(L, grid, mg, mx, p);
    }
    reduce_partials(L, partials, p.S, (int64_t)C * K, dwd, accumulate, gmax);
}

}  // namespace sc
