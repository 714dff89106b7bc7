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
// Roles: warps 0-3 epilogue (TMEM -> shared memory -> diagonal sums), warps 4-11 operand preparation
// (x is converted to the type of gu and masked by the sample length, in place; two groups of four warps
// take alternate steps), warp 12 TMA producer (one box per lane: issuing a TMA copy costs a thread
// about a hundred cycles, so the boxes of a step are issued side by side), warp 13 MMA issuer.  Every wait is bounded; on expiry the CTA raises the status word and leaves.
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

constexpr int WT_STAGES = 4;               // at most; 3 when the x window needs four 64-frame boxes
constexpr int WT_RING_BYTES = 163840;      // stage = two time blocks x (128 frames of gu + 192 or 256 frames of x) x 32 samples
constexpr int WT_THREADS = 448;
constexpr int WT_ACC_COLS = 256;
constexpr int WT_MAX_CHUNKS = 64;
constexpr int WT_STG_PITCH = 36;                     // floats per staging row
constexpr int WT_STG_FLOATS = 63 * WT_STG_PITCH;     // per epilogue warp
constexpr int WT_XW = 128;

struct WtParams {
    float* partials; const int* len_in; const int* len_out; int* status;
    float* dwd; const float* gmax; int accumulate;   // used when a channel is not split: the result is written directly
    int B, C, T, K, Pa, delta;
    int BB;              // samples per contraction step (16 or 32)
    int nxb;             // 64-frame boxes in the x window
    int N;               // accumulator columns in use
    int nchunks, ntb;    // contraction steps per channel = nchunks * ntb; a step is a PAIR of 128-frame time blocks
    int nstages, stage_bytes;
    int S, ks_per_split; // splits per channel
    int units;           // C * S
    int prep;            // 1: the x window needs converting and/or masking
    int mask;            // 1: x may be non-zero at or beyond the sample length
};

template <typename T> struct FmtW;
template <> struct FmtW<__half> { static constexpr uint32_t v = 0; };
template <> struct FmtW<__nv_bfloat16> { static constexpr uint32_t v = 1; };

// One 16-byte vector (8 frames) of x: convert TX -> TG and zero the frames at or beyond `nvalid`.
// amax collects the largest magnitude seen (a bf16 value of 2^16 or more has no half counterpart).
template <typename TG, typename TX>
__device__ __forceinline__ uint4 prep8(uint4 raw, int nvalid, float& amax) {
    uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    if (!std::is_same<TG, TX>::value) {
        // bf16 -> half through fp32: a bf16 is the upper half of the float with the same value
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
            amax = fmaxf(amax, fmaxf(fabsf(lo), fabsf(hi)));
            const __half2 h = __floats2half2_rn(lo, hi);
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
    }
    if (nvalid < 8) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (2 * i >= nvalid) w[i] = 0u;
            else if (2 * i + 1 >= nvalid) w[i] &= 0x0000FFFFu;
        }
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ void bar_sync_named(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Walks the contraction steps of one unit: (chunk, tb) advance without divisions; a step is skipped when
// its time block lies past every sample of its chunk (never the unit's first step, so that an
// accumulator is always written).  Every role walks the same sequence.
struct StepWalk {
    int ks, ks0, ks1, chunk, tb, ntb, cl;
    const int* chunk_len;
    __device__ __forceinline__ void begin(int sp, int ks_per_split, int ks_total, int ntb_, const int* cl_) {
        ks0 = sp * ks_per_split; ks1 = min(ks0 + ks_per_split, ks_total); ks = ks0; ntb = ntb_; chunk_len = cl_;
        chunk = ks0 / ntb; tb = ks0 - chunk * ntb;
        cl = chunk < WT_MAX_CHUNKS ? chunk_len[chunk] : (1 << 30);
    }
    __device__ __forceinline__ bool more() const { return ks < ks1; }
    __device__ __forceinline__ bool on() const { return ks == ks0 || tb * 256 < cl; }
    __device__ __forceinline__ void next() {
        ++ks;
        if (++tb == ntb) { tb = 0; ++chunk; cl = chunk < WT_MAX_CHUNKS ? chunk_len[chunk] : (1 << 30); }
    }
};
// ring position: stage index and phase parity, advanced without a modulo
struct Ring {
    int s = 0, ph = 0, n;
    __device__ __forceinline__ explicit Ring(int nstages) : n(nstages) {}
    __device__ __forceinline__ void advance() { if (++s == n) { s = 0; ph ^= 1; } }
};

template <typename TG, typename TX>
__global__ void __launch_bounds__(WT_THREADS, 1)
dw_wgrad_tc_kernel(const __grid_constant__ CUtensorMap mapG, const __grid_constant__ CUtensorMap mapX, WtParams p) {
    pdl_launch_dependents();
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + WT_RING_BYTES);
    uint64_t* conv = full + WT_STAGES;
    uint64_t* empty = conv + WT_STAGES;
    uint64_t* acc_full = empty + WT_STAGES;    // [2]
    uint64_t* acc_empty = acc_full + 2;        // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    int* chunk_len = reinterpret_cast<int*>(tmem_slot + 2);                 // [WT_MAX_CHUNKS]
    // staging rows are read with 16-byte loads: keep the block 16-byte aligned (barriers etc. take < 512 bytes)
    float* stg_all = reinterpret_cast<float*>(smem + WT_RING_BYTES + 512);   // [4][63][36]
    float* xw = stg_all + 4 * WT_STG_FLOATS;                                // [4][160]
    int* epi_fail = reinterpret_cast<int*>(xw + 4 * WT_XW);                 // set when an epilogue wait expired

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g_bytes = 2 * p.BB * 128, box_bytes = p.BB * 128;
    const int x_bytes = p.nxb * box_bytes;
    const int stage_tx = 2 * (g_bytes + x_bytes);

    if (tid == 0) {
        for (int s = 0; s < WT_STAGES; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&conv[s], 4); ptx::mbar_init(&empty[s], 1); }
        for (int i = 0; i < 2; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], 128); }
        *epi_fail = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&mapG);
        ptx::prefetch_tensormap(&mapX);
    }
    pdl_wait();                                        // the barrier set-up above overlaps the previous kernel's tail
    // longest output length in every sample chunk: time blocks past it hold only zeros of gu
    for (int ch = tid; ch < p.nchunks && ch < WT_MAX_CHUNKS; ch += WT_THREADS) {
        int m = 0;
        for (int b = ch * p.BB; b < min(p.B, (ch + 1) * p.BB); ++b) m = max(m, min(p.len_out[b], p.T));
        chunk_len[ch] = m;
    }
    // the skewed staging is written on the same parallelogram every time; the rest stays zero
    for (int i = tid; i < 4 * WT_STG_FLOATS; i += WT_THREADS) stg_all[i] = 0.f;
    if (warp == 0) { ptx::tmem_alloc(tmem_slot, 2 * WT_ACC_COLS); ptx::tmem_relinquish(); }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int ks_total = p.nchunks * p.ntb;

    if (warp == 12) {                                  // ---- TMA producer: one box per lane ----
        Ring rg(p.nstages); bool dead = false;
        // lane -> (time block of the pair, box): boxes 0-1 are gu, boxes 2.. the x window
        const int per = 2 + p.nxb;
        const int hb = lane / per, bx = lane - hb * per;
        const bool is_g = bx < 2;
        const int q = bx - 2;
        const bool active = lane < 2 * per;
        const void* map = is_g ? (const void*)&mapG : (const void*)&mapX;
        const int dst_off = is_g ? hb * g_bytes + bx * box_bytes : 2 * g_bytes + hb * x_bytes + q * box_bytes;
        const int t_off = 128 * hb + (is_g ? 64 * bx : 64 * q - p.Pa);
        for (int unit = blockIdx.x; unit < p.units && !dead; unit += gridDim.x) {
            const int c = unit / p.S, sp = unit - c * p.S;
            StepWalk w; w.begin(sp, p.ks_per_split, ks_total, p.ntb, chunk_len);
            for (; w.more(); w.next()) {
                if (!w.on()) continue;
                bool ok = true;
                if (lane == 0) {
                    ok = ptx::mbar_wait(&empty[rg.s], rg.ph ^ 1);
                    if (ok) ptx::mbar_arrive_expect_tx(&full[rg.s], stage_tx);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { if (lane == 0) raise_status(p.status, kErrTimeout); dead = true; break; }
                if (active)
                    ptx::tma_load_3d(smem + rg.s * p.stage_bytes + dst_off, map, &full[rg.s], w.tb * 256 + t_off, c,
                                     w.chunk * p.BB);
                rg.advance();
            }
        }
    } else if (warp == 13) {
        if (lane == 0) {                               // ---- MMA issuer ----
            const uint32_t idesc = ptx::instr_desc(FmtW<TG>::v, 1u, 1u, 128, (uint32_t)p.N);
            // descriptors differ from step to step only in the start-address field
            const uint64_t dbase = ptx::smem_desc(0, box_bytes, 1024);
            const uint32_t smem_a = ptx::smem_u32(smem);
            const int nkk = p.BB / 16;
            Ring rg(p.nstages); int j = 0; bool dead = false;
            for (int unit = blockIdx.x; unit < p.units && !dead; unit += gridDim.x, ++j) {
                const int c = unit / p.S, sp = unit - c * p.S;
                (void)c;
                const int buf = j & 1;
                if (!ptx::mbar_wait(&acc_empty[buf], ((j >> 1) & 1) ^ 1)) { raise_status(p.status, kErrTimeout); break; }
                ptx::tc_fence_after();
                uint32_t accum = 0;
                StepWalk w; w.begin(sp, p.ks_per_split, ks_total, p.ntb, chunk_len);
                for (; w.more(); w.next()) {
                    if (!w.on()) continue;
                    // conv[s] completes only after the preparation warps have seen full[s] complete
                    if (!ptx::mbar_wait(&conv[rg.s], rg.ph)) {
                        raise_status(p.status, kErrTimeout); dead = true; break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t aG = smem_a + rg.s * p.stage_bytes;
#pragma unroll 1
                    for (int hb = 0; hb < 2; ++hb) {
                        uint64_t dG = dbase | (uint64_t)(((aG + hb * g_bytes) & 0x3FFFFu) >> 4);
                        uint64_t dX = dbase | (uint64_t)(((aG + 2 * g_bytes + hb * x_bytes) & 0x3FFFFu) >> 4);
                        for (int kk = 0; kk < nkk; ++kk) {
                            ptx::mma_f16(tmem + buf * WT_ACC_COLS, dG, dX, idesc, accum);
                            accum = 1u; dG += 2048 >> 4; dX += 2048 >> 4;
                        }
                    }
                    ptx::mma_commit(&empty[rg.s]);
                    rg.advance();
                }
                if (!dead) ptx::mma_commit(&acc_full[buf]);
            }
        }
        __syncwarp();
    } else if (warp >= 4) {                            // ---- operand preparation: two groups of four warps ----
        // group 0 (warps 4-7) takes the even ring steps, group 1 (warps 8-11) the odd ones
        const int grp = (warp - 4) >> 2;
        const int ctid = tid - 128 - 128 * grp;
        // Vector v = ctid + 128 i of the window sits in box v / (8 BB), sample row (v / 8) % BB, 16-byte slot
        // v % 8.  The slot and the row's low bits do not depend on i, so the frame offset inside a box is
        // a per-thread constant (128-byte swizzle: logical slot = physical slot ^ (row % 8)).
        const int lb = (p.BB == 32) ? 5 : 4;
        const int nvec_t = (p.nxb * p.BB) >> 4;                 // vectors per thread and step (<= 8)
        const int r0 = ctid >> 3;
        const int toff = 8 * ((ctid & 7) ^ (r0 & 7));
        Ring rg(p.nstages); int it = 0; bool dead = false; float amax = 0.f;
        for (int unit = blockIdx.x; unit < p.units && !dead; unit += gridDim.x) {
            const int c = unit / p.S, sp = unit - c * p.S;
            (void)c;
            StepWalk w; w.begin(sp, p.ks_per_split, ks_total, p.ntb, chunk_len);
            for (; w.more(); w.next()) {
                if (!w.on()) continue;
                if ((it & 1) == grp) {
                    const bool ok = ptx::mbar_wait_warp(&full[rg.s], rg.ph);
                    if (!ok) { if (lane == 0) raise_status(p.status, kErrTimeout); dead = true; break; }
                    if (p.prep) {
#pragma unroll 1
                        for (int hb = 0; hb < 2; ++hb) {
                            uint4* sX = reinterpret_cast<uint4*>(smem + rg.s * p.stage_bytes + 2 * g_bytes + hb * x_bytes);
                            const int tx0 = w.tb * 256 + 128 * hb - p.Pa + toff, b0 = w.chunk * p.BB;
                            // frames left before the sample's end, for this thread's (at most two) rows
                            int left0 = 1 << 30, left1 = 1 << 30;
                            if (p.mask) {
                                const int ba = b0 + r0, bb = b0 + r0 + 16;
                                left0 = (ba < p.B ? min(p.len_in[ba], p.T) : 0) - tx0;
                                left1 = (bb < p.B ? min(p.len_in[bb], p.T) : 0) - tx0;
                            }
                            uint4 raw[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) if (i < nvec_t) raw[i] = sX[ctid + 128 * i];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                if (i < nvec_t) {
                                    const int v = ctid + 128 * i;
                                    const int left = (((v >> 3) & 16) & (p.BB - 1)) ? left1 : left0;
                                    sX[v] = prep8<TG, TX>(raw[i], left - 64 * (v >> (3 + lb)), amax);
                                }
                            }
                        }
                        ptx::fence_proxy_async();
                    }
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&conv[rg.s]);
                }
                rg.advance(); ++it;
            }
        }
        if (amax >= 65536.f) raise_status(p.status, kErrRange);
    } else {                                           // ---- epilogue (warps 0-3) ----
        // Warp e owns accumulator rows j = 32 e + l (lane l) and reads them in 32-column chunks
        // (columns 32 e + 32 q + i).  The entry of tap k in row j is column j + delta + k, so inside a chunk
        // it lies on the diagonal d = i - l + 31 = delta + k - 32 q + 31.  Each lane scatters its 32 values
        // to staging row d (pitch 36 floats: conflict-free both ways), and a lane then sums whole staging
        // rows d = lane and d = lane + 32 with 16-byte loads: all of them belong to taps
        // k = lane + 1 - delta + 32 n with n = q - 1 and n = q.
        float* stg = stg_all + warp * WT_STG_FLOATS;
        const int nq = (62 + p.delta + p.K) / 32;          // 32-column chunks this warp reads (<= 6)
        int j = 0;
        for (int unit = blockIdx.x; unit < p.units; unit += gridDim.x, ++j) {
            const int c = unit / p.S, sp = unit - c * p.S;
            const int buf = j & 1;
            const bool ok = ptx::mbar_wait_warp(&acc_full[buf], (j >> 1) & 1, 64);
            if (!ok && lane == 0) { raise_status(p.status, kErrTimeout); atomicExch(epi_fail, 1); }
            bar_sync_named(1, 128);                        // the four warps leave together or not at all
            if (*reinterpret_cast<volatile int*>(epi_fail)) break;
            ptx::tc_fence_after();
            float acc[7] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};   // acc[n + 1]: tap lane + 1 - delta + 32 n
#pragma unroll
            for (int q = 0; q < 6; ++q) {
                if (q < nq) {
                    uint32_t r[32];
                    ptx::tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + buf * WT_ACC_COLS + warp * 32 + q * 32, r);
                    ptx::tmem_ld_wait();
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 32; ++i) stg[(i + 31 - lane) * WT_STG_PITCH + lane] = __uint_as_float(r[i]);
                    __syncwarp();
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int d = lane + 32 * h;
                        if (d < 63) {
                            const float4* row = reinterpret_cast<const float4*>(stg + d * WT_STG_PITCH);
                            float s0 = 0.f, s1 = 0.f;
#pragma unroll
                            for (int v = 0; v < 8; v += 2) {
                                const float4 x0 = row[v], x1 = row[v + 1];
                                s0 += (x0.x + x0.y) + (x0.z + x0.w);
                                s1 += (x1.x + x1.y) + (x1.z + x1.w);
                            }
                            acc[q + h] += s0 + s1;
                        }
                    }
                }
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(&acc_empty[buf]);             // accumulator buffer may be overwritten
#pragma unroll
            for (int n = 0; n < 7; ++n) {
                const int k = lane + 1 - p.delta + 32 * (n - 1);
                if (k >= 0 && k < p.K) xw[warp * WT_XW + k] = acc[n];
            }
            bar_sync_named(1, 128);
            if (tid < p.K) {
                const float v = ((xw[tid] + xw[WT_XW + tid]) + xw[2 * WT_XW + tid]) + xw[3 * WT_XW + tid];
                if (p.S == 1) {        // no split: finish here (undo the gradient scale, accumulate) and skip the reduction pass
                    const float r = p.gmax ? v * (1.f / pow2_scale(*p.gmax)) : v;
                    float* dst = p.dwd + (size_t)c * p.K + tid;
                    *dst = p.accumulate ? *dst + r : r;
                } else {
                    p.partials[((size_t)sp * p.C + c) * p.K + tid] = v;
                }
            }
            bar_sync_named(1, 128);
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem, 2 * WT_ACC_COLS);
}

constexpr int kWtSmem = WT_RING_BYTES + 1024 /* alignment */ + 512 /* barriers, chunk lengths */ +
                        4 * WT_STG_FLOATS * 4 + 4 * WT_XW * 4 + 16;
static_assert((3 * WT_STAGES + 4) * 8 + 8 + WT_MAX_CHUNKS * 4 <= 512, "barrier block");

template <typename TG, typename TX>
void launch_wt(const Launch& L, int grid, const CUtensorMap& mg, const CUtensorMap& mx, const WtParams& p) {
    auto kern = dw_wgrad_tc_kernel<TG, TX>;
    set_max_smem_once<dw_wgrad_tc_kernel<TG, TX>>(kWtSmem);
    launch_k(L, kern, grid, WT_THREADS, kWtSmem, mg, mx, p);
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
        p.dwd = dwd; p.gmax = gmax; p.accumulate = accumulate;
        p.B = B; p.C = C; p.T = T; p.K = K;
        p.Pa = (P + 7) / 8 * 8; p.delta = p.Pa - P;
        p.BB = B >= 32 ? 32 : 16;
        p.N = (127 + K + p.delta + 15) / 16 * 16;
        p.nxb = (p.N + 63) / 64;
        p.stage_bytes = 2 * (2 + p.nxb) * p.BB * 128;
        p.nstages = std::min(WT_STAGES, WT_RING_BYTES / p.stage_bytes);
        p.nchunks = (B + p.BB - 1) / p.BB;
        p.ntb = (T + 255) / 256;                              // pairs of 128-frame time blocks
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
    if (p.S > 1) reduce_partials(L, partials, p.S, (int64_t)C * K, dwd, accumulate, gmax);
}

}  // namespace sc
