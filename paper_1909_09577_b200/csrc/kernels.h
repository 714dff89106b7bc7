// Internal launcher interface between the C-ABI layer (api.cu) and the kernel files.
// Every function enqueues on L.stream and returns; all pointers are device pointers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <utility>
#include <vector>

namespace sc {

// Kernel classes, for launch counting and per-class event timing.
enum KClass : int {
    KC_LENGTHS = 0, KC_DW_FWD, KC_DW_DGRAD, KC_DW_WGRAD, KC_PW_FWD, KC_PW_DGRAD, KC_PW_WGRAD,
    KC_BN_STATS, KC_BN_FINALIZE, KC_BN_APPLY, KC_BN_BWD_REDUCE, KC_BN_BWD_FINALIZE, KC_BN_BWD_APPLY,
    KC_EW, KC_REDUCE, KC_COUNT
};
const char* kclass_name(int c);

// Optional event timing of one kernel class (or all): a start/stop event pair brackets each launch
// of the selected class on the launching stream; totals are read back after a synchronise.
struct Prof {
    int filter = -2;                       // -2 off, -1 every class, >= 0 one class
    std::vector<cudaEvent_t> events;       // pool, pairs
    struct Rec { int cls; int e0; double bytes, flops; };
    std::vector<Rec> recs;
    size_t used = 0;
};

struct Launch {
    cudaStream_t stream;
    int* status;          // device status word
    int64_t* counter;     // host launch counter
    Prof* prof = nullptr;
    int simt_only = 0;    // 1: never take a tensor-core kernel (used by tests)
    int pdl = 1;          // 1: launch with programmatic stream serialization (see pdl_sync in common.cuh)
    void count(int n = 1) const { if (counter) *counter += n; }
};

// Launches `kern` on L.stream; with L.pdl the launch carries the programmatic-stream-serialization attribute, so
// the kernel may begin (up to its pdl_wait()) before the previous kernel on the stream has completed.
template <typename K, typename... Args>
inline void launch_k(const Launch& L, K kern, dim3 grid, dim3 block, size_t smem, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = L.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = L.pdl ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// Brackets the launches of one launcher call.  bytes/flops are the algorithmic figures of the call.
struct KScope {
    const Launch& L; int slot = -1;
    KScope(const Launch& l, int cls, double bytes, double flops) : L(l) {
        Prof* p = L.prof;
        if (!p || p->filter == -2 || (p->filter >= 0 && p->filter != cls)) return;
        if (p->used + 2 > p->events.size()) return;
        slot = (int)p->used; p->used += 2;
        p->recs.push_back({cls, slot, bytes, flops});
        cudaEventRecord(p->events[slot], L.stream);
    }
    ~KScope() { if (slot >= 0) cudaEventRecord(L.prof->events[slot + 1], L.stream); }
};

// Device the context was created on (-1 for a null context).
}  // namespace sc
struct sc_ctx;
namespace sc {
int ctx_device(const sc_ctx* ctx);

// Launches one CTA that waits, with a short poll limit, on an mbarrier that nothing ever signals: the wait
// must run out, raise the timeout status and return (exercises the bounded-wait exit of the kernels).
void selftest_bounded_wait(const Launch& L);

// cudaFuncAttributeMaxDynamicSharedMemorySize is a per-device property of a kernel: set it once per
// (kernel, device), keyed by the current device.
template <auto Kern> inline void set_max_smem_once(int smem) {
    static unsigned long long done = 0;      // one bit per device ordinal
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && ((done >> dev) & 1ull)) return;
    cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (dev >= 0 && dev < 64) done |= 1ull << dev;
}

// ---- lengths -------------------------------------------------------------------------------
// len_out[b] = ceil(len_in[b]/stride); *nvalid = sum_b len_out[b]; flags lengths outside [1,T_in].
// blk_off (nullable, int [B+1]): exclusive prefix sum of ceil(len_out[b] / 64), the number of 64-frame blocks
// of each sample that hold at least one valid frame; blk_off[B] is their total.
void lengths(const Launch& L, const int* len_in, int B, int T_in, int stride, int* len_out, int* nvalid,
             int* blk_off = nullptr);

// ---- depthwise ------------------------------------------------------------------------------
// u[b,c,t] = sum_k wd[c,k] * x[b,c,t*s+k*dil-P] (x masked by len_in), written as 0 for t >= len_out[b];
// P = (dil*(K-1))/2 zeros on the left ("same" padding; any K >= 1, dil >= 1).
// x and wd in `dtype`, u in `odt` (values beyond the half range are clamped and flagged).
void dw_fwd(const Launch& L, int dtype, int odt, const void* x, const void* wd, void* u, const int* len_in,
            const int* len_out, int B, int C, int T, int Tp, int K, int s, int dil = 1);
// dx[b,c,tau] = [tau < len_in[b]] * (sum_{k,t: t*s+k-P=tau} wd[c,k]*gu[b,c,t] + add1 + add2)
// gu in `odt` and pre-multiplied by pow2_scale(*gmax) when gmax is non-null; wd, add1, add2, dx in `dtype`.
void dw_dgrad(const Launch& L, int dtype, int odt, const void* gu, const void* wd, void* dx, const void* add1,
              const void* add2, const float* gmax, const int* len_in, const int* len_out, int B, int C, int T,
              int Tp, int K, int s, int dil = 1);
// dwd[c,k] (+)= sum_{b,t<len_out} gu[b,c,t] * x[b,c,t*s+k-P] (x masked by len_in).
// partials: float [B*C*K] scratch.
void dw_wgrad(const Launch& L, int dtype, int odt, const void* gu, const void* x, float* dwd, float* partials,
              int accumulate, const float* gmax, const int* len_in, const int* len_out, int B, int C, int T,
              int Tp, int K, int s, int dil = 1);
size_t dw_wgrad_scratch_bytes(int B, int C, int K);
// Tensor-core form of the stride-1 tap gradient (16-bit types, B >= 16, K <= 127): same result as dw_wgrad.
// x_clean != 0 promises that x is already zero at and beyond len_in.  partials: float [8*C*K] at least.
struct TcState;
bool dw_wgrad_tc_supported(const TcState* st, int dtype, int B, int T, int K, int s);
void dw_wgrad_tc(const TcState* st, const Launch& L, int dtype, int odt, const void* gu, const void* x, float* dwd,
                 float* partials, int accumulate, const float* gmax, const int* len_in, const int* len_out, int B,
                 int C, int T, int K, int x_clean);
// TMA-fed tensor-core forms of the stride-1 depthwise forward / input gradient (16-bit types, B >= 16,
// K + padding slack <= 129): same results as dw_fwd / dw_dgrad.  x_clean != 0 promises that x is already
// zero at and beyond len_in.
bool dw_tma_supported(const TcState* st, int dtype, int B, int T, int K, int s);
void dw_tma_fwd(const TcState* st, const Launch& L, int dtype, int odt, const void* x, const void* wd, void* u,
                const int* len_in, const int* len_out, int B, int C, int T, int K, int x_clean);
void dw_tma_dgrad(const TcState* st, const Launch& L, int dtype, int odt, const void* gu, const void* wd, void* dx,
                  const void* add1, const void* add2, const float* gmax, const int* len_in, const int* len_out, int B,
                  int C, int T, int K);
// Tensor-core forms of the stride-1 depthwise forward / input gradient (16-bit types, K <= 129).
bool dw_tc_supported(int dtype, int T, int K, int s);
void dw_tc_fwd(const Launch& L, int dtype, int odt, const void* x, const void* wd, void* u, const int* len_in,
               const int* len_out, int B, int C, int T, int K);
void dw_tc_dgrad(const Launch& L, int dtype, int odt, const void* gu, const void* wd, void* dx, const void* add1,
                 const void* add2, const float* gmax, const int* len_in, const int* len_out, int B, int C, int T,
                 int K);
// out = [t < len[b]] * (a + b + c)   (b, c nullable)
void ew_add_masked(const Launch& L, int dtype, void* out, const void* a, const void* b, const void* c,
                   const int* len, int B, int C, int T);

// ---- pointwise, SIMT (any shape, fp32 accumulate) ------------------------------------------
// v[b,o,t] = [t<len_out[b]] * (sum_c w[o,c]*u[b,c,t] + bias[o]); v is stored in out_dtype
// (a float16 result beyond the half range is clamped and flagged)
void gemm_fwd_simt(const Launch& L, int dtype, const void* w, const void* u, const float* bias, void* v,
                   int out_dtype, const int* len_out, int B, int Cin, int Cout, int Tp);
// gu[b,c,t] = sum_o w[o,c]*gv[b,o,t]
void gemm_dgrad_simt(const Launch& L, int dtype, const void* w, const void* gv, void* gu, int B, int Cin,
                     int Cout, int Tp);
// dw[o,c] (+)= sum_{b,t} gv[b,o,t]*u[b,c,t];  partials: float [nsplit*Cout*Cin]
void gemm_wgrad_simt(const Launch& L, int dtype, const void* gv, const void* u, float* dw, float* partials,
                     int accumulate, int B, int Cin, int Cout, int Tp, const float* gmax = nullptr);
size_t gemm_wgrad_simt_scratch_bytes(int B, int Cin, int Cout);
// out[i] (+)= (sum_s partials[s*n + i]) / pow2_scale(*gmax), fixed order (gmax nullable: no scaling)
void reduce_partials(const Launch& L, const float* partials, int nsplit, int64_t n, float* out, int accumulate,
                     const float* gmax = nullptr);
// dst (half) = src (bf16), n elements
void convert_bf16_to_f16(const Launch& L, const void* src, void* dst, int64_t n);
// the same for up to 48 arrays in one launch
struct ConvertList { const void* src[48]; void* dst[48]; int n[48]; int count; };
void convert_bf16_to_f16_many(const Launch& L, const ConvertList& list);

// ---- non-separable convolution (block variant; k_conv_simt.cu) ---------------------------------
// w [Cout, Cin, K] and x [B, Cin, T] in `dtype`; v [B, Cout, Tp] in out_dtype (dtype, or F16 for BF16 operands).
// "Same" padding with (dil * (K - 1)) / 2 zeros on the left; the input is read as zero from len_in[b] on, the
// result is zero from len_out[b] on.  gv zero in padding is not assumed.
void conv_fwd_simt(const Launch& L, int dtype, const void* w, const void* x, const float* bias, void* v, int out_dtype,
                   const int* len_in, const int* len_out, int B, int Cin, int Cout, int T, int Tp, int K, int stride, int dil);
void conv_dgrad_simt(const Launch& L, int dtype, const void* w, const void* gv, void* dx, const int* len_in, const int* len_out,
                     int B, int Cin, int Cout, int T, int Tp, int K, int stride, int dil);
size_t conv_wgrad_scratch_bytes(int B, int Cin, int Cout, int K);
void conv_wgrad_simt(const Launch& L, int dtype, const void* gv, const void* x, float* dw, float* partials, int accumulate,
                     const int* len_in, const int* len_out, int B, int Cin, int Cout, int T, int Tp, int K, int stride, int dil);

// ---- batch norm -----------------------------------------------------------------------------
// Per-(b,channel) row moments over t < len_out[b]: partials[(b*C+o)] = (sum, M2 about the row mean).
void bn_stats(const Launch& L, int vdtype, const void* v, const int* len_out, int B, int C, int Tp,
              float2* partials);
// Merge partials in a fixed order. parts_per_b tiles of tile_w frames per sample.
// mean/invstd [C]; running stats optional.
void bn_finalize(const Launch& L, const float2* partials, int parts_per_b, int tile_w, const int* len_out,
                 const int* nvalid, int B, int C, float eps, float momentum, float* mean, float* invstd,
                 float* running_mean, float* running_var);

// The same merge for the per-(CTA, channel) float4 (count, sum, M2, -) partials of the flattened-block
// contraction: `grid` CTAs, tiles_m M tiles of rows_per_tile channels, CTA c took the unit range
// [c U / grid, (c+1) U / grid) with U = tiles_m * blk_off[B] (M tile major).
void bn_finalize_flat(const Launch& L, const float4* partials, int grid, int tiles_m, int rows_per_tile,
                      const int* blk_off, const int* nvalid, int B, int C, float eps, float momentum, float* mean,
                      float* invstd, float* running_mean, float* running_var);

// Storage types.  T = activation type.  NT = type of the pointwise result v, which the contraction's
// epilogue writes once and which is kept for the backward pass: float for fp32 activations, half for
// both 16-bit activation types (11 significand bits; bf16's 8 bits on v alone would use most of the
// error budget).  The normalised value vhat = (v - mean) * invstd is never stored: the forward apply
// step and the backward kernels recompute it from v with the same two float operations, so the ReLU
// decision derived from it is the same bit on both sides.
inline int ntype_of(int dtype) { return dtype == 0 ? 0 : 1; }
inline size_t dtype_size(int dtype) { return dtype == 0 ? 4 : 2; }
// OT = type of the tensors that only the library sees between the depthwise and pointwise steps
// (u, and in the backward pass gv and gu): float for fp32; half for BOTH 16-bit activation types when
// the layer has a depthwise step (bf16 activations would otherwise pay a second 8-bit-mantissa rounding
// on every contraction operand); the activation type itself for layers without a depthwise step,
// whose contraction operand is the layer input.
inline int otype_of(int dtype, int has_dw) { return (dtype == 2 && has_dw) ? 1 : dtype; }

// Division of a 32-bit index by a run-time constant without a divide instruction (multiply-high and two
// shifts; exact for every 32-bit numerator).  The flattened elementwise kernels split their thread index
// into (row, position) and a row into (sample, channel) with it.
struct FastDiv {
    uint32_t mul = 1, sh1 = 0, sh2 = 0;
    FastDiv() = default;
    explicit FastDiv(uint32_t d) {
        uint32_t l = 0;
        while (l < 32 && (1ull << l) < d) ++l;
        mul = (uint32_t)(((1ull << 32) * ((1ull << l) - d)) / d + 1);
        sh1 = l < 1 ? l : 1; sh2 = l > 0 ? l - 1 : 0;
    }
#ifdef __CUDACC__
    __device__ __forceinline__ uint32_t div(uint32_t n) const {
        const uint32_t t = __umulhi(n, mul);
        return (t + ((n - t) >> sh1)) >> sh2;
    }
#endif
};

struct ApplyArgs {
    const void* v; const float *mean, *invstd, *gamma, *beta;          // main branch (v in NT)
    int residual;                                  // 0 none, 1 identity, 2 projection
    const void* xres;                              // identity source [B,C,Tp], T
    const void* vr; const float *mean_r, *invstd_r, *gamma_r, *beta_r; // projection branch (vr in NT)
    void* y; const int* len_out;
    int B, C, Tp, has_relu, res_before_relu;
    FastDiv dvpr, dC;                              // by Tp / 8 and by C (set by bn_apply)
};
void bn_apply(const Launch& L, int dtype, const ApplyArgs& a);

struct BnBwdArgs {
    const void* g; const void* y; const void* v; const void* vr;          // v, vr in NT
    const float* mean; const float* mean_r;
    const float* invstd; const float* invstd_r;
    const float *gamma, *beta;                     // for the relu-then-add gate
    const int* len_out; const int* nvalid;
    int B, C, Tp, has_bn, has_relu, res_before_relu, residual;
    float4* partials;                              // [B*C*nslots]
    float* amax_part;                              // [B*C*nslots] max |gated gradient| (only with gmax)
    int nslots;                                    // partial slots per (sample, channel) row; set by bn_bwd_reduce
    int vpw, vpw_shift;                            // 8-frame vectors per warp of the flattened reduce (a power of two) and its log2; set by bn_bwd_reduce
    float* gmax;                                   // device scalar: bound on |gv| over the tensor (nullable)
    int gv_dtype;                                  // storage type of gv (OT)
    float4* coef; float4* coef_r;                  // [C]: (k, c1, c2, unused)
    void* gv; void* gvr; void* gres;               // outputs of the apply step (gvr: proj, gres: identity)
    int gv_scaled;                                 // gv is multiplied by pow2_scale(*gmax) (gmax must be set)
    // Optional half copies for the weight-gradient contractions of bf16 layers whose gv / gvr stay in
    // bf16 (8 significand bits): multiplied by pow2_scale(*gmax), rounded with error diffusion.
    void* gv16; void* gvr16;
    FastDiv dvpr, dC;                              // by Tp / 8 and by C (set by the launchers)
};
void bn_bwd_reduce(const Launch& L, int dtype, BnBwdArgs& a);
// partial slots per row that bn_bwd_reduce may use for rows of Tp frames (for scratch sizing)
inline int bn_bwd_max_slots(int Tp) { return Tp / 256 + 2; }
void bn_bwd_finalize(const Launch& L, const BnBwdArgs& a, const float* gamma, const float* gamma_r,
                     float* dgamma, float* dbeta, float* dgamma_r, float* dbeta_r, float* dbias,
                     int accumulate);
// bn_bwd_reduce followed by bn_bwd_finalize, or -- for the encoder's block shape -- one kernel with a CTA per
// channel that does both.
void bn_bwd_reduce_finalize(const Launch& L, int dtype, BnBwdArgs& a, const float* gamma, const float* gamma_r,
                            float* dgamma, float* dbeta, float* dgamma_r, float* dbeta_r, float* dbias, int accumulate);
void bn_bwd_apply(const Launch& L, int dtype, const BnBwdArgs& a);

// ---- decoder tail / evaluation mode ---------------------------------------------------------------
// y[b,:,t] = [t < len_out[b]] * (z[b,:,t] - log(sum_c exp(z[b,c,t]))), z in float32
void log_softmax_fwd(const Launch& L, int dtype, const float* z, void* y, const int* len_out, int B, int C, int Tp);
// dz[b,c,t] = [t < len_out[b]] * (g[b,c,t] - exp(logp[b,c,t]) * sum_c' g[b,c',t])
void log_softmax_bwd(const Launch& L, int dtype, void* dz, const void* g, const void* logp, const int* len_out, int B,
                     int C, int Tp);
// invstd[o] = 1 / sqrt(var[o] + eps)
void invstd_from_var(const Launch& L, const float* var, float eps, float* invstd, int C);

// out (half) = [t<len[b]] ? in (bf16) : 0; values beyond the half range are clamped and flagged
void mask_convert_f16(const Launch& L, void* out, const void* in, const int* len, int B, int C, int T);
// masked copy: out = [t<len[b]] ? in : 0
void mask_copy(const Launch& L, int dtype, void* out, const void* in, const int* len, int B, int C, int T);

}  // namespace sc
