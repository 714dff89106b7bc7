// C-ABI layer: argument validation, workspace planning and the launch sequence of one block and of
// the whole encoder.  All arithmetic lives in the kernel files; this file only orders launches.
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/sepconv.h"
#include "common.cuh"
#include "kernels.h"
#include "tc_gemm.h"

using namespace sc;

struct sc_ctx {
    int device = 0;
    int sm_count = 0;
    int* status_dev = nullptr;
    int64_t launches = 0;
    int gemm_mode = 0;
    TcState tc;
    Prof prof;
    // A second, library-owned stream: kernels that are off the critical path of a layer (weight gradients, the
    // residual projection's contraction) run there, forked from and joined back into the caller's stream with
    // events, so that they fill the SMs a latency-bound kernel of the critical path leaves idle.
    cudaStream_t side = nullptr;
    cudaEvent_t ev[8] = {};     // backward fork, (unused), done[0], done[1], forward fork, forward join, done[2], (unused)
    int overlap = 1;
    int pdl = 1;          // launch kernels with programmatic stream serialization
};

namespace sc {
int ctx_device(const sc_ctx* ctx) { return ctx ? ctx->device : -1; }
const char* kclass_name(int c) {
    static const char* n[KC_COUNT] = {"lengths", "dw_fwd", "dw_dgrad", "dw_wgrad", "pw_fwd", "pw_dgrad", "pw_wgrad",
                                      "bn_stats", "bn_finalize", "bn_apply", "bn_bwd_reduce", "bn_bwd_finalize",
                                      "bn_bwd_apply", "elementwise", "reduce_partials"};
    return (c >= 0 && c < KC_COUNT) ? n[c] : "?";
}
}  // namespace sc

namespace {

size_t esize(int dtype) { return dtype == SC_F32 ? 4 : 2; }

// Bump allocator over the caller's workspace; with base == nullptr it only measures.
struct Bump {
    char* base; size_t off = 0, cap;
    Bump(void* b, size_t c) : base((char*)b), cap(c) {}
    void* take(size_t bytes) {
        size_t o = (off + 255) & ~(size_t)255;
        off = o + bytes;
        return base ? base + o : nullptr;
    }
    bool ok() const { return base == nullptr || off <= cap; }
};

struct Dims { int B, Cin, Cout, Cres, T, Tp, K, s, dil; bool plain, full; };   // plain: odd K, adjacent taps; full: non-separable convolution

int desc_dims(const sc_block_desc* d, Dims* o) {
    if (!d) return SC_ERR_NULL;
    if (d->io_dtype < 0 || d->io_dtype > 2) return SC_ERR_INCOMPATIBLE;
    if (d->B < 1 || d->C_in < 1 || d->C_out < 1 || d->T_in < 1) return SC_ERR_DIM_INCOMPATIBLE;
    o->B = d->B; o->Cin = d->C_in; o->Cout = d->C_out; o->T = d->T_in;
    o->full = d->full_conv != 0;
    if (o->full && (d->has_dw || d->log_softmax)) return SC_ERR_UNSUPPORTED;
    const bool taps = d->has_dw || o->full;       // the K-tap step: depthwise, or the non-separable convolution
    o->K = taps ? d->K : 1; o->s = taps ? d->stride : 1;
    o->dil = (taps && d->dilation > 1) ? d->dilation : 1;
    if (d->dilation < 0 || o->K < 1) return SC_ERR_UNSUPPORTED;
    if (o->s != 1 && o->s != 2) return SC_ERR_UNSUPPORTED;
    o->plain = o->dil == 1 && (o->K & 1);
    o->Tp = (o->T - 1) / o->s + 1;            // "same" padding: dil * (K - 1) zeros in total
    o->Cres = d->C_res > 0 ? d->C_res : d->C_in;
    if (d->residual < 0 || d->residual > 2) return SC_ERR_UNSUPPORTED;
    if (d->residual == SC_RES_IDENTITY && o->Cres != o->Cout) return SC_ERR_UNSUPPORTED;
    if (d->residual != SC_RES_NONE && !d->has_bn) return SC_ERR_UNSUPPORTED;
    if (!d->has_bn && d->has_relu) return SC_ERR_UNSUPPORTED;
    if (d->has_bn && d->has_bias) return SC_ERR_UNSUPPORTED;   // a bias before batch norm cancels
    if (d->log_softmax && (d->has_bn || d->has_relu || d->residual != SC_RES_NONE)) return SC_ERR_UNSUPPORTED;
    return SC_OK;
}

int check_tensor(const sc_tensor* t, int dtype, int64_t B, int64_t C, int64_t T) {
    if (!t || !t->ptr) return SC_ERR_NULL;
    if (t->dtype != dtype || t->rank != 3) return SC_ERR_INCOMPATIBLE;
    const int64_t want[3] = {B, C, T};
    const int wtag[3] = {SC_AX_BATCH, SC_AX_CHANNEL, SC_AX_TIME};
    bool tags_ok = true, sizes_ok = true;
    for (int i = 0; i < 3; ++i) { tags_ok &= (t->tag[i] == wtag[i]); sizes_ok &= (t->size[i] == want[i]); }
    if (!tags_ok) {
        // same axes in another order -> transposed; otherwise not a [batch, channel, time] tensor
        int seen = 0;
        for (int i = 0; i < 3; ++i) if (t->tag[i] >= 0 && t->tag[i] <= 2) seen |= 1 << t->tag[i];
        return seen == 7 ? SC_ERR_TRANSPOSED : SC_ERR_INCOMPATIBLE;
    }
    if (!sizes_ok) return SC_ERR_DIM_INCOMPATIBLE;
    if (t->stride[2] != 1 || t->stride[1] != T || t->stride[0] != C * T) return SC_ERR_TRANSPOSED;
    if (((uintptr_t)t->ptr & 15) != 0) return SC_ERR_ALIGNMENT;
    return SC_OK;
}

struct BlockIO {                 // raw pointers after validation
    const void* x; const void* xres; void* y;
    const int* len_in; int* len_out; int* nvalid; int* blk_off;
    bool x_clean, res_clean;     // inputs known to be zero in padded frames
    bool lengths_ready;          // len_out / nvalid already computed
    void* w16_keep;              // optional: where to leave the float16 copy of wp for the backward pass
    bool w16_ready;              // w16_keep already holds the copy
};

// Type of the library-internal contraction operands (u, gv, gu) of this layer.
int op_dtype(const sc_block_desc* d) { return otype_of(d->io_dtype, d->has_dw && d->has_bn); }

// ---- forward scratch ---------------------------------------------------------------------------
struct FwdScratch { void* partials; void* partials_r; void *xr, *w16; float* zf32; int* len_out; int* nvalid; int* blk_off; };

void plan_fwd(const sc_block_desc* d, const Dims& m, Bump& ws, FwdScratch* f, const TcState* tc) {
    f->len_out = (int*)ws.take(sizeof(int) * m.B);
    f->nvalid = (int*)ws.take(sizeof(int));
    f->blk_off = (int*)ws.take(sizeof(int) * (m.B + 1));
    f->partials = ws.take(tc_stats_bytes(m.B, m.Cout, m.Tp));
    f->partials_r = (d->residual == SC_RES_PROJ) ? ws.take(tc_stats_bytes(m.B, m.Cout, m.Tp)) : nullptr;
    f->zf32 = d->log_softmax ? (float*)ws.take(sizeof(float) * m.B * m.Cout * m.Tp) : nullptr;
    f->xr = (d->residual == SC_RES_PROJ) ? ws.take(esize(d->io_dtype) * m.B * m.Cres * m.Tp) : nullptr;
    f->w16 = (op_dtype(d) != d->io_dtype) ? ws.take((size_t)2 * m.Cout * m.Cin) : nullptr;
}

// v = w * u for every sample (stored once, in the type it is kept in for the backward pass), plus masked
// batch statistics.
void pointwise_bn(sc_ctx* ctx, const Launch& L, const sc_block_desc* d, const Dims& m, int Cin, int opdt,
                  const void* w, const void* u, void* v, const int* len_out, const int* nvalid, const int* blk_off,
                  float* mean, float* invstd, void* partials, float* rmean, float* rvar) {
    const int vdt = ntype_of(d->io_dtype);
    StatsLayout sl;
    if (ctx->gemm_mode == 0 && tc_fwd_supported(&ctx->tc, opdt, Cin, m.Cout, m.Tp))
        tc_gemm_fwd(&ctx->tc, L, opdt, w, u, nullptr, v, vdt, len_out, blk_off, m.B, Cin, m.Cout, m.Tp, partials, &sl);
    else
        gemm_fwd_simt(L, opdt, w, u, nullptr, v, vdt, len_out, m.B, Cin, m.Cout, m.Tp);
    if (sl.kind == 2) {
        bn_finalize_flat(L, (const float4*)partials, sl.grid, sl.tiles_m, sl.rows_per_tile, blk_off, nvalid, m.B, m.Cout,
                         d->bn_eps, d->bn_momentum, mean, invstd, rmean, rvar);
        return;
    }
    if (sl.kind == 0) { bn_stats(L, vdt, v, len_out, m.B, m.Cout, m.Tp, (float2*)partials); sl.parts_per_b = 1; sl.tile_w = m.Tp; }
    bn_finalize(L, (const float2*)partials, sl.parts_per_b, sl.tile_w, len_out, nvalid, m.B, m.Cout, d->bn_eps, d->bn_momentum,
                mean, invstd, rmean, rvar);
}

// The launch context of the side stream (same status word, counters and profile), or L itself when overlap is off.
Launch side_launch(sc_ctx* ctx, const Launch& L) {
    Launch s = L;
    if (ctx->overlap && ctx->side) s.stream = ctx->side;
    return s;
}
// side stream waits for everything enqueued on L.stream so far
void fork_to_side(sc_ctx* ctx, const Launch& L, cudaEvent_t ev) {
    if (!(ctx->overlap && ctx->side)) return;
    cudaEventRecord(ev, L.stream);
    cudaStreamWaitEvent(ctx->side, ev, 0);
}
void record_side(sc_ctx* ctx, cudaEvent_t ev) { if (ctx->overlap && ctx->side) cudaEventRecord(ev, ctx->side); }
void wait_side(sc_ctx* ctx, const Launch& L, cudaEvent_t ev) { if (ctx->overlap && ctx->side) cudaStreamWaitEvent(L.stream, ev, 0); }

// Evaluation mode: fixed running statistics take the place of the batch statistics.
struct InferStats { const float *mean, *var, *mean_r, *var_r; };

// v = w * u without statistics (evaluation mode); invstd <- 1 / sqrt(var + eps)
void pointwise_fixed(sc_ctx* ctx, const Launch& L, const sc_block_desc* d, const Dims& m, int Cin, int opdt, const void* w,
                     const void* u, void* v, const int* len_out, const int* blk_off, const float* var, float* invstd) {
    const int vdt = ntype_of(d->io_dtype);
    if (ctx->gemm_mode == 0 && tc_fwd_supported(&ctx->tc, opdt, Cin, m.Cout, m.Tp))
        tc_gemm_fwd(&ctx->tc, L, opdt, w, u, nullptr, v, vdt, len_out, blk_off, m.B, Cin, m.Cout, m.Tp, nullptr, nullptr);
    else
        gemm_fwd_simt(L, opdt, w, u, nullptr, v, vdt, len_out, m.B, Cin, m.Cout, m.Tp);
    invstd_from_var(L, var, d->bn_eps, invstd, m.Cout);
}

int block_fwd_impl(sc_ctx* ctx, const Launch& L, const sc_block_desc* d, const Dims& m, BlockIO io,
                   const sc_block_params* p, sc_block_saved* sv, float* rmean, float* rvar,
                   const FwdScratch& f, const InferStats* inf = nullptr) {
    const int dt = d->io_dtype;
    if (!io.lengths_ready) lengths(L, io.len_in, m.B, m.T, m.s, io.len_out, io.nvalid, io.blk_off);
    const int odt = op_dtype(d);
    if (d->has_bn && d->residual == SC_RES_PROJ) {
        // the residual projection does not depend on the main branch: its contraction and statistics go to the
        // side stream and are joined just before the apply step
        fork_to_side(ctx, L, ctx->ev[4]);
        const Launch Ls = side_launch(ctx, L);
        const void* xr = io.xres;
        if (!io.res_clean) { mask_copy(Ls, dt, f.xr, io.xres, io.len_out, m.B, m.Cres, m.Tp); xr = f.xr; }
        if (inf) pointwise_fixed(ctx, Ls, d, m, m.Cres, dt, p->wr, xr, sv->vr, io.len_out, io.blk_off, inf->var_r, sv->invstd_r);
        else pointwise_bn(ctx, Ls, d, m, m.Cres, dt, p->wr, xr, sv->vr, io.len_out, io.nvalid, io.blk_off, sv->mean_r,
                          sv->invstd_r, f.partials_r, nullptr, nullptr);
        record_side(ctx, ctx->ev[5]);
    }
    if (m.full) {
        // block variant: one K-tap convolution over all input channels (it masks its input by len_in itself)
        if (!d->has_bn) {
            conv_fwd_simt(L, dt, p->wp, io.x, d->has_bias ? p->bias : nullptr, io.y, dt, io.len_in, io.len_out, m.B, m.Cin, m.Cout,
                          m.T, m.Tp, m.K, m.s, m.dil);
            return SC_OK;
        }
        const int vdt = ntype_of(dt);
        conv_fwd_simt(L, dt, p->wp, io.x, nullptr, sv->v, vdt, io.len_in, io.len_out, m.B, m.Cin, m.Cout, m.T, m.Tp, m.K, m.s, m.dil);
        if (inf) {
            invstd_from_var(L, inf->var, d->bn_eps, sv->invstd, m.Cout);
        } else {
            bn_stats(L, vdt, sv->v, io.len_out, m.B, m.Cout, m.Tp, (float2*)f.partials);
            bn_finalize(L, (const float2*)f.partials, 1, m.Tp, io.len_out, io.nvalid, m.B, m.Cout, d->bn_eps, d->bn_momentum, sv->mean,
                        sv->invstd, rmean, rvar);
        }
    }
    const void* u = nullptr;
    if (m.full) {
    } else if (d->has_dw) {
        if (ctx->gemm_mode == 0 && m.plain && dw_tma_supported(&ctx->tc, dt, m.B, m.T, m.K, m.s))
            dw_tma_fwd(&ctx->tc, L, dt, odt, io.x, p->wd, sv->u, io.len_in, io.len_out, m.B, m.Cin, m.T, m.K,
                       io.x_clean ? 1 : 0);
        else
            dw_fwd(L, dt, odt, io.x, p->wd, sv->u, io.len_in, io.len_out, m.B, m.Cin, m.T, m.Tp, m.K, m.s, m.dil);
        u = sv->u;
    } else if (io.x_clean) {
        u = io.x;
    } else {
        mask_copy(L, dt, sv->u, io.x, io.len_in, m.B, m.Cin, m.T);
        u = sv->u;
    }
    if (!d->has_bn) {   // linear layer: y = mask * (w u + bias), or its log-softmax over the channels
        // with the decoder tail the class scores stay in float32 until the log-softmax has been taken
        void* z = d->log_softmax ? (void*)f.zf32 : io.y;
        const int zdt = d->log_softmax ? (int)SC_F32 : dt;
        if (ctx->gemm_mode == 0 && tc_fwd_supported(&ctx->tc, dt, m.Cin, m.Cout, m.Tp)) {
            tc_gemm_fwd(&ctx->tc, L, dt, p->wp, u, d->has_bias ? p->bias : nullptr, z, zdt, io.len_out, io.blk_off, m.B,
                        m.Cin, m.Cout, m.Tp, nullptr, nullptr);
        } else {
            gemm_fwd_simt(L, dt, p->wp, u, d->has_bias ? p->bias : nullptr, z, zdt, io.len_out, m.B, m.Cin, m.Cout, m.Tp);
        }
        if (d->log_softmax) log_softmax_fwd(L, dt, f.zf32, io.y, io.len_out, m.B, m.Cout, m.Tp);
        return SC_OK;
    }
    const void* wp_op = p->wp;
    if (odt != dt && !m.full) {
        void* dst = io.w16_keep ? io.w16_keep : f.w16;
        if (!(io.w16_keep && io.w16_ready)) convert_bf16_to_f16(L, p->wp, dst, (int64_t)m.Cout * m.Cin);
        wp_op = dst;
    }
    if (m.full) {}
    else if (inf) pointwise_fixed(ctx, L, d, m, m.Cin, odt, wp_op, u, sv->v, io.len_out, io.blk_off, inf->var, sv->invstd);
    else pointwise_bn(ctx, L, d, m, m.Cin, odt, wp_op, u, sv->v, io.len_out, io.nvalid, io.blk_off, sv->mean, sv->invstd,
                      f.partials, rmean, rvar);
    ApplyArgs a{};
    a.v = sv->v; a.mean = inf ? inf->mean : sv->mean; a.invstd = sv->invstd; a.gamma = p->gamma; a.beta = p->beta;
    a.residual = d->residual; a.y = io.y; a.len_out = io.len_out;
    a.B = m.B; a.C = m.Cout; a.Tp = m.Tp; a.has_relu = d->has_relu; a.res_before_relu = d->res_before_relu;
    if (d->residual == SC_RES_IDENTITY) a.xres = io.xres;
    if (d->residual == SC_RES_PROJ) {
        a.vr = sv->vr; a.mean_r = inf ? inf->mean_r : sv->mean_r; a.invstd_r = sv->invstd_r; a.gamma_r = p->gamma_r; a.beta_r = p->beta_r;
        wait_side(ctx, L, ctx->ev[5]);      // the projection branch (enqueued above on the side stream) is complete
    }
    bn_apply(L, dt, a);
    return SC_OK;
}

// ---- backward scratch --------------------------------------------------------------------------
struct BwdScratch {
    int* len_out; int* nvalid; int* blk_off;
    float4 *partials, *coef, *coef_r;
    float *amax_part, *gmax;
    void *gv, *gvr, *gres, *gu, *gxr, *xr, *w16, *dz;
    void *gv16, *gvr16, *x16, *xr16;     // half copies for the weight gradients of bf16 layers (see block_bwd_impl)
    float* wpart; size_t wpart_bytes;
};

void plan_bwd(const sc_block_desc* d, const Dims& m, Bump& ws, BwdScratch* s, const TcState* tc) {
    const size_t e = esize(d->io_dtype);
    // gu holds the gradient w.r.t. the pointwise operand [B, C_in, T']; with the non-separable convolution it is the
    // staging tensor of the input gradient [B, C_in, T]
    const size_t act_out = e * m.B * m.Cout * m.Tp, act_in = e * m.B * m.Cin * (m.full ? m.T : m.Tp);
    s->len_out = (int*)ws.take(sizeof(int) * m.B);
    s->nvalid = (int*)ws.take(sizeof(int));
    s->blk_off = (int*)ws.take(sizeof(int) * (m.B + 1));
    s->partials = (float4*)ws.take(sizeof(float4) * m.B * m.Cout * bn_bwd_max_slots(m.Tp));
    s->coef = (float4*)ws.take(sizeof(float4) * m.Cout);
    s->coef_r = (float4*)ws.take(sizeof(float4) * m.Cout);
    s->amax_part = (float*)ws.take(sizeof(float) * m.B * m.Cout * bn_bwd_max_slots(m.Tp));
    s->gmax = (float*)ws.take(sizeof(float));
    s->w16 = (op_dtype(d) != d->io_dtype) ? ws.take((size_t)2 * m.Cout * m.Cin) : nullptr;
    s->gv = ws.take(act_out);
    s->dz = d->log_softmax ? ws.take(act_out) : nullptr;
    s->gvr = d->residual == SC_RES_PROJ ? ws.take(act_out) : nullptr;
    s->gres = d->residual == SC_RES_IDENTITY ? ws.take(act_out) : nullptr;
    s->gu = ws.take(act_in);
    s->gxr = d->residual == SC_RES_PROJ ? ws.take(e * m.B * m.Cres * m.Tp) : nullptr;
    s->xr = d->residual == SC_RES_PROJ ? ws.take(e * m.B * m.Cres * m.Tp) : nullptr;
    const bool bf = d->io_dtype == SC_BF16 && d->has_bn && !m.full;
    s->gv16 = (bf && !d->has_dw) ? ws.take(act_out) : nullptr;
    s->x16 = (bf && !d->has_dw) ? ws.take(act_in) : nullptr;
    s->gvr16 = (bf && d->residual == SC_RES_PROJ) ? ws.take(act_out) : nullptr;
    s->xr16 = (bf && d->residual == SC_RES_PROJ) ? ws.take(e * m.B * m.Cres * m.Tp) : nullptr;
    size_t wb = gemm_wgrad_simt_scratch_bytes(m.B, std::max(m.Cin, m.Cres), m.Cout);
    wb = std::max(wb, tc_wgrad_scratch_bytes(tc, std::max(m.Cin, m.Cres), m.Cout));
    wb = std::max(wb, dw_wgrad_scratch_bytes(m.B, m.Cin, m.K));
    if (m.full) wb = std::max(wb, conv_wgrad_scratch_bytes(m.B, m.Cin, m.Cout, m.K));
    s->wpart = (float*)ws.take(wb);
    s->wpart_bytes = wb;
}

void pointwise_wgrad(sc_ctx* ctx, const Launch& L, int dt, const void* gv, const void* u, float* dw,
                     float* part, int acc, int B, int Cin, int Cout, int Tp, const int* len_out,
                     const float* gmax) {
    if (ctx->gemm_mode == 0 && tc_wgrad_supported(&ctx->tc, dt, Cin, Cout, Tp))
        tc_gemm_wgrad(&ctx->tc, L, dt, gv, u, dw, part, acc, B, Cin, Cout, Tp, len_out, gmax);
    else
        gemm_wgrad_simt(L, dt, gv, u, dw, part, acc, B, Cin, Cout, Tp, gmax);
}
void pointwise_dgrad(sc_ctx* ctx, const Launch& L, int dt, const void* w, const void* gv, void* gu, int B,
                     int Cin, int Cout, int Tp, const int* len_out, const int* blk_off) {
    if (ctx->gemm_mode == 0 && tc_dgrad_supported(&ctx->tc, dt, Cin, Cout, Tp))
        tc_gemm_dgrad(&ctx->tc, L, dt, w, gv, gu, B, Cin, Cout, Tp, len_out, blk_off);
    else
        gemm_dgrad_simt(L, dt, w, gv, gu, B, Cin, Cout, Tp);
}

struct BwdIO {
    const void *dy, *x, *xres, *y;
    void *dx, *dx_res; const void* dx_add;
    const int* len_in; const int* len_out; const int* nvalid; const int* blk_off;
    bool x_clean, res_clean;
    const void* w16_kept;        // float16 copy of wp left by the forward pass (optional)
    cudaEvent_t done;            // recorded on the side stream after this layer's last side-stream kernel
    float* gmax_zeroed;          // optional: a float the caller has already set to zero, used for the |gv| bound
                                 // (a memset between two kernels would end the programmatic overlap of that pair)
};

int block_bwd_impl(sc_ctx* ctx, const Launch& L, const sc_block_desc* d, const Dims& m, BwdIO io,
                   const sc_block_params* p, const sc_block_saved* sv, sc_block_grads* g, int acc,
                   const BwdScratch& s) {
    const int dt = d->io_dtype;
    const int odt = op_dtype(d);
    // gv (and gu after it) is kept scaled by a power of two whenever it is a library-internal 16-bit
    // tensor, so that neither a tiny nor a huge upstream gradient leaves the half range
    // bf16 layers whose gv / gvr stay in bf16 (no depthwise step; the residual projection) get a scaled
    // half copy of that gradient, and of the other operand, for their weight-gradient contraction: with
    // 8 significand bits the rounding of the gradient alone uses most of the error budget of dwp / dwr
    const bool tc_ok = ctx->gemm_mode == 0;
    const bool half_gv = dt == SC_BF16 && d->has_bn && !d->has_dw && !m.full && s.gv16 && tc_ok &&
                         tc_wgrad_supported(&ctx->tc, SC_F16, m.Cin, m.Cout, m.Tp);
    const bool half_gvr = dt == SC_BF16 && d->has_bn && d->residual == SC_RES_PROJ && s.gvr16 && tc_ok &&
                          tc_wgrad_supported(&ctx->tc, SC_F16, m.Cres, m.Cout, m.Tp);
    float* gmax = (dt != SC_F32 && d->has_bn && (d->has_dw || half_gv || half_gvr)) ? (io.gmax_zeroed ? io.gmax_zeroed : s.gmax) : nullptr;
    if (gmax && !io.gmax_zeroed) cudaMemsetAsync(gmax, 0, sizeof(float), L.stream);
    const void* dy = io.dy;
    if (d->log_softmax) {      // upstream gradient is w.r.t. the log-probabilities: back through the log-softmax first
        log_softmax_bwd(L, dt, s.dz, io.dy, io.y, io.len_out, m.B, m.Cout, m.Tp);
        dy = s.dz;
    }
    BnBwdArgs a{};
    a.amax_part = s.amax_part; a.gmax = gmax; a.gv_dtype = odt;
    a.gv_scaled = (gmax && d->has_dw) ? 1 : 0;
    a.gv16 = half_gv ? s.gv16 : nullptr; a.gvr16 = half_gvr ? s.gvr16 : nullptr;
    a.g = dy; a.y = io.y; a.v = sv->v; a.vr = sv->vr;
    a.mean = sv->mean; a.mean_r = sv->mean_r; a.invstd = sv->invstd; a.invstd_r = sv->invstd_r; a.gamma = p->gamma; a.beta = p->beta;
    a.len_out = io.len_out; a.nvalid = io.nvalid;
    a.B = m.B; a.C = m.Cout; a.Tp = m.Tp; a.has_bn = d->has_bn; a.has_relu = d->has_relu;
    a.res_before_relu = d->res_before_relu; a.residual = d->residual;
    a.partials = s.partials; a.coef = s.coef; a.coef_r = s.coef_r;
    a.gv = s.gv; a.gvr = s.gvr;
    // identity residual: its gradient is the gated upstream gradient itself
    a.gres = (d->residual == SC_RES_IDENTITY) ? (io.dx_res ? io.dx_res : s.gres) : nullptr;
    bn_bwd_reduce_finalize(L, dt, a, p->gamma, p->gamma_r, g->dgamma, g->dbeta, g->dgamma_r, g->dbeta_r,
                           d->has_bias ? g->dbias : nullptr, acc);
    bn_bwd_apply(L, dt, a);

    // The weight gradients are off the critical path (nothing later in the backward pass reads them): they run on the
    // side stream.  They are enqueued after the input-gradient kernels of this stream: the host issues launches in
    // program order, and kernels of the critical path that sit behind side-stream launches in that order start late
    // whenever the GPU is ahead of the host.  One event, recorded behind this layer's last main-stream kernel, releases
    // them (an event between two kernels ends the programmatic overlap of that pair, so there is only one per layer);
    // they then overlap the next layer's main-stream kernels.
    const Launch Ls = side_launch(ctx, L);
    auto weight_gradients = [&]() {
        fork_to_side(ctx, L, ctx->ev[0]);               // gv, gvr, gu and the half copies are complete
        const void* u = d->has_dw ? sv->u : (io.x_clean ? io.x : sv->u);
        if (m.full) {
            conv_wgrad_simt(Ls, dt, s.gv, io.x, g->dwp, s.wpart, acc, io.len_in, io.len_out, m.B, m.Cin, m.Cout, m.T, m.Tp, m.K, m.s, m.dil);
        } else if (half_gv) {
            mask_convert_f16(Ls, s.x16, io.x, io.len_in, m.B, m.Cin, m.T);
            pointwise_wgrad(ctx, Ls, SC_F16, s.gv16, s.x16, g->dwp, s.wpart, acc, m.B, m.Cin, m.Cout, m.Tp, io.len_out, gmax);
        } else {
            pointwise_wgrad(ctx, Ls, odt, s.gv, u, g->dwp, s.wpart, acc, m.B, m.Cin, m.Cout, m.Tp, io.len_out,
                            a.gv_scaled ? gmax : nullptr);
        }
        if (d->residual == SC_RES_PROJ) {
            if (half_gvr) {
                mask_convert_f16(Ls, s.xr16, io.xres, io.len_out, m.B, m.Cres, m.Tp);
                pointwise_wgrad(ctx, Ls, SC_F16, s.gvr16, s.xr16, g->dwr, s.wpart, acc, m.B, m.Cres, m.Cout, m.Tp, io.len_out, gmax);
            } else {
                const void* xr = io.xres;
                if (!io.res_clean) { mask_copy(Ls, dt, s.xr, io.xres, io.len_out, m.B, m.Cres, m.Tp); xr = s.xr; }
                pointwise_wgrad(ctx, Ls, dt, s.gvr, xr, g->dwr, s.wpart, acc, m.B, m.Cres, m.Cout, m.Tp, io.len_out, nullptr);
            }
        }
        if (d->has_dw && !m.full) {
            if (ctx->gemm_mode == 0 && m.plain && dw_wgrad_tc_supported(&ctx->tc, dt, m.B, m.T, m.K, m.s))
                dw_wgrad_tc(&ctx->tc, Ls, dt, odt, s.gu, io.x, g->dwd, s.wpart, acc, gmax, io.len_in, io.len_out, m.B, m.Cin,
                            m.T, m.K, io.x_clean ? 1 : 0);
            else
                dw_wgrad(Ls, dt, odt, s.gu, io.x, g->dwd, s.wpart, acc, gmax, io.len_in, io.len_out, m.B, m.Cin, m.T, m.Tp, m.K, m.s, m.dil);
        }
    };

    const void* wp_op = p->wp;
    if (odt != dt && !m.full) {
        if (io.w16_kept) wp_op = io.w16_kept;
        else { convert_bf16_to_f16(L, p->wp, s.w16, (int64_t)m.Cout * m.Cin); wp_op = s.w16; }
    }
    const void* extra = nullptr;    // residual-path gradient to fold into dx
    if (d->residual == SC_RES_PROJ) {
        void* tgt = io.dx_res ? io.dx_res : s.gxr;
        if (io.dx_res || io.dx) pointwise_dgrad(ctx, L, dt, p->wr, s.gvr, tgt, m.B, m.Cres, m.Cout, m.Tp, io.len_out, io.blk_off);
        if (!io.dx_res) extra = s.gxr;
    } else if (d->residual == SC_RES_IDENTITY && !io.dx_res) {
        extra = s.gres;
    }

    if (m.full) {
        if (io.dx) {
            void* tgt = (!io.dx_add && !extra) ? io.dx : s.gu;
            conv_dgrad_simt(L, dt, p->wp, s.gv, tgt, io.len_in, io.len_out, m.B, m.Cin, m.Cout, m.T, m.Tp, m.K, m.s, m.dil);
            if (tgt != io.dx) ew_add_masked(L, dt, io.dx, s.gu, io.dx_add, extra, io.len_in, m.B, m.Cin, m.T);
        }
    } else if (d->has_dw) {
        pointwise_dgrad(ctx, L, odt, wp_op, s.gv, s.gu, m.B, m.Cin, m.Cout, m.Tp, io.len_out, io.blk_off);
        if (io.dx) {
            if (ctx->gemm_mode == 0 && m.plain && dw_tma_supported(&ctx->tc, dt, m.B, m.T, m.K, m.s))
                dw_tma_dgrad(&ctx->tc, L, dt, odt, s.gu, p->wd, io.dx, io.dx_add, extra, gmax, io.len_in, io.len_out, m.B,
                             m.Cin, m.T, m.K);
            else
                dw_dgrad(L, dt, odt, s.gu, p->wd, io.dx, io.dx_add, extra, gmax, io.len_in, io.len_out, m.B, m.Cin, m.T,
                         m.Tp, m.K, m.s, m.dil);
        }
    } else if (io.dx) {
        if (!io.dx_add && !extra) {
            pointwise_dgrad(ctx, L, dt, p->wp, s.gv, io.dx, m.B, m.Cin, m.Cout, m.Tp, io.len_out, io.blk_off);
        } else {
            pointwise_dgrad(ctx, L, dt, p->wp, s.gv, s.gu, m.B, m.Cin, m.Cout, m.Tp, io.len_out, io.blk_off);
            ew_add_masked(L, dt, io.dx, s.gu, io.dx_add, extra, io.len_in, m.B, m.Cin, m.T);
        }
    }
    weight_gradients();
    // the caller joins: it waits for io.done on its stream before it reuses this scratch or returns
    if (io.done) record_side(ctx, io.done);
    return SC_OK;
}

int check_params(const sc_block_desc* d, const sc_block_params* p) {
    if (!p || !p->wp) return SC_ERR_NULL;
    if (d->has_dw && !p->wd) return SC_ERR_NULL;
    if (d->has_bn && (!p->gamma || !p->beta)) return SC_ERR_NULL;
    if (d->has_bias && !p->bias) return SC_ERR_NULL;
    if (d->residual == SC_RES_PROJ && (!p->wr || !p->gamma_r || !p->beta_r)) return SC_ERR_NULL;
    return SC_OK;
}
int check_saved(const sc_block_desc* d, const sc_block_saved* s, bool x_clean) {
    if (!s) return SC_ERR_NULL;
    if (!d->full_conv && (d->has_dw || !x_clean) && !s->u) return SC_ERR_NULL;
    if (d->has_bn && (!s->v || !s->mean || !s->invstd)) return SC_ERR_NULL;
    if (d->residual == SC_RES_PROJ && (!s->vr || !s->mean_r || !s->invstd_r)) return SC_ERR_NULL;
    return SC_OK;
}
int check_grads(const sc_block_desc* d, const sc_block_grads* g) {
    if (!g || !g->dwp) return SC_ERR_NULL;
    if (d->has_dw && !g->dwd) return SC_ERR_NULL;
    if (d->has_bn && (!g->dgamma || !g->dbeta)) return SC_ERR_NULL;
    if (d->has_bias && !g->dbias) return SC_ERR_NULL;
    if (d->residual == SC_RES_PROJ && (!g->dwr || !g->dgamma_r || !g->dbeta_r)) return SC_ERR_NULL;
    return SC_OK;
}

int finish(sc_ctx* ctx) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { fprintf(stderr, "sepconv: CUDA error: %s\n", cudaGetErrorString(e)); return SC_ERR_CUDA; }
    (void)ctx;
    return SC_OK;
}

#define SC_TRY(expr) do { int _r = (expr); if (_r != SC_OK) return _r; } while (0)

}  // namespace

// =================================================================================================
extern "C" {

int sepconv_ctx_create(sc_ctx** out, int device) {
    if (!out) return SC_ERR_NULL;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SC_ERR_CUDA;
    if (prop.major != 10) return SC_ERR_ARCH;
    if (cudaSetDevice(device) != cudaSuccess) return SC_ERR_CUDA;
    sc_ctx* c = new (std::nothrow) sc_ctx();
    if (!c) return SC_ERR_CUDA;
    c->device = device;
    c->sm_count = prop.multiProcessorCount;
    if (cudaMalloc(&c->status_dev, 64) != cudaSuccess) { delete c; return SC_ERR_CUDA; }
    cudaMemset(c->status_dev, 0, 64);
    int r = tc_init(&c->tc, device, c->sm_count);
    if (r != SC_OK) { cudaFree(c->status_dev); delete c; return r; }
    bool ok = cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < 8 && ok; ++i) ok = cudaEventCreateWithFlags(&c->ev[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { sepconv_ctx_destroy(c); return SC_ERR_CUDA; }
    *out = c;
    return SC_OK;
}

void sepconv_ctx_destroy(sc_ctx* ctx) {
    if (!ctx) return;
    for (cudaEvent_t e : ctx->prof.events) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->ev) if (e) cudaEventDestroy(e);
    if (ctx->side) cudaStreamDestroy(ctx->side);
    cudaFree(ctx->status_dev);
    tc_destroy(&ctx->tc);
    delete ctx;
}

int sepconv_last_status(sc_ctx* ctx, void* stream) {
    if (!ctx) return SC_ERR_NULL;
    int h = 0;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(&h, ctx->status_dev, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SC_ERR_CUDA;
    if (cudaMemsetAsync(ctx->status_dev, 0, sizeof(int), st) != cudaSuccess) return SC_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SC_ERR_CUDA;
    return h;
}

const char* sepconv_strerror(int s) {
    switch (s) {
        case SC_OK: return "ok";
        case SC_ERR_NULL: return "a required pointer is null";
        case SC_ERR_INCOMPATIBLE: return "incompatible tensor type (dtype, rank or axis tags)";
        case SC_ERR_DIM_INCOMPATIBLE: return "an axis size disagrees with the descriptor";
        case SC_ERR_TRANSPOSED: return "axes are transposed or the tensor is not dense [batch, channel, time]";
        case SC_ERR_ALIGNMENT: return "pointer is not 16-byte aligned";
        case SC_ERR_UNSUPPORTED: return "unsupported block configuration";
        case SC_ERR_WORKSPACE: return "workspace is null or too small";
        case SC_ERR_LENGTHS: return "a length lies outside [1, T]";
        case SC_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
        case SC_ERR_ARCH: return "device is not compute capability 10.x";
        case SC_ERR_CUDA: return "a CUDA call failed";
        case SC_ERR_RANGE: return "an intermediate value left the float16 range and was clamped";
        default: return "unknown status";
    }
}

int sepconv_selftest_bounded_wait(sc_ctx* ctx, void* cuda_stream) {
    if (!ctx) return SC_ERR_NULL;
    Launch L{(cudaStream_t)cuda_stream, ctx->status_dev, &ctx->launches, &ctx->prof, ctx->gemm_mode, ctx->pdl};
    selftest_bounded_wait(L);
    return finish(ctx);
}

int sepconv_set_tile_shape(sc_ctx* ctx, int shape) {
    if (!ctx) return SC_ERR_NULL;
    if (shape < 0 || shape > 5) return SC_ERR_UNSUPPORTED;
    ctx->tc.flat_shape = shape;
    return SC_OK;
}

int sepconv_set_overlap(sc_ctx* ctx, int on) {
    if (!ctx) return SC_ERR_NULL;
    if (on < 0 || on > 3) return SC_ERR_UNSUPPORTED;
    ctx->overlap = on & 1;
    ctx->pdl = (on >> 1) & 1;
    return SC_OK;
}

int sepconv_set_gemm_mode(sc_ctx* ctx, int mode) {
    if (!ctx) return SC_ERR_NULL;
    if (mode != 0 && mode != 1) return SC_ERR_UNSUPPORTED;
    ctx->gemm_mode = mode;
    return SC_OK;
}

int64_t sepconv_launch_count(sc_ctx* ctx) { return ctx ? ctx->launches : 0; }

int sepconv_profile_begin(sc_ctx* ctx, int kernel_class, int max_launches) {
    if (!ctx) return SC_ERR_NULL;
    if (kernel_class < -1 || kernel_class >= KC_COUNT || max_launches < 1) return SC_ERR_UNSUPPORTED;
    Prof& p = ctx->prof;
    while (p.events.size() < (size_t)2 * max_launches) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return SC_ERR_CUDA;
        p.events.push_back(e);
    }
    p.recs.clear(); p.used = 0; p.filter = kernel_class;
    return SC_OK;
}

int sepconv_profile_end(sc_ctx* ctx, void* cuda_stream, double* ms, int64_t* launches, double* bytes,
                        double* flops) {
    if (!ctx || !ms || !launches || !bytes || !flops) return SC_ERR_NULL;
    Prof& p = ctx->prof;
    p.filter = -2;
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return SC_ERR_CUDA;
    for (int c = 0; c < KC_COUNT; ++c) { ms[c] = 0; launches[c] = 0; bytes[c] = 0; flops[c] = 0; }
    for (const Prof::Rec& r : p.recs) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, p.events[r.e0], p.events[r.e0 + 1]) != cudaSuccess) return SC_ERR_CUDA;
        ms[r.cls] += t; launches[r.cls] += 1; bytes[r.cls] += r.bytes; flops[r.cls] += r.flops;
    }
    p.recs.clear(); p.used = 0;
    return SC_OK;
}

int sepconv_kernel_class_count(void) { return KC_COUNT; }
const char* sepconv_kernel_class_name(int c) { return kclass_name(c); }

int sepconv_workspace_bytes(const sc_block_desc* desc, size_t* fwd, size_t* bwd) {
    Dims m;
    SC_TRY(desc_dims(desc, &m));
    if (fwd) { Bump b(nullptr, 0); FwdScratch f; plan_fwd(desc, m, b, &f, nullptr); *fwd = b.off + 256; }
    if (bwd) { Bump b(nullptr, 0); BwdScratch s; plan_bwd(desc, m, b, &s, nullptr); *bwd = b.off + 256; }
    return SC_OK;
}

int sepconv_fwd(sc_ctx* ctx, const sc_block_desc* desc, const sc_tensor* x, const sc_tensor* x_res,
                const int32_t* lengths_dev, const sc_block_params* params, sc_tensor* y,
                int32_t* out_lengths_dev, sc_block_saved* saved, float* running_mean, float* running_var,
                void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!ctx || !lengths_dev) return SC_ERR_NULL;
    Dims m;
    SC_TRY(desc_dims(desc, &m));
    const int dt = desc->io_dtype;
    SC_TRY(check_tensor(x, dt, m.B, m.Cin, m.T));
    SC_TRY(check_tensor(y, dt, m.B, m.Cout, m.Tp));
    if (desc->residual != SC_RES_NONE) {
        if (x_res) SC_TRY(check_tensor(x_res, dt, m.B, m.Cres, m.Tp));
        else if (m.s != 1 || m.Cres != m.Cin) return SC_ERR_UNSUPPORTED;
    }
    SC_TRY(check_params(desc, params));
    SC_TRY(check_saved(desc, saved, false));
    if (!workspace) return SC_ERR_WORKSPACE;
    Bump ws(workspace, workspace_bytes);
    FwdScratch f;
    plan_fwd(desc, m, ws, &f, &ctx->tc);
    if (!ws.ok()) return SC_ERR_WORKSPACE;
    Launch L{(cudaStream_t)cuda_stream, ctx->status_dev, &ctx->launches, &ctx->prof, ctx->gemm_mode, ctx->pdl};
    BlockIO io{};
    io.x = x->ptr; io.xres = desc->residual != SC_RES_NONE ? (x_res ? x_res->ptr : x->ptr) : nullptr;
    io.y = y->ptr; io.len_in = lengths_dev; io.len_out = f.len_out; io.nvalid = f.nvalid; io.blk_off = f.blk_off;
    io.x_clean = false; io.res_clean = false; io.lengths_ready = false;
    SC_TRY(block_fwd_impl(ctx, L, desc, m, io, params, saved, running_mean, running_var, f));
    if (out_lengths_dev)
        cudaMemcpyAsync(out_lengths_dev, f.len_out, sizeof(int) * m.B, cudaMemcpyDeviceToDevice, L.stream);
    return finish(ctx);
}

namespace {
// scratch of the evaluation-mode forward: the training forward's scratch plus the tensors that call would save
struct InferScratch { FwdScratch f; sc_block_saved sv; };
void plan_infer(const sc_block_desc* d, const Dims& m, Bump& ws, InferScratch* q, const TcState* tc) {
    plan_fwd(d, m, ws, &q->f, tc);
    memset(&q->sv, 0, sizeof(q->sv));
    const size_t e = esize(d->io_dtype), en = dtype_size(ntype_of(d->io_dtype));
    q->sv.u = ws.take(e * m.B * m.Cin * m.Tp);
    if (d->has_bn) { q->sv.v = ws.take(en * m.B * m.Cout * m.Tp); q->sv.invstd = (float*)ws.take(4 * m.Cout); }
    if (d->residual == SC_RES_PROJ) { q->sv.vr = ws.take(en * m.B * m.Cout * m.Tp); q->sv.invstd_r = (float*)ws.take(4 * m.Cout); }
}
}  // namespace

int sepconv_infer_workspace_bytes(const sc_block_desc* desc, size_t* bytes) {
    if (!bytes) return SC_ERR_NULL;
    Dims m;
    SC_TRY(desc_dims(desc, &m));
    Bump b(nullptr, 0); InferScratch q; plan_infer(desc, m, b, &q, nullptr);
    *bytes = b.off + 256;
    return SC_OK;
}

int sepconv_infer(sc_ctx* ctx, const sc_block_desc* desc, const sc_tensor* x, const sc_tensor* x_res,
                  const int32_t* lengths_dev, const sc_block_params* params, const float* running_mean,
                  const float* running_var, const float* running_mean_r, const float* running_var_r, sc_tensor* y,
                  int32_t* out_lengths_dev, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!ctx || !lengths_dev) return SC_ERR_NULL;
    Dims m;
    SC_TRY(desc_dims(desc, &m));
    const int dt = desc->io_dtype;
    SC_TRY(check_tensor(x, dt, m.B, m.Cin, m.T));
    SC_TRY(check_tensor(y, dt, m.B, m.Cout, m.Tp));
    if (desc->residual != SC_RES_NONE) {
        if (x_res) SC_TRY(check_tensor(x_res, dt, m.B, m.Cres, m.Tp));
        else if (m.s != 1 || m.Cres != m.Cin) return SC_ERR_UNSUPPORTED;
    }
    SC_TRY(check_params(desc, params));
    if (desc->has_bn && (!running_mean || !running_var)) return SC_ERR_NULL;
    if (desc->residual == SC_RES_PROJ && (!running_mean_r || !running_var_r)) return SC_ERR_NULL;
    if (!workspace) return SC_ERR_WORKSPACE;
    Bump ws(workspace, workspace_bytes);
    InferScratch q;
    plan_infer(desc, m, ws, &q, &ctx->tc);
    if (!ws.ok()) return SC_ERR_WORKSPACE;
    Launch L{(cudaStream_t)cuda_stream, ctx->status_dev, &ctx->launches, &ctx->prof, ctx->gemm_mode, ctx->pdl};
    BlockIO io{};
    io.x = x->ptr; io.xres = desc->residual != SC_RES_NONE ? (x_res ? x_res->ptr : x->ptr) : nullptr;
    io.y = y->ptr; io.len_in = lengths_dev; io.len_out = q.f.len_out; io.nvalid = q.f.nvalid; io.blk_off = q.f.blk_off;
    InferStats inf{running_mean, running_var, running_mean_r, running_var_r};
    SC_TRY(block_fwd_impl(ctx, L, desc, m, io, params, &q.sv, nullptr, nullptr, q.f, &inf));
    if (out_lengths_dev)
        cudaMemcpyAsync(out_lengths_dev, q.f.len_out, sizeof(int) * m.B, cudaMemcpyDeviceToDevice, L.stream);
    return finish(ctx);
}

int sepconv_bwd(sc_ctx* ctx, const sc_block_desc* desc, const sc_tensor* dy, const sc_tensor* x,
                const sc_tensor* x_res, const sc_tensor* y, const int32_t* lengths_dev,
                const sc_block_params* params, const sc_block_saved* saved, sc_tensor* dx,
                sc_tensor* dx_res, const sc_tensor* dx_add, sc_block_grads* grads, int accumulate,
                void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!ctx || !lengths_dev) return SC_ERR_NULL;
    Dims m;
    SC_TRY(desc_dims(desc, &m));
    const int dt = desc->io_dtype;
    SC_TRY(check_tensor(dy, dt, m.B, m.Cout, m.Tp));
    SC_TRY(check_tensor(x, dt, m.B, m.Cin, m.T));
    SC_TRY(check_tensor(y, dt, m.B, m.Cout, m.Tp));
    SC_TRY(check_tensor(dx, dt, m.B, m.Cin, m.T));
    if (dx_add) SC_TRY(check_tensor(dx_add, dt, m.B, m.Cin, m.T));
    if (desc->residual != SC_RES_NONE) {
        if (x_res) SC_TRY(check_tensor(x_res, dt, m.B, m.Cres, m.Tp));
        else if (m.s != 1 || m.Cres != m.Cin) return SC_ERR_UNSUPPORTED;
        if (dx_res) SC_TRY(check_tensor(dx_res, dt, m.B, m.Cres, m.Tp));
        else if (m.s != 1 || m.Cres != m.Cin) return SC_ERR_UNSUPPORTED;
        // folding the residual path's gradient into dx is only meaningful when the residual source is x itself
        else if (x_res && x_res->ptr != x->ptr) return SC_ERR_UNSUPPORTED;
    }
    SC_TRY(check_params(desc, params));
    SC_TRY(check_saved(desc, saved, false));
    SC_TRY(check_grads(desc, grads));
    if (!workspace) return SC_ERR_WORKSPACE;
    Bump ws(workspace, workspace_bytes);
    BwdScratch s;
    plan_bwd(desc, m, ws, &s, &ctx->tc);
    if (!ws.ok()) return SC_ERR_WORKSPACE;
    Launch L{(cudaStream_t)cuda_stream, ctx->status_dev, &ctx->launches, &ctx->prof, ctx->gemm_mode, ctx->pdl};
    lengths(L, lengths_dev, m.B, m.T, m.s, s.len_out, s.nvalid, s.blk_off);
    BwdIO io{};
    io.dy = dy->ptr; io.x = x->ptr; io.y = y->ptr;
    io.xres = desc->residual != SC_RES_NONE ? (x_res ? x_res->ptr : x->ptr) : nullptr;
    io.dx = dx->ptr; io.dx_res = (desc->residual != SC_RES_NONE && dx_res) ? dx_res->ptr : nullptr;
    io.dx_add = dx_add ? dx_add->ptr : nullptr;
    io.len_in = lengths_dev; io.len_out = s.len_out; io.nvalid = s.nvalid; io.blk_off = s.blk_off;
    io.x_clean = false; io.res_clean = false;
    io.done = ctx->ev[2];
    SC_TRY(block_bwd_impl(ctx, L, desc, m, io, params, saved, grads, accumulate, s));
    wait_side(ctx, L, ctx->ev[2]);
    return finish(ctx);
}

// ---- encoder ---------------------------------------------------------------------------------
namespace {
struct LayerPlan {
    sc_block_desc d; Dims m;
    sc_block_saved sv; void* y; int* len_out; int* nvalid; int* blk_off; void* w16;
    bool own_lengths;
};
// Backward layer i works in scratch region i % kScratchRegions: its weight-gradient kernels (side stream) may still
// read their operands while the next layers already write their own, and the main stream waits for them only when it
// comes back to the region, kScratchRegions layers later.  (Three regions measured slower than two: weight gradients
// that may lag two layers behind take SMs from the critical path more often than the wait costs.)
constexpr int kScratchRegions = 2;
struct EncPlan {
    std::vector<LayerPlan> L;
    void* gbuf[2];
    std::vector<void*> pend;       // per layer: where the residual gradients for that layer's input collect (or null)
    void* pend_tmp;                // a second residual gradient for a source that already holds one lands here first
    float* gmax_all;               // one |gv| bound per layer, zeroed by one memset at the start of the call
    size_t bytes;
    size_t scratch_mark;           // offset where the shared per-layer scratch starts
    size_t scratch_size;           // its size; kScratchRegions regions of that size in all (backward layers rotate)
};

int plan_encoder(const sc_encoder_desc* e, void* base, size_t cap, EncPlan* P, const TcState* tc) {
    if (!e || !e->layers || e->n_layers < 1) return SC_ERR_NULL;
    Bump ws(base, cap);
    P->L.resize(e->n_layers);
    int B = e->layers[0].B, T = e->layers[0].T_in, C = e->layers[0].C_in;
    size_t max_act = 0, max_res = 0;
    // Residual spans [source, layer]: the residual path's gradient waits in a pending buffer from the backward step of
    // `layer` down to that of `source`.  Spans that do not overlap share a buffer (the five blocks of the QuartzNet
    // encoder use one); spans that overlap or nest get buffers of their own; several layers may share a source (their
    // gradients are summed in the source's buffer).
    const int nl = e->n_layers;
    std::vector<int> last_user(nl, -1), users(nl, 0);
    std::vector<size_t> res_bytes(nl, 0);
    for (int i = 0; i < nl; ++i) {
        if (e->layers[i].residual == SC_RES_NONE || !e->res_from || e->res_from[i] < 0 || e->res_from[i] == i) continue;
        if (e->res_from[i] > i) return SC_ERR_UNSUPPORTED;
        last_user[e->res_from[i]] = i; ++users[e->res_from[i]];
    }
    for (int i = 0; i < e->n_layers; ++i) {
        LayerPlan& lp = P->L[i];
        lp.d = e->layers[i];
        lp.d.B = B; lp.d.T_in = T;
        if (lp.d.C_in != C) return SC_ERR_DIM_INCOMPATIBLE;
        if (lp.d.io_dtype != e->layers[0].io_dtype) return SC_ERR_INCOMPATIBLE;
        if (lp.d.residual != SC_RES_NONE) {
            int j = e->res_from ? e->res_from[i] : -1;
            if (j < 0) j = i;
            if (j > i) return SC_ERR_UNSUPPORTED;
            lp.d.C_res = e->layers[j].C_in;
        }
        SC_TRY(desc_dims(&lp.d, &lp.m));
        const Dims& m = lp.m;
        const size_t es = esize(lp.d.io_dtype);
        if (lp.d.residual != SC_RES_NONE) {
            int j = (e->res_from && e->res_from[i] >= 0) ? e->res_from[i] : i;
            if (P->L[j].m.T != m.Tp) return SC_ERR_UNSUPPORTED;
            max_res = std::max(max_res, es * m.B * m.Cres * m.Tp);
            if (j != i) res_bytes[j] = es * m.B * m.Cres * m.Tp;
        }
        lp.own_lengths = (i == 0) || (m.s != 1);
        if (lp.own_lengths) {
            lp.len_out = (int*)ws.take(sizeof(int) * B); lp.nvalid = (int*)ws.take(sizeof(int));
            lp.blk_off = (int*)ws.take(sizeof(int) * (B + 1));
        } else { lp.len_out = P->L[i - 1].len_out; lp.nvalid = P->L[i - 1].nvalid; lp.blk_off = P->L[i - 1].blk_off; }
        memset(&lp.sv, 0, sizeof(lp.sv));
        if (lp.d.has_dw) lp.sv.u = ws.take(es * B * m.Cin * m.Tp);
        else if (i == 0) lp.sv.u = ws.take(es * B * m.Cin * m.Tp);
        if (lp.d.has_bn) {
            lp.sv.v = ws.take(dtype_size(ntype_of(lp.d.io_dtype)) * B * m.Cout * m.Tp);
            lp.sv.mean = (float*)ws.take(4 * m.Cout); lp.sv.invstd = (float*)ws.take(4 * m.Cout);
        }
        if (lp.d.residual == SC_RES_PROJ) {
            lp.sv.vr = ws.take(dtype_size(ntype_of(lp.d.io_dtype)) * B * m.Cout * m.Tp);
            lp.sv.mean_r = (float*)ws.take(4 * m.Cout); lp.sv.invstd_r = (float*)ws.take(4 * m.Cout);
        }
        lp.y = (i + 1 < e->n_layers) ? ws.take(es * B * m.Cout * m.Tp) : nullptr;
        lp.w16 = (op_dtype(&lp.d) != lp.d.io_dtype) ? ws.take((size_t)2 * m.Cout * m.Cin) : nullptr;
        max_act = std::max(max_act, es * B * (size_t)m.Cin * m.T);
        max_act = std::max(max_act, es * B * (size_t)m.Cout * m.Tp);
        C = m.Cout; T = m.Tp;
    }
    // shared scratch: plan every layer from the same offset and keep the maximum
    const size_t mark = ws.off;
    size_t hi = mark;
    for (int i = 0; i < e->n_layers; ++i) {
        Bump b(base, cap); b.off = mark; FwdScratch f; plan_fwd(&P->L[i].d, P->L[i].m, b, &f, tc); hi = std::max(hi, b.off);
        Bump c(base, cap); c.off = mark; BwdScratch s; plan_bwd(&P->L[i].d, P->L[i].m, c, &s, tc); hi = std::max(hi, c.off);
    }
    hi = (hi + 255) & ~(size_t)255;
    ws.off = hi + (size_t)(kScratchRegions - 1) * (hi - mark);
    P->scratch_size = hi - mark;
    P->gbuf[0] = ws.take(max_act); P->gbuf[1] = ws.take(max_act);
    {
        // interval colouring in source order: a buffer whose span ended strictly before this source is free again
        struct Buf { int end; size_t bytes; };
        std::vector<Buf> bufs;
        std::vector<int> colour(nl, -1);
        bool need_tmp = false;
        for (int j = 0; j < nl; ++j) {
            if (last_user[j] < 0) continue;
            if (users[j] > 1) need_tmp = true;
            int c = -1;
            for (size_t q = 0; q < bufs.size(); ++q) if (bufs[q].end < j) { c = (int)q; break; }
            if (c < 0) { bufs.push_back(Buf{0, 0}); c = (int)bufs.size() - 1; }
            bufs[c].end = last_user[j]; bufs[c].bytes = std::max(bufs[c].bytes, res_bytes[j]);
            colour[j] = c;
        }
        std::vector<void*> addr(bufs.size(), nullptr);
        for (size_t q = 0; q < bufs.size(); ++q) addr[q] = ws.take(bufs[q].bytes);
        P->pend.assign(nl, nullptr);
        for (int j = 0; j < nl; ++j) if (colour[j] >= 0) P->pend[j] = addr[colour[j]];
        P->pend_tmp = need_tmp ? ws.take(max_res) : nullptr;
    }
    P->gmax_all = (float*)ws.take(sizeof(float) * e->n_layers);
    P->bytes = ws.off + 256;
    if (!ws.ok()) return SC_ERR_WORKSPACE;
    P->scratch_mark = mark;
    return SC_OK;
}

sc_block_params layer_params(const void* blob, const int64_t* off) {
    auto at = [&](int j) -> const void* { return off[j] < 0 ? nullptr : (const char*)blob + off[j]; };
    sc_block_params p;
    p.wd = at(0); p.wp = at(1); p.gamma = (const float*)at(2); p.beta = (const float*)at(3);
    p.bias = (const float*)at(4); p.wr = at(5); p.gamma_r = (const float*)at(6); p.beta_r = (const float*)at(7);
    return p;
}
sc_block_grads layer_grads(void* blob, const int64_t* off) {
    auto at = [&](int j) -> float* { return off[j] < 0 ? nullptr : (float*)((char*)blob + off[j]); };
    sc_block_grads g;
    g.dwd = at(0); g.dwp = at(1); g.dgamma = at(2); g.dbeta = at(3); g.dbias = at(4);
    g.dwr = at(5); g.dgamma_r = at(6); g.dbeta_r = at(7);
    return g;
}
}  // namespace

int encoder_workspace_bytes(const sc_encoder_desc* desc, size_t* bytes) {
    if (!bytes) return SC_ERR_NULL;
    EncPlan P;
    SC_TRY(plan_encoder(desc, nullptr, 0, &P, nullptr));
    *bytes = P.bytes;
    return SC_OK;
}

int encoder_infer_workspace_bytes(const sc_encoder_desc* desc, size_t* bytes) {
    return encoder_workspace_bytes(desc, bytes);      // the same plan: per-layer buffers double as scratch
}

int encoder_infer(sc_ctx* ctx, const sc_encoder_desc* e, const sc_tensor* x, const int32_t* lengths_dev,
                  const void* params_blob, const int64_t* param_offsets, const void* running_blob,
                  const int64_t* running_offsets, sc_tensor* out, int32_t* out_lengths_dev, void* workspace,
                  size_t workspace_bytes, void* cuda_stream) {
    if (!ctx || !lengths_dev || !params_blob || !param_offsets || !running_blob || !running_offsets) return SC_ERR_NULL;
    if (!workspace) return SC_ERR_WORKSPACE;
    EncPlan P;
    SC_TRY(plan_encoder(e, workspace, workspace_bytes, &P, &ctx->tc));
    const int n = e->n_layers;
    const Dims& m0 = P.L[0].m; const Dims& ml = P.L[n - 1].m;
    const int dt = P.L[0].d.io_dtype;
    SC_TRY(check_tensor(x, dt, m0.B, m0.Cin, m0.T));
    SC_TRY(check_tensor(out, dt, ml.B, ml.Cout, ml.Tp));
    Launch L{(cudaStream_t)cuda_stream, ctx->status_dev, &ctx->launches, &ctx->prof, ctx->gemm_mode, ctx->pdl};
    auto input_of = [&](int i) -> const void* { return i == 0 ? x->ptr : P.L[i - 1].y; };
    auto res_src = [&](int i) -> int { return (e->res_from && e->res_from[i] >= 0) ? e->res_from[i] : i; };
    auto stat = [&](int i, int j) -> const float* {
        const int64_t o = running_offsets[4 * i + j];
        return o < 0 ? nullptr : (const float*)((const char*)running_blob + o);
    };
    for (int i = 0; i < n; ++i) {
        LayerPlan& lp = P.L[i];
        sc_block_params prm = layer_params(params_blob, param_offsets + 8 * i);
        SC_TRY(check_params(&lp.d, &prm));
        InferStats inf{stat(i, 0), stat(i, 1), stat(i, 2), stat(i, 3)};
        if (lp.d.has_bn && (!inf.mean || !inf.var)) return SC_ERR_NULL;
        if (lp.d.residual == SC_RES_PROJ && (!inf.mean_r || !inf.var_r)) return SC_ERR_NULL;
        Bump b(workspace, workspace_bytes); b.off = P.scratch_mark;
        FwdScratch f; plan_fwd(&lp.d, lp.m, b, &f, &ctx->tc);
        BlockIO io{};
        io.x = input_of(i);
        io.xres = lp.d.residual != SC_RES_NONE ? input_of(res_src(i)) : nullptr;
        io.y = (i + 1 < n) ? lp.y : out->ptr;
        io.len_in = i == 0 ? lengths_dev : P.L[i - 1].len_out; io.len_out = lp.len_out; io.nvalid = lp.nvalid; io.blk_off = lp.blk_off;
        io.x_clean = i > 0; io.res_clean = lp.d.residual != SC_RES_NONE && res_src(i) > 0;
        io.lengths_ready = !lp.own_lengths;
        io.w16_keep = lp.w16; io.w16_ready = false;
        SC_TRY(block_fwd_impl(ctx, L, &lp.d, lp.m, io, &prm, &lp.sv, nullptr, nullptr, f, &inf));
    }
    if (out_lengths_dev)
        cudaMemcpyAsync(out_lengths_dev, P.L[n - 1].len_out, sizeof(int) * m0.B, cudaMemcpyDeviceToDevice, L.stream);
    return finish(ctx);
}

int encoder_fwd_bwd(sc_ctx* ctx, const sc_encoder_desc* e, const sc_tensor* x, const int32_t* lengths_dev,
                    const void* params_blob, const int64_t* param_offsets, const sc_tensor* dlogits,
                    sc_tensor* logits, int32_t* out_lengths_dev, void* grads_blob,
                    const int64_t* grad_offsets, sc_tensor* dx, int accumulate, void* workspace,
                    size_t workspace_bytes, void* cuda_stream) {
    if (!ctx || !lengths_dev || !params_blob || !param_offsets || !grads_blob || !grad_offsets) return SC_ERR_NULL;
    if (!workspace) return SC_ERR_WORKSPACE;
    EncPlan P;
    SC_TRY(plan_encoder(e, workspace, workspace_bytes, &P, &ctx->tc));
    const int n = e->n_layers;
    const size_t mark = P.scratch_mark;
    const Dims& m0 = P.L[0].m; const Dims& ml = P.L[n - 1].m;
    const int dt = P.L[0].d.io_dtype;
    SC_TRY(check_tensor(x, dt, m0.B, m0.Cin, m0.T));
    SC_TRY(check_tensor(logits, dt, ml.B, ml.Cout, ml.Tp));
    SC_TRY(check_tensor(dlogits, dt, ml.B, ml.Cout, ml.Tp));
    if (dx) SC_TRY(check_tensor(dx, dt, m0.B, m0.Cin, m0.T));
    std::vector<sc_block_params> prm(n);
    std::vector<sc_block_grads> grd(n);
    for (int i = 0; i < n; ++i) {
        prm[i] = layer_params(params_blob, param_offsets + 8 * i);
        grd[i] = layer_grads(grads_blob, grad_offsets + 8 * i);
        SC_TRY(check_params(&P.L[i].d, &prm[i]));
        SC_TRY(check_grads(&P.L[i].d, &grd[i]));
    }
    Launch L{(cudaStream_t)cuda_stream, ctx->status_dev, &ctx->launches, &ctx->prof, ctx->gemm_mode, ctx->pdl};
    auto input_of = [&](int i) -> const void* { return i == 0 ? x->ptr : P.L[i - 1].y; };
    auto len_in_of = [&](int i) -> const int* { return i == 0 ? lengths_dev : P.L[i - 1].len_out; };
    auto res_src = [&](int i) -> int { return (e->res_from && e->res_from[i] >= 0) ? e->res_from[i] : i; };

    cudaMemsetAsync(P.gmax_all, 0, sizeof(float) * n, L.stream);
    // float16 copies of the pointwise weights of every layer that needs one: one launch
    {
        ConvertList cl; cl.count = 0;
        for (int i = 0; i < n; ++i) {
            if (!P.L[i].w16) continue;
            if (cl.count == 48) { convert_bf16_to_f16_many(L, cl); cl.count = 0; }
            cl.src[cl.count] = prm[i].wp; cl.dst[cl.count] = P.L[i].w16; cl.n[cl.count] = P.L[i].m.Cout * P.L[i].m.Cin;
            ++cl.count;
        }
        convert_bf16_to_f16_many(L, cl);
    }
    // forward
    for (int i = 0; i < n; ++i) {
        LayerPlan& lp = P.L[i];
        Bump b(workspace, workspace_bytes); b.off = mark;
        FwdScratch f; plan_fwd(&lp.d, lp.m, b, &f, &ctx->tc);
        BlockIO io{};
        io.x = input_of(i);
        io.xres = lp.d.residual != SC_RES_NONE ? input_of(res_src(i)) : nullptr;
        io.y = (i + 1 < n) ? lp.y : logits->ptr;
        io.len_in = len_in_of(i); io.len_out = lp.len_out; io.nvalid = lp.nvalid; io.blk_off = lp.blk_off;
        io.x_clean = i > 0; io.res_clean = lp.d.residual != SC_RES_NONE && res_src(i) > 0;
        io.lengths_ready = !lp.own_lengths;
        io.w16_keep = lp.w16; io.w16_ready = true;
        SC_TRY(block_fwd_impl(ctx, L, &lp.d, lp.m, io, &prm[i], &lp.sv, nullptr, nullptr, f));
    }
    if (out_lengths_dev)
        cudaMemcpyAsync(out_lengths_dev, P.L[n - 1].len_out, sizeof(int) * m0.B, cudaMemcpyDeviceToDevice, L.stream);

    // backward
    const void* g = dlogits->ptr;
    std::vector<char> has_pending(n, 0);
    bool side_busy[kScratchRegions] = {};
    cudaEvent_t done_ev[3] = {ctx->ev[2], ctx->ev[3], ctx->ev[6]};
    for (int i = n - 1; i >= 0; --i) {
        LayerPlan& lp = P.L[i];
        // this layer reuses the scratch region of layer i + kScratchRegions: that layer's side-stream kernels must be done
        const int region = i % kScratchRegions;
        if (side_busy[region]) wait_side(ctx, L, done_ev[region]);
        Bump b(workspace, workspace_bytes); b.off = mark + (size_t)region * P.scratch_size;
        BwdScratch s; plan_bwd(&lp.d, lp.m, b, &s, &ctx->tc);
        BwdIO io{};
        io.done = done_ev[region]; side_busy[region] = true;
        io.dy = g; io.x = input_of(i); io.y = (i + 1 < n) ? lp.y : logits->ptr;
        io.xres = lp.d.residual != SC_RES_NONE ? input_of(res_src(i)) : nullptr;
        io.dx = (i == 0) ? (dx ? dx->ptr : nullptr) : P.gbuf[i & 1];
        io.dx_res = nullptr;
        const int src = res_src(i);
        const bool to_pending = lp.d.residual != SC_RES_NONE && src != i;
        const bool second = to_pending && has_pending[src];       // the source's buffer already holds a gradient
        if (to_pending) { io.dx_res = second ? P.pend_tmp : P.pend[src]; has_pending[src] = 1; }
        io.dx_add = has_pending[i] ? P.pend[i] : nullptr;
        io.len_in = len_in_of(i); io.len_out = lp.len_out; io.nvalid = lp.nvalid; io.blk_off = lp.blk_off;
        io.x_clean = i > 0; io.res_clean = lp.d.residual != SC_RES_NONE && res_src(i) > 0;
        io.w16_kept = lp.w16;
        io.gmax_zeroed = P.gmax_all + i;
        SC_TRY(block_bwd_impl(ctx, L, &lp.d, lp.m, io, &prm[i], &lp.sv, &grd[i], accumulate, s));
        if (second)
            ew_add_masked(L, dt, P.pend[src], P.pend[src], P.pend_tmp, nullptr, len_in_of(src), P.L[src].m.B, P.L[src].m.Cin, P.L[src].m.T);
        g = io.dx;
    }
    for (int q = 0; q < kScratchRegions; ++q) if (side_busy[q]) wait_side(ctx, L, done_ev[q]);     // join before returning
    return finish(ctx);
}

}  // extern "C"
