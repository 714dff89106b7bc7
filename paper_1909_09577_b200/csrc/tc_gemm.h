// Tensor-core (tcgen05 + TMEM + TMA) pointwise contractions for 16-bit activations.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include "kernels.h"

namespace sc {

struct TcState {
    void* encode_fn = nullptr;   // cuTensorMapEncodeTiled, resolved through the runtime
    int sm_count = 0;
    bool ready = false;
    bool persistent = true;      // forward / input gradient: persistent warp-specialised kernel
};

int tc_init(TcState* st, int device, int sm_count);

// Encodes a tiled tensor map (128-byte swizzle, zero fill outside the tensor) for a dense 16-bit tensor
// whose dimensions, innermost first, are dims[0..rank-1]; map_out points to a CUtensorMap.
bool tc_make_map(const TcState* st, void* map_out, int dtype, const void* base, int rank, const uint64_t* dims,
                 const uint32_t* box);

// Upper bound on statistics partials per sample that the fused epilogue may emit.
int tc_max_parts_per_sample(int Tp);

bool tc_fwd_supported(const TcState* st, int dtype, int Cin, int Cout, int Tp);
bool tc_dgrad_supported(const TcState* st, int dtype, int Cin, int Cout, int Tp);
bool tc_wgrad_supported(const TcState* st, int dtype, int Cin, int Cout, int Tp);
size_t tc_wgrad_scratch_bytes(const TcState* st, int Cin, int Cout);

// v[b,o,t] = [t < len_out[b]] * (sum_c w[o,c] u[b,c,t] + bias[o]), stored in out_dtype.  When `partials` is non-null the
// epilogue also writes per-(sample, time-tile, channel) (sum, M2) over valid frames, computed from the
// fp32 accumulators, and reports the tiling through parts_per_b / tile_w; returns true if it did.
bool tc_gemm_fwd(const TcState* st, const Launch& L, int dtype, const void* w, const void* u, const float* bias,
                 void* v, int out_dtype, const int* len_out, int B, int Cin, int Cout, int Tp, float2* partials,
                 int* parts_per_b, int* tile_w);
// gu[b,c,t] = sum_o w[o,c] gv[b,o,t]
void tc_gemm_dgrad(const TcState* st, const Launch& L, int dtype, const void* w, const void* gv, void* gu, int B,
                   int Cin, int Cout, int Tp, const int* len_out);
// dw[o,c] (+)= sum_{b,t} gv[b,o,t] u[b,c,t]
void tc_gemm_wgrad(const TcState* st, const Launch& L, int dtype, const void* gv, const void* u, float* dw,
                   float* partials, int accumulate, int B, int Cin, int Cout, int Tp, const int* len_out,
                   const float* gmax = nullptr);

}  // namespace sc
