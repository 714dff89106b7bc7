// Tensor-core (tcgen05 + TMEM + TMA) pointwise contractions for 16-bit activations.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include "kernels.h"

namespace sc {

struct TcMapCache;
struct TcState {
    void* encode_fn = nullptr;   // cuTensorMapEncodeTiled, resolved through the runtime
    TcMapCache* map_cache = nullptr;   // encoded tensor maps of this context (tc_make_map); calls on one context are not concurrent
    int sm_count = 0;
    bool ready = false;
    bool persistent = true;      // forward / input gradient: persistent warp-specialised kernel
    bool flat = true;            // ... over the flattened list of valid 64-frame blocks (needs blk_off)
    int flat_shape = 0;          // tile shape of that kernel: 0 = 256 x 256 (one accumulator), 1 = 256 x 128 and
                                 // 2 = 128 x 256 (two accumulators: the epilogue overlaps the next tile's MMAs)
};

int tc_init(TcState* st, int device, int sm_count);
void tc_destroy(TcState* st);

// Encodes a tiled tensor map (128-byte swizzle by default, 64-byte with swizzle_bytes = 64; zero fill outside the
// tensor) for a dense 16-bit tensor whose dimensions, innermost first, are dims[0..rank-1]; map_out points to a
// CUtensorMap.
bool tc_make_map(const TcState* st, void* map_out, int dtype, const void* base, int rank, const uint64_t* dims,
                 const uint32_t* box, int swizzle_bytes = 128);

// Upper bound on statistics partials per sample that the fused epilogue may emit.
int tc_max_parts_per_sample(int Tp);
// Bytes of statistics scratch the forward contraction may need for C_out channels (either partial layout).
size_t tc_stats_bytes(int B, int Cout, int Tp);

// How the forward contraction left its batch-norm partial statistics.
//   kind 0: none (the caller computes them from the stored result)
//   kind 1: float2 (sum, M2) per (sample, time tile, channel): parts_per_b tiles of tile_w frames per sample
//   kind 2: float4 (count, sum, M2, -) per (CTA, channel) of the flattened-block kernel: `grid` CTAs,
//           tiles_m M tiles of rows_per_tile channels; CTA c took the units [c U / grid, (c+1) U / grid) of the
//           U = tiles_m * (number of valid 64-frame blocks) units, M tile major
struct StatsLayout { int kind = 0, parts_per_b = 1, tile_w = 0, grid = 0, tiles_m = 0, rows_per_tile = 0; };

bool tc_fwd_supported(const TcState* st, int dtype, int Cin, int Cout, int Tp);
bool tc_dgrad_supported(const TcState* st, int dtype, int Cin, int Cout, int Tp);
bool tc_wgrad_supported(const TcState* st, int dtype, int Cin, int Cout, int Tp);
size_t tc_wgrad_scratch_bytes(const TcState* st, int Cin, int Cout);

// v[b,o,t] = [t < len_out[b]] * (sum_c w[o,c] u[b,c,t] + bias[o]), stored in out_dtype.  When `partials` is non-null the
// epilogue also writes per-(sample, time-tile, channel) (sum, M2) over valid frames, computed from the
// fp32 accumulators, and reports the tiling through parts_per_b / tile_w; returns true if it did.
// blk_off (int [B+1], exclusive prefix of ceil(len_out[b]/64), from lengths()) selects the flattened-block
// kernel when it is given and B is small enough for its shared-memory copy.
void tc_gemm_fwd(const TcState* st, const Launch& L, int dtype, const void* w, const void* u, const float* bias,
                 void* v, int out_dtype, const int* len_out, const int* blk_off, int B, int Cin, int Cout, int Tp,
                 void* partials, StatsLayout* layout);
// gu[b,c,t] = sum_o w[o,c] gv[b,o,t]
void tc_gemm_dgrad(const TcState* st, const Launch& L, int dtype, const void* w, const void* gv, void* gu, int B,
                   int Cin, int Cout, int Tp, const int* len_out, const int* blk_off);
// dw[o,c] (+)= sum_{b,t} gv[b,o,t] u[b,c,t]
void tc_gemm_wgrad(const TcState* st, const Launch& L, int dtype, const void* gv, const void* u, float* dw,
                   float* partials, int accumulate, int B, int Cin, int Cout, int Tp, const int* len_out,
                   const float* gmax = nullptr);

}  // namespace sc
