// Internal declarations shared by the translation units of libhgf_b200.so (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/hgf.h"

#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ < 1000)
#error "libhgf_b200 is written for sm_100a only"
#endif

namespace hgf {

// ---- launch accounting and the device-side status word ------------------------------------
void count_launch(int n = 1);
unsigned int *device_status_word();  // per-device word in global memory; nonzero = a wait gave up

// ---- workspace layout (all sections 256-byte aligned) --------------------------------------
//   xq       [M][d_in]   int8     quantised activations
//   gamma_x  [M]         float    per-token scales (floored at 1e-5)
//   row_sum  [M]         int32    sum_k xq[m][k]  (the packed codes are t + 1, so
//                                 sum_k t*xq = sum_k c*xq - row_sum)
//   h        [M][r]      float    SiLU(x A)
//   h16      [M][64]     half     the same, fp16 and zero-padded to 64 columns (GEMM path only)
struct WsLayout {
    size_t xq, gamma_x, row_sum, h, h16, total;
};

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static inline WsLayout ws_layout(int64_t M, int64_t d_in, int32_t r, bool gemm_path) {
    WsLayout L;
    size_t off = 0;
    L.xq = off;      off += align_up((size_t)M * (size_t)d_in, 256);
    L.gamma_x = off; off += align_up((size_t)M * 4, 256);
    L.row_sum = off; off += align_up((size_t)M * 4, 256);
    L.h = off;       off += align_up((size_t)M * (size_t)(r > 0 ? r : 1) * 4, 256);
    L.h16 = off;     off += gemm_path ? align_up((size_t)M * 64 * 2, 256) : 0;
    L.total = off ? off : 256;
    return L;
}

// ---- kernel parameter blocks ----------------------------------------------------------------
struct PrologueParams {
    const __nv_bfloat16 *x;  // [M][K]
    const __half *At;        // [r][K], nullable when r == 0
    int8_t *xq;              // [M][K]
    float *gamma_x;          // [M]
    int32_t *row_sum;        // [M], nullable
    float *h;                // [M][r]
    __half *h16;             // [M][64] or null
    int8_t *dbg_xq;          // nullable debug copies
    float *dbg_gamma_x;
    float *dbg_h;
    int M, K, r;
    uint32_t flags;
};

// One layer problem of a decode launch (M <= 16).  tile_begin = index of its first 16-row tile in
// the launch-wide tile numbering.
struct DecodeProblem {
    const uint8_t *packed;   // [N][K/4]
    const int8_t *xq;        // [M][K]
    const float *gamma_x;    // [M]
    const int32_t *row_sum;  // [M]
    const float *h;          // [M][r]
    const __half *Bt;        // [N][r]
    const float *gate;       // [N]
    void *y;                 // [M][N] fp32 or bf16
    int32_t *dbg_y_int;      // nullable
    float gw_over_127;       // gamma_W / 127
    int M, K, N, r;
    uint32_t flags;
    int tile_begin;
};

struct DecodeLaunch {
    const DecodeProblem *probs;  // device array, or null for a single problem passed by value
    int n_probs;
    int total_tiles;
    int S;                       // K slices per row tile (chosen by the launcher)
};

// host-side launchers (each enqueues on `stream` and returns the CUDA error of the launch)
cudaError_t launch_quant(const PrologueParams &p, cudaStream_t stream);
cudaError_t launch_decode_prologue(const PrologueParams &p, bool pdl, cudaStream_t stream);
cudaError_t launch_decode_prologue_group(const PrologueParams *d_pps, const int *d_blk_begin, int n, int total_blocks,
                                         bool pdl, cudaStream_t stream);
cudaError_t launch_lora_down_gemm(const PrologueParams &p, cudaStream_t stream);
cudaError_t launch_decode_gemv(const DecodeLaunch &L, const DecodeProblem *single, int max_M, int min_steps, bool pdl,
                               cudaStream_t stream);

struct GemmParams {
    const int8_t *xq;        // [M][K]
    const uint8_t *packed;   // [N][K/4]
    const float *gamma_x;    // [M]
    const int32_t *row_sum;  // [M]
    const __half *h16;       // [M][64]
    const __half *Bt;        // [N][r]
    const float *gate;       // [N]
    void *y;                 // [M][N]
    int32_t *dbg_y_int;
    float gw_over_127;
    int M, K, N, r;
    uint32_t flags;
};
// Returns cudaSuccess or an error; *status distinguishes tensor-map failures.
cudaError_t launch_prefill_gemm(const GemmParams &p, cudaStream_t stream);

// ---- small device helpers ---------------------------------------------------------------------
__device__ __forceinline__ float bf16lo_to_float(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_to_float(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float silu_f(float z) { return z / (1.0f + expf(-z)); }

}  // namespace hgf
