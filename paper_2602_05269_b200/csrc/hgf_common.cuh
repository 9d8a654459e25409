// Internal declarations shared by the translation units of libhgf_b200.so (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>

#include <atomic>

#include "../../include/hgf.h"

#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ < 1000)
#error "libhgf_b200 is written for sm_100a only"
#endif

namespace hgf {

// ---- launch accounting and the device-side status word ------------------------------------
void count_launch(int n = 1);
unsigned int *device_status_word();  // per-device word in global memory; nonzero = a wait gave up

// ---- per-device launch set-up -----------------------------------------------------------------
// A process may drive several GPUs: the SM count and the opt-in to large dynamic shared memory
// (an attribute of the kernel on ONE device) are looked up for the device that is current.
constexpr int kMaxDevices = 64;
int current_device();      // ordinal of the current device, or -1
int device_sm_count();     // SM count of the current device (cached per device), 0 if it cannot be queried
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per device; `done` is a per-kernel bit mask
// of the devices already set up (one static instance beside each kernel's launcher).
template <typename Kernel>
static inline cudaError_t ensure_dynamic_smem(Kernel kernel, int bytes, std::atomic<unsigned long long> &done) {
    const int dev = current_device();
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    const unsigned long long bit = 1ull << dev;
    if (done.load(std::memory_order_acquire) & bit) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    done.fetch_or(bit, std::memory_order_release);
    return cudaSuccess;
}

// ---- packed weight layout ---------------------------------------------------------------------
// Tiles of 16 output rows x 256 input columns, 1 KiB each, row-major inside the tile (64 bytes per
// row), tiles ordered with the column-tile index fastest.  d_in is padded to a multiple of 256 and
// d_out to a multiple of 16 with code 1 (weight 0).
static inline int64_t padded_k(int64_t d_in) { return (d_in + 255) / 256 * 256; }
static inline int64_t row_tiles(int64_t d_out) { return (d_out + 15) / 16; }
// Base-3 layout (five codes per byte): tiles of 16 output rows x 320 input columns, also 1 KiB each.
static inline int64_t padded_k_b3(int64_t d_in) { return (d_in + 319) / 320 * 320; }

// ---- workspace layout (all sections 256-byte aligned) --------------------------------------
//   xq       [M][d_in]   int8     quantised activations
//   gamma_x  [M]         float    per-token scales (floored at 1e-5)
//   row_sum  [M]         int32    sum_k xq[m][k]  (the packed codes are t + 1, so
//                                 sum_k t*xq = sum_k c*xq - row_sum)
//   h        [M][r]      float    SiLU(x A)
//   h_hi     [M][r]      half     fp16 rounding of h          (decode path only)
//   h_lo     [M][r]      half     fp16 rounding of h - h_hi   (decode path only)
//   hpart    [r/16][slices][8][32] float  partial sums of x A per K slice (decode path only; see LoraItem)
//   h16      [M][64]     half     h in fp16, zero-padded to 64 columns (GEMM path only)
//   tok_sc   [M]         float    gamma_x[m] * gamma_W / 127 (GEMM path only)
//   gb16     [N][64]     half     gate[n] * B[j][n], zero-padded to 64 columns (GEMM path only)
// On the GEMM path the per-token arrays have room for M rounded up to 128: the kernel fetches them
// 128 tokens at a time (what lies past M is never used).
struct WsLayout {
    size_t xq, gamma_x, row_sum, h, h_hi, h_lo, hpart, h16, tok_sc, gb16, w2, total;
};

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static inline WsLayout ws_layout(int64_t M, int64_t d_in, int64_t d_out, int32_t r, bool gemm_path, bool base3 = false) {
    WsLayout L;
    size_t off = 0;
    const size_t rr = (size_t)(r > 0 ? r : 1);
    L.xq = off;      off += align_up((size_t)M * (size_t)d_in, 256);
    L.gamma_x = off; off += align_up((size_t)M * 4, 256);
    const size_t Mp = gemm_path ? align_up((size_t)M, 128) : (size_t)M;
    L.row_sum = off; off += align_up(Mp * 4, 256);
    L.h = off;       off += align_up((size_t)M * rr * 4, 256);
    L.h_hi = off;    off += gemm_path ? 0 : align_up((size_t)M * rr * 2, 256);
    L.h_lo = off;    off += gemm_path ? 0 : align_up((size_t)M * rr * 2, 256);
    L.hpart = off;   off += (gemm_path || r <= 0) ? 0 : (size_t)(r / 16) * (size_t)((d_in + 255) / 256) * 1024;
    L.h16 = off;     off += gemm_path ? align_up((size_t)M * 64 * 2, 256) : 0;
    L.tok_sc = off;  off += gemm_path ? align_up(Mp * 4, 256) : 0;
    L.gb16 = off;    off += (gemm_path && r > 0) ? align_up((size_t)d_out * 64 * 2, 256) : 0;
    // GEMM path on base-3 weights: the layer's two-bit tiles, rewritten from the base-3 bytes before the GEMM
    L.w2 = off;      off += (gemm_path && base3) ? align_up((size_t)((d_out + 15) / 16) * (size_t)((d_in + 255) / 256) * 1024, 256) : 0;
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
    float *hpart;            // decode path, optional: per (16 columns of H, K slice) the 8 x 32 partial sums of x A
    __half *h_hi, *h_lo;     // [M][r] each (decode path) or null
    __half *h16;             // [M][64] (GEMM path) or null
    int8_t *dbg_xq;          // nullable debug copies
    float *dbg_gamma_x;
    float *dbg_h;
    int M, K, r;
    uint32_t flags;
    int nslices;             // K slices behind hpart
};
static_assert(sizeof(PrologueParams) <= 128, "the decode prologue's parameter block: see GemmPrologueExtra");

// What the GEMM path's prologue kernels produce beyond PrologueParams (kept apart so that the decode
// kernels' parameter block stays as small as it was).
struct GemmPrologueExtra {
    float *tok_sc;           // [M] gamma_x * gamma_W / 127, or null
    __half *gb16;            // [N][64] gate * B^T, or null
    const __half *Bt;        // [N][r]
    const float *gate;       // [N]
    float gw_over_127;
    int N;
    int tokens_per_block;    // set by the launcher of the GEMM path's prologue kernel
    int gate_group;          // channels per gate value (1 = one per channel)
    int split_round;         // set by the launcher: the rounding pass runs as a launch of its own (round_rows_kernel)
};

// LayerNorm front end (Appendix E of the paper): parameters and where the statistics go.
struct FrontEnd {
    const float *ln_w;       // [K]
    const float *ln_b;       // [K]
    float *dbg_mean;         // [M], nullable
    float *dbg_rstd;         // [M], nullable
    float eps;
};

// Cost of one 16-row tile of a decode problem, the unit in which a launch is cut into equal shares:
// its 1 KiB weight tiles, plus what the switch to the row tile and its epilogue take, counted in
// weight tiles (measured: a layer with short rows runs slower per byte than one with long rows by
// about this much per row tile).
constexpr int kRowTileOverhead = 6;
// 1 KiB weight tiles per 16-row tile: 256 columns each at two bits per weight, 320 in the base-3 layout.
__host__ __device__ inline int weight_steps(int K, uint32_t flags) { return (flags & HGF_FLAG_BASE3) ? (K + 319) / 320 : (K + 255) >> 8; }
__host__ __device__ inline long long row_tile_cost(int K, uint32_t flags) { return (long long)weight_steps(K, flags) + kRowTileOverhead; }

// One layer problem of a decode launch (M <= 16).  tile_begin = index of its first 16-row tile in
// the launch-wide tile numbering; cost_begin = sum of the costs of all row tiles of earlier problems.
struct DecodeProblem {
    const uint8_t *packed;   // tiled layout, see above
    const int8_t *xq;        // [M][K]
    const float *gamma_x;    // [M]
    const int32_t *row_sum;  // [M]
    const __half *h_hi;      // [M][r]
    const __half *h_lo;      // [M][r]
    const float *hpart;      // group launches: partial sums of x A per (16-column tile, K slice), else null
    int nslices;             // K slices per tile in hpart
    const __half *Bt;        // [N][r]
    const float *gate;       // [N]
    void *y;                 // [M][N] fp32 or bf16
    int32_t *dbg_y_int;      // nullable
    float gw_over_127;       // gamma_W / 127
    int M, K, N, r;
    uint32_t flags;
    int tile_begin;
    long long cost_begin;
    int gate_group;          // channels per gate value: 1, or a multiple of 16 (a row tile then has one gate)
};

struct DecodeLaunch {
    const DecodeProblem *probs;  // device array, or null for a single problem passed by value
    int n_probs;
    int total_tiles;
    long long total_cost;        // cost of all row tiles of all problems
    int max_M;                   // largest token count of any problem
    int xq_smem_bytes;           // shared memory for the largest problem's activations
    int ring_slots;              // weight-ring slots per warp (set by the launcher)
    uint32_t flags;              // the launch's layout flag (HGF_FLAG_BASE3) for a group; a single problem carries its own
    const int4 *cta_range;       // per CTA: first tile, end tile, first problem (device array), or null
};

// host-side launchers (each enqueues on `stream` and returns the CUDA error of the launch)
cudaError_t launch_quant(const PrologueParams &p, const GemmPrologueExtra &x, cudaStream_t stream);
cudaError_t launch_decode_prologue(const PrologueParams &p, bool pdl, cudaStream_t stream);
// The same with the LayerNorm front end: the row blocks normalise before they quantise.
cudaError_t launch_decode_prologue_ln(const PrologueParams &p, const FrontEnd &fe, bool pdl, cudaStream_t stream);
// GEMM path with the front end: normalise + quantise every token (one block per row); the LoRA part
// runs in launch_gemm_prologue with p.xq == nullptr (its quantisation switched off).
cudaError_t launch_ln_quant(const PrologueParams &p, const GemmPrologueExtra &x, const FrontEnd &fe, cudaStream_t stream);
// Group prologue.  A quantisation item is one token row.  A LoRA item is 16 columns of H (rows
// 16 jt .. 16 jt + 15 of A^T) over one K slice of a problem; its 16 x 16 partial sums of x A go to
// `hpart` as [8 accumulator registers][32 lanes] floats, and the GEMV adds the slices of a tile in
// slice order.  Slices are 512 columns when every problem of the group has M <= 8, else 256.
struct LoraItem {
    const __half *At;          // row 16 jt of A^T, first column of the slice
    const __nv_bfloat16 *x;    // token 0, first column of the slice
    float *hpart;              // this item's 8 x 32 floats
    int K;                     // row pitch of A^T and x
    int kvalid_M;              // (columns of the slice inside K) << 8 | M
};
struct QuantItem {
    const __nv_bfloat16 *x;    // the token's row
    int8_t *xq;                // its quantised row
    float *gamma_x;            // its scale
    int32_t *row_sum;          // its sum of quantised values
    int K;
    float eps;                 // LayerNorm front end (ln_w non-null): normalise the row before quantising it
    const float *ln_w, *ln_b;  // [K] each, or null
    float *mean_out, *rstd_out;  // nullable: where this row's statistics go
};
__host__ __device__ inline int prologue_slice_k(int max_M) { return max_M <= 8 ? 512 : 256; }
cudaError_t launch_decode_prologue_group(const QuantItem *d_quant_items, int n_quant,
                                         const LoraItem *d_lora_items, int n_lora, int max_M, bool pdl,
                                         cudaStream_t stream);
cudaError_t launch_gemm_prologue(const PrologueParams &p, const GemmPrologueExtra &x, cudaStream_t stream);
// base-3 bytes of a layer -> its two-bit tiles (the GEMM path's weight format)
cudaError_t launch_repack_b3(const void *packed_b3, int64_t d_out, int64_t d_in, void *packed2, cudaStream_t stream);
cudaError_t launch_decode_gemv(const DecodeLaunch &L, const DecodeProblem *single, bool pdl, cudaStream_t stream);
// Shared memory the decode kernel needs for one problem's activations, and the largest it accepts.
int decode_xq_smem_bytes(int M, int K, uint32_t flags);
int decode_xq_smem_limit(uint32_t flags);
// Grid of the decode GEMV for a launch with that many row tiles (0 if the device cannot be queried).
int decode_grid(int total_tiles);

struct GemmParams {
    const int8_t *xq;        // [M][K]
    const uint8_t *packed;   // tiled layout, see above
    const float *gamma_x;    // [M]
    const int32_t *row_sum;  // [M]
    const __half *h16;       // [M][64]
    const float *tok_sc;     // [M] (room for M rounded up to 128)
    const __half *gb16;      // [N][64]
    void *y;                 // [M][N]
    int32_t *dbg_y_int;
    float gw_over_127;
    int M, K, N, r;
    uint32_t flags;
};
cudaError_t launch_prefill_gemm(const GemmParams &p, cudaStream_t stream);
cudaError_t launch_wait_timeout_selftest(unsigned long long limit_ns, cudaStream_t stream);

// ---- small device helpers ---------------------------------------------------------------------
__device__ __forceinline__ float bf16lo_to_float(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_to_float(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float silu_f(float z) { return z / (1.0f + expf(-z)); }

}  // namespace hgf
