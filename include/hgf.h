/*
 * hgf.h - C ABI of the B200 (sm_100a) forward pass of the Hybrid Gated Flow dual-stream linear layer.
 *
 * The layer (paper, Algorithm 1 "HGF 1.0 Forward Pass (Inference Mode)"):
 *
 *     gamma_x[m] = max_k |x[m][k]|                                   (per-token scale)
 *     xq[m][k]   = Clip(Round(x[m][k] / gamma_x[m] * 127), -127, 127)   (int8)
 *     Y_int      = xq  x  T^T            T in {-1,0,1}^(d_out x d_in)   (integer GEMM)
 *     Y_tern     = Y_int * gamma_x[m] * gamma_W / 127
 *     H          = SiLU(x A)             A in R^(d_in x r)
 *     Y_corr     = H B                   B in R^(r x d_out)
 *     y          = Y_tern + g * Y_corr
 *
 * Conventions for every call
 *   - Plain C ABI, no exceptions; every call that can fail returns an hgf_status.
 *   - Unless a parameter says "host", tensor pointers are DEVICE pointers owned by the caller.
 *     The library never frees, keeps or reallocates them.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Forward calls only
 *     enqueue work and return without synchronising; they allocate nothing.
 *   - All tensors are dense and row-major; all device pointers must be 16-byte aligned.
 *   - The library is CUDA-only: there is no CPU fallback.  Without a usable device a call
 *     returns HGF_ERR_CUDA.
 */
#ifndef HGF_H
#define HGF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HGF_OK = 0,
    HGF_ERR_INVALID_ARG = 1,       /* null pointer, non-positive size, unknown flag */
    HGF_ERR_UNSUPPORTED_SHAPE = 2, /* d_in % 64 != 0, r not in {0,16,32,48,64}, M too large, ... */
    HGF_ERR_MISALIGNED = 3,        /* a device pointer is not 16-byte aligned */
    HGF_ERR_WORKSPACE = 4,         /* workspace missing or smaller than hgf_workspace_bytes() */
    HGF_ERR_CUDA = 5,              /* a CUDA runtime/driver call failed (launch error, no device) */
    HGF_ERR_TIMEOUT = 6,           /* a bounded device-side wait gave up (reported by hgf_check_status) */
    HGF_ERR_TOO_LARGE = 7          /* the problem needs more scratch than HGF_STATIC_SCRATCH_BYTES */
} hgf_status;

/* flags of hgf_linear_forward / hgf_workspace_bytes */
#define HGF_FLAG_OUT_BF16 0x1u /* y is bfloat16 instead of fp32 */
#define HGF_FLAG_NO_SILU 0x2u  /* correction is (x A) B, without the SiLU the paper defines */
#define HGF_FLAG_FORCE_GEMM 0x4u /* route to the tensor-core GEMM path even when M <= 16 (a small batch whose
                                    consumer wants the GEMM path's bf16 tiles; also how the tests reach that
                                    path on decode-sized inputs) */

#define HGF_FLAG_NO_PDL 0x8u     /* do not use programmatic dependent launch (see hgf_linear_forward) */
#define HGF_FLAG_BASE3 0x10u     /* `packed` is in the base-3 layout of hgf_pack_ternary_b3 */

/* Largest token count the register-resident decode path handles; above it the GEMM path runs. */
#define HGF_DECODE_MAX_M 16

/* Optional copies of intermediate results, for parity checks.  Device pointers, each nullable. */
typedef struct {
    int8_t *xq;      /* [M][d_in]   quantised activations (Algorithm 1, step 2) */
    float *gamma_x;  /* [M]         per-token scales, after the 1e-5 floor (step 1) */
    int32_t *y_int;  /* [M][d_out]  integer accumulators sum_k xq[m][k] T[n][k] (step 3) */
    float *h;        /* [M][r]      SiLU(x A) (steps 5-6) */
} hgf_debug_out;

/*
 * Size in bytes of the packed form of a d_out x d_in ternary matrix.
 * Packed layout (the paper fixes none; it only states 1.58 bits of information per weight):
 * two bits per weight, code c = t + 1 in {0,1,2}.  The matrix is cut into tiles of 16 output rows
 * by 256 input columns; d_out is padded up to a multiple of 16 and d_in up to a multiple of 256
 * with zero weights (code 1).  A tile is 1024 bytes: its 16 rows one after the other, 64 bytes per
 * row.  Tiles are stored with the column-tile index running fastest: tile (R, C) starts at byte
 * (R * (d_in_padded / 256) + C) * 1024, so the 16 rows of a row tile are one contiguous run.  The
 * 64 bytes of a row are 16 little-endian 32-bit words; word i holds the weights whose column
 * inside the tile is 16 i .. 16 i + 15, and with that column written 16 i + 4 j + b (j, b in 0..3)
 * the code sits in bits 8 b + 2 j and 8 b + 2 j + 1.  So (word >> 2 j) & 0x03030303 is four
 * consecutive-column codes, one per byte.
 * Returns ceil(d_out / 16) * 16 * ceil(d_in / 256) * 256 / 4, or 0 for invalid sizes
 * (d_in % 64 != 0 or non-positive).
 */
size_t hgf_packed_bytes(int64_t d_out, int64_t d_in);

/*
 * Offline weight preparation (paper, Definition "Absmax Quantization", Section 2.2):
 *     gamma_W = mean |W|,  t = Clip(Round(W / gamma_W), -1, 1)   (boundaries at +-gamma_W/2,
 *     a weight exactly on a boundary becomes 0), then 2-bit packing as above.
 * W: device, fp32 [d_out][d_in].  packed: device, hgf_packed_bytes(d_out, d_in) bytes.
 * gamma_out: HOST pointer, receives gamma_W (sum in double, rounded once to fp32).
 * This call allocates a small temporary, synchronises `stream` and is not meant for the hot path.
 * Requires d_in % 64 == 0.
 */
hgf_status hgf_pack_ternary(const float *W, int64_t d_out, int64_t d_in, void *packed,
                            float *gamma_out, void *stream);

/* Inverse of the packing: T[n][k] in {-1,0,1} as int8, device [d_out][d_in].  Enqueue only. */
hgf_status hgf_unpack_ternary(const void *packed, int64_t d_out, int64_t d_in, int8_t *T,
                              void *stream);

/*
 * The same weights at 1.6 bits each: five codes per byte as the base-3 number
 * c0 + 3 c1 + 9 c2 + 27 c3 + 81 c4 (0..242), the nearest byte-aligned packing to the log2(3) = 1.58
 * bits the paper counts per ternary weight (Introduction, the T_max bound; Section 4.2, the
 * effective bit-width).  It takes a fifth off the weight stream of the memory-bound decode path at
 * the price of a table look-up per byte; forward calls take it with HGF_FLAG_BASE3.  The decode
 * path (M <= HGF_DECODE_MAX_M) computes straight from the base-3 bytes.  The compute-bound GEMM path
 * reads two-bit tiles: given base-3 weights, hgf_linear_forward first rewrites the layer's tiles into
 * its workspace (one small launch; hgf_workspace_bytes with the flag includes the room), so a model
 * stored at 1.6 bits needs no second copy of its weights for prefill.  Groups and the allocation-free
 * entry point take base-3 weights on the decode path only.
 * Layout: tiles of 16 output rows by 320 input columns (d_out padded to 16, d_in to 320, with zero
 * weights); a tile is 1024 bytes, its 16 rows one after the other, 64 bytes per row; tile (R, C)
 * starts at byte (R * (d_in_padded / 320) + C) * 1024.  Byte q = 16 t + j (t in 0..3, j in 0..15) of a
 * row holds in digit e < 4 the code of tile column col(j, t) + e and in digit 4 the code of tile column
 * col(16 + j / 4, t) + j % 4, with col(p, t) = 32 (p / 2) + 16 (p % 2) + 4 t.  Examples: column 0 is
 * digit 0 of byte 0, column 5 digit 1 of byte 16, column 16 digit 0 of byte 1, column 47 digit 3 of
 * byte 50, column 256 digit 4 of byte 0, column 319 digit 4 of byte 63.
 * hgf_packed_bytes_b3 returns ceil(d_out / 16) * 16 * ceil(d_in / 320) * 320 / 5, or 0 for invalid
 * sizes.  Arguments and behaviour of the other two calls are those of their two-bit counterparts.
 */
size_t hgf_packed_bytes_b3(int64_t d_out, int64_t d_in);
hgf_status hgf_pack_ternary_b3(const float *W, int64_t d_out, int64_t d_in, void *packed,
                               float *gamma_out, void *stream);
hgf_status hgf_unpack_ternary_b3(const void *packed, int64_t d_out, int64_t d_in, int8_t *T,
                                 void *stream);

/* Bytes of caller-provided scratch hgf_linear_forward needs for this problem (never 0). */
size_t hgf_workspace_bytes(int64_t M, int64_t d_in, int64_t d_out, int32_t r, uint32_t flags);

/*
 * The layer forward pass (paper, Algorithm 1; Definitions "Dynamic Activation Quantization",
 * "Low-Rank Correction", "Gated Fusion").
 *
 *   x       [M][d_in]      bfloat16
 *   packed  from hgf_pack_ternary, gamma = its gamma_W
 *   At      [r][d_in]      fp16: the transpose of the paper's A (d_in contiguous)
 *   Bt      [d_out][r]     fp16: the transpose of the paper's B (r contiguous)
 *   gate    [d_out]        fp32: the evaluated gate g = tanh(alpha), one value per output
 *                          channel (the paper's scalar gate is the constant vector)
 *   y       [M][d_out]     fp32, or bfloat16 with HGF_FLAG_OUT_BF16
 *   workspace              device scratch of at least hgf_workspace_bytes(...) bytes, 256-byte
 *                          aligned; holds xq, gamma_x, row sums and H between the kernels
 *   dbg                    nullable; see hgf_debug_out
 *
 * r = 0, or any of At/Bt/gate null, computes the pure ternary layer (Y_tern only).
 * The per-token scale is floored at 1e-5 (an all-zero token yields zeros).
 * Requirements: M >= 1; d_in % 64 == 0; d_out >= 1; r in {0,16,32,48,64}; 16-byte aligned
 * pointers.  M <= HGF_DECODE_MAX_M runs the bandwidth-bound GEMV path, larger M the tcgen05
 * int8 GEMM path (which additionally needs d_out % 8 == 0).  The GEMV path keeps the layer's
 * quantised activations in shared memory; a problem with (M + 1) * (d_in_padded + 64) above about
 * 104 KiB (no shape of the paper's model classes at M <= 16) takes the GEMM path as well.
 * Calls on the same workspace must not overlap on the device.
 * Launch overlap: the decode kernels are launched with programmatic stream serialization and start
 * fetching `packed` before the preceding work on `stream` has finished (they wait for that work
 * before touching x, the workspace or y).  packed, At, Bt and gate must therefore not be written
 * by work still pending on `stream`; pass HGF_FLAG_NO_PDL if they might be.
 */
hgf_status hgf_linear_forward(const void *x, int64_t M, const void *packed, float gamma,
                              int64_t d_in, int64_t d_out, const void *At, const void *Bt,
                              int32_t r, const float *gate, void *y, void *workspace,
                              size_t workspace_bytes, const hgf_debug_out *dbg, uint32_t flags,
                              void *stream);

/*
 * The two launches of hgf_linear_forward separately (both bits together are hgf_linear_forward):
 * HGF_PHASE_PROLOGUE runs Algorithm 1 steps 1-2 and 5-6 (activation quantisation, H = SiLU(x A))
 * into the workspace; HGF_PHASE_GEMV runs steps 3-4 and 7-8 (the ternary contraction - GEMV or
 * tensor-core GEMM, whichever path the problem takes - with dequantisation, up-projection and gated
 * fusion) from what the last prologue call with the same arguments left in the workspace.  For
 * timing the two kernels apart, and for callers that re-run the contraction of an unchanged input.
 */
#define HGF_PHASE_PROLOGUE 0x1u
#define HGF_PHASE_GEMV 0x2u
hgf_status hgf_linear_forward_phases(const void *x, int64_t M, const void *packed, float gamma,
                                     int64_t d_in, int64_t d_out, const void *At, const void *Bt,
                                     int32_t r, const float *gate, void *y, void *workspace,
                                     size_t workspace_bytes, const hgf_debug_out *dbg, uint32_t flags,
                                     uint32_t phases, void *stream);

/*
 * The layer with the front end and the gate granularity of the paper's reference module
 * (Appendix E): ScientificBitLinear.forward normalises each token with a LayerNorm over d_in before
 * it quantises it, AdaptiveDualPathLinear.forward feeds the RAW token to the correction path, and
 * HeadAdaptiveDiffAttention gates per attention head.
 *
 *     xn[m][k]   = ((x[m][k] - mean[m]) * rstd[m]) * ln_weight[k] + ln_bias[k]
 *                  mean, rstd = 1 / sqrt(var + eps) of token m (biased variance); every operation one
 *                  binary32 operation, in this order (the rounded value decides the int8 code)
 *     gamma_x[m] = max(max_k |xn[m][k]|, 1e-5);  xq = Clip(Round(xn * (127 / gamma_x)), -127, 127),
 *                  binary32 as in the listing (a product, not a quotient)
 *     y          = Y_int * gamma_x * gamma_W / 127 + gate[n / gate_group] * (SiLU(x A) B)[m][n]
 *
 * ln_weight, ln_bias: device fp32 [d_in]; both null = no LayerNorm (the call then is
 * hgf_linear_forward with a grouped gate).  gate holds ceil(d_out / gate_group) values: gate_group
 * 0 or 1 = one per channel, d_out / n_heads = one per head, >= d_out = the paper's scalar gate;
 * it must be 1, a multiple of 16, or >= d_out.  mean_out / rstd_out: nullable device fp32 [M], receive
 * the statistics the kernels used (for parity checks).  Everything else as hgf_linear_forward, same
 * workspace size.  With a LayerNorm the GEMM path takes one more launch (normalise + quantise).
 */
typedef struct {
    const float *ln_weight;
    const float *ln_bias;
    float eps;
    int64_t gate_group;
    float *mean_out;
    float *rstd_out;
} hgf_front_end;
hgf_status hgf_linear_forward_ln(const void *x, int64_t M, const void *packed, float gamma,
                                 int64_t d_in, int64_t d_out, const void *At, const void *Bt,
                                 int32_t r, const float *gate, void *y, void *workspace,
                                 size_t workspace_bytes, const hgf_debug_out *dbg,
                                 const hgf_front_end *front_end, uint32_t flags, void *stream);

/*
 * hgf_linear_forward for callers that cannot hand over a workspace.  (The paper has no counterpart:
 * this is a convenience of the library, not a step of the method.)
 *
 * Who needs it: code that runs where device memory may not be allocated - a serving loop whose
 * memory plan was fixed at start-up and is fully spent, a plug-in inside a host framework that owns
 * every byte of device memory through its own pool and forbids cudaMalloc behind its back, or a
 * latency-critical decode thread for which cudaMalloc's implicit device-wide synchronisation is a
 * stall it cannot afford.  Such a caller still owns x, the weights and y, but has nowhere to get
 * the few hundred KiB of scratch that the layer's kernels exchange intermediate results through.
 *
 * This entry point takes that scratch from an array that is part of the library image itself
 * (HGF_STATIC_SCRATCH_BYTES of device memory, held by every GPU that loads the library until the
 * process exits).  It calls no allocator of any kind.  Arguments are those of hgf_linear_forward
 * without workspace and debug outputs; results are the same.
 *
 * Limits: only decode-sized problems (those hgf_linear_forward serves with its GEMV path, M <=
 * HGF_DECODE_MAX_M) with hgf_workspace_bytes(M, d_in, d_out, r, flags) <= HGF_STATIC_SCRATCH_BYTES.
 * The scratch holds M * d_in bytes of quantised activations plus (r / 16) * ceil(d_in / 256) KiB of
 * partial sums of x A and a few KiB of per-token values: with r = 64 that is every model shape of
 * the paper at M = 16 up to d_in = 6656 and at M = 1 up to d_in = 16384; M = 1, d_in = 32768, r = 64
 * does not fit.  A problem that needs more returns HGF_ERR_TOO_LARGE; an unsupported rank, or a
 * problem that would take the GEMM path, HGF_ERR_UNSUPPORTED_SHAPE; nothing is launched then.
 *
 * Sharing: all calls on a device use the same array, and it keeps what the last call left in it.
 * Nothing in it has to be cleared (each call writes every value before reading it), but two calls
 * whose kernels may run at the same time - different streams, or different host threads without
 * ordering between their streams - would overwrite each other's intermediates: order them.
 *
 * Set-up: the first call on each device looks up the array's device address (the current device
 * must be the one the pointers belong to).  Make that first call before starting any stream
 * capture.
 */
#define HGF_STATIC_SCRATCH_BYTES (288u * 1024u)
hgf_status hgf_linear_forward_static(const void *x, int64_t M, const void *packed, float gamma,
                                     int64_t d_in, int64_t d_out, const void *At, const void *Bt,
                                     int32_t r, const float *gate, void *y, uint32_t flags,
                                     void *stream);

/*
 * A group of independent decode-sized layer problems served by one pair of launches.  The paper's
 * blocks evaluate several HGF layers on the same or on unrelated inputs with no dependency between
 * them (Section 2.4, Definition "HGF Attention Projections": Q, K and V are three HGF layers of the
 * same X; the MLP's two up-projections likewise), and each is small against the launch latency,
 * so a group streams all their packed weights in one pass.  Each problem is exactly one
 * hgf_linear_forward with M <= HGF_DECODE_MAX_M (same argument meaning, same requirements).
 * Problems that name the same x (same pointer, M and d_in) are quantised once and share the
 * result; their LoRA down-projections stay separate, since each has its own A.
 *
 * hgf_group_create records the problems (pointers are kept, not the data: x, y and the weights
 * stay owned by the caller and must stay valid) and allocates the group's descriptors and
 * workspace on the current device; it is a set-up call, not for the hot path.
 * hgf_group_forward only enqueues: one prologue launch and one GEMV launch for the whole group,
 * which streams the packed weights of all its problems as one sequence split evenly over the SMs.
 * Forward calls of one group must not overlap on the device.  hgf_group_destroy frees the group
 * (the caller makes sure no forward is still running).
 */
typedef struct {
    const void *x;      /* [M][d_in] bf16 */
    int64_t M;
    const void *packed; /* from hgf_pack_ternary */
    float gamma;
    int64_t d_in, d_out;
    const void *At;     /* [r][d_in] fp16, nullable */
    const void *Bt;     /* [d_out][r] fp16, nullable */
    int32_t r;
    const float *gate;  /* [d_out] fp32, nullable */
    void *y;            /* [M][d_out] fp32, or bf16 with HGF_FLAG_OUT_BF16 */
} hgf_problem;

typedef struct hgf_group hgf_group;

hgf_status hgf_group_create(const hgf_problem *problems /* host array */, int32_t n, uint32_t flags,
                            hgf_group **out);
/*
 * The same with a front end per problem (front_ends: host array of n entries, or null for none):
 * the LayerNorm in front of the quantiser and the gate granularity of hgf_linear_forward_ln.  This is
 * the paper's attention block in one group (Appendix E, HeadAdaptiveDiffAttention): Q, K and V are
 * three HGF layers of the same x, each behind a LayerNorm of its own, with one gate per head.
 * Problems on the same x share a quantisation only if they also name the same LayerNorm parameters.
 * The parameter arrays are kept by pointer, like the other tensors; mean_out / rstd_out, if given,
 * are written by every forward.
 */
hgf_status hgf_group_create_ln(const hgf_problem *problems /* host array */,
                               const hgf_front_end *front_ends /* host array, nullable */, int32_t n,
                               uint32_t flags, hgf_group **out);
hgf_status hgf_group_forward(hgf_group *group, void *stream);
/*
 * The two launches of hgf_group_forward separately, for measurement: HGF_PHASE_PROLOGUE runs
 * Algorithm 1 steps 1-2 and 5-6 (activation quantisation, H = SiLU(x A)) into the group's
 * workspace, HGF_PHASE_GEMV steps 3-4 and 7-8 from what the last prologue left there.  Both bits
 * together are hgf_group_forward.
 */
hgf_status hgf_group_forward_phases(hgf_group *group, uint32_t phases, void *stream);
/*
 * Parity-check access to problem `index` of a group (Algorithm 1, steps 1-3 as the group's own
 * kernels compute them).  y_int: nullable device buffer [M][d_out] owned by the caller; from the
 * next forward on, the GEMV also writes the problem's integer accumulators there (null switches
 * that off again).  views: nullable host struct that receives device pointers INTO the group's
 * workspace - xq [M][d_in] and gamma_x [M] as the last forward left them (problems that share an
 * input share these) - plus y_int as passed; h is set to null (the group keeps x A in K slices).
 * A set-up call: it synchronises the device; no forward of the group may be running.
 */
hgf_status hgf_group_debug(hgf_group *group, int32_t index, int32_t *y_int, hgf_debug_out *views);
void hgf_group_destroy(hgf_group *group);

/*
 * Step a1 alone (paper, Definition "Dynamic Activation Quantization"): xq, gamma_x and the row
 * sums sum_k xq[m][k] (row_sum nullable).  Enqueue only.
 */
hgf_status hgf_act_quant(const void *x, int64_t M, int64_t d_in, int8_t *xq, float *gamma_x,
                         int32_t *row_sum, void *stream);

/*
 * Causal differential attention forward on the outputs of the HGF attention projections (paper,
 * Section 2.4, Definitions "HGF Attention Projections" and "Differential Attention"):
 *     O = ( Softmax(Q1 K1^T / sqrt(d_h)) - lambda * Softmax(Q2 K2^T / sqrt(d_h)) ) V * out_scale
 * per batch element and head; token i attends to tokens j <= i.
 *   q, k   [B*L][2 * n_heads * head_dim]  bfloat16, token-major as the Q and K projections write them
 *          (HGF_FLAG_OUT_BF16): the first n_heads * head_dim columns are the heads of stream 1, the
 *          rest those of stream 2 ([Q1; Q2] of the Definition)
 *   v      [B*L][n_heads * head_dim]      bfloat16 (the V projection, width d / 2)
 *   out    [B*L][n_heads * head_dim]      fp32, or bfloat16 with HGF_FLAG_OUT_BF16 (the input of the
 *          output projection)
 *   lambda the learnable scalar (hgf_diff_lambda0(head_dim) is its initial value 0.8 - 0.6 exp(-0.3 d_h));
 *   out_scale 1 for the Definition; the reference module of Appendix E multiplies by 0.5.
 * head_dim 64 or 128; B, n_heads <= 65535, L <= 2^24, B * L < 2^31 (else HGF_ERR_UNSUPPORTED_SHAPE); 16-byte
 * aligned pointers.  Enqueue only; no workspace.  The probabilities enter the second product rounded to
 * bfloat16 (fp32 accumulation); a bounded wait that ran out is reported by hgf_check_status.
 */
hgf_status hgf_diff_attention_forward(const void *q, const void *k, const void *v, int64_t B, int64_t L,
                                      int32_t n_heads, int32_t head_dim, float lambda, float out_scale,
                                      void *out, uint32_t flags, void *stream);
double hgf_diff_lambda0(double head_dim);

/*
 * Straight-through backward pass of the layer (paper, Section 2.2, Definition "Straight-Through
 * Estimator"): the forward pass of hgf_linear_forward is differentiated with both quantisers treated
 * as the identity (every activation lies inside its clipping range; the weight gradient is passed
 * unchanged, as in the reference module), everything else exactly.  With Xd = x~ gamma_x / 127,
 * Wd = gamma_W t, Z = x A, H = SiLU(Z) and dY the gradient with respect to y:
 *     dW = dY^T Xd                          [d_out][d_in]  (gradient for the latent fp32 weights)
 *     dX = dY Wd + dZ A^T                   [M][d_in],   dZ = ((dY (.) g) B^T) (.) SiLU'(Z)
 *     dAt = dZ^T x  [r][d_in],  dBt = g (.) (dY^T H)  [d_out][r],  dgate = sum_m dY (.) (H B)  [d_out]
 * (dgate is with respect to the evaluated gate g; d alpha = dgate (1 - g^2) is the caller's.)
 * x, packed, gamma, At, Bt, gate as in the forward call; dy [M][d_out] bfloat16.  Every output is fp32
 * and nullable (skipped).  The matrix products run on the tensor cores with bf16 operands and fp32
 * accumulation (the precision the paper trains in): dY, x and t enter exactly; Xd, A, g (.) B, H, dZ and
 * dZ / gamma_W (the low-rank term of dX is accumulated together with dY t and the sum scaled by gamma_W)
 * are rounded to bf16.  Requirements: d_in % 64 == 0, d_out % 8 == 0, M <= 2^22, r in {0,16,32,48,64};
 * 16-byte aligned pointers; workspace of hgf_backward_workspace_bytes(...) bytes, 256-byte aligned (it
 * holds the operands above and the partial sums of the thin products; its contents are scratch).
 * Flags: HGF_FLAG_NO_SILU.  Enqueue only; errors of the launches come back as HGF_ERR_CUDA, a bounded
 * wait that ran out through hgf_check_status.
 */
typedef struct {
    float *dx;
    float *dW;
    float *dAt;
    float *dBt;
    float *dgate;
} hgf_grads;
size_t hgf_backward_workspace_bytes(int64_t M, int64_t d_in, int64_t d_out, int32_t r);
hgf_status hgf_linear_backward(const void *x, int64_t M, const void *packed, float gamma, int64_t d_in,
                               int64_t d_out, const void *At, const void *Bt, int32_t r, const float *gate,
                               const void *dy, const hgf_grads *grads, void *workspace,
                               size_t workspace_bytes, uint32_t flags, void *stream);

/*
 * Device-side waits in the GEMM path are bounded; when one gives up the kernel records it and
 * returns.  This call synchronises `stream`, reads and clears that record, and returns
 * HGF_ERR_TIMEOUT if a wait gave up since the last check (HGF_OK otherwise).
 */
hgf_status hgf_check_status(void *stream);

/*
 * Exercises that error path without any fault: enqueues a one-warp kernel whose bounded wait (the
 * one every role of the GEMM kernel uses, with a limit of `limit_us` microseconds, 1 .. 1000000,
 * instead of two seconds) sits on a barrier that nothing ever completes.  The wait gives up, records
 * it and the kernel returns normally; the next hgf_check_status reports HGF_ERR_TIMEOUT once and the
 * device stays usable.  For tests of the callers' handling of HGF_ERR_TIMEOUT.
 */
hgf_status hgf_selftest_wait_timeout(uint32_t limit_us, void *stream);

/* Memory-wall bound of the paper's introduction: T_max = B_mem / (P * b / 8) tokens/s. */
double hgf_tmax_tokens_per_s(double bmem_bytes_per_s, double params, double bits_per_param);

/* Kernels launched by this library in this process so far (for launch accounting). */
uint64_t hgf_launch_count(void);

const char *hgf_status_string(hgf_status s);

#ifdef __cplusplus
}
#endif
#endif /* HGF_H */
