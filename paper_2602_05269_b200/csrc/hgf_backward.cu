// Straight-through backward pass of the HGF layer (paper, Section 2.2, Definition "Straight-Through
// Estimator"; the forward pass it differentiates is Algorithm 1 with both quantisers treated as the
// identity):
//     dW = dY^T Xd,  dX = dY Wd + dZ A^T,  dZ = ((dY (.) g) B^T) (.) SiLU'(x A),
//     dA = x^T dZ,   dB = g (.) (H^T dY),   dg = sum_m dY (.) (H B)
// with Xd = x~ gamma_x / 127 and Wd = gamma_W t.  Seven matrix products on one generic tcgen05 bf16 GEMM
// (C = A B^T, both operands with the contraction index contiguous), plus preparation kernels that bring
// the operands into that form: transposes of dY, x, x~ and of the small matrices, and the ternary codes
// expanded as a transposed bf16 matrix.  The quantised activations enter as exact bf16 integers
// (|x~| <= 127) and the per-token scale is folded into dY; the ternary codes enter as exact -1 / 0 / +1.
#include "hgf_tc.cuh"

namespace hgf {

// ---- generic GEMM on the 5th-generation tensor cores: C[I][J] (fp32) = alpha * A B^T (+ C) ----------
// A is stored [I][Cn], B [J][Cn], both bf16 with the contraction index contiguous ("K-major"): the form
// TMA stages with the 128-byte swizzle and tcgen05.mma reads straight from shared memory.  Operands
// that the backward pass has the other way round are transposed by the preparation kernels below.
// Persistent, one CTA per SM, six warps: warp 0 stages operand tiles with TMA (128 rows of A, BN rows
// of B, 64 contraction elements = 128 bytes per row and stage), one lane of warp 1 issues
// tcgen05.mma.kind::f16 (bf16 inputs, 128 x BN x 16 per instruction, fp32 accumulators in tensor memory,
// two of them so that a tile's epilogue runs under the next tile's main loop), warps 2-5 read the
// accumulator back (tcgen05.ld) and write C.  Rows and columns past the matrices, and contraction
// elements past Cn, are zeros from TMA's out-of-bounds fill; stores are guarded.  Every wait is bounded.
constexpr int kTBM = 128, kTBK = 64, kTThreads = 192;

struct TcGemmArgs {
    float *C;
    int I, J, Cn, ldc;
    float alpha;
    int accumulate;
};

template <int BN>
struct TcCfg {
    static constexpr int STAGES = BN == 256 ? 4 : 6;
    static constexpr int A_BYTES = kTBM * 128, B_BYTES = BN * 128, STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int OFF_BAR = STAGES * STAGE_BYTES;
    static constexpr int BAR_FULL = 0, BAR_EMPTY = STAGES, BAR_ACCFULL = 2 * STAGES, BAR_ACCEMPTY = 2 * STAGES + 2, BAR_COUNT = 2 * STAGES + 4;
    static constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;
    static constexpr uint32_t IDESC = (1u << 4) /*f32*/ | (1u << 7) /*A bf16*/ | (1u << 10) /*B bf16*/ |
                                      ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(kTBM >> 4) << 24);
    static constexpr int TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;
};

template <int BN>
__global__ void __launch_bounds__(kTThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const TcGemmArgs g,
               unsigned int *status) {
    using C = TcCfg<BN>;
    extern __shared__ uint8_t tc_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)tc_smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem), bar0 = sbase + C::OFF_BAR;
    auto bar = [&](int i) { return bar0 + 8u * i; };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::OFF_BAR + C::BAR_COUNT * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_BAR + C::BAR_COUNT * 8 + 4);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles_i = (g.I + kTBM - 1) / kTBM, tiles_j = (g.J + BN - 1) / BN, num_tiles = tiles_i * tiles_j;
    const int kblocks = (g.Cn + kTBK - 1) / kTBK;

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(bar(C::BAR_FULL + s), 1);
            mbar_init(bar(C::BAR_EMPTY + s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(C::BAR_ACCFULL + b), 1);
            mbar_init(bar(C::BAR_ACCEMPTY + b), 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        fence_proxy_async();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(C::TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        int s = 0;
        uint32_t ph = 0;
        uint32_t issued[C::STAGES] = {};
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
            const int i0 = (tile / tiles_j) * kTBM, j0 = (tile % tiles_j) * BN;
            for (int kb = 0; kb < kblocks; ++kb) {
                ok = mbar_wait(bar(C::BAR_EMPTY + s), ph ^ 1u, abort_flag, status, 0x800u + s);
                if (!(ok = __all_sync(0xffffffffu, ok))) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(C::BAR_FULL + s), C::STAGE_BYTES);
                    tma_load_2d(sbase + s * C::STAGE_BYTES, &tmap_a, kb * kTBK, i0, bar(C::BAR_FULL + s));
                    tma_load_2d(sbase + s * C::STAGE_BYTES + C::A_BYTES, &tmap_b, kb * kTBK, j0, bar(C::BAR_FULL + s));
                }
                ++issued[s];
                if (++s == C::STAGES) { s = 0; ph ^= 1u; }
            }
        }
        for (int q = 0; q < C::STAGES; ++q)  // never leave with a copy in flight
            if (issued[q]) {
                const uint32_t par = (issued[q] - 1u) & 1u;
                for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar(C::BAR_FULL + q), par); ++i) {}
            }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0, it = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++it) {
                const int b = it & 1;
                const uint32_t acc = tmem_base + b * BN;
                if (it >= 2 && !(ok = mbar_wait(bar(C::BAR_ACCEMPTY + b), (uint32_t)((it >> 1) - 1) & 1u, abort_flag, status, 0x810u)))
                    break;
                tc_fence_after();
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!(ok = mbar_wait(bar(C::BAR_FULL + s), ph, abort_flag, status, 0x820u + s))) break;
                    tc_fence_after();
                    const uint64_t adesc = make_sw128_desc(sbase + s * C::STAGE_BYTES);
                    const uint64_t bdesc = make_sw128_desc(sbase + s * C::STAGE_BYTES + C::A_BYTES);
#pragma unroll
                    for (int kk = 0; kk < kTBK / 16; ++kk)  // 16 bf16 = 32 bytes of a row per MMA
                        mma_f16(acc, adesc + 2u * kk, bdesc + 2u * kk, C::IDESC, (kb | kk) ? 1u : 0u);
                    tc_commit(bar(C::BAR_EMPTY + s));
                    if (++s == C::STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                tc_commit(bar(C::BAR_ACCFULL + b));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int q = warp & 3;  // tensor-memory lane quarter this warp may access
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++it) {
            const int i0 = (tile / tiles_j) * kTBM, j0 = (tile % tiles_j) * BN;
            const int b = it & 1;
            ok = mbar_wait(bar(C::BAR_ACCFULL + b), (uint32_t)(it >> 1) & 1u, abort_flag, status, 0x830u);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;
            tc_fence_after();
            const int i = i0 + 32 * q + lane;  // this thread's row of C = its tensor-memory lane
            const uint32_t lane_base = tmem_base + ((uint32_t)(32 * q) << 16) + b * BN;
            for (int cc = 0; cc < BN; cc += 32) {
                if (j0 + cc >= g.J) break;  // (warp-uniform)
                uint32_t v[32];
                tmem_ld32(lane_base + cc, v);
                tmem_ld_wait();
                if (i < g.I) {
                    float *row = g.C + (size_t)i * g.ldc + j0 + cc;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (j0 + cc + 4 * u < g.J) {  // J is a multiple of 4
                            float4 o = make_float4(g.alpha * __uint_as_float(v[4 * u]), g.alpha * __uint_as_float(v[4 * u + 1]),
                                                   g.alpha * __uint_as_float(v[4 * u + 2]), g.alpha * __uint_as_float(v[4 * u + 3]));
                            float4 *dst = reinterpret_cast<float4 *>(row + 4 * u);
                            if (g.accumulate) { const float4 c = *dst; o.x += c.x; o.y += c.y; o.z += c.z; o.w += c.w; }
                            *dst = o;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(C::BAR_ACCEMPTY + b));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(C::TMEM_COLS) : "memory");
    }
}

template <int BN>
static cudaError_t tc_gemm_bn(const CUtensorMap &ma, const CUtensorMap &mb, const TcGemmArgs &g, cudaStream_t stream) {
    static std::atomic<unsigned long long> attr_done{0};
    cudaError_t e = ensure_dynamic_smem(tc_gemm_kernel<BN>, TcCfg<BN>::SMEM_BYTES, attr_done);
    if (e != cudaSuccess) return e;
    const int sms = device_sm_count();
    if (!sms) return cudaErrorInvalidDevice;
    const int tiles = ((g.I + kTBM - 1) / kTBM) * ((g.J + BN - 1) / BN);
    unsigned int *status = device_status_word();
    if (!status) return cudaErrorMemoryAllocation;
    tc_gemm_kernel<BN><<<tiles < sms ? tiles : sms, kTThreads, TcCfg<BN>::SMEM_BYTES, stream>>>(ma, mb, g, status);
    count_launch();
    return cudaGetLastError();
}

// C[I][J] = alpha * A[I][Cn] B[J][Cn]^T (+ C); lda, ldb in elements (multiples of 8), bases 16-byte aligned.
static cudaError_t tc_gemm(const __nv_bfloat16 *A, int lda, const __nv_bfloat16 *B, int ldb, float *C, int ldc, int I, int J, int Cn,
                           float alpha, bool accumulate, cudaStream_t stream) {
    const int BN = J > 128 ? 256 : (J > 64 ? 128 : 64);
    CUtensorMap ma, mb;
    if (!make_map_2d(&ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, A, (uint64_t)Cn, (uint64_t)I, (uint64_t)lda * 2, kTBK, kTBM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, B, (uint64_t)Cn, (uint64_t)J, (uint64_t)ldb * 2, kTBK, (uint32_t)BN, CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;
    TcGemmArgs g = {C, I, J, Cn, ldc, alpha, accumulate ? 1 : 0};
    return BN == 256 ? tc_gemm_bn<256>(ma, mb, g, stream) : (BN == 128 ? tc_gemm_bn<128>(ma, mb, g, stream) : tc_gemm_bn<64>(ma, mb, g, stream));
}

// ---- operand preparation ---------------------------------------------------------------------------
// Transposes go through a 32 x 33 shared-memory tile; a block of 32 x 8 threads handles 32 x 32 elements.
// ldt = row pitch of the transposed outputs (the row count rounded up to 8: 16-byte rows for TMA).

// dY [M][N] bf16 -> dY^T [N][ldt], (dY * gamma_x[m] / 127)^T [N][ldt], and dY * gate[n] [M][N] (each nullable).
__global__ void __launch_bounds__(256) bw_prepare_dy_kernel(const __nv_bfloat16 *dy, const float *gamma_x, const float *gate, int M, int N,
                                                            int ldt, __nv_bfloat16 *dy_t, __nv_bfloat16 *dys_t, __nv_bfloat16 *dyg) {
    __shared__ float tile[32][33];
    __shared__ float tile_s[32][33];
    const int n0 = blockIdx.x * 32, m0 = blockIdx.y * 32, tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int r = ty; r < 32; r += 8) {
        const int m = m0 + r, n = n0 + tx;
        float v = 0.0f;
        if (m < M && n < N) v = __bfloat162float(dy[(size_t)m * N + n]);
        tile[r][tx] = v;
        tile_s[r][tx] = m < M ? v * (gamma_x[m] * (1.0f / 127.0f)) : 0.0f;
        if (dyg && m < M && n < N) dyg[(size_t)m * N + n] = __float2bfloat16_rn(v * gate[n]);
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int n = n0 + r, m = m0 + tx;
        if (n < N && m < M) {
            if (dy_t) dy_t[(size_t)n * ldt + m] = __float2bfloat16_rn(tile[tx][r]);
            if (dys_t) dys_t[(size_t)n * ldt + m] = __float2bfloat16_rn(tile_s[tx][r]);
        }
    }
}

// src [R][Cc] (bf16, fp16, int8 or fp32, by `kind` 0..3) -> dst [Cc][ldt] bf16, optionally also a plain bf16 copy [R][Cc].
__global__ void __launch_bounds__(256) bw_transpose_kernel(const void *src, int kind, int R, int Cc, int ldt, __nv_bfloat16 *dst_t,
                                                           __nv_bfloat16 *dst_plain) {
    __shared__ float tile[32][33];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32, tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int rr = ty; rr < 32; rr += 8) {
        const int r = r0 + rr, c = c0 + tx;
        float v = 0.0f;
        if (r < R && c < Cc) {
            const size_t o = (size_t)r * Cc + c;
            v = kind == 0 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(src)[o])
              : kind == 1 ? __half2float(reinterpret_cast<const __half *>(src)[o])
              : kind == 2 ? (float)reinterpret_cast<const int8_t *>(src)[o]
                          : reinterpret_cast<const float *>(src)[o];
            if (dst_plain) dst_plain[o] = __float2bfloat16_rn(v);
        }
        tile[rr][tx] = v;
    }
    __syncthreads();
    for (int rr = ty; rr < 32; rr += 8) {
        const int c = c0 + rr, r = r0 + tx;
        if (c < Cc && r < R) dst_t[(size_t)c * ldt + r] = __float2bfloat16_rn(tile[tx][rr]);
    }
}

// Ternary codes of the packed matrix as a transposed bf16 matrix T^T [K][N] of -1 / 0 / +1.  One block per
// packed 1 KiB tile (16 rows x 256 columns): expanded into shared memory, written as 256 rows of 16 values.
__global__ void __launch_bounds__(256) bw_expand_ternary_t_kernel(const uint32_t *packed, int N, int K, int steps, __nv_bfloat16 *Tt) {
    __shared__ __nv_bfloat16 tile[256][16];
    const size_t t = blockIdx.x;
    const int n0 = (int)(t / steps) * 16, k0 = (int)(t % steps) * 256;
    {
        const int w = threadIdx.x, r = w >> 4, kw = w & 15;  // word w of the tile: row r, columns 16 kw ..
        const uint32_t word = packed[t * 256 + w];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t e = (word >> (2 * j)) & 0x03030303u;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int c = (e >> (8 * b)) & 0xff;
                tile[16 * kw + 4 * j + b][r] = __float2bfloat16_rn((float)(c == 3 ? 0 : c - 1));
            }
        }
    }
    __syncthreads();
    const int k = k0 + (int)threadIdx.x;
    if (k < K) {
        if (n0 + 16 <= N) {
            uint4 *dst = reinterpret_cast<uint4 *>(Tt + (size_t)k * N + n0);  // N is a multiple of 8: 16-byte aligned
            const uint4 *srcv = reinterpret_cast<const uint4 *>(&tile[threadIdx.x][0]);
            dst[0] = srcv[0];
            dst[1] = srcv[1];
        } else {
            for (int r = 0; n0 + r < N; ++r) Tt[(size_t)k * N + n0 + r] = tile[threadIdx.x][r];
        }
    }
}

// Z (fp32 [M][r]) -> H = act(Z) as bf16 [M][r] and SiLU'(Z) as fp32 (in place of Z).
__global__ void __launch_bounds__(256) bw_act_kernel(float *z, size_t n, int no_silu, __nv_bfloat16 *h) {
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    const float v = z[i];
    const float sg = 1.0f / (1.0f + expf(-v));
    h[i] = __float2bfloat16_rn(no_silu ? v : v * sg);
    z[i] = no_silu ? 1.0f : sg * (1.0f + v * (1.0f - sg));
}

// dZ = dH * SiLU'(Z), rounded to bf16.
__global__ void __launch_bounds__(256) bw_dz_kernel(const float *dh, const float *dact, size_t n, __nv_bfloat16 *dz) {
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i < n) dz[i] = __float2bfloat16_rn(dh[i] * dact[i]);
}

// From G[n][j] = sum_m dY[m][n] H[m][j]: dBt[n][j] = gate[n] G[n][j] (in place), dgate[n] = sum_j G[n][j] Bt[n][j].
__global__ void __launch_bounds__(256) bw_gate_kernel(float *G, const __half *Bt, const float *gate, int N, int r, float *dgate) {
    const int n = blockIdx.x * 256 + threadIdx.x;
    if (n >= N) return;
    float dg = 0.0f;
    const float gn = gate[n];
    for (int j = 0; j < r; ++j) {
        const float v = G[(size_t)n * r + j];
        dg = fmaf(v, __half2float(Bt[(size_t)n * r + j]), dg);
        G[(size_t)n * r + j] = gn * v;
    }
    if (dgate) dgate[n] = dg;
}

struct BwLayout {
    size_t xq, gamma_x, x_t, xq_t, T_t, dy_t, dys_t, dyg, At_b, At_t, Bt_t, z, h_b, h_t, dh, dz_b, dz_t, G, total;
};
static BwLayout bw_layout(int64_t M, int64_t K, int64_t N, int32_t r) {
    BwLayout L;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += align_up(bytes, 256); return o; };
    const size_t rr = (size_t)(r > 0 ? r : 16), Mp = (size_t)(M + 7) / 8 * 8;
    L.xq = take((size_t)M * K);
    L.gamma_x = take((size_t)M * 4);
    L.x_t = take((size_t)K * Mp * 2);
    L.xq_t = take((size_t)K * Mp * 2);
    L.T_t = take((size_t)K * N * 2);
    L.dy_t = take((size_t)N * Mp * 2);
    L.dys_t = take((size_t)N * Mp * 2);
    L.dyg = take((size_t)M * N * 2);
    L.At_b = take(rr * K * 2);
    L.At_t = take((size_t)K * rr * 2);
    L.Bt_t = take(rr * N * 2);
    L.z = take((size_t)M * rr * 4);
    L.h_b = take((size_t)M * rr * 2);
    L.h_t = take(rr * Mp * 2);
    L.dh = take((size_t)M * rr * 4);
    L.dz_b = take((size_t)M * rr * 2);
    L.dz_t = take(rr * Mp * 2);
    L.G = take((size_t)N * rr * 4);
    L.total = off;
    return L;
}

}  // namespace hgf

using namespace hgf;

extern "C" size_t hgf_backward_workspace_bytes(int64_t M, int64_t d_in, int64_t d_out, int32_t r) {
    if (M <= 0 || d_in <= 0 || d_out <= 0 || r < 0) return 256;
    return bw_layout(M, d_in, d_out, r).total;
}

extern "C" hgf_status hgf_linear_backward(const void *x, int64_t M, const void *packed, float gamma, int64_t d_in, int64_t d_out,
                                          const void *At, const void *Bt, int32_t r, const float *gate, const void *dy,
                                          const hgf_grads *grads, void *workspace, size_t workspace_bytes, uint32_t flags,
                                          void *stream_) {
    if (!x || !packed || !dy || !grads || M <= 0 || d_in <= 0 || d_out <= 0 || r < 0) return HGF_ERR_INVALID_ARG;
    if (flags & ~HGF_FLAG_NO_SILU) return HGF_ERR_INVALID_ARG;
    if (!At || !Bt || !gate) r = 0;
    if (d_in % 64 != 0 || d_out % 8 != 0 || d_in > 65536 || d_out > (1 << 24) || M > (1 << 22)) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (r != 0 && r != 16 && r != 32 && r != 48 && r != 64) return HGF_ERR_UNSUPPORTED_SHAPE;
    const uintptr_t bits = (uintptr_t)x | (uintptr_t)packed | (uintptr_t)dy | (uintptr_t)At | (uintptr_t)Bt | (uintptr_t)gate |
                           (uintptr_t)grads->dx | (uintptr_t)grads->dW | (uintptr_t)grads->dAt | (uintptr_t)grads->dBt |
                           (uintptr_t)grads->dgate;
    if (bits & 15u) return HGF_ERR_MISALIGNED;
    const BwLayout L = bw_layout(M, d_in, d_out, r);
    if (!workspace || workspace_bytes < L.total) return HGF_ERR_WORKSPACE;
    if (((uintptr_t)workspace) & 255u) return HGF_ERR_MISALIGNED;
    cudaStream_t stream = (cudaStream_t)stream_;
    char *ws = (char *)workspace;
    const int Mi = (int)M, K = (int)d_in, N = (int)d_out, Mp = (Mi + 7) / 8 * 8;
    auto bf = [&](size_t off) { return (__nv_bfloat16 *)(ws + off); };
    auto blocks1 = [](size_t n) { return (unsigned)((n + 255) / 256); };
    auto tgrid = [](int R, int Cc) { return dim3((unsigned)((Cc + 31) / 32), (unsigned)((R + 31) / 32)); };
    bool ok = true;
    auto gemm = [&](const __nv_bfloat16 *A, int lda, const __nv_bfloat16 *B, int ldb, float *C, int ldc, int I, int J, int Cn, float alpha,
                    bool acc) { ok = ok && tc_gemm(A, lda, B, ldb, C, ldc, I, J, Cn, alpha, acc, stream) == cudaSuccess; };
    const bool need_t = grads->dW || (r && (grads->dAt || grads->dBt || grads->dgate));  // products that contract over the tokens

    // Algorithm 1, steps 1-2 again: the quantised activations and their scales
    PrologueParams pp = {};
    pp.x = (const __nv_bfloat16 *)x;
    pp.xq = (int8_t *)(ws + L.xq);
    pp.gamma_x = (float *)(ws + L.gamma_x);
    pp.M = Mi;
    pp.K = K;
    pp.flags = HGF_FLAG_NO_PDL;
    if (launch_quant(pp, GemmPrologueExtra{}, stream) != cudaSuccess) return HGF_ERR_CUDA;

    bw_prepare_dy_kernel<<<tgrid(Mi, N), 256, 0, stream>>>((const __nv_bfloat16 *)dy, pp.gamma_x, gate, Mi, N, Mp,
                                                           need_t ? bf(L.dy_t) : nullptr, grads->dW ? bf(L.dys_t) : nullptr,
                                                           r ? bf(L.dyg) : nullptr);
    count_launch();
    if (grads->dW) {  // dW[n][k] = sum_m dYs[m][n] x~[m][k]
        bw_transpose_kernel<<<tgrid(Mi, K), 256, 0, stream>>>(pp.xq, 2, Mi, K, Mp, bf(L.xq_t), nullptr);
        count_launch();
        gemm(bf(L.dys_t), Mp, bf(L.xq_t), Mp, grads->dW, K, N, K, Mi, 1.0f, false);
    }
    if (grads->dx) {  // dX = gamma_W (dY T)
        const int steps = (int)(padded_k(d_in) / 256);
        bw_expand_ternary_t_kernel<<<(unsigned)(row_tiles(d_out) * steps), 256, 0, stream>>>((const uint32_t *)packed, N, K, steps, bf(L.T_t));
        count_launch();
        gemm((const __nv_bfloat16 *)dy, N, bf(L.T_t), N, grads->dx, K, Mi, K, N, gamma, false);
    }
    if (r) {
        float *z = (float *)(ws + L.z), *dh = (float *)(ws + L.dh), *G = grads->dBt ? grads->dBt : (float *)(ws + L.G);
        bw_transpose_kernel<<<tgrid(r, K), 256, 0, stream>>>(At, 1, r, K, r, bf(L.At_t), bf(L.At_b));       // A^T [r][K] -> [K][r]
        bw_transpose_kernel<<<tgrid(N, r), 256, 0, stream>>>(Bt, 1, N, r, N, bf(L.Bt_t), nullptr);          // B^T [N][r] -> [r][N]
        count_launch(2);
        gemm((const __nv_bfloat16 *)x, K, bf(L.At_b), K, z, r, Mi, r, K, 1.0f, false);                      // Z = x A
        bw_act_kernel<<<blocks1((size_t)M * r), 256, 0, stream>>>(z, (size_t)M * r, (flags & HGF_FLAG_NO_SILU) ? 1 : 0, bf(L.h_b));
        gemm(bf(L.dyg), N, bf(L.Bt_t), N, dh, r, Mi, r, N, 1.0f, false);                                    // dH = (dY g) B^T
        bw_dz_kernel<<<blocks1((size_t)M * r), 256, 0, stream>>>(dh, z, (size_t)M * r, bf(L.dz_b));
        count_launch(2);
        if (grads->dx) gemm(bf(L.dz_b), r, bf(L.At_t), r, grads->dx, K, Mi, K, r, 1.0f, true);             // dX += dZ A^T
        if (grads->dAt) {                                                                                   // dA^T = dZ^T x
            bw_transpose_kernel<<<tgrid(Mi, r), 256, 0, stream>>>(bf(L.dz_b), 0, Mi, r, Mp, bf(L.dz_t), nullptr);
            bw_transpose_kernel<<<tgrid(Mi, K), 256, 0, stream>>>(x, 0, Mi, K, Mp, bf(L.x_t), nullptr);
            count_launch(2);
            gemm(bf(L.dz_t), Mp, bf(L.x_t), Mp, grads->dAt, K, r, K, Mi, 1.0f, false);
        }
        if (grads->dBt || grads->dgate) {                                                                   // G = dY^T H
            bw_transpose_kernel<<<tgrid(Mi, r), 256, 0, stream>>>(bf(L.h_b), 0, Mi, r, Mp, bf(L.h_t), nullptr);
            count_launch();
            gemm(bf(L.dy_t), Mp, bf(L.h_t), Mp, G, r, N, r, Mi, 1.0f, false);
            bw_gate_kernel<<<blocks1((size_t)N), 256, 0, stream>>>(G, (const __half *)Bt, gate, N, r, grads->dgate);
            count_launch();
        }
    }
    return (ok && cudaGetLastError() == cudaSuccess) ? HGF_OK : HGF_ERR_CUDA;
}
