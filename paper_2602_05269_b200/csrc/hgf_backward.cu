// Straight-through backward pass of the HGF layer (paper, Section 2.2, Definition "Straight-Through
// Estimator"; the forward pass it differentiates is Algorithm 1 with both quantisers treated as the
// identity):
//     dW = dY^T Xd,  dX = dY Wd + dZ A^T,  dZ = ((dY (.) g) B^T) (.) SiLU'(x A),
//     dA = x^T dZ,   dB = g (.) (H^T dY),   dg = sum_m dY (.) (H B)
// with Xd = x~ gamma_x / 127 and Wd = gamma_W t.  Seven matrix products around one generic bf16 GEMM
// (warp-level MMA m16n8k16, fp32 accumulate, operands staged with 16-byte asynchronous copies and read
// with ldmatrix, transposed or not, so that no operand is ever transposed in memory), plus small
// elementwise kernels that prepare its operands.  The quantised activations enter as exact bf16 integers
// (|x~| <= 127) and the per-token scale is folded into dY; the ternary codes enter as exact -1 / 0 / +1.
#include "hgf_common.cuh"

namespace hgf {

// ---- generic GEMM: C[I][J] (fp32) = alpha * sum_c A(i, c) B(c, j) (+ C) --------------------------------
// A_T = false: A is stored [I][C] (contraction contiguous); true: [C][I].
// B_T = false: B is stored [J][C] (contraction contiguous); true: [C][J].
// Row pitches lda / ldb / ldc in elements; every contiguous extent is a multiple of 8 elements.
constexpr int kGBM = 128, kGBN = 128, kGBK = 32, kGThreads = 256;

struct GemmArgs {
    const __nv_bfloat16 *A, *B;
    float *C;
    int I, J, Cn;          // extents: rows of C, columns of C, contraction
    int lda, ldb, ldc;
    float alpha;
    int accumulate;        // add to what C holds
};

__device__ __forceinline__ void bw_mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void bw_ldsm4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void bw_ldsm4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void bw_cp16(uint32_t dst, const void *src, uint32_t bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}

// Shared-memory tiles keep the source's orientation.  Not transposed: [128 rows (i or j)][32 c], row pitch
// 80 bytes; transposed: [32 rows (c)][128 (i or j)], row pitch 272 bytes (both spread eight consecutive
// rows over the eight 16-byte bank groups).
constexpr int kPitchN = kGBK * 2 + 16, kPitchT = kGBM * 2 + 16;
constexpr int kTileBytesG = kGBM * kPitchN > kGBK * kPitchT ? kGBM * kPitchN : kGBK * kPitchT;

template <bool A_T, bool B_T>
__global__ void __launch_bounds__(kGThreads) bw_gemm_kernel(const GemmArgs g) {
    __shared__ __align__(128) uint8_t smem[2][2][kTileBytesG];  // [stage][A | B]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wi = warp >> 2, wj = warp & 3;                    // warp grid 2 x 4: warp tile 64 x 32
    const int i0 = blockIdx.y * kGBM, j0 = blockIdx.x * kGBN;
    const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(&smem[0][0][0]);

    auto stage_tile = [&](const __nv_bfloat16 *M, int ld, bool transposed, int f0, int fext, int c0, uint32_t dst) {
        // f = free index (i or j), c = contraction index
        if (!transposed) {  // rows f, 4 pieces of 8 contraction elements
            for (int u = tid; u < kGBM * 4; u += kGThreads) {
                const int r = u >> 2, pc = u & 3, f = f0 + r, c = c0 + 8 * pc;
                const bool in = f < fext && c < g.Cn;
                bw_cp16(dst + r * kPitchN + 16 * pc, in ? M + (size_t)f * ld + c : M, in ? 16u : 0u);
            }
        } else {            // rows c, 16 pieces of 8 free elements
            for (int u = tid; u < kGBK * 16; u += kGThreads) {
                const int r = u >> 4, pc = u & 15, c = c0 + r, f = f0 + 8 * pc;
                const bool in = c < g.Cn && f < fext;
                bw_cp16(dst + r * kPitchT + 16 * pc, in ? M + (size_t)c * ld + f : M, in ? 16u : 0u);
            }
        }
    };
    auto stage = [&](int kt, int st) {
        stage_tile(g.A, g.lda, A_T, i0, g.I, kt * kGBK, sbase + (st * 2 + 0) * kTileBytesG);
        stage_tile(g.B, g.ldb, B_T, j0, g.J, kt * kGBK, sbase + (st * 2 + 1) * kTileBytesG);
        asm volatile("cp.async.commit_group;\n" ::: "memory");
    };

    float acc[4][4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[a][b][c] = 0.0f;

    const int nk = (g.Cn + kGBK - 1) / kGBK;
    stage(0, 0);
    const int mi = lane >> 3, mr = lane & 7;  // ldmatrix: this lane addresses row mr of matrix mi
    for (int kt = 0; kt < nk; ++kt) {
        const int st = kt & 1;
        if (kt + 1 < nk) stage(kt + 1, st ^ 1);
        if (kt + 1 < nk) asm volatile("cp.async.wait_group 1;\n" ::: "memory");
        else asm volatile("cp.async.wait_all;\n" ::: "memory");
        __syncthreads();
        const uint32_t sa = sbase + (st * 2 + 0) * kTileBytesG, sb = sbase + (st * 2 + 1) * kTileBytesG;
#pragma unroll
        for (int ks = 0; ks < kGBK / 16; ++ks) {
            uint32_t af[4][4];
#pragma unroll
            for (int fi = 0; fi < 4; ++fi) {
                const int ib = 64 * wi + 16 * fi;
                if (!A_T)  // matrices: (i, c), (i + 8, c), (i, c + 8), (i + 8, c + 8)
                    bw_ldsm4(sa + (ib + 8 * (mi & 1) + mr) * kPitchN + (16 * ks + 8 * (mi >> 1)) * 2, af[fi]);
                else       // stored [c][i]: the same four blocks, each read transposed
                    bw_ldsm4_t(sa + (16 * ks + 8 * (mi >> 1) + mr) * kPitchT + (ib + 8 * (mi & 1)) * 2, af[fi]);
            }
#pragma unroll
            for (int fp = 0; fp < 2; ++fp) {  // two 8-column tiles of C per ldmatrix
                uint32_t bf[4];
                const int jb = 32 * wj + 16 * fp;
                if (!B_T)  // stored [j][c]: matrices (j, c), (j, c + 8), (j + 8, c), (j + 8, c + 8)
                    bw_ldsm4(sb + (jb + 8 * (mi >> 1) + mr) * kPitchN + (16 * ks + 8 * (mi & 1)) * 2, bf);
                else       // stored [c][j]: matrices (c, j), (c + 8, j), (c, j + 8), (c + 8, j + 8), transposed
                    bw_ldsm4_t(sb + (16 * ks + 8 * (mi & 1) + mr) * kPitchT + (jb + 8 * (mi >> 1)) * 2, bf);
#pragma unroll
                for (int fi = 0; fi < 4; ++fi) {
                    bw_mma_bf16(acc[fi][2 * fp], af[fi], bf[0], bf[1]);
                    bw_mma_bf16(acc[fi][2 * fp + 1], af[fi], bf[2], bf[3]);
                }
            }
        }
        __syncthreads();
    }

    const int gq = lane >> 2, t = lane & 3;
#pragma unroll
    for (int fi = 0; fi < 4; ++fi)
#pragma unroll
        for (int fj = 0; fj < 4; ++fj)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int i = i0 + 64 * wi + 16 * fi + gq + 8 * hh, j = j0 + 32 * wj + 8 * fj + 2 * t;
                if (i < g.I && j < g.J) {  // J is even: the pair is inside together
                    float2 *dst = reinterpret_cast<float2 *>(g.C + (size_t)i * g.ldc + j);
                    float2 v = make_float2(g.alpha * acc[fi][fj][2 * hh], g.alpha * acc[fi][fj][2 * hh + 1]);
                    if (g.accumulate) { const float2 o = *dst; v.x += o.x; v.y += o.y; }
                    *dst = v;
                }
            }
}

template <bool A_T, bool B_T>
static cudaError_t bw_gemm(const GemmArgs &g, cudaStream_t stream) {
    const dim3 grid((unsigned)((g.J + kGBN - 1) / kGBN), (unsigned)((g.I + kGBM - 1) / kGBM));
    bw_gemm_kernel<A_T, B_T><<<grid, kGThreads, 0, stream>>>(g);
    count_launch();
    return cudaGetLastError();
}

// ---- operand preparation ---------------------------------------------------------------------------
// Ternary codes of the packed matrix as bf16 -1 / 0 / +1, [N][K] row-major (one thread per packed word).
__global__ void __launch_bounds__(256) bw_expand_ternary_kernel(const uint32_t *packed, int N, int K, int steps, size_t n_words,
                                                                __nv_bfloat16 *T) {
    const size_t w = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (w >= n_words) return;
    const int kw = (int)(w & 15), r = (int)((w >> 4) & 15);
    const size_t tile = w >> 8;
    const int n = (int)(tile / steps) * 16 + r, k0 = (int)(tile % steps) * 256 + kw * 16;
    if (n >= N || k0 >= K) return;
    const uint32_t word = packed[w];
    uint32_t o[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t e = (word >> (2 * j)) & 0x03030303u;
#pragma unroll
        for (int b = 0; b < 4; b += 2) {
            const int c0 = (e >> (8 * b)) & 0xff, c1 = (e >> (8 * b + 8)) & 0xff;
            const __nv_bfloat162 v = __floats2bfloat162_rn((float)(c0 == 3 ? 0 : c0 - 1), (float)(c1 == 3 ? 0 : c1 - 1));
            o[2 * j + (b >> 1)] = *reinterpret_cast<const uint32_t *>(&v);
        }
    }
    uint4 *dst = reinterpret_cast<uint4 *>(T + (size_t)n * K + k0);
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
}

// Per element of dY [M][N]: dYs = dY * gamma_x[m] / 127 and dYg = dY * gate[n], both rounded to bf16.
__global__ void __launch_bounds__(256) bw_scale_dy_kernel(const __nv_bfloat16 *dy, const float *gamma_x, const float *gate, int M, int N,
                                                          __nv_bfloat16 *dys, __nv_bfloat16 *dyg) {
    const size_t idx = ((size_t)blockIdx.x * 256 + threadIdx.x) * 2;
    if (idx >= (size_t)M * N) return;
    const int m = (int)(idx / N), n = (int)(idx % N);
    const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(dy + idx));
    const float s = gamma_x[m] * (1.0f / 127.0f);
    *reinterpret_cast<__nv_bfloat162 *>(dys + idx) = __floats2bfloat162_rn(v.x * s, v.y * s);
    if (dyg) *reinterpret_cast<__nv_bfloat162 *>(dyg + idx) = __floats2bfloat162_rn(v.x * gate[n], v.y * gate[n + 1]);
}

__global__ void __launch_bounds__(256) bw_int8_to_bf16_kernel(const int8_t *src, size_t n, __nv_bfloat16 *dst) {
    const size_t i = ((size_t)blockIdx.x * 256 + threadIdx.x) * 4;
    if (i >= n) return;
    const char4 v = *reinterpret_cast<const char4 *>(src + i);
    *reinterpret_cast<__nv_bfloat162 *>(dst + i) = __floats2bfloat162_rn((float)v.x, (float)v.y);
    *reinterpret_cast<__nv_bfloat162 *>(dst + i + 2) = __floats2bfloat162_rn((float)v.z, (float)v.w);
}

__global__ void __launch_bounds__(256) bw_half_to_bf16_kernel(const __half *src, size_t n, __nv_bfloat16 *dst) {
    const size_t i = ((size_t)blockIdx.x * 256 + threadIdx.x) * 2;
    if (i >= n) return;
    const float2 v = __half22float2(*reinterpret_cast<const __half2 *>(src + i));
    *reinterpret_cast<__nv_bfloat162 *>(dst + i) = __floats2bfloat162_rn(v.x, v.y);
}

// Z (fp32 [M][r]) -> H = act(Z) as bf16 and SiLU'(Z) as fp32 (in place of Z).
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
    size_t xq, gamma_x, xq_b, T_b, dys, dyg, At_b, Bt_b, z, h_b, dh, dz_b, G, total;
};
static BwLayout bw_layout(int64_t M, int64_t K, int64_t N, int32_t r) {
    BwLayout L;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += align_up(bytes, 256); return o; };
    const size_t rr = (size_t)(r > 0 ? r : 16);
    L.xq = take((size_t)M * K);
    L.gamma_x = take((size_t)M * 4);
    L.xq_b = take((size_t)M * K * 2);
    L.T_b = take((size_t)N * K * 2);
    L.dys = take((size_t)M * N * 2);
    L.dyg = take((size_t)M * N * 2);
    L.At_b = take(rr * K * 2);
    L.Bt_b = take((size_t)N * rr * 2);
    L.z = take((size_t)M * rr * 4);
    L.h_b = take((size_t)M * rr * 2);
    L.dh = take((size_t)M * rr * 4);
    L.dz_b = take((size_t)M * rr * 2);
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
    const int Mi = (int)M, K = (int)d_in, N = (int)d_out;
    auto blocks = [](size_t n, int per) { return (unsigned)((n + (size_t)per * 256 - 1) / ((size_t)per * 256)); };
    bool ok = true;
    auto gemm = [&](bool at, bool bt, const void *A, int lda, const void *B, int ldb, float *C, int ldc, int I, int J, int Cn, float alpha,
                    bool acc) {
        GemmArgs g = {(const __nv_bfloat16 *)A, (const __nv_bfloat16 *)B, C, I, J, Cn, lda, ldb, ldc, alpha, acc ? 1 : 0};
        cudaError_t e = at ? (bt ? bw_gemm<true, true>(g, stream) : bw_gemm<true, false>(g, stream))
                           : (bt ? bw_gemm<false, true>(g, stream) : bw_gemm<false, false>(g, stream));
        ok = ok && e == cudaSuccess;
    };

    // Algorithm 1, steps 1-2 again: the quantised activations and their scales
    PrologueParams pp = {};
    pp.x = (const __nv_bfloat16 *)x;
    pp.xq = (int8_t *)(ws + L.xq);
    pp.gamma_x = (float *)(ws + L.gamma_x);
    pp.M = Mi;
    pp.K = K;
    pp.flags = HGF_FLAG_NO_PDL;
    if (launch_quant(pp, GemmPrologueExtra{}, stream) != cudaSuccess) return HGF_ERR_CUDA;

    __nv_bfloat16 *dys = (__nv_bfloat16 *)(ws + L.dys), *dyg = r ? (__nv_bfloat16 *)(ws + L.dyg) : nullptr;
    bw_scale_dy_kernel<<<blocks((size_t)M * N, 2), 256, 0, stream>>>((const __nv_bfloat16 *)dy, pp.gamma_x, gate, Mi, N, dys, dyg);
    count_launch();
    if (grads->dW) {  // dW[n][k] = sum_m dYs[m][n] x~[m][k]
        bw_int8_to_bf16_kernel<<<blocks((size_t)M * K, 4), 256, 0, stream>>>(pp.xq, (size_t)M * K, (__nv_bfloat16 *)(ws + L.xq_b));
        count_launch();
        gemm(true, true, dys, N, ws + L.xq_b, K, grads->dW, K, N, K, Mi, 1.0f, false);
    }
    if (grads->dx) {  // dX = gamma_W (dY T)
        const int steps = (int)(padded_k(d_in) / 256);
        const size_t n_words = (size_t)row_tiles(d_out) * steps * 256;
        bw_expand_ternary_kernel<<<blocks(n_words, 1), 256, 0, stream>>>((const uint32_t *)packed, N, K, steps, n_words,
                                                                         (__nv_bfloat16 *)(ws + L.T_b));
        count_launch();
        gemm(false, true, dy, N, ws + L.T_b, K, (float *)grads->dx, K, Mi, K, N, gamma, false);
    }
    if (r) {
        __nv_bfloat16 *At_b = (__nv_bfloat16 *)(ws + L.At_b), *Bt_b = (__nv_bfloat16 *)(ws + L.Bt_b);
        float *z = (float *)(ws + L.z), *dh = (float *)(ws + L.dh), *G = grads->dBt ? grads->dBt : (float *)(ws + L.G);
        __nv_bfloat16 *h_b = (__nv_bfloat16 *)(ws + L.h_b), *dz_b = (__nv_bfloat16 *)(ws + L.dz_b);
        bw_half_to_bf16_kernel<<<blocks((size_t)r * K, 2), 256, 0, stream>>>((const __half *)At, (size_t)r * K, At_b);
        bw_half_to_bf16_kernel<<<blocks((size_t)N * r, 2), 256, 0, stream>>>((const __half *)Bt, (size_t)N * r, Bt_b);
        count_launch(2);
        gemm(false, false, x, K, At_b, K, z, r, Mi, r, K, 1.0f, false);                 // Z = x A
        bw_act_kernel<<<blocks((size_t)M * r, 1), 256, 0, stream>>>(z, (size_t)M * r, (flags & HGF_FLAG_NO_SILU) ? 1 : 0, h_b);
        gemm(false, true, dyg, N, Bt_b, r, dh, r, Mi, r, N, 1.0f, false);               // dH = (dY g) B^T
        bw_dz_kernel<<<blocks((size_t)M * r, 1), 256, 0, stream>>>(dh, z, (size_t)M * r, dz_b);
        count_launch(2);
        if (grads->dx) gemm(false, true, dz_b, r, At_b, K, (float *)grads->dx, K, Mi, K, r, 1.0f, true);   // dX += dZ A^T
        if (grads->dAt) gemm(true, true, dz_b, r, x, K, grads->dAt, K, r, K, Mi, 1.0f, false);            // dA^T = dZ^T x
        if (grads->dBt || grads->dgate) {
            gemm(true, true, dy, N, h_b, r, G, r, N, r, Mi, 1.0f, false);                                // G = dY^T H
            bw_gate_kernel<<<(unsigned)((N + 255) / 256), 256, 0, stream>>>(G, (const __half *)Bt, gate, N, r, grads->dgate);
            count_launch();
        }
    }
    return (ok && cudaGetLastError() == cudaSuccess) ? HGF_OK : HGF_ERR_CUDA;
}
