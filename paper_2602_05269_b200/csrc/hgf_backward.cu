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

// ---- generic GEMM on the 5th-generation tensor cores: C[I][J] (fp32) = alpha * sum_c A[i][c] B[j][c] (+ C) ----
// Either operand may be stored with the contraction index contiguous ([rows][Cn], "K-major") or with its
// row index contiguous ([Cn][rows], "MN-major"): tcgen05.mma reads both forms from shared memory (the
// instruction descriptor says which), so no operand of the backward pass is ever transposed in memory.
// A K-major tile of R rows x 64 contraction elements is one TMA box of R rows of 128 bytes; an MN-major
// tile is R / 64 boxes of 64 contraction rows of 128 bytes (64 operand rows each), 8 KiB apart; both use
// the 128-byte swizzle.  The contraction may continue over a second pair of operands (A2, B2: the
// low-rank term of dX), and may be split over several CTAs that write partial sums which a second
// kernel adds up in a fixed order.
// Persistent, one CTA per SM, six warps: warp 0 stages operand tiles with TMA, one lane of warp 1 issues
// tcgen05.mma.kind::f16 (bf16 inputs, 128 x BN x 16 per instruction, fp32 accumulators in tensor memory,
// two of them so that a tile's epilogue runs under the next tile's main loop), warps 2-5 read the
// accumulator back (tcgen05.ld) and write C.  Rows and columns past the matrices, and contraction
// elements past Cn, are zeros from TMA's out-of-bounds fill; stores are guarded.  Every wait is bounded.
constexpr int kTBM = 128, kTBK = 64, kTThreads = 192, kTBox = 64 * 128;

struct TcGemmArgs {
    float *C;          // output, or the partial sums [splits][I][ldc] when splits > 1
    int I, J, ldc;
    int kb1, kb2;      // 64-element contraction blocks of the first and of the second operand pair
    int splits, kb_per_split;
    int n_half;        // splits == 1 only: the last n_half / 2 tiles are worked as halves of BN / 2 columns (see tc_gemm)
    int a_mn, b_mn;    // operand forms (both pairs alike)
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
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               const __grid_constant__ CUtensorMap tmap_a2, const __grid_constant__ CUtensorMap tmap_b2, const TcGemmArgs g,
               unsigned int *status) {
    using C = TcCfg<BN>;
    extern __shared__ uint8_t tc_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)tc_smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem), bar0 = sbase + C::OFF_BAR;
    auto bar = [&](int i) { return bar0 + 8u * i; };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::OFF_BAR + C::BAR_COUNT * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_BAR + C::BAR_COUNT * 8 + 4);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles_i = (g.I + kTBM - 1) / kTBM, tiles_j = (g.J + BN - 1) / BN, tiles_ij = tiles_i * tiles_j;
    const int n_full = tiles_ij - g.n_half / 2;  // tiles worked whole (all of them unless n_half > 0)
    const int num_work = g.n_half ? n_full + g.n_half : tiles_ij * g.splits, kb_all = g.kb1 + g.kb2;
    // work item w: output tile w % tiles_ij, contraction blocks [kb_lo, kb_hi) of split w / tiles_ij; with
    // half tiles (one split): items past n_full are the two halves of the remaining tiles, in turn
    auto kb_lo = [&](int w) { return g.n_half ? 0 : (w / tiles_ij) * g.kb_per_split; };
    auto kb_hi = [&](int w) {
        if (g.n_half) return kb_all;
        const int e = (w / tiles_ij + 1) * g.kb_per_split;
        return e < kb_all ? e : kb_all;
    };
    auto tile_of = [&](int w, int &i0, int &j0, int &bn) {
        int tile = w % tiles_ij, half = 0;
        bn = BN;
        if (g.n_half && w >= n_full) {
            tile = n_full + (w - n_full) / 2;
            half = (w - n_full) & 1;
            bn = BN / 2;
        }
        i0 = (tile / tiles_j) * kTBM;
        j0 = (tile % tiles_j) * BN + half * (BN / 2);
    };

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
        for (int w = blockIdx.x; ok && w < num_work; w += gridDim.x) {
            int i0, j0, bn;
            tile_of(w, i0, j0, bn);
            for (int kb = kb_lo(w); kb < kb_hi(w); ++kb) {
                ok = mbar_wait(bar(C::BAR_EMPTY + s), ph ^ 1u, abort_flag, status, 0x800u + s);
                if (!(ok = __all_sync(0xffffffffu, ok))) break;
                if (lane == 0) {
                    const bool second = kb >= g.kb1;
                    const CUtensorMap *ma = second ? &tmap_a2 : &tmap_a, *mb = second ? &tmap_b2 : &tmap_b;
                    const int c0 = (second ? kb - g.kb1 : kb) * kTBK;
                    const uint32_t dst_a = sbase + s * C::STAGE_BYTES, dst_b = dst_a + C::A_BYTES, full = bar(C::BAR_FULL + s);
                    mbar_arrive_expect_tx(full, C::A_BYTES + (g.b_mn ? bn * 128 : C::B_BYTES));  // (a K-major box always has BN rows)
                    if (g.a_mn) {
                        for (int h = 0; h < kTBM / 64; ++h) tma_load_2d(dst_a + h * kTBox, ma, i0 + 64 * h, c0, full);
                    } else {
                        tma_load_2d(dst_a, ma, c0, i0, full);
                    }
                    if (g.b_mn) {
                        for (int h = 0; h < bn / 64; ++h) tma_load_2d(dst_b + h * kTBox, mb, j0 + 64 * h, c0, full);
                    } else {
                        tma_load_2d(dst_b, mb, c0, j0, full);
                    }
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
            const uint32_t idesc = C::IDESC | (g.a_mn ? 1u << 15 : 0u) | (g.b_mn ? 1u << 16 : 0u);
            const uint32_t a_step = g.a_mn ? (16 * 128) >> 4 : 32 >> 4, b_step = g.b_mn ? (16 * 128) >> 4 : 32 >> 4;  // 16 contraction elements
            for (int w = blockIdx.x; ok && w < num_work; w += gridDim.x, ++it) {
                const int b = it & 1;
                const uint32_t acc = tmem_base + b * BN;
                if (it >= 2 && !(ok = mbar_wait(bar(C::BAR_ACCEMPTY + b), (uint32_t)((it >> 1) - 1) & 1u, abort_flag, status, 0x810u)))
                    break;
                tc_fence_after();
                const int lo = kb_lo(w), hi = kb_hi(w);
                int ti0, tj0, bn;
                tile_of(w, ti0, tj0, bn);
                const uint32_t idesc_w = (idesc & ~(0x3fu << 17)) | ((uint32_t)(bn >> 3) << 17);
                for (int kb = lo; kb < hi; ++kb) {
                    if (!(ok = mbar_wait(bar(C::BAR_FULL + s), ph, abort_flag, status, 0x820u + s))) break;
                    tc_fence_after();
                    const uint32_t sa = sbase + s * C::STAGE_BYTES, sb = sa + C::A_BYTES;
                    const uint64_t adesc = g.a_mn ? make_sw128_mn_desc(sa, kTBox) : make_sw128_desc(sa);
                    const uint64_t bdesc = g.b_mn ? make_sw128_mn_desc(sb, kTBox) : make_sw128_desc(sb);
#pragma unroll
                    for (int kk = 0; kk < kTBK / 16; ++kk)
                        mma_f16(acc, adesc + (uint64_t)(a_step * kk), bdesc + (uint64_t)(b_step * kk), idesc_w, (kb > lo || kk) ? 1u : 0u);
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
        for (int w = blockIdx.x; ok && w < num_work; w += gridDim.x, ++it) {
            int i0, j0, bn;
            tile_of(w, i0, j0, bn);
            float *Cw = g.C + (g.n_half ? (size_t)0 : (size_t)(w / tiles_ij) * g.I * g.ldc);
            const int b = it & 1;
            ok = mbar_wait(bar(C::BAR_ACCFULL + b), (uint32_t)(it >> 1) & 1u, abort_flag, status, 0x830u);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;
            tc_fence_after();
            const int i = i0 + 32 * q + lane;  // this thread's row of C = its tensor-memory lane
            const uint32_t lane_base = tmem_base + ((uint32_t)(32 * q) << 16) + b * BN;
            const bool empty = kb_lo(w) >= kb_hi(w);  // a split past the end of the contraction: zeros
            for (int cc = 0; cc < bn; cc += 32) {
                if (j0 + cc >= g.J) break;  // (warp-uniform)
                uint32_t v[32];
                tmem_ld32(lane_base + cc, v);
                tmem_ld_wait();
                if (i < g.I) {
                    float *row = Cw + (size_t)i * g.ldc + j0 + cc;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (j0 + cc + 4 * u < g.J) {  // J is a multiple of 4
                            float4 o = make_float4(g.alpha * __uint_as_float(v[4 * u]), g.alpha * __uint_as_float(v[4 * u + 1]),
                                                   g.alpha * __uint_as_float(v[4 * u + 2]), g.alpha * __uint_as_float(v[4 * u + 3]));
                            if (empty) o = make_float4(0.f, 0.f, 0.f, 0.f);
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
// Sum of the partial results of a split contraction, in split order: C = alpha * sum_s P[s] (+ C).
__global__ void __launch_bounds__(256) tc_reduce_kernel(const float4 *P, int splits, size_t n4, float alpha, int accumulate, float4 *C) {
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= n4) return;
    float4 a = P[i];
    for (int s = 1; s < splits; ++s) {
        const float4 b = P[(size_t)s * n4 + i];
        a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
    }
    a.x *= alpha; a.y *= alpha; a.z *= alpha; a.w *= alpha;
    if (accumulate) { const float4 c = C[i]; a.x += c.x; a.y += c.y; a.z += c.z; a.w += c.w; }
    C[i] = a;
}

// One operand: `rows` x `cn` values; mn = stored [cn][rows] (row index contiguous), else [rows][cn]; ld in elements.
struct TcOperand {
    const __nv_bfloat16 *p;
    int ld;
    bool mn;
};

static bool tc_map(CUtensorMap *m, const TcOperand &o, int rows, int cn, int tile_rows) {
    if (o.mn) return make_map_2d(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, o.p, (uint64_t)rows, (uint64_t)cn, (uint64_t)o.ld * 2, 64, kTBK, CU_TENSOR_MAP_SWIZZLE_128B);
    return make_map_2d(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, o.p, (uint64_t)cn, (uint64_t)rows, (uint64_t)o.ld * 2, kTBK, (uint32_t)tile_rows, CU_TENSOR_MAP_SWIZZLE_128B);
}

template <int BN>
static cudaError_t tc_gemm_bn(const CUtensorMap *maps, const TcGemmArgs &g, cudaStream_t stream) {
    static std::atomic<unsigned long long> attr_done{0};
    cudaError_t e = ensure_dynamic_smem(tc_gemm_kernel<BN>, TcCfg<BN>::SMEM_BYTES, attr_done);
    if (e != cudaSuccess) return e;
    const int sms = device_sm_count();
    if (!sms) return cudaErrorInvalidDevice;
    const int tiles = ((g.I + kTBM - 1) / kTBM) * ((g.J + BN - 1) / BN);
    const int work = g.n_half ? tiles + g.n_half / 2 : tiles * g.splits;
    unsigned int *status = device_status_word();
    if (!status) return cudaErrorMemoryAllocation;
    tc_gemm_kernel<BN><<<work < sms ? work : sms, kTThreads, TcCfg<BN>::SMEM_BYTES, stream>>>(maps[0], maps[1], maps[2], maps[3], g, status);
    count_launch();
    return cudaGetLastError();
}

// C[I][J] = alpha * (A B^T + A2 B2^T) (+ C).  A2.p == nullptr: one pair only.  Both pairs have the same
// operand forms.  `partials` (splits_max * I * ldc floats) enables splitting the contraction when the
// output has fewer tiles than the device has SMs; ldc must then be J.  Bases 16-byte aligned, ld % 8 == 0.
static cudaError_t tc_gemm(TcOperand A, TcOperand B, int Cn, TcOperand A2, TcOperand B2, int Cn2, float *C, int ldc, int I, int J,
                           float alpha, bool accumulate, float *partials, int splits_max, cudaStream_t stream) {
    const int BN = J > 128 ? 256 : (J > 64 ? 128 : 64);
    CUtensorMap maps[4];
    if (!tc_map(&maps[0], A, I, Cn, kTBM) || !tc_map(&maps[1], B, J, Cn, BN)) return cudaErrorInvalidValue;
    maps[2] = maps[0];
    maps[3] = maps[1];
    if (A2.p && (!tc_map(&maps[2], A2, I, Cn2, kTBM) || !tc_map(&maps[3], B2, J, Cn2, BN))) return cudaErrorInvalidValue;
    TcGemmArgs g = {};
    g.I = I; g.J = J; g.ldc = ldc;
    g.kb1 = (Cn + kTBK - 1) / kTBK;
    g.kb2 = A2.p ? (Cn2 + kTBK - 1) / kTBK : 0;
    g.a_mn = A.mn; g.b_mn = B.mn;
    const int kb_all = g.kb1 + g.kb2, tiles = ((I + kTBM - 1) / kTBM) * ((J + BN - 1) / BN), sms = device_sm_count();
    int splits = 1;
    if (partials && ldc == J && sms > 0 && tiles * 2 <= sms) {
        splits = sms / tiles;
        if (splits > splits_max) splits = splits_max;
        if (splits > kb_all / 4) splits = kb_all / 4 > 0 ? kb_all / 4 : 1;   // at least four blocks per split
    }
    // Tail of the tile schedule: when the tiles left for the last round of the persistent CTAs would keep at most
    // half of the SMs busy, they are worked as twice as many tiles of half the width, which fills the round.
    if (splits == 1 && BN == 256 && B.mn && sms > 0 && tiles > sms && tiles % sms != 0 && 2 * (tiles % sms) <= sms &&
        J % 256 == 0)
        g.n_half = 2 * (tiles % sms);
    g.kb_per_split = (kb_all + splits - 1) / splits;
    g.splits = (kb_all + g.kb_per_split - 1) / g.kb_per_split;  // no empty split
    if (g.splits == 1) {
        g.C = C; g.alpha = alpha; g.accumulate = accumulate ? 1 : 0;
    } else {
        g.C = partials; g.alpha = 1.0f; g.accumulate = 0;
    }
    cudaError_t e = BN == 256 ? tc_gemm_bn<256>(maps, g, stream) : (BN == 128 ? tc_gemm_bn<128>(maps, g, stream) : tc_gemm_bn<64>(maps, g, stream));
    if (e != cudaSuccess || g.splits == 1) return e;
    const size_t n4 = (size_t)I * J / 4;
    tc_reduce_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, stream>>>((const float4 *)partials, g.splits, n4, alpha, accumulate ? 1 : 0, (float4 *)C);
    count_launch();
    return cudaGetLastError();
}

// ---- operand preparation ---------------------------------------------------------------------------
// Xd = x~ gamma_x / 127 as bf16 [M][K] (eight values per thread).
__global__ void __launch_bounds__(256) bw_dequant_kernel(const int8_t *xq, const float *gamma_x, int K, size_t n8, __nv_bfloat16 *xd) {
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= n8) return;
    const float s = gamma_x[(i * 8) / (size_t)K] * (1.0f / 127.0f);
    const uint2 w = reinterpret_cast<const uint2 *>(xq)[i];
    const uint32_t ww[2] = {w.x, w.y};
    uint32_t o[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const int c0 = (int)(int8_t)(ww[h >> 1] >> (16 * (h & 1))), c1 = (int)(int8_t)(ww[h >> 1] >> (16 * (h & 1) + 8));
        const __nv_bfloat162 v = __floats2bfloat162_rn((float)c0 * s, (float)c1 * s);
        o[h] = *reinterpret_cast<const uint32_t *>(&v);
    }
    reinterpret_cast<uint4 *>(xd)[i] = make_uint4(o[0], o[1], o[2], o[3]);
}

// Ternary codes of the packed matrix as a bf16 matrix T [N][K] of -1 / 0 / +1 (one packed word = 16 columns per thread).
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

// fp16 -> bf16, optionally times a per-row factor (the gate folded into B^T).
__global__ void __launch_bounds__(256) bw_half_to_bf16_kernel(const __half *src, const float *row_scale, int cols, size_t n, __nv_bfloat16 *dst) {
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    const float s = row_scale ? row_scale[i / (size_t)cols] : 1.0f;
    dst[i] = __float2bfloat16_rn(__half2float(src[i]) * s);
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

// dZ = dH * SiLU'(Z), rounded to bf16, and dZ * scale (the copy that enters dX next to gamma_W dY T).
__global__ void __launch_bounds__(256) bw_dz_kernel(const float *dh, const float *dact, size_t n, float scale, __nv_bfloat16 *dz,
                                                    __nv_bfloat16 *dz_scaled) {
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    const float v = dh[i] * dact[i];
    dz[i] = __float2bfloat16_rn(v);
    dz_scaled[i] = __float2bfloat16_rn(v * scale);
}

// From G[n][j] = sum_m dY[m][n] H[m][j]: dBt[n][j] = gate[n] G[n][j] (in place), dgate[n] = sum_j G[n][j] Bt[n][j].
// One warp per output channel n (its r values are contiguous).
__global__ void __launch_bounds__(256) bw_gate_kernel(float *G, const __half *Bt, const float *gate, int N, int r, float *dgate) {
    const int n = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (n >= N) return;
    float dg = 0.0f;
    const float gn = gate[n];
    for (int j = lane; j < r; j += 32) {
        const float v = G[(size_t)n * r + j];
        dg = fmaf(v, __half2float(Bt[(size_t)n * r + j]), dg);
        G[(size_t)n * r + j] = gn * v;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dg += __shfl_xor_sync(0xffffffffu, dg, o);
    if (dgate && lane == 0) dgate[n] = dg;
}

constexpr int kBwSplitsMax = 16;

struct BwLayout {
    size_t xq, gamma_x, xd, T, At_b, gBt, z, h_b, dh, dz_b, dzs_b, G, partials, total;
};
static BwLayout bw_layout(int64_t M, int64_t K, int64_t N, int32_t r) {
    BwLayout L;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += align_up(bytes, 256); return o; };
    const size_t rr = (size_t)(r > 0 ? r : 16);
    L.xq = take((size_t)M * K);
    L.gamma_x = take((size_t)M * 4);
    L.xd = take((size_t)M * K * 2);
    L.T = take((size_t)N * K * 2);
    L.At_b = take(rr * K * 2);
    L.gBt = take((size_t)N * rr * 2);
    L.z = take((size_t)M * rr * 4);
    L.h_b = take((size_t)M * rr * 2);
    L.dh = take((size_t)M * rr * 4);
    L.dz_b = take((size_t)M * rr * 2);
    L.dzs_b = take((size_t)M * rr * 2);
    L.G = take((size_t)N * rr * 4);
    const size_t big = (size_t)(M > N ? (M > K ? M : K) : (N > K ? N : K));
    L.partials = take((size_t)kBwSplitsMax * big * rr * 4);  // split contractions all have r as one output extent
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
    auto bf = [&](size_t off) { return (__nv_bfloat16 *)(ws + off); };
    auto blocks1 = [](size_t n) { return (unsigned)((n + 255) / 256); };
    const TcOperand none = {nullptr, 0, false};
    float *partials = (float *)(ws + L.partials);
    bool ok = true;
    auto gemm = [&](TcOperand A, TcOperand B, int Cn, TcOperand A2, TcOperand B2, int Cn2, float *C, int ldc, int I, int J, float alpha,
                    bool acc, bool may_split) {
        ok = ok && tc_gemm(A, B, Cn, A2, B2, Cn2, C, ldc, I, J, alpha, acc, may_split ? partials : nullptr, kBwSplitsMax, stream) == cudaSuccess;
    };
    const TcOperand dy_k = {(const __nv_bfloat16 *)dy, N, false};  // dY as [M rows][N contraction]
    const TcOperand dy_mn = {(const __nv_bfloat16 *)dy, N, true};  // dY as [N rows] contracted over its M stored rows
    const TcOperand x_k = {(const __nv_bfloat16 *)x, K, false}, x_mn = {(const __nv_bfloat16 *)x, K, true};

    if (grads->dW) {  // Algorithm 1, steps 1-2 again, then dW[n][k] = sum_m dY[m][n] Xd[m][k]
        PrologueParams pp = {};
        pp.x = (const __nv_bfloat16 *)x;
        pp.xq = (int8_t *)(ws + L.xq);
        pp.gamma_x = (float *)(ws + L.gamma_x);
        pp.M = Mi;
        pp.K = K;
        pp.flags = HGF_FLAG_NO_PDL;
        if (launch_quant(pp, GemmPrologueExtra{}, stream) != cudaSuccess) return HGF_ERR_CUDA;
        const size_t n8 = (size_t)M * K / 8;
        bw_dequant_kernel<<<blocks1(n8), 256, 0, stream>>>(pp.xq, pp.gamma_x, K, n8, bf(L.xd));
        count_launch();
        gemm(dy_mn, TcOperand{bf(L.xd), K, true}, Mi, none, none, 0, grads->dW, K, N, K, 1.0f, false, false);
    }
    const bool fold = gamma > 1e-20f;  // the low-rank term of dX rides in the same contraction, pre-divided by gamma_W
    if (grads->dx) {
        const int steps = (int)(padded_k(d_in) / 256);
        const size_t n_words = (size_t)row_tiles(d_out) * steps * 256;
        bw_expand_ternary_kernel<<<blocks1(n_words), 256, 0, stream>>>((const uint32_t *)packed, N, K, steps, n_words, bf(L.T));
        count_launch();
    }
    const TcOperand T_mn = {bf(L.T), K, true};  // T [N][K]: rows k of the product, contracted over n
    if (!r) {
        if (grads->dx) gemm(dy_k, T_mn, N, none, none, 0, grads->dx, K, Mi, K, gamma, false, false);
        return (ok && cudaGetLastError() == cudaSuccess) ? HGF_OK : HGF_ERR_CUDA;
    }
    float *z = (float *)(ws + L.z), *dh = (float *)(ws + L.dh), *G = grads->dBt ? grads->dBt : (float *)(ws + L.G);
    bw_half_to_bf16_kernel<<<blocks1((size_t)r * K), 256, 0, stream>>>((const __half *)At, nullptr, K, (size_t)r * K, bf(L.At_b));
    bw_half_to_bf16_kernel<<<blocks1((size_t)N * r), 256, 0, stream>>>((const __half *)Bt, gate, r, (size_t)N * r, bf(L.gBt));
    count_launch(2);
    const TcOperand At_k = {bf(L.At_b), K, false}, At_mn = {bf(L.At_b), K, true};
    gemm(x_k, At_k, K, none, none, 0, z, r, Mi, r, 1.0f, false, true);                                       // Z = x A
    bw_act_kernel<<<blocks1((size_t)M * r), 256, 0, stream>>>(z, (size_t)M * r, (flags & HGF_FLAG_NO_SILU) ? 1 : 0, bf(L.h_b));
    gemm(dy_k, TcOperand{bf(L.gBt), r, true}, N, none, none, 0, dh, r, Mi, r, 1.0f, false, true);            // dH = dY (g (.) B^T)
    bw_dz_kernel<<<blocks1((size_t)M * r), 256, 0, stream>>>(dh, z, (size_t)M * r, fold ? 1.0f / gamma : 1.0f, bf(L.dz_b), bf(L.dzs_b));
    count_launch(2);
    if (grads->dx) {                                                                                         // dX = gamma_W dY T + dZ A^T
        const TcOperand dzs_k = {bf(L.dzs_b), r, false};
        if (fold) {
            gemm(dy_k, T_mn, N, dzs_k, At_mn, r, grads->dx, K, Mi, K, gamma, false, false);
        } else {
            gemm(dy_k, T_mn, N, none, none, 0, grads->dx, K, Mi, K, gamma, false, false);
            gemm(dzs_k, At_mn, r, none, none, 0, grads->dx, K, Mi, K, 1.0f, true, false);
        }
    }
    if (grads->dAt)                                                                                          // dA^T[j][k] = sum_m dZ[m][j] x[m][k]
        gemm(TcOperand{bf(L.dz_b), r, true}, x_mn, Mi, none, none, 0, grads->dAt, K, r, K, 1.0f, false, true);
    if (grads->dBt || grads->dgate) {                                                                        // G[n][j] = sum_m dY[m][n] H[m][j]
        gemm(dy_mn, TcOperand{bf(L.h_b), r, true}, Mi, none, none, 0, G, r, N, r, 1.0f, false, true);
        bw_gate_kernel<<<(unsigned)((N + 7) / 8), 256, 0, stream>>>(G, (const __half *)Bt, gate, N, r, grads->dgate);
        count_launch();
    }
    return (ok && cudaGetLastError() == cudaSuccess) ? HGF_OK : HGF_ERR_CUDA;
}
