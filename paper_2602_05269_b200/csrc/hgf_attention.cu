// Causal differential attention forward (paper, Section 2.4, Definition "Differential Attention"):
//     O = ( Softmax(Q1 K1^T / sqrt(d_h)) - lambda * Softmax(Q2 K2^T / sqrt(d_h)) ) V
// on the outputs of the HGF attention projections (Definition "HGF Attention Projections": Q, K of
// width d, V of width d / 2), per batch element and head.
//
#include <cmath>

#include "hgf_tc.cuh"

namespace hgf {

struct AttnParams {
    const __nv_bfloat16 *q, *k, *v;  // q, k [B*L][2*h*dh]; v [B*L][h*dh]
    void *out;                       // [B*L][h*dh] fp32 or bf16
    int B, L, h;
    float lambda, out_scale, scale_log2;  // scale_log2 = log2(e) / sqrt(dh)
    uint32_t flags;
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}

// One CTA of twelve warps per (batch element, head, tile of 128 queries), both streams:
//   warp 0      TMA producer: the two query tiles once, then per key tile K of stream 1, K of stream 2 and V
//               (KV keys: 128 for head_dim 64, 64 for head_dim 128; 128-byte swizzle, three stages)
//   warp 1      one lane issues tcgen05.mma.kind::f16: S_s = Q_s K_s^T (128 x KV, fp32, tensor memory), and
//               O_s += P_s V with P_s (bf16) read from tensor memory and V read from its stored form
//               (key rows of 128 bytes: the second operand with its row index contiguous)
//   warps 4-7   softmax of stream 1, warps 8-11 of stream 2: a thread owns one query row; it reads S_s
//               (tcgen05.ld), keeps a reference maximum and the sum, rescales its row of O_s in tensor memory
//               when the maximum moved far, and writes P_s = exp2(scale (s - reference)) as bf16 pairs (tcgen05.st)
// The issuer takes the streams in turn - P_s V of tile j, then S_s of tile j + 1 - so that one stream's
// matrix products run under the other stream's exponentials.  Tensor-memory columns: S_1, S_2, O_1, O_2,
// P_1, P_2 = 3 KV + 2 head_dim <= 512.  At the end O_1 / l_1 - lambda O_2 / l_2 is formed from the two
// accumulators by the thread pair that owns the row.  Every wait is bounded.
constexpr int kTaBM = 128, kTaThreads = 384, kTaStages = 3;
constexpr float kTaSlack = 8.0f;

template <int DH>
struct TaCfg {
    static constexpr int KV = DH == 64 ? 128 : 64, NBLK = DH / 64;
    static constexpr int Q_BYTES = NBLK * kTaBM * 128;             // one stream's query tile
    static constexpr int K_BYTES = NBLK * KV * 128, V_BYTES = NBLK * KV * 128, V_BLOCK = KV * 128;
    static constexpr int STAGE = 2 * K_BYTES + V_BYTES;
    static constexpr int OFF_RING = 2 * Q_BYTES, OFF_BAR = OFF_RING + kTaStages * STAGE;
    static constexpr int BAR_Q = 0, BAR_KVFULL = 1, BAR_KVEMPTY = 1 + kTaStages, BAR_SFULL = 1 + 2 * kTaStages,
                         BAR_PFULL = BAR_SFULL + 2, BAR_FINAL = BAR_PFULL + 2, BAR_COUNT = BAR_FINAL + 1;
    static constexpr int OFF_L = OFF_BAR + 256;                    // [2][128] floats
    static constexpr int SMEM_BYTES = OFF_L + 2 * kTaBM * 4 + 1024;
    static constexpr int COL_S = 0, COL_O = 2 * KV, COL_P = 2 * KV + 2 * DH;  // stream s: + s KV, + s DH, + s KV / 2
    static constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(KV >> 3) << 17) | ((uint32_t)(kTaBM >> 4) << 24);
    static constexpr uint32_t IDESC_PV = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(kTaBM >> 4) << 24);
};

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

template <int DH>
__global__ void __launch_bounds__(kTaThreads, 1)
ta_diff_attention_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                         const __grid_constant__ CUtensorMap tmap_v, const AttnParams p, unsigned int *status) {
    using C = TaCfg<DH>;
    constexpr int KV = C::KV;
    extern __shared__ uint8_t ta_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)ta_smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem), bar0 = sbase + C::OFF_BAR;
    auto bar = [&](int i) { return bar0 + 8u * i; };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::OFF_BAR + C::BAR_COUNT * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_BAR + C::BAR_COUNT * 8 + 4);
    float *s_l = reinterpret_cast<float *>(smem + C::OFF_L);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int L = p.L, h = p.h, nqt = (L + kTaBM - 1) / kTaBM;
    const int qt = nqt - 1 - (int)(blockIdx.x / (unsigned)(p.B * h));  // the long tiles (late queries) start first
    const int bh = (int)(blockIdx.x % (unsigned)(p.B * h)), b = bh / h, hd = bh % h;
    const int q0 = qt * kTaBM, tok0 = b * L;
    const int keys = q0 + kTaBM < L ? q0 + kTaBM : L;  // keys 0 .. keys - 1 are visible to this tile
    const int J = (keys + KV - 1) / KV;

    if (tid == 0) {
        mbar_init(bar(C::BAR_Q), 1);
        for (int s = 0; s < kTaStages; ++s) {
            mbar_init(bar(C::BAR_KVFULL + s), 1);
            mbar_init(bar(C::BAR_KVEMPTY + s), 1);
        }
        for (int st = 0; st < 2; ++st) {
            mbar_init(bar(C::BAR_SFULL + st), 1);
            mbar_init(bar(C::BAR_PFULL + st), 4);
        }
        mbar_init(bar(C::BAR_FINAL), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        fence_proxy_async();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        uint32_t issued[kTaStages] = {};
        bool ok = true;
        if (lane == 0) {
            mbar_arrive_expect_tx(bar(C::BAR_Q), 2 * C::Q_BYTES);
            for (int st = 0; st < 2; ++st)
                for (int blk = 0; blk < C::NBLK; ++blk)
                    tma_load_2d(sbase + st * C::Q_BYTES + blk * kTaBM * 128, &tmap_q, (st * h + hd) * DH + 64 * blk, tok0 + q0, bar(C::BAR_Q));
        }
        for (int j = 0; j < J; ++j) {
            const int s = j % kTaStages;
            ok = mbar_wait(bar(C::BAR_KVEMPTY + s), (uint32_t)((j / kTaStages) & 1) ^ 1u, abort_flag, status, 0xa00u + s);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;
            if (lane == 0) {
                const uint32_t dst = sbase + C::OFF_RING + s * C::STAGE, full = bar(C::BAR_KVFULL + s);
                mbar_arrive_expect_tx(full, C::STAGE);
                for (int blk = 0; blk < C::NBLK; ++blk) {
                    tma_load_2d(dst + blk * KV * 128, &tmap_k, hd * DH + 64 * blk, tok0 + j * KV, full);
                    tma_load_2d(dst + C::K_BYTES + blk * KV * 128, &tmap_k, (h + hd) * DH + 64 * blk, tok0 + j * KV, full);
                    tma_load_2d(dst + 2 * C::K_BYTES + blk * C::V_BLOCK, &tmap_v, hd * DH + 64 * blk, tok0 + j * KV, full);
                }
            }
            ++issued[s];
        }
        for (int q = 0; q < kTaStages; ++q)  // never leave with a copy in flight
            if (issued[q]) {
                const uint32_t par = (issued[q] - 1u) & 1u;
                for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar(C::BAR_KVFULL + q), par); ++i) {}
            }
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar(C::BAR_Q), 0); ++i) {}
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            bool ok = true;
            auto issue_s = [&](int st, int s) {  // S_st = Q_st K_st^T from stage s
                const uint32_t qa = sbase + st * C::Q_BYTES, ka = sbase + C::OFF_RING + s * C::STAGE + st * C::K_BYTES;
#pragma unroll
                for (int blk = 0; blk < C::NBLK; ++blk) {
                    const uint64_t adesc = make_sw128_desc(qa + blk * kTaBM * 128), bdesc = make_sw128_desc(ka + blk * KV * 128);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_f16(tmem_base + C::COL_S + st * KV, adesc + 2u * kk, bdesc + 2u * kk, C::IDESC_S, (blk | kk) ? 1u : 0u);
                }
                tc_commit(bar(C::BAR_SFULL + st));
            };
            auto issue_pv = [&](int st, int s, bool first) {  // O_st (+)= P_st V from stage s
                const uint64_t bdesc = make_sw128_mn_desc(sbase + C::OFF_RING + s * C::STAGE + 2 * C::K_BYTES, C::V_BLOCK);
#pragma unroll
                for (int kk = 0; kk < KV / 16; ++kk)
                    mma_f16_ts(tmem_base + C::COL_O + st * DH, tmem_base + C::COL_P + st * (KV / 2) + 8 * kk, bdesc + (uint64_t)(128 * kk),
                               C::IDESC_PV, (!first || kk) ? 1u : 0u);
            };
            ok = mbar_wait(bar(C::BAR_Q), 0, abort_flag, status, 0xa10u);
            ok = ok && mbar_wait(bar(C::BAR_KVFULL + 0), 0, abort_flag, status, 0xa11u);
            if (ok) {
                tc_fence_after();
                issue_s(0, 0);
                issue_s(1, 0);
            }
            for (int j = 0; ok && j < J; ++j) {
                const int s = j % kTaStages, s1 = (j + 1) % kTaStages;
                for (int st = 0; st < 2; ++st) {
                    if (!(ok = mbar_wait(bar(C::BAR_PFULL + st), (uint32_t)(j & 1), abort_flag, status, 0xa20u + st))) break;
                    tc_fence_after();
                    issue_pv(st, s, j == 0);
                    if (st == 1) tc_commit(bar(C::BAR_KVEMPTY + s));
                    if (j + 1 < J) {
                        if (st == 0 && !(ok = mbar_wait(bar(C::BAR_KVFULL + s1), (uint32_t)(((j + 1) / kTaStages) & 1), abort_flag, status, 0xa30u + s1)))
                            break;
                        tc_fence_after();
                        issue_s(st, s1);
                    }
                }
            }
            if (ok) tc_commit(bar(C::BAR_FINAL));
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ softmax of one stream, one row per thread
        const int st = warp >= 8 ? 1 : 0, quarter = warp & 3, row = 32 * quarter + lane, qi = q0 + row;
        const uint32_t lane_base = tmem_base + ((uint32_t)(32 * quarter) << 16);
        const uint32_t s_addr = lane_base + C::COL_S + st * KV, o_addr = lane_base + C::COL_O + st * DH, p_addr = lane_base + C::COL_P + st * (KV / 2);
        const float c = p.scale_log2;
        float m = -1e30f, l = 0.0f;
        bool ok = true;
        for (int j = 0; j < J; ++j) {
            ok = mbar_wait(bar(C::BAR_SFULL + st), (uint32_t)(j & 1), abort_flag, status, 0xa40u + st);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;
            tc_fence_after();
            const int k0 = j * KV;
            const bool diag = k0 + KV - 1 > q0;  // some key of the tile lies after some query of the tile
            // pass 1: the row's maximum (two chunks of 32 scores in flight)
            float mx = -1e30f;
#pragma unroll
            for (int cc = 0; cc < KV; cc += 64) {
                uint32_t v0[32], v1[32];
                tmem_ld32(s_addr + cc, v0);
                tmem_ld32(s_addr + cc + 32, v1);
                tmem_ld_wait();
                if (diag) {
#pragma unroll
                    for (int u = 0; u < 32; ++u) {
                        if (k0 + cc + u <= qi) mx = fmaxf(mx, __uint_as_float(v0[u]));
                        if (k0 + cc + 32 + u <= qi) mx = fmaxf(mx, __uint_as_float(v1[u]));
                    }
                } else {
                    float m0 = __uint_as_float(v0[0]), m1 = __uint_as_float(v1[0]);
#pragma unroll
                    for (int u = 1; u < 32; ++u) {
                        m0 = fmaxf(m0, __uint_as_float(v0[u]));
                        m1 = fmaxf(m1, __uint_as_float(v1[u]));
                    }
                    mx = fmaxf(mx, fmaxf(m0, m1));
                }
            }
            // The reference point of the exponentials follows the maximum only when the maximum has moved by more
            // than kTaSlack (in log2 units): probabilities then stay below 2^kTaSlack, and O and l are rescaled
            // rarely instead of at nearly every tile.  (The final O / l does not depend on the reference point.)
            float m_new = m;
            if ((mx - m) * c > (j == 0 ? -1.0f : kTaSlack)) m_new = mx;
            if (j > 0 && __any_sync(0xffffffffu, m_new != m)) {
                const float alpha = ex2_approx((m - m_new) * c);
                l *= alpha;
#pragma unroll
                for (int cc = 0; cc < DH; cc += 32) {
                    uint32_t v[32];
                    tmem_ld32(o_addr + cc, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int u = 0; u < 32; ++u) v[u] = __float_as_uint(__uint_as_float(v[u]) * alpha);
                    tmem_st32(o_addr + cc, v);
                }
            }
            // pass 2: probabilities as bf16 pairs, 64 keys at a time
            const float mc = m_new * c;
#pragma unroll
            for (int cc = 0; cc < KV; cc += 64) {
                uint32_t v0[32], v1[32], pk[32];
                tmem_ld32(s_addr + cc, v0);
                tmem_ld32(s_addr + cc + 32, v1);
                tmem_ld_wait();
                if (diag) {
#pragma unroll
                    for (int u = 0; u < 32; ++u) {
                        if (k0 + cc + u > qi) v0[u] = 0xff800000u;       // -inf: probability 0
                        if (k0 + cc + 32 + u > qi) v1[u] = 0xff800000u;
                    }
                }
                float l0 = 0.0f, l1 = 0.0f;
#pragma unroll
                for (int u = 0; u < 32; u += 2) {
                    const float pa0 = ex2_approx(fmaf(__uint_as_float(v0[u]), c, -mc)), pa1 = ex2_approx(fmaf(__uint_as_float(v0[u + 1]), c, -mc));
                    const float pb0 = ex2_approx(fmaf(__uint_as_float(v1[u]), c, -mc)), pb1 = ex2_approx(fmaf(__uint_as_float(v1[u + 1]), c, -mc));
                    l0 += pa0 + pa1;
                    l1 += pb0 + pb1;
                    pk[u >> 1] = pack_bf16(pa0, pa1);
                    pk[16 + (u >> 1)] = pack_bf16(pb0, pb1);
                }
                l += l0 + l1;
                tmem_st32(p_addr + (cc >> 1), pk);
            }
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(C::BAR_PFULL + st));
            m = m_new;
        }
        if (ok) {
            ok = mbar_wait(bar(C::BAR_FINAL), 0, abort_flag, status, 0xa50u);
            ok = __all_sync(0xffffffffu, ok);
        }
        s_l[st * kTaBM + row] = l;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp >= 4 && !*abort_flag) {
        // (O_1 / l_1 - lambda O_2 / l_2) out_scale: stream s's thread of a row writes half s of the row's columns
        const int st = warp >= 8 ? 1 : 0, quarter = warp & 3, row = 32 * quarter + lane, qi = q0 + row;
        const uint32_t lane_base = tmem_base + ((uint32_t)(32 * quarter) << 16);
        const float w1 = p.out_scale / s_l[row], w2 = p.out_scale * p.lambda / s_l[kTaBM + row];
        const size_t obase = (size_t)(tok0 + qi) * ((size_t)h * DH) + (size_t)hd * DH;
#pragma unroll
        for (int cc = st * (DH / 2); cc < (st + 1) * (DH / 2); cc += 32) {
            uint32_t v1[32], v2[32];
            tmem_ld32(lane_base + C::COL_O + cc, v1);
            tmem_ld32(lane_base + C::COL_O + DH + cc, v2);
            tmem_ld_wait();
            if (qi < L) {
                if (p.flags & HGF_FLAG_OUT_BF16) {
                    uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(p.out) + obase + cc);
#pragma unroll
                    for (int u = 0; u < 32; u += 8) {
                        uint32_t o[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            o[e] = pack_bf16(__uint_as_float(v1[u + 2 * e]) * w1 - __uint_as_float(v2[u + 2 * e]) * w2,
                                             __uint_as_float(v1[u + 2 * e + 1]) * w1 - __uint_as_float(v2[u + 2 * e + 1]) * w2);
                        dst[u >> 3] = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                } else {
                    float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.out) + obase + cc);
#pragma unroll
                    for (int u = 0; u < 32; u += 4)
                        dst[u >> 2] = make_float4(__uint_as_float(v1[u]) * w1 - __uint_as_float(v2[u]) * w2,
                                                  __uint_as_float(v1[u + 1]) * w1 - __uint_as_float(v2[u + 1]) * w2,
                                                  __uint_as_float(v1[u + 2]) * w1 - __uint_as_float(v2[u + 2]) * w2,
                                                  __uint_as_float(v1[u + 3]) * w1 - __uint_as_float(v2[u + 3]) * w2);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

template <int DH>
static cudaError_t launch_attention_tc(const AttnParams &p, cudaStream_t stream) {
    using C = TaCfg<DH>;
    static std::atomic<unsigned long long> attr_done{0};
    cudaError_t e = ensure_dynamic_smem(ta_diff_attention_kernel<DH>, C::SMEM_BYTES, attr_done);
    if (e != cudaSuccess) return e;
    unsigned int *status = device_status_word();
    if (!status) return cudaErrorMemoryAllocation;
    const uint64_t rows = (uint64_t)p.B * p.L, dq = (uint64_t)2 * p.h * DH, dv = (uint64_t)p.h * DH;
    CUtensorMap mq, mk, mv;
    if (!make_map_2d(&mq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p.q, dq, rows, dq * 2, 64, kTaBM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&mk, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p.k, dq, rows, dq * 2, 64, C::KV, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&mv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p.v, dv, rows, dv * 2, 64, C::KV, CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;
    const unsigned grid = (unsigned)(((p.L + kTaBM - 1) / kTaBM) * p.B * p.h);
    ta_diff_attention_kernel<DH><<<grid, kTaThreads, C::SMEM_BYTES, stream>>>(mq, mk, mv, p, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hgf

using namespace hgf;

extern "C" hgf_status hgf_diff_attention_forward(const void *q, const void *k, const void *v, int64_t B, int64_t L,
                                                 int32_t n_heads, int32_t head_dim, float lambda, float out_scale, void *out,
                                                 uint32_t flags, void *stream) {
    if (!q || !k || !v || !out || B <= 0 || L <= 0 || n_heads <= 0) return HGF_ERR_INVALID_ARG;
    if (flags & ~HGF_FLAG_OUT_BF16) return HGF_ERR_INVALID_ARG;
    if ((head_dim != 64 && head_dim != 128) || B > 65535 || n_heads > 65535 || L > (1 << 24)) return HGF_ERR_UNSUPPORTED_SHAPE;
    // token rows and CTAs are counted in 32 bits
    if (B * L > 0x7fffffffll || (uint64_t)B * (uint64_t)n_heads * (uint64_t)((L + kTaBM - 1) / kTaBM) > 0x7fffffffull) return HGF_ERR_UNSUPPORTED_SHAPE;
    if ((((uintptr_t)q) | ((uintptr_t)k) | ((uintptr_t)v) | ((uintptr_t)out)) & 15u) return HGF_ERR_MISALIGNED;
    AttnParams p = {};
    p.q = (const __nv_bfloat16 *)q;
    p.k = (const __nv_bfloat16 *)k;
    p.v = (const __nv_bfloat16 *)v;
    p.out = out;
    p.B = (int)B;
    p.L = (int)L;
    p.h = n_heads;
    p.lambda = lambda;
    p.out_scale = out_scale;
    p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)head_dim));
    p.flags = flags;
    const cudaError_t e = head_dim == 64 ? launch_attention_tc<64>(p, (cudaStream_t)stream) : launch_attention_tc<128>(p, (cudaStream_t)stream);
    return e == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
}

extern "C" double hgf_diff_lambda0(double head_dim) { return 0.8 - 0.6 * exp(-0.3 * head_dim); }
