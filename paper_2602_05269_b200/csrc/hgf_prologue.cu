// Prologue kernels: per-token absmax int8 quantisation (Algorithm 1, steps 1-2) and the LoRA
// down-projection H = SiLU(x A) (Algorithm 1, steps 5-6).
#include "hgf_common.cuh"

namespace hgf {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ int warp_sum_i(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Round-to-nearest-even of the exact quotient 127 x / gamma for a bf16 x.
//
// Reference form: 127 x is exact in fp32, the IEEE division is correctly rounded and k + 1/2 is
// representable, so rintf of the rounded quotient equals the rounding of the exact one.
__device__ __forceinline__ int quant1_div(float x, float gamma) {
    float q = rintf(__fdiv_rn(127.0f * x, gamma));
    q = fminf(fmaxf(q, -127.0f), 127.0f);
    return __float2int_rn(q);
}
// Division- and conversion-free form, for gamma = max |x| over bf16 values (so gamma is a bf16 value
// itself, i.e. not the 1e-5 floor).  Adding 1.5 * 2^23 in one fma rounds x * (127 / gamma) to an
// integer (nearest, ties to even) in the low mantissa bits - a candidate that can only be wrong on
// an exact tie of the true quotient.  The residual 127 x - q gamma is exact in one fma (127 x and
// q gamma each have at most 15 significant bits), and the exact quotient is q + residual / gamma:
// off a tie the candidate is always right (checked over every pair of bf16 mantissas and every
// exponent gap in exact arithmetic), so it stands unless 2 |residual| = gamma with q odd: a tie goes
// to the even neighbour, one step towards the residual's sign (2 |residual| > gamma cannot occur).
// No F2I / FRND: those run at an eighth of the FMA rate and bounded the quantisation kernels.
struct QuantScale {
    float gamma, half_gamma, inv127;  // inv127 = 127 / gamma
    bool fast;                        // gamma is a bf16 value
};
__device__ __forceinline__ QuantScale make_quant_scale(float gamma) {
    QuantScale s;
    s.gamma = gamma;
    s.half_gamma = 0.5f * gamma;
    s.inv127 = __fdiv_rn(127.0f, gamma);
    s.fast = (__float_as_uint(gamma) & 0xffffu) == 0u;
    return s;
}
// Largest magnitude of the eight bf16 values of a 16-byte unit, on the bit patterns: without the sign
// bit a bf16 pattern orders like its magnitude, so a packed 16-bit maximum does two values at a time.
__device__ __forceinline__ uint32_t absmax8_bits(uint32_t acc, const uint4 &v) {
    acc = __vmaxu2(acc, v.x & 0x7fff7fffu);
    acc = __vmaxu2(acc, v.y & 0x7fff7fffu);
    acc = __vmaxu2(acc, v.z & 0x7fff7fffu);
    return __vmaxu2(acc, v.w & 0x7fff7fffu);
}
__device__ __forceinline__ float absmax_bits_to_float(uint32_t acc) {
    const uint32_t hi = acc >> 16, lo = acc & 0xffffu;
    return __uint_as_float((hi > lo ? hi : lo) << 16);
}
// The eight values of a 16-byte unit -> eight int8 (two words), their sum added to `sum`.
// The fast form, arranged for throughput: the candidate's low byte is already the low
// byte of the magic-constant sum's bit pattern (its mantissa holds 2^22 + q in two's complement), so
// the bytes are packed straight from those patterns, and the tie test of all eight values is one
// predicate; only a unit that holds an exact tie (rare) goes back over its values to move the odd
// candidates to their even neighbours.
__device__ __forceinline__ uint2 quant8(const uint4 &v, const QuantScale &s, int &sum) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t b[8];
    if (s.fast) {
        constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23
        float xf[8], res[8];
        bool tie = false;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            xf[e] = (e & 1) ? bf16hi_to_float(w[e >> 1]) : bf16lo_to_float(w[e >> 1]);
            const float tm = fmaf(xf[e], s.inv127, kMagic);
            res[e] = fmaf(kMagic - tm, s.gamma, 127.0f * xf[e]);  // 127 x - q gamma, exact
            tie = tie || fabsf(res[e]) == s.half_gamma;
            b[e] = __float_as_uint(tm);
        }
        if (tie) {
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (fabsf(res[e]) == s.half_gamma && (b[e] & 1u)) b[e] += res[e] > 0.0f ? 1u : 0xffffffffu;
        }
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e)
            b[e] = (uint32_t)quant1_div((e & 1) ? bf16hi_to_float(w[e >> 1]) : bf16lo_to_float(w[e >> 1]), s.gamma);
    }
    uint32_t o[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t p01 = __byte_perm(b[4 * h], b[4 * h + 1], 0x0040), p23 = __byte_perm(b[4 * h + 2], b[4 * h + 3], 0x0040);
        o[h] = __byte_perm(p01, p23, 0x5410);
        sum = __dp4a((int)o[h], 0x01010101, sum);
    }
    return make_uint2(o[0], o[1]);
}

// One block quantises one token row.
__device__ __forceinline__ void quant_row(const PrologueParams &p, int m, float *tok_sc = nullptr, float gw_over_127 = 0.0f) {
    __shared__ float s_red_f[kWarps];
    __shared__ int s_red_i[kWarps];
    const int K = p.K, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint4 *xv = reinterpret_cast<const uint4 *>(p.x + (size_t)m * K);
    const int nv = K / 8;

    uint32_t abits = 0u;
    for (int i = tid; i < nv; i += kThreads) abits = absmax8_bits(abits, xv[i]);
    float amax = warp_max(absmax_bits_to_float(abits));
    if (lane == 0) s_red_f[warp] = amax;
    __syncthreads();
    float g = s_red_f[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) g = fmaxf(g, s_red_f[w]);
    g = fmaxf(g, 1e-5f);
    const QuantScale qs = make_quant_scale(g);

    int sum = 0;
    uint2 *qv = reinterpret_cast<uint2 *>(p.xq + (size_t)m * K);
    uint2 *dq = p.dbg_xq ? reinterpret_cast<uint2 *>(p.dbg_xq + (size_t)m * K) : nullptr;
    for (int i = tid; i < nv; i += kThreads) {
        const uint2 o = quant8(xv[i], qs, sum);
        qv[i] = o;
        if (dq) dq[i] = o;
    }
    sum = warp_sum_i(sum);
    if (lane == 0) s_red_i[warp] = sum;
    __syncthreads();
    if (tid == 0) {
        int tot = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) tot += s_red_i[w];
        if (p.row_sum) p.row_sum[m] = tot;
        if (tok_sc) tok_sc[m] = g * gw_over_127;
        p.gamma_x[m] = g;
        if (p.dbg_gamma_x) p.dbg_gamma_x[m] = g;
    }
}

// ---- LayerNorm front end (Appendix E, ScientificBitLinear.forward) -----------------------------------
// One binary32 operation each, in this order: the rounded value decides the int8 code.
__device__ __forceinline__ float ln_value(float x, float mean, float rstd, float w, float b) {
    return __fadd_rn(__fmul_rn(__fmul_rn(__fsub_rn(x, mean), rstd), w), b);
}
__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = (e & 1) ? bf16hi_to_float(w[e >> 1]) : bf16lo_to_float(w[e >> 1]);
}
__device__ __forceinline__ double block_sum_d(double v, double *s_red, int lane, int warp) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();  // the previous use of s_red is over
    if (lane == 0) s_red[warp] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += s_red[w];
    return t;
}
// One block normalises and quantises one token row: mean and variance (two passes, summed in double),
// the row's largest |xn|, then the codes - the listing's binary32 arithmetic: scale = 127 / gamma_x,
// code = rint(xn * scale).  The row is read from L1/L2 in every pass.
__device__ __forceinline__ void quant_row_ln(const PrologueParams &p, const FrontEnd &fe, int m, float *tok_sc, float gw_over_127) {
    __shared__ double s_red_d[kWarps];
    __shared__ float s_red_f[kWarps];
    __shared__ int s_red_i[kWarps];
    const int K = p.K, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint4 *xv = reinterpret_cast<const uint4 *>(p.x + (size_t)m * K);
    const int nv = K / 8;
    float f[8];

    double sum = 0.0;
    for (int i = tid; i < nv; i += kThreads) {
        unpack8(xv[i], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) sum += (double)f[e];
    }
    const double mean_d = block_sum_d(sum, s_red_d, lane, warp) / (double)K;
    double ss = 0.0;
    for (int i = tid; i < nv; i += kThreads) {
        unpack8(xv[i], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const double d = (double)f[e] - mean_d;
            ss += d * d;
        }
    }
    const double var = block_sum_d(ss, s_red_d, lane, warp) / (double)K;
    const float mean = (float)mean_d, rstd = (float)(1.0 / sqrt(var + (double)fe.eps));

    float amax = 0.0f;
    for (int i = tid; i < nv; i += kThreads) {
        unpack8(xv[i], f);
        const float4 w0 = *reinterpret_cast<const float4 *>(fe.ln_w + 8 * i), w1 = *reinterpret_cast<const float4 *>(fe.ln_w + 8 * i + 4);
        const float4 b0 = *reinterpret_cast<const float4 *>(fe.ln_b + 8 * i), b1 = *reinterpret_cast<const float4 *>(fe.ln_b + 8 * i + 4);
        const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w}, b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(ln_value(f[e], mean, rstd, w[e], b[e])));
    }
    amax = warp_max(amax);
    if (lane == 0) s_red_f[warp] = amax;
    __syncthreads();
    float g = s_red_f[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) g = fmaxf(g, s_red_f[w]);
    g = fmaxf(g, 1e-5f);
    const float scale = __fdiv_rn(127.0f, g);

    int sum_q = 0;
    uint2 *qv = reinterpret_cast<uint2 *>(p.xq + (size_t)m * K);
    uint2 *dq = p.dbg_xq ? reinterpret_cast<uint2 *>(p.dbg_xq + (size_t)m * K) : nullptr;
    for (int i = tid; i < nv; i += kThreads) {
        unpack8(xv[i], f);
        const float4 w0 = *reinterpret_cast<const float4 *>(fe.ln_w + 8 * i), w1 = *reinterpret_cast<const float4 *>(fe.ln_w + 8 * i + 4);
        const float4 b0 = *reinterpret_cast<const float4 *>(fe.ln_b + 8 * i), b1 = *reinterpret_cast<const float4 *>(fe.ln_b + 8 * i + 4);
        const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w}, b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
        uint32_t c[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            float q = rintf(__fmul_rn(ln_value(f[e], mean, rstd, w[e], b[e]), scale));
            q = fminf(fmaxf(q, -127.0f), 127.0f);
            c[e] = (uint32_t)__float2int_rn(q);
        }
        uint32_t o[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t p01 = __byte_perm(c[4 * h], c[4 * h + 1], 0x0040), p23 = __byte_perm(c[4 * h + 2], c[4 * h + 3], 0x0040);
            o[h] = __byte_perm(p01, p23, 0x5410);
            sum_q = __dp4a((int)o[h], 0x01010101, sum_q);
        }
        qv[i] = make_uint2(o[0], o[1]);
        if (dq) dq[i] = make_uint2(o[0], o[1]);
    }
    sum_q = warp_sum_i(sum_q);
    if (lane == 0) s_red_i[warp] = sum_q;
    __syncthreads();
    if (tid == 0) {
        int tot = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) tot += s_red_i[w];
        if (p.row_sum) p.row_sum[m] = tot;
        if (tok_sc) tok_sc[m] = g * gw_over_127;
        p.gamma_x[m] = g;
        if (p.dbg_gamma_x) p.dbg_gamma_x[m] = g;
        if (fe.dbg_mean) fe.dbg_mean[m] = mean;
        if (fe.dbg_rstd) fe.dbg_rstd[m] = rstd;
    }
}

__device__ __forceinline__ void mma_tf32(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ldg_nc_u4(const void *ptr) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(ptr));
    return v;
}

// One block computes 16 columns of H (rows 16 jt .. 16 jt + 15 of A^T) for up to 16 tokens:
// H[m][j] = act(sum_k x[m][k] A[k][j]) on the warp-level tf32 MMA.  bf16 and fp16 values are both
// exactly representable in tf32 (8 exponent, 10 mantissa bits), so the products are formed from
// exact inputs and accumulated in fp32.  The rows of A^T are the 16-row operand, the tokens the
// 8-column operand; the warps split K in 32-element chunks and their partial sums are added in a
// fixed order through shared memory.  NT = number of 8-token tiles.
// With `hpart` the block covers only the 32-column chunks [cbeg, cend) of K and parks its raw sums
// there (MMA accumulator layout: [register][lane]); the GEMV adds the slices and applies the SiLU.
template <int NT>
__device__ __forceinline__ void lora_down_tile(const PrologueParams &p, int jt, int cbeg, int cend, float *hpart) {
    __shared__ float s_red[kWarps][NT * 4][32];
    const int K = p.K, M = p.M, r = p.r, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const __half *rowA = p.At + (size_t)(16 * jt + g) * K + 8 * t;
    const __half *rowB = rowA + (size_t)8 * K;
    const __nv_bfloat16 *xr[NT];
    bool tok_ok[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        tok_ok[nt] = g + 8 * nt < M;
        xr[nt] = p.x + (size_t)(tok_ok[nt] ? g + 8 * nt : 0) * K + 8 * t;
    }
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[nt][c] = 0.0f;

    const int nchunks = cend;
    constexpr int U = 4;  // chunks in flight per warp
    for (int c0 = cbeg + warp; c0 < nchunks; c0 += U * kWarps) {
        uint4 av[U], bv[U], xv[U][NT];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = c0 + u * kWarps;
            av[u] = bv[u] = make_uint4(0u, 0u, 0u, 0u);
            if (c < nchunks) {
                av[u] = ldg_nc_u4(rowA + 32 * c);
                bv[u] = ldg_nc_u4(rowB + 32 * c);
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                xv[u][nt] = make_uint4(0u, 0u, 0u, 0u);
                if (c < nchunks && tok_ok[nt]) xv[u][nt] = *reinterpret_cast<const uint4 *>(xr[nt] + 32 * c);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t aw[4] = {av[u].x, av[u].y, av[u].z, av[u].w};
            const uint32_t bw[4] = {bv[u].x, bv[u].y, bv[u].z, bv[u].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                // elements 2 i and 2 i + 1 of this lane's eight take the k slots t and t + 4 of the MMA
                const float2 fa = __half22float2(*reinterpret_cast<const __half2 *>(&aw[i]));
                const float2 fb = __half22float2(*reinterpret_cast<const __half2 *>(&bw[i]));
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint32_t xw = (&xv[u][nt].x)[i];
                    mma_tf32(acc[nt], __float_as_uint(fa.x), __float_as_uint(fb.x), __float_as_uint(fa.y),
                             __float_as_uint(fb.y), xw << 16, xw & 0xffff0000u);
                }
            }
        }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) s_red[warp][nt * 4 + c][lane] = acc[nt][c];
    __syncthreads();
    if (tid < NT * 4 * 32) {
        const int idx = tid >> 5, ln = tid & 31, nt = idx >> 2, c = idx & 3;
        float z = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) z += s_red[w][idx][ln];
        // accumulator register c of lane (g, t): row g + 8 (c >> 1), token 8 nt + 2 t + (c & 1)
        const int j = 16 * jt + (ln >> 2) + 8 * (c >> 1), m = 8 * nt + 2 * (ln & 3) + (c & 1);
        if (hpart) {
            hpart[idx * 32 + ln] = z;
        } else if (m < M) {
            const float h = (p.flags & HGF_FLAG_NO_SILU) ? z : silu_f(z);
            const size_t o = (size_t)m * r + j;
            p.h[o] = h;
            if (p.dbg_h) p.dbg_h[o] = h;
            if (p.h_hi) {
                const __half hi = __float2half_rn(h);
                p.h_hi[o] = hi;
                p.h_lo[o] = __float2half_rn(h - __half2float(hi));
            }
        }
    }
}

__device__ __forceinline__ void lora_down_block(const PrologueParams &p, int jt, int cbeg, int cend, float *hpart) {
    if (p.M <= 8) lora_down_tile<1>(p, jt, cbeg, cend, hpart); else lora_down_tile<2>(p, jt, cbeg, cend, hpart);
}

// Many rows of up to 4096 elements (quantisation alone): one warp per token row, the row held in registers between the maximum and
// the rounding (U 16-byte units per lane), so a row costs one trip to memory, no block-wide
// synchronisation, and the per-row overhead (scale, reductions) is spread over 8 U elements per lane.
template <int U>
__global__ void __launch_bounds__(kThreads) quant_rows_kernel(const PrologueParams p, const GemmPrologueExtra x) {
    asm volatile("griddepcontrol.wait;\n" ::: "memory");  // see gemm_prologue_kernel
    const int lane = threadIdx.x & 31, m = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (m >= p.M) return;
    const int K = p.K, nv = K / 8;
    const uint4 *xv = reinterpret_cast<const uint4 *>(p.x + (size_t)m * K);
    uint4 v[U];
    uint32_t abits = 0u;
#pragma unroll
    for (int u = 0; u < U; ++u) v[u] = lane + 32 * u < nv ? xv[lane + 32 * u] : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int u = 0; u < U; ++u) abits = absmax8_bits(abits, v[u]);
    const float g = fmaxf(warp_max(absmax_bits_to_float(abits)), 1e-5f);
    const QuantScale qs = make_quant_scale(g);
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");  // the row is in registers: the next launch may be set up
    int sum = 0;
    uint2 *qv = reinterpret_cast<uint2 *>(p.xq + (size_t)m * K);
    uint2 *dq = p.dbg_xq ? reinterpret_cast<uint2 *>(p.dbg_xq + (size_t)m * K) : nullptr;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (lane + 32 * u < nv) {
            const uint2 o = quant8(v[u], qs, sum);
            qv[lane + 32 * u] = o;
            if (dq) dq[lane + 32 * u] = o;
        }
    }
    sum = warp_sum_i(sum);
    if (lane == 0) {
        if (p.row_sum) p.row_sum[m] = sum;
        if (x.tok_sc) x.tok_sc[m] = g * x.gw_over_127;
        p.gamma_x[m] = g;
        if (p.dbg_gamma_x) p.dbg_gamma_x[m] = g;
    }
}

__global__ void __launch_bounds__(kThreads) quant_kernel(const PrologueParams p, const GemmPrologueExtra x) {
    quant_row(p, blockIdx.x, x.tok_sc, x.gw_over_127);
}

// Programmatic dependent launch: no-ops when the launch carries no such attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }

// Decode prologue: blocks [0, M) quantise one token each; the others compute 16 columns of H each,
// over all of K, or - with a scratch for partial sums - over one K slice each (slice-major), which
// shortens the chain of dependent loads from K / 1024 rounds to one or two.
__global__ void __launch_bounds__(kThreads) decode_prologue_kernel(const PrologueParams p) {
    pdl_launch_dependents();  // the GEMV that follows may start streaming its weights
    pdl_wait();               // x, and the workspace this kernel overwrites, belong to earlier work
    if ((int)blockIdx.x < p.M)
        quant_row(p, blockIdx.x);
    else if (p.hpart) {
        const int lb = blockIdx.x - p.M, jts = p.r / 16, sl = lb / jts, jt = lb - sl * jts;
        const int per = prologue_slice_k(p.M) / 32, cbeg = sl * per, cend = cbeg + per < p.K / 32 ? cbeg + per : p.K / 32;
        lora_down_block(p, jt, cbeg, cend, p.hpart + ((size_t)jt * p.nslices + sl) * 256);
    } else {
        lora_down_block(p, blockIdx.x - p.M, 0, p.K / 32, nullptr);
    }
}

// The same with the LayerNorm front end: the row blocks normalise before they quantise; the
// correction path's blocks read the raw x as before.
__global__ void __launch_bounds__(kThreads) decode_prologue_ln_kernel(const PrologueParams p, const FrontEnd fe) {
    pdl_launch_dependents();
    pdl_wait();
    if ((int)blockIdx.x < p.M)
        quant_row_ln(p, fe, blockIdx.x, nullptr, 0.0f);
    else if (p.hpart) {
        const int lb = blockIdx.x - p.M, jts = p.r / 16, sl = lb / jts, jt = lb - sl * jts;
        const int per = prologue_slice_k(p.M) / 32, cbeg = sl * per, cend = cbeg + per < p.K / 32 ? cbeg + per : p.K / 32;
        lora_down_block(p, jt, cbeg, cend, p.hpart + ((size_t)jt * p.nslices + sl) * 256);
    } else {
        lora_down_block(p, blockIdx.x - p.M, 0, p.K / 32, nullptr);
    }
}

// GEMM path with the front end: one block per token row.
__global__ void __launch_bounds__(kThreads) ln_quant_kernel(const PrologueParams p, const GemmPrologueExtra x, const FrontEnd fe) {
    pdl_wait();
    quant_row_ln(p, fe, blockIdx.x, x.tok_sc, x.gw_over_127);
}

// ---- group prologue: persistent CTAs, one warp per work item ------------------------------------
// The rows of A^T are the bulk of what a decode prologue reads, and a group has thousands of small
// pieces of them, each behind a chain of dependent memory latencies.  Here the grid stays resident
// (one CTA of 8 warps per SM) and every warp walks the item tables with a grid-wide stride.  For a
// LoRA item the warp requests everything the item reads at once - per lane up to 32 + 16 asynchronous
// 16-byte copies into its own part of shared memory, which serves as a register extension: a lane
// reads back only what it requested itself - while the next item's descriptor is already on its
// way, then runs the tf32 MMAs (rows of A^T are the 16-row operand, tokens the 8-column operand) and
// parks the 16 x 16 partial sums; the GEMV adds a tile's K slices in slice order.
constexpr int kPgWarps = 8;
constexpr int kPgThreads = kPgWarps * 32;

// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros and reads nothing.
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ uint4 pg_lds_u4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

// One warp quantises one token row (Algorithm 1, steps 1-2).  The row is brought into the warp's
// shared-memory buffer with asynchronous copies, all requested at once, so both passes (maximum,
// then rounding) read it from there; a row longer than the buffer goes through in pieces and is
// fetched a second time for the second pass.
__device__ void warp_quant_row(const QuantItem &q, uint32_t buf_u32, const uint8_t *buf, int buf_bytes, int lane) {
    const int K = q.K, piece = buf_bytes / 2;  // elements per piece (a multiple of 256)
    const int npieces = (K + piece - 1) / piece;
    auto fetch = [&](int pc) {  // units of 8 elements; lane-strided, so a lane reads back its own units
        const int n = (K - pc * piece < piece ? K - pc * piece : piece) / 8;
        for (int i = lane; i < n; i += 32) cp_async_16(buf_u32 + 16 * i, q.x + (size_t)pc * piece + 8 * i, 16u);
        asm volatile("cp.async.commit_group;\n" ::: "memory");
        asm volatile("cp.async.wait_all;\n" ::: "memory");
        return n;
    };
    uint32_t abits = 0u;
    int n = 0;
    for (int pc = 0; pc < npieces; ++pc) {
        n = fetch(pc);
        for (int i = lane; i < n; i += 32) abits = absmax8_bits(abits, *reinterpret_cast<const uint4 *>(buf + 16 * i));
    }
    const float g = fmaxf(warp_max(absmax_bits_to_float(abits)), 1e-5f);
    const QuantScale qs = make_quant_scale(g);
    int sum = 0;
    for (int pc = 0; pc < npieces; ++pc) {
        if (npieces > 1) n = fetch(pc);
        uint2 *qv = reinterpret_cast<uint2 *>(q.xq + (size_t)pc * piece);
        for (int i = lane; i < n; i += 32) qv[i] = quant8(*reinterpret_cast<const uint4 *>(buf + 16 * i), qs, sum);
    }
    sum = warp_sum_i(sum);
    if (lane == 0) {
        *q.row_sum = sum;
        *q.gamma_x = g;
    }
}

// The same for a row behind the LayerNorm front end (Appendix E of the paper): statistics in two passes
// summed in double, the largest |xn|, then the codes - the arithmetic of quant_row_ln, one warp per
// row, each pass reading the row from L1 / L2.
__device__ void warp_quant_row_ln(const QuantItem &q, int lane) {
    const int K = q.K, nv = K / 8;
    const uint4 *xv = reinterpret_cast<const uint4 *>(q.x);
    float f[8];
    double sum = 0.0;
    for (int i = lane; i < nv; i += 32) {
        unpack8(xv[i], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) sum += (double)f[e];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const double mean_d = sum / (double)K;
    double ss = 0.0;
    for (int i = lane; i < nv; i += 32) {
        unpack8(xv[i], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const double d = (double)f[e] - mean_d;
            ss += d * d;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const float mean = (float)mean_d, rstd = (float)(1.0 / sqrt(ss / (double)K + (double)q.eps));
    auto load_wb = [&](int i, float (&w)[8], float (&b)[8]) {
        const float4 w0 = *reinterpret_cast<const float4 *>(q.ln_w + 8 * i), w1 = *reinterpret_cast<const float4 *>(q.ln_w + 8 * i + 4);
        const float4 b0 = *reinterpret_cast<const float4 *>(q.ln_b + 8 * i), b1 = *reinterpret_cast<const float4 *>(q.ln_b + 8 * i + 4);
        w[0] = w0.x; w[1] = w0.y; w[2] = w0.z; w[3] = w0.w; w[4] = w1.x; w[5] = w1.y; w[6] = w1.z; w[7] = w1.w;
        b[0] = b0.x; b[1] = b0.y; b[2] = b0.z; b[3] = b0.w; b[4] = b1.x; b[5] = b1.y; b[6] = b1.z; b[7] = b1.w;
    };
    float amax = 0.0f, w[8], b[8];
    for (int i = lane; i < nv; i += 32) {
        unpack8(xv[i], f);
        load_wb(i, w, b);
#pragma unroll
        for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(ln_value(f[e], mean, rstd, w[e], b[e])));
    }
    const float g = fmaxf(warp_max(amax), 1e-5f);
    const float scale = __fdiv_rn(127.0f, g);
    int sum_q = 0;
    uint2 *qv = reinterpret_cast<uint2 *>(q.xq);
    for (int i = lane; i < nv; i += 32) {
        unpack8(xv[i], f);
        load_wb(i, w, b);
        uint32_t c[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            float v = rintf(__fmul_rn(ln_value(f[e], mean, rstd, w[e], b[e]), scale));
            v = fminf(fmaxf(v, -127.0f), 127.0f);
            c[e] = (uint32_t)__float2int_rn(v);
        }
        uint32_t o[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t p01 = __byte_perm(c[4 * h], c[4 * h + 1], 0x0040), p23 = __byte_perm(c[4 * h + 2], c[4 * h + 3], 0x0040);
            o[h] = __byte_perm(p01, p23, 0x5410);
            sum_q = __dp4a((int)o[h], 0x01010101, sum_q);
        }
        qv[i] = make_uint2(o[0], o[1]);
    }
    sum_q = warp_sum_i(sum_q);
    if (lane == 0) {
        *q.row_sum = sum_q;
        *q.gamma_x = g;
        if (q.mean_out) *q.mean_out = mean;
        if (q.rstd_out) *q.rstd_out = rstd;
    }
}

// The LayerNorm front end for many rows (the GEMM path): one warp per token row, eight rows per block, the
// row's passes (mean, variance, largest |xn|, codes) all from L1 with warp shuffles between them - one block
// per row spent its time in block-wide barriers between the passes.
__global__ void __launch_bounds__(kThreads) ln_quant_rows_kernel(const PrologueParams p, const GemmPrologueExtra x, const FrontEnd fe) {
    pdl_wait();
    const int lane = threadIdx.x & 31, m = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (m >= p.M) return;
    QuantItem q;
    q.x = p.x + (size_t)m * p.K;
    q.xq = p.xq + (size_t)m * p.K;
    q.gamma_x = p.gamma_x + m;
    q.row_sum = p.row_sum + m;
    q.K = p.K;
    q.eps = fe.eps;
    q.ln_w = fe.ln_w;
    q.ln_b = fe.ln_b;
    q.mean_out = fe.dbg_mean ? fe.dbg_mean + m : nullptr;
    q.rstd_out = fe.dbg_rstd ? fe.dbg_rstd + m : nullptr;
    warp_quant_row_ln(q, lane);
    __syncwarp();
    if (lane == 0) {  // (reads back what this lane wrote)
        const float g = p.gamma_x[m];
        if (x.tok_sc) x.tok_sc[m] = g * x.gw_over_127;
        if (p.dbg_gamma_x) p.dbg_gamma_x[m] = g;
    }
    if (p.dbg_xq) {  // each lane copies the units it wrote itself
        const uint2 *qv = reinterpret_cast<const uint2 *>(q.xq);
        uint2 *dq = reinterpret_cast<uint2 *>(p.dbg_xq + (size_t)m * p.K);
        for (int i = lane; i < p.K / 8; i += 32) dq[i] = qv[i];
    }
}

template <int NT>
__global__ void __launch_bounds__(kPgThreads, 1)
decode_prologue_group_kernel(const QuantItem *quant_items, int n_quant, const LoraItem *lora, int n_lora) {
    constexpr int CH = 16 / NT;                       // 32-column chunks per item
    constexpr int kWarpBytes = CH * (1024 + 512 * NT);  // per chunk: two rows of A^T and NT rows of x, 16 bytes per lane
    extern __shared__ __align__(128) uint8_t pg_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
    const int gw = blockIdx.x * kPgWarps + warp, nw = gridDim.x * kPgWarps;
    const uint32_t buf = (uint32_t)__cvta_generic_to_shared(pg_smem) + warp * kWarpBytes + 16 * lane;

    pdl_launch_dependents();
    // the item tables are written at set-up, not by the preceding work
    uint4 d0 = make_uint4(0u, 0u, 0u, 0u), d1 = d0;
    if (gw < n_lora) {
        d0 = reinterpret_cast<const uint4 *>(lora + gw)[0];
        d1 = reinterpret_cast<const uint4 *>(lora + gw)[1];
    }
    // LoRA items are dealt from the first warp up, quantisation items from the last warp down, so the
    // warps with one LoRA item fewer take the rows
    const int q_first = nw - 1 - gw;
    QuantItem q = {};
    if (q_first < n_quant) q = quant_items[q_first];
    pdl_wait();  // x, and the scratch this kernel overwrites, belong to earlier work

    for (int i = q_first; i < n_quant; i += nw) {
        QuantItem q_next = q;
        if (i + nw < n_quant) q_next = quant_items[i + nw];  // travels while this row is worked on
        if (q.ln_w) warp_quant_row_ln(q, lane);
        else warp_quant_row(q, buf - 16 * lane, pg_smem + warp * kWarpBytes, kWarpBytes, lane);
        q = q_next;
    }

    for (int i = gw; i < n_lora; i += nw) {
        const LoraItem it = {reinterpret_cast<const __half *>(((uint64_t)d0.y << 32) | d0.x),
                             reinterpret_cast<const __nv_bfloat16 *>(((uint64_t)d0.w << 32) | d0.z),
                             reinterpret_cast<float *>(((uint64_t)d1.y << 32) | d1.x), (int)d1.z, (int)d1.w};
        const int K = it.K, M = it.kvalid_M & 0xff, nchunks = (it.kvalid_M >> 8) / 32;
        // everything this item reads, requested at once
        const __half *rowA = it.At + (size_t)g * K + 8 * t;
        const __half *rowB = rowA + (size_t)8 * K;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const bool in = c < nchunks;
            cp_async_16(buf + c * 1024, in ? rowA + 32 * c : it.At, in ? 16u : 0u);
            cp_async_16(buf + c * 1024 + 512, in ? rowB + 32 * c : it.At, in ? 16u : 0u);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const bool tok = g + 8 * nt < M;
            const __nv_bfloat16 *xr = it.x + (size_t)(tok ? g + 8 * nt : 0) * K + 8 * t;
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const bool in = tok && c < nchunks;
                cp_async_16(buf + CH * 1024 + (c * NT + nt) * 512, in ? xr + 32 * c : it.x, in ? 16u : 0u);
            }
        }
        asm volatile("cp.async.commit_group;\n" ::: "memory");
        if (i + nw < n_lora) {  // the next item's descriptor travels meanwhile
            d0 = reinterpret_cast<const uint4 *>(lora + i + nw)[0];
            d1 = reinterpret_cast<const uint4 *>(lora + i + nw)[1];
        }
        asm volatile("cp.async.wait_all;\n" ::: "memory");

        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[nt][c] = 0.0f;
#pragma unroll 4
        for (int c = 0; c < CH; ++c) {
            const uint4 av = pg_lds_u4(buf + c * 1024), bv = pg_lds_u4(buf + c * 1024 + 512);
            uint4 xv[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) xv[nt] = pg_lds_u4(buf + CH * 1024 + (c * NT + nt) * 512);
            const uint32_t aw[4] = {av.x, av.y, av.z, av.w};
            const uint32_t bw[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                // elements 2 e and 2 e + 1 of this lane's eight take the k slots t and t + 4 of the MMA
                const float2 fa = __half22float2(*reinterpret_cast<const __half2 *>(&aw[e]));
                const float2 fb = __half22float2(*reinterpret_cast<const __half2 *>(&bw[e]));
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint32_t xw = (&xv[nt].x)[e];
                    mma_tf32(acc[nt], __float_as_uint(fa.x), __float_as_uint(fb.x), __float_as_uint(fa.y),
                             __float_as_uint(fb.y), xw << 16, xw & 0xffff0000u);
                }
            }
        }
        // park the partial sums: [register 0..7][lane]
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c) __stcg(it.hpart + (nt * 4 + c) * 32 + lane, acc[nt][c]);
    }
}

static cudaLaunchConfig_t prologue_cfg(int blocks, bool pdl, cudaStream_t stream, cudaLaunchAttribute *attr);

// ---- GEMM-path prologue in one kernel -------------------------------------------------------------
// Quantisation (Algorithm 1, steps 1-2) and the LoRA down-projection (steps 5-6) of a block of 32
// tokens, reading x from HBM once.  First pass: x and the rows of A^T travel through a three-stage
// ring of 256-column chunks (16-byte asynchronous copies); every warp takes 32 columns of a chunk,
// feeds them to the tf32 MMA (tokens are the 16-row operand, 8 columns of H the 8-column operand;
// bf16 and fp16 values are exact in tf32) and, since every element of x passes through exactly one
// lane's registers on the way, keeps the running maximum of |x| of its rows.  Then the warps' partial
// sums of x A are added in a fixed order, and the block's rows - still in L2 - are read again and
// rounded with the now known scales.  JT = r / 8 column tiles of H; JT = 0 quantises only.
constexpr int kFpThreads = 256;
constexpr int kFpWarps = kFpThreads / 32;
constexpr int kFpTokens = 32;
constexpr int kFpChunk = 256;                        // columns per stage
constexpr int kFpPitch = kFpChunk * 2 + 64;          // bytes per staged row: neighbouring rows on the other 16 banks
constexpr int kFpStages = 3;
__host__ __device__ constexpr int fp_stage_bytes(int r) { return (kFpTokens + r) * kFpPitch; }
__host__ __device__ constexpr int fp_smem_bytes(int r) {
    return kFpStages * fp_stage_bytes(r) > kFpWarps * kFpTokens * r * 4 ? kFpStages * fp_stage_bytes(r)
                                                                         : kFpWarps * kFpTokens * r * 4;
}

template <int JT>
__global__ void __launch_bounds__(kFpThreads) gemm_prologue_kernel(const PrologueParams p, const GemmPrologueExtra x) {
    extern __shared__ __align__(128) uint8_t fp_smem[];
    __shared__ float s_amax[kFpWarps][kFpTokens];
    __shared__ float s_gamma[kFpTokens];
    constexpr int r = 8 * JT;
    pdl_wait();  // x, and the workspace this kernel overwrites, belong to earlier work
    const int tpb = x.tokens_per_block;  // tokens this launch gives a block (at most kFpTokens)
    const int token_blocks = (p.M + tpb - 1) / tpb;
    if ((int)blockIdx.x >= token_blocks) {
        // the remaining blocks prepare the up-projection's operand: row n of B^T times its channel's
        // gate, fp16, padded to 64 columns (one 16-byte piece per thread)
        if constexpr (JT > 0) {
            const int idx = ((int)blockIdx.x - token_blocks) * kFpThreads + (int)threadIdx.x, n = idx >> 3, c = idx & 7;
            if (n < x.N) {
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (c * 8 < r) {
                    v = *reinterpret_cast<const uint4 *>(x.Bt + (size_t)n * r + c * 8);
                    const float g = x.gate[x.gate_group > 1 ? n / x.gate_group : n];
                    __half2 *h2 = reinterpret_cast<__half2 *>(&v);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float2 f = __half22float2(h2[k]);
                        h2[k] = __floats2half2_rn(g * f.x, g * f.y);
                    }
                }
                *reinterpret_cast<uint4 *>(x.gb16 + (size_t)n * 64 + c * 8) = v;
            }
        }
        return;
    }
    const int K = p.K, M = p.M;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int m0 = blockIdx.x * tpb;
    const uint32_t smem_u32 = (uint32_t)__cvta_generic_to_shared(fp_smem);
    constexpr int kStage = fp_stage_bytes(r);
    const int nchunks = (K + kFpChunk - 1) / kFpChunk;

    // One chunk into one stage: 32 (+ r) rows of 32 16-byte units; rows past M and columns past K are
    // zeros.  A thread copies unit `lane` of rows warp, warp + 8, ...: the same ones in every chunk.
    constexpr int kRowsPerThread = (kFpTokens + r) / kFpWarps;
    const uint8_t *src_row[kRowsPerThread];
    bool row_ok[kRowsPerThread];
#pragma unroll
    for (int q = 0; q < kRowsPerThread; ++q) {
        const int row = warp + kFpWarps * q;
        if (row < kFpTokens) {
            row_ok[q] = row < tpb && m0 + row < M;
            src_row[q] = reinterpret_cast<const uint8_t *>(p.x + (size_t)(row_ok[q] ? m0 + row : 0) * K) + 16 * lane;
        } else {
            row_ok[q] = true;
            src_row[q] = reinterpret_cast<const uint8_t *>(p.At + (size_t)(row - kFpTokens) * K) + 16 * lane;
        }
    }
    auto fetch = [&](int c, int stage) {
        const uint32_t dst = smem_u32 + stage * kStage + warp * kFpPitch + 16 * lane;
        const int k = c * kFpChunk + 8 * lane;
        const bool col_ok = k < K;
#pragma unroll
        for (int q = 0; q < kRowsPerThread; ++q) {
            const bool in = col_ok && row_ok[q];
            cp_async_16(dst + q * kFpWarps * kFpPitch, src_row[q] + (in ? (size_t)c * kFpChunk * 2 : 0), in ? 16u : 0u);
        }
        asm volatile("cp.async.commit_group;\n" ::: "memory");
    };

    float acc[2][JT > 0 ? JT : 1][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < (JT > 0 ? JT : 1); ++b)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[a][b][c] = 0.0f;
    uint32_t amax[2][2] = {{0u, 0u}, {0u, 0u}};  // rows 16 mt + 8 hh + g, packed maxima of the bit patterns

#pragma unroll
    for (int sg = 0; sg < kFpStages - 1; ++sg) {
        if (sg < nchunks) fetch(sg, sg);
        else asm volatile("cp.async.commit_group;\n" ::: "memory");
    }
    for (int c = 0; c < nchunks; ++c) {
        asm volatile("cp.async.wait_group %0;\n" ::"n"(kFpStages - 2) : "memory");
        __syncthreads();  // chunk c has landed for every thread, and everyone is done with chunk c - 1
        if (c + kFpStages - 1 < nchunks) fetch(c + kFpStages - 1, (c + kFpStages - 1) % kFpStages);
        else asm volatile("cp.async.commit_group;\n" ::: "memory");

        const uint32_t st = smem_u32 + (c % kFpStages) * kStage + 64 * warp + 16 * t;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            if (16 * mt >= tpb) break;  // a block of up to 16 tokens has no second tile
            const uint4 x0 = pg_lds_u4(st + (16 * mt + g) * kFpPitch), x1 = pg_lds_u4(st + (16 * mt + 8 + g) * kFpPitch);
            amax[mt][0] = absmax8_bits(amax[mt][0], x0);
            amax[mt][1] = absmax8_bits(amax[mt][1], x1);
            if constexpr (JT > 0) {
                // elements 2 i and 2 i + 1 of this lane's eight take the k slots t and t + 4 of MMA i
                uint32_t xs[4][4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t w0 = (&x0.x)[i], w1 = (&x1.x)[i];
                    xs[i][0] = w0 << 16; xs[i][1] = w1 << 16; xs[i][2] = w0 & 0xffff0000u; xs[i][3] = w1 & 0xffff0000u;
                }
#pragma unroll
                for (int jt = 0; jt < JT; ++jt) {
                    const uint4 a4 = pg_lds_u4(st + (kFpTokens + 8 * jt + g) * kFpPitch);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 bf = __half22float2(*reinterpret_cast<const __half2 *>(&(&a4.x)[i]));
                        mma_tf32(acc[mt][jt], xs[i][0], xs[i][1], xs[i][2], xs[i][3], __float_as_uint(bf.x), __float_as_uint(bf.y));
                    }
                }
            }
        }
    }
    asm volatile("cp.async.wait_all;\n" ::: "memory");

    // the rows' maxima: over the four lanes that share a row, then over the warps
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            float a = absmax_bits_to_float(amax[mt][hh]);
            a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 1));
            a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 2));
            if (t == 0) s_amax[warp][16 * mt + 8 * hh + g] = a;
        }
    __syncthreads();  // also: every warp is done with the ring, which the partial sums now reuse
    if (tid < kFpTokens) {
        float a = s_amax[0][tid];
#pragma unroll
        for (int w = 1; w < kFpWarps; ++w) a = fmaxf(a, s_amax[w][tid]);
        s_gamma[tid] = fmaxf(a, 1e-5f);
    }
    if constexpr (JT > 0) {
        float *s_acc = reinterpret_cast<float *>(fp_smem);  // [warps][32 tokens][r]
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int jt = 0; jt < JT; ++jt) {
                float *base = s_acc + ((size_t)warp * kFpTokens + 16 * mt) * r + 8 * jt;
                base[g * r + 2 * t] = acc[mt][jt][0];
                base[g * r + 2 * t + 1] = acc[mt][jt][1];
                base[(g + 8) * r + 2 * t] = acc[mt][jt][2];
                base[(g + 8) * r + 2 * t + 1] = acc[mt][jt][3];
            }
    }
    __syncthreads();
    if constexpr (JT > 0) {
        const float *s_acc = reinterpret_cast<const float *>(fp_smem);
        for (int e = tid; e < kFpTokens * r; e += kFpThreads) {
            const int ml = e / r, j = e % r, m = m0 + ml;
            float z = 0.0f;
#pragma unroll
            for (int w = 0; w < kFpWarps; ++w) z += s_acc[w * kFpTokens * r + e];
            const float h = (p.flags & HGF_FLAG_NO_SILU) ? z : silu_f(z);
            if (ml < tpb && m < M) {
                p.h[(size_t)m * r + j] = h;
                if (p.dbg_h) p.dbg_h[(size_t)m * r + j] = h;
                if (p.h16) p.h16[(size_t)m * 64 + j] = __float2half_rn(h);
            }
        }
        if constexpr (JT < 8) {  // zero padding of the fp16 copy up to 64 columns
            if (p.h16)
                for (int e = tid; e < kFpTokens * (64 - r); e += kFpThreads) {
                    const int ml = e / (64 - r), j = r + e % (64 - r), m = m0 + ml;
                    if (ml < tpb && m < M) p.h16[(size_t)m * 64 + j] = __float2half_rn(0.0f);
                }
        }
    }

    // The launch that follows (the GEMM) may be set up from here on; it waits for this grid's completion
    // before it reads.  (Not earlier: blocks of a dependent launch that sit waiting on an SM slow the
    // blocks still working there.)
    pdl_launch_dependents();

    if (!p.xq) return;  // the LayerNorm front end quantises in a kernel of its own
    if (x.split_round) {  // the rounding pass is the next launch: leave it the scales
        if (tid < tpb && m0 + tid < M) {
            const float gm = s_gamma[tid];
            p.gamma_x[m0 + tid] = gm;
            if (x.tok_sc) x.tok_sc[m0 + tid] = gm * x.gw_over_127;
            if (p.dbg_gamma_x) p.dbg_gamma_x[m0 + tid] = gm;
        }
        return;
    }

    // second pass: the warps round the block's rows, warp w rows w, w + 8, ...
    const int nv = K / 8;
#pragma unroll 1
    for (int rr = 0; rr < kFpTokens / kFpWarps; ++rr) {
        const int ml = warp + kFpWarps * rr, m = m0 + ml;
        if (ml >= tpb || m >= M) break;
        const float gm = s_gamma[ml];
        const QuantScale qs = make_quant_scale(gm);
        const uint4 *xv = reinterpret_cast<const uint4 *>(p.x + (size_t)m * K);
        uint2 *qv = reinterpret_cast<uint2 *>(p.xq + (size_t)m * K);
        uint2 *dq = p.dbg_xq ? reinterpret_cast<uint2 *>(p.dbg_xq + (size_t)m * K) : nullptr;
        int sum = 0;
        int i = lane;
        for (; i + 96 < nv; i += 128) {  // four units in flight per lane
            const uint4 v0 = xv[i], v1 = xv[i + 32], v2 = xv[i + 64], v3 = xv[i + 96];
            const uint2 o0 = quant8(v0, qs, sum), o1 = quant8(v1, qs, sum), o2 = quant8(v2, qs, sum), o3 = quant8(v3, qs, sum);
            qv[i] = o0; qv[i + 32] = o1; qv[i + 64] = o2; qv[i + 96] = o3;
            if (dq) { dq[i] = o0; dq[i + 32] = o1; dq[i + 64] = o2; dq[i + 96] = o3; }
        }
        for (; i < nv; i += 32) {
            const uint2 o = quant8(xv[i], qs, sum);
            qv[i] = o;
            if (dq) dq[i] = o;
        }
        sum = warp_sum_i(sum);
        if (lane == 0) {
            if (p.row_sum) p.row_sum[m] = sum;
            if (x.tok_sc) x.tok_sc[m] = gm * x.gw_over_127;
            p.gamma_x[m] = gm;
            if (p.dbg_gamma_x) p.dbg_gamma_x[m] = gm;
        }
    }
}

// The rounding pass as a launch of its own: one warp per token row, the scale taken from gamma_x.  At 64
// registers a thread four blocks share an SM (32 warps), which this arithmetic-bound pass needs: inside the
// kernel above it runs at 16 warps per SM and takes twice as long.  The rows are read from L2.
__global__ void __launch_bounds__(kThreads, 4) round_rows_kernel(const PrologueParams p) {
    pdl_wait();               // the scales come from the launch before
    pdl_launch_dependents();  // the GEMM may set itself up; it waits for this grid before it reads
    const int lane = threadIdx.x & 31, m = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (m >= p.M) return;
    const int K = p.K, nv = K / 8;
    const QuantScale qs = make_quant_scale(p.gamma_x[m]);
    const uint4 *xv = reinterpret_cast<const uint4 *>(p.x + (size_t)m * K);
    uint2 *qv = reinterpret_cast<uint2 *>(p.xq + (size_t)m * K);
    uint2 *dq = p.dbg_xq ? reinterpret_cast<uint2 *>(p.dbg_xq + (size_t)m * K) : nullptr;
    int sum = 0;
    int i = lane;
    for (; i + 96 < nv; i += 128) {  // four units in flight per lane
        const uint4 v0 = xv[i], v1 = xv[i + 32], v2 = xv[i + 64], v3 = xv[i + 96];
        const uint2 o0 = quant8(v0, qs, sum), o1 = quant8(v1, qs, sum), o2 = quant8(v2, qs, sum), o3 = quant8(v3, qs, sum);
        qv[i] = o0; qv[i + 32] = o1; qv[i + 64] = o2; qv[i + 96] = o3;
        if (dq) { dq[i] = o0; dq[i + 32] = o1; dq[i + 64] = o2; dq[i + 96] = o3; }
    }
    for (; i < nv; i += 32) {
        const uint2 o = quant8(xv[i], qs, sum);
        qv[i] = o;
        if (dq) dq[i] = o;
    }
    sum = warp_sum_i(sum);
    if (lane == 0 && p.row_sum) p.row_sum[m] = sum;
}

template <int JT>
static cudaError_t launch_gemm_prologue_jt(const PrologueParams &p, const GemmPrologueExtra &x, int blocks, cudaStream_t stream) {
    // Never more than two blocks per SM (the launcher spreads the rows over twice the SM count of
    // blocks): blocks that start as SMs come free at the tail of the preceding launch would otherwise
    // pile up four to an SM on the first SMs free and leave the others idle.
    constexpr int smem = fp_smem_bytes(8 * JT) > 80 * 1024 ? fp_smem_bytes(8 * JT) : 80 * 1024;
    static std::atomic<unsigned long long> attr_done{0};
    {
        cudaError_t e = ensure_dynamic_smem(gemm_prologue_kernel<JT>, smem, attr_done);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchAttribute attr[1];
    cudaLaunchConfig_t cfg = prologue_cfg(blocks, !(p.flags & HGF_FLAG_NO_PDL), stream, attr);
    cfg.blockDim = dim3(kFpThreads);
    cfg.dynamicSmemBytes = smem;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_prologue_kernel<JT>, p, x);
    return e != cudaSuccess ? e : cudaGetLastError();
}

// Quantisation and (r > 0) LoRA down-projection of the GEMM path, plus gate * B^T for its epilogue.
cudaError_t launch_gemm_prologue(const PrologueParams &p, const GemmPrologueExtra &x, cudaStream_t stream) {
    // Tokens per block: as many blocks as are resident at once share the rows evenly; beyond that a
    // block takes its full 32.
    const int sm_count = device_sm_count();
    if (!sm_count) return cudaErrorInvalidDevice;
    const int per_sm = p.r >= 48 ? 1 : 2;  // blocks that fit an SM (shared memory: 138 KB and more from rank 48 on)
    int tpb = (p.M + per_sm * sm_count - 1) / (per_sm * sm_count);
    tpb = (tpb + 3) / 4 * 4;
    tpb = tpb < 8 ? 8 : (tpb > kFpTokens ? kFpTokens : tpb);
    GemmPrologueExtra xx = x;
    xx.tokens_per_block = tpb;
    // The rounding pass as a second launch where there is enough of x to pay for a launch: it then runs at twice
    // the occupancy, and the GEMM's set-up overlaps it (measured per layer, M = 8192: 118.8 -> 117.0 us at
    // K = 2048, 141.3 -> 134.3 us at K = 5632; M = 4096: 209.7 -> 205.1 us at K = 11008, unchanged at K = 4096).
    const size_t x_bytes = (size_t)p.M * p.K * 2;
    xx.split_round = (p.xq && p.r > 0 && x_bytes >= ((size_t)8 << 20)) ? 1 : 0;
    const int blocks = (p.M + tpb - 1) / tpb + ((p.r > 0 && x.gb16) ? (x.N * 8 + kFpThreads - 1) / kFpThreads : 0);
    cudaError_t e;
    switch (p.r) {
        case 0: e = launch_gemm_prologue_jt<0>(p, xx, blocks, stream); break;
        case 16: e = launch_gemm_prologue_jt<2>(p, xx, blocks, stream); break;
        case 32: e = launch_gemm_prologue_jt<4>(p, xx, blocks, stream); break;
        case 48: e = launch_gemm_prologue_jt<6>(p, xx, blocks, stream); break;
        case 64: e = launch_gemm_prologue_jt<8>(p, xx, blocks, stream); break;
        default: return cudaErrorInvalidValue;
    }
    count_launch();
    if (e == cudaSuccess && xx.split_round) {
        cudaLaunchAttribute attr[1];
        cudaLaunchConfig_t cfg = prologue_cfg((p.M + kWarps - 1) / kWarps, !(p.flags & HGF_FLAG_NO_PDL), stream, attr);
        e = cudaLaunchKernelEx(&cfg, round_rows_kernel, p);
        count_launch();
        if (e == cudaSuccess) e = cudaGetLastError();
    }
    return e;
}

// Quantisation alone.  Many rows: one warp per row while a row fits its registers, else the GEMM
// path's prologue kernel without its LoRA part; few rows: one block per row.
cudaError_t launch_quant(const PrologueParams &p, const GemmPrologueExtra &x, cudaStream_t stream) {
    const int nv = p.K / 8, row_blocks = (p.M + kWarps - 1) / kWarps;
    if (p.M >= 256 && nv <= 32 * 8) {
        cudaLaunchAttribute attr[1];
        cudaLaunchConfig_t cfg = prologue_cfg(row_blocks, !(p.flags & HGF_FLAG_NO_PDL), stream, attr);
        cudaError_t e = cudaLaunchKernelEx(&cfg, quant_rows_kernel<8>, p, x);
        if (e != cudaSuccess) return e;
    } else if (p.M >= 256 && nv <= 32 * 16) {
        cudaLaunchAttribute attr[1];
        cudaLaunchConfig_t cfg = prologue_cfg(row_blocks, !(p.flags & HGF_FLAG_NO_PDL), stream, attr);
        cudaError_t e = cudaLaunchKernelEx(&cfg, quant_rows_kernel<16>, p, x);
        if (e != cudaSuccess) return e;
    } else if (p.M >= 2 * kFpTokens) {
        PrologueParams q = p;
        q.r = 0;
        return launch_gemm_prologue(q, x, stream);
    } else {
        quant_kernel<<<p.M, kThreads, 0, stream>>>(p, x);
    }
    count_launch();
    return cudaGetLastError();
}

cudaLaunchConfig_t prologue_cfg(int blocks, bool pdl, cudaStream_t stream, cudaLaunchAttribute *attr) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cfg;
}

cudaError_t launch_decode_prologue(const PrologueParams &p, bool pdl, cudaStream_t stream) {
    cudaLaunchAttribute attr[1];
    cudaLaunchConfig_t cfg = prologue_cfg(p.M + (p.r / 16) * (p.hpart ? p.nslices : 1), pdl, stream, attr);
    cudaError_t e = cudaLaunchKernelEx(&cfg, decode_prologue_kernel, p);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_decode_prologue_ln(const PrologueParams &p, const FrontEnd &fe, bool pdl, cudaStream_t stream) {
    cudaLaunchAttribute attr[1];
    cudaLaunchConfig_t cfg = prologue_cfg(p.M + (p.r / 16) * (p.hpart ? p.nslices : 1), pdl, stream, attr);
    cudaError_t e = cudaLaunchKernelEx(&cfg, decode_prologue_ln_kernel, p, fe);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_ln_quant(const PrologueParams &p, const GemmPrologueExtra &x, const FrontEnd &fe, cudaStream_t stream) {
    cudaLaunchAttribute attr[1];
    const bool by_warp = p.row_sum != nullptr && p.M >= 64;  // many rows: one warp each; few: one block each
    cudaLaunchConfig_t cfg = prologue_cfg(by_warp ? (p.M + kWarps - 1) / kWarps : p.M, !(p.flags & HGF_FLAG_NO_PDL), stream, attr);
    cudaError_t e = by_warp ? cudaLaunchKernelEx(&cfg, ln_quant_rows_kernel, p, x, fe) : cudaLaunchKernelEx(&cfg, ln_quant_kernel, p, x, fe);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_decode_prologue_group(const QuantItem *d_quant_items, int n_quant, const LoraItem *d_lora_items, int n_lora, int max_M, bool pdl,
                                         cudaStream_t stream) {
    static std::atomic<unsigned long long> attr_done1{0}, attr_done2{0};
    const int sm_count = device_sm_count();
    if (!sm_count) return cudaErrorInvalidDevice;
    const int smem1 = kPgWarps * 16 * (1024 + 512), smem2 = kPgWarps * 8 * (1024 + 1024);
    {
        cudaError_t e = ensure_dynamic_smem(decode_prologue_group_kernel<1>, smem1, attr_done1);
        if (e != cudaSuccess) return e;
        e = ensure_dynamic_smem(decode_prologue_group_kernel<2>, smem2, attr_done2);
        if (e != cudaSuccess) return e;
    }
    const int most = n_lora > n_quant ? n_lora : n_quant;
    int blocks = (most + kPgWarps - 1) / kPgWarps;
    blocks = blocks < sm_count ? blocks : sm_count;
    if (blocks < 1) blocks = 1;
    cudaLaunchAttribute attr[1];
    cudaLaunchConfig_t cfg = prologue_cfg(blocks, pdl, stream, attr);
    cfg.blockDim = dim3(kPgThreads);
    cudaError_t e;
    if (max_M <= 8) {
        cfg.dynamicSmemBytes = smem1;
        e = cudaLaunchKernelEx(&cfg, decode_prologue_group_kernel<1>, d_quant_items, n_quant, d_lora_items, n_lora);
    } else {
        cfg.dynamicSmemBytes = smem2;
        e = cudaLaunchKernelEx(&cfg, decode_prologue_group_kernel<2>, d_quant_items, n_quant, d_lora_items, n_lora);
    }
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace hgf
