// Causal differential attention forward (paper, Section 2.4, Definition "Differential Attention"):
//     O = ( Softmax(Q1 K1^T / sqrt(d_h)) - lambda * Softmax(Q2 K2^T / sqrt(d_h)) ) V
// on the outputs of the HGF attention projections (Definition "HGF Attention Projections": Q, K of
// width d, V of width d / 2), per batch element and head.
//
// One CTA of four warps per (batch element, head, tile of 64 queries); a warp owns 16 query rows.
// Keys and values go through shared memory in tiles of 64 (16-byte asynchronous copies); both streams'
// scores are formed on the warp-level bf16 MMA (m16n8k16, fp32 accumulate) with the query fragments
// held in registers, the softmax is the running-maximum form in fp32 (base-2 exponentials), the
// probabilities go back into the MMA as bf16 first operands, and the two streams share the value tile.
// The two streams' outputs are normalised and combined once, at the end.  No tensor-memory path here:
// the block is small against the linear layers around it and is built for parity, not for the roofline.
#include <cmath>

#include "hgf_common.cuh"

namespace hgf {

constexpr int kAtBM = 64, kAtBN = 64, kAtThreads = 128;

struct AttnParams {
    const __nv_bfloat16 *q, *k, *v;  // q, k [B*L][2*h*dh]; v [B*L][h*dh]
    void *out;                       // [B*L][h*dh] fp32 or bf16
    int B, L, h;
    float lambda, out_scale, scale_log2;  // scale_log2 = log2(e) / sqrt(dh)
    uint32_t flags;
};

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void at_cp_async_16(uint32_t dst, const void *src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}

template <int DH>
__global__ void __launch_bounds__(kAtThreads) diff_attention_kernel(const AttnParams p) {
    constexpr int PITCH = DH * 2 + 16;          // bytes per staged row: eight rows 16 bytes apart in the banks
    constexpr int TILE = kAtBN * PITCH;
    constexpr int KS = DH / 16, DN = DH / 8;    // k steps of Q K^T, 8-column tiles of the output
    extern __shared__ __align__(128) uint8_t at_smem[];  // K of stream 1, K of stream 2, V
    const uint32_t sm = (uint32_t)__cvta_generic_to_shared(at_smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;  // the long tiles (late queries) start first
    const int hd = blockIdx.y, b = blockIdx.z;
    const int L = p.L, dq = 2 * p.h * DH, dv = p.h * DH;
    const int q0 = qt * kAtBM, row0 = q0 + 16 * warp + g, row1 = row0 + 8;
    const size_t tok0 = (size_t)b * L;

    // query fragments of both streams (first operand of S = Q K^T), zeros past the sequence
    uint32_t qa[2][KS][4];
#pragma unroll
    for (int s = 0; s < 2; ++s) {
        const __nv_bfloat16 *r0 = p.q + (tok0 + (row0 < L ? row0 : 0)) * dq + (s * p.h + hd) * DH + 2 * t;
        const __nv_bfloat16 *r1 = p.q + (tok0 + (row1 < L ? row1 : 0)) * dq + (s * p.h + hd) * DH + 2 * t;
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) {
            qa[s][kk][0] = row0 < L ? *reinterpret_cast<const uint32_t *>(r0 + 16 * kk) : 0u;
            qa[s][kk][1] = row1 < L ? *reinterpret_cast<const uint32_t *>(r1 + 16 * kk) : 0u;
            qa[s][kk][2] = row0 < L ? *reinterpret_cast<const uint32_t *>(r0 + 16 * kk + 8) : 0u;
            qa[s][kk][3] = row1 < L ? *reinterpret_cast<const uint32_t *>(r1 + 16 * kk + 8) : 0u;
        }
    }
    float o[2][DN][4];
    float mx[2][2], ls[2][2];  // running maximum (base-2 scaled scores) and this thread's part of the running sum
#pragma unroll
    for (int s = 0; s < 2; ++s) {
#pragma unroll
        for (int d = 0; d < DN; ++d)
#pragma unroll
            for (int c = 0; c < 4; ++c) o[s][d][c] = 0.0f;
        mx[s][0] = mx[s][1] = -INFINITY;
        ls[s][0] = ls[s][1] = 0.0f;
    }

    const int q_end = q0 + kAtBM < L ? q0 + kAtBM : L;  // keys up to the tile's last query
    const int n_kt = (q_end + kAtBN - 1) / kAtBN;
    for (int kt = 0; kt < n_kt; ++kt) {
        const int j0 = kt * kAtBN;
        __syncthreads();  // the previous tile has been consumed
        // stage K1, K2, V rows j0 .. j0 + 63 (zeros past the sequence): DH / 8 16-byte pieces per row and tensor
        for (int u = tid; u < 3 * kAtBN * (DH / 8); u += kAtThreads) {
            const int which = u / (kAtBN * (DH / 8)), rem = u - which * (kAtBN * (DH / 8)), r = rem / (DH / 8), c = rem - r * (DH / 8);
            const int j = j0 + r;
            const bool in = j < L;
            const __nv_bfloat16 *src = which < 2 ? p.k + (tok0 + (in ? j : 0)) * dq + (which * p.h + hd) * DH + 8 * c
                                                 : p.v + (tok0 + (in ? j : 0)) * dv + hd * DH + 8 * c;
            at_cp_async_16(sm + which * TILE + r * PITCH + 16 * c, src, in ? 16u : 0u);
        }
        asm volatile("cp.async.commit_group;\n" ::: "memory");
        asm volatile("cp.async.wait_all;\n" ::: "memory");
        __syncthreads();

        const bool diag = j0 + kAtBN > q0 + 16 * warp;  // this warp's rows meet the causal boundary (or the end) in this tile
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            float sc[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) sc[nt][c] = 0.0f;
#pragma unroll
            for (int kk = 0; kk < KS; ++kk)
#pragma unroll
                for (int np = 0; np < 4; ++np) {  // two 8-key tiles per ldmatrix
                    uint32_t kb[4];
                    const int i = lane >> 3, r = lane & 7;
                    ldmatrix_x4(sm + s * TILE + ((2 * np + (i >> 1)) * 8 + r) * PITCH + (16 * kk + 8 * (i & 1)) * 2, kb);
                    mma_bf16(sc[2 * np], qa[s][kk][0], qa[s][kk][1], qa[s][kk][2], qa[s][kk][3], kb[0], kb[1]);
                    mma_bf16(sc[2 * np + 1], qa[s][kk][0], qa[s][kk][1], qa[s][kk][2], qa[s][kk][3], kb[2], kb[3]);
                }
            // scale to base 2, mask (key after the query, or past the sequence), row maxima
            float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int j = j0 + 8 * nt + 2 * t + (c & 1), i = (c >> 1) ? row1 : row0;
                    float v = sc[nt][c] * p.scale_log2;
                    if (diag && (j > i || j >= L)) v = -INFINITY;
                    sc[nt][c] = v;
                    tmax[c >> 1] = fmaxf(tmax[c >> 1], v);
                }
            float alpha[2];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                tmax[hh] = fmaxf(tmax[hh], __shfl_xor_sync(0xffffffffu, tmax[hh], 1));
                tmax[hh] = fmaxf(tmax[hh], __shfl_xor_sync(0xffffffffu, tmax[hh], 2));
                const float m_new = fmaxf(mx[s][hh], tmax[hh]);
                // (a row wholly masked so far - only rows past the sequence - keeps -inf and contributes zeros)
                alpha[hh] = m_new == -INFINITY ? 1.0f : exp2f(mx[s][hh] - m_new);
                mx[s][hh] = m_new;
                ls[s][hh] *= alpha[hh];
            }
            uint32_t pa[4][4];  // probabilities as first operands: 16 keys per step
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                float e[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float m = mx[s][c >> 1];
                    e[c] = m == -INFINITY ? 0.0f : exp2f(sc[nt][c] - m);
                    ls[s][c >> 1] += e[c];
                }
                pa[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(e[0], e[1]);
                pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(e[2], e[3]);
            }
#pragma unroll
            for (int d = 0; d < DN; ++d) {
                o[s][d][0] *= alpha[0]; o[s][d][1] *= alpha[0];
                o[s][d][2] *= alpha[1]; o[s][d][3] *= alpha[1];
            }
#pragma unroll
            for (int k2 = 0; k2 < 4; ++k2)
#pragma unroll
                for (int dp = 0; dp < DN / 2; ++dp) {  // two 8-column tiles of V per ldmatrix
                    uint32_t vb[4];
                    const int i = lane >> 3, r = lane & 7;
                    ldmatrix_x4_trans(sm + 2 * TILE + (16 * k2 + 8 * (i & 1) + r) * PITCH + ((2 * dp + (i >> 1)) * 8) * 2, vb);
                    mma_bf16(o[s][2 * dp], pa[k2][0], pa[k2][1], pa[k2][2], pa[k2][3], vb[0], vb[1]);
                    mma_bf16(o[s][2 * dp + 1], pa[k2][0], pa[k2][1], pa[k2][2], pa[k2][3], vb[2], vb[3]);
                }
        }
    }

    // normalise each stream, combine, store
    float inv[2][2];
#pragma unroll
    for (int s = 0; s < 2; ++s)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            float l = ls[s][hh];
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            inv[s][hh] = l > 0.0f ? 1.0f / l : 0.0f;
        }
    const bool out_bf16 = (p.flags & HGF_FLAG_OUT_BF16) != 0;
#pragma unroll
    for (int d = 0; d < DN; ++d)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int row = hh ? row1 : row0;
            if (row >= L) continue;
            const float y0 = (o[0][d][2 * hh] * inv[0][hh] - p.lambda * o[1][d][2 * hh] * inv[1][hh]) * p.out_scale;
            const float y1 = (o[0][d][2 * hh + 1] * inv[0][hh] - p.lambda * o[1][d][2 * hh + 1] * inv[1][hh]) * p.out_scale;
            const size_t off = (tok0 + row) * dv + hd * DH + 8 * d + 2 * t;
            if (out_bf16)
                *reinterpret_cast<uint32_t *>(reinterpret_cast<__nv_bfloat16 *>(p.out) + off) = pack_bf16(y0, y1);
            else
                *reinterpret_cast<float2 *>(reinterpret_cast<float *>(p.out) + off) = make_float2(y0, y1);
        }
}

template <int DH>
static cudaError_t launch_attention_dh(const AttnParams &p, cudaStream_t stream) {
    static std::atomic<unsigned long long> attr_done{0};
    constexpr int smem = 3 * kAtBN * (DH * 2 + 16);
    cudaError_t e = ensure_dynamic_smem(diff_attention_kernel<DH>, smem, attr_done);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)((p.L + kAtBM - 1) / kAtBM), (unsigned)p.h, (unsigned)p.B);
    diff_attention_kernel<DH><<<grid, kAtThreads, smem, stream>>>(p);
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
    const cudaError_t e = head_dim == 64 ? launch_attention_dh<64>(p, (cudaStream_t)stream) : launch_attention_dh<128>(p, (cudaStream_t)stream);
    return e == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
}

extern "C" double hgf_diff_lambda0(double head_dim) { return 0.8 - 0.6 * exp(-0.3 * head_dim); }
