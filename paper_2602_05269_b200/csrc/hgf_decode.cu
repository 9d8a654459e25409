// Decode path, M <= 16 tokens: one pass over the packed ternary weights (Algorithm 1, step 3),
// with the dequantisation (step 4), the LoRA up-projection (step 7) and the gated fusion (step 8)
// fused into the epilogue.
//
// The kernel is bound by the packed-weight stream from HBM.  Each thread fetches 128-bit
// pieces of two weight rows, expands the 2-bit codes in registers with one AND per register,
// and feeds them to the warp-level int8 tensor-core MMA (m16n8k32, u8 x s8 -> s32): the 16-row
// operand holds weight rows, the 8-column operand holds the tokens.  The AND masks keep the
// codes in place, i.e. scaled by 1, 4, 16 or 64; each scale has its own accumulator and the
// exact quotients are added at the end.  Codes are t + 1, so sum_k t x~ = sum_k c x~ - sum_k x~.
#include "hgf_common.cuh"

namespace hgf {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kRowsPerBlock = 16;

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ld_stream_u4(const void *ptr) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(ptr));
    return v;
}

// NT = number of 8-token tiles (1: M <= 8, 2: M <= 16).
//
// Work split: a block owns 16 consecutive output rows; its 8 warps split K in steps of 256.
// In a step, thread (g = lane / 4, t = lane % 4) holds 64 consecutive k (k0 + 64 t ...) of rows
// g and g + 8, and the matching 64 int8 activations of token g.  Within those 64, word i and
// mask j select k = 16 i + 4 j + (0..3): MMA (j, h) multiplies words 2h, 2h+1 under mask j with
// the activation words (2h, j) and (2h+1, j).
template <int NT>
__global__ void __launch_bounds__(kDecThreads) decode_gemv_kernel(const DecodeParams p) {
    __shared__ int s_red[kDecWarps][kRowsPerBlock][8 * NT];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int K = p.K, N = p.N, M = p.M;
    const int n0 = blockIdx.x * kRowsPerBlock;
    const int rowA = min(n0 + g, N - 1), rowB = min(n0 + g + 8, N - 1);
    const size_t row_bytes = (size_t)K / 4;
    const uint8_t *wA = p.packed + (size_t)rowA * row_bytes;
    const uint8_t *wB = p.packed + (size_t)rowB * row_bytes;

    int acc[NT][4][4];
#pragma unroll
    for (int a = 0; a < NT; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[a][b][c] = 0;

    const int nsteps = (K + 255) / 256;
#pragma unroll 2
    for (int step = warp; step < nsteps; step += kDecWarps) {
        const int k = step * 256 + 64 * t;
        // K % 64 == 0: a thread's 64-wide piece is either whole or absent.  Absent pieces are
        // zeros (code 0 times activation 0); every lane still executes the warp-wide MMAs.
        const bool valid = k < K;
        const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
        const uint4 P = valid ? ld_stream_u4(wA + k / 4) : zero4;
        const uint4 Q = valid ? ld_stream_u4(wB + k / 4) : zero4;
        const uint32_t pw[4] = {P.x, P.y, P.z, P.w};
        const uint32_t qw[4] = {Q.x, Q.y, Q.z, Q.w};
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int tok = 8 * nt + g;
            uint32_t xw[4][4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                uint4 v = zero4;
                if (valid && tok < M) v = reinterpret_cast<const uint4 *>(p.xq + (size_t)tok * K + k)[u];
                xw[u][0] = v.x; xw[u][1] = v.y; xw[u][2] = v.z; xw[u][3] = v.w;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t mask = 0x03030303u << (2 * j);
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    mma_u8s8(acc[nt][j], pw[2 * h] & mask, qw[2 * h] & mask, pw[2 * h + 1] & mask,
                             qw[2 * h + 1] & mask, xw[2 * h][j], xw[2 * h + 1][j]);
            }
        }
    }

    // exact rescale of the four accumulators, then the cross-warp sum
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        int v[4];
#pragma unroll
        for (int c = 0; c < 4; ++c)
            v[c] = acc[nt][0][c] + (acc[nt][1][c] >> 2) + (acc[nt][2][c] >> 4) + (acc[nt][3][c] >> 6);
        s_red[warp][g][8 * nt + 2 * t] = v[0];
        s_red[warp][g][8 * nt + 2 * t + 1] = v[1];
        s_red[warp][g + 8][8 * nt + 2 * t] = v[2];
        s_red[warp][g + 8][8 * nt + 2 * t + 1] = v[3];
    }
    __syncthreads();

    // epilogue: thread -> (row, token); adjacent threads own adjacent output channels
    if (tid < kRowsPerBlock * 8 * NT) {
        const int row = tid % kRowsPerBlock, tok = tid / kRowsPerBlock, n = n0 + row;
        if (tok < M && n < N) {
            int s = 0;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) s += s_red[w][row][tok];
            const int y_int = s - p.row_sum[tok];
            float y = (float)y_int * (p.gamma_x[tok] * p.gw_over_127);
            if (p.r > 0) {
                float corr = 0.0f;
                const uint4 *bv = reinterpret_cast<const uint4 *>(p.Bt + (size_t)n * p.r);
                const float4 *hv = reinterpret_cast<const float4 *>(p.h + (size_t)tok * p.r);
                for (int q = 0; q < p.r / 8; ++q) {
                    uint4 b4 = bv[q];
                    float4 h0 = hv[2 * q], h1 = hv[2 * q + 1];
                    const __half2 *b2 = reinterpret_cast<const __half2 *>(&b4);
                    float2 f0 = __half22float2(b2[0]), f1 = __half22float2(b2[1]);
                    float2 f2 = __half22float2(b2[2]), f3 = __half22float2(b2[3]);
                    corr = fmaf(h0.x, f0.x, corr); corr = fmaf(h0.y, f0.y, corr);
                    corr = fmaf(h0.z, f1.x, corr); corr = fmaf(h0.w, f1.y, corr);
                    corr = fmaf(h1.x, f2.x, corr); corr = fmaf(h1.y, f2.y, corr);
                    corr = fmaf(h1.z, f3.x, corr); corr = fmaf(h1.w, f3.y, corr);
                }
                y = fmaf(p.gate[n], corr, y);
            }
            const size_t o = (size_t)tok * N + n;
            if (p.flags & HGF_FLAG_OUT_BF16)
                reinterpret_cast<__nv_bfloat16 *>(p.y)[o] = __float2bfloat16_rn(y);
            else
                reinterpret_cast<float *>(p.y)[o] = y;
            if (p.dbg_y_int) p.dbg_y_int[o] = y_int;
        }
    }
}

cudaError_t launch_decode_gemv(const DecodeParams &p, cudaStream_t stream) {
    const int blocks = (p.N + kRowsPerBlock - 1) / kRowsPerBlock;
    if (p.M <= 8)
        decode_gemv_kernel<1><<<blocks, kDecThreads, 0, stream>>>(p);
    else
        decode_gemv_kernel<2><<<blocks, kDecThreads, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hgf
