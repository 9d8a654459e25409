// Offline weight preparation: absmean scale, ternary codes, 2-bit packing (and its inverse).
// Paper: Section 2.2, Definition "Absmax Quantization" (the scale is the mean of |W|).
#include "hgf_common.cuh"

namespace hgf {

constexpr int kAbsBlocks = 1024;
constexpr int kAbsThreads = 256;

// Stage 1: per-block sums of |W| in double (fixed grid-stride order, fixed tree -> deterministic).
__global__ void __launch_bounds__(kAbsThreads) abs_sum_partial_kernel(const float4 *W4, size_t n4,
                                                                      double *partials) {
    double acc = 0.0;
    for (size_t i = (size_t)blockIdx.x * kAbsThreads + threadIdx.x; i < n4;
         i += (size_t)gridDim.x * kAbsThreads) {
        float4 v = W4[i];
        acc += (double)fabsf(v.x) + (double)fabsf(v.y) + (double)fabsf(v.z) + (double)fabsf(v.w);
    }
    __shared__ double red[kAbsThreads];
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int s = kAbsThreads / 2; s > 0; s >>= 1) {
        if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) partials[blockIdx.x] = red[0];
}

// Stage 2: one warp adds the partials (fixed order: lane-strided, then a fixed shuffle tree) and
// rounds the mean once to fp32.
__global__ void abs_sum_final_kernel(const double *partials, int n, double count, float *gamma) {
    double acc = 0.0;
    for (int i = threadIdx.x; i < n; i += 32) acc += partials[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (threadIdx.x == 0) *gamma = (float)(acc / count);
}

// Decomposition of a packed word index into its place in the matrix.  Words are numbered in storage
// order: 16 per row segment, 16 row segments per tile, column tiles fastest, then row tiles.
struct WordPos {
    int64_t n, k0;  // output row and first of the 16 input columns the word covers
};
__device__ __forceinline__ WordPos word_pos(size_t w, int64_t steps) {
    const int64_t kw = (int64_t)(w & 15), r = (int64_t)((w >> 4) & 15);
    const int64_t tile = (int64_t)(w >> 8);
    WordPos p;
    p.n = (tile / steps) * 16 + r;
    p.k0 = (tile % steps) * 256 + kw * 16;
    return p;
}

// Stage 3: one thread per 32-bit packed word (16 weights).  Weight k0 + 4 j + b goes to bits
// 8 b + 2 j of the word; code = t + 1; t = sign(w) * [|w| > gamma/2].  Padding words hold code 1.
__global__ void __launch_bounds__(256) ternarise_pack_kernel(const float *W, int64_t N, int64_t K, int64_t steps,
                                                             size_t n_words, const float *gamma, uint32_t *packed) {
    size_t w = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (w >= n_words) return;
    const WordPos p = word_pos(w, steps);
    uint32_t word = 0x55555555u;
    if (p.n < N && p.k0 < K) {
        const float half = 0.5f * *gamma;  // exact
        const float4 *src = reinterpret_cast<const float4 *>(W + p.n * K + p.k0);
        word = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float4 v = src[j];
            float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                uint32_t c = e[b] > half ? 2u : (e[b] < -half ? 0u : 1u);
                word |= c << (8 * b + 2 * j);
            }
        }
    }
    packed[w] = word;
}

__global__ void __launch_bounds__(256) unpack_kernel(const uint32_t *packed, int64_t N, int64_t K, int64_t steps,
                                                     size_t n_words, int8_t *T) {
    size_t w = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (w >= n_words) return;
    const WordPos p = word_pos(w, steps);
    if (p.n >= N || p.k0 >= K) return;
    uint32_t word = packed[w];
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t e = (word >> (2 * j)) & 0x03030303u;  // codes 0..3 per byte
        uint32_t r = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            int c = (e >> (8 * b)) & 0xff;
            int t = c == 3 ? 0 : c - 1;
            r |= (uint32_t)(t & 0xff) << (8 * b);
        }
        o[j] = r;
    }
    *reinterpret_cast<uint4 *>(T + p.n * K + p.k0) = make_uint4(o[0], o[1], o[2], o[3]);
}

// ---- base-3 layout: five codes per byte ---------------------------------------------------------
// Tiles of 16 rows x 320 columns, 64 bytes per row.  Byte q = 16 t + j of a row holds, as digits of a
// base-3 number, the codes of tile columns col(j, t) + 0..3 (digits 0..3) and col(16 + j / 4, t) + j % 4
// (digit 4), col(p, t) = 32 (p / 2) + 16 (p % 2) + 4 t: lane t of the decode kernel's warp MMA then
// finds the operand registers of its ten MMAs in its own 16 bytes of the row.
__host__ __device__ inline int b3_col(int p, int t) { return 32 * (p >> 1) + 16 * (p & 1) + 4 * t; }

// One thread per packed byte.
__global__ void __launch_bounds__(256) ternarise_pack_b3_kernel(const float *W, int64_t N, int64_t K, int64_t steps,
                                                                size_t n_bytes, const float *gamma, uint8_t *packed) {
    size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= n_bytes) return;
    const int q = (int)(i & 63), row = (int)((i >> 6) & 15);
    const int64_t tile = (int64_t)(i >> 10);
    const int64_t n = (tile / steps) * 16 + row, k_tile = (tile % steps) * 320;
    const int t = q >> 4, j = q & 15;
    const float half = 0.5f * *gamma;  // exact
    int cols[5];
#pragma unroll
    for (int e = 0; e < 4; ++e) cols[e] = b3_col(j, t) + e;
    cols[4] = b3_col(16 + (j >> 2), t) + (j & 3);
    int v = 0, power = 1;
#pragma unroll
    for (int e = 0; e < 5; ++e) {
        const int64_t k = k_tile + cols[e];
        int c = 1;  // padding: weight 0
        if (n < N && k < K) {
            const float w = W[n * K + k];
            c = w > half ? 2 : (w < -half ? 0 : 1);
        }
        v += c * power;
        power *= 3;
    }
    packed[i] = (uint8_t)v;
}

// One thread per weight.
__global__ void __launch_bounds__(256) unpack_b3_kernel(const uint8_t *packed, int64_t N, int64_t K, int64_t steps, int8_t *T) {
    const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (idx >= N * K) return;
    const int64_t n = idx / K, k = idx % K;
    const int col = (int)(k % 320), p = 2 * (col / 32) + (col % 32) / 16, t = (col % 16) / 4, e = col % 4;
    const int j = p < 16 ? p : 4 * (p - 16) + e;
    const int digit = p < 16 ? e : 4;
    const size_t off = (size_t)((n / 16) * steps + k / 320) * 1024 + (size_t)(n % 16) * 64 + 16 * t + j;
    int v = packed[off];
    int c = 1;
    if (v <= 242) {
        for (int d = 0; d < digit; ++d) v /= 3;
        c = v % 3;
    }
    T[idx] = (int8_t)(c - 1);
}

// Base-3 bytes -> two-bit tiles (the GEMM path reads only those).  One thread per two-bit word: its sixteen
// codes are digits of up to sixteen bytes of the row's 64 in the base-3 tile that holds those columns.
__global__ void __launch_bounds__(256) repack_b3_kernel(const uint8_t *packed_b3, int64_t N, int64_t K, int64_t steps2, int64_t steps3,
                                                        size_t n_words, uint32_t *packed2) {
    const size_t w = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (w >= n_words) return;
    const WordPos p = word_pos(w, steps2);
    uint32_t word = 0x55555555u;
    if (p.n < N && p.k0 < K) {
        word = 0;
        const uint8_t *row_base = packed_b3 + (size_t)(p.n / 16) * steps3 * 1024 + (size_t)(p.n % 16) * 64;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int64_t k = p.k0 + i;  // K is a multiple of 64: the word's sixteen columns are all inside the matrix
            const int col = (int)(k % 320), q = 2 * (col / 32) + (col % 32) / 16, t = (col % 16) / 4, e = col % 4;
            const int j = q < 16 ? q : 4 * (q - 16) + e, digit = q < 16 ? e : 4;
            int v = row_base[(size_t)(k / 320) * 1024 + 16 * t + j];
            int c = 1;
            if (v <= 242) {
                for (int d = 0; d < digit; ++d) v /= 3;
                c = v % 3;
            }
            word |= (uint32_t)c << (8 * (i & 3) + 2 * (i >> 2));
        }
    }
    packed2[w] = word;
}

cudaError_t launch_repack_b3(const void *packed_b3, int64_t d_out, int64_t d_in, void *packed2, cudaStream_t stream) {
    const int64_t steps2 = padded_k(d_in) / 256, steps3 = padded_k_b3(d_in) / 320;
    const size_t n_words = (size_t)row_tiles(d_out) * steps2 * 256;
    repack_b3_kernel<<<(unsigned)((n_words + 255) / 256), 256, 0, stream>>>((const uint8_t *)packed_b3, d_out, d_in, steps2, steps3, n_words,
                                                                            (uint32_t *)packed2);
    count_launch();
    return cudaGetLastError();
}

// gamma_W = mean |W| into *gamma_dev (two launches; partials: kAbsBlocks doubles)
static void enqueue_gamma(const float *W, size_t n, double *partials, float *gamma_dev, cudaStream_t stream) {
    abs_sum_partial_kernel<<<kAbsBlocks, kAbsThreads, 0, stream>>>((const float4 *)W, n / 4, partials);
    abs_sum_final_kernel<<<1, 32, 0, stream>>>(partials, kAbsBlocks, (double)n, gamma_dev);
}

}  // namespace hgf

using namespace hgf;

extern "C" size_t hgf_packed_bytes_b3(int64_t d_out, int64_t d_in) {
    if (d_out <= 0 || d_in <= 0 || d_in % 64 != 0) return 0;
    return (size_t)row_tiles(d_out) * 16 * (size_t)padded_k_b3(d_in) / 5;
}

extern "C" hgf_status hgf_pack_ternary_b3(const float *W, int64_t d_out, int64_t d_in, void *packed, float *gamma_out,
                                          void *stream_) {
    if (!W || !packed || !gamma_out || d_out <= 0 || d_in <= 0) return HGF_ERR_INVALID_ARG;
    if (d_in % 64 != 0) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (((uintptr_t)W | (uintptr_t)packed) & 15) return HGF_ERR_MISALIGNED;
    cudaStream_t stream = (cudaStream_t)stream_;
    void *tmp = nullptr;
    if (cudaMalloc(&tmp, kAbsBlocks * sizeof(double) + 256) != cudaSuccess) return HGF_ERR_CUDA;
    float *gamma_dev = (float *)((char *)tmp + kAbsBlocks * sizeof(double));
    enqueue_gamma(W, (size_t)d_out * (size_t)d_in, (double *)tmp, gamma_dev, stream);
    const int64_t steps = padded_k_b3(d_in) / 320;
    const size_t n_bytes = (size_t)row_tiles(d_out) * (size_t)steps * 1024;
    ternarise_pack_b3_kernel<<<(unsigned)((n_bytes + 255) / 256), 256, 0, stream>>>(W, d_out, d_in, steps, n_bytes, gamma_dev,
                                                                                    (uint8_t *)packed);
    count_launch(3);
    cudaError_t e = cudaMemcpyAsync(gamma_out, gamma_dev, sizeof(float), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    cudaError_t e2 = cudaGetLastError();
    cudaFree(tmp);
    return (e == cudaSuccess && e2 == cudaSuccess) ? HGF_OK : HGF_ERR_CUDA;
}

extern "C" hgf_status hgf_unpack_ternary_b3(const void *packed, int64_t d_out, int64_t d_in, int8_t *T, void *stream_) {
    if (!packed || !T || d_out <= 0 || d_in <= 0) return HGF_ERR_INVALID_ARG;
    if (d_in % 64 != 0 || d_out * d_in > ((int64_t)1 << 40)) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (((uintptr_t)T | (uintptr_t)packed) & 15) return HGF_ERR_MISALIGNED;
    const int64_t steps = padded_k_b3(d_in) / 320, n = d_out * d_in;
    unpack_b3_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)stream_>>>((const uint8_t *)packed, d_out, d_in, steps, T);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
}

extern "C" size_t hgf_packed_bytes(int64_t d_out, int64_t d_in) {
    if (d_out <= 0 || d_in <= 0 || d_in % 64 != 0) return 0;
    return (size_t)row_tiles(d_out) * 16 * (size_t)padded_k(d_in) / 4;
}

extern "C" hgf_status hgf_pack_ternary(const float *W, int64_t d_out, int64_t d_in, void *packed,
                                       float *gamma_out, void *stream_) {
    if (!W || !packed || !gamma_out || d_out <= 0 || d_in <= 0) return HGF_ERR_INVALID_ARG;
    if (d_in % 64 != 0) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (((uintptr_t)W | (uintptr_t)packed) & 15) return HGF_ERR_MISALIGNED;
    cudaStream_t stream = (cudaStream_t)stream_;
    size_t n = (size_t)d_out * (size_t)d_in;
    void *tmp = nullptr;
    if (cudaMalloc(&tmp, kAbsBlocks * sizeof(double) + 256) != cudaSuccess) return HGF_ERR_CUDA;
    double *partials = (double *)tmp;
    float *gamma_dev = (float *)((char *)tmp + kAbsBlocks * sizeof(double));
    abs_sum_partial_kernel<<<kAbsBlocks, kAbsThreads, 0, stream>>>((const float4 *)W, n / 4, partials);
    abs_sum_final_kernel<<<1, 32, 0, stream>>>(partials, kAbsBlocks, (double)n, gamma_dev);
    const int64_t steps = padded_k(d_in) / 256;
    size_t n_words = (size_t)row_tiles(d_out) * (size_t)steps * 256;
    ternarise_pack_kernel<<<(unsigned)((n_words + 255) / 256), 256, 0, stream>>>(W, d_out, d_in, steps, n_words, gamma_dev,
                                                                                 (uint32_t *)packed);
    count_launch(3);
    cudaError_t e = cudaMemcpyAsync(gamma_out, gamma_dev, sizeof(float), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    cudaError_t e2 = cudaGetLastError();
    cudaFree(tmp);
    return (e == cudaSuccess && e2 == cudaSuccess) ? HGF_OK : HGF_ERR_CUDA;
}

extern "C" hgf_status hgf_unpack_ternary(const void *packed, int64_t d_out, int64_t d_in, int8_t *T,
                                         void *stream_) {
    if (!packed || !T || d_out <= 0 || d_in <= 0) return HGF_ERR_INVALID_ARG;
    if (d_in % 64 != 0) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (((uintptr_t)T | (uintptr_t)packed) & 15) return HGF_ERR_MISALIGNED;
    const int64_t steps = padded_k(d_in) / 256;
    size_t n_words = (size_t)row_tiles(d_out) * (size_t)steps * 256;
    unpack_kernel<<<(unsigned)((n_words + 255) / 256), 256, 0, (cudaStream_t)stream_>>>((const uint32_t *)packed, d_out, d_in,
                                                                                        steps, n_words, T);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
}
