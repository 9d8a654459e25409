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

}  // namespace hgf

using namespace hgf;

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
