// Decode path, M <= 16 tokens: one pass over the packed ternary weights (Algorithm 1, step 3),
// with the dequantisation (step 4), the LoRA up-projection (step 7) and the gated fusion (step 8)
// fused into the epilogue.  One launch serves one layer or a group of independent layers.
//
// The kernel is bound by the packed-weight stream from HBM.  A work item is 16 consecutive
// output rows of one layer (optionally one of S interleaved K slices of them) and belongs to one
// warp.  Each lane fetches 128-bit pieces of two weight rows, four steps (4 x 256 k) ahead of
// their use, expands the 2-bit codes in registers with one AND per register and feeds them to the
// warp-level int8 tensor-core MMA (m16n8k32, u8 x s8 -> s32): the 16-row operand holds weight
// rows, the 8-column operand holds the tokens.  The AND masks keep the codes in place, i.e. scaled
// by 1, 4, 16 or 64; each scale has its own accumulator and the exact quotients are added at the
// end.  Codes are t + 1, so sum_k t x~ = sum_k c x~ - sum_k x~ (the row sums come from the
// quantisation kernel).  Before an item's epilogue the warp already has the first loads of its
// next item in flight, so the weight stream does not pause.
#include "hgf_common.cuh"

namespace hgf {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kTileRows = 16;
constexpr int kDepth = 4;  // steps of weight loads in flight per warp

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
__device__ __forceinline__ void prefetch_l2(const void *ptr) {
    asm volatile("prefetch.global.L2 [%0];\n" ::"l"(ptr));
}
// Programmatic dependent launch: both are no-ops when the launch carries no such attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }

struct Item {
    const uint8_t *wA, *wB;  // this lane's two weight rows, already offset by 16 t bytes
    const int8_t *xq;        // activations of token g, already offset by 64 t
    int K, M, first_step, nsteps, prob, n0;
};

__device__ __forceinline__ const DecodeProblem &problem_of(const DecodeLaunch &L, const DecodeProblem &single,
                                                           int prob) {
    return L.probs ? L.probs[prob] : single;
}

// Work item `tile` (a global row-tile index over all problems of the launch), K slice ks of S.
__device__ __forceinline__ Item make_item(const DecodeLaunch &L, const DecodeProblem &single, int tile, int ks,
                                          int S, int g, int t) {
    Item it;
    it.nsteps = 0;
    it.prob = -1;
    if (tile >= L.total_tiles) return it;
    int prob = 0;
    if (L.probs) {  // last problem whose tile_begin <= tile
        int lo = 0, hi = L.n_probs - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (L.probs[mid].tile_begin <= tile) lo = mid; else hi = mid - 1;
        }
        prob = lo;
    }
    const DecodeProblem &P = problem_of(L, single, prob);
    const int K = P.K, N = P.N;
    const int n0 = (tile - P.tile_begin) * kTileRows;
    const size_t row_bytes = (size_t)K / 4;
    it.wA = P.packed + (size_t)min(n0 + g, N - 1) * row_bytes + 16 * t;
    it.wB = P.packed + (size_t)min(n0 + g + 8, N - 1) * row_bytes + 16 * t;
    it.xq = P.xq + (size_t)g * K + 64 * t;
    it.K = K;
    it.M = P.M;
    it.first_step = ks;
    const int total = (K + 255) / 256;
    it.nsteps = ks < total ? (total - ks + S - 1) / S : 0;
    it.prob = prob;
    it.n0 = n0;
    return it;
}

// NT = number of 8-token tiles (1: M <= 8, 2: M <= 16).
template <int NT>
__global__ void __launch_bounds__(kDecThreads, 2) decode_gemv_kernel(const DecodeLaunch L, const DecodeProblem single) {
    __shared__ int s_red[kDecWarps][kTileRows][8 * NT];

    pdl_launch_dependents();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int S = L.S;                       // K slices per row tile: 1, 2, 4 or 8
    const int tiles_per_cta = kDecWarps / S;
    const int my_tile = warp / S, ks = warp % S;
    const int n_cta_items = (L.total_tiles + tiles_per_cta - 1) / tiles_per_cta;

    uint4 ringA[kDepth], ringB[kDepth];
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);

    auto fetch = [&](const Item &it, int i, uint4 &a, uint4 &b) {
        // step i of the item; K % 64 == 0, so a lane's 64-wide piece is either whole or absent
        const int step = it.first_step + i * S;
        const bool valid = i < it.nsteps && step * 256 + 64 * t < it.K;
        a = valid ? ld_stream_u4(it.wA + (size_t)step * 64) : zero4;
        b = valid ? ld_stream_u4(it.wB + (size_t)step * 64) : zero4;
    };

    int ci = blockIdx.x;
    Item cur = make_item(L, single, ci < n_cta_items ? ci * tiles_per_cta + my_tile : L.total_tiles, ks, S, g, t);
#pragma unroll
    for (int j = 0; j < kDepth; ++j) fetch(cur, j, ringA[j], ringB[j]);

    // everything above reads only weights; the activations come from the preceding launch
    pdl_wait();

    for (; ci < n_cta_items; ci += gridDim.x) {
        int acc[NT][4][4];
#pragma unroll
        for (int a = 0; a < NT; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[a][b][c] = 0;

        for (int s0 = 0; s0 < cur.nsteps; s0 += kDepth) {
#pragma unroll
            for (int j = 0; j < kDepth; ++j) {
                const int i = s0 + j;
                if (i < cur.nsteps) {  // warp-uniform
                    const uint32_t pw[4] = {ringA[j].x, ringA[j].y, ringA[j].z, ringA[j].w};
                    const uint32_t qw[4] = {ringB[j].x, ringB[j].y, ringB[j].z, ringB[j].w};
                    const int k = (cur.first_step + i * S) * 256;  // + 64 t is folded into cur.xq
                    const bool kvalid = k + 64 * t < cur.K;
                    fetch(cur, i + kDepth, ringA[j], ringB[j]);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        uint32_t xw[4][4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            uint4 v = zero4;
                            if (kvalid && 8 * nt + g < cur.M)
                                v = *reinterpret_cast<const uint4 *>(cur.xq + (size_t)(8 * nt) * cur.K + k + 16 * u);
                            xw[u][0] = v.x; xw[u][1] = v.y; xw[u][2] = v.z; xw[u][3] = v.w;
                        }
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj) {
                            const uint32_t mask = 0x03030303u << (2 * jj);
#pragma unroll
                            for (int h = 0; h < 2; ++h)
                                mma_u8s8(acc[nt][jj], pw[2 * h] & mask, qw[2 * h] & mask, pw[2 * h + 1] & mask,
                                         qw[2 * h + 1] & mask, xw[2 * h][jj], xw[2 * h + 1][jj]);
                        }
                    }
                }
            }
        }

        // start the next item's weight stream before this item's epilogue
        const int cn = ci + gridDim.x;
        const Item nxt = make_item(L, single, cn < n_cta_items ? cn * tiles_per_cta + my_tile : L.total_tiles, ks, S, g, t);
#pragma unroll
        for (int j = 0; j < kDepth; ++j) fetch(nxt, j, ringA[j], ringB[j]);

        // exact rescale of the four accumulators
        int v[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c)
                v[nt][c] = acc[nt][0][c] + (acc[nt][1][c] >> 2) + (acc[nt][2][c] >> 4) + (acc[nt][3][c] >> 6);

        if (S > 1) {  // sum the K slices of a row tile through shared memory
            __syncthreads();  // previous item's readers are done
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                s_red[warp][g][8 * nt + 2 * t] = v[nt][0];
                s_red[warp][g][8 * nt + 2 * t + 1] = v[nt][1];
                s_red[warp][g + 8][8 * nt + 2 * t] = v[nt][2];
                s_red[warp][g + 8][8 * nt + 2 * t + 1] = v[nt][3];
            }
            __syncthreads();
            if (ks == 0) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    int s0 = 0, s1 = 0, s2 = 0, s3 = 0;
                    for (int w = 0; w < S; ++w) {
                        s0 += s_red[warp + w][g][8 * nt + 2 * t];
                        s1 += s_red[warp + w][g][8 * nt + 2 * t + 1];
                        s2 += s_red[warp + w][g + 8][8 * nt + 2 * t];
                        s3 += s_red[warp + w][g + 8][8 * nt + 2 * t + 1];
                    }
                    v[nt][0] = s0; v[nt][1] = s1; v[nt][2] = s2; v[nt][3] = s3;
                }
            }
        }

        // epilogue: lane l handles output row l / 2 and one half of the rank-r dot product
        if (ks == 0 && cur.prob >= 0) {
            const DecodeProblem &P = problem_of(L, single, cur.prob);
            const int row = lane >> 1, half = lane & 1, n = cur.n0 + row, r = P.r, hr = r >> 1;
            const bool n_ok = n < P.N;
            const int nc = n_ok ? n : P.N - 1;
            uint4 bq[4];  // this lane's half of row n of B^T, as fp16 pairs
#pragma unroll
            for (int q = 0; q < 4; ++q)
                bq[q] = q * 8 < hr ? *reinterpret_cast<const uint4 *>(P.Bt + (size_t)nc * r + half * hr + q * 8) : zero4;
            const float gate = r > 0 ? P.gate[nc] : 0.0f;
            const int owner_base = (row & 7) * 4;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int mm = 0; mm < 8; ++mm) {
                    const int m = 8 * nt + mm;
                    if (m < P.M) {  // warp-uniform
                        // C[row][m] lives in lane (row % 8) * 4 + mm / 2, register (row / 8) * 2 + mm % 2
                        const int src = owner_base + (mm >> 1);
                        const int lo = __shfl_sync(0xffffffffu, v[nt][mm & 1], src);
                        const int hi = __shfl_sync(0xffffffffu, v[nt][2 + (mm & 1)], src);
                        const int y_int = (row < 8 ? lo : hi) - P.row_sum[m];
                        float corr = 0.0f;
                        if (r > 0) {
                            const float4 *hv = reinterpret_cast<const float4 *>(P.h + (size_t)m * r + half * hr);
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                if (q * 8 < hr) {
                                    const __half2 *b2 = reinterpret_cast<const __half2 *>(&bq[q]);
                                    const float4 h0 = hv[2 * q], h1 = hv[2 * q + 1];
                                    const float2 f0 = __half22float2(b2[0]), f1 = __half22float2(b2[1]);
                                    const float2 f2 = __half22float2(b2[2]), f3 = __half22float2(b2[3]);
                                    corr = fmaf(h0.x, f0.x, corr); corr = fmaf(h0.y, f0.y, corr);
                                    corr = fmaf(h0.z, f1.x, corr); corr = fmaf(h0.w, f1.y, corr);
                                    corr = fmaf(h1.x, f2.x, corr); corr = fmaf(h1.y, f2.y, corr);
                                    corr = fmaf(h1.z, f3.x, corr); corr = fmaf(h1.w, f3.y, corr);
                                }
                            }
                        }
                        corr += __shfl_xor_sync(0xffffffffu, corr, 1);
                        if (half == 0 && n_ok) {
                            const float y = fmaf(gate, corr, (float)y_int * (P.gamma_x[m] * P.gw_over_127));
                            const size_t o = (size_t)m * P.N + n;
                            if (P.flags & HGF_FLAG_OUT_BF16)
                                reinterpret_cast<__nv_bfloat16 *>(P.y)[o] = __float2bfloat16_rn(y);
                            else
                                reinterpret_cast<float *>(P.y)[o] = y;
                            if (P.dbg_y_int) P.dbg_y_int[o] = y_int;
                        }
                    }
                }
            }
        }
        cur = nxt;
    }
}

// K slices per row tile: enough items to give every resident warp one, at least one step each.
static int choose_slices(int total_tiles, int min_steps, int warp_slots) {
    int S = 1;
    while (S < kDecWarps && total_tiles * S < warp_slots && min_steps >= 2 * S) S *= 2;
    return S;
}

cudaError_t launch_decode_gemv(const DecodeLaunch &L_in, const DecodeProblem *single, int max_M, int min_steps,
                               bool pdl, cudaStream_t stream) {
    static int sm_count = 0;
    if (!sm_count) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
    }
    DecodeLaunch L = L_in;
    const int warp_slots = sm_count * 2 * kDecWarps;
    L.S = choose_slices(L.total_tiles, min_steps, warp_slots);
    const int tiles_per_cta = kDecWarps / L.S;
    const int n_cta_items = (L.total_tiles + tiles_per_cta - 1) / tiles_per_cta;
    const int grid = n_cta_items < sm_count * 2 ? n_cta_items : sm_count * 2;
    DecodeProblem dummy = {};
    const DecodeProblem &sp = single ? *single : dummy;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kDecThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    cudaError_t e = max_M <= 8 ? cudaLaunchKernelEx(&cfg, decode_gemv_kernel<1>, L, sp)
                               : cudaLaunchKernelEx(&cfg, decode_gemv_kernel<2>, L, sp);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace hgf
