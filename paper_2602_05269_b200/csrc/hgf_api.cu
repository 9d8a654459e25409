// C-ABI entry points: argument validation, workspace carving, routing between the decode GEMV
// path (M <= 16) and the tcgen05 GEMM path.  No compute happens on the host and there is no CPU
// fallback: without a CUDA device every forward call fails with HGF_ERR_CUDA.
#include <atomic>

#include "hgf_common.cuh"

namespace hgf {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

// Device-side status word (nonzero after a bounded wait gave up).  A file-scope device variable:
// nothing is allocated for it at run time.
__device__ unsigned int g_status_word = 0;

unsigned int *device_status_word() {
    static thread_local int cached_dev = -1;
    static thread_local unsigned int *cached_ptr = nullptr;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    if (dev != cached_dev) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_status_word) != cudaSuccess) return nullptr;
        cached_dev = dev;
        cached_ptr = (unsigned int *)ptr;
    }
    return cached_ptr;
}

static bool misaligned(const void *p) { return p && (((uintptr_t)p) & 15u); }

}  // namespace hgf

using namespace hgf;

extern "C" size_t hgf_workspace_bytes(int64_t M, int64_t d_in, int64_t d_out, int32_t r, uint32_t flags) {
    (void)d_out;
    if (M <= 0 || d_in <= 0 || r < 0) return 256;
    const bool gemm = M > HGF_DECODE_MAX_M || (flags & HGF_FLAG_FORCE_GEMM);
    return ws_layout(M, d_in, r, gemm).total;
}

extern "C" hgf_status hgf_act_quant(const void *x, int64_t M, int64_t d_in, int8_t *xq, float *gamma_x,
                                    int32_t *row_sum, void *stream) {
    if (!x || !xq || !gamma_x || M <= 0 || d_in <= 0) return HGF_ERR_INVALID_ARG;
    if (d_in % 64 != 0 || M > (1 << 24) || d_in > (1 << 20)) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (misaligned(x) || misaligned(xq) || misaligned(gamma_x)) return HGF_ERR_MISALIGNED;
    PrologueParams pp = {};
    pp.x = (const __nv_bfloat16 *)x;
    pp.xq = xq;
    pp.gamma_x = gamma_x;
    pp.row_sum = row_sum;
    pp.M = (int)M;
    pp.K = (int)d_in;
    return launch_quant(pp, (cudaStream_t)stream) == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
}

extern "C" hgf_status hgf_linear_forward(const void *x, int64_t M, const void *packed, float gamma, int64_t d_in,
                                         int64_t d_out, const void *At, const void *Bt, int32_t r,
                                         const float *gate, void *y, void *workspace, size_t workspace_bytes,
                                         const hgf_debug_out *dbg, uint32_t flags, void *stream_) {
    if (!x || !packed || !y || M <= 0 || d_in <= 0 || d_out <= 0 || r < 0) return HGF_ERR_INVALID_ARG;
    if (flags & ~(HGF_FLAG_OUT_BF16 | HGF_FLAG_NO_SILU | HGF_FLAG_FORCE_GEMM)) return HGF_ERR_INVALID_ARG;
    if (!At || !Bt || !gate) r = 0;  // pure ternary layer
    if (d_in % 64 != 0 || d_in > 65536 || d_out > (1 << 24) || M > (1 << 22)) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (r != 0 && r != 16 && r != 32 && r != 48 && r != 64) return HGF_ERR_UNSUPPORTED_SHAPE;
    const bool gemm = M > HGF_DECODE_MAX_M || (flags & HGF_FLAG_FORCE_GEMM);
    if (gemm && (d_out % 8 != 0)) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (misaligned(x) || misaligned(packed) || misaligned(y) || misaligned(At) || misaligned(Bt) || misaligned(gate))
        return HGF_ERR_MISALIGNED;
    if (dbg && (misaligned(dbg->xq) || misaligned(dbg->gamma_x) || misaligned(dbg->y_int) || misaligned(dbg->h)))
        return HGF_ERR_MISALIGNED;
    const WsLayout L = ws_layout(M, d_in, r, gemm);
    if (!workspace || workspace_bytes < L.total) return HGF_ERR_WORKSPACE;
    if (((uintptr_t)workspace) & 255u) return HGF_ERR_MISALIGNED;
    cudaStream_t stream = (cudaStream_t)stream_;
    char *ws = (char *)workspace;

    PrologueParams pp = {};
    pp.x = (const __nv_bfloat16 *)x;
    pp.At = r ? (const __half *)At : nullptr;
    pp.xq = (int8_t *)(ws + L.xq);
    pp.gamma_x = (float *)(ws + L.gamma_x);
    pp.row_sum = (int32_t *)(ws + L.row_sum);
    pp.h = (float *)(ws + L.h);
    pp.h16 = gemm ? (__half *)(ws + L.h16) : nullptr;
    pp.dbg_xq = dbg ? dbg->xq : nullptr;
    pp.dbg_gamma_x = dbg ? dbg->gamma_x : nullptr;
    pp.dbg_h = (dbg && r) ? dbg->h : nullptr;
    pp.M = (int)M;
    pp.K = (int)d_in;
    pp.r = r;
    pp.flags = flags;

    const float gw = (float)((double)gamma / 127.0);

    if (!gemm) {
        if (launch_decode_prologue(pp, stream) != cudaSuccess) return HGF_ERR_CUDA;
        DecodeParams dp = {};
        dp.packed = (const uint8_t *)packed;
        dp.xq = pp.xq;
        dp.gamma_x = pp.gamma_x;
        dp.row_sum = pp.row_sum;
        dp.h = pp.h;
        dp.Bt = (const __half *)Bt;
        dp.gate = gate;
        dp.y = y;
        dp.dbg_y_int = dbg ? dbg->y_int : nullptr;
        dp.gw_over_127 = gw;
        dp.M = (int)M;
        dp.K = (int)d_in;
        dp.N = (int)d_out;
        dp.r = r;
        dp.flags = flags;
        return launch_decode_gemv(dp, stream) == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
    }

    if (launch_quant(pp, stream) != cudaSuccess) return HGF_ERR_CUDA;
    if (r && launch_lora_down_gemm(pp, stream) != cudaSuccess) return HGF_ERR_CUDA;
    GemmParams gp = {};
    gp.xq = pp.xq;
    gp.packed = (const uint8_t *)packed;
    gp.gamma_x = pp.gamma_x;
    gp.row_sum = pp.row_sum;
    gp.h16 = pp.h16;
    gp.Bt = (const __half *)Bt;
    gp.gate = gate;
    gp.y = y;
    gp.dbg_y_int = dbg ? dbg->y_int : nullptr;
    gp.gw_over_127 = gw;
    gp.M = (int)M;
    gp.K = (int)d_in;
    gp.N = (int)d_out;
    gp.r = r;
    gp.flags = flags;
    return launch_prefill_gemm(gp, stream) == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
}

extern "C" hgf_status hgf_check_status(void *stream) {
    unsigned int *w = device_status_word();
    if (!w) return HGF_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return HGF_ERR_CUDA;
    unsigned int v = 0;
    if (cudaMemcpy(&v, w, sizeof v, cudaMemcpyDeviceToHost) != cudaSuccess) return HGF_ERR_CUDA;
    if (v) {
        unsigned int zero = 0;
        cudaMemcpy(w, &zero, sizeof zero, cudaMemcpyHostToDevice);
        return HGF_ERR_TIMEOUT;
    }
    return HGF_OK;
}

extern "C" double hgf_tmax_tokens_per_s(double bmem_bytes_per_s, double params, double bits_per_param) {
    return bmem_bytes_per_s / (params * bits_per_param / 8.0);
}

extern "C" uint64_t hgf_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

extern "C" const char *hgf_status_string(hgf_status s) {
    switch (s) {
        case HGF_OK: return "ok";
        case HGF_ERR_INVALID_ARG: return "invalid argument";
        case HGF_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case HGF_ERR_MISALIGNED: return "misaligned pointer";
        case HGF_ERR_WORKSPACE: return "workspace missing or too small";
        case HGF_ERR_CUDA: return "CUDA error";
        case HGF_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    }
    return "unknown status";
}
