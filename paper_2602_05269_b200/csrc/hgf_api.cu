// C-ABI entry points: argument validation, workspace carving, routing between the decode GEMV
// path (M <= 16) and the tcgen05 GEMM path.  No compute happens on the host and there is no CPU
// fallback: without a CUDA device every forward call fails with HGF_ERR_CUDA.
#include <atomic>
#include <new>
#include <unordered_map>
#include <vector>

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

int current_device() {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

int device_sm_count() {
    static std::atomic<int> cache[kMaxDevices];
    const int dev = current_device();
    if (dev < 0 || dev >= kMaxDevices) return 0;
    int n = cache[dev].load(std::memory_order_acquire);
    if (!n) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 0;
        cache[dev].store(n, std::memory_order_release);
    }
    return n;
}

static bool misaligned(const void *p) { return p && (((uintptr_t)p) & 15u); }

// The decode path keeps a problem's quantised activations in shared memory; problems too large
// for that (and every M > 16) take the GEMM path.
static bool takes_gemm_path(int64_t M, int64_t d_in, uint32_t flags) {
    if (M > HGF_DECODE_MAX_M || (flags & HGF_FLAG_FORCE_GEMM)) return true;
    return decode_xq_smem_bytes((int)M, (int)d_in, flags) > decode_xq_smem_limit(flags);
}

}  // namespace hgf

using namespace hgf;

extern "C" size_t hgf_workspace_bytes(int64_t M, int64_t d_in, int64_t d_out, int32_t r, uint32_t flags) {
    if (M <= 0 || d_in <= 0 || d_in > 65536 || r < 0) return 256;
    return ws_layout(M, d_in, d_out, r, takes_gemm_path(M, d_in, flags), (flags & HGF_FLAG_BASE3) != 0).total;
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
    return launch_quant(pp, GemmPrologueExtra{}, (cudaStream_t)stream) == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
}

namespace hgf {

// Validates one layer problem.  On HGF_OK, *r_eff is the rank actually used (0 for a pure
// ternary layer) and *gemm tells which path the problem takes.
static hgf_status validate_problem(const void *x, int64_t M, const void *packed, int64_t d_in, int64_t d_out,
                                   const void *At, const void *Bt, int32_t r, const float *gate, const void *y,
                                   uint32_t flags, int32_t *r_eff, bool *gemm) {
    if (!x || !packed || !y || M <= 0 || d_in <= 0 || d_out <= 0 || r < 0) return HGF_ERR_INVALID_ARG;
    if (flags & ~(HGF_FLAG_OUT_BF16 | HGF_FLAG_NO_SILU | HGF_FLAG_FORCE_GEMM | HGF_FLAG_NO_PDL | HGF_FLAG_BASE3)) return HGF_ERR_INVALID_ARG;
    if (!At || !Bt || !gate) r = 0;  // pure ternary layer
    if (d_in % 64 != 0 || d_in > 65536 || d_out > (1 << 24) || M > (1 << 22)) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (r != 0 && r != 16 && r != 32 && r != 48 && r != 64) return HGF_ERR_UNSUPPORTED_SHAPE;
    *gemm = takes_gemm_path(M, d_in, flags);
    if (*gemm && (d_out % 8 != 0)) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (misaligned(x) || misaligned(packed) || misaligned(y) || misaligned(At) || misaligned(Bt) || misaligned(gate))
        return HGF_ERR_MISALIGNED;
    *r_eff = r;
    return HGF_OK;
}

static void fill_params(const void *x, int64_t M, const void *packed, float gamma, int64_t d_in, int64_t d_out,
                        const void *At, const void *Bt, int32_t r, const float *gate, void *y, char *ws,
                        const WsLayout &L, bool gemm, const hgf_debug_out *dbg, uint32_t flags, PrologueParams *pp,
                        DecodeProblem *dp) {
    *pp = PrologueParams{};
    pp->x = (const __nv_bfloat16 *)x;
    pp->At = r ? (const __half *)At : nullptr;
    pp->xq = (int8_t *)(ws + L.xq);
    pp->gamma_x = (float *)(ws + L.gamma_x);
    pp->row_sum = (int32_t *)(ws + L.row_sum);
    pp->h = (float *)(ws + L.h);
    pp->h_hi = gemm ? nullptr : (__half *)(ws + L.h_hi);
    pp->h_lo = gemm ? nullptr : (__half *)(ws + L.h_lo);
    pp->h16 = gemm ? (__half *)(ws + L.h16) : nullptr;
    pp->dbg_xq = dbg ? dbg->xq : nullptr;
    pp->dbg_gamma_x = dbg ? dbg->gamma_x : nullptr;
    pp->dbg_h = (dbg && r) ? dbg->h : nullptr;
    // decode path: unless H itself is asked for, x A is computed in K slices by more blocks and the
    // GEMV adds the slices
    if (!gemm && r && !pp->dbg_h) {
        pp->hpart = (float *)(ws + L.hpart);
        pp->nslices = (int)((d_in + prologue_slice_k((int)M) - 1) / prologue_slice_k((int)M));
    }
    pp->M = (int)M;
    pp->K = (int)d_in;
    pp->r = r;
    pp->flags = flags;
    if (dp) {
        *dp = DecodeProblem{};
        dp->packed = (const uint8_t *)packed;
        dp->xq = pp->xq;
        dp->gamma_x = pp->gamma_x;
        dp->row_sum = pp->row_sum;
        dp->h_hi = pp->h_hi;
        dp->h_lo = pp->h_lo;
        dp->hpart = pp->hpart;
        dp->nslices = pp->hpart ? pp->nslices : 0;
        dp->Bt = (const __half *)Bt;
        dp->gate = gate;
        dp->y = y;
        dp->dbg_y_int = dbg ? dbg->y_int : nullptr;
        dp->gw_over_127 = (float)((double)gamma / 127.0);
        dp->M = (int)M;
        dp->K = (int)d_in;
        dp->N = (int)d_out;
        dp->r = r;
        dp->flags = flags;
        dp->tile_begin = 0;
        dp->cost_begin = 0;
        dp->gate_group = 1;
    }
}

static hgf_status forward_impl(const void *x, int64_t M, const void *packed, float gamma, int64_t d_in, int64_t d_out,
                               const void *At, const void *Bt, int32_t r, const float *gate, void *y, void *workspace,
                               size_t workspace_bytes, const hgf_debug_out *dbg, const hgf_front_end *fe_in, uint32_t flags,
                               uint32_t phases, void *stream_);

}  // namespace hgf

extern "C" hgf_status hgf_linear_forward(const void *x, int64_t M, const void *packed, float gamma, int64_t d_in,
                                         int64_t d_out, const void *At, const void *Bt, int32_t r,
                                         const float *gate, void *y, void *workspace, size_t workspace_bytes,
                                         const hgf_debug_out *dbg, uint32_t flags, void *stream_) {
    return hgf_linear_forward_phases(x, M, packed, gamma, d_in, d_out, At, Bt, r, gate, y, workspace, workspace_bytes, dbg,
                                     flags, HGF_PHASE_PROLOGUE | HGF_PHASE_GEMV, stream_);
}

extern "C" hgf_status hgf_linear_forward_phases(const void *x, int64_t M, const void *packed, float gamma, int64_t d_in,
                                                int64_t d_out, const void *At, const void *Bt, int32_t r,
                                                const float *gate, void *y, void *workspace, size_t workspace_bytes,
                                                const hgf_debug_out *dbg, uint32_t flags, uint32_t phases, void *stream_) {
    return forward_impl(x, M, packed, gamma, d_in, d_out, At, Bt, r, gate, y, workspace, workspace_bytes, dbg, nullptr, flags,
                        phases, stream_);
}

extern "C" hgf_status hgf_linear_forward_ln(const void *x, int64_t M, const void *packed, float gamma, int64_t d_in,
                                            int64_t d_out, const void *At, const void *Bt, int32_t r, const float *gate,
                                            void *y, void *workspace, size_t workspace_bytes, const hgf_debug_out *dbg,
                                            const hgf_front_end *front_end, uint32_t flags, void *stream_) {
    if (!front_end) return HGF_ERR_INVALID_ARG;
    return forward_impl(x, M, packed, gamma, d_in, d_out, At, Bt, r, gate, y, workspace, workspace_bytes, dbg, front_end, flags,
                        HGF_PHASE_PROLOGUE | HGF_PHASE_GEMV, stream_);
}

// Validates a front-end description (nullable) and turns it into the kernels' form.
static hgf_status parse_front_end(const hgf_front_end *fe_in, int64_t d_out, bool *ln, int *gate_group, FrontEnd *fe) {
    *ln = false;
    *gate_group = 1;
    *fe = FrontEnd{};
    if (!fe_in) return HGF_OK;
    if ((fe_in->ln_weight == nullptr) != (fe_in->ln_bias == nullptr) || !(fe_in->eps >= 0.0f)) return HGF_ERR_INVALID_ARG;
    if ((((uintptr_t)fe_in->ln_weight) | ((uintptr_t)fe_in->ln_bias)) & 15u) return HGF_ERR_MISALIGNED;
    if (fe_in->gate_group < 0) return HGF_ERR_INVALID_ARG;
    if (fe_in->gate_group > 1) {
        if (fe_in->gate_group >= d_out) *gate_group = (int)((d_out + 15) / 16 * 16);  // scalar gate: one group holds every row tile
        else if (fe_in->gate_group % 16 == 0) *gate_group = (int)fe_in->gate_group;
        else return HGF_ERR_UNSUPPORTED_SHAPE;
    }
    *ln = fe_in->ln_weight != nullptr;
    fe->ln_w = fe_in->ln_weight;
    fe->ln_b = fe_in->ln_bias;
    fe->dbg_mean = fe_in->mean_out;
    fe->dbg_rstd = fe_in->rstd_out;
    fe->eps = fe_in->eps;
    return HGF_OK;
}

hgf_status hgf::forward_impl(const void *x, int64_t M, const void *packed, float gamma, int64_t d_in, int64_t d_out,
                                    const void *At, const void *Bt, int32_t r, const float *gate, void *y, void *workspace,
                                    size_t workspace_bytes, const hgf_debug_out *dbg, const hgf_front_end *fe_in, uint32_t flags,
                                    uint32_t phases, void *stream_) {
    if (!phases || (phases & ~(HGF_PHASE_PROLOGUE | HGF_PHASE_GEMV))) return HGF_ERR_INVALID_ARG;
    const bool do_prologue = (phases & HGF_PHASE_PROLOGUE) != 0, do_main = (phases & HGF_PHASE_GEMV) != 0;
    bool gemm = false;
    hgf_status st = validate_problem(x, M, packed, d_in, d_out, At, Bt, r, gate, y, flags, &r, &gemm);
    if (st != HGF_OK) return st;
    if (dbg && (misaligned(dbg->xq) || misaligned(dbg->gamma_x) || misaligned(dbg->y_int) || misaligned(dbg->h)))
        return HGF_ERR_MISALIGNED;
    const WsLayout L = ws_layout(M, d_in, d_out, r, gemm, (flags & HGF_FLAG_BASE3) != 0);
    if (!workspace || workspace_bytes < L.total) return HGF_ERR_WORKSPACE;
    if (((uintptr_t)workspace) & 255u) return HGF_ERR_MISALIGNED;
    cudaStream_t stream = (cudaStream_t)stream_;
    const bool pdl = !(flags & HGF_FLAG_NO_PDL);

    // front end (Appendix E): LayerNorm before the quantiser, grouped gate
    bool ln = false;
    int gate_group = 1;
    FrontEnd fe = {};
    {
        hgf_status fst = parse_front_end(fe_in, d_out, &ln, &gate_group, &fe);
        if (fst != HGF_OK) return fst;
    }

    PrologueParams pp;
    DecodeProblem dp;
    fill_params(x, M, packed, gamma, d_in, d_out, At, Bt, r, gate, y, (char *)workspace, L, gemm, dbg, flags, &pp, &dp);
    dp.gate_group = gate_group;

    if (!gemm) {
        if (do_prologue && (ln ? launch_decode_prologue_ln(pp, fe, pdl, stream) : launch_decode_prologue(pp, pdl, stream)) != cudaSuccess)
            return HGF_ERR_CUDA;
        if (!do_main) return HGF_OK;
        DecodeLaunch dl = {};
        dl.probs = nullptr;
        dl.n_probs = 1;
        dl.total_tiles = (int)row_tiles(d_out);
        dl.total_cost = (long long)dl.total_tiles * row_tile_cost((int)d_in, flags);
        dl.max_M = (int)M;
        dl.xq_smem_bytes = decode_xq_smem_bytes((int)M, (int)d_in, flags);
        return launch_decode_gemv(dl, &dp, pdl, stream) == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
    }

    // Base-3 weights on the GEMM path: the tensor-core kernel reads two-bit tiles, so the layer's tiles are
    // rewritten from the base-3 bytes into the workspace first (a few microseconds; the prefill is bound by
    // arithmetic, not by the weight bytes the base-3 layout saves).
    const void *packed2 = packed;
    if (do_main && (flags & HGF_FLAG_BASE3)) {
        if (launch_repack_b3(packed, d_out, d_in, (char *)workspace + L.w2, stream) != cudaSuccess) return HGF_ERR_CUDA;
        packed2 = (char *)workspace + L.w2;
    }
    GemmPrologueExtra gx = {};
    gx.tok_sc = (float *)((char *)workspace + L.tok_sc);
    gx.gb16 = r ? (__half *)((char *)workspace + L.gb16) : nullptr;
    gx.Bt = (const __half *)Bt;
    gx.gate = gate;
    gx.gw_over_127 = dp.gw_over_127;
    gx.N = (int)d_out;
    gx.gate_group = gate_group;
    if (do_prologue && ln) {
        // the correction path's part of the prologue on the raw tokens (its own quantisation switched off),
        // then one launch that normalises and quantises
        if (r) {
            PrologueParams lora_only = pp;
            lora_only.xq = nullptr;
            if (launch_gemm_prologue(lora_only, gx, stream) != cudaSuccess) return HGF_ERR_CUDA;
        }
        if (launch_ln_quant(pp, gx, fe, stream) != cudaSuccess) return HGF_ERR_CUDA;
    } else if (do_prologue && (r ? launch_gemm_prologue(pp, gx, stream) : launch_quant(pp, gx, stream)) != cudaSuccess) {
        return HGF_ERR_CUDA;
    }
    if (!do_main) return HGF_OK;
    GemmParams gp = {};
    gp.xq = pp.xq;
    gp.packed = (const uint8_t *)packed2;
    gp.gamma_x = pp.gamma_x;
    gp.row_sum = pp.row_sum;
    gp.h16 = pp.h16;
    gp.tok_sc = gx.tok_sc;
    gp.gb16 = gx.gb16;
    gp.y = y;
    gp.dbg_y_int = dbg ? dbg->y_int : nullptr;
    gp.gw_over_127 = dp.gw_over_127;
    gp.M = (int)M;
    gp.K = (int)d_in;
    gp.N = (int)d_out;
    gp.r = r;
    gp.flags = flags;
    return launch_prefill_gemm(gp, stream) == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
}

// ---- a forward call that allocates nothing ------------------------------------------------------
// Scratch for callers that cannot provide a workspace: part of the library image, one copy per
// device that loads it.  In host code the name below is only a handle for the symbol, never a
// device address; the address a kernel can use comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_static_scratch[HGF_STATIC_SCRATCH_BYTES];

namespace hgf {
static void *static_scratch_address() {
    constexpr int kMaxDevices = 64;
    static std::atomic<void *> cache[kMaxDevices];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    void *ptr = cache[dev].load(std::memory_order_acquire);
    if (!ptr) {
        if (cudaGetSymbolAddress((void **)&ptr, g_static_scratch) != cudaSuccess || !ptr) return nullptr;
        cache[dev].store(ptr, std::memory_order_release);
    }
    return ptr;
}
}  // namespace hgf

extern "C" hgf_status hgf_linear_forward_static(const void *x, int64_t M, const void *packed, float gamma, int64_t d_in,
                                                int64_t d_out, const void *At, const void *Bt, int32_t r,
                                                const float *gate, void *y, uint32_t flags, void *stream) {
    if (M <= 0 || d_in <= 0 || d_out <= 0 || r < 0) return HGF_ERR_INVALID_ARG;
    if (flags & HGF_FLAG_FORCE_GEMM) return HGF_ERR_INVALID_ARG;
    if (d_in % 64 != 0 || d_in > 65536 || M > HGF_DECODE_MAX_M) return HGF_ERR_UNSUPPORTED_SHAPE;
    const int32_t r_eff = (At && Bt && gate) ? r : 0;
    if (r_eff != 0 && r_eff != 16 && r_eff != 32 && r_eff != 48 && r_eff != 64) return HGF_ERR_UNSUPPORTED_SHAPE;
    if (ws_layout(M, d_in, d_out, r_eff, false).total > (size_t)HGF_STATIC_SCRATCH_BYTES) return HGF_ERR_TOO_LARGE;
    if (takes_gemm_path(M, d_in, flags)) return HGF_ERR_UNSUPPORTED_SHAPE;
    void *scratch = static_scratch_address();
    if (!scratch) return HGF_ERR_CUDA;
    return hgf_linear_forward(x, M, packed, gamma, d_in, d_out, At, Bt, r, gate, y, scratch, HGF_STATIC_SCRATCH_BYTES,
                              nullptr, flags, stream);
}

// ---- groups of independent decode problems --------------------------------------------------------
struct hgf_group {
    int n, total_tiles, max_M, xq_smem_bytes, device;
    std::vector<DecodeProblem> h_probs;  // host copy of the descriptors (hgf_group_debug edits one and re-uploads it)
    long long total_cost;
    uint32_t flags;
    void *d_mem;              // one allocation: descriptors, block offsets, workspaces
    DecodeProblem *d_probs;
    PrologueParams *d_pps;
    QuantItem *d_quant_items; // prologue: one per (problem, token)
    LoraItem *d_lora_items;   // prologue: one per (problem, 16 columns of H, K slice)
    int n_quant, n_lora;
    int4 *d_cta_range;        // per GEMV CTA: (first tile, end tile, first problem, 0)
    int grid;
};

extern "C" hgf_status hgf_group_create(const hgf_problem *problems, int32_t n, uint32_t flags, hgf_group **out) {
    return hgf_group_create_ln(problems, nullptr, n, flags, out);
}

extern "C" hgf_status hgf_group_create_ln(const hgf_problem *problems, const hgf_front_end *front_ends, int32_t n, uint32_t flags,
                                          hgf_group **out) {
    if (!problems || !out || n <= 0 || n > 65536) return HGF_ERR_INVALID_ARG;
    if (flags & HGF_FLAG_FORCE_GEMM) return HGF_ERR_INVALID_ARG;
    *out = nullptr;
    std::vector<PrologueParams> pps((size_t)n);
    std::vector<DecodeProblem> dps((size_t)n);
    std::vector<QuantItem> qitems;
    std::vector<LoraItem> litems;
    std::vector<WsLayout> lay((size_t)n);
    std::vector<int32_t> ranks((size_t)n);
    std::vector<FrontEnd> fes((size_t)n);
    std::vector<int> gate_groups((size_t)n, 1);
    std::vector<char> lns((size_t)n, 0);
    size_t ws_total = 0;
    int tiles = 0, max_M = 0, xq_smem = 0;
    long long cost = 0;
    int64_t tiles64 = 0;
    for (int i = 0; i < n; ++i) {
        const hgf_problem &q = problems[i];
        bool gemm = false;
        int32_t r = q.r;
        hgf_status st = validate_problem(q.x, q.M, q.packed, q.d_in, q.d_out, q.At, q.Bt, q.r, q.gate, q.y, flags, &r, &gemm);
        if (st != HGF_OK) return st;
        if (gemm) return HGF_ERR_UNSUPPORTED_SHAPE;  // groups hold decode-sized problems only
        {
            bool ln = false;
            st = parse_front_end(front_ends ? front_ends + i : nullptr, q.d_out, &ln, &gate_groups[i], &fes[i]);
            if (st != HGF_OK) return st;
            lns[i] = ln ? 1 : 0;
        }
        ranks[i] = r;
        lay[i] = ws_layout(q.M, q.d_in, q.d_out, r, false);
        ws_total += lay[i].total;
        // the kernels number the launch's row tiles (and the items of the prologue) with 32-bit integers
        tiles64 += row_tiles(q.d_out);
        if (tiles64 > (int64_t)1 << 30) return HGF_ERR_UNSUPPORTED_SHAPE;
    }
    const size_t off_probs = 0;
    const size_t off_pps = align_up(off_probs + sizeof(DecodeProblem) * (size_t)n, 256);
    // prologue items, and the scratch of the LoRA items: per problem (r / 16) x slices x 8 x 32 floats
    int all_M = 0;
    for (int i = 0; i < n; ++i) all_M = problems[i].M > all_M ? (int)problems[i].M : all_M;
    const int slice_k = prologue_slice_k(all_M);
    size_t n_quant = 0, n_lora = 0;
    for (int i = 0; i < n; ++i) {
        n_quant += (size_t)problems[i].M;  // an upper bound: problems that share x share their items
        n_lora += ((size_t)ranks[i] / 16) * (size_t)((problems[i].d_in + slice_k - 1) / slice_k);
    }
    if (n_quant > ((size_t)1 << 30) || n_lora > ((size_t)1 << 30)) return HGF_ERR_UNSUPPORTED_SHAPE;
    const size_t off_qit = align_up(off_pps + sizeof(PrologueParams) * (size_t)n, 256);
    const size_t off_lit = align_up(off_qit + sizeof(QuantItem) * n_quant, 256);
    const size_t off_cta = align_up(off_lit + sizeof(LoraItem) * n_lora, 256);
    const size_t off_hpart = align_up(off_cta + sizeof(int4) * 1024, 256);
    const size_t off_ws = align_up(off_hpart + n_lora * 8 * 32 * sizeof(float), 256);
    void *mem = nullptr;
    if (cudaMalloc(&mem, off_ws + ws_total) != cudaSuccess) return HGF_ERR_CUDA;
    char *ws = (char *)mem + off_ws;
    float *hpart = (float *)((char *)mem + off_hpart);
    std::unordered_map<const void *, int> first_with_x;
    for (int i = 0; i < n; ++i) {
        const hgf_problem &q = problems[i];
        fill_params(q.x, q.M, q.packed, q.gamma, q.d_in, q.d_out, q.At, q.Bt, ranks[i], q.gate, q.y, ws, lay[i], false,
                    nullptr, flags, &pps[i], &dps[i]);
        ws += lay[i].total;
        dps[i].tile_begin = tiles;
        dps[i].cost_begin = cost;
        dps[i].gate_group = gate_groups[i];
        // problems on the same input (Q, K and V of an attention block; the two up-projections of its
        // MLP) share one quantisation: a later one reads the first one's x~, scales and row sums
        int first = i;
        {
            auto seen = first_with_x.find(q.x);
            // (projections behind LayerNorms of their own - the paper's Q, K and V each have one - are
            // quantised separately unless they name the same parameters)
            if (seen == first_with_x.end()) first_with_x.emplace(q.x, i);
            else if (problems[seen->second].M == q.M && problems[seen->second].d_in == q.d_in &&
                     fes[seen->second].ln_w == fes[i].ln_w && fes[seen->second].ln_b == fes[i].ln_b &&
                     (!lns[i] || fes[seen->second].eps == fes[i].eps))
                first = seen->second;
        }
        if (first != i) {
            pps[i].xq = pps[first].xq;
            pps[i].gamma_x = pps[first].gamma_x;
            pps[i].row_sum = pps[first].row_sum;
            dps[i].xq = dps[first].xq;
            dps[i].gamma_x = dps[first].gamma_x;
            dps[i].row_sum = dps[first].row_sum;
        }
        {
            const int slices = (int)((q.d_in + slice_k - 1) / slice_k), jts = ranks[i] / 16;
            dps[i].hpart = jts ? hpart : nullptr;
            dps[i].nslices = jts ? slices : 0;
            for (int m = 0; first == i && m < (int)q.M; ++m) {
                QuantItem qi = {};
                qi.x = pps[i].x + (size_t)m * q.d_in;
                qi.xq = pps[i].xq + (size_t)m * q.d_in;
                qi.gamma_x = pps[i].gamma_x + m;
                qi.row_sum = pps[i].row_sum + m;
                qi.K = (int)q.d_in;
                if (lns[i]) {
                    qi.eps = fes[i].eps;
                    qi.ln_w = fes[i].ln_w;
                    qi.ln_b = fes[i].ln_b;
                    qi.mean_out = fes[i].dbg_mean ? fes[i].dbg_mean + m : nullptr;
                    qi.rstd_out = fes[i].dbg_rstd ? fes[i].dbg_rstd + m : nullptr;
                }
                qitems.push_back(qi);
            }
            for (int sl = 0; sl < slices; ++sl)      // slice-major: neighbouring warps share x
                for (int jt = 0; jt < jts; ++jt) {
                    const int64_t k0 = (int64_t)sl * slice_k, kvalid = q.d_in - k0 < slice_k ? q.d_in - k0 : slice_k;
                    LoraItem it;
                    it.At = (const __half *)q.At + (size_t)16 * jt * q.d_in + k0;
                    it.x = (const __nv_bfloat16 *)q.x + k0;
                    it.hpart = hpart + ((size_t)jt * slices + sl) * 8 * 32;
                    it.K = (int)q.d_in;
                    it.kvalid_M = (int)(kvalid << 8) | (int)q.M;
                    litems.push_back(it);
                }
            hpart += (size_t)jts * slices * 8 * 32;
        }
        tiles += (int)row_tiles(q.d_out);
        cost += (long long)row_tiles(q.d_out) * row_tile_cost((int)q.d_in, flags);
        max_M = q.M > max_M ? (int)q.M : max_M;
        const int xb = decode_xq_smem_bytes((int)q.M, (int)q.d_in, flags);
        xq_smem = xb > xq_smem ? xb : xq_smem;
    }
    hgf_group *g = new (std::nothrow) hgf_group();
    if (!g) { cudaFree(mem); return HGF_ERR_CUDA; }
    g->n = n; g->total_tiles = tiles; g->max_M = max_M; g->xq_smem_bytes = xq_smem;
    g->total_cost = cost;
    g->flags = flags; g->d_mem = mem;
    g->d_probs = (DecodeProblem *)((char *)mem + off_probs);
    g->d_pps = (PrologueParams *)((char *)mem + off_pps);
    g->d_quant_items = (QuantItem *)((char *)mem + off_qit);
    g->d_lora_items = (LoraItem *)((char *)mem + off_lit);
    g->n_quant = (int)qitems.size();
    g->n_lora = (int)litems.size();
    g->d_cta_range = (int4 *)((char *)mem + off_cta);
    cudaGetDevice(&g->device);
    // the GEMV's split of the launch-wide tile sequence into equal contiguous shares, one per CTA
    g->grid = decode_grid(tiles);
    std::vector<int4> ranges;
    if (g->grid > 0 && g->grid <= 1024) {
        auto tile_of_cost = [&](long long c, int *prob) {
            int lo = 0, hi = n - 1;
            while (lo < hi) {  // last problem with cost_begin <= c
                const int mid = (lo + hi + 1) >> 1;
                if (dps[mid].cost_begin <= c) lo = mid; else hi = mid - 1;
            }
            const long long steps = row_tile_cost(dps[lo].K, flags), tl = row_tiles(dps[lo].N);
            long long local = (c - dps[lo].cost_begin + steps - 1) / steps;
            if (local > tl) local = tl;
            *prob = lo;
            return dps[lo].tile_begin + (int)local;
        };
        for (int c = 0; c < g->grid; ++c) {
            int p0 = 0, p1 = 0;
            const int t0 = tile_of_cost(cost * c / g->grid, &p0);
            const int t1 = c + 1 == g->grid ? tiles : tile_of_cost(cost * (c + 1) / g->grid, &p1);
            while (p0 + 1 < n && dps[p0 + 1].tile_begin <= t0) ++p0;  // the problem that holds tile t0
            ranges.push_back(make_int4(t0, t1, p0, 0));
        }
    } else {
        g->d_cta_range = nullptr;  // the kernel works its share out itself
    }
    bool ok = cudaMemcpy(g->d_probs, dps.data(), sizeof(DecodeProblem) * (size_t)n, cudaMemcpyHostToDevice) == cudaSuccess &&
              cudaMemcpy(g->d_pps, pps.data(), sizeof(PrologueParams) * (size_t)n, cudaMemcpyHostToDevice) == cudaSuccess &&
              cudaMemcpy(g->d_quant_items, qitems.data(), sizeof(QuantItem) * qitems.size(), cudaMemcpyHostToDevice) == cudaSuccess &&
              (litems.empty() || cudaMemcpy(g->d_lora_items, litems.data(), sizeof(LoraItem) * litems.size(),
                                            cudaMemcpyHostToDevice) == cudaSuccess) &&
              (ranges.empty() ||
               cudaMemcpy(g->d_cta_range, ranges.data(), sizeof(int4) * ranges.size(), cudaMemcpyHostToDevice) == cudaSuccess);
    if (!ok) { cudaFree(mem); delete g; return HGF_ERR_CUDA; }
    g->h_probs = std::move(dps);
    *out = g;
    return HGF_OK;
}

extern "C" hgf_status hgf_group_debug(hgf_group *g, int32_t index, int32_t *y_int, hgf_debug_out *views) {
    if (!g || index < 0 || index >= g->n) return HGF_ERR_INVALID_ARG;
    if (misaligned(y_int)) return HGF_ERR_MISALIGNED;
    DecodeProblem &P = g->h_probs[(size_t)index];
    if (P.dbg_y_int != y_int) {
        P.dbg_y_int = y_int;
        if (cudaMemcpy(g->d_probs + index, &P, sizeof(DecodeProblem), cudaMemcpyHostToDevice) != cudaSuccess) return HGF_ERR_CUDA;
    }
    if (views) {
        views->xq = const_cast<int8_t *>(P.xq);
        views->gamma_x = const_cast<float *>(P.gamma_x);
        views->y_int = y_int;
        views->h = nullptr;
    }
    return HGF_OK;
}

extern "C" hgf_status hgf_group_forward_phases(hgf_group *g, uint32_t phases, void *stream_) {
    if (!g || !phases || (phases & ~(HGF_PHASE_PROLOGUE | HGF_PHASE_GEMV))) return HGF_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    const bool pdl = !(g->flags & HGF_FLAG_NO_PDL);
    if ((phases & HGF_PHASE_PROLOGUE) &&
        launch_decode_prologue_group(g->d_quant_items, g->n_quant, g->d_lora_items, g->n_lora, g->max_M, pdl,
                                     stream) != cudaSuccess)
        return HGF_ERR_CUDA;
    if (!(phases & HGF_PHASE_GEMV)) return HGF_OK;
    DecodeLaunch dl = {};
    dl.probs = g->d_probs;
    dl.n_probs = g->n;
    dl.total_tiles = g->total_tiles;
    dl.total_cost = g->total_cost;
    dl.max_M = g->max_M;
    dl.xq_smem_bytes = g->xq_smem_bytes;
    dl.cta_range = g->grid == decode_grid(g->total_tiles) ? g->d_cta_range : nullptr;
    dl.flags = g->flags;
    return launch_decode_gemv(dl, nullptr, pdl, stream) == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
}

extern "C" hgf_status hgf_group_forward(hgf_group *g, void *stream) {
    return hgf_group_forward_phases(g, HGF_PHASE_PROLOGUE | HGF_PHASE_GEMV, stream);
}

extern "C" void hgf_group_destroy(hgf_group *g) {
    if (!g) return;
    cudaFree(g->d_mem);
    delete g;
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

extern "C" hgf_status hgf_selftest_wait_timeout(uint32_t limit_us, void *stream) {
    if (limit_us == 0 || limit_us > 1000000u) return HGF_ERR_INVALID_ARG;
    return launch_wait_timeout_selftest((unsigned long long)limit_us * 1000ull, (cudaStream_t)stream) == cudaSuccess ? HGF_OK : HGF_ERR_CUDA;
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
        case HGF_ERR_TOO_LARGE: return "the problem needs more scratch than the library's built-in array holds";
    }
    return "unknown status";
}
