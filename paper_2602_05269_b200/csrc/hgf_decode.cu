// Decode path, M <= 16 tokens: one pass over the packed ternary weights (Algorithm 1, step 3),
// with the dequantisation (step 4), the LoRA up-projection (step 7) and the gated fusion (step 8)
// fused into the epilogue.  One launch serves one layer or a group of independent layers.
//
// The kernel is bound by the packed-weight stream from HBM, so it is built around keeping that
// stream busy.  One persistent CTA of 16 warps per SM.  The weights of all problems of the launch
// form one long sequence of 1 KiB tiles (16 output rows x 256 input columns); it is cut into
// contiguous shares of equal cost (weight tiles plus a fixed charge per row tile), one per CTA.
// Every warp owns a private ring of shared-memory slots (two of 4 KiB, or three to four of 2 KiB)
// that one of its lanes keeps filled with bulk asynchronous copies (cp.async.bulk, completion on an
// mbarrier), several tiles ahead of their use and across row-tile, layer and (under programmatic
// dependent launch) kernel boundaries, so the number of bytes in flight does not depend on what
// the math is doing.  A warp consumes a row tile (16 output rows, all of K or a K slice of it):
// per 1 KiB tile two 128-bit shared-memory loads per lane bring the 2-bit codes in the register
// layout of the warp-level int8 MMA (m16n8k32, u8 x s8 -> s32; the 16-row operand holds weight
// rows, the 8-column operand the tokens), one AND per register isolates the codes in place (scaled
// by 1, 4, 16 or 64; each scale has its own accumulator and the exact quotients are added at the
// end).  Codes are t + 1, so sum_k t x~ = sum_k c x~ - sum_k x~ (the row sums come from the
// quantisation kernel).  The quantised activations of the layer at hand sit in shared memory.
// The epilogue runs the rank-r up-projection on the same MMA unit (f16 inputs; SiLU(x A) enters as
// an fp16 value plus an fp16 residual, so nothing is lost against fp32), in the accumulator layout
// of the integer result, and writes y.
#include "hgf_common.cuh"

namespace hgf {

constexpr int kDecWarps = 16;
constexpr int kDecThreads = kDecWarps * 32;
constexpr int kTileBytes = 1024;     // one 16 x 256 weight tile
// A warp's ring is either two slots of four tiles (fewer, larger copies and hand-overs: measured
// 6 % faster) or, when the activations leave no room for that, three to four slots of two tiles.
constexpr int kBigSlotTiles = 4, kBigSlots = 2;
constexpr int kSmallSlotTiles = 2;
constexpr int kMaxSlots = 4;         // slots per warp ring at most (barriers are laid out for that many)
constexpr int kMinSlots = 3;         // small slots at least: what bounds the activations' share of shared memory
constexpr int kXqPad = 64;           // row padding of the activations in shared memory (bank spread)
constexpr int kHPitch = 72;          // halves per row of H in shared memory (r <= 64, + 8 bank spread)

// shared-memory map: fixed part, then the activations, then the rings
constexpr int kOffBars = 0;
constexpr int kOffSmall = kOffBars + kDecWarps * kMaxSlots * 8;
struct SegSmall {                    // per-problem values the epilogue needs
    float scale[16];                 // gamma_x[m] * gamma_W / 127
    int row_sum[16];
    __half h_hi[16][kHPitch];
    __half h_lo[16][kHPitch];
    void *y;
    int32_t *dbg_y_int;
    const float *gate;
    uint32_t flags;
    int gate_group;
};
constexpr int kOffRed = kOffSmall + 2 * (int)sizeof(SegSmall);
constexpr int kRedBytes = kDecWarps * 8 * 32 * 4;  // per warp: up to 8 accumulator registers per lane
constexpr int kOffFlags = kOffRed + kRedBytes;
constexpr int kOffXq = (kOffFlags + 64 + 127) / 128 * 128;
constexpr int kSmemLimit = 227 * 1024;
// Base-3 weights: the decode table (byte value -> its first four codes, one per byte of a word) is
// a static shared array with one copy per lane (entry b of lane l at word 32 b + l), so that a warp's
// 32 look-ups of unrelated bytes never meet in a bank.  A byte's fifth code is found arithmetically.
constexpr int kLutBytes = 256 * 32 * 4;
constexpr int kXqLimit = (kSmemLimit - kOffXq - kMinSlots * kDecWarps * kSmallSlotTiles * kTileBytes) / 128 * 128;

constexpr unsigned long long kDecWaitLimitNs = 2000000000ull;  // bounded waits give up after two seconds

// Rows of activations kept in shared memory: the M tokens, plus one row of zeros that stands in for
// the absent tokens of the 8-token tiles.
int decode_xq_smem_bytes(int M, int K, uint32_t flags) {
    const int Kp = (flags & HGF_FLAG_BASE3) ? (int)padded_k_b3(K) : (int)padded_k(K);
    return (M + (M < 16 ? 1 : 0)) * (Kp + kXqPad);
}
// (With the base-3 table in shared memory a ring of two small slots per warp is accepted, which gives
// the same limit as three slots without the table.)
int decode_xq_smem_limit(uint32_t flags) {
    if (!(flags & HGF_FLAG_BASE3)) return kXqLimit;
    return (kSmemLimit - kOffXq - kLutBytes - 2 * kDecWarps * kSmallSlotTiles * kTileBytes) / 128 * 128;
}

// ---- PTX wrappers -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t dsmem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void dmbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ bool dmbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// One bulk copy global -> shared of `bytes` (a multiple of 16; both addresses 16-byte aligned),
// completing on the mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void bulk_prefetch_l2(const void *src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void *ptr) {
    asm volatile("prefetch.global.L2 [%0];\n" ::"l"(ptr));
}
__device__ __forceinline__ unsigned long long dec_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
    return t;
}
// Programmatic dependent launch: both are no-ops when the launch carries no such attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }

// ---- work decomposition -------------------------------------------------------------------------
// A segment is the run of row tiles of one problem that falls into this CTA's share.  Its tiles are
// dealt to the 16 warps in rounds of 16 whole tiles; a last round with fewer tiles than warps
// splits each tile's K range into slices so that every warp has work, and the slices are added
// through shared memory.
struct Seg {
    int p;                   // problem index
    int lo, hi;              // launch-wide tile range [lo, hi) of the segment
    int tile_begin;          // first launch-wide tile of the problem
    int nsteps;              // 1 KiB tiles per row tile (padded K / 256)
    const uint8_t *packed;
};
struct Item {
    int tile_local;          // row tile inside the problem
    int ks0, ks1;            // column tiles [ks0, ks1)
    int S, slice;            // number of K slices of the row tile, and this warp's
    bool valid;
};

__device__ __forceinline__ const DecodeProblem &problem_of(const DecodeLaunch &L, const DecodeProblem &single, int p) {
    return L.probs ? L.probs[p] : single;
}
__device__ __forceinline__ int b3_col(int p, int t) { return 32 * (p >> 1) + 16 * (p & 1) + 4 * t; }
__device__ __forceinline__ int tiles_of(int N) { return (N + 15) >> 4; }

// Smallest launch-wide tile index at which the cost of all earlier row tiles is >= cost.
__device__ int tile_of_cost(const DecodeLaunch &L, const DecodeProblem &single, long long cost) {
    int lo = 0, hi = L.n_probs - 1;
    while (lo < hi) {  // last problem with cost_begin <= cost
        const int mid = (lo + hi + 1) >> 1;
        if (problem_of(L, single, mid).cost_begin <= cost) lo = mid; else hi = mid - 1;
    }
    const DecodeProblem &P = problem_of(L, single, lo);
    const long long steps = row_tile_cost(P.K, P.flags);
    const int tiles = tiles_of(P.N);
    long long local = (cost - P.cost_begin + steps - 1) / steps;
    if (local > tiles) local = tiles;
    return P.tile_begin + (int)local;
}

// First segment (first = true) or the one after `s`, inside the CTA's tile range [t0, t1).
// p_first >= 0 names the problem that holds tile t0 (saves the search).
__device__ bool next_segment(const DecodeLaunch &L, const DecodeProblem &single, int t0, int t1, bool first, Seg &s,
                             int p_first = -1) {
    if (t0 >= t1) return false;
    int p;
    if (first && p_first >= 0) {
        p = p_first;
    } else if (first) {
        int lo = 0, hi = L.n_probs - 1;
        while (lo < hi) {  // last problem with tile_begin <= t0
            const int mid = (lo + hi + 1) >> 1;
            if (problem_of(L, single, mid).tile_begin <= t0) lo = mid; else hi = mid - 1;
        }
        p = lo;
    } else {
        p = s.p + 1;
    }
    for (; p < L.n_probs; ++p) {
        const DecodeProblem &P = problem_of(L, single, p);
        const int tb = P.tile_begin, te = tb + tiles_of(P.N);
        if (tb >= t1) return false;
        const int lo = t0 > tb ? t0 : tb, hi = t1 < te ? t1 : te;
        if (lo < hi) {
            s.p = p; s.lo = lo; s.hi = hi; s.tile_begin = tb; s.nsteps = weight_steps(P.K, P.flags); s.packed = P.packed;
            return true;
        }
    }
    return false;
}
__device__ __forceinline__ int seg_rounds(const Seg &s) { return (s.hi - s.lo + kDecWarps - 1) / kDecWarps; }

__device__ __forceinline__ Item seg_item(const Seg &s, int round, int warp) {
    const int n = s.hi - s.lo, full = n / kDecWarps, rem = n % kDecWarps;
    Item it;
    if (round < full) {
        it.tile_local = s.lo - s.tile_begin + round * kDecWarps + warp;
        it.ks0 = 0; it.ks1 = s.nsteps; it.S = 1; it.slice = 0; it.valid = true;
    } else {
        int S = kDecWarps / rem;
        S = S < s.nsteps ? S : s.nsteps;
        const int tix = warp / S, sl = warp - tix * S;
        it.valid = tix < rem;
        it.tile_local = s.lo - s.tile_begin + full * kDecWarps + tix;
        it.ks0 = sl * s.nsteps / S; it.ks1 = (sl + 1) * s.nsteps / S;
        it.S = S; it.slice = sl;
    }
    return it;
}

// The copy-issuing side of a warp's ring: walks the same item sequence as the consumer.  All
// lanes keep the (warp-uniform) state; lane 0 issues.
struct Producer {
    Seg seg;
    int round, rounds;
    int left;                // 1 KiB tiles of the current item not yet requested
    const uint8_t *src;      // the next of them
    const __half *bt_src;    // rows of B^T the item's epilogue reads (requested after its last tile)
    int bt_bytes;            // 0 when the item has no epilogue of its own or the layer has no correction
    bool done;
};

// NT = number of 8-token tiles (1: M <= 8, 2: M <= 16); ST = tiles per ring slot; B3 = the weights
// are in the base-3 layout (tiles of 320 columns, decoded through a table in shared memory).
template <int NT, int ST, bool B3>
__global__ void __launch_bounds__(kDecThreads, 1)
decode_gemv_kernel(const DecodeLaunch L, const DecodeProblem single, unsigned int *status) {
    constexpr int kSlotTiles = ST, kSlotBytes = ST * kTileBytes;
    constexpr int kTileCols = B3 ? 320 : 256;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int slots = L.ring_slots;  // slots of this warp's ring, kSlotBytes each
    uint8_t *ring = smem + kOffXq + ((L.xq_smem_bytes + 127) & ~127) + warp * slots * kSlotBytes;
    const uint32_t ring_u32 = dsmem_u32(ring);
    const uint32_t bars_u32 = dsmem_u32(smem + kOffBars) + warp * kMaxSlots * 8;
    SegSmall *small = reinterpret_cast<SegSmall *>(smem + kOffSmall);
    int *red = reinterpret_cast<int *>(smem + kOffRed);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffFlags);
    int8_t *xq_s = reinterpret_cast<int8_t *>(smem + kOffXq);

    pdl_launch_dependents();
    if (tid == 0) *abort_flag = 0;
    uint32_t lut_lane = 0;  // shared-window address of this lane's copy of the table
    if constexpr (B3) {
        // Values above 242 never occur in a packed matrix; they decode as zero weights (code 1).
        __shared__ __align__(128) uint32_t b3_lut[256 * 32];
        for (int i = tid; i < 256 * 32; i += kDecThreads) {
            const int b = i >> 5;
            b3_lut[i] = b <= 242 ? ((uint32_t)(b % 3) | ((uint32_t)(b / 3 % 3) << 8) | ((uint32_t)(b / 9 % 3) << 16) | ((uint32_t)(b / 27 % 3) << 24))
                                 : 0x01010101u;
        }
        lut_lane = dsmem_u32(b3_lut) + 4 * lane;
    }
    if (lane == 0) {
        for (int s = 0; s < slots; ++s) dmbar_init(bars_u32 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncthreads();

    // this CTA's share of the launch-wide tile sequence
    int t0, t1, p_first = -1;
    if (L.cta_range) {  // precomputed on the host for a group
        const int4 cr = L.cta_range[blockIdx.x];
        t0 = cr.x; t1 = cr.y; p_first = cr.z;
    } else {
        const long long c0 = L.total_cost * (long long)blockIdx.x / (long long)gridDim.x;
        const long long c1 = L.total_cost * (long long)(blockIdx.x + 1) / (long long)gridDim.x;
        t0 = tile_of_cost(L, single, c0);
        t1 = (blockIdx.x + 1 == gridDim.x) ? L.total_tiles : tile_of_cost(L, single, c1);
    }

    // ---- producer ------------------------------------------------------------------------------
    // A slot receives up to kSlotTiles consecutive tiles of one item; items are cut into slots from
    // their first tile on, so the consumer knows each slot's size from its own position.
    Producer pr;
    pr.left = 0; pr.round = -1; pr.rounds = 0; pr.src = nullptr; pr.bt_src = nullptr; pr.bt_bytes = 0;
    pr.done = !next_segment(L, single, t0, t1, true, pr.seg, p_first);
    if (!pr.done) pr.rounds = seg_rounds(pr.seg);

    auto next_item = [&]() {  // slow path of the producer: find this warp's next item with work
        while (!pr.done && pr.left == 0) {
            if (++pr.round >= pr.rounds) {
                if (!next_segment(L, single, t0, t1, false, pr.seg)) { pr.done = true; break; }
                pr.rounds = seg_rounds(pr.seg);
                pr.round = 0;
            }
            const Item it = seg_item(pr.seg, pr.round, warp);
            if (it.valid && it.ks0 < it.ks1) {
                pr.left = it.ks1 - it.ks0;
                pr.src = pr.seg.packed + ((size_t)it.tile_local * pr.seg.nsteps + it.ks0) * kTileBytes;
                if (it.slice == 0) {  // this warp runs the row tile's epilogue
                    const DecodeProblem &P = problem_of(L, single, pr.seg.p);
                    const int r = P.r, n0 = it.tile_local * 16, rows = P.N - n0 < 16 ? P.N - n0 : 16;
                    pr.bt_bytes = rows * r * 2;
                    pr.bt_src = P.Bt + (size_t)n0 * r;
                }
            }
        }
    };
    // Request the next slot's worth of this warp's sequence into `slot`: up to kSlotTiles consecutive
    // tiles of an item, or (after the item's last tile) the rows of B^T for its epilogue.
    auto produce = [&](int slot) {
        const uint32_t dst = ring_u32 + slot * kSlotBytes, bar = bars_u32 + 8 * slot;
        if (pr.left == 0) {
            if (pr.bt_bytes) {
                if (lane == 0) bulk_load(dst, pr.bt_src, (uint32_t)pr.bt_bytes, bar);
                pr.bt_bytes = 0;
                return;
            }
            next_item();
            if (pr.done) return;
        }
        const int n = pr.left < kSlotTiles ? pr.left : kSlotTiles;
        if (lane == 0) bulk_load(dst, pr.src, (uint32_t)(n * kTileBytes), bar);
        pr.src += n * kTileBytes;
        pr.left -= n;
    };
#pragma unroll 1
    for (int i = 0; i < slots; ++i) produce(i);

    // everything above reads only weights; the activations come from the preceding launch
    pdl_wait();

    // ---- consumer ------------------------------------------------------------------------------
    int cslot = 0;          // slot the next tiles arrive in
    uint32_t cpar = 0;      // and its mbarrier phase
    bool ok = true;         // false once a wait gave up (this warp stops computing but keeps the barriers)
    Seg seg;
    int seg_idx = 0;
    for (bool more = next_segment(L, single, t0, t1, true, seg, p_first); more;
         more = next_segment(L, single, t0, t1, false, seg), ++seg_idx) {
        const DecodeProblem &Pg = problem_of(L, single, seg.p);
        const int K = Pg.K, M = Pg.M, N = Pg.N, r = Pg.r;
        const int Kp = seg.nsteps * kTileCols, pitch = Kp + kXqPad;
        SegSmall &sm = small[seg_idx & 1];

        // stage the problem's activations and per-token values (all reads of the previous
        // segment's activations ended at the barrier that closed it)
        {
            const int8_t *xq_g = Pg.xq;
            // Shared-memory order of a token's bytes, per 256-column tile: the lane with t = lane % 4
            // owns columns 64 t .. 64 t + 63; of each 32 of them (4-byte groups G0 .. G7) it reads two
            // 16-byte units, [G0 G4 G1 G5] and [G2 G6 G3 G7], so that the two registers one MMA takes
            // (columns c .. c + 3 and c + 16 .. c + 19) come out of one load next to each other.  Unit
            // u = 0 .. 3 of lane t sits at byte 64 u + 16 t of the tile: the four lanes of a token read
            // 64 consecutive bytes, and the row padding puts the next token on the other banks.
            const int groups_per_row = Kp >> 5;
            if (M < 16)  // the row of zeros
                for (int u = tid; u < (Kp >> 4); u += kDecThreads)
                    *reinterpret_cast<uint4 *>(xq_s + (size_t)M * pitch + 16 * u) = make_uint4(0u, 0u, 0u, 0u);
            if (B3) {
                // Base-3 tiles have 320 columns; lane t's five 16-byte units of a tile sit at bytes
                // 64 u + 16 t of it and hold, four bytes each, the columns col(4 u + i, t) .. + 3, i = 0..3 -
                // the second operands of the MMAs whose first operands come out of the lane's 16 weight bytes.
                const int units_per_row = seg.nsteps * 20;
                for (int v = tid; v < M * units_per_row; v += kDecThreads) {
                    const int m = v / units_per_row, rem = v - m * units_per_row, c = rem / 20, ut = rem - c * 20, u = ut >> 2, tt = ut & 3;
                    uint32_t r4[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int k = c * 320 + b3_col(4 * u + i, tt);
                        r4[i] = k < K ? *reinterpret_cast<const uint32_t *>(xq_g + (size_t)m * K + k) : 0u;
                    }
                    *reinterpret_cast<uint4 *>(xq_s + (size_t)m * pitch + c * 320 + 64 * u + 16 * tt) = make_uint4(r4[0], r4[1], r4[2], r4[3]);
                }
            }
            for (int u = tid; !B3 && u < M * groups_per_row; u += kDecThreads) {
                const int m = u / groups_per_row, q = u - m * groups_per_row;
                uint4 v0 = make_uint4(0u, 0u, 0u, 0u), v1 = v0;
                if (32 * q < K) {
                    v0 = *reinterpret_cast<const uint4 *>(xq_g + (size_t)m * K + 32 * q);
                    v1 = *reinterpret_cast<const uint4 *>(xq_g + (size_t)m * K + 32 * q + 16);
                }
                const int tq = q & 7, tt = tq >> 1, h = tq & 1;
                int8_t *dst = xq_s + (size_t)m * pitch + ((q >> 3) << 8) + 16 * tt + 128 * h;
                *reinterpret_cast<uint4 *>(dst) = make_uint4(v0.x, v1.x, v0.y, v1.y);
                *reinterpret_cast<uint4 *>(dst + 64) = make_uint4(v0.z, v1.z, v0.w, v1.w);
            }
            if (tid < 16) {
                sm.scale[tid] = tid < M ? Pg.gamma_x[tid] * Pg.gw_over_127 : 0.0f;
                sm.row_sum[tid] = tid < M ? Pg.row_sum[tid] : 0;
            }
            if (tid == 32) { sm.y = Pg.y; sm.dbg_y_int = Pg.dbg_y_int; sm.gate = Pg.gate; sm.flags = Pg.flags; sm.gate_group = Pg.gate_group; }
            if (Pg.nslices > 0) {
                // group launch: H = act(sum over K slices of the parked partial sums of x A), slices in
                // order.  The partial sums sit in the tf32 MMA's accumulator layout: column j = 16 jt + jl
                // and token m are register 4 (m / 8) + 2 (jl / 8) + (m % 2) of lane 4 (jl % 8) + (m % 8) / 2.
                const float *hp = Pg.hpart;
                const int ns = Pg.nslices;
                const bool no_silu = (Pg.flags & HGF_FLAG_NO_SILU) != 0;
                for (int u = tid; u < M * r; u += kDecThreads) {
                    const int m = u / r, j = u - m * r, jt = j >> 4, jl = j & 15;
                    const int idx = 4 * (m >> 3) + 2 * (jl >> 3) + (m & 1), ln = 4 * (jl & 7) + ((m & 7) >> 1);
                    const float *src = hp + ((size_t)jt * ns * 8 + idx) * 32 + ln;
                    float z = 0.0f;
                    int sl = 0;
                    for (; sl + 4 <= ns; sl += 4) {  // four loads in flight, added in slice order
                        const float z0 = __ldcg(src + (size_t)sl * 256), z1 = __ldcg(src + (size_t)(sl + 1) * 256);
                        const float z2 = __ldcg(src + (size_t)(sl + 2) * 256), z3 = __ldcg(src + (size_t)(sl + 3) * 256);
                        z += z0; z += z1; z += z2; z += z3;
                    }
                    for (; sl < ns; ++sl) z += __ldcg(src + (size_t)sl * 256);
                    const float h = no_silu ? z : silu_f(z);
                    const __half hi = __float2half_rn(h);
                    sm.h_hi[m][j] = hi;
                    sm.h_lo[m][j] = __float2half_rn(h - __half2float(hi));
                }
            } else {
                const int words = r >> 1;  // 32-bit words per row of H
                const uint32_t *hi_g = reinterpret_cast<const uint32_t *>(Pg.h_hi), *lo_g = reinterpret_cast<const uint32_t *>(Pg.h_lo);
                for (int u = tid; u < M * words; u += kDecThreads) {
                    const int m = u / words, w = u - m * words;
                    reinterpret_cast<uint32_t *>(&sm.h_hi[m][0])[w] = hi_g[u];
                    reinterpret_cast<uint32_t *>(&sm.h_lo[m][0])[w] = lo_g[u];
                }
            }
        }
        __syncthreads();

        // Bounded wait for the slot the next part of this warp's sequence arrives in.
        auto wait_slot = [&]() -> bool {
            const uint32_t bar = bars_u32 + 8 * cslot;
            bool got = dmbar_try_wait(bar, cpar);
            if (__all_sync(0xffffffffu, got)) return true;  // the whole warp takes the same path
            unsigned long long t_start = 0;
            uint32_t polls = 0;
            while (!got && !(got = dmbar_try_wait(bar, cpar))) {
                if ((++polls & 255u) == 0) {
                    const unsigned long long now = dec_timer_ns();
                    if (t_start == 0) t_start = now;
                    else if (now - t_start > kDecWaitLimitNs || *abort_flag) break;
                }
            }
            if (!got) { *abort_flag = 1; if (lane == 0) atomicExch(status, 0x500u + (unsigned)warp); }
            return __all_sync(0xffffffffu, got);
        };
        auto release_slot = [&]() {  // every lane has read the slot: refill it, move on
            __syncwarp();
            produce(cslot);
            if (++cslot == slots) { cslot = 0; cpar ^= 1u; }
        };
        // Epilogue of one row tile: dequantise, add the gated rank-r correction, store.  v holds
        // sum_k c x~ in the MMA accumulator layout: register c of token tile nt is row g + 8 (c >> 1),
        // token 8 nt + 2 t + (c & 1).  The correction runs on the f16 MMA: the tile's rows of B^T (which
        // arrive in a ring slot of their own) are the 16-row operand, H^T (fp16 value + fp16 residual)
        // the 8-column operand.  Returns false if the wait for B^T gave up.
        auto epilogue = [&](int n0, const int (&v)[NT][4]) -> bool {
            float corr[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) corr[nt][c] = 0.0f;
            float gA = 0.0f, gB = 0.0f;
            if (r > 0) {
                const float *gate = sm.gate;
                if (sm.gate_group > 1) {  // grouped gate (per head, or scalar): groups are whole row tiles
                    gA = gB = __ldg(gate + n0 / sm.gate_group);
                } else {
                    gA = __ldg(gate + (n0 + g < N ? n0 + g : N - 1));
                    gB = __ldg(gate + (n0 + g + 8 < N ? n0 + g + 8 : N - 1));
                }
                if (!wait_slot()) return false;
                const int rows = N - n0 < 16 ? N - n0 : 16;
                const uint32_t *bA = reinterpret_cast<const uint32_t *>(ring + cslot * kSlotBytes) + (g < rows ? g : rows - 1) * (r >> 1) + t;
                const uint32_t *bB = reinterpret_cast<const uint32_t *>(ring + cslot * kSlotBytes) + (g + 8 < rows ? g + 8 : rows - 1) * (r >> 1) + t;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    if (16 * kk < r) {
                        const uint32_t a0 = bA[8 * kk], a1 = bB[8 * kk], a2 = bA[8 * kk + 4], a3 = bB[8 * kk + 4];
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            uint32_t h0 = 0, h1 = 0, l0 = 0, l1 = 0;
                            if (g + 8 * nt < M) {
                                const uint32_t *hh = reinterpret_cast<const uint32_t *>(&sm.h_hi[g + 8 * nt][0]);
                                const uint32_t *hl = reinterpret_cast<const uint32_t *>(&sm.h_lo[g + 8 * nt][0]);
                                h0 = hh[8 * kk + t]; h1 = hh[8 * kk + 4 + t];
                                l0 = hl[8 * kk + t]; l1 = hl[8 * kk + 4 + t];
                            }
                            mma_f16(corr[nt], a0, a1, a2, a3, h0, h1);
                            mma_f16(corr[nt], a0, a1, a2, a3, l0, l1);
                        }
                    }
                }
                release_slot();
            }
            void *y_out = sm.y;
            int32_t *dbg_y_int = sm.dbg_y_int;
            const bool out_bf16 = (sm.flags & HGF_FLAG_OUT_BF16) != 0;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int m = 8 * nt + 2 * t + (c & 1), n = n0 + g + 8 * (c >> 1);
                    if (m < M && n < N) {
                        const int y_int = v[nt][c] - sm.row_sum[m];
                        const float y = fmaf(c >> 1 ? gB : gA, corr[nt][c], (float)y_int * sm.scale[m]);
                        const size_t o = (size_t)m * N + n;
                        if (out_bf16)
                            reinterpret_cast<__nv_bfloat16 *>(y_out)[o] = __float2bfloat16_rn(y);
                        else
                            reinterpret_cast<float *>(y_out)[o] = y;
                        if (dbg_y_int) dbg_y_int[o] = y_int;
                    }
                }
            return true;
        };

        const int rounds = seg_rounds(seg);
        const int full_rounds = (seg.hi - seg.lo) / kDecWarps;
        int last_tile = -1, last_S = 1;  // the row tile whose epilogue this warp runs after the barrier

        // this lane's activation bytes: token g + 8 nt (an absent token reads the row of zeros), units
        // at bytes 16 t + 64 u of each tile
        const int8_t *xrow[NT];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) xrow[nt] = xq_s + (size_t)(g + 8 * nt < M ? g + 8 * nt : M) * pitch + 16 * t;

        for (int round = 0; round < rounds; ++round) {
            const Item it = seg_item(seg, round, warp);
            if (!it.valid || it.ks0 >= it.ks1) continue;

            int acc[NT][4][4];
#pragma unroll
            for (int a = 0; a < NT; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b)
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[a][b][c] = 0;

            // one 16 x 256 tile at shared-memory address `wt` against the activations at `xt`
            auto compute_tile = [&](const uint8_t *wt, const int8_t *const (&xt)[NT]) {
                const uint4 pq = *reinterpret_cast<const uint4 *>(wt);
                const uint4 qq = *reinterpret_cast<const uint4 *>(wt + 512);
                const uint32_t pw[4] = {pq.x, pq.y, pq.z, pq.w};
                const uint32_t qw[4] = {qq.x, qq.y, qq.z, qq.w};
                if constexpr (B3) {
                    // The lane's 16 bytes of row g (pw) and of row g + 8 (qw): byte 4 w + e gives, through the
                    // table, the first operand of one half of MMA 2 w + e / 2 (four codes), and the fifth codes
                    // of a word's four bytes together make one operand register of MMAs 8 and 9.
                    uint32_t f5g[4], f5h[4];
                    // fifth codes of a word's four bytes, one per byte: [b >= 81] + [b >= 162], from carries
                    // into bit 7 of the bytes' low seven bits (no carry crosses a byte: 127 + 94 < 256)
                    auto fifth = [](uint32_t w) {
                        const uint32_t u = w & 0x7f7f7f7fu;
                        const uint32_t ge81 = ((u + 0x2f2f2f2fu) | w) & 0x80808080u;
                        const uint32_t ge162 = (u + 0x5e5e5e5eu) & w & 0x80808080u;
                        return (ge81 >> 7) + (ge162 >> 7);
                    };
                    auto look_up = [&](uint32_t w, int e) {
                        // byte e of w, times 128 (the table's stride), plus the lane's base address
                        const uint32_t idx = (e == 0 ? (w << 7) : (w >> (8 * e - 7))) & 0x7f80u;
                        uint32_t v;
                        asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(lut_lane + idx));
                        return v;
                    };
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        uint32_t ag[4], ah[4];
                        f5g[w] = fifth(pw[w]);
                        f5h[w] = fifth(qw[w]);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            ag[e] = look_up(pw[w], e);
                            ah[e] = look_up(qw[w], e);
                        }
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const uint4 xv = *reinterpret_cast<const uint4 *>(xt[nt] + 64 * w);
                            mma_u8s8(acc[nt][0], ag[0], ah[0], ag[1], ah[1], xv.x, xv.y);
                            mma_u8s8(acc[nt][0], ag[2], ah[2], ag[3], ah[3], xv.z, xv.w);
                        }
                    }
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint4 xv = *reinterpret_cast<const uint4 *>(xt[nt] + 64 * 4);
                        mma_u8s8(acc[nt][0], f5g[0], f5h[0], f5g[1], f5h[1], xv.x, xv.y);
                        mma_u8s8(acc[nt][0], f5g[2], f5h[2], f5g[3], f5h[3], xv.z, xv.w);
                    }
                } else {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint4 xa[NT], xb[NT];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        xa[nt] = *reinterpret_cast<const uint4 *>(xt[nt] + 64 * (2 * h));
                        xb[nt] = *reinterpret_cast<const uint4 *>(xt[nt] + 64 * (2 * h + 1));
                    }
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        const uint32_t mask = 0x03030303u << (2 * jj);
                        const uint32_t a0 = pw[2 * h] & mask, a1 = qw[2 * h] & mask;
                        const uint32_t a2 = pw[2 * h + 1] & mask, a3 = qw[2 * h + 1] & mask;
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const uint4 &xv = jj < 2 ? xa[nt] : xb[nt];
                            if (jj & 1) mma_u8s8(acc[nt][jj], a0, a1, a2, a3, xv.z, xv.w);
                            else mma_u8s8(acc[nt][jj], a0, a1, a2, a3, xv.x, xv.y);
                        }
                    }
                }
                }
            };
            const int8_t *xt[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) xt[nt] = xrow[nt] + it.ks0 * kTileCols;
            const int ntiles = it.ks1 - it.ks0;
            for (int left = ntiles; left > 0 && ok;) {  // slot by slot; the last may hold fewer tiles
                if (!(ok = wait_slot())) break;  // stop computing and copying; requested slots stay outstanding
                const uint8_t *sl = ring + cslot * kSlotBytes + 16 * lane;
                const int n = left < kSlotTiles ? left : kSlotTiles;
#pragma unroll
                for (int q = 0; q < kSlotTiles; ++q) {
                    if (q < n) {
                        compute_tile(sl + q * kTileBytes, xt);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) xt[nt] += kTileCols;
                    }
                }
                release_slot();
                left -= n;
            }

            // exact rescale of the four accumulators
            int v[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    v[nt][c] = acc[nt][0][c] + (acc[nt][1][c] >> 2) + (acc[nt][2][c] >> 4) + (acc[nt][3][c] >> 6);

            if (round < full_rounds) {  // a whole row tile: its epilogue runs right away
                if (ok) ok = epilogue(it.tile_local * 16, v);
                continue;
            }
            // last round: park the sums (K slices are added after the barrier)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) red[(warp * 8 + nt * 4 + c) * 32 + lane] = v[nt][c];
            if (it.slice == 0) { last_tile = it.tile_local; last_S = it.S; }
        }

        __syncthreads();  // partial sums are parked; every read of this segment's activations is done

        // ---- epilogue of the last round (after adding K slices) ----------------------------------
        if (ok && last_tile >= 0) {
            int v[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    int s = 0;
                    for (int w = 0; w < last_S; ++w) s += red[((warp + w) * 8 + nt * 4 + c) * 32 + lane];
                    v[nt][c] = s;
                }
            ok = epilogue(last_tile * 16, v);
        }
    }

    // A warp that stopped early still has copies in flight: wait (bounded) for them before leaving.
    if (!ok) {
        for (int q = 0; q < slots; ++q) {
            for (uint32_t i = 0; i < (1u << 16) && !dmbar_try_wait(bars_u32 + 8 * cslot, cpar); ++i) {}
            if (++cslot == slots) { cslot = 0; cpar ^= 1u; }
        }
    }
}

int decode_grid(int total_tiles) {
    const int sms = device_sm_count();
    return total_tiles < sms ? total_tiles : sms;
}

template <int NT, int ST, bool B3>
static cudaError_t launch_decode_variant(cudaLaunchConfig_t &cfg, const DecodeLaunch &L, const DecodeProblem &sp, unsigned int *status) {
    static std::atomic<unsigned long long> attr_done{0};
    cudaError_t e = ensure_dynamic_smem(decode_gemv_kernel<NT, ST, B3>, kSmemLimit - (B3 ? kLutBytes : 0), attr_done);
    if (e != cudaSuccess) return e;
    return cudaLaunchKernelEx(&cfg, decode_gemv_kernel<NT, ST, B3>, L, sp, status);
}
template <bool B3>
static cudaError_t launch_decode_layout(cudaLaunchConfig_t &cfg, const DecodeLaunch &L, const DecodeProblem &sp, unsigned int *status, bool big) {
    if (L.max_M <= 8)
        return big ? launch_decode_variant<1, kBigSlotTiles, B3>(cfg, L, sp, status) : launch_decode_variant<1, kSmallSlotTiles, B3>(cfg, L, sp, status);
    return big ? launch_decode_variant<2, kBigSlotTiles, B3>(cfg, L, sp, status) : launch_decode_variant<2, kSmallSlotTiles, B3>(cfg, L, sp, status);
}

cudaError_t launch_decode_gemv(const DecodeLaunch &L_in, const DecodeProblem *single, bool pdl, cudaStream_t stream) {
    const int grid = decode_grid(L_in.total_tiles);
    if (grid <= 0) return cudaErrorInvalidDevice;
    if (L_in.xq_smem_bytes > decode_xq_smem_limit(single ? single->flags : L_in.flags)) return cudaErrorInvalidValue;
    unsigned int *status = device_status_word();
    if (!status) return cudaErrorMemoryAllocation;
    DecodeLaunch L = L_in;
    // the ring beside the activations: two slots of four tiles if they fit, else as many slots of two
    // tiles as shared memory allows
    const bool b3 = ((single ? single->flags : L_in.flags) & HGF_FLAG_BASE3) != 0;
    const int lut = b3 ? kLutBytes : 0;
    const int xq_bytes = (L.xq_smem_bytes + 127) & ~127;
    const int room = kSmemLimit - kOffXq - lut - xq_bytes;
    const bool big = room >= kDecWarps * kBigSlots * kBigSlotTiles * kTileBytes;
    const int slot_bytes = (big ? kBigSlotTiles : kSmallSlotTiles) * kTileBytes;
    int slots = big ? kBigSlots : room / (kDecWarps * slot_bytes);
    slots = slots > kMaxSlots ? kMaxSlots : slots;
    L.ring_slots = slots;
    DecodeProblem dummy = {};
    const DecodeProblem &sp = single ? *single : dummy;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kDecThreads);
    cfg.dynamicSmemBytes = (size_t)(kOffXq + xq_bytes + kDecWarps * slots * slot_bytes);  // (the table is static shared memory)
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    cudaError_t e = b3 ? launch_decode_layout<true>(cfg, L, sp, status, big) : launch_decode_layout<false>(cfg, L, sp, status, big);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace hgf
