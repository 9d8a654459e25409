// GEMM path (M > 16 tokens): Y_int = X~ x T^T on the 5th-generation tensor cores
// (tcgen05.mma kind::i8, int32 accumulator in tensor memory), with the dequantisation, the LoRA
// up-projection (a small tcgen05.mma kind::f16 on top of the dequantised accumulator, with the gate
// folded into B) and the gated fusion in the epilogue.  Algorithm 1, steps 3, 4, 7, 8.
//
// The ternary weights are the MMA's first operand and are read from TENSOR MEMORY: the tensor core
// cannot read 2-bit codes, and expanding them to int8 in shared memory costs four times their bytes
// in shared-memory writes plus the same again when the MMA reads them - more than the port has.
// Here four warps expand a packed 128 x 256 tile straight from its 8 KiB in shared memory into
// registers (one 128-channel row per thread: a shift and a mask per register) and store it with two
// tcgen05.st into the operand's place in tensor memory, so shared memory carries only the int8
// activation tile (TMA in, MMA out) and the packed codes.  The output tile is therefore
// 128 output channels (tensor-memory lanes, MMA M) x 128 tokens (columns, MMA N); two accumulators
// alternate, so the epilogue of a tile runs under the main loop of the next.  A pipeline stage is
// 256 input columns (eight MMAs): every hand-over between the roles costs a shared-memory round
// trip, and the single MMA-issuing thread can only afford one per 512 tensor-core clocks.
//
// One persistent CTA per SM, 16 warps with fixed roles:
//   warp 0      producer (all lanes): per stage the int8 activation tile as two 128 tokens x 128 B
//               boxes (128-byte swizzle) and the packed weights of 128 channels (eight contiguous
//               1 KiB tiles of the tiled weight layout, one bulk copy each); per tile what its
//               epilogue needs: row sums, scales, the H tile and the (g B)^T tile
//   warp 1      allocates tensor memory; one lane issues the MMAs of every other pipeline stage (and the
//               correction MMAs) and commits to mbarriers
//   warp 11     one lane issues the MMAs of the stages in between
//   warps 2-5, 12-15  epilogue, two warps per tensor-memory lane quarter (32 channels), one for each
//               half of the tile's tokens: dequantise the accumulator in place (tcgen05.ld /
//               tcgen05.st), wait for the correction MMA, read the result, transpose it through shared
//               memory and store y with TMA
//   warps 6-9   expand the packed tile into tensor memory
//   warp 10     producer of the packed codes (eight contiguous 1 KiB tiles of the tiled weight layout
//               per stage, one bulk copy each), in a ring that runs ahead of the activations'
// Codes are c = t + 1 (both operands are declared signed 8-bit; 0, 1, 2 read the same either way);
// sum_k t x~ = sum_k c x~ - sum_k x~ is restored in the epilogue from the row sums.
//
// Every wait is bounded: when one gives up, the CTA records it in the device status word, all
// roles leave their loops, in-flight bulk copies are drained, tensor memory is freed and the
// kernel returns.
#include "hgf_tc.cuh"

namespace hgf {

constexpr int TILE_C = 128;   // output channels per tile (MMA M, tensor-memory lanes)
constexpr int TILE_T = 128;   // tokens per tile (MMA N, accumulator columns)
constexpr int KBLK = 256;      // input columns per pipeline stage: one column tile of the packed layout
constexpr int X_HALF_BYTES = TILE_T * 128;       // 16 KiB: 128 tokens x 128 columns, one 128-byte-swizzled operand tile
constexpr int X_TILE_BYTES = 2 * X_HALF_BYTES;   // 32 KiB per stage
constexpr int P_TILE_BYTES = TILE_C * KBLK / 4;  // 8 KiB: 8 weight tiles of 16 rows x 256 columns
constexpr int TOKV_BYTES = TILE_T * 8;           // row sums and scales of the tile's tokens
constexpr int STORE_BUF_BYTES = 2048;            // per epilogue warp: 32 channels x 32 tokens (bf16) or x 16 tokens (fp32)
constexpr int GEMM_THREADS = 512;  // 16 warps
// tensor memory: two accumulators of 128 columns, then one weight operand of 64 columns (= 256 int8 per lane) per stage
constexpr int TMEM_COLS = 512, ACC_COLS = TILE_T, A_COL = 2 * ACC_COLS, A_STAGE_COLS = KBLK / 4;

// Shared-memory map and barrier slots of a kernel variant.  NS = pipeline stages (activation tile +
// packed codes in shared memory, weight operand in tensor memory).  OPSB = bytes per row of the
// correction's two operand tiles: 128 (64 fp16, any rank), or 64 when r <= 32 - which leaves room
// for a fourth stage.
template <int NS, int OPSB>
struct Cfg {
    static constexpr int STAGES = NS;
    static constexpr int PSTAGES = NS + 1;  // the packed codes run one stage further ahead than the activations
    static constexpr int LORA_H_BYTES = TILE_T * OPSB, LORA_B_BYTES = TILE_C * OPSB;
    static constexpr int OFF_X = 0;
    static constexpr int OFF_LH = OFF_X + NS * X_TILE_BYTES;
    static constexpr int OFF_LB = OFF_LH + 2 * LORA_H_BYTES;  // the epilogue's operands are double-buffered like the accumulators
    static constexpr int OFF_P = OFF_LB + 2 * LORA_B_BYTES;
    static constexpr int OFF_TOKV = OFF_P + PSTAGES * P_TILE_BYTES;
    static constexpr int OFF_ST = OFF_TOKV + 2 * TOKV_BYTES;
    static constexpr int OFF_BAR = OFF_ST + 8 * STORE_BUF_BYTES;
    static constexpr int SMEM_BYTES = OFF_BAR + 512 + 1024;  // + slack for the 1024-byte alignment of the base
    // barrier slots (8 bytes each) inside the OFF_BAR block
    static constexpr int BAR_FULL = 0, BAR_EMPTY = BAR_FULL + NS, BAR_PFULL = BAR_EMPTY + NS, BAR_PEMPTY = BAR_PFULL + PSTAGES,
                         BAR_ACCFULL = BAR_PEMPTY + PSTAGES,
                         BAR_ACCEMPTY = BAR_ACCFULL + 2, BAR_LORAREADY = BAR_ACCEMPTY + 2, BAR_LORADONE = BAR_LORAREADY + 2,
                         BAR_OPSFULL = BAR_LORADONE + 2, BAR_OPSEMPTY = BAR_OPSFULL + 2, BAR_TURN = BAR_OPSEMPTY + 2,
                         BAR_COUNT = BAR_TURN + 2;
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
    static_assert(BAR_COUNT * 8 + 16 <= 512, "barrier block too small");
    static_assert(A_COL + NS * A_STAGE_COLS <= TMEM_COLS, "tensor memory budget");
};

// Instruction descriptor: D format (bits 4-5), A format (7-9), B format (10-12), K-major A and B,
// N >> 3 (17-22), M >> 4 (24-28).
constexpr uint32_t IDESC_I8 = (2u << 4) /*s32*/ | (1u << 7) /*A s8*/ | (1u << 10) /*B s8*/ |
                              ((uint32_t)(TILE_T >> 3) << 17) | ((uint32_t)(TILE_C >> 4) << 24);
constexpr uint32_t IDESC_F16 = (1u << 4) /*f32*/ | (0u << 7) /*A f16*/ | (0u << 10) /*B f16*/ |
                               ((uint32_t)(TILE_T >> 3) << 17) | ((uint32_t)(TILE_C >> 4) << 24);

template <bool OUT_BF16, int NS, int OPSB>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
prefill_gemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_h,
                    const __grid_constant__ CUtensorMap tmap_gb, const __grid_constant__ CUtensorMap tmap_y,
                    const GemmParams p, unsigned int *status) {
    using C = Cfg<NS, OPSB>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + C::OFF_BAR;
    auto bar = [&](int i) { return bar0 + 8u * i; };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::OFF_BAR + C::BAR_COUNT * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_BAR + C::BAR_COUNT * 8 + 4);
    static_assert(TILE_T == 128, "the epilogue's staging loops are written for 128-token tiles");

    // the next launch in the stream, if it asks for it, may be set up while this one runs (it waits
    // for this grid's completion before it touches memory)
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles_t = (p.M + TILE_T - 1) / TILE_T, tiles_c = (p.N + TILE_C - 1) / TILE_C;
    const int num_tiles = tiles_t * tiles_c;
    const int kblocks = (p.K + KBLK - 1) / KBLK;
    const bool has_lora = p.r > 0;

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            // FULL: the stage's activation tile has landed (producer's arrival + bytes) and the four unpack
            // warps have put the weight operand into tensor memory, so the MMA thread waits on this one
            // barrier only (it is a single thread and every barrier operation costs it a shared-memory
            // round trip).  EMPTY: the MMAs that read the stage are complete (one commit; the producer
            // and the unpack warps both wait on it).
            mbar_init(bar(C::BAR_FULL + s), 1 + 4);
            mbar_init(bar(C::BAR_EMPTY + s), 1);
        }
        for (int j = 0; j < C::PSTAGES; ++j) {
            // the packed codes have a ring of their own, filled ahead of the activations: the expansion into
            // tensor memory then starts the moment a stage's MMAs are complete, in parallel with the reload
            // of the activation tile, instead of after it
            mbar_init(bar(C::BAR_PFULL + j), 1);
            mbar_init(bar(C::BAR_PEMPTY + j), 4);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(C::BAR_ACCFULL + b), 2);  // one commit from each of the two MMA-issuing threads
            mbar_init(bar(C::BAR_TURN + b), 1);
            mbar_init(bar(C::BAR_ACCEMPTY + b), 8);
            mbar_init(bar(C::BAR_LORAREADY + b), 8);
            mbar_init(bar(C::BAR_LORADONE + b), 1);
            mbar_init(bar(C::BAR_OPSFULL + b), 1);
            mbar_init(bar(C::BAR_OPSEMPTY + b), 8);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        fence_proxy_async();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Everything above touches only this CTA's own shared and tensor memory; what follows reads what
    // the prologue launch wrote (a no-op unless the launch carries the programmatic-dependency attribute).
    asm volatile("griddepcontrol.wait;\n" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // The whole warp walks the loop (a single thread issuing ten copies per two k blocks, each
        // with its address arithmetic, cannot keep up with the MMAs): every lane polls the barriers,
        // lane 0 posts the byte counts and the activation tile, lanes 0-7 one weight tile each.
        {
            int s = 0;
            uint32_t ph = 0;
            uint32_t issued[C::STAGES] = {}, ops_issued[2] = {};
            int pit = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                const int t0 = (tile % tiles_t) * TILE_T, c0 = (tile / tiles_t) * TILE_C;
                {
                    // what the tile's epilogue needs, into the buffer of the tile's accumulator: row sums and
                    // scales of the 128 tokens, and with a correction the H tile and the (g B)^T tile
                    const int b = pit & 1;
                    ok = mbar_wait(bar(C::BAR_OPSEMPTY + b), ((uint32_t)(pit >> 1) & 1u) ^ 1u, abort_flag, status, 0x120u + b);
                    if (!(ok = __all_sync(0xffffffffu, ok))) break;
                    if (lane == 0) {
                        mbar_arrive_expect_tx(bar(C::BAR_OPSFULL + b), 2u * TILE_T * 4u + (has_lora ? C::LORA_H_BYTES + C::LORA_B_BYTES : 0));
                        bulk_load_1d(sbase + C::OFF_TOKV + b * TOKV_BYTES, p.row_sum + t0, TILE_T * 4u, bar(C::BAR_OPSFULL + b));
                        bulk_load_1d(sbase + C::OFF_TOKV + b * TOKV_BYTES + TILE_T * 4, p.tok_sc + t0, TILE_T * 4u, bar(C::BAR_OPSFULL + b));
                        if (has_lora) {
                            tma_load_2d(sbase + C::OFF_LH + b * C::LORA_H_BYTES, &tmap_h, 0, t0, bar(C::BAR_OPSFULL + b));
                            tma_load_2d(sbase + C::OFF_LB + b * C::LORA_B_BYTES, &tmap_gb, 0, c0, bar(C::BAR_OPSFULL + b));
                        }
                    }
                    ++ops_issued[b];
                    ++pit;
                }
                for (int kb = 0; kb < kblocks; ++kb) {
                    ok = mbar_wait(bar(C::BAR_EMPTY + s), ph ^ 1u, abort_flag, status, 0x100u + s);
                    if (!(ok = __all_sync(0xffffffffu, ok))) break;
                    if (lane == 0) {
                        // 256 columns of 128 tokens as two 128-byte-swizzled tiles (columns past K read as zeros)
                        mbar_arrive_expect_tx(bar(C::BAR_FULL + s), X_TILE_BYTES);
                        tma_load_2d(sbase + C::OFF_X + s * X_TILE_BYTES, &tmap_x, kb * KBLK, t0, bar(C::BAR_FULL + s));
                        tma_load_2d(sbase + C::OFF_X + s * X_TILE_BYTES + X_HALF_BYTES, &tmap_x, kb * KBLK + 128, t0, bar(C::BAR_FULL + s));
                    }
                    ++issued[s];
                    if (++s == C::STAGES) { s = 0; ph ^= 1u; }
                }
            }
            // drain: wait (bounded) until every copy this warp issued has landed, so that the CTA
            // never exits with a bulk copy in flight (immediate when the consumers ran to the end)
            for (int q = 0; q < C::STAGES; ++q)
                if (issued[q]) {
                    const uint32_t par = (issued[q] - 1u) & 1u;
                    for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar(C::BAR_FULL + q), par); ++i) {}
                }
            for (int q = 0; q < 2; ++q)
                if (ops_issued[q]) {
                    const uint32_t par = (ops_issued[q] - 1u) & 1u;
                    for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar(C::BAR_OPSFULL + q), par); ++i) {}
                }
        }
    } else if (warp == 1 || warp == 11) {
        // ------------------------------------------------------------------ MMA issuers
        // Tile `it` accumulates into accumulator it % 2, so the epilogue of one tile runs under the main
        // loop of the next.  With a correction, the epilogue first rewrites the accumulator as fp32
        // (dequantised), then the first issuer adds (g B) H^T onto it with one more MMA, slipped in between
        // the k blocks of the tile in progress as soon as the epilogue is ready for it.
        //
        // TWO threads issue the integer MMAs, in turns: the stages are numbered through the whole tile
        // sequence and warp 1 takes the even ones, warp 11 the odd ones.  The tensor pipe holds hardly any
        // MMA in reserve and takes a 128 x 128 x 32 one about as fast as it executes it (64 clocks), so with
        // a single issuing thread it idles while that thread waits on barriers, commits and keeps its
        // books - about as long per stage as the stage's eight MMAs run.  Here one thread does all that
        // for its next stage while the other's MMAs run, and only the hand-over itself is exposed.  Order
        // between the two threads' MMAs on the shared accumulator is established the documented way: after
        // its stage a thread executes tcgen05.fence::before_thread_sync and arrives on the other's TURN
        // barrier; the other waits there and executes tcgen05.fence::after_thread_sync before its first MMA.
        // Each thread commits the stages it issued (EMPTY) and, at the end of a tile, ACCFULL (two arrivals).
        const int half = warp == 1 ? 0 : 1;
        if (lane == 0) {
            bool ok = true;
            int it = 0, pend = -1;  // pend: tile whose correction MMA is still to be issued (first issuer only)
            int gs = 0;             // stage number, counted through all tiles of this CTA
            const uint64_t xdesc0 = make_sw128_desc(sbase + C::OFF_X);
            auto issue_lora = [&](int t) {
                const int b = t & 1;
                tc_fence_after();
                const uint32_t la = sbase + C::OFF_LB + b * C::LORA_B_BYTES, lh = sbase + C::OFF_LH + b * C::LORA_H_BYTES;
                const uint64_t adesc = OPSB == 128 ? make_sw128_desc(la) : make_sw64_desc(la);
                const uint64_t bdesc = OPSB == 128 ? make_sw128_desc(lh) : make_sw64_desc(lh);
#pragma unroll
                for (int kk = 0; kk < OPSB / 32; ++kk)  // K = 16 fp16 (32 bytes of a row) per MMA, on top of the fp32 values
                    mma_f16(tmem_base + b * ACC_COLS, adesc + 2u * kk, bdesc + 2u * kk, IDESC_F16, 1u);
                tc_commit(bar(C::BAR_LORADONE + b));
            };
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++it) {
                const int b = it & 1;
                const uint32_t acc = tmem_base + b * ACC_COLS;
                bool acc_mine = false;  // this thread has waited for the accumulator's release
                for (int kb = 0; kb < kblocks; ++kb, ++gs) {
                    if ((gs & 1) != half) continue;
                    if (!acc_mine) {
                        if (it >= 2 && !(ok = mbar_wait(bar(C::BAR_ACCEMPTY + b), (uint32_t)((it >> 1) - 1) & 1u, abort_flag, status, 0x200u)))
                            break;
                        acc_mine = true;
                    }
                    if (half == 0 && pend >= 0 && mbar_try_wait(bar(C::BAR_LORAREADY + (pend & 1)), (uint32_t)(pend >> 1) & 1u)) {
                        issue_lora(pend);
                        pend = -1;
                    }
                    const int s = gs % C::STAGES;
                    const uint32_t ph = (uint32_t)(gs / C::STAGES) & 1u;
                    if (!(ok = mbar_wait(bar(C::BAR_FULL + s), ph, abort_flag, status, 0x210u + s))) break;
                    // the other thread has issued stage gs - 1
                    if (gs > 0 && !(ok = mbar_wait_spin(bar(C::BAR_TURN + half), (uint32_t)((gs - 1) >> 1) & 1u, abort_flag, status, 0x240u + half)))
                        break;
                    tc_fence_after();
                    const uint64_t bdesc = xdesc0 + (uint64_t)(s * (X_TILE_BYTES >> 4));
                    const uint32_t a_tmem = tmem_base + A_COL + s * A_STAGE_COLS;
                    // per MMA 32 int8: 8 columns of the weight operand, 32 bytes of a token row; the stage's
                    // second 128 columns sit in the second swizzled tile
                    mma_i8_ts(acc, a_tmem, bdesc, IDESC_I8, kb ? 1u : 0u);
                    mma_i8_ts(acc, a_tmem + 8u, bdesc + 2u, IDESC_I8, 1u);
                    mma_i8_ts(acc, a_tmem + 16u, bdesc + 4u, IDESC_I8, 1u);
                    mma_i8_ts(acc, a_tmem + 24u, bdesc + 6u, IDESC_I8, 1u);
                    mma_i8_ts(acc, a_tmem + 32u, bdesc + (X_HALF_BYTES >> 4), IDESC_I8, 1u);
                    mma_i8_ts(acc, a_tmem + 40u, bdesc + (X_HALF_BYTES >> 4) + 2u, IDESC_I8, 1u);
                    mma_i8_ts(acc, a_tmem + 48u, bdesc + (X_HALF_BYTES >> 4) + 4u, IDESC_I8, 1u);
                    mma_i8_ts(acc, a_tmem + 56u, bdesc + (X_HALF_BYTES >> 4) + 6u, IDESC_I8, 1u);
                    tc_fence_before();
                    mbar_arrive(bar(C::BAR_TURN + (half ^ 1)));  // the other thread's turn
                    tc_commit(bar(C::BAR_EMPTY + s));
                }
                if (!ok) break;
                tc_commit(bar(C::BAR_ACCFULL + b));
                if (half != 0) continue;
                if (pend >= 0) {  // the previous tile's correction has to be out before its accumulator's next turn
                    if (!(ok = mbar_wait(bar(C::BAR_LORAREADY + (pend & 1)), (uint32_t)(pend >> 1) & 1u, abort_flag, status, 0x230u)))
                        break;
                    issue_lora(pend);
                    pend = -1;
                }
                if (has_lora) pend = it;
            }
            if (half == 0 && ok && pend >= 0 &&
                mbar_wait(bar(C::BAR_LORAREADY + (pend & 1)), (uint32_t)(pend >> 1) & 1u, abort_flag, status, 0x231u))
                issue_lora(pend);
        }
    } else if (warp < 6 || warp >= 12) {
        // ------------------------------------------------------------------ epilogue warps
        // Eight of them: the warp pair of a tensor-memory lane quarter (32 output channels) shares the
        // tile's 128 tokens, 64 each, so a tile's epilogue takes half as long as with one warp per
        // quarter - with the two issuing threads the main loop of a short-K tile is over sooner than that.
        const int e2 = warp < 6 ? 0 : 1;                  // which 64 tokens of the tile
        const int q = warp & 3;                           // tensor-memory lane quarter this warp may access
        constexpr int HALF_T = TILE_T / 2;
        constexpr int W = OUT_BF16 ? 32 : 16;             // tokens per staging step (2 KiB of staging either way)
        uint8_t *buf = smem + C::OFF_ST + (4 * e2 + q) * STORE_BUF_BYTES;
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++it) {
            const int t0 = (tile % tiles_t) * TILE_T, c0 = (tile / tiles_t) * TILE_C;
            const int b = it & 1;
            const uint32_t par = (uint32_t)(it >> 1) & 1u;
            // the tile's row sums and scales (and the correction's operands) were fetched by the producer
            const int *tok_rs = reinterpret_cast<const int *>(smem + C::OFF_TOKV + b * TOKV_BYTES);
            const float *tok_sc = reinterpret_cast<const float *>(tok_rs + TILE_T);
            ok = mbar_wait(bar(C::BAR_OPSFULL + b), par, abort_flag, status, 0x320u + b);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;

            const int n = c0 + 32 * q + lane;  // this thread's output channel = its tensor-memory lane
            const bool n_ok = n < p.N;

            ok = mbar_wait(bar(C::BAR_ACCFULL + b), par, abort_flag, status, 0x300u);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;  // the whole warp leaves together
            tc_fence_after();
            const uint32_t lane_base = tmem_base + ((uint32_t)(32 * q) << 16) + b * ACC_COLS;

            // int32 sums -> fp32 (Y_int - row sum) * scale, for the WN tokens from cc on
            // (the per-token values are read as vectors ahead of the arithmetic: a shared-memory load per
            // element in the dependent chain costs its full latency every time)
            auto dequant_chunk = [&](int cc, auto &ai) {
                constexpr int WN = (int)(sizeof(ai) / sizeof(uint32_t));
                if (p.dbg_y_int && n_ok) {
#pragma unroll
                    for (int j = 0; j < WN; ++j)
                        if (t0 + cc + j < p.M) p.dbg_y_int[(size_t)(t0 + cc + j) * p.N + n] = (int)ai[j] - tok_rs[cc + j];
                }
#pragma unroll
                for (int v = 0; v < WN / 4; ++v) {
                    const int4 rs4 = *reinterpret_cast<const int4 *>(tok_rs + cc + 4 * v);
                    const float4 sc4 = *reinterpret_cast<const float4 *>(tok_sc + cc + 4 * v);
                    ai[4 * v + 0] = __float_as_uint((float)((int)ai[4 * v + 0] - rs4.x) * sc4.x);
                    ai[4 * v + 1] = __float_as_uint((float)((int)ai[4 * v + 1] - rs4.y) * sc4.y);
                    ai[4 * v + 2] = __float_as_uint((float)((int)ai[4 * v + 2] - rs4.z) * sc4.z);
                    ai[4 * v + 3] = __float_as_uint((float)((int)ai[4 * v + 3] - rs4.w) * sc4.w);
                }
            };
            if (has_lora) {
                // first pass: dequantise in place (int32 -> fp32), then let the MMA warp add the correction
                for (int cc = HALF_T * e2; cc < HALF_T * (e2 + 1); cc += 32) {
                    uint32_t ai[32];
                    tmem_ld32(lane_base + cc, ai);
                    tmem_ld_wait();
                    dequant_chunk(cc, ai);
                    tmem_st32(lane_base + cc, ai);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(C::BAR_LORAREADY + b));
                ok = mbar_wait(bar(C::BAR_LORADONE + b), par, abort_flag, status, 0x310u);
                if (!(ok = __all_sync(0xffffffffu, ok))) break;
                tc_fence_after();
            }

            // read the result, transpose it through shared memory (a thread holds one channel of W
            // tokens; y wants the channels of a token next to each other) and store with TMA
            for (int cc = HALF_T * e2; cc < HALF_T * (e2 + 1); cc += W) {
                uint32_t ai[W];
                if constexpr (W == 32) tmem_ld32(lane_base + cc, ai); else tmem_ld16(lane_base + cc, ai);
                tmem_ld_wait();
                if (!has_lora) dequant_chunk(cc, ai);
                // the buffer was handed to a TMA store one chunk ago: wait until it was read
                if (lane == 0) bulk_wait_read<0>();
                __syncwarp();
                if (OUT_BF16) {
#pragma unroll
                    for (int j = 0; j < W; ++j)
                        reinterpret_cast<__nv_bfloat16 *>(buf)[j * 32 + lane] = __float2bfloat16_rn(__uint_as_float(ai[j]));
                } else {
#pragma unroll
                    for (int j = 0; j < W; ++j) reinterpret_cast<uint32_t *>(buf)[j * 32 + lane] = ai[j];
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&tmap_y, c0 + 32 * q, t0 + cc, smem_u32(buf));
                    bulk_commit();
                }
            }
            // all tensor-memory reads of this tile are done: hand the accumulator back to the MMA warps
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar(C::BAR_ACCEMPTY + b));
                mbar_arrive(bar(C::BAR_OPSEMPTY + b));
            }
        }
        if (lane == 0) bulk_wait_read<0>();
        __syncwarp();
    } else if (warp == 10) {
        // ------------------------------------------------------------------ packed-code producer
        // Its own warp and ring: the codes run ahead of the activations, so the expansion into tensor
        // memory starts the moment a stage's MMAs are complete, in parallel with the reload of the
        // activation tile.  Per stage the 1 KiB tiles (16 rows x 256 columns) of 8 consecutive row tiles,
        // one bulk copy per lane (row tiles past the matrix are left out).
        int pj = 0;
        uint32_t pph = 0;
        uint32_t pissued[C::PSTAGES] = {};
        bool ok = true;
        const int steps = (p.K + 255) >> 8, n_row_tiles = (p.N + 15) >> 4;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
            const int rt0 = ((tile / tiles_t) * TILE_C) >> 4;
            const int nrt = n_row_tiles - rt0 < TILE_C / 16 ? n_row_tiles - rt0 : TILE_C / 16;
            const uint8_t *psrc = p.packed + (size_t)(rt0 + (lane < nrt ? lane : 0)) * steps * 1024;
            for (int kb = 0; kb < kblocks; ++kb) {
                ok = mbar_wait(bar(C::BAR_PEMPTY + pj), pph ^ 1u, abort_flag, status, 0x110u + pj);
                if (!(ok = __all_sync(0xffffffffu, ok))) break;
                if (lane == 0) mbar_arrive_expect_tx(bar(C::BAR_PFULL + pj), (uint32_t)nrt * 1024u);
                __syncwarp();
                if (lane < nrt)
                    bulk_load_1d(sbase + C::OFF_P + pj * P_TILE_BYTES + lane * 1024, psrc + (size_t)kb * 1024, 1024u, bar(C::BAR_PFULL + pj));
                ++pissued[pj];
                if (++pj == C::PSTAGES) { pj = 0; pph ^= 1u; }
            }
        }
        for (int q = 0; q < C::PSTAGES; ++q)
            if (pissued[q]) {
                const uint32_t par = (pissued[q] - 1u) & 1u;
                for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(bar(C::BAR_PFULL + q), par); ++i) {}
            }
    } else {
        // ------------------------------------------------------------------ unpack warps
        const int q = warp & 3;              // tensor-memory lane quarter this warp may access
        const int row = 32 * q + lane;       // this thread's channel row of the tile = its tensor-memory lane
        int s = 0, pj = 0;
        uint32_t ph = 0, pph = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
            for (int kb = 0; kb < kblocks; ++kb) {
                // the stage's packed codes have landed, and the MMAs that read this stage's previous operand
                // are complete
                ok = mbar_wait(bar(C::BAR_PFULL + pj), pph, abort_flag, status, 0x400u + pj) &&
                     mbar_wait(bar(C::BAR_EMPTY + s), ph ^ 1u, abort_flag, status, 0x410u + s);
                if (!(ok = __all_sync(0xffffffffu, ok))) break;  // the whole warp leaves together
                // this row's 64 bytes hold the stage's 256 columns; register 4 i + j of a half = columns
                // 16 i + 4 j .. + 3, one code per byte
                const uint8_t *prow = smem + C::OFF_P + pj * P_TILE_BYTES + row * 64;
                const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + A_COL + s * A_STAGE_COLS;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const uint4 lo = *reinterpret_cast<const uint4 *>(prow + 32 * half);
                    const uint4 hi = *reinterpret_cast<const uint4 *>(prow + 32 * half + 16);
                    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
                    uint32_t a[32];
#pragma unroll
                    for (int i = 0; i < 8; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) a[4 * i + j] = (w[i] >> (2 * j)) & 0x03030303u;
                    tmem_st32(taddr + 32 * half, a);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar(C::BAR_FULL + s));
                    mbar_arrive(bar(C::BAR_PEMPTY + pj));
                }
                if (++pj == C::PSTAGES) { pj = 0; pph ^= 1u; }
                if (++s == C::STAGES) { s = 0; ph ^= 1u; }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// The bounded wait on a barrier that nothing completes: it gives up after `limit_ns`, records that
// in the status word and the kernel returns (the error path of every role above, exercised alone).
__global__ void wait_timeout_selftest_kernel(unsigned long long limit_ns, unsigned int *status) {
    __shared__ __align__(8) unsigned long long bar_mem;
    __shared__ int abort_mem;
    const uint32_t bar = smem_u32(&bar_mem);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        abort_mem = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait(bar, 0u, &abort_mem, status, 0x700u, limit_ns);
}

cudaError_t launch_wait_timeout_selftest(unsigned long long limit_ns, cudaStream_t stream) {
    unsigned int *status = device_status_word();
    if (!status) return cudaErrorMemoryAllocation;
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(limit_ns, status);
    count_launch();
    return cudaGetLastError();
}

// ---- host side: tensor maps and launch -----------------------------------------------------------
template <bool OUT_BF16, int NS, int OPSB>
static cudaError_t launch_variant(const CUtensorMap &mx, const CUtensorMap &mh, const CUtensorMap &mgb, const CUtensorMap &my,
                                  const GemmParams &p, int grid, unsigned int *status, cudaStream_t stream) {
    static std::atomic<unsigned long long> attr_done{0};
    constexpr int smem = Cfg<NS, OPSB>::SMEM_BYTES;
    {
        cudaError_t e = ensure_dynamic_smem(prefill_gemm_kernel<OUT_BF16, NS, OPSB>, smem, attr_done);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (p.flags & HGF_FLAG_NO_PDL) ? 0 : 1;  // set-up (barriers, tensor memory) may overlap the prologue's tail
    cudaError_t e = cudaLaunchKernelEx(&cfg, prefill_gemm_kernel<OUT_BF16, NS, OPSB>, mx, mh, mgb, my, p, status);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_prefill_gemm(const GemmParams &p, cudaStream_t stream) {
    const int sm_count = device_sm_count();
    if (!sm_count) return cudaErrorInvalidDevice;
    const bool bf16 = (p.flags & HGF_FLAG_OUT_BF16) != 0;
    const bool narrow = p.r <= 32;  // 64-byte operand rows for the correction, and room for a fourth stage
    CUtensorMap mx, mh, mgb, my;
    if (!make_map_2d(&mx, CU_TENSOR_MAP_DATA_TYPE_UINT8, p.xq, (uint64_t)p.K, (uint64_t)p.M, (uint64_t)p.K, 128, TILE_T,
                     CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;
    if (p.r > 0) {  // H [M][64] and (g B)^T [N][64] fp16: tiles of 128 rows; the first 32 or all 64 columns
        const uint32_t cols = narrow ? 32 : 64;
        const CUtensorMapSwizzle sw = narrow ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
        if (!make_map_2d(&mh, CU_TENSOR_MAP_DATA_TYPE_UINT16, p.h16, 64, (uint64_t)p.M, 128, cols, TILE_T, sw)) return cudaErrorInvalidValue;
        if (!make_map_2d(&mgb, CU_TENSOR_MAP_DATA_TYPE_UINT16, p.gb16, 64, (uint64_t)p.N, 128, cols, TILE_C, sw)) return cudaErrorInvalidValue;
    } else {
        mh = mx;
        mgb = mx;
    }
    if (!make_map_2d(&my, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, p.y, (uint64_t)p.N,
                     (uint64_t)p.M, (uint64_t)p.N * (bf16 ? 2 : 4), 32, bf16 ? 32 : 16, CU_TENSOR_MAP_SWIZZLE_NONE))
        return cudaErrorInvalidValue;
    const int tiles = ((p.M + TILE_T - 1) / TILE_T) * ((p.N + TILE_C - 1) / TILE_C);
    const int grid = tiles < sm_count ? tiles : sm_count;
    unsigned int *status = device_status_word();
    if (!status) return cudaErrorMemoryAllocation;
    cudaError_t e;
    if (narrow)
        e = bf16 ? launch_variant<true, 4, 64>(mx, mh, mgb, my, p, grid, status, stream)
                 : launch_variant<false, 4, 64>(mx, mh, mgb, my, p, grid, status, stream);
    else
        e = bf16 ? launch_variant<true, 3, 128>(mx, mh, mgb, my, p, grid, status, stream)
                 : launch_variant<false, 3, 128>(mx, mh, mgb, my, p, grid, status, stream);
    count_launch();
    return e;
}

}  // namespace hgf
